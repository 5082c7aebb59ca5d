/*
 * ats.h — C ABI of the tensor-granularity hybrid-placement forward library (B200, sm_100a).
 *
 * The library executes the per-tensor forward of 4-bit block-quantized transformer weights under
 * a per-tensor placement: every weight tensor is one operator (paper Section 3 and 4.3.1: the unit
 * that is placed and scheduled is a tensor with a size s_i and a value r_i); a GPU memory budget M
 * and a placement b decide which tensors stay resident in GPU memory (Section 4.3.2, Algorithm 1);
 * the others live in pinned host memory and are copied into temporary GPU buffers by a transfer
 * stream while a compute stream runs the operators, ordered by events (Section 4.2.1, 4.2.2).
 * For MoE operators only the experts the current tokens selected are moved (Section 4.2.2, 4.4.1).
 *
 * Conventions
 *  - Every function returns an int32 status: ATS_OK (0) or a negative ATS_ERR_* code; the text of the
 *    last error of a context is available from ats_last_error().  Nothing throws or aborts.
 *  - Pointers are marked HOST or DEVICE.  Device pointers must belong to the context's device.
 *  - Compute calls are asynchronous: they validate their arguments, enqueue work on the context's
 *    compute / transfer streams and return.  Invalid arguments are rejected before anything is
 *    enqueued.  An asynchronous CUDA error surfaces at a later call or at ats_sync() as ATS_ERR_CUDA.
 *  - One host thread per context.  The caller owns every buffer it passes; the library owns the
 *    pinned host store and lays the resident region / staging ring / workspace out inside the
 *    caller's arena.
 *  - Quantization format ATS_FMT_Q4B32 (the workload's "INT4"; the paper only names the bit width,
 *    Section 5.1): signed 4-bit codes in [-8,7], blocks of 32 consecutive k of one output row, one
 *    fp16 scale per block, w[n][k] = scale[n][k/32] * code[n][k].
 *    Interchange layout at this ABI: codes row-major [E][N][K/2] bytes, byte j of a row holds code 2j
 *    in bits 0..3 and code 2j+1 in bits 4..7 as two's-complement nibbles; scales row-major fp16
 *    [E][N][K/32].  E = n_experts (1 for a dense tensor).  The library repacks internally.
 */
#ifndef ATS_H_
#define ATS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ats_ctx ats_ctx;

enum {
  ATS_OK = 0,
  ATS_ERR_INVALID = -1,     /* bad argument / unknown id / non-finite scale */
  ATS_ERR_SHAPE = -2,       /* shape rule violated (k_in % 32 != 0, mismatching layer shapes, ...) */
  ATS_ERR_NOMEM = -3,       /* host allocation failed, or workspace too small */
  ATS_ERR_BUDGET = -4,      /* GPU-placed entries do not fit the arena, or a slice does not fit a ring slot */
  ATS_ERR_STATE = -5,       /* call not legal in the current state (e.g. compute before placement) */
  ATS_ERR_CUDA = -6,        /* a CUDA call failed; the context is poisoned */
  ATS_ERR_TIMEOUT = -7,     /* ats_sync() gave up waiting */
  ATS_ERR_UNSUPPORTED = -8  /* legal but not implemented configuration */
};

enum { ATS_HOST = 0, ATS_GPU = 1 };             /* placement b_i (Section 4.3.2) */
enum { ATS_FMT_Q4B32 = 0, ATS_FMT_F16 = 1, ATS_FMT_W16 = 2, ATS_FMT_MXFP4 = 3 };
/* F16: small auxiliary tensors (router weight [k_in][n_out], norm gain [n_out]): always resident, no placement.
 * W16: an unquantized fp16 weight matrix [n_out][k_in] (the paper runs one of its models with FP16 weights, Section 5.1):
 * a dense tensor (n_experts = 1, k_in a multiple of 8) placed and streamed like a Q4B32 tensor (2 bytes per weight);
 * ats_linear and ats_lm_head take it, and so do ats_layer_decode / ats_layer_decode_host / ats_layer_prefill for a dense
 * layer whose seven matrices are all W16 (mixed formats within a layer: ATS_ERR_INVALID; MoE layers: Q4B32 experts only;
 * fp32 accumulation, the same roundings between operators as the quantized layer; the norm runs as a launch of its
 * own and fused groups (QKV, gate|up) become one GEMV launch or one GEMM per matrix).  ats_moe_linear, ats_embed and
 * ats_dequantize take 4-bit tensors only.
 * MXFP4: the microscaling 4-bit format, the other 4-bit format the paper evaluates (Section 5.1).  Interchange layout:
 * codes uint8 [E][n_out][k_in/2], byte j of a row = element 2j in bits 0..3 and element 2j+1 in bits 4..7, each element a
 * 4-bit float (sign, 2 exponent bits with bias 1, 1 mantissa bit, exponent 0 subnormal: 0, 0.5, 1, 1.5, 2, 3, 4, 6 and
 * their negatives); scales uint8 [E][n_out][k_in/32], one biased exponent per block of 32: 2^(byte - 127).  Byte 255
 * (not a number): ATS_ERR_INVALID; exponents outside -23 .. 13 (bytes 104 .. 140): ATS_ERR_UNSUPPORTED, because every
 * weight must be an fp16 value (it is the tensor-core operand).  Inside the library the tensor has the slice layout and
 * size of a Q4B32 tensor (the scale kept as an fp16 power of two) and takes every call a Q4B32 tensor takes, dense or
 * stacked; weights are exact in both the GEMV and the GEMM.  The single-token streaming kernels have a mode for this
 * format (twice an element is an integer, looked up per nibble and fed to the same integer dot products). */
enum { ATS_OUT_F32 = 0, ATS_OUT_F16 = 1 };      /* ats_dequantize output */
enum { ATS_MODE_DECODE = 0, ATS_MODE_PREFILL = 1 };

/* ats_config.flags */
enum {
  ATS_FLAG_POISON_SLOTS = 1u,     /* debug: fill a ring slot with 0xFF after its consumer, so premature reuse shows */
  ATS_FLAG_SKIP_SCALE_CHECK = 2u, /* do not scan scales for Inf/NaN at registration */
  ATS_FLAG_TIME_KERNELS = 4u,     /* bracket every GEMV / grouped GEMV / GEMM launch with CUDA events (see ats_stats.timed_*) */
  ATS_FLAG_NO_PDL = 8u,           /* launch every kernel fully serialized (no programmatic dependent launch overlap) */
  ATS_FLAG_NO_GEMM_PAIR = 32u,    /* do not run large GEMMs as pairs of CTAs on two SMs (tcgen05 cta_group::2): the single-CTA kernel only */
  ATS_FLAG_MOE_RING_ONLY = 16u,   /* Decode-step MoE stages with host-placed experts always take the staging ring (ids to
                                     the host, one cudaMemcpyAsync per chunk of every selected host-placed slice on the
                                     transfer stream, counted in ats_stats.streamed_bytes / copies / host_syncs).
                                     Without this flag the library uses the zero-copy path of Sections 4.1 / 4.2.1 where it
                                     can (the pinned host store is mapped into the device's address space and every stacked
                                     tensor has a device table of slice addresses, resident copy or place in the store):
                                     one token: the grouped-expert kernels pick each selected slice's address by the expert
                                     id on the device and stream a host-placed slice over PCIe straight into their
                                     shared-memory ring: no ids on the host, no staging slot, no event (these reads are not
                                     counted in streamed_bytes / copies / host_syncs); several tokens: the ids go to the
                                     host, and the distinct selected host-placed experts are gathered into the part of the
                                     workspace beyond the call's own buffers by one launch of an SM-driven copy kernel (each
                                     slice crosses PCIe once; counted in streamed_bytes, not in copies) when that part holds
                                     them; otherwise the ring.  Same arithmetic and the same results on every path. */
};
/* ats_layer_desc.flags */
enum { ATS_LAYER_NO_TOPK_RENORM = 1u /* gates = full softmax entries instead of softmax over the top-k */ };

typedef struct {
  void* arena;             /* DEVICE, 256-byte aligned; workspace, staging ring and resident region are carved from it */
  uint64_t arena_bytes;
  void* compute_stream;    /* cudaStream_t on which operators run (0 = legacy default stream) */
  void* transfer_stream;   /* cudaStream_t for host->device weight copies; must differ from compute_stream */
  uint32_t ring_slots;     /* number of equal staging slots (temporary GPU buffers, Section 4.2.1); 0 = no streaming */
  uint64_t slot_bytes;     /* bytes of one slot; every streamed tensor / expert slice must fit one slot */
  uint64_t chunk_bytes;    /* a streamed slice is copied as ceil(bytes/chunk_bytes) cudaMemcpyAsync calls */
  uint64_t workspace_bytes;/* activation scratch (>= 1024; for ats_layer_* pass ats_workspace_bytes()) */
  int32_t device;          /* CUDA device ordinal of the arena and streams */
  uint32_t flags;
} ats_config;

/* Create a context.  cfg is copied.  ATS_ERR_INVALID for null/misaligned arena, equal streams, an arena
 * smaller than workspace + ring.  The arena and streams stay owned by the caller and must outlive the context. */
int32_t ats_init(const ats_config* cfg /*HOST*/, ats_ctx** out /*HOST*/);
/* Synchronises both streams, frees the pinned store and every event.  The arena is not touched. */
int32_t ats_destroy(ats_ctx* ctx);
/* Text of the last error recorded on ctx (valid until the next failing call); "" if none. */
const char* ats_last_error(const ats_ctx* ctx);

/* A tensor record (Section 4.3.2: size s_i, value r_i, switching cost c_i). */
typedef struct {
  uint32_t fmt;        /* ATS_FMT_* */
  uint32_t n_experts;  /* 1 = dense tensor; > 1 = stacked expert tensor [E][n_out][k_in] */
  uint32_t n_out;      /* output features N */
  uint32_t k_in;       /* input features K (Q4B32, MXFP4: multiple of 32) */
  uint32_t layer;      /* informational */
  uint32_t role;       /* informational */
  int64_t value;       /* r_i, the benefit of residency; < 0 selects the default r_i = byte size */
  int64_t switch_cost; /* c_i >= 0, charged when tensor i and its predecessor get different backends */
} ats_tensor_desc;

/* Register a tensor.  codes/scales are HOST pointers in the interchange layout; they are repacked into the
 * library's pinned store before return and may be freed afterwards.  ATS_FMT_F16 tensors pass their fp16 data as
 * `codes` (scales = NULL); they are small, always GPU-resident and take no part in placement.
 * Tensors must be registered in execution order (that order is the sequence Algorithm 1 runs over).
 * Registration after ats_set_placement/ats_plan_placement invalidates the placement (state: unplaced).
 * Errors: ATS_ERR_SHAPE (k_in % 32, zero dims), ATS_ERR_INVALID (non-finite scale, null), ATS_ERR_NOMEM. */
int32_t ats_register_tensor(ats_ctx* ctx, const ats_tensor_desc* desc /*HOST*/, const void* codes /*HOST*/,
                            const void* scales /*HOST*/, int32_t* out_id /*HOST*/);

/* Bytes one (tensor, expert) slice occupies in the library's format: N*K/2 code bytes + N*(K/32) fp16 scales. */
int32_t ats_tensor_slice_bytes(const ats_ctx* ctx, int32_t id, uint64_t* out_bytes /*HOST*/);

/* Explicit placement (the decision vector b of Section 4.3.2).  Entry i places tensor ids[i], expert slice
 * experts[i] (-1 = the whole tensor, all slices) on where[i] (ATS_HOST / ATS_GPU).  Entries not named are ATS_HOST.
 * Rebuilds the resident region (copies GPU-placed slices into the arena, synchronously).
 * ATS_ERR_BUDGET if the GPU entries do not fit arena - workspace - ring, or a HOST slice exceeds slot_bytes
 * (or ring_slots == 0 while something is placed on the host). */
int32_t ats_set_placement(ats_ctx* ctx, const int32_t* ids /*HOST*/, const int32_t* experts /*HOST*/,
                          const uint8_t* where /*HOST*/, uint32_t n);

/* Algorithm 1 (static tensor placement): knapsack DP over the registered weight tensors (Q4B32 and W16) in registration order with
 * sizes s_i = ceil(bytes/granule), budget M = floor(budget_bytes/granule), values r_i and switch costs c_i;
 * for a model with expert tensors the expert / non-expert partition rule of Algorithm 1 applies (a stacked expert
 * tensor is one item).  granule_bytes = 0 selects 1 MiB (the paper quantizes at MB granularity).
 * Applies the result like ats_set_placement and writes one ATS_HOST/ATS_GPU byte per weight tensor (registration
 * order) to out_where[0..n) if non-null; n must then equal the number of weight tensors. */
int32_t ats_plan_placement(ats_ctx* ctx, uint64_t budget_bytes, uint32_t granule_bytes, uint8_t* out_where /*HOST*/,
                           uint32_t n);
int32_t ats_get_placement(const ats_ctx* ctx, int32_t id, int32_t expert, uint8_t* out_where /*HOST*/);

/* The per-tensor operator: y[m][n] = sum_k w[n][k] x[m][k], fp32 accumulation, fp16 output.
 * x DEVICE fp16 row-major [M][k_in]; y DEVICE fp16 row-major [M][n_out].  M <= 8 runs the memory-bound GEMV with exact
 * weights (scale * code in fp32): one or two rows on the streaming kernel (integer dot products on the CUDA cores), three
 * to eight rows on mma.sync tensor-core instructions, odd shapes on a generic kernel; M > 8 runs the tensor-core GEMM
 * (weights rounded once to fp16 operands).
 * Activations inside the single-row streaming kernel (also used by ats_layer_decode, ats_lm_head and the single-token MoE
 * stages): every block of 32 fp16 activations is re-expressed as 16-bit block fixed point, xi = rn(x * 2^sh) with
 * |xi| <= 32752, i.e. each element is rounded within 2^-17 of its block's largest magnitude (fp16 itself resolves that
 * maximum to 2^-11); block dot products are then exact integers and blocks are summed in fp32.  The perturbation of an
 * output is bounded by 2^-17 * sum over blocks of (block maximum * sum of |w| in the block), about 1e-5 of its scale for
 * the workloads here.  A block that holds an Inf or a NaN activation contributes NaN (as the plain definition would give
 * Inf or NaN), so a non-finite input never turns into a finite output.
 * If the tensor is placed on the host it is streamed through the ring for this call. */
int32_t ats_linear(ats_ctx* ctx, int32_t id, const void* x /*DEVICE*/, void* y /*DEVICE*/, uint32_t M);

/* Empirical performance density (Section 4.3.1: k_i = t_i / s_i from measured operator times).  Times ats_linear on dense
 * weight tensor `id` over M rows (x, y DEVICE scratch as ats_linear takes them), `iters` back-to-back calls after a warm-up,
 * with CUDA events on the compute stream: once with the tensor resident (*t_resident_us, the paper's t^g) and once with it
 * placed on the host and streamed through the ring (*t_host_us: the steady-state cost of leaving it off the GPU; this
 * library has no CPU executor, so that is what stands where the paper has t^c).  The caller forms k = t / bytes and the
 * residency benefit r_i = t_host - t_resident and hands it to Algorithm 1 through ats_set_tensor_value.
 * The call replaces the placement while it measures (this tensor alone on the GPU / on the host, everything else on the
 * host) and puts the previous one back before it returns; it synchronises, and its launches and copies count in the
 * statistics like any other call's.  ATS_ERR_BUDGET if the tensor fits neither the
 * resident region nor a ring slot.  Stacked expert tensors: ATS_ERR_INVALID (profile the operator through ats_moe_linear).
 * ats_set_tensor_value: replaces r_i (value < 0: the default, the tensor's byte size) and c_i of a registered weight tensor;
 * the placement in force stays until the next ats_plan_placement. */
int32_t ats_profile_tensor(ats_ctx* ctx, int32_t id, const void* x /*DEVICE*/, void* y /*DEVICE*/, uint32_t M, uint32_t iters,
                           double* t_resident_us /*HOST*/, double* t_host_us /*HOST*/);
int32_t ats_set_tensor_value(ats_ctx* ctx, int32_t id, int64_t value, int64_t switch_cost);

/* ats_linear for callers that must not allocate.  (The paper has no counterpart; this is a packaging variant.)
 * Some hosts of this library cannot hand it device memory beyond their tensors: code running inside a captured or
 * replayed region, plug-ins of an inference server whose memory pool is frozen after start-up, or a process that
 * has given all device memory to another allocator.  ats_linear needs scratch for its split-K partial sums when
 * M > 8 and takes it from the workspace the caller allocated; this entry point takes it instead from a fixed array of
 * ATS_STATIC_SCRATCH_BYTES that is part of the library's device image, so that it calls no cudaMalloc / cudaFree /
 * allocating routine of any library.  Same arguments as ats_linear and the same kernels, so the same result (bit for bit
 * whenever both pick the same split-K plan, which holds unless the 8 MiB here admit a plan ats_linear's workspace did
 * not: k_in >= 8192 with M >= 1024; within the tolerance of the operator otherwise), with these differences:
 *  - dense ATS_FMT_Q4B32 and ATS_FMT_MXFP4 tensors only (ATS_FMT_W16: ATS_ERR_INVALID);
 *  - the context still needs the first kilobyte of a workspace (workspace_bytes >= 1024, set at ats_init): that is
 *    where the attention counters and, on systems without mapped pinned memory, the status word live.  Nothing else of
 *    the workspace is touched;
 *  - the tensor must be GPU-placed (streaming would need the ring) -> ATS_ERR_STATE otherwise;
 *  - if the split-K plan ats_linear would pick with unlimited workspace needs more than ATS_STATIC_SCRATCH_BYTES for its
 *    partial sums, the call fails with ATS_ERR_NOMEM and the text says how much was needed (no smaller plan is tried);
 *  - every GPU that loads the library holds the array from load to exit; all calls (all contexts, all streams of a
 *    process) share it, and nothing in it has to start at zero: each call fully writes the partials it later reads.
 *    Two calls that overlap on the GPU (different streams) would overwrite each other's partials: keep them on one stream;
 *  - the first call on a device looks the array's device address up (cudaGetSymbolAddress) and caches it; make that
 *    first call before any stream capture begins. */
#define ATS_STATIC_SCRATCH_BYTES (8ull << 20)
int32_t ats_linear_static_scratch(ats_ctx* ctx, int32_t id, const void* x /*DEVICE*/, void* y /*DEVICE*/, uint32_t M);

/* Router: logits = h W_r (fp16 weights [hidden][E], fp32 accumulation); ids[m][0..k) = the k largest logits in
 * descending order, equal logits -> lower expert index first; gates = softmax over the selected logits.
 * h DEVICE fp16 [M][hidden]; ids_dev DEVICE int32 [M][k]; gates_dev DEVICE fp32 [M][k].  k <= 32, E <= 1024. */
int32_t ats_route_topk(ats_ctx* ctx, int32_t router_id, const void* h /*DEVICE*/, uint32_t M, uint32_t k,
                       int32_t* ids_dev /*DEVICE*/, float* gates_dev /*DEVICE*/);

/* Top-k routed expert GEMV on a stacked expert tensor: y[m][j][:] = W[ids[m][j]] x[m][:] (x_per_slot = 0, x [M][K])
 * or W[ids[m][j]] x[m][j][:] (x_per_slot = 1, x [M][k][K]); fp16 in, fp32 accumulation, fp16 out [M][k][n_out].
 * M*k <= 256.  Every id must lie in [0, n_experts).  With host-placed slices the ids are checked on the host
 * (ATS_ERR_INVALID before anything is enqueued); when every slice is resident they are only seen by the kernel, which
 * then computes with expert 0 in place of an id out of range and raises the context's status word: the next ats_sync
 * returns ATS_ERR_INVALID and the context is poisoned.  (ats_route_topk always writes ids in range, also for a row of
 * NaN activations, whose gates are NaN.)  If any expert slice of the tensor is host-placed the call copies ids to the host and waits for them
 * (the one host synchronisation on the path: expert transfer cannot start before routing is known, Section 4.2.2),
 * then streams only the selected host-placed slices (distinct over the batch, ascending expert id). */
int32_t ats_moe_linear(ats_ctx* ctx, int32_t id, const void* x /*DEVICE*/, const int32_t* ids_dev /*DEVICE*/,
                       void* y /*DEVICE*/, uint32_t M, uint32_t k, uint32_t x_per_slot);

/* One decoder layer.  Tensor ids; -1 = absent.  Attention part runs if wq >= 0; the FFN part is dense SwiGLU if
 * n_experts == 0, else a top-k MoE of SwiGLU experts (w_gate/w_up/w_down stacked, router F16 [hidden][E]).
 * Math: h = RMSNorm(x; attn_norm); q,k,v = W h; rotary embedding (half-split pairs, angle pos*theta^(-2i/d)) on q,k;
 * K/V of the new token(s) are written to the caches as fp16 first; causal grouped-query attention with scale
 * 1/sqrt(head_dim), query head hq reading kv head hq/(n_q/n_kv); x1 = x + W_o a; h2 = RMSNorm(x1; ffn_norm);
 * y = x1 + W_down(silu(W_gate h2) * (W_up h2))  (MoE: y = x1 + sum_j gate_j FFN_{e_j}(h2) in rank order). */
typedef struct {
  int32_t attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down, router;
  uint32_t hidden, n_q_heads, n_kv_heads, head_dim, ffn, n_experts, top_k, kv_capacity;
  float rms_eps;
  float rope_theta;  /* 0 = no rotary embedding */
  uint32_t flags;    /* ATS_LAYER_* */
} ats_layer_desc;

/* Decode: M tokens, each one step of its own sequence.  With an attention part M must be 1 (one sequence; the token
 * sits at cache position `pos` = number of past tokens, pos < kv_capacity); an FFN-only layer (wq = -1) takes M <= 32.
 * x_in, x_out DEVICE fp16 [M][hidden] (may alias); k_cache, v_cache DEVICE fp16 [n_kv_heads][kv_capacity][head_dim],
 * caller-owned, updated in place (ignored when wq = -1).  Streams host-placed tensors of the layer through the ring. */
int32_t ats_layer_decode(ats_ctx* ctx, const ats_layer_desc* desc /*HOST*/, const void* x_in /*DEVICE*/,
                         void* x_out /*DEVICE*/, void* k_cache /*DEVICE*/, void* v_cache /*DEVICE*/, uint32_t pos,
                         uint32_t M);
/* The same decode step driven from HOST buffers, as a caller that holds activations on the host sees it: brings x_in
 * (HOST fp16 [M][hidden]) into the workspace, runs ats_layer_decode on the compute stream, brings the result into x_out
 * (HOST fp16 [M][hidden]) and returns when x_out is valid.  The caches stay on the DEVICE.  Needs 2 * M * hidden * 2 bytes
 * of workspace beyond ats_layer_decode's (ats_workspace_bytes includes them).
 * Any host memory works (two cudaMemcpyAsync and a wait for the stream).  When both buffers lie inside ranges registered
 * with ats_register_host_buffer, only x_in is copied: the layer's last kernel stores the result row straight into x_out,
 * and the call returns as soon as the device has written a completion word that the host polls (bounded; it falls back
 * to waiting for the stream).
 * The status word of the context is looked at before returning: ATS_ERR_TIMEOUT if a kernel gave up a bounded wait.
 * Errors as ats_layer_decode, plus ATS_ERR_CUDA from the copies or the wait. */
int32_t ats_layer_decode_host(ats_ctx* ctx, const ats_layer_desc* desc /*HOST*/, const void* x_in /*HOST*/,
                              void* x_out /*HOST*/, void* k_cache /*DEVICE*/, void* v_cache /*DEVICE*/, uint32_t pos,
                              uint32_t M);
/* Pinned host memory the caller will pass to host-driven calls (ats_layer_decode_host).  [ptr, ptr + bytes) must be
 * page-locked memory that the device can address (cudaHostAlloc / cudaHostRegister, or a framework's pinned allocation),
 * 16-byte aligned; the library keeps the range's device alias and lets kernels read and write the memory directly.
 * LIFETIME: the range must stay allocated and pinned until ats_unregister_host_buffer (which first waits for the compute
 * stream) or ats_destroy; the library never looks a raw address up again on its own, so a buffer that was freed and whose
 * address was reused is the caller's error only if it is still registered.  Buffers that are not registered are served
 * by ordinary copies.  ATS_ERR_INVALID if the memory is not pinned and mapped. */
int32_t ats_register_host_buffer(ats_ctx* ctx, void* ptr /*HOST*/, uint64_t bytes);
int32_t ats_unregister_host_buffer(ats_ctx* ctx, void* ptr /*HOST*/);

/* Prefill: T tokens of one sequence at cache positions pos0 .. pos0+T-1 (pos0+T <= kv_capacity); projections run as
 * dequantize-fused tensor-core GEMMs.  Same buffers as decode with M = T.
 * Layers with routed experts (the MoE prefill of Section 5's workloads): every (token, slot) pair becomes a row, rows
 * are sorted by expert on the host from the routing ids (one synchronisation per call; T * top_k <= 65536) and each
 * projection is ONE grouped GEMM launch in which every expert multiplies its own block of rows with its own slice;
 * y = rn16(x1 + sum_j gate_j d_j) with the expert outputs d_j rounded to fp16 as every GEMM output of the prefill
 * contract is.  Host-placed experts that some token selected are brought into the part of the workspace that lies beyond
 * ats_workspace_bytes(desc, T) by one SM-driven copy launch (bulk-async copies from the mapped pinned store, the copy
 * kernel of Section 4.2.1; counted in ats_stats.streamed_bytes, not in copies) when that part holds them; otherwise the
 * GEMMs read those slices in place over PCIe, which is several times slower.  Same results either way. */
int32_t ats_layer_prefill(ats_ctx* ctx, const ats_layer_desc* desc /*HOST*/, const void* x_in /*DEVICE*/,
                          void* x_out /*DEVICE*/, void* k_cache /*DEVICE*/, void* v_cache /*DEVICE*/, uint32_t pos0,
                          uint32_t T);

/* Workspace a layer call needs: pass the largest value over the calls you will make as ats_config.workspace_bytes. */
uint64_t ats_workspace_bytes(const ats_layer_desc* desc /*HOST*/, uint32_t max_tokens);

/* Block dequantization of one (tensor, expert) slice (expert = 0 for a dense tensor) from the library's internal
 * format: out[n][k] = scale*code as fp32 (exact) or rounded once to fp16.  out_dev DEVICE [n_out][k_in].
 * Reads the resident copy if the slice is GPU-placed, else streams it through the ring. */
int32_t ats_dequantize(ats_ctx* ctx, int32_t id, int32_t expert, void* out_dev /*DEVICE*/, uint32_t out_fmt);

/* The numerics contract of a mode: bit i of *fp16_edge_mask set = the layer rounds intermediate i to fp16, for
 * i over {h, q, k, v, q_rot, a, o, x1, h2, g, u, act, d}; *weight_mode 0 = weights exact (scale*code in fp32),
 * 1 = weights rounded once to fp16 (tensor-core operands).  Cache entries and x_out are always fp16. */
int32_t ats_get_numerics(const ats_ctx* ctx, uint32_t mode, uint32_t* fp16_edge_mask /*HOST*/,
                         uint32_t* weight_mode /*HOST*/);

#define ATS_STATS_LIST 512
typedef struct {
  uint64_t resident_bytes;   /* Q4B32 slices placed on the GPU */
  uint64_t aux_bytes;        /* F16 tensors (always resident) */
  uint64_t host_store_bytes; /* pinned host store */
  uint64_t streamed_bytes;   /* host->device weight bytes since the last ats_reset_stats */
  uint64_t copies;           /* cudaMemcpyAsync calls for those bytes */
  uint64_t kernel_launches;  /* kernels launched by the library since the last reset */
  uint64_t ring_reuses;      /* copies that had to wait for a slot's previous consumer */
  uint64_t host_syncs;       /* host waits for routing ids */
  /* With ATS_FLAG_TIME_KERNELS: per kernel family (0 GEMV, 1 grouped-expert GEMV, 2 tensor-core GEMM) since the last
   * reset: launches, summed device time of the completed launches (CUDA events on the compute stream) and the
   * algorithmic work they did (families 0,1: bytes = weights + activations in + out; family 2: flops = 2*T*N*K). */
  uint64_t timed_launches[3];
  uint64_t timed_work[3];
  double timed_ms[3];
  uint32_t n_streamed;       /* streamed slices since the last reset (list below holds the first ATS_STATS_LIST) */
  uint32_t reserved;
  int32_t streamed_ids[ATS_STATS_LIST];
  int32_t streamed_experts[ATS_STATS_LIST];
} ats_stats;
/* Kernel times are read from events here: call after ats_sync() so that every timed launch has completed. */
int32_t ats_get_stats(ats_ctx* ctx, ats_stats* out /*HOST*/);
/* Replace the context's flags (ATS_FLAG_*) at run time, e.g. to switch kernel timing on for a profiling pass. */
int32_t ats_set_flags(ats_ctx* ctx, uint32_t flags);
int32_t ats_reset_stats(ats_ctx* ctx);

/* Wait for everything enqueued so far by polling events; ATS_ERR_TIMEOUT after timeout_ms (0 = wait without limit),
 * ATS_ERR_CUDA if a kernel or copy failed.  Then the context's status word is read: ATS_ERR_TIMEOUT if a kernel gave up
 * one of its bounded waits, ATS_ERR_INVALID if a kernel met a token or expert id out of range; either poisons the
 * context (its results are invalid).  The word lives in pinned host memory, so the calls that wait on the host anyway
 * (ats_layer_decode_host, and the MoE calls that fetch routing ids) check it too. */
int32_t ats_sync(ats_ctx* ctx, uint32_t timeout_ms);

/* Measure host->device copy bandwidth from the library's own kind of pinned memory into the arena's ring:
 * `bytes` (<= ring size) copied `reps` times, best time.  Synchronous.  Writes GB/s (1e9 bytes/s). */
int32_t ats_measure_h2d(ats_ctx* ctx, uint64_t bytes, uint32_t reps, double* out_gbs /*HOST*/);

/* Measure what the device delivers to a kernel that only READS: the first `bytes` of the arena (at least 256 MiB, more
 * than the L2 holds) are read once per pass by a kernel with the streaming GEMV's access pattern (bulk-async copies into
 * shared memory, nothing done with the data), `reps` passes after a warm-up pass, best time.  Synchronous; the arena's
 * contents are not changed.  Writes GB/s (1e9 bytes/s): the read-only ceiling to hold the GEMV's achieved bandwidth
 * against, beside the nominal figure and a copy benchmark (which also writes and reaches less). */
int32_t ats_measure_hbm_read(ats_ctx* ctx, uint64_t bytes, uint32_t reps, double* out_gbs /*HOST*/);

/* Test hook: make the next n streaming copies fail as if cudaMemcpyAsync had returned an error (host-side fault
 * injection; nothing faults on the device).  The failing call returns ATS_ERR_CUDA and the context is poisoned. */
int32_t ats_debug_fail_copies(ats_ctx* ctx, uint32_t n);

/* Test hook for the failure path of the streaming single-token GEMV (nothing faults, nothing hangs): from now on that
 * kernel's bounded waits give up after limit_cycles SM clock cycles (0 = the default of about a second), and its producer
 * leaves out the weight copies of tile `withhold_tile` of every launch (-1 = none), so the consumers of that tile wait in
 * vain, run into the limit, raise the context's device status word and return; every other CTA finishes normally.  The
 * next ats_sync (or ats_layer_decode_host) then returns ATS_ERR_TIMEOUT and the context is poisoned; other contexts of the
 * process are unaffected.  Applies to dense single-token GEMV launches only (ats_linear with M = 1, ats_layer_decode). */
int32_t ats_debug_gemv_wait(ats_ctx* ctx, uint64_t limit_cycles, int32_t withhold_tile);
/* Timing hook: ats_layer_decode leaves out the launches whose bit is set (dense layers: 1 = QKV GEMV, 2 = attention,
 * 4 = O GEMV, 8 = gate/up GEMV, 16 = down GEMV; routed-expert FFN with every expert resident: 32 = router, 64 = experts'
 * gate/up stage, 128 = experts' down stage, 256 = gated sum; the skipped router leaves the ids of an earlier call in
 * place, so run one full call first); the outputs of such a call are stale.  0 restores the full step.  Used by the
 * benchmark to time the GEMV launches of a step without the attention launch between them. */
int32_t ats_debug_skip_stages(ats_ctx* ctx, uint32_t mask);

/* The two ends of a whole-model loop around the layer calls (Section 5's workloads run whole models).
 * ats_embed: rows token_ids[m] of a Q4B32 table [vocab = n_out][hidden = k_in], dequantized to fp16 (scale * code rounded
 * once, as ats_dequantize writes it): out DEVICE fp16 [M][k_in].  token_ids DEVICE int32 [M]; an id outside [0, n_out)
 * gives a row of zeros and makes the next ats_sync fail.  A host-placed table is read in place through the mapped pinned
 * store (a few rows per call), never streamed whole.
 * ats_lm_head: logits = W_head * RMSNorm(x; norm_id gain, eps), x DEVICE fp16 [M][hidden], logits DEVICE fp16 [M][vocab];
 * the normalised row is rounded to fp16 before the product (the contract's edge "h").  M = 1 runs as one launch of the
 * streaming GEMV with the norm as its prologue (hidden <= 4096 and a shape that kernel takes); otherwise a norm launch
 * into `scratch` (DEVICE fp16 [M][hidden], caller-provided, may be NULL only for the one-launch case) and ats_linear.
 * A W16 or MXFP4 head always takes the second form (scratch required). */
int32_t ats_embed(ats_ctx* ctx, int32_t id, const int32_t* token_ids /*DEVICE*/, uint32_t M, void* out /*DEVICE*/);
int32_t ats_lm_head(ats_ctx* ctx, int32_t norm_id, int32_t head_id, float eps, const void* x /*DEVICE*/, void* logits /*DEVICE*/,
                    uint32_t M, void* scratch /*DEVICE*/);

/* Debug/test hook: device address and byte size of an intermediate of the most recent ats_layer_decode call shape
 * (which = 0 h, 1 qkv (fp32 [q|k|v]), 2 q_rot (fp32), 3 a (fp16), 4 x1 (fp32), 5 h2 (fp16), 6 act (fp16), 7 d (fp32, MoE),
 * 8 ids (int32, MoE), 9 gates (fp32, MoE)).  The workspace is reused by every call; read it after ats_sync(). */
int32_t ats_debug_decode_buffer(ats_ctx* ctx, const ats_layer_desc* desc /*HOST*/, uint32_t M, uint32_t which,
                                void** out_dev /*HOST*/, uint64_t* out_bytes /*HOST*/);

/* Same for ats_layer_prefill with T tokens: which = 0 h, 1 qkv (fp16 [T][q|k|v]), 2 q_rot, 3 a, 4 o, 5 x1, 6 h2,
 * 7 gate|up (fp16 [T][2*ffn]), 8 act, 9 d; all fp16. */
int32_t ats_debug_prefill_buffer(ats_ctx* ctx, const ats_layer_desc* desc /*HOST*/, uint32_t T, uint32_t which,
                                 void** out_dev /*HOST*/, uint64_t* out_bytes /*HOST*/);

/* ---- host-only utilities (no context, no GPU needed) ---- */

/* Algorithm 1 on caller-supplied arrays (all HOST): n tensors in execution order with sizes s[i] (units), values r[i],
 * switch costs c[i] (c[0] unused), is_expert[i] (0/1; null = dense model), budget M units.  Writes ATS_HOST/ATS_GPU to
 * out_b[0..n) and, if non-null, the value of the placement objective of Section 4.3.2 to *out_objective. */
int32_t ats_host_solve_placement(const int64_t* s, const int64_t* r, const int64_t* c, const uint8_t* is_expert, uint32_t n,
                                 int64_t M, uint8_t* out_b, int64_t* out_objective);
/* Interchange layout -> the library's internal slice layout (n_out*k_in/2 code bytes followed by n_out*k_in/32 fp16
 * scales) and back; out_* are HOST buffers of the same sizes as the inputs.  The round trip is the identity. */
/* The row order of the MoE prefill's grouped GEMMs (host only): the stable sort of the P (token, slot) pairs by expert id.
 * ids[p] in [0, E); order[r] = the pair at sorted position r; pos[p] = the sorted position of pair p; off[e] = first
 * position of expert e, off[E] = P; *max_rows = the largest expert's row count.  ATS_ERR_INVALID for an id out of range. */
int32_t ats_host_group_pairs(const int32_t* ids, uint32_t P, uint32_t E, int32_t* order, int32_t* pos, int32_t* off,
                             int32_t* max_rows);
int32_t ats_host_repack_q4(const void* codes, const void* scales, void* out_slice, uint32_t n_out, uint32_t k_in);
int32_t ats_host_unpack_q4(const void* slice, void* out_codes, void* out_scales, uint32_t n_out, uint32_t k_in);

/* Load-aware dynamic transfer (Section 4.4), host only.  A round runs tensors 0..n-1 in order; b[i] (ATS_HOST / ATS_GPU) is
 * the default backend from static placement, t_gpu[i] / t_host[i] the current execution times of tensor i's operator on the
 * GPU / on the host, c[i] the activation-transfer cost paid when tensors i-1 and i run on different backends (c[0] unused),
 * w[i] the weight-transfer time of tensor i (for an expert operator in a decode round: of the activated experts only).  All
 * times in one unit, finite and >= 0 (else ATS_ERR_INVALID).
 *
 * ats_host_dynamic_transfer: Algorithm 2.  Writes the runtime backend assignment to out_rb[0..n): resident tensors stay on
 * the GPU; a host tensor stays or is promoted (out_rb[i] = ATS_GPU), in which case out_start[i] (optional array) is the
 * tensor after which its weight transfer starts, ATS_ROUND_START for the start of the round; ATS_NO_TRANSFER elsewhere.
 * *out_latency (optional) = the round latency T of Section 4.4.1 for that plan: execution times on the runtime backends +
 * switch costs + for every promoted tensor the part of w[i] that the default-path work between its start point and i does
 * not hide.  Between a start point and its promoted tensor nothing else is promoted.  O(n^2) time, O(n) space.
 * ats_host_transfer_latency: T for a caller-given plan (ATS_ERR_INVALID if a resident tensor is moved off the GPU or a
 * start index is not before its tensor; whether the start points are admissible is the caller's business).
 * ats_host_deviation: ComputeDeviation of Algorithm 3, read as the largest relative change |cur - prev| / prev over the n
 * measured quantities (a quantity leaving 0 counts as infinite, one staying 0 as none).
 * ats_host_reschedule: Algorithm 3.  m_ref / m_cur are measurement snapshots [4n] = t_gpu | t_host | c | w.  If the
 * deviation of m_cur from m_ref is below eps, or less than tau has passed since *t_last, nothing changes (the previous
 * rb / start stay, *out_replanned = 0); otherwise Algorithm 2 runs on m_cur into rb / start (start optional), m_cur becomes
 * the reference, *t_last = t_now and *out_replanned = 1; rebuilding the execution plan for the new assignment is the
 * caller's step.  The paper uses eps = 0.15 and tau = 5 x the recent time per output token. */
enum { ATS_ROUND_START = -1, ATS_NO_TRANSFER = -2 };
int32_t ats_host_dynamic_transfer(const uint8_t* b, const double* t_gpu, const double* t_host, const double* c, const double* w,
                                  uint32_t n, uint8_t* out_rb, int32_t* out_start, double* out_latency);
int32_t ats_host_transfer_latency(const uint8_t* rb, const int32_t* start, const uint8_t* b, const double* t_gpu, const double* t_host,
                                  const double* c, const double* w, uint32_t n, double* out_latency);
double ats_host_deviation(const double* m_prev, const double* m_cur, uint32_t n);
int32_t ats_host_reschedule(const uint8_t* b, uint32_t n, double* m_ref, const double* m_cur, double eps, double tau, double t_now,
                            double* t_last, uint8_t* rb, int32_t* start, int32_t* out_replanned);

#ifdef __cplusplus
}
#endif
#endif /* ATS_H_ */
