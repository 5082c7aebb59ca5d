// Internal declarations shared by the host runtime and the CUDA kernels of the ats library.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/ats.h"

namespace ats {

constexpr int kBlock = 32;        // weights per quantization block
constexpr uint64_t kAlign = 256;  // alignment of every region / slice inside the arena

inline uint64_t align_up(uint64_t v, uint64_t a = kAlign) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// Internal weight format "Q4B32i" of one (tensor, expert) slice:
//   [codes: N rows x K/2 bytes][scales: N rows x K/32 fp16], the slice padded to 256 bytes.
// Codes are stored per 32-bit word (8 consecutive k of a row): nibble position p of the word holds
//   p = 0,1,2,3 -> k = 0,2,4,6 ;  p = 4,5,6,7 -> k = 1,3,5,7
// as offset-binary u = code + 8.  With that order (word >> 8s) & 0x000F000F yields the fp16 pair
// (k, k+1) after OR-ing the 1024.0 exponent, with no per-nibble shifts.
// ---------------------------------------------------------------------------------------------
struct Slice {
  uint8_t where = ATS_HOST;
  uint8_t* dev = nullptr;  // resident copy (null when host-placed)
};

struct Tensor {
  ats_tensor_desc d{};
  uint64_t codes_bytes = 0;   // per slice
  uint64_t slice_bytes = 0;   // codes + scales (what streaming moves and the statistics count)
  uint64_t slice_stride = 0;  // slice_bytes padded to 256 (distance between slices in host store / resident region)
  uint8_t* host = nullptr;    // pinned store, n_experts * slice_stride bytes (F16: the raw fp16 data)
  uint64_t host_bytes = 0;
  uint8_t* f16_dev = nullptr;  // F16 tensors: device copy
  std::vector<Slice> slices;
  bool any_host = true;        // some slice is host-placed
  bool contiguous_dev = false; // all slices resident, at dev0 + e * slice_stride
  // expert-stacked tensors: device array of one address per slice, the resident copy or the slice's place in the pinned
  // host store as the device sees it (mapped memory); null for single-slice tensors
  const uint8_t** slice_tab_dev = nullptr;
  const uint8_t* host_dev = nullptr;  // the pinned store as the device addresses it (null when it is not mapped)
};

struct RingSlot {
  cudaEvent_t ready = nullptr;  // recorded on the transfer stream after the slot's copies
  cudaEvent_t freed = nullptr;  // recorded on the compute stream after the slot's consumer
  bool used = false;            // freed has been recorded at least once
  bool busy = false;            // holds a slice whose consumer has not been enqueued yet
};

// One streamed slice of the current call (an entry of the per-call execution plan).
struct Fetch {
  int tensor = -1;
  int expert = 0;
  int slot = -1;
  bool enqueued = false;  // copy is on the transfer stream
  bool waited = false;    // compute stream already waits on the slot's ready event
};

}  // namespace ats

struct ats_ctx {
  ats_config cfg{};
  cudaStream_t cs = nullptr, ts = nullptr;
  std::string err;
  bool poisoned = false;
  bool placed = false;
  std::vector<ats::Tensor> tensors;
  // arena layout
  uint8_t* ws = nullptr;        // workspace
  uint8_t* ring = nullptr;      // ring_slots * slot_stride
  uint64_t slot_stride = 0;
  uint8_t* resident = nullptr;  // start of aux + resident region
  uint64_t resident_cap = 0;
  std::vector<ats::RingSlot> slots;
  // per-call streaming plan
  std::vector<ats::Fetch> plan;
  size_t plan_next = 0;  // next plan entry whose copy is not enqueued yet
  uint32_t next_slot = 0;
  // pinned scratch for routing ids (host side of the one synchronisation on the MoE path)
  int32_t* ids_host = nullptr;
  // pinned host buffers the caller registered for host-driven calls (ats_register_host_buffer): host range -> device alias
  struct HostBuf {
    const uint8_t* host;
    uint64_t bytes;
    uint8_t* dev;
  };
  std::vector<HostBuf> host_bufs;
  volatile int* done_host = nullptr;  // pinned completion word of host-driven calls (written by the device)
  int* done_dev = nullptr;            // ... as the device addresses it (null: the store is not mapped)
  int done_seq = 0;
  uint8_t* stage_host = nullptr;  // pinned scratch for per-call tables (MoE prefill: slice addresses, copy list)
  cudaEvent_t ids_event = nullptr;
  cudaEvent_t sync_event = nullptr;
  uint32_t fail_copies = 0;
  // test hooks (ats_debug_gemv_wait, ats_debug_skip_stages)
  long long dbg_wait_limit = 0;
  int dbg_withhold_plus1 = 0;
  uint32_t dbg_skip = 0;
  // The status word kernels raise when a bounded wait expires or an id is out of range.  It lives in pinned host memory
  // that the device addresses directly (dev_status is that alias), so every call that already waits on the host can look
  // at it without a copy; on a system where the store cannot be mapped it is the first word of the workspace and only
  // ats_sync reads it (with a copy).
  int* dev_status = nullptr;
  int* host_status = nullptr;
  bool status_mapped = false;
  bool ws_reserved = false;   // the workspace holds the reserved first kilobyte (attention counters, fallback status word)
  int sm_count = 148;
  std::vector<double> rope_inv;  // cached theta^(-2i/d)
  float rope_theta = -1.f;
  int rope_d = 0;
  ats_stats stats{};
  // kernel timing (ATS_FLAG_TIME_KERNELS): event pairs in launch order, family per pair
  std::vector<cudaEvent_t> tev;
  std::vector<uint8_t> tev_family;
  size_t tev_used = 0;  // events handed out (2 per timed launch)
};

namespace ats {

int32_t fail(ats_ctx* c, int32_t code, const char* fmt, ...);
int32_t check_cuda(ats_ctx* c, cudaError_t e, const char* what);

// ----------------------------------------------------------------------------- kernel launchers
// All launchers enqueue on `st`, return the cudaError of the launch and count launches in *n_launch.

struct GemvSeg {
  const uint8_t* base;  // slice base (codes, then scales)
  int n_rows;
};
enum GemvMode {
  GEMV_OUT_F32 = 0,        // y32[m][row] = acc
  GEMV_OUT_F16 = 1,        // y16[m][row] = rn16(acc)
  GEMV_RES16_OUT_F32 = 2,  // y32 = float(res16) + acc
  GEMV_RES32_OUT_F16 = 3,  // y16 = rn16(res32 + acc)
  GEMV_SWIGLU_F16 = 4,     // seg[0] = gate, seg[1] = up (same n_rows): y16 = rn16(silu(g) * u)
  GEMV_RES16_OUT_F16 = 5   // y16 = rn16(float(res16) + acc)
};
struct GemvParams {
  GemvSeg seg[3];
  int n_seg;
  int K;
  int M;
  const __half* x;
  int ldx;
  float* y32;
  __half* y16;
  int ldy;
  const float* res32;
  const __half* res16;
  int ldres;
  int mode;
  // optional RMSNorm prologue (M = 1): x = rn16(norm_x * norm_gain / sqrt(mean(norm_x^2) + norm_eps)); exactly one of
  // norm_x16 / norm_x32 is set when norm_gain is; norm_out (optional) receives the normalised operand
  const __half* norm_x16;
  const float* norm_x32;
  const __half* norm_gain;
  float norm_eps;
  __half* norm_out;
  int pdl;  // allow the launch to overlap the tail of the preceding kernel (programmatic dependent launch)
  int w16;  // the segments are unquantized fp16 matrices [n_rows][K] (launch_gemv_w16; no norm prologue)
  int mx;   // the segments hold microscaling 4-bit floats (same slice layout, power-of-two fp16 block scales): generic kernel only
  // test hooks of the streaming kernel (ats_debug_gemv_wait): limit of its bounded waits in SM cycles (0 = the default of
  // about a second) and, plus one, the tile whose weight copies its producer leaves out (0 = none)
  long long dbg_wait_limit;
  int dbg_withhold_tile_plus1;
};
cudaError_t launch_gemv(const GemvParams& p, cudaStream_t st, uint64_t* n_launch);
// fp16-weight GEMV (kernels_decode.cu): the same segments, epilogue modes and fp32 accumulation as launch_gemv over
// unquantized fp16 matrices; M <= 8, K a multiple of 8, x given (the norm prologue fields are ignored)
cudaError_t launch_gemv_w16(const GemvParams& p, cudaStream_t st, uint64_t* n_launch);
// few-row GEMV of the 4-bit formats on mma.sync (kernels_gemv_mma.cu): same segments and epilogues as launch_gemv, x given
bool gemv_mma_eligible(const GemvParams& p);
cudaError_t launch_gemv_mma(const GemvParams& p, cudaStream_t st, uint64_t* n_launch);
// the streaming single-token kernel (kernels_gemv_stream.cu): shapes it accepts, and its launcher
bool gemv_stream_eligible(const GemvParams& p);
cudaError_t launch_gemv_stream(const GemvParams& p, int* status, int sm_count, cudaStream_t st, uint64_t* n_launch);

// Grouped-expert GEMV: job j multiplies the slice w0[j] (and w1[j] for SwiGLU) with activation row xrow[j] and
// writes output row j_out[j].  Implicit mode (n_jobs_explicit == 0): job p = 0..P-1 uses expert ids[p] of a
// contiguous resident tensor.
// Function attributes (the dynamic shared-memory limit) are per device: a launcher sets them the first time it runs on
// each device.  `done` holds one bit per device ordinal; setting an attribute twice is harmless, so no lock is needed.
inline bool first_use_on_device(uint64_t* done) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
  if ((*done >> dev) & 1ull) return false;
  *done |= 1ull << dev;
  return true;
}

// Launch with the programmatic-dependent-launch attribute: the kernel may start while its predecessor in the stream is
// still finishing; every kernel launched this way executes griddepcontrol.wait before it touches the predecessor's data.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dep(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int pdl, int cluster_x,
                              Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[na].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
  ++na;
  if (cluster_x > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = cluster_x;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

constexpr int kMoeJobsPerLaunch = 64;
struct MoeJobs {
  const uint8_t* w0[kMoeJobsPerLaunch];
  const uint8_t* w1[kMoeJobsPerLaunch];
  int16_t xrow[kMoeJobsPerLaunch];
  int16_t orow[kMoeJobsPerLaunch];
  int n;
};
struct MoeGemvParams {
  // implicit addressing
  const uint8_t* base0;
  const uint8_t* base1;
  uint64_t stride;
  const int32_t* ids;  // [P]
  const uint8_t* const* tab0;  // optional per-expert slice addresses (device array); when set they replace base + id * stride
  const uint8_t* const* tab1;
  int x_div;           // activation row of pair p is p / x_div (k when one x per token, 1 when one per slot)
  int P;
  int n_experts;       // ids outside [0, n_experts) are replaced by 0 and raise *status (implicit addressing)
  int* status;
  // common
  int n_rows, K;
  const __half* x;
  int ldx;
  float* y32;
  __half* y16;
  int ldy;
  int mode;  // GEMV_OUT_F32, GEMV_OUT_F16 or GEMV_SWIGLU_F16
  int mx;    // microscaling 4-bit floats instead of integer codes (generic kernel only)
};
cudaError_t launch_moe_gemv(const MoeGemvParams& p, const MoeJobs* jobs /*null = implicit*/, cudaStream_t st,
                            uint64_t* n_launch);
// the streaming kernel's grouped-expert form (kernels_gemv_stream.cu): shapes it accepts, and its launcher
bool moe_gemv_stream_eligible(const MoeGemvParams& p);
cudaError_t launch_moe_gemv_stream(const MoeGemvParams& p, const MoeJobs* jobs /*null = implicit*/, int* status, int sm_count,
                                   int pdl, cudaStream_t st, uint64_t* n_launch);

// reads `bytes` of device memory once with the streaming GEMV's access pattern and drops them (kernels_gemv_stream.cu)
cudaError_t launch_hbm_read_probe(const uint8_t* src, uint64_t bytes, int* status, int sm_count, cudaStream_t st);

cudaError_t launch_dequant(const uint8_t* slice, int n_rows, int K, void* out, int out_f16, int mx, cudaStream_t st,
                           uint64_t* n_launch);
cudaError_t launch_embed_rows(const uint8_t* slice, int n_rows, int K, const int32_t* ids, int M, __half* out, int* status,
                              int mx, cudaStream_t st, uint64_t* n_launch, int pdl = 0);
cudaError_t launch_rmsnorm(const void* x, int x_is_f32, const __half* gain, __half* out, int M, int H, float eps,
                           cudaStream_t st, uint64_t* n_launch, int pdl = 0);
// decode attention, fused with the rotary embedding and the KV append (kernels_decode.cu)
constexpr int kAttnMaxCounters = 192;  // arrival counters of the decode attention in the workspace's reserved head
struct AttnDecodeParams {
  const float* qkv;   // [q | k | v] fp32 of the new token
  float* q_rot_out;   // optional copy of the rotated query (debug / tests)
  __half* kc;
  __half* vc;
  float* part;        // [n_q][splits][d + 2] scratch
  int* counters;      // [n_kv * hsplit] zero between launches
  __half* a16;        // [n_q * d]
  int n_q, n_kv, group, cap, pos;
  int hsplit;         // CTAs that share a kv head's query heads (set by the launcher)
  float scale;
  float cs[128];      // (cos, sin) of pos * theta^(-2i/d), i < d/2
};
int attn_decode_splits(int n_ctx);
size_t attn_decode_scratch_floats(int n_q, int d, int n_ctx);
cudaError_t launch_attn_decode_fused(AttnDecodeParams p, int d, int pdl, cudaStream_t st, uint64_t* n_launch);
cudaError_t launch_router_topk(const __half* h, const __half* wr, int M, int H, int E, int k, int renorm, int32_t* ids,
                               float* gates, cudaStream_t st, uint64_t* n_launch, int pdl = 0);
cudaError_t launch_router_topk_norm(const __half* h, const __half* wr, int M, int H, int E, int k, int renorm, int32_t* ids,
                                    float* gates, const void* norm_x, int norm_x_f32, const __half* norm_gain, float eps,
                                    cudaStream_t st, uint64_t* n_launch, int pdl = 0);
// y16[m] = rn16(res[m] + sum_j gates[m][j] * d32[m*k + j])   (res fp16 or fp32)
cudaError_t launch_moe_combine(const void* res, int res_is_f32, const float* gates, const float* d32, __half* y16,
                               int M, int k, int H, cudaStream_t st, uint64_t* n_launch, int pdl = 0);
cudaError_t launch_fill(void* p, uint64_t bytes, uint8_t v, cudaStream_t st, uint64_t* n_launch);
// host-driven calls (kernels_decode.cu): the completion word written once everything before it in the stream is done
cudaError_t launch_signal_done(int* done_alias, int seq, int pdl, cudaStream_t st, uint64_t* n_launch);

// prefill
cudaError_t launch_rope_append_prefill(const __half* qkv16, int ld, __half* q_rot16, __half* kc, __half* vc, int T,
                                       int n_q, int n_kv, int d, int cap, int pos0, float theta, cudaStream_t st,
                                       uint64_t* n_launch, int pdl = 0);
cudaError_t launch_attn_prefill(const __half* q_rot16, const __half* kc, const __half* vc, __half* a16, int T, int n_q,
                                int n_kv, int d, int cap, int pos0, cudaStream_t st, uint64_t* n_launch, int pdl = 0);
// MoE prefill helpers (kernels_prefill.cu): rows gathered in expert order, and the gated sum back in token order
cudaError_t launch_moe_gather_rows(const __half* h, const int* order, int k, __half* xs, int P, int H, cudaStream_t st,
                                   uint64_t* n_launch, int pdl = 0);
cudaError_t launch_moe_combine_sorted(const __half* res, const float* gates, const __half* d, const int* pos, __half* y, int T, int k,
                                      int H, cudaStream_t st, uint64_t* n_launch, int pdl = 0);
// SM-driven gather of host-placed slices into device memory (kernels_prefill.cu): chunks of at most 32 KB, src in the
// mapped pinned store, both addresses and sizes multiples of 16 bytes
struct CopyChunk {
  const uint8_t* src;
  uint8_t* dst;
  uint32_t bytes;
  uint32_t pad;
};
constexpr uint32_t kCopyChunkBytes = 32 * 1024;
cudaError_t launch_host_gather(const CopyChunk* list, int n, int* status, int sm_count, cudaStream_t st, uint64_t* n_launch,
                               int pdl = 0);
cudaError_t launch_swiglu16(const __half* gu, int ld, int ffn, __half* act, int T, cudaStream_t st, uint64_t* n_launch,
                            int pdl = 0);

// Tensor-core GEMM  Y[T][n_rows] (fp16, leading dimension ldy) = X[T][K] (fp16, ld = ldx) * W^T for up to 3 weight
// segments laid side by side in Y.  `scratch` holds split-K partials (gemm_scratch_bytes()).
struct GemmParams {
  GemvSeg seg[3];
  int n_seg;
  int K;
  int T;
  const __half* x;
  int ldx;
  __half* y;
  int ldy;
  void* scratch;
  uint64_t scratch_bytes;
  int* status;  // device word raised when a bounded wait expires
  // optional fused residual: y2[t][c] = rn16(res[t][c] + y[t][c]) with y the fp16-rounded product (both ld = ldy)
  const __half* res;
  __half* y2;
  int pdl;  // programmatic dependent launch allowed (see launch_dep)
  // grouped form (MoE prefill): the T activation rows are sorted by expert; expert e owns rows grp_off[e] .. grp_off[e+1]-1
  // and multiplies them with slice e of every segment (seg[i].base + e * grp_stride, or grp_tab[i][e] where a table is
  // given: device or mapped host addresses).  No split-K, no residual.
  int w16;                  // seg[0].base is an unquantized fp16 matrix [n_rows][K] (one segment, no grouping)
  int mx;                   // the slices hold microscaling 4-bit floats (same layout as the integer codes)
  const int* grp_off;       // DEVICE [n_groups + 1]; null = plain GEMM
  int n_groups;
  int grp_max_rows;         // the largest expert's row count (sizes the grid)
  uint64_t grp_stride;
  const uint8_t* const* grp_tab[3];
};
uint64_t gemm_scratch_bytes(int T, int n_total, int K);
cudaError_t launch_gemm(const GemmParams& p, cudaStream_t st, uint64_t* n_launch, std::string* err);
// y = rn16(sum over splits of partial[s][T][ldy]) (+ optional residual into y2), splits in ascending order (kernels_gemm.cu)
cudaError_t launch_gemm_splitk_reduce(const float* partial, __half* y, int T, int n_cols, int ldy, int splits, const __half* res, __half* y2,
                                      int pdl, cudaStream_t st, uint64_t* n_launch);
// GEMMs as pairs of CTAs (kernels_gemm_pair.cu): shapes they take, and their launcher
bool gemm_pair_eligible(const GemmParams& p);
cudaError_t launch_gemm_pair(const GemmParams& p, cudaStream_t st, uint64_t* n_launch, std::string* err);
// fixed split-K scratch inside the library's device image (no allocation): capacity, and its address on the current device
uint64_t gemm_static_scratch_capacity();
cudaError_t gemm_static_scratch(void** out);

// host-side pieces
void repack_q4(const uint8_t* codes_in, const uint16_t* scales_in, uint8_t* slice_out, uint64_t n_rows, uint64_t K);
// the microscaling format into the same slice layout: elements keep their encoding, scale bytes become fp16 powers of two
void repack_mxfp4(const uint8_t* codes_in, const uint8_t* scale_bytes_in, uint8_t* slice_out, uint64_t n_rows, uint64_t K);
// Algorithm 1's dense solver; returns placement bytes (ATS_HOST/ATS_GPU) and the objective.
void solve_knapsack_dp(const std::vector<int64_t>& s, const std::vector<int64_t>& r, const std::vector<int64_t>& c,
                       int64_t M, std::vector<uint8_t>* b, int64_t* objective);
void static_placement(const std::vector<int64_t>& s, const std::vector<int64_t>& r, const std::vector<int64_t>& c,
                      const std::vector<uint8_t>& is_expert, int64_t M, std::vector<uint8_t>* b);

}  // namespace ats
