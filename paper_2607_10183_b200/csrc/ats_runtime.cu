// Host runtime of the ats library: context, tensor registry, placement, resident region, staging ring,
// per-call execution plan and the C ABI entry points.  All device work goes through the launchers declared in
// ats_internal.h; there is no CPU compute path.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <chrono>
#include <thread>

#include "ats_internal.h"

namespace ats {

int32_t fail(ats_ctx* c, int32_t code, const char* fmt, ...) {
  if (c) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    c->err = buf;
  }
  return code;
}

int32_t check_cuda(ats_ctx* c, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return ATS_OK;
  c->poisoned = true;
  return fail(c, ATS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define ATS_CUDA(call)                                       \
  do {                                                       \
    int32_t _s = ats::check_cuda(ctx, (call), #call);        \
    if (_s != ATS_OK) return _s;                             \
  } while (0)
#define ATS_TRY(expr)              \
  do {                             \
    int32_t _s = (expr);           \
    if (_s != ATS_OK) return _s;   \
  } while (0)

constexpr int kMaxPairs = 65536;  // (token, slot) pairs of one MoE call at most: ids, then the prefill's sort arrays, in ctx->ids_host
constexpr size_t kStageHostBytes = 1 << 20;  // pinned scratch for per-call tables
constexpr uint64_t kWsReserved = 1024;  // status word + attention counters at the start of the workspace
static_assert((64 + kAttnMaxCounters) * sizeof(int) <= kWsReserved, "the attention counters start at int 64 of the reserved head");

// Kernel timing: a pair of events around one launch on the compute stream.
constexpr size_t kMaxTimedLaunches = 1 << 16;
struct TimedLaunch {
  ats_ctx* ctx;
  cudaEvent_t stop = nullptr;
  TimedLaunch(ats_ctx* c, int family, uint64_t work) : ctx(c) {
    if (!(c->cfg.flags & ATS_FLAG_TIME_KERNELS) || c->tev_used / 2 >= kMaxTimedLaunches) return;
    while (c->tev.size() < c->tev_used + 2) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      c->tev.push_back(e);
    }
    cudaEvent_t start = c->tev[c->tev_used];
    stop = c->tev[c->tev_used + 1];
    if (c->tev_family.size() < c->tev_used / 2 + 1) c->tev_family.resize(c->tev_used / 2 + 1);
    c->tev_family[c->tev_used / 2] = (uint8_t)family;
    c->tev_used += 2;
    c->stats.timed_launches[family]++;
    c->stats.timed_work[family] += work;
    cudaEventRecord(start, c->cs);
  }
  ~TimedLaunch() {
    if (stop) cudaEventRecord(stop, ctx->cs);
  }
};

static uint64_t gemv_work_bytes(const GemvParams& p) {
  uint64_t rows = 0;
  for (int i = 0; i < p.n_seg; ++i) rows += (uint64_t)p.seg[i].n_rows;
  const uint64_t K = (uint64_t)p.K, M = (uint64_t)p.M;
  const uint64_t out_rows = p.mode == GEMV_SWIGLU_F16 ? rows / 2 : rows;
  const uint64_t out_b = (p.mode == GEMV_OUT_F32 || p.mode == GEMV_RES16_OUT_F32) ? 4 : 2;
  const uint64_t w_bytes = p.w16 ? rows * K * 2 : rows * K / 2 + rows * (K / 32) * 2;
  return w_bytes + M * K * 2 + M * out_rows * out_b;
}

static int32_t precheck(ats_ctx* ctx, bool need_placement) {
  if (!ctx) return ATS_ERR_INVALID;
  if (ctx->poisoned) return fail(ctx, ATS_ERR_CUDA, "context is poisoned by an earlier CUDA error: %s", ctx->err.c_str());
  if (need_placement && !ctx->placed)
    return fail(ctx, ATS_ERR_STATE, "no placement: call ats_set_placement or ats_plan_placement first");
  if (need_placement && !ctx->ws_reserved)
    return fail(ctx, ATS_ERR_NOMEM, "workspace_bytes must be at least %llu", (unsigned long long)kWsReserved);
  return ATS_OK;
}

// Look at the status word after a wait that the call makes anyway (mapped word: a plain read of pinned memory).
static int32_t check_status(ats_ctx* ctx) {
  if (!ctx->status_mapped) return ATS_OK;
  const int v = *reinterpret_cast<volatile int*>(ctx->host_status);
  if (v == 0) return ATS_OK;
  ctx->poisoned = true;
  if (v == 6 || v == 7)
    return fail(ctx, ATS_ERR_INVALID, "a kernel met an id out of range (status %d: %s); results are invalid", v,
                v == 6 ? "token id" : "expert id");
  return fail(ctx, ATS_ERR_TIMEOUT, "a kernel gave up a bounded wait (status %d); results are invalid", v);
}

static Tensor* get_tensor(ats_ctx* ctx, int32_t id, uint32_t fmt) {
  if (id < 0 || (size_t)id >= ctx->tensors.size()) return nullptr;
  Tensor* t = &ctx->tensors[id];
  return t->d.fmt == fmt ? t : nullptr;
}
// tensors that take part in placement: block-quantized or fp16 weight matrices
static bool placeable(const Tensor& t) { return t.d.fmt == ATS_FMT_Q4B32 || t.d.fmt == ATS_FMT_W16 || t.d.fmt == ATS_FMT_MXFP4; }
// the two 4-bit block formats share the slice layout and every kernel that reads it
static bool four_bit(const Tensor& t) { return t.d.fmt == ATS_FMT_Q4B32 || t.d.fmt == ATS_FMT_MXFP4; }
static Tensor* get_4bit(ats_ctx* ctx, int32_t id) {
  if (id < 0 || (size_t)id >= ctx->tensors.size()) return nullptr;
  Tensor* t = &ctx->tensors[id];
  return four_bit(*t) ? t : nullptr;
}
static Tensor* get_weight(ats_ctx* ctx, int32_t id) {
  if (id < 0 || (size_t)id >= ctx->tensors.size()) return nullptr;
  Tensor* t = &ctx->tensors[id];
  return placeable(*t) ? t : nullptr;
}

// ------------------------------------------------------------------------------------ streaming ring
// The per-call execution plan is the ordered list ctx->plan of slices to stream.  Copies are issued in plan order into
// ring slots taken round-robin; a slot is reused only after the consumer of its previous content has been enqueued on
// the compute stream (its `freed` event is then what the transfer stream waits for).

static void plan_begin(ats_ctx* ctx) {
  ctx->plan.clear();
  ctx->plan_next = 0;
}

static int plan_add(ats_ctx* ctx, int tensor, int expert) {
  Fetch f;
  f.tensor = tensor;
  f.expert = expert;
  ctx->plan.push_back(f);
  return (int)ctx->plan.size() - 1;
}

static int plan_find(const ats_ctx* ctx, int tensor, int expert) {
  for (size_t i = 0; i < ctx->plan.size(); ++i)
    if (ctx->plan[i].tensor == tensor && ctx->plan[i].expert == expert) return (int)i;
  return -1;
}

static int32_t pump(ats_ctx* ctx) {
  const uint32_t S = ctx->cfg.ring_slots;
  while (ctx->plan_next < ctx->plan.size()) {
    if (S == 0) return fail(ctx, ATS_ERR_BUDGET, "a host-placed tensor needs streaming but ring_slots is 0");
    RingSlot& slot = ctx->slots[ctx->next_slot];
    if (slot.busy) break;
    Fetch& f = ctx->plan[ctx->plan_next];
    const Tensor& t = ctx->tensors[f.tensor];
    if (t.slice_bytes > ctx->cfg.slot_bytes)
      return fail(ctx, ATS_ERR_BUDGET, "slice of tensor %d (%llu bytes) does not fit a ring slot (%llu bytes)", f.tensor,
                  (unsigned long long)t.slice_bytes, (unsigned long long)ctx->cfg.slot_bytes);
    if (slot.used) {
      ATS_CUDA(cudaStreamWaitEvent(ctx->ts, slot.freed, 0));
      ctx->stats.ring_reuses++;
    }
    uint8_t* dst = ctx->ring + (uint64_t)ctx->next_slot * ctx->slot_stride;
    const uint8_t* src = t.host + (uint64_t)f.expert * t.slice_stride;
    const uint64_t chunk = ctx->cfg.chunk_bytes ? ctx->cfg.chunk_bytes : t.slice_bytes;
    for (uint64_t off = 0; off < t.slice_bytes; off += chunk) {
      const uint64_t nb = std::min<uint64_t>(chunk, t.slice_bytes - off);
      if (ctx->fail_copies) {
        ctx->fail_copies--;
        ctx->poisoned = true;
        return fail(ctx, ATS_ERR_CUDA, "cudaMemcpyAsync failed (injected) while streaming tensor %d", f.tensor);
      }
      ATS_CUDA(cudaMemcpyAsync(dst + off, src + off, nb, cudaMemcpyHostToDevice, ctx->ts));
      ctx->stats.copies++;
    }
    ATS_CUDA(cudaEventRecord(slot.ready, ctx->ts));
    ctx->stats.streamed_bytes += t.slice_bytes;
    if (ctx->stats.n_streamed < ATS_STATS_LIST) {
      ctx->stats.streamed_ids[ctx->stats.n_streamed] = f.tensor;
      ctx->stats.streamed_experts[ctx->stats.n_streamed] = f.expert;
    }
    ctx->stats.n_streamed++;
    f.slot = (int)ctx->next_slot;
    f.enqueued = true;
    slot.busy = true;
    ctx->next_slot = (ctx->next_slot + 1) % S;
    ctx->plan_next++;
  }
  return ATS_OK;
}

// Make the compute stream wait for plan entry idx and return where its bytes land.
static int32_t acquire(ats_ctx* ctx, int idx, const uint8_t** out) {
  Fetch& f = ctx->plan[idx];
  if (!f.enqueued) {
    ATS_TRY(pump(ctx));
    if (!f.enqueued)
      return fail(ctx, ATS_ERR_BUDGET, "staging ring too small: %u slots cannot hold the slices one operator consumes together",
                  ctx->cfg.ring_slots);
  }
  if (!f.waited) {
    ATS_CUDA(cudaStreamWaitEvent(ctx->cs, ctx->slots[f.slot].ready, 0));
    f.waited = true;
  }
  *out = ctx->ring + (uint64_t)f.slot * ctx->slot_stride;
  return ATS_OK;
}

// The consumer of plan entry idx is on the compute stream: its slot may be refilled after it.
static int32_t release(ats_ctx* ctx, int idx) {
  Fetch& f = ctx->plan[idx];
  RingSlot& slot = ctx->slots[f.slot];
  if (ctx->cfg.flags & ATS_FLAG_POISON_SLOTS)
    ATS_CUDA(launch_fill(ctx->ring + (uint64_t)f.slot * ctx->slot_stride, ctx->slot_stride, 0xFF, ctx->cs,
                         &ctx->stats.kernel_launches));
  ATS_CUDA(cudaEventRecord(slot.freed, ctx->cs));
  slot.used = true;
  slot.busy = false;
  return pump(ctx);
}

// A dense tensor as a kernel operand: resident pointer, or a plan entry to acquire.
struct Operand {
  const Tensor* t = nullptr;
  int id = -1;
  int fetch = -1;  // plan index, -1 = resident
  const uint8_t* ptr = nullptr;
};

static void plan_dense(ats_ctx* ctx, int id, Operand* op) {
  op->id = id;
  op->t = &ctx->tensors[id];
  if (op->t->slices[0].where == ATS_GPU) {
    op->ptr = op->t->slices[0].dev;
    op->fetch = -1;
  } else {
    op->fetch = plan_add(ctx, id, 0);
  }
}

static int32_t acquire_ops(ats_ctx* ctx, Operand* ops, int n) {
  for (int i = 0; i < n; ++i)
    if (ops[i].fetch >= 0) ATS_TRY(acquire(ctx, ops[i].fetch, &ops[i].ptr));
  return ATS_OK;
}
static int32_t release_ops(ats_ctx* ctx, Operand* ops, int n) {
  for (int i = 0; i < n; ++i)
    if (ops[i].fetch >= 0) ATS_TRY(release(ctx, ops[i].fetch));
  return ATS_OK;
}
static int count_streamed(const Operand* ops, int n) {
  int c = 0;
  for (int i = 0; i < n; ++i) c += ops[i].fetch >= 0;
  return c;
}

// One GEMV: the streaming kernel where the shapes allow it (one row of a 4-bit format; two rows as two launches), else the
// fp16-weight kernel, the mma.sync kernel (4-bit formats, three to eight rows) or the generic kernel, preceded by a
// separate RMSNorm launch when a norm prologue was asked for.  Which kernel runs depends on format and shapes only, never on placement.
static int32_t launch_gemv_any(ats_ctx* ctx, GemvParams p) {
  p.pdl = (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1;
  p.dbg_wait_limit = ctx->dbg_wait_limit;
  p.dbg_withhold_tile_plus1 = ctx->dbg_withhold_plus1;
  if (gemv_stream_eligible(p)) {
    TimedLaunch tl(ctx, 0, gemv_work_bytes(p));
    ATS_CUDA(launch_gemv_stream(p, ctx->dev_status, ctx->sm_count, ctx->cs, &ctx->stats.kernel_launches));
    return ATS_OK;
  }
  if (p.M == 2 && !p.w16) {
    // Two rows: the single-row streaming kernel once per row is faster than the generic kernel over both (two launches at
    // about 8 us against one of 19 us for 14336 x 4096), and each row gets exactly the single-row result.
    GemvParams q = p;
    q.M = 1;
    if (gemv_stream_eligible(q)) {
      for (int r = 0; r < 2; ++r) {
        TimedLaunch tl(ctx, 0, gemv_work_bytes(q));
        ATS_CUDA(launch_gemv_stream(q, ctx->dev_status, ctx->sm_count, ctx->cs, &ctx->stats.kernel_launches));
        if (q.x) q.x += q.ldx;
        if (q.norm_x16) q.norm_x16 += q.K;
        if (q.norm_x32) q.norm_x32 += q.K;
        if (q.norm_out) q.norm_out += q.K;
        if (q.y32) q.y32 += q.ldy;
        if (q.y16) q.y16 += q.ldy;
        if (q.res32) q.res32 += q.ldres;
        if (q.res16) q.res16 += q.ldres;
      }
      return ATS_OK;
    }
  }
  if (p.norm_gain) {
    if (!p.norm_out) return fail(ctx, ATS_ERR_INVALID, "internal: norm prologue without an output buffer");
    ATS_CUDA(launch_rmsnorm(p.norm_x32 ? (const void*)p.norm_x32 : (const void*)p.norm_x16, p.norm_x32 != nullptr, p.norm_gain,
                            p.norm_out, p.M, p.K, p.norm_eps, ctx->cs, &ctx->stats.kernel_launches));
    p.x = p.norm_out;
    p.norm_gain = nullptr;
  }
  TimedLaunch tl(ctx, 0, gemv_work_bytes(p));
  if (p.w16)
    ATS_CUDA(launch_gemv_w16(p, ctx->cs, &ctx->stats.kernel_launches));
  else if (p.M >= 3 && gemv_mma_eligible(p))  // from three rows on the tensor-core form is the faster one (its cost does not grow with M)
    ATS_CUDA(launch_gemv_mma(p, ctx->cs, &ctx->stats.kernel_launches));
  else
    ATS_CUDA(launch_gemv(p, ctx->cs, &ctx->stats.kernel_launches));
  return ATS_OK;
}

// GEMV over 1..3 dense tensors whose outputs lie side by side.  When the ring cannot hold all streamed operands of
// the group at once the segments run one by one (same per-row arithmetic, so results do not depend on it).
static int32_t run_gemv_group(ats_ctx* ctx, Operand* ops, int n, GemvParams p) {
  p.K = (int)ops[0].t->d.k_in;
  p.w16 = ops[0].t->d.fmt == ATS_FMT_W16;  // a group shares one format (check_layer)
  p.mx = ops[0].t->d.fmt == ATS_FMT_MXFP4;
  if (count_streamed(ops, n) <= (int)ctx->cfg.ring_slots || n == 1) {
    ATS_TRY(acquire_ops(ctx, ops, n));
    p.n_seg = n;
    for (int i = 0; i < n; ++i) p.seg[i] = GemvSeg{ops[i].ptr, (int)ops[i].t->d.n_out};
    ATS_TRY(launch_gemv_any(ctx, p));
    return release_ops(ctx, ops, n);
  }
  if (p.mode == GEMV_SWIGLU_F16)
    return fail(ctx, ATS_ERR_BUDGET, "fused gate/up needs 2 ring slots when both tensors are host-placed");
  int row0 = 0;
  for (int i = 0; i < n; ++i) {
    ATS_TRY(acquire_ops(ctx, ops + i, 1));
    GemvParams q = p;
    q.n_seg = 1;
    q.seg[0] = GemvSeg{ops[i].ptr, (int)ops[i].t->d.n_out};
    if (q.y32) q.y32 += row0;
    if (q.y16) q.y16 += row0;
    if (q.res32) q.res32 += row0;
    if (q.res16) q.res16 += row0;
    ATS_TRY(launch_gemv_any(ctx, q));
    ATS_TRY(release_ops(ctx, ops + i, 1));
    row0 += (int)ops[i].t->d.n_out;
  }
  return ATS_OK;
}

static int32_t run_gemm_group(ats_ctx* ctx, Operand* ops, int n, GemmParams p) {
  p.K = (int)ops[0].t->d.k_in;
  p.status = ctx->dev_status;
  p.w16 = ops[0].t->d.fmt == ATS_FMT_W16;  // a group shares one format (check_layer)
  p.mx = ops[0].t->d.fmt == ATS_FMT_MXFP4;
  std::string err;
  // fp16 weight tiles come through one tensor map per matrix: such a group always runs matrix by matrix
  if ((count_streamed(ops, n) <= (int)ctx->cfg.ring_slots && !p.w16) || n == 1) {
    ATS_TRY(acquire_ops(ctx, ops, n));
    p.n_seg = n;
    uint64_t rows = 0;
    for (int i = 0; i < n; ++i) {
      p.seg[i] = GemvSeg{ops[i].ptr, (int)ops[i].t->d.n_out};
      rows += ops[i].t->d.n_out;
    }
    cudaError_t e;
    {
      TimedLaunch tl(ctx, 2, 2ull * (uint64_t)p.T * rows * (uint64_t)p.K);
      if (!(ctx->cfg.flags & ATS_FLAG_NO_GEMM_PAIR) && gemm_pair_eligible(p))
        e = launch_gemm_pair(p, ctx->cs, &ctx->stats.kernel_launches, &err);
      else
        e = launch_gemm(p, ctx->cs, &ctx->stats.kernel_launches, &err);
    }
    if (e != cudaSuccess) return check_cuda(ctx, e, err.empty() ? "launch_gemm" : err.c_str());
    return release_ops(ctx, ops, n);
  }
  int row0 = 0;
  for (int i = 0; i < n; ++i) {
    ATS_TRY(acquire_ops(ctx, ops + i, 1));
    GemmParams q = p;
    q.n_seg = 1;
    q.seg[0] = GemvSeg{ops[i].ptr, (int)ops[i].t->d.n_out};
    q.y += row0;
    cudaError_t e;
    {
      TimedLaunch tl(ctx, 2, 2ull * (uint64_t)q.T * (uint64_t)q.seg[0].n_rows * (uint64_t)q.K);
      if (!(ctx->cfg.flags & ATS_FLAG_NO_GEMM_PAIR) && gemm_pair_eligible(q))
        e = launch_gemm_pair(q, ctx->cs, &ctx->stats.kernel_launches, &err);
      else
        e = launch_gemm(q, ctx->cs, &ctx->stats.kernel_launches, &err);
    }
    if (e != cudaSuccess) return check_cuda(ctx, e, err.empty() ? "launch_gemm" : err.c_str());
    ATS_TRY(release_ops(ctx, ops + i, 1));
    row0 += (int)ops[i].t->d.n_out;
  }
  return ATS_OK;
}

// ------------------------------------------------------------------------------------ workspace
struct Bump {
  uint8_t* base;
  uint64_t cap, off = 0;
  bool ok = true;
  Bump(uint8_t* b, uint64_t c) : base(b), cap(c) {}
  void* take(uint64_t bytes) {
    const uint64_t o = align_up(off);
    off = o + bytes;
    if (off > cap) ok = false;
    return base ? base + o : nullptr;
  }
};

struct LayerWs {
  // decode
  __half* h16 = nullptr;
  float* qkv32 = nullptr;
  float* qrot32 = nullptr;
  float* attn_scratch = nullptr;
  __half* a16 = nullptr;
  float* x1_32 = nullptr;
  __half* h2_16 = nullptr;
  __half* act16 = nullptr;
  float* d32 = nullptr;
  int32_t* ids = nullptr;
  float* gates = nullptr;
  // prefill
  __half* qkv16 = nullptr;
  __half* qrot16 = nullptr;
  __half* o16 = nullptr;
  __half* x1_16 = nullptr;
  __half* gu16 = nullptr;
  __half* d16 = nullptr;
  void* gemm_scratch = nullptr;
  uint64_t gemm_scratch_bytes = 0;
  // MoE prefill: rows in expert order
  __half* xs16 = nullptr;
  int* order = nullptr;
  int* pos = nullptr;
  int* grp_off = nullptr;
  uint64_t total = 0;
  bool ok = true;
};

static LayerWs layout_decode(const ats_layer_desc& L, uint32_t M, uint8_t* base, uint64_t cap) {
  LayerWs w;
  Bump b(base, cap);
  b.take(kWsReserved);
  const uint64_t H = L.hidden, qd = (uint64_t)L.n_q_heads * L.head_dim, kvd = (uint64_t)L.n_kv_heads * L.head_dim;
  if (L.wq >= 0) {
    w.h16 = (__half*)b.take(M * H * 2);
    w.qkv32 = (float*)b.take(M * (qd + 2 * kvd) * 4);
    w.qrot32 = (float*)b.take(M * qd * 4);
    w.attn_scratch = (float*)b.take(attn_decode_scratch_floats((int)L.n_q_heads, (int)L.head_dim, (int)L.kv_capacity) * 4);
    w.a16 = (__half*)b.take(M * qd * 2);
    w.x1_32 = (float*)b.take(M * H * 4);
  }
  w.h2_16 = (__half*)b.take(M * H * 2);
  if (L.n_experts == 0) {
    w.act16 = (__half*)b.take((uint64_t)M * L.ffn * 2);
  } else {
    const uint64_t P = (uint64_t)M * L.top_k;
    w.act16 = (__half*)b.take(P * L.ffn * 2);
    w.d32 = (float*)b.take(P * H * 4);
    w.ids = (int32_t*)b.take(P * 4);
    w.gates = (float*)b.take(P * 4);
  }
  w.total = align_up(b.off);
  w.ok = b.ok;
  return w;
}

static LayerWs layout_prefill(const ats_layer_desc& L, uint32_t T, uint8_t* base, uint64_t cap) {
  LayerWs w;
  Bump b(base, cap);
  b.take(kWsReserved);
  const uint64_t H = L.hidden, qd = (uint64_t)L.n_q_heads * L.head_dim, kvd = (uint64_t)L.n_kv_heads * L.head_dim;
  uint64_t scratch = 0;
  if (L.wq >= 0) {
    w.h16 = (__half*)b.take(T * H * 2);
    w.qkv16 = (__half*)b.take(T * (qd + 2 * kvd) * 2);
    w.qrot16 = (__half*)b.take(T * qd * 2);
    w.a16 = (__half*)b.take(T * qd * 2);
    w.o16 = (__half*)b.take(T * H * 2);
    w.x1_16 = (__half*)b.take(T * H * 2);
    scratch = std::max(scratch, gemm_scratch_bytes((int)T, (int)(qd + 2 * kvd), (int)H));
    scratch = std::max(scratch, gemm_scratch_bytes((int)T, (int)H, (int)qd));
  }
  w.h2_16 = (__half*)b.take(T * H * 2);
  if (L.n_experts) {
    // every (token, slot) pair is a row of the expert GEMMs
    const uint64_t P = (uint64_t)T * L.top_k;
    w.ids = (int32_t*)b.take(P * 4);
    w.gates = (float*)b.take(P * 4);
    w.order = (int*)b.take(P * 4);
    w.pos = (int*)b.take(P * 4);
    w.grp_off = (int*)b.take(((uint64_t)L.n_experts + 1) * 4);
    w.xs16 = (__half*)b.take(P * H * 2);
    w.gu16 = (__half*)b.take(P * 2 * L.ffn * 2);
    w.act16 = (__half*)b.take(P * L.ffn * 2);
    w.d16 = (__half*)b.take(P * H * 2);
  } else {
    w.gu16 = (__half*)b.take((uint64_t)T * 2 * L.ffn * 2);
    w.act16 = (__half*)b.take((uint64_t)T * L.ffn * 2);
    w.d16 = (__half*)b.take(T * H * 2);
    scratch = std::max(scratch, gemm_scratch_bytes((int)T, (int)(2 * L.ffn), (int)H));
    scratch = std::max(scratch, gemm_scratch_bytes((int)T, (int)H, (int)L.ffn));
  }
  w.gemm_scratch = b.take(scratch);
  w.gemm_scratch_bytes = scratch;
  w.total = align_up(b.off);
  w.ok = b.ok;
  return w;
}

// ------------------------------------------------------------------------------------ placement
static int32_t apply_placement(ats_ctx* ctx) {
  // everything enqueued so far may still read the old resident region
  ATS_CUDA(cudaStreamSynchronize(ctx->cs));
  ATS_CUDA(cudaStreamSynchronize(ctx->ts));
  uint64_t off = 0, resident = 0, aux = 0;
  for (Tensor& t : ctx->tensors) {
    if (t.d.fmt == ATS_FMT_F16) {
      off = align_up(off) + t.host_bytes;
      aux += t.host_bytes;
      continue;
    }
    if (t.slices.size() > 1) off = align_up(off) + t.slices.size() * sizeof(uint8_t*);  // the slice address table
    for (Slice& s : t.slices)
      if (s.where == ATS_GPU) {
        off = align_up(off) + t.slice_stride;
        resident += t.slice_bytes;
      } else if (ctx->cfg.ring_slots == 0 || t.slice_bytes > ctx->cfg.slot_bytes) {
        return fail(ctx, ATS_ERR_BUDGET, "host-placed slice of %llu bytes cannot be streamed (ring_slots %u, slot_bytes %llu)",
                    (unsigned long long)t.slice_bytes, ctx->cfg.ring_slots, (unsigned long long)ctx->cfg.slot_bytes);
      }
  }
  if (off > ctx->resident_cap)
    return fail(ctx, ATS_ERR_BUDGET, "placement needs %llu resident bytes, arena has %llu after workspace and ring",
                (unsigned long long)off, (unsigned long long)ctx->resident_cap);
  off = 0;
  for (Tensor& t : ctx->tensors) {
    if (t.d.fmt == ATS_FMT_F16) {
      off = align_up(off);
      t.f16_dev = ctx->resident + off;
      ATS_CUDA(cudaMemcpyAsync(t.f16_dev, t.host, t.host_bytes, cudaMemcpyHostToDevice, ctx->ts));
      off += t.host_bytes;
      continue;
    }
    t.any_host = false;
    t.contiguous_dev = true;
    t.slice_tab_dev = nullptr;
    t.host_dev = nullptr;
    if (t.slices.size() > 1) {
      off = align_up(off);
      t.slice_tab_dev = reinterpret_cast<const uint8_t**>(ctx->resident + off);
      off += t.slices.size() * sizeof(uint8_t*);
    }
    uint8_t* prev = nullptr;
    for (size_t e = 0; e < t.slices.size(); ++e) {
      Slice& s = t.slices[e];
      if (s.where == ATS_GPU) {
        off = align_up(off);
        s.dev = ctx->resident + off;
        ATS_CUDA(cudaMemcpyAsync(s.dev, t.host + e * t.slice_stride, t.slice_bytes, cudaMemcpyHostToDevice, ctx->ts));
        off += t.slice_stride;
        if (prev && s.dev != prev + t.slice_stride) t.contiguous_dev = false;
        prev = s.dev;
      } else {
        s.dev = nullptr;
        t.any_host = true;
        t.contiguous_dev = false;
      }
    }
  }
  // slice address tables: the resident copy, or the slice inside the pinned host store at the address the device sees
  for (Tensor& t : ctx->tensors) {
    if (!t.slice_tab_dev) continue;
    void* host_dev = nullptr;
    if (cudaHostGetDevicePointer(&host_dev, t.host, 0) != cudaSuccess) {
      cudaGetLastError();
      t.slice_tab_dev = nullptr;  // the store is not mapped on this system: the ring path remains
      continue;
    }
    t.host_dev = static_cast<const uint8_t*>(host_dev);
    std::vector<const uint8_t*> tab(t.slices.size());
    for (size_t e = 0; e < t.slices.size(); ++e)
      tab[e] = t.slices[e].where == ATS_GPU ? t.slices[e].dev : static_cast<const uint8_t*>(host_dev) + e * t.slice_stride;
    ATS_CUDA(cudaMemcpyAsync(const_cast<uint8_t**>(t.slice_tab_dev), tab.data(), tab.size() * sizeof(uint8_t*), cudaMemcpyHostToDevice,
                             ctx->ts));
    ATS_CUDA(cudaStreamSynchronize(ctx->ts));  // `tab` is pageable and goes out of scope
  }
  ATS_CUDA(cudaStreamSynchronize(ctx->ts));
  ctx->stats.resident_bytes = resident;
  ctx->stats.aux_bytes = aux;
  for (RingSlot& s : ctx->slots) s.busy = false;
  ctx->placed = true;
  return ATS_OK;
}

// ------------------------------------------------------------------------------------ MoE stages
// One grouped GEMV stage over P = M*k (token, slot) pairs on stacked tensors t0 (and t1 for the fused SwiGLU stage).
// ids_host == null: every slice is resident and contiguous, the kernel indexes experts from device ids.
// Otherwise pairs on resident experts run first (overlapping the copies), then the streamed experts in ascending order
// in groups that fit the ring.
// One grouped-expert GEMV launch: the streaming kernel where the shapes allow it, else the generic one.
static cudaError_t launch_moe_gemv_any(ats_ctx* ctx, const MoeGemvParams& p, const MoeJobs* jobs) {
  if (moe_gemv_stream_eligible(p))
    return launch_moe_gemv_stream(p, jobs, ctx->dev_status, ctx->sm_count, (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1, ctx->cs,
                                  &ctx->stats.kernel_launches);
  return launch_moe_gemv(p, jobs, ctx->cs, &ctx->stats.kernel_launches);
}

static int32_t run_moe_stage(ats_ctx* ctx, int id0, int id1, const int32_t* ids_dev, const int32_t* ids_host,
                             MoeGemvParams p, const uint8_t* const* call_tab0 = nullptr, const uint8_t* const* call_tab1 = nullptr) {
  const Tensor& t0 = ctx->tensors[id0];
  const Tensor* t1 = id1 >= 0 ? &ctx->tensors[id1] : nullptr;
  p.n_rows = (int)t0.d.n_out;
  p.K = (int)t0.d.k_in;
  p.stride = t0.slice_stride;
  p.ids = ids_dev;
  p.mx = t0.d.fmt == ATS_FMT_MXFP4;
  p.n_experts = (int)t0.slices.size();
  p.status = ctx->dev_status;
  if (!ids_host) {
    if (call_tab0) {  // per-call tables: resident copies, or slices the copy kernel has gathered into the workspace
      p.tab0 = call_tab0;
      p.tab1 = call_tab1;
    } else if (t0.contiguous_dev && (!t1 || t1->contiguous_dev)) {
      p.base0 = t0.slices[0].dev;
      p.base1 = t1 ? t1->slices[0].dev : nullptr;
    } else {  // device-initiated gather: addresses from the per-tensor tables
      p.tab0 = t0.slice_tab_dev;
      p.tab1 = t1 ? t1->slice_tab_dev : nullptr;
    }
    TimedLaunch tl(ctx, 1, (uint64_t)p.P * ((t1 ? 2 : 1) * t0.slice_bytes + (uint64_t)p.K * 2 + (uint64_t)p.n_rows * 2));
    ATS_CUDA(launch_moe_gemv_any(ctx, p, nullptr));
    return ATS_OK;
  }
  const int P = p.P;
  MoeJobs jobs;
  jobs.n = 0;
  auto flush = [&]() -> int32_t {
    if (jobs.n == 0) return ATS_OK;
    TimedLaunch tl(ctx, 1, (uint64_t)jobs.n * ((t1 ? 2 : 1) * t0.slice_bytes + (uint64_t)p.K * 2 + (uint64_t)p.n_rows * 2));
    ATS_CUDA(launch_moe_gemv_any(ctx, p, &jobs));
    jobs.n = 0;
    return ATS_OK;
  };
  auto add_job = [&](int pair, const uint8_t* w0, const uint8_t* w1) -> int32_t {
    jobs.w0[jobs.n] = w0;
    jobs.w1[jobs.n] = w1;
    jobs.xrow[jobs.n] = (int16_t)(pair / p.x_div);
    jobs.orow[jobs.n] = (int16_t)pair;
    if (++jobs.n == kMoeJobsPerLaunch) return flush();
    return ATS_OK;
  };
  auto is_res = [&](int e) {
    return t0.slices[e].where == ATS_GPU && (!t1 || t1->slices[e].where == ATS_GPU);
  };
  // resident experts first
  for (int pr = 0; pr < P; ++pr) {
    const int e = ids_host[pr];
    if (is_res(e)) ATS_TRY(add_job(pr, t0.slices[e].dev, t1 ? t1->slices[e].dev : nullptr));
  }
  ATS_TRY(flush());
  // streamed experts, ascending, in groups whose slices fit the ring together
  std::vector<int> sel;
  for (int pr = 0; pr < P; ++pr)
    if (!is_res(ids_host[pr])) sel.push_back(ids_host[pr]);
  std::sort(sel.begin(), sel.end());
  sel.erase(std::unique(sel.begin(), sel.end()), sel.end());
  size_t i = 0;
  while (i < sel.size()) {
    std::vector<int> fetches;
    size_t j = i;
    int need = 0;
    while (j < sel.size()) {
      const int e = sel[j];
      const int n_e = (t0.slices[e].where == ATS_HOST) + (t1 && t1->slices[e].where == ATS_HOST);
      if (need + n_e > (int)ctx->cfg.ring_slots) break;
      need += n_e;
      ++j;
    }
    if (j == i) return fail(ctx, ATS_ERR_BUDGET, "staging ring too small for one expert's gate and up slices");
    for (size_t q = i; q < j; ++q) {
      const int e = sel[q];
      const uint8_t *w0 = t0.slices[e].dev, *w1 = t1 ? t1->slices[e].dev : nullptr;
      if (t0.slices[e].where == ATS_HOST) {
        const int f = plan_find(ctx, id0, e);
        ATS_TRY(acquire(ctx, f, &w0));
        fetches.push_back(f);
      }
      if (t1 && t1->slices[e].where == ATS_HOST) {
        const int f = plan_find(ctx, id1, e);
        ATS_TRY(acquire(ctx, f, &w1));
        fetches.push_back(f);
      }
      for (int pr = 0; pr < P; ++pr)
        if (ids_host[pr] == e) ATS_TRY(add_job(pr, w0, w1));
    }
    ATS_TRY(flush());
    for (int f : fetches) ATS_TRY(release(ctx, f));
    i = j;
  }
  return ATS_OK;
}

// Bring the routing ids to the host (the single host synchronisation of the MoE path) and validate them.
static int32_t fetch_ids(ats_ctx* ctx, const int32_t* ids_dev, int P, int E) {
  ATS_CUDA(cudaMemcpyAsync(ctx->ids_host, ids_dev, (size_t)P * 4, cudaMemcpyDeviceToHost, ctx->cs));
  ATS_CUDA(cudaEventRecord(ctx->ids_event, ctx->cs));
  ATS_CUDA(cudaEventSynchronize(ctx->ids_event));
  ctx->stats.host_syncs++;
  ATS_TRY(check_status(ctx));
  for (int i = 0; i < P; ++i)
    if (ctx->ids_host[i] < 0 || ctx->ids_host[i] >= E)
      return fail(ctx, ATS_ERR_INVALID, "routing id %d out of range [0,%d)", ctx->ids_host[i], E);
  return ATS_OK;
}

// Plan the streamed slices of an MoE stage set: for each selected expert (ascending) the host-placed gate and up
// slices, then the host-placed down slices (only selected experts move, Section 4.2.2).
static void plan_moe(ats_ctx* ctx, const int32_t* ids_host, int P, const int* tensor_ids, int n_first, int n_total) {
  std::vector<int> sel(ids_host, ids_host + P);
  std::sort(sel.begin(), sel.end());
  sel.erase(std::unique(sel.begin(), sel.end()), sel.end());
  for (int e : sel)
    for (int t = 0; t < n_first; ++t)
      if (ctx->tensors[tensor_ids[t]].slices[e].where == ATS_HOST) plan_add(ctx, tensor_ids[t], e);
  for (int t = n_first; t < n_total; ++t)
    for (int e : sel)
      if (ctx->tensors[tensor_ids[t]].slices[e].where == ATS_HOST) plan_add(ctx, tensor_ids[t], e);
}

// The device alias of [p, p + bytes) if it lies inside a registered host buffer, else null.
static const uint8_t* find_host_buffer(const ats_ctx* ctx, const void* p, uint64_t bytes) {
  const uint8_t* q = static_cast<const uint8_t*>(p);
  for (const ats_ctx::HostBuf& b : ctx->host_bufs)
    if (q >= b.host && q + bytes <= b.host + b.bytes) return b.dev + (q - b.host);
  return nullptr;
}

// (cos, sin) of pos * theta^(-2i/d) for i < d/2, formed in fp64 on the host and rounded to fp32.  The inverse
// frequencies are cached per (theta, d).
static void rope_table(ats_ctx* ctx, float theta, int d, int pos, float* cs) {
  const int half = d / 2;
  if (theta == 0.f) {
    for (int i = 0; i < half; ++i) {
      cs[2 * i] = 1.f;
      cs[2 * i + 1] = 0.f;
    }
    return;
  }
  if (ctx->rope_theta != theta || ctx->rope_d != d) {
    ctx->rope_inv.resize(half);
    for (int i = 0; i < half; ++i) ctx->rope_inv[i] = pow((double)theta, -2.0 * (double)i / (double)d);
    ctx->rope_theta = theta;
    ctx->rope_d = d;
  }
  for (int i = 0; i < half; ++i) {
    const double a = (double)pos * ctx->rope_inv[i];
    cs[2 * i] = (float)cos(a);
    cs[2 * i + 1] = (float)sin(a);
  }
}

}  // namespace ats

using namespace ats;

// ====================================================================================== C ABI
extern "C" {

int32_t ats_init(const ats_config* cfg, ats_ctx** out) {
  if (!cfg || !out) return ATS_ERR_INVALID;
  *out = nullptr;
  if (!cfg->arena || ((uintptr_t)cfg->arena % kAlign) != 0) return ATS_ERR_INVALID;
  if (cfg->compute_stream == cfg->transfer_stream) return ATS_ERR_INVALID;
  const uint64_t slot_stride = align_up(cfg->slot_bytes);
  const uint64_t ws = align_up(cfg->workspace_bytes);
  const uint64_t ring_bytes = (uint64_t)cfg->ring_slots * slot_stride;
  if (ws + ring_bytes > cfg->arena_bytes) return ATS_ERR_INVALID;
  if (cfg->ring_slots && cfg->slot_bytes == 0) return ATS_ERR_INVALID;
  if (cudaSetDevice(cfg->device) != cudaSuccess) return ATS_ERR_CUDA;
  ats_ctx* ctx = new (std::nothrow) ats_ctx();
  if (!ctx) return ATS_ERR_NOMEM;
  ctx->cfg = *cfg;
  ctx->cs = (cudaStream_t)cfg->compute_stream;
  ctx->ts = (cudaStream_t)cfg->transfer_stream;
  ctx->ws = (uint8_t*)cfg->arena;
  ctx->ring = ctx->ws + ws;
  ctx->slot_stride = slot_stride;
  ctx->resident = ctx->ring + ring_bytes;
  ctx->resident_cap = cfg->arena_bytes - ws - ring_bytes;
  ctx->slots.resize(cfg->ring_slots);
  bool ok = true;
  for (RingSlot& s : ctx->slots) {
    ok &= cudaEventCreateWithFlags(&s.ready, cudaEventDisableTiming) == cudaSuccess;
    ok &= cudaEventCreateWithFlags(&s.freed, cudaEventDisableTiming) == cudaSuccess;
  }
  ok &= cudaEventCreateWithFlags(&ctx->ids_event, cudaEventDisableTiming) == cudaSuccess;
  ok &= cudaEventCreateWithFlags(&ctx->sync_event, cudaEventDisableTiming) == cudaSuccess;
  ok &= cudaHostAlloc((void**)&ctx->ids_host, (3 * (size_t)kMaxPairs + 2048) * sizeof(int32_t), cudaHostAllocDefault) == cudaSuccess;
  ok &= cudaHostAlloc((void**)&ctx->host_status, 128, cudaHostAllocMapped) == cudaSuccess;
  ok &= cudaHostAlloc((void**)&ctx->stage_host, kStageHostBytes, cudaHostAllocDefault) == cudaSuccess;
  if (ws >= kWsReserved) {
    ctx->ws_reserved = true;
    ctx->dev_status = (int*)ctx->ws;
    ok &= cudaMemsetAsync(ctx->ws, 0, kWsReserved, ctx->cs) == cudaSuccess;
    ok &= cudaStreamSynchronize(ctx->cs) == cudaSuccess;
  }
  if (ok) {
    memset(ctx->host_status, 0, 128);
    void* alias = nullptr;
    if (cudaHostGetDevicePointer(&alias, ctx->host_status, 0) == cudaSuccess && alias) {
      ctx->dev_status = static_cast<int*>(alias);
      ctx->status_mapped = true;
      ctx->done_host = ctx->host_status + 16;  // its own 64-byte line
      ctx->done_dev = static_cast<int*>(alias) + 16;
    } else {
      cudaGetLastError();
    }
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess && sms > 0) ctx->sm_count = sms;
  if (!ok) {
    ats_destroy(ctx);
    return ATS_ERR_CUDA;
  }
  *out = ctx;
  return ATS_OK;
}

int32_t ats_destroy(ats_ctx* ctx) {
  if (!ctx) return ATS_ERR_INVALID;
  cudaStreamSynchronize(ctx->cs);
  cudaStreamSynchronize(ctx->ts);
  for (Tensor& t : ctx->tensors)
    if (t.host) cudaFreeHost(t.host);
  for (RingSlot& s : ctx->slots) {
    if (s.ready) cudaEventDestroy(s.ready);
    if (s.freed) cudaEventDestroy(s.freed);
  }
  for (cudaEvent_t e : ctx->tev) cudaEventDestroy(e);
  if (ctx->ids_event) cudaEventDestroy(ctx->ids_event);
  if (ctx->sync_event) cudaEventDestroy(ctx->sync_event);
  if (ctx->ids_host) cudaFreeHost(ctx->ids_host);
  if (ctx->stage_host) cudaFreeHost(ctx->stage_host);
  if (ctx->host_status) cudaFreeHost(ctx->host_status);
  delete ctx;
  return ATS_OK;
}

const char* ats_last_error(const ats_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int32_t ats_register_tensor(ats_ctx* ctx, const ats_tensor_desc* d, const void* codes, const void* scales,
                            int32_t* out_id) {
  ATS_TRY(precheck(ctx, false));
  if (!d || !codes || !out_id) return fail(ctx, ATS_ERR_INVALID, "null argument");
  if (d->fmt != ATS_FMT_Q4B32 && d->fmt != ATS_FMT_F16 && d->fmt != ATS_FMT_W16 && d->fmt != ATS_FMT_MXFP4)
    return fail(ctx, ATS_ERR_INVALID, "unknown format %u", d->fmt);
  if (d->n_out == 0 || d->k_in == 0 || d->n_experts == 0) return fail(ctx, ATS_ERR_SHAPE, "zero dimension");
  if (d->switch_cost < 0) return fail(ctx, ATS_ERR_INVALID, "switch_cost must be >= 0");
  Tensor t;
  t.d = *d;
  if (d->fmt == ATS_FMT_F16) {
    if (d->n_experts != 1) return fail(ctx, ATS_ERR_SHAPE, "F16 tensors are not stacked");
    t.host_bytes = (uint64_t)d->n_out * d->k_in * 2;
    if (cudaHostAlloc((void**)&t.host, t.host_bytes, cudaHostAllocDefault) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, ATS_ERR_NOMEM, "pinned allocation of %llu bytes failed", (unsigned long long)t.host_bytes);
    }
    memcpy(t.host, codes, t.host_bytes);
  } else if (d->fmt == ATS_FMT_W16) {
    if (d->n_experts != 1) return fail(ctx, ATS_ERR_SHAPE, "W16 tensors are not stacked");
    if (d->k_in % 8) return fail(ctx, ATS_ERR_SHAPE, "k_in = %u is not a multiple of 8", d->k_in);
    t.codes_bytes = (uint64_t)d->n_out * d->k_in * 2;
    t.slice_bytes = t.codes_bytes;
    t.slice_stride = align_up(t.slice_bytes);
    t.host_bytes = t.slice_stride;
    if (cudaHostAlloc((void**)&t.host, t.host_bytes, cudaHostAllocDefault) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, ATS_ERR_NOMEM, "pinned allocation of %llu bytes failed", (unsigned long long)t.host_bytes);
    }
    memcpy(t.host, codes, t.slice_bytes);
    if (t.slice_stride > t.slice_bytes) memset(t.host + t.slice_bytes, 0, t.slice_stride - t.slice_bytes);
    t.slices.resize(1);
    if (t.d.value < 0) t.d.value = (int64_t)t.slice_bytes;
  } else {
    if (d->k_in % kBlock) return fail(ctx, ATS_ERR_SHAPE, "k_in = %u is not a multiple of 32", d->k_in);
    if (!scales) return fail(ctx, ATS_ERR_INVALID, "null scales");
    const uint64_t N = d->n_out, K = d->k_in, E = d->n_experts;
    t.codes_bytes = N * K / 2;
    t.slice_bytes = t.codes_bytes + N * (K / kBlock) * 2;
    t.slice_stride = align_up(t.slice_bytes);
    t.host_bytes = E * t.slice_stride;
    const bool mx = d->fmt == ATS_FMT_MXFP4;
    if (mx) {
      // every weight must be an fp16 value (the tensor-core operand and the fp16 dequantized form): 0.5 * 2^e >= 2^-24
      // and 6 * 2^e <= 65504 give e = byte - 127 in [-23, 13]; 255 encodes "not a number"
      const uint8_t* s = (const uint8_t*)scales;
      const uint64_t ns = E * N * (K / kBlock);
      for (uint64_t i = 0; i < ns; ++i) {
        if (s[i] == 255) return fail(ctx, ATS_ERR_INVALID, "block scale %llu is NaN (byte 255)", (unsigned long long)i);
        if (s[i] < 104 || s[i] > 140)
          return fail(ctx, ATS_ERR_UNSUPPORTED, "block scale %llu has exponent %d: supported range is -23 .. 13", (unsigned long long)i,
                      (int)s[i] - 127);
      }
    } else if (!(ctx->cfg.flags & ATS_FLAG_SKIP_SCALE_CHECK)) {
      const uint16_t* s = (const uint16_t*)scales;
      const uint64_t ns = E * N * (K / kBlock);
      for (uint64_t i = 0; i < ns; ++i)
        if ((s[i] & 0x7C00u) == 0x7C00u) return fail(ctx, ATS_ERR_INVALID, "scale %llu is Inf or NaN", (unsigned long long)i);
    }
    if (cudaHostAlloc((void**)&t.host, t.host_bytes, cudaHostAllocDefault) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, ATS_ERR_NOMEM, "pinned allocation of %llu bytes failed", (unsigned long long)t.host_bytes);
    }
    for (uint64_t e = 0; e < E; ++e) {
      uint8_t* dst = t.host + e * t.slice_stride;
      if (mx)
        repack_mxfp4((const uint8_t*)codes + e * t.codes_bytes, (const uint8_t*)scales + e * N * (K / kBlock), dst, N, K);
      else
        repack_q4((const uint8_t*)codes + e * t.codes_bytes, (const uint16_t*)scales + e * N * (K / kBlock), dst, N, K);
      if (t.slice_stride > t.slice_bytes) memset(dst + t.slice_bytes, 0, t.slice_stride - t.slice_bytes);
    }
    t.slices.resize(E);
    if (t.d.value < 0) t.d.value = (int64_t)(E * t.slice_bytes);
  }
  ctx->stats.host_store_bytes += t.host_bytes;
  ctx->tensors.push_back(std::move(t));
  ctx->placed = false;
  *out_id = (int32_t)ctx->tensors.size() - 1;
  return ATS_OK;
}

int32_t ats_tensor_slice_bytes(const ats_ctx* ctx, int32_t id, uint64_t* out_bytes) {
  if (!ctx || !out_bytes || id < 0 || (size_t)id >= ctx->tensors.size()) return ATS_ERR_INVALID;
  const Tensor& t = ctx->tensors[id];
  *out_bytes = t.d.fmt == ATS_FMT_F16 ? t.host_bytes : t.slice_bytes;
  return ATS_OK;
}

int32_t ats_set_placement(ats_ctx* ctx, const int32_t* ids, const int32_t* experts, const uint8_t* where, uint32_t n) {
  ATS_TRY(precheck(ctx, false));
  if (n && (!ids || !where)) return fail(ctx, ATS_ERR_INVALID, "null argument");
  for (uint32_t i = 0; i < n; ++i) {
    Tensor* t = get_weight(ctx, ids[i]);
    if (!t) return fail(ctx, ATS_ERR_INVALID, "entry %u: id %d is not a registered weight tensor", i, ids[i]);
    const int32_t e = experts ? experts[i] : -1;
    if (e < -1 || e >= (int32_t)t->slices.size()) return fail(ctx, ATS_ERR_INVALID, "entry %u: expert %d out of range", i, e);
    if (where[i] != ATS_HOST && where[i] != ATS_GPU) return fail(ctx, ATS_ERR_INVALID, "entry %u: placement %u", i, where[i]);
  }
  for (Tensor& t : ctx->tensors)
    for (Slice& s : t.slices) s.where = ATS_HOST;
  for (uint32_t i = 0; i < n; ++i) {
    Tensor& t = ctx->tensors[ids[i]];
    const int32_t e = experts ? experts[i] : -1;
    if (e < 0)
      for (Slice& s : t.slices) s.where = where[i];
    else
      t.slices[e].where = where[i];
  }
  ctx->placed = false;
  return apply_placement(ctx);
}

int32_t ats_plan_placement(ats_ctx* ctx, uint64_t budget_bytes, uint32_t granule_bytes, uint8_t* out_where, uint32_t n) {
  ATS_TRY(precheck(ctx, false));
  const uint64_t G = granule_bytes ? granule_bytes : (1u << 20);
  std::vector<int64_t> s, r, c;
  std::vector<uint8_t> is_exp;
  std::vector<int> idx;
  for (size_t i = 0; i < ctx->tensors.size(); ++i) {
    const Tensor& t = ctx->tensors[i];
    if (!placeable(t)) continue;
    const uint64_t bytes = t.slice_bytes * t.slices.size();
    s.push_back((int64_t)((bytes + G - 1) / G));
    r.push_back(t.d.value);
    c.push_back(t.d.switch_cost);
    is_exp.push_back(t.slices.size() > 1);
    idx.push_back((int)i);
  }
  if (out_where && n != idx.size())
    return fail(ctx, ATS_ERR_INVALID, "out_where holds %u entries, %zu weight tensors are registered", n, idx.size());
  std::vector<uint8_t> b;
  static_placement(s, r, c, is_exp, (int64_t)(budget_bytes / G), &b);
  for (size_t j = 0; j < idx.size(); ++j)
    for (Slice& sl : ctx->tensors[idx[j]].slices) sl.where = b[j];
  if (out_where) memcpy(out_where, b.data(), b.size());
  ctx->placed = false;
  return apply_placement(ctx);
}

int32_t ats_get_placement(const ats_ctx* ctx, int32_t id, int32_t expert, uint8_t* out_where) {
  if (!ctx || !out_where) return ATS_ERR_INVALID;
  if (id < 0 || (size_t)id >= ctx->tensors.size()) return ATS_ERR_INVALID;
  const Tensor& t = ctx->tensors[id];
  if (t.d.fmt == ATS_FMT_F16) {
    *out_where = ATS_GPU;
    return ATS_OK;
  }
  if (expert < 0) expert = 0;
  if ((size_t)expert >= t.slices.size()) return ATS_ERR_INVALID;
  *out_where = t.slices[expert].where;
  return ATS_OK;
}

int32_t ats_linear(ats_ctx* ctx, int32_t id, const void* x, void* y, uint32_t M) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_weight(ctx, id);
  if (!t || t->slices.size() != 1) return fail(ctx, ATS_ERR_INVALID, "id %d is not a dense weight tensor", id);
  if (!x || !y) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  if (M == 0) return ATS_OK;
  plan_begin(ctx);
  Operand op;
  plan_dense(ctx, id, &op);
  ATS_TRY(pump(ctx));
  if (M <= 8) {
    GemvParams p{};
    p.M = (int)M;
    p.x = (const __half*)x;
    p.ldx = (int)t->d.k_in;
    p.y16 = (__half*)y;
    p.ldy = (int)t->d.n_out;
    p.mode = GEMV_OUT_F16;
    return run_gemv_group(ctx, &op, 1, p);
  }
  GemmParams g{};
  g.T = (int)M;
  g.x = (const __half*)x;
  g.ldx = (int)t->d.k_in;
  g.y = (__half*)y;
  g.ldy = (int)t->d.n_out;
  g.scratch_bytes = gemm_scratch_bytes((int)M, (int)t->d.n_out, (int)t->d.k_in);
  if (g.scratch_bytes + kWsReserved > align_up(ctx->cfg.workspace_bytes))
    return fail(ctx, ATS_ERR_NOMEM, "workspace too small for the GEMM: need %llu bytes",
                (unsigned long long)(g.scratch_bytes + kWsReserved));
  g.scratch = ctx->ws + kWsReserved;
  return run_gemm_group(ctx, &op, 1, g);
}

// Empirical performance density (Section 4.3.1): the measured time of one tensor's operator with the tensor resident and
// with the tensor placed on the host, from which the caller forms k_i = t_i / s_i and the residency benefit r_i.
int32_t ats_profile_tensor(ats_ctx* ctx, int32_t id, const void* x, void* y, uint32_t M, uint32_t iters, double* t_resident_us,
                           double* t_host_us) {
  ATS_TRY(precheck(ctx, false));
  Tensor* t = get_weight(ctx, id);
  if (!t || t->slices.size() != 1) return fail(ctx, ATS_ERR_INVALID, "id %d is not a dense weight tensor", id);
  if (!x || !y || !t_resident_us || !t_host_us || M == 0 || iters == 0) return fail(ctx, ATS_ERR_INVALID, "null pointer or zero count");
  // the placement in force is put back afterwards
  std::vector<uint8_t> saved;
  for (Tensor& u : ctx->tensors)
    for (Slice& sl : u.slices) saved.push_back(sl.where);
  const bool was_placed = ctx->placed;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  ATS_CUDA(cudaEventCreate(&e0));
  cudaError_t ce = cudaEventCreate(&e1);
  if (ce != cudaSuccess) {
    cudaEventDestroy(e0);
    return check_cuda(ctx, ce, "cudaEventCreate");
  }
  auto restore = [&]() -> int32_t {
    size_t k = 0;
    for (Tensor& u : ctx->tensors)
      for (Slice& sl : u.slices) sl.where = saved[k++];
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    ctx->placed = false;
    return was_placed ? apply_placement(ctx) : ATS_OK;
  };
  int32_t st = ATS_OK;
  for (int mode = 0; mode < 2 && st == ATS_OK; ++mode) {
    // this tensor alone decides: everything else sits on the host and is not touched
    for (Tensor& u : ctx->tensors)
      if (placeable(u))
        for (Slice& sl : u.slices) sl.where = ATS_HOST;
    t->slices[0].where = mode == 0 ? ATS_GPU : ATS_HOST;
    ctx->placed = false;
    st = apply_placement(ctx);
    for (uint32_t i = 0; i < 2 && st == ATS_OK; ++i) st = ats_linear(ctx, id, x, y, M);  // warm-up
    if (st != ATS_OK) break;
    if ((ce = cudaEventRecord(e0, ctx->cs)) != cudaSuccess) break;
    for (uint32_t i = 0; i < iters && st == ATS_OK; ++i) st = ats_linear(ctx, id, x, y, M);
    if (st != ATS_OK) break;
    if ((ce = cudaEventRecord(e1, ctx->cs)) != cudaSuccess) break;
    if ((ce = cudaEventSynchronize(e1)) != cudaSuccess) break;
    float ms = 0.f;
    if ((ce = cudaEventElapsedTime(&ms, e0, e1)) != cudaSuccess) break;
    *(mode == 0 ? t_resident_us : t_host_us) = (double)ms * 1e3 / iters;
  }
  if (ce != cudaSuccess) {
    restore();
    return check_cuda(ctx, ce, "ats_profile_tensor timing");
  }
  if (st != ATS_OK) {
    const std::string why = ctx->err;
    restore();
    ctx->err = why;
    return st;
  }
  return restore();
}

int32_t ats_set_tensor_value(ats_ctx* ctx, int32_t id, int64_t value, int64_t switch_cost) {
  ATS_TRY(precheck(ctx, false));
  Tensor* t = get_weight(ctx, id);
  if (!t) return fail(ctx, ATS_ERR_INVALID, "id %d is not a weight tensor", id);
  if (switch_cost < 0) return fail(ctx, ATS_ERR_INVALID, "switch_cost must be >= 0");
  t->d.value = value < 0 ? (int64_t)(t->slices.size() * t->slice_bytes) : value;
  t->d.switch_cost = switch_cost;
  return ATS_OK;
}

static int32_t check_f16(ats_ctx* ctx, int32_t id, uint32_t n_out, uint32_t k_in, const char* name);

int32_t ats_embed(ats_ctx* ctx, int32_t id, const int32_t* token_ids, uint32_t M, void* out) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_4bit(ctx, id);
  if (!t || t->slices.size() != 1) return fail(ctx, ATS_ERR_INVALID, "id %d is not a dense 4-bit tensor", id);
  if (!token_ids || !out) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  if (M == 0) return ATS_OK;
  const uint8_t* ptr = t->slices[0].dev;
  if (t->slices[0].where != ATS_GPU) {
    // a host-placed table: the rows are read where they are (a lookup touches a few kilobytes of a table of hundreds of
    // megabytes)
    if (!t->host_dev) {
      void* alias = nullptr;
      if (cudaHostGetDevicePointer(&alias, t->host, 0) != cudaSuccess) {
        cudaGetLastError();
        return fail(ctx, ATS_ERR_UNSUPPORTED, "host-placed embedding table: the pinned store is not mapped into the device");
      }
      t->host_dev = static_cast<const uint8_t*>(alias);
    }
    ptr = t->host_dev;
  }
  const int pdl = (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1;
  ATS_CUDA(launch_embed_rows(ptr, (int)t->d.n_out, (int)t->d.k_in, token_ids, (int)M, (__half*)out, ctx->dev_status, t->d.fmt == ATS_FMT_MXFP4, ctx->cs,
                             &ctx->stats.kernel_launches, pdl));
  return ATS_OK;
}

int32_t ats_lm_head(ats_ctx* ctx, int32_t norm_id, int32_t head_id, float eps, const void* x, void* logits, uint32_t M, void* scratch) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_weight(ctx, head_id);
  if (!t || t->slices.size() != 1) return fail(ctx, ATS_ERR_INVALID, "id %d is not a dense weight tensor", head_id);
  ATS_TRY(check_f16(ctx, norm_id, t->d.k_in, 1, "final norm"));
  if (!x || !logits) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  if (M == 0) return ATS_OK;
  const __half* gain = (const __half*)ctx->tensors[norm_id].f16_dev;
  const int K = (int)t->d.k_in, N = (int)t->d.n_out;
  if (M == 1) {
    GemvParams p{};
    p.M = 1;
    p.norm_x16 = (const __half*)x;
    p.norm_gain = gain;
    p.norm_eps = eps;
    p.norm_out = (__half*)scratch;
    p.x = (const __half*)scratch;  // used only when the norm runs as its own launch
    p.ldx = K;
    p.y16 = (__half*)logits;
    p.ldy = N;
    p.mode = GEMV_OUT_F16;
    GemvParams probe = p;
    probe.K = K;
    probe.n_seg = 1;
    probe.seg[0] = GemvSeg{nullptr, N};
    probe.w16 = t->d.fmt == ATS_FMT_W16;
    probe.mx = t->d.fmt == ATS_FMT_MXFP4;
    if (!scratch && !gemv_stream_eligible(probe))
      return fail(ctx, ATS_ERR_INVALID, "ats_lm_head needs `scratch` for this shape (the norm runs as a launch of its own)");
    plan_begin(ctx);
    Operand op;
    plan_dense(ctx, head_id, &op);
    ATS_TRY(pump(ctx));
    return run_gemv_group(ctx, &op, 1, p);
  }
  if (!scratch) return fail(ctx, ATS_ERR_INVALID, "ats_lm_head with M > 1 needs `scratch`");
  const int pdl = (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1;
  ATS_CUDA(launch_rmsnorm(x, 0, gain, (__half*)scratch, (int)M, K, eps, ctx->cs, &ctx->stats.kernel_launches, pdl));
  return ats_linear(ctx, head_id, scratch, logits, M);
}

int32_t ats_linear_static_scratch(ats_ctx* ctx, int32_t id, const void* x, void* y, uint32_t M) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_4bit(ctx, id);
  if (!t || t->slices.size() != 1) return fail(ctx, ATS_ERR_INVALID, "id %d is not a dense 4-bit tensor", id);
  if (!x || !y) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  if (t->slices[0].where != ATS_GPU)
    return fail(ctx, ATS_ERR_STATE, "tensor %d is host-placed: the no-allocation entry point only runs resident tensors", id);
  if (M == 0) return ATS_OK;
  plan_begin(ctx);
  Operand op;
  plan_dense(ctx, id, &op);
  if (M <= 8) {  // the GEMV needs no scratch at all
    GemvParams p{};
    p.M = (int)M;
    p.x = (const __half*)x;
    p.ldx = (int)t->d.k_in;
    p.y16 = (__half*)y;
    p.ldy = (int)t->d.n_out;
    p.mode = GEMV_OUT_F16;
    return run_gemv_group(ctx, &op, 1, p);
  }
  const uint64_t need = gemm_scratch_bytes((int)M, (int)t->d.n_out, (int)t->d.k_in);
  if (need > gemm_static_scratch_capacity())
    return fail(ctx, ATS_ERR_NOMEM, "split-K partials of %u x %u x %u need %llu bytes, the static scratch holds %llu", M, t->d.n_out,
                t->d.k_in, (unsigned long long)need, (unsigned long long)gemm_static_scratch_capacity());
  void* scratch = nullptr;
  ATS_CUDA(gemm_static_scratch(&scratch));
  GemmParams g{};
  g.T = (int)M;
  g.x = (const __half*)x;
  g.ldx = (int)t->d.k_in;
  g.y = (__half*)y;
  g.ldy = (int)t->d.n_out;
  g.scratch = scratch;
  g.scratch_bytes = gemm_static_scratch_capacity();
  return run_gemm_group(ctx, &op, 1, g);
}

int32_t ats_dequantize(ats_ctx* ctx, int32_t id, int32_t expert, void* out_dev, uint32_t out_fmt) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_4bit(ctx, id);
  if (!t) return fail(ctx, ATS_ERR_INVALID, "id %d is not a 4-bit tensor", id);
  if (expert < 0 || (size_t)expert >= t->slices.size()) return fail(ctx, ATS_ERR_INVALID, "expert %d out of range", expert);
  if (!out_dev || out_fmt > ATS_OUT_F16) return fail(ctx, ATS_ERR_INVALID, "bad output argument");
  plan_begin(ctx);
  const uint8_t* ptr = t->slices[expert].dev;
  int f = -1;
  if (t->slices[expert].where == ATS_HOST) {
    f = plan_add(ctx, id, expert);
    ATS_TRY(pump(ctx));
    ATS_TRY(acquire(ctx, f, &ptr));
  }
  ATS_CUDA(launch_dequant(ptr, (int)t->d.n_out, (int)t->d.k_in, out_dev, out_fmt == ATS_OUT_F16, t->d.fmt == ATS_FMT_MXFP4, ctx->cs,
                          &ctx->stats.kernel_launches));
  if (f >= 0) ATS_TRY(release(ctx, f));
  return ATS_OK;
}

int32_t ats_route_topk(ats_ctx* ctx, int32_t router_id, const void* h, uint32_t M, uint32_t k, int32_t* ids_dev,
                       float* gates_dev) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_tensor(ctx, router_id, ATS_FMT_F16);
  if (!t) return fail(ctx, ATS_ERR_INVALID, "id %d is not an F16 router tensor", router_id);
  if (!h || !ids_dev || !gates_dev) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  const uint32_t E = t->d.n_out;
  if (k == 0 || k > 32 || k > E || E > 1024) return fail(ctx, ATS_ERR_SHAPE, "top-k %u of %u experts unsupported", k, E);
  if (M == 0) return ATS_OK;
  ATS_CUDA(launch_router_topk((const __half*)h, (const __half*)t->f16_dev, (int)M, (int)t->d.k_in, (int)E, (int)k, 1,
                              ids_dev, gates_dev, ctx->cs, &ctx->stats.kernel_launches));
  return ATS_OK;
}

int32_t ats_moe_linear(ats_ctx* ctx, int32_t id, const void* x, const int32_t* ids_dev, void* y, uint32_t M, uint32_t k,
                       uint32_t x_per_slot) {
  ATS_TRY(precheck(ctx, true));
  Tensor* t = get_4bit(ctx, id);
  if (!t) return fail(ctx, ATS_ERR_INVALID, "id %d is not a 4-bit tensor", id);
  if (!x || !y || !ids_dev) return fail(ctx, ATS_ERR_INVALID, "null pointer");
  const uint32_t P = M * k;
  if (P == 0) return ATS_OK;
  if (P > 256) return fail(ctx, ATS_ERR_SHAPE, "M*k = %u exceeds 256", P);
  MoeGemvParams p{};
  p.P = (int)P;
  p.x_div = x_per_slot ? 1 : (int)k;
  p.x = (const __half*)x;
  p.ldx = (int)t->d.k_in;
  p.y16 = (__half*)y;
  p.ldy = (int)t->d.n_out;
  p.mode = GEMV_OUT_F16;
  plan_begin(ctx);
  const int32_t* ids_host = nullptr;
  if (t->any_host || !t->contiguous_dev) {
    ATS_TRY(fetch_ids(ctx, ids_dev, (int)P, (int)t->slices.size()));
    ids_host = ctx->ids_host;
    const int tid = id;
    plan_moe(ctx, ids_host, (int)P, &tid, 1, 1);
    ATS_TRY(pump(ctx));
  }
  return run_moe_stage(ctx, id, -1, ids_dev, ids_host, p);
}

// A layer's weight matrices share one format: Q4B32 (dense or stacked experts) or, for dense layers, fp16 (W16).
static int32_t check_q4(ats_ctx* ctx, int32_t id, uint32_t fmt, uint32_t n_out, uint32_t k_in, uint32_t n_experts, const char* name) {
  Tensor* t = get_tensor(ctx, id, fmt);
  if (!t)
    return fail(ctx, ATS_ERR_INVALID, "layer tensor %s (id %d) is not a registered %s tensor (a layer's weight matrices share one format)",
                name, id, fmt == ATS_FMT_W16 ? "W16" : fmt == ATS_FMT_MXFP4 ? "MXFP4" : "Q4B32");
  if (t->d.n_out != n_out || t->d.k_in != k_in || t->slices.size() != n_experts)
    return fail(ctx, ATS_ERR_SHAPE, "layer tensor %s is [%zu][%u][%u], the layer needs [%u][%u][%u]", name, t->slices.size(),
                t->d.n_out, t->d.k_in, n_experts, n_out, k_in);
  return ATS_OK;
}
static int32_t check_f16(ats_ctx* ctx, int32_t id, uint32_t n_out, uint32_t k_in, const char* name) {
  Tensor* t = get_tensor(ctx, id, ATS_FMT_F16);
  if (!t) return fail(ctx, ATS_ERR_INVALID, "layer tensor %s (id %d) is not a registered F16 tensor", name, id);
  if ((uint64_t)t->d.n_out * t->d.k_in != (uint64_t)n_out * k_in)
    return fail(ctx, ATS_ERR_SHAPE, "layer tensor %s has %u x %u elements, the layer needs %u x %u", name, t->d.k_in, t->d.n_out,
                k_in, n_out);
  return ATS_OK;
}

static int32_t check_layer(ats_ctx* ctx, const ats_layer_desc* L, bool prefill) {
  if (!L) return fail(ctx, ATS_ERR_INVALID, "null layer descriptor");
  if (L->hidden == 0 || L->ffn == 0) return fail(ctx, ATS_ERR_SHAPE, "zero hidden/ffn size");
  if (L->hidden % 32 || L->ffn % 32) return fail(ctx, ATS_ERR_SHAPE, "hidden and ffn must be multiples of 32");
  // the format of w_gate decides: every other matrix of the layer must have it too
  uint32_t fmt = ATS_FMT_Q4B32;
  if (Tensor* tg = get_weight(ctx, L->w_gate)) fmt = tg->d.fmt;
  if (fmt == ATS_FMT_W16 && L->n_experts) return fail(ctx, ATS_ERR_UNSUPPORTED, "MoE layers take 4-bit expert tensors");
  if (L->wq >= 0) {
    if (L->head_dim != 64 && L->head_dim != 128) return fail(ctx, ATS_ERR_UNSUPPORTED, "head_dim %u (64 or 128)", L->head_dim);
    if (L->n_kv_heads == 0 || L->n_q_heads % L->n_kv_heads) return fail(ctx, ATS_ERR_SHAPE, "n_q_heads %% n_kv_heads != 0");
    if (L->n_q_heads / L->n_kv_heads > 8) return fail(ctx, ATS_ERR_UNSUPPORTED, "more than 8 query heads per kv head");
    if (L->n_kv_heads > (uint32_t)kAttnMaxCounters) return fail(ctx, ATS_ERR_UNSUPPORTED, "more than %d kv heads", kAttnMaxCounters);
    const uint32_t qd = L->n_q_heads * L->head_dim, kvd = L->n_kv_heads * L->head_dim;
    ATS_TRY(check_f16(ctx, L->attn_norm, L->hidden, 1, "attn_norm"));
    ATS_TRY(check_q4(ctx, L->wq, fmt, qd, L->hidden, 1, "wq"));
    ATS_TRY(check_q4(ctx, L->wk, fmt, kvd, L->hidden, 1, "wk"));
    ATS_TRY(check_q4(ctx, L->wv, fmt, kvd, L->hidden, 1, "wv"));
    ATS_TRY(check_q4(ctx, L->wo, fmt, L->hidden, qd, 1, "wo"));
    if (L->kv_capacity == 0) return fail(ctx, ATS_ERR_SHAPE, "kv_capacity is 0");
    if (!prefill && (L->kv_capacity > 131072 || L->n_q_heads > 192))
      return fail(ctx, ATS_ERR_UNSUPPORTED, "decode attention supports kv_capacity <= 131072 and <= 192 query heads");
  }
  ATS_TRY(check_f16(ctx, L->ffn_norm, L->hidden, 1, "ffn_norm"));
  const uint32_t E = L->n_experts ? L->n_experts : 1;
  if (L->n_experts) {
    if (L->top_k == 0 || L->top_k > 32 || L->top_k > L->n_experts || L->n_experts > 1024)
      return fail(ctx, ATS_ERR_SHAPE, "top_k %u of %u experts unsupported", L->top_k, L->n_experts);
    ATS_TRY(check_f16(ctx, L->router, L->n_experts, L->hidden, "router"));
  }
  ATS_TRY(check_q4(ctx, L->w_gate, fmt, L->ffn, L->hidden, E, "w_gate"));
  ATS_TRY(check_q4(ctx, L->w_up, fmt, L->ffn, L->hidden, E, "w_up"));
  ATS_TRY(check_q4(ctx, L->w_down, fmt, L->hidden, L->ffn, E, "w_down"));
  return ATS_OK;
}

uint64_t ats_workspace_bytes(const ats_layer_desc* L, uint32_t max_tokens) {
  if (!L || max_tokens == 0) return 0;
  uint64_t need = layout_decode(*L, std::min<uint32_t>(max_tokens, 32), nullptr, ~0ull).total;
  need = std::max(need, layout_prefill(*L, max_tokens, nullptr, ~0ull).total);
  // staging rows of ats_layer_decode_host (input and output), each padded to the arena alignment
  need += 2 * align_up((uint64_t)std::min<uint32_t>(max_tokens, 32) * L->hidden * 2);
  return need + kAlign;
}

int32_t ats_layer_decode(ats_ctx* ctx, const ats_layer_desc* L, const void* x_in, void* x_out, void* k_cache,
                         void* v_cache, uint32_t pos, uint32_t M) {
  ATS_TRY(precheck(ctx, true));
  ATS_TRY(check_layer(ctx, L, false));
  if (!x_in || !x_out) return fail(ctx, ATS_ERR_INVALID, "null activation pointer");
  const bool attn = L->wq >= 0;
  if (M == 0) return ATS_OK;
  if (attn && M != 1) return fail(ctx, ATS_ERR_UNSUPPORTED, "decode with attention takes M = 1 (one sequence)");
  if (!attn && M > 32) return fail(ctx, ATS_ERR_SHAPE, "FFN-only decode takes M <= 32");
  if (L->n_experts == 0 && M > 8) return fail(ctx, ATS_ERR_SHAPE, "dense decode takes M <= 8");
  if (attn && (!k_cache || !v_cache)) return fail(ctx, ATS_ERR_INVALID, "null cache pointer");
  if (attn && pos >= L->kv_capacity) return fail(ctx, ATS_ERR_SHAPE, "pos %u >= kv_capacity %u", pos, L->kv_capacity);
  LayerWs w = layout_decode(*L, M, ctx->ws, align_up(ctx->cfg.workspace_bytes));
  if (!w.ok) return fail(ctx, ATS_ERR_NOMEM, "workspace too small: layer needs %llu bytes", (unsigned long long)w.total);
  uint64_t* nl = &ctx->stats.kernel_launches;
  const int H = (int)L->hidden, d = (int)L->head_dim, nq = (int)L->n_q_heads, nkv = (int)L->n_kv_heads;
  const int qd = nq * d, kvd = nkv * d;

  // the execution plan of this call: dense host-placed tensors in execution order
  plan_begin(ctx);
  Operand qkv[3], wo, gu[2], wd;
  if (attn) {
    plan_dense(ctx, L->wq, &qkv[0]);
    plan_dense(ctx, L->wk, &qkv[1]);
    plan_dense(ctx, L->wv, &qkv[2]);
    plan_dense(ctx, L->wo, &wo);
  }
  if (L->n_experts == 0) {
    plan_dense(ctx, L->w_gate, &gu[0]);
    plan_dense(ctx, L->w_up, &gu[1]);
    plan_dense(ctx, L->w_down, &wd);
  }
  ATS_TRY(pump(ctx));

  const int pdl = (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1;
  if (attn) {
    GemvParams p{};
    p.M = (int)M;
    p.norm_x16 = (const __half*)x_in;
    p.norm_gain = (const __half*)ctx->tensors[L->attn_norm].f16_dev;
    p.norm_eps = L->rms_eps;
    p.norm_out = w.h16;
    p.ldx = H;
    p.y32 = w.qkv32;
    p.ldy = qd + 2 * kvd;
    p.mode = GEMV_OUT_F32;
    const uint32_t skip = ctx->dbg_skip;
    if (!(skip & 1)) ATS_TRY(run_gemv_group(ctx, qkv, 3, p));
    AttnDecodeParams ap{};
    ap.qkv = w.qkv32;
    ap.q_rot_out = w.qrot32;
    ap.kc = (__half*)k_cache;
    ap.vc = (__half*)v_cache;
    ap.part = w.attn_scratch;
    ap.counters = reinterpret_cast<int*>(ctx->ws) + 64;
    ap.a16 = w.a16;
    ap.n_q = nq;
    ap.n_kv = nkv;
    ap.group = nq / nkv;
    ap.cap = (int)L->kv_capacity;
    ap.pos = (int)pos;
    rope_table(ctx, L->rope_theta, d, (int)pos, ap.cs);
    if (!(skip & 2)) ATS_CUDA(launch_attn_decode_fused(ap, d, pdl, ctx->cs, nl));
    GemvParams o{};
    o.M = (int)M;
    o.x = w.a16;
    o.ldx = qd;
    o.y32 = w.x1_32;
    o.ldy = H;
    o.res16 = (const __half*)x_in;
    o.ldres = H;
    o.mode = GEMV_RES16_OUT_F32;
    if (!(skip & 4)) ATS_TRY(run_gemv_group(ctx, &wo, 1, o));
  }
  if (L->n_experts == 0) {
    GemvParams g{};
    g.M = (int)M;
    if (attn) g.norm_x32 = w.x1_32; else g.norm_x16 = (const __half*)x_in;
    g.norm_gain = (const __half*)ctx->tensors[L->ffn_norm].f16_dev;
    g.norm_eps = L->rms_eps;
    g.norm_out = w.h2_16;
    g.ldx = H;
    g.y16 = w.act16;
    g.ldy = (int)L->ffn;
    g.mode = GEMV_SWIGLU_F16;
    if (count_streamed(gu, 2) > (int)ctx->cfg.ring_slots)
      return fail(ctx, ATS_ERR_BUDGET, "fused gate/up needs 2 ring slots when both tensors are host-placed");
    const uint32_t skip2 = ctx->dbg_skip;
    if (!(skip2 & 8)) ATS_TRY(run_gemv_group(ctx, gu, 2, g));
    GemvParams dn{};
    dn.M = (int)M;
    dn.x = w.act16;
    dn.ldx = (int)L->ffn;
    dn.y16 = (__half*)x_out;
    dn.ldy = H;
    dn.ldres = H;
    if (attn) {
      dn.res32 = w.x1_32;
      dn.mode = GEMV_RES32_OUT_F16;
    } else {
      dn.res16 = (const __half*)x_in;
      dn.mode = GEMV_RES16_OUT_F16;
    }
    if (skip2 & 16) return ATS_OK;
    return run_gemv_group(ctx, &wd, 1, dn);
  }
  // ---- MoE FFN
  const int k = (int)L->top_k, P = (int)M * k, E = (int)L->n_experts;
  // the FFN norm runs inside the router launch; the normalised rows land in h2_16 for the expert kernels
  const uint32_t mskip = ctx->dbg_skip;  // timing hook: 32 router, 64 gate/up stage, 128 down stage, 256 combine
  if (!(mskip & 32))
    ATS_CUDA(launch_router_topk_norm(w.h2_16, (const __half*)ctx->tensors[L->router].f16_dev, (int)M, H, E, k,
                                     (L->flags & ATS_LAYER_NO_TOPK_RENORM) ? 0 : 1, w.ids, w.gates, attn ? (const void*)w.x1_32 : x_in,
                                     attn ? 1 : 0, (const __half*)ctx->tensors[L->ffn_norm].f16_dev, L->rms_eps, ctx->cs, nl, pdl));
  const Tensor &tg = ctx->tensors[L->w_gate], &tu = ctx->tensors[L->w_up], &td = ctx->tensors[L->w_down];
  bool implicit = tg.contiguous_dev && tu.contiguous_dev && td.contiguous_dev;
  if (!implicit && M == 1 && !(ctx->cfg.flags & ATS_FLAG_MOE_RING_ONLY) && tg.slice_tab_dev && tu.slice_tab_dev && td.slice_tab_dev) {
    // the kernels find every selected slice themselves, in device memory or in the mapped host store: no ids on the
    // host, no ring (shapes the streaming kernel does not take keep the ring path).  One token only: its k experts are
    // distinct, so every host-placed slice crosses PCIe once; with several tokens, pairs that share an expert would each
    // read it again, and the ring path, which moves every distinct expert once, is the better one.
    MoeGemvParams probe1{}, probe2{};
    probe1.K = H; probe1.n_rows = (int)L->ffn; probe1.mode = GEMV_SWIGLU_F16;
    probe1.mx = probe2.mx = tg.d.fmt == ATS_FMT_MXFP4;
    probe2.K = (int)L->ffn; probe2.n_rows = H; probe2.mode = GEMV_OUT_F32;
    if (moe_gemv_stream_eligible(probe1) && moe_gemv_stream_eligible(probe2)) implicit = true;
  }
  const int32_t* ids_host = nullptr;
  const uint8_t* const* call_tab[3] = {nullptr, nullptr, nullptr};
  if (!implicit) {
    ATS_TRY(fetch_ids(ctx, w.ids, P, E));
    ids_host = ctx->ids_host;
    // Several tokens (unless ATS_FLAG_MOE_RING_ONLY): the distinct selected host-placed experts are gathered into the
    // workspace beyond this call's buffers by one launch of the copy kernel (every slice crosses PCIe once, no per-copy
    // cost), when that room exists and the streaming kernel takes the shapes; the stages then run as one launch each
    // over per-call address tables.  Otherwise: the staging ring.
    bool staged = false;
    if (!(ctx->cfg.flags & ATS_FLAG_MOE_RING_ONLY) && tg.host_dev && tu.host_dev && td.host_dev) {
      MoeGemvParams probe1{}, probe2{};
      probe1.K = H; probe1.n_rows = (int)L->ffn; probe1.mode = GEMV_SWIGLU_F16;
      probe1.mx = probe2.mx = tg.d.fmt == ATS_FMT_MXFP4;
    probe1.mx = probe2.mx = tg.d.fmt == ATS_FMT_MXFP4;
      probe2.K = (int)L->ffn; probe2.n_rows = H; probe2.mode = GEMV_OUT_F32;
      const Tensor* ts3[3] = {&tg, &tu, &td};
      std::vector<uint8_t> sel(E, 0);
      for (int pr = 0; pr < P; ++pr) sel[ids_host[pr]] = 1;
      uint64_t need = 0;
      int n_host = 0;
      for (const Tensor* t : ts3)
        for (int e = 0; e < E; ++e)
          if (sel[e] && t->slices[e].where != ATS_GPU) {
            need += t->slice_stride;
            ++n_host;
          }
      const uint64_t tab_bytes = align_up(3ull * E * sizeof(uint8_t*));
      const uint64_t list_bytes = align_up(((need + kCopyChunkBytes - 1) / kCopyChunkBytes + n_host) * sizeof(CopyChunk));
      const uint64_t room = align_up(ctx->cfg.workspace_bytes) - w.total;
      if (moe_gemv_stream_eligible(probe1) && moe_gemv_stream_eligible(probe2) && tab_bytes + list_bytes + need <= room &&
          tab_bytes + list_bytes <= kStageHostBytes) {
        uint8_t* dev_tab = ctx->ws + w.total;
        uint8_t* dev_list = dev_tab + tab_bytes;
        uint8_t* stage = dev_list + list_bytes;
        const uint8_t** tab_h = reinterpret_cast<const uint8_t**>(ctx->stage_host);
        CopyChunk* list_h = reinterpret_cast<CopyChunk*>(ctx->stage_host + tab_bytes);
        int nc = 0;
        uint64_t so = 0;
        for (int i = 0; i < 3; ++i) {
          const Tensor* t = ts3[i];
          for (int e = 0; e < E; ++e) {
            const Slice& sl = t->slices[e];
            if (sl.where == ATS_GPU) {
              tab_h[i * E + e] = sl.dev;
            } else if (sel[e]) {
              tab_h[i * E + e] = stage + so;
              const uint8_t* src = t->host_dev + (uint64_t)e * t->slice_stride;
              for (uint64_t o = 0; o < t->slice_stride; o += kCopyChunkBytes)
                list_h[nc++] = CopyChunk{src + o, stage + so + o, (uint32_t)std::min<uint64_t>(kCopyChunkBytes, t->slice_stride - o), 0};
              so += t->slice_stride;
            } else {
              tab_h[i * E + e] = t->host_dev + (uint64_t)e * t->slice_stride;  // not selected: never read
            }
          }
        }
        ATS_CUDA(cudaMemcpyAsync(dev_tab, ctx->stage_host, tab_bytes + (size_t)nc * sizeof(CopyChunk), cudaMemcpyHostToDevice, ctx->cs));
        ATS_CUDA(launch_host_gather(reinterpret_cast<const CopyChunk*>(dev_list), nc, ctx->dev_status, ctx->sm_count, ctx->cs, nl, pdl));
        for (int i = 0; i < 3; ++i) call_tab[i] = reinterpret_cast<const uint8_t* const*>(dev_tab) + (size_t)i * E;
        ctx->stats.streamed_bytes += need;
        staged = true;
        ids_host = nullptr;  // the stages take the ids on the device
      }
    }
    if (!staged) {
      const int tids[3] = {L->w_gate, L->w_up, L->w_down};
      plan_moe(ctx, ids_host, P, tids, 2, 3);
      ATS_TRY(pump(ctx));
    }
  }
  MoeGemvParams s1{};
  s1.P = P;
  s1.x_div = k;
  s1.x = w.h2_16;
  s1.ldx = H;
  s1.y16 = w.act16;
  s1.ldy = (int)L->ffn;
  s1.mode = GEMV_SWIGLU_F16;
  if (!(mskip & 64)) ATS_TRY(run_moe_stage(ctx, L->w_gate, L->w_up, w.ids, ids_host, s1, call_tab[0], call_tab[1]));
  MoeGemvParams s2{};
  s2.P = P;
  s2.x_div = 1;
  s2.x = w.act16;
  s2.ldx = (int)L->ffn;
  s2.y32 = w.d32;
  s2.ldy = H;
  s2.mode = GEMV_OUT_F32;
  if (!(mskip & 128)) ATS_TRY(run_moe_stage(ctx, L->w_down, -1, w.ids, ids_host, s2, call_tab[2], nullptr));
  if (!(mskip & 256))
    ATS_CUDA(launch_moe_combine(attn ? (const void*)w.x1_32 : x_in, attn ? 1 : 0, w.gates, w.d32, (__half*)x_out, (int)M, k, H,
                              ctx->cs, nl, pdl));
  return ATS_OK;
}

int32_t ats_layer_decode_host(ats_ctx* ctx, const ats_layer_desc* L, const void* x_in, void* x_out, void* k_cache,
                              void* v_cache, uint32_t pos, uint32_t M) {
  ATS_TRY(precheck(ctx, true));
  ATS_TRY(check_layer(ctx, L, false));
  if (!x_in || !x_out) return fail(ctx, ATS_ERR_INVALID, "null activation pointer");
  if (M == 0) return ATS_OK;
  if (M > 32) return fail(ctx, ATS_ERR_SHAPE, "decode takes M <= 32");
  // the staging rows sit behind everything the device call lays out in the workspace
  const LayerWs w = layout_decode(*L, M, nullptr, ~0ull);
  const uint64_t row_bytes = (uint64_t)M * L->hidden * 2, stage = align_up(row_bytes);
  const uint64_t need = w.total + 2 * stage;
  if (need > align_up(ctx->cfg.workspace_bytes))
    return fail(ctx, ATS_ERR_NOMEM, "workspace too small: host-driven decode needs %llu bytes", (unsigned long long)need);
  uint8_t* xin_dev = ctx->ws + w.total;
  uint8_t* xout_dev = xin_dev + stage;
  // Buffers the caller registered (pinned, mapped): the layer's last kernel writes the result row straight into the host
  // buffer (a few kilobytes of posted writes over PCIe) and the call returns when the device has written the completion
  // word, which costs less than the device-to-host copy and the wake-up from a stream wait.  The input row still goes
  // through the copy engine: fetching it with a small kernel was measured and is slower (58.3 against 54.7 us per step).
  const uint8_t* in_alias = find_host_buffer(ctx, x_in, row_bytes);
  uint8_t* out_alias = const_cast<uint8_t*>(find_host_buffer(ctx, x_out, row_bytes));
  const bool fast = in_alias && out_alias && ctx->done_dev && row_bytes % 16 == 0;
  ATS_CUDA(cudaMemcpyAsync(xin_dev, x_in, row_bytes, cudaMemcpyHostToDevice, ctx->cs));
  ATS_TRY(ats_layer_decode(ctx, L, xin_dev, fast ? (void*)out_alias : (void*)xout_dev, k_cache, v_cache, pos, M));
  if (fast) {
    // A one-thread kernel behind the layer writes the word.  (Letting the last CTA of the layer's last GEMV write it, after a
    // system-wide fence in every CTA, was measured and is slower: 57.8 against 54.9 us per step.)
    const int seq = ++ctx->done_seq;
    ATS_CUDA(launch_signal_done(ctx->done_dev, seq, (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1, ctx->cs, &ctx->stats.kernel_launches));
    // bounded poll (about two seconds), then the stream itself decides
    const auto t0 = std::chrono::steady_clock::now();
    uint32_t spins = 0;
    while (*ctx->done_host != seq) {
      if ((++spins & 0xFFFFu) == 0) {
        if (cudaStreamQuery(ctx->cs) != cudaErrorNotReady) break;  // finished (or failed) without the word: settle below
        if (std::chrono::steady_clock::now() - t0 > std::chrono::seconds(2)) break;
      }
    }
    if (*ctx->done_host != seq) ATS_CUDA(cudaStreamSynchronize(ctx->cs));
  } else {
    if (!fast) ATS_CUDA(cudaMemcpyAsync(x_out, xout_dev, row_bytes, cudaMemcpyDeviceToHost, ctx->cs));
    ATS_CUDA(cudaStreamSynchronize(ctx->cs));
  }
  return check_status(ctx);
}

int32_t ats_register_host_buffer(ats_ctx* ctx, void* ptr, uint64_t bytes) {
  ATS_TRY(precheck(ctx, false));
  if (!ptr || bytes == 0) return fail(ctx, ATS_ERR_INVALID, "null buffer");
  cudaPointerAttributes pa{};
  if (cudaPointerGetAttributes(&pa, ptr) != cudaSuccess || pa.type != cudaMemoryTypeHost || !pa.devicePointer ||
      (reinterpret_cast<uintptr_t>(pa.devicePointer) & 15) != 0) {
    cudaGetLastError();
    return fail(ctx, ATS_ERR_INVALID, "buffer %p is not pinned host memory the device can address (16-byte aligned)", ptr);
  }
  ats_unregister_host_buffer(ctx, ptr);
  ctx->host_bufs.push_back(ats_ctx::HostBuf{static_cast<const uint8_t*>(ptr), bytes, static_cast<uint8_t*>(pa.devicePointer)});
  return ATS_OK;
}

int32_t ats_unregister_host_buffer(ats_ctx* ctx, void* ptr) {
  if (!ctx) return ATS_ERR_INVALID;
  for (size_t i = 0; i < ctx->host_bufs.size(); ++i)
    if (ctx->host_bufs[i].host == ptr) {
      // nothing enqueued may still write through the alias
      cudaStreamSynchronize(ctx->cs);
      ctx->host_bufs.erase(ctx->host_bufs.begin() + (long)i);
      return ATS_OK;
    }
  return ATS_OK;
}

int32_t ats_layer_prefill(ats_ctx* ctx, const ats_layer_desc* L, const void* x_in, void* x_out, void* k_cache,
                          void* v_cache, uint32_t pos0, uint32_t T) {
  ATS_TRY(precheck(ctx, true));
  ATS_TRY(check_layer(ctx, L, true));
  if (!x_in || !x_out) return fail(ctx, ATS_ERR_INVALID, "null activation pointer");
  if (T == 0) return ATS_OK;
  const bool attn = L->wq >= 0;
  if (attn && (!k_cache || !v_cache)) return fail(ctx, ATS_ERR_INVALID, "null cache pointer");
  if (attn && (uint64_t)pos0 + T > L->kv_capacity)
    return fail(ctx, ATS_ERR_SHAPE, "pos0 + T = %llu exceeds kv_capacity %u", (unsigned long long)pos0 + T, L->kv_capacity);
  LayerWs w = layout_prefill(*L, T, ctx->ws, align_up(ctx->cfg.workspace_bytes));
  if (!w.ok) return fail(ctx, ATS_ERR_NOMEM, "workspace too small: prefill of %u tokens needs %llu bytes", T, (unsigned long long)w.total);
  uint64_t* nl = &ctx->stats.kernel_launches;
  const int H = (int)L->hidden, d = (int)L->head_dim, nq = (int)L->n_q_heads, nkv = (int)L->n_kv_heads;
  const int qd = nq * d, kvd = nkv * d;

  plan_begin(ctx);
  Operand qkv[3], wo, gu[2], wd;
  if (attn) {
    plan_dense(ctx, L->wq, &qkv[0]);
    plan_dense(ctx, L->wk, &qkv[1]);
    plan_dense(ctx, L->wv, &qkv[2]);
    plan_dense(ctx, L->wo, &wo);
  }
  const bool moe = L->n_experts != 0;
  if (moe) {
    if ((uint64_t)T * L->top_k > (uint64_t)kMaxPairs)
      return fail(ctx, ATS_ERR_SHAPE, "MoE prefill takes T * top_k <= %d pairs per call", kMaxPairs);
    for (int id : {L->w_gate, L->w_up, L->w_down}) {
      const Tensor& t = ctx->tensors[id];
      if (!t.contiguous_dev && !t.slice_tab_dev)
        return fail(ctx, ATS_ERR_UNSUPPORTED, "MoE prefill with host-placed experts needs the pinned store mapped into the device");
    }
  } else {
    plan_dense(ctx, L->w_gate, &gu[0]);
    plan_dense(ctx, L->w_up, &gu[1]);
    plan_dense(ctx, L->w_down, &wd);
  }
  ATS_TRY(pump(ctx));

  const int pdl = (ctx->cfg.flags & ATS_FLAG_NO_PDL) ? 0 : 1;
  GemmParams g{};
  g.T = (int)T;
  g.scratch = w.gemm_scratch;
  g.scratch_bytes = w.gemm_scratch_bytes;
  g.pdl = pdl;
  const __half* resid = (const __half*)x_in;
  if (attn) {
    ATS_CUDA(launch_rmsnorm(x_in, 0, (const __half*)ctx->tensors[L->attn_norm].f16_dev, w.h16, (int)T, H, L->rms_eps, ctx->cs, nl, pdl));
    g.x = w.h16;
    g.ldx = H;
    g.y = w.qkv16;
    g.ldy = qd + 2 * kvd;
    ATS_TRY(run_gemm_group(ctx, qkv, 3, g));
    ATS_CUDA(launch_rope_append_prefill(w.qkv16, qd + 2 * kvd, w.qrot16, (__half*)k_cache, (__half*)v_cache, (int)T, nq, nkv, d,
                                        (int)L->kv_capacity, (int)pos0, L->rope_theta, ctx->cs, nl, pdl));
    ATS_CUDA(launch_attn_prefill(w.qrot16, (const __half*)k_cache, (const __half*)v_cache, w.a16, (int)T, nq, nkv, d,
                                 (int)L->kv_capacity, (int)pos0, ctx->cs, nl, pdl));
    g.x = w.a16;
    g.ldx = qd;
    g.y = w.o16;
    g.ldy = H;
    g.res = (const __half*)x_in;  // x1 = rn16(x + o) in the GEMM's own epilogue (or its split-K reduction)
    g.y2 = w.x1_16;
    ATS_TRY(run_gemm_group(ctx, &wo, 1, g));
    g.res = nullptr;
    g.y2 = nullptr;
    resid = w.x1_16;
  }
  ATS_CUDA(launch_rmsnorm(resid, 0, (const __half*)ctx->tensors[L->ffn_norm].f16_dev, w.h2_16, (int)T, H, L->rms_eps, ctx->cs, nl, pdl));
  if (moe) {
    // Routed FFN over T tokens: every (token, slot) pair becomes a row; rows are sorted by expert so that each expert's
    // rows are one contiguous block of a grouped GEMM (one launch for all experts).  The sort runs on the host from the
    // routing ids (one synchronisation per call); expert slices are read where they are: resident copies, or the pinned
    // host store through its device mapping for host-placed experts (every slice is read once per 128 of its rows).
    const int k = (int)L->top_k, E = (int)L->n_experts, P = (int)T * k, F = (int)L->ffn;
    ATS_CUDA(launch_router_topk(w.h2_16, (const __half*)ctx->tensors[L->router].f16_dev, (int)T, H, E, k,
                                (L->flags & ATS_LAYER_NO_TOPK_RENORM) ? 0 : 1, w.ids, w.gates, ctx->cs, nl, pdl));
    ATS_TRY(fetch_ids(ctx, w.ids, P, E));
    int32_t* order_h = ctx->ids_host + kMaxPairs;       // sorted position -> pair
    int32_t* pos_h = ctx->ids_host + 2 * kMaxPairs;     // pair -> sorted position
    int32_t* off_h = ctx->ids_host + 3 * kMaxPairs;     // expert -> first sorted position; [E] = P
    int max_rows = 0;
    if (ats_host_group_pairs(ctx->ids_host, (uint32_t)P, (uint32_t)E, order_h, pos_h, off_h, &max_rows) != ATS_OK)
      return fail(ctx, ATS_ERR_INVALID, "routing ids out of range");
    ATS_CUDA(cudaMemcpyAsync(w.order, order_h, (size_t)P * 4, cudaMemcpyHostToDevice, ctx->cs));
    ATS_CUDA(cudaMemcpyAsync(w.pos, pos_h, (size_t)P * 4, cudaMemcpyHostToDevice, ctx->cs));
    ATS_CUDA(cudaMemcpyAsync(w.grp_off, off_h, (size_t)(E + 1) * 4, cudaMemcpyHostToDevice, ctx->cs));
    ATS_CUDA(launch_moe_gather_rows(w.h2_16, w.order, k, w.xs16, P, H, ctx->cs, nl, pdl));
    const Tensor &tg = ctx->tensors[L->w_gate], &tu = ctx->tensors[L->w_up], &td = ctx->tensors[L->w_down];
    auto slice0 = [](const Tensor& t) -> const uint8_t* { return t.contiguous_dev ? t.slices[0].dev : nullptr; };
    // Host-placed experts that some token selected: one SM-driven gather brings their slices into what the workspace has
    // left beyond this layer's buffers, and per-call address tables point the GEMMs there.  Without that room (or
    // without a mapped store) the GEMMs read the slices in place through the per-tensor tables (slower: 32-byte reads).
    const uint8_t* const* call_tab[3] = {nullptr, nullptr, nullptr};
    {
      const Tensor* ts3[3] = {&tg, &tu, &td};
      uint64_t need = 0;
      int n_host = 0;
      for (const Tensor* t : ts3)
        if (!t->contiguous_dev && t->host_dev)
          for (int e = 0; e < E; ++e)
            if (off_h[e + 1] > off_h[e] && t->slices[e].where != ATS_GPU) {
              need += t->slice_stride;
              ++n_host;
            }
      const uint64_t tab_bytes = align_up(3ull * E * sizeof(uint8_t*));
      const uint64_t n_chunks = n_host ? (need + kCopyChunkBytes - 1) / kCopyChunkBytes + n_host : 0;
      const uint64_t list_bytes = align_up(n_chunks * sizeof(CopyChunk));
      const uint64_t room = align_up(ctx->cfg.workspace_bytes) - w.total;
      if (n_host && tab_bytes + list_bytes + need <= room && tab_bytes + list_bytes <= kStageHostBytes) {
        uint8_t* dev_tab = ctx->ws + w.total;
        uint8_t* dev_list = dev_tab + tab_bytes;
        uint8_t* stage = dev_list + list_bytes;
        const uint8_t** tab_h = reinterpret_cast<const uint8_t**>(ctx->stage_host);
        CopyChunk* list_h = reinterpret_cast<CopyChunk*>(ctx->stage_host + tab_bytes);
        int nc = 0;
        uint64_t so = 0;
        for (int i = 0; i < 3; ++i) {
          const Tensor* t = ts3[i];
          for (int e = 0; e < E; ++e) {
            const Slice& sl = t->slices[e];
            if (sl.where == ATS_GPU) {
              tab_h[i * E + e] = sl.dev;
            } else if (off_h[e + 1] > off_h[e] && t->host_dev) {
              tab_h[i * E + e] = stage + so;
              const uint8_t* src = t->host_dev + (uint64_t)e * t->slice_stride;
              for (uint64_t o = 0; o < t->slice_stride; o += kCopyChunkBytes)
                list_h[nc++] = CopyChunk{src + o, stage + so + o, (uint32_t)std::min<uint64_t>(kCopyChunkBytes, t->slice_stride - o), 0};
              so += t->slice_stride;
            } else {
              tab_h[i * E + e] = t->host_dev ? t->host_dev + (uint64_t)e * t->slice_stride : nullptr;  // no rows: never read
            }
          }
        }
        ATS_CUDA(cudaMemcpyAsync(dev_tab, ctx->stage_host, tab_bytes + (size_t)nc * sizeof(CopyChunk), cudaMemcpyHostToDevice, ctx->cs));
        ATS_CUDA(launch_host_gather(reinterpret_cast<const CopyChunk*>(dev_list), nc, ctx->dev_status, ctx->sm_count, ctx->cs, nl, pdl));
        for (int i = 0; i < 3; ++i) call_tab[i] = reinterpret_cast<const uint8_t* const*>(dev_tab) + (size_t)i * E;
        ctx->stats.streamed_bytes += need;
      }
    }
    std::string err;
    GemmParams m{};
    m.T = P;
    m.pdl = pdl;
    m.status = ctx->dev_status;
    m.grp_off = w.grp_off;
    m.n_groups = E;
    m.grp_max_rows = max_rows;
    m.mx = tg.d.fmt == ATS_FMT_MXFP4;
    // gate | up side by side
    m.n_seg = 2;
    m.K = H;
    m.seg[0] = GemvSeg{slice0(tg), F};
    m.seg[1] = GemvSeg{slice0(tu), F};
    m.grp_stride = tg.slice_stride;
    m.grp_tab[0] = call_tab[0] ? call_tab[0] : tg.contiguous_dev ? nullptr : tg.slice_tab_dev;
    m.grp_tab[1] = call_tab[1] ? call_tab[1] : tu.contiguous_dev ? nullptr : tu.slice_tab_dev;
    m.x = w.xs16;
    m.ldx = H;
    m.y = w.gu16;
    m.ldy = 2 * F;
    cudaError_t ce = launch_gemm(m, ctx->cs, nl, &err);
    if (ce != cudaSuccess) return check_cuda(ctx, ce, err.empty() ? "launch_gemm (expert gate/up)" : err.c_str());
    ATS_CUDA(launch_swiglu16(w.gu16, 2 * F, F, w.act16, P, ctx->cs, nl, pdl));
    m.n_seg = 1;
    m.K = F;
    m.seg[0] = GemvSeg{slice0(td), H};
    m.grp_stride = td.slice_stride;
    m.grp_tab[0] = call_tab[2] ? call_tab[2] : td.contiguous_dev ? nullptr : td.slice_tab_dev;
    m.grp_tab[1] = nullptr;
    m.x = w.act16;
    m.ldx = F;
    m.y = w.d16;
    m.ldy = H;
    ce = launch_gemm(m, ctx->cs, nl, &err);
    if (ce != cudaSuccess) return check_cuda(ctx, ce, err.empty() ? "launch_gemm (expert down)" : err.c_str());
    ATS_CUDA(launch_moe_combine_sorted(resid, w.gates, w.d16, w.pos, (__half*)x_out, (int)T, k, H, ctx->cs, nl, pdl));
    return ATS_OK;
  }
  g.x = w.h2_16;
  g.ldx = H;
  g.y = w.gu16;
  g.ldy = 2 * (int)L->ffn;
  ATS_TRY(run_gemm_group(ctx, gu, 2, g));
  ATS_CUDA(launch_swiglu16(w.gu16, 2 * (int)L->ffn, (int)L->ffn, w.act16, (int)T, ctx->cs, nl, pdl));
  g.x = w.act16;
  g.ldx = (int)L->ffn;
  g.y = w.d16;
  g.ldy = H;
  g.res = resid;  // y = rn16(x1 + d)
  g.y2 = (__half*)x_out;
  ATS_TRY(run_gemm_group(ctx, &wd, 1, g));
  return ATS_OK;
}

int32_t ats_get_numerics(const ats_ctx* ctx, uint32_t mode, uint32_t* fp16_edge_mask, uint32_t* weight_mode) {
  if (!ctx || !fp16_edge_mask || !weight_mode) return ATS_ERR_INVALID;
  // edge bits: h=0 q=1 k=2 v=3 q_rot=4 a=5 o=6 x1=7 h2=8 g=9 u=10 act=11 d=12
  if (mode == ATS_MODE_DECODE) {
    *fp16_edge_mask = (1u << 0) | (1u << 5) | (1u << 8) | (1u << 11);  // the GEMV inputs h, a, h2, act
    *weight_mode = 0;
  } else if (mode == ATS_MODE_PREFILL) {
    *fp16_edge_mask = (1u << 13) - 1;  // every intermediate is stored as fp16
    *weight_mode = 1;
  } else {
    return ATS_ERR_INVALID;
  }
  return ATS_OK;
}

int32_t ats_get_stats(ats_ctx* ctx, ats_stats* out) {
  if (!ctx || !out) return ATS_ERR_INVALID;
  for (int f = 0; f < 3; ++f) ctx->stats.timed_ms[f] = 0.0;
  for (size_t i = 0; i + 1 < ctx->tev_used; i += 2) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->tev[i], ctx->tev[i + 1]) == cudaSuccess)
      ctx->stats.timed_ms[ctx->tev_family[i / 2]] += ms;
    else
      cudaGetLastError();  // launch not finished yet: not counted
  }
  *out = ctx->stats;
  return ATS_OK;
}

int32_t ats_set_flags(ats_ctx* ctx, uint32_t flags) {
  if (!ctx) return ATS_ERR_INVALID;
  ctx->cfg.flags = flags;
  return ATS_OK;
}

int32_t ats_reset_stats(ats_ctx* ctx) {
  if (!ctx) return ATS_ERR_INVALID;
  ats_stats& s = ctx->stats;
  s.streamed_bytes = s.copies = s.kernel_launches = s.ring_reuses = s.host_syncs = 0;
  s.n_streamed = 0;
  for (int f = 0; f < 3; ++f) {
    s.timed_launches[f] = s.timed_work[f] = 0;
    s.timed_ms[f] = 0.0;
  }
  ctx->tev_used = 0;
  return ATS_OK;
}

int32_t ats_sync(ats_ctx* ctx, uint32_t timeout_ms) {
  if (!ctx) return ATS_ERR_INVALID;
  if (ctx->poisoned) return fail(ctx, ATS_ERR_CUDA, "context is poisoned: %s", std::string(ctx->err).c_str());
  const auto t0 = std::chrono::steady_clock::now();
  cudaStream_t streams[2] = {ctx->ts, ctx->cs};
  for (cudaStream_t st : streams) {
    ATS_CUDA(cudaEventRecord(ctx->sync_event, st));
    // short waits (a decode step) are polled without yielding the core: a sleep costs more than the step; after a
    // millisecond the wait backs off to sleeping polls
    for (uint32_t polls = 0;; ++polls) {
      cudaError_t e = cudaEventQuery(ctx->sync_event);
      if (e == cudaSuccess) break;
      if (e != cudaErrorNotReady) return check_cuda(ctx, e, "ats_sync");
      if ((polls & 63u) != 63u) continue;
      const auto us = std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now() - t0).count();
      if (timeout_ms && us >= 1000ll * (long long)timeout_ms)
        return fail(ctx, ATS_ERR_TIMEOUT, "ats_sync: still running after %u ms", timeout_ms);
      if (us > 1000) std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return check_cuda(ctx, e, "asynchronous error");
  if (ctx->status_mapped) return check_status(ctx);
  if (ctx->dev_status) {
    ATS_CUDA(cudaMemcpyAsync(ctx->host_status, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->cs));
    ATS_CUDA(cudaStreamSynchronize(ctx->cs));
    if (*ctx->host_status != 0) {
      ctx->poisoned = true;
      return fail(ctx, ATS_ERR_TIMEOUT, "a kernel raised the status word (%d); results are invalid", *ctx->host_status);
    }
  }
  return ATS_OK;
}

int32_t ats_measure_h2d(ats_ctx* ctx, uint64_t bytes, uint32_t reps, double* out_gbs) {
  ATS_TRY(precheck(ctx, false));
  if (!out_gbs || bytes == 0 || reps == 0) return fail(ctx, ATS_ERR_INVALID, "bad argument");
  const uint64_t ring_bytes = (uint64_t)ctx->cfg.ring_slots * ctx->slot_stride;
  if (bytes > ring_bytes) return fail(ctx, ATS_ERR_BUDGET, "%llu bytes exceed the ring (%llu)", (unsigned long long)bytes, (unsigned long long)ring_bytes);
  ATS_CUDA(cudaStreamSynchronize(ctx->cs));
  ATS_CUDA(cudaStreamSynchronize(ctx->ts));
  void* hbuf = nullptr;
  if (cudaHostAlloc(&hbuf, bytes, cudaHostAllocDefault) != cudaSuccess) {
    cudaGetLastError();
    return fail(ctx, ATS_ERR_NOMEM, "pinned allocation of %llu bytes failed", (unsigned long long)bytes);
  }
  memset(hbuf, 1, bytes);
  cudaEvent_t a, b;
  cudaEventCreate(&a);
  cudaEventCreate(&b);
  float best = 1e30f;
  int32_t st = ATS_OK;
  for (uint32_t r = 0; r < reps && st == ATS_OK; ++r) {
    cudaEventRecord(a, ctx->ts);
    cudaError_t e = cudaMemcpyAsync(ctx->ring, hbuf, bytes, cudaMemcpyHostToDevice, ctx->ts);
    cudaEventRecord(b, ctx->ts);
    if (e == cudaSuccess) e = cudaEventSynchronize(b);
    st = check_cuda(ctx, e, "ats_measure_h2d copy");
    float ms = 0;
    if (st == ATS_OK && cudaEventElapsedTime(&ms, a, b) == cudaSuccess && ms > 0) best = std::min(best, ms);
  }
  cudaEventDestroy(a);
  cudaEventDestroy(b);
  cudaFreeHost(hbuf);
  if (st != ATS_OK) return st;
  *out_gbs = (double)bytes / (best * 1e-3) / 1e9;
  return ATS_OK;
}

int32_t ats_measure_hbm_read(ats_ctx* ctx, uint64_t bytes, uint32_t reps, double* out_gbs) {
  ATS_TRY(precheck(ctx, false));
  if (!out_gbs || reps == 0) return fail(ctx, ATS_ERR_INVALID, "bad argument");
  bytes = std::min<uint64_t>(bytes, ctx->cfg.arena_bytes) / (16 * 1024) * (16 * 1024);
  if (bytes < (256ull << 20))
    return fail(ctx, ATS_ERR_BUDGET, "the probe reads at least 256 MiB of the arena (twice the L2), the arena holds %llu bytes",
                (unsigned long long)ctx->cfg.arena_bytes);
  ATS_CUDA(cudaStreamSynchronize(ctx->cs));
  cudaEvent_t a = nullptr, b = nullptr;
  ATS_CUDA(cudaEventCreate(&a));
  cudaError_t e = cudaEventCreate(&b);
  float best = 1e30f;
  for (uint32_t r = 0; r < reps + 1 && e == cudaSuccess; ++r) {  // the first pass warms up
    cudaEventRecord(a, ctx->cs);
    e = launch_hbm_read_probe(static_cast<const uint8_t*>(ctx->cfg.arena), bytes, ctx->dev_status, ctx->sm_count, ctx->cs);
    cudaEventRecord(b, ctx->cs);
    if (e == cudaSuccess) e = cudaEventSynchronize(b);
    float ms = 0.f;
    if (e == cudaSuccess && r > 0 && cudaEventElapsedTime(&ms, a, b) == cudaSuccess && ms > 0) best = std::min(best, ms);
  }
  cudaEventDestroy(a);
  if (b) cudaEventDestroy(b);
  if (e != cudaSuccess) return check_cuda(ctx, e, "ats_measure_hbm_read");
  *out_gbs = (double)bytes / (best * 1e-3) / 1e9;
  return check_status(ctx);
}

int32_t ats_debug_decode_buffer(ats_ctx* ctx, const ats_layer_desc* L, uint32_t M, uint32_t which, void** out_dev,
                                uint64_t* out_bytes) {
  if (!ctx || !L || !out_dev || !out_bytes || M == 0) return ATS_ERR_INVALID;
  LayerWs w = layout_decode(*L, M, ctx->ws, align_up(ctx->cfg.workspace_bytes));
  if (!w.ok) return fail(ctx, ATS_ERR_NOMEM, "workspace too small");
  const uint64_t H = L->hidden, qd = (uint64_t)L->n_q_heads * L->head_dim, kvd = (uint64_t)L->n_kv_heads * L->head_dim;
  const uint64_t P = (uint64_t)M * (L->n_experts ? L->top_k : 1);
  switch (which) {
    case 0: *out_dev = w.h16; *out_bytes = M * H * 2; break;
    case 1: *out_dev = w.qkv32; *out_bytes = M * (qd + 2 * kvd) * 4; break;
    case 2: *out_dev = w.qrot32; *out_bytes = M * qd * 4; break;
    case 3: *out_dev = w.a16; *out_bytes = M * qd * 2; break;
    case 4: *out_dev = w.x1_32; *out_bytes = M * H * 4; break;
    case 5: *out_dev = w.h2_16; *out_bytes = M * H * 2; break;
    case 6: *out_dev = w.act16; *out_bytes = P * L->ffn * 2; break;
    case 7: *out_dev = w.d32; *out_bytes = P * H * 4; break;
    case 8: *out_dev = w.ids; *out_bytes = P * 4; break;
    case 9: *out_dev = w.gates; *out_bytes = P * 4; break;
    default: return fail(ctx, ATS_ERR_INVALID, "unknown buffer %u", which);
  }
  if (!*out_dev) return fail(ctx, ATS_ERR_INVALID, "buffer %u is not part of this layer", which);
  return ATS_OK;
}

int32_t ats_debug_prefill_buffer(ats_ctx* ctx, const ats_layer_desc* L, uint32_t T, uint32_t which, void** out_dev,
                                 uint64_t* out_bytes) {
  if (!ctx || !L || !out_dev || !out_bytes || T == 0) return ATS_ERR_INVALID;
  LayerWs w = layout_prefill(*L, T, ctx->ws, align_up(ctx->cfg.workspace_bytes));
  if (!w.ok) return fail(ctx, ATS_ERR_NOMEM, "workspace too small");
  const uint64_t H = L->hidden, qd = (uint64_t)L->n_q_heads * L->head_dim, kvd = (uint64_t)L->n_kv_heads * L->head_dim;
  switch (which) {
    case 0: *out_dev = w.h16; *out_bytes = T * H * 2; break;
    case 1: *out_dev = w.qkv16; *out_bytes = T * (qd + 2 * kvd) * 2; break;
    case 2: *out_dev = w.qrot16; *out_bytes = T * qd * 2; break;
    case 3: *out_dev = w.a16; *out_bytes = T * qd * 2; break;
    case 4: *out_dev = w.o16; *out_bytes = T * H * 2; break;
    case 5: *out_dev = w.x1_16; *out_bytes = T * H * 2; break;
    case 6: *out_dev = w.h2_16; *out_bytes = T * H * 2; break;
    case 7: *out_dev = w.gu16; *out_bytes = (uint64_t)T * 2 * L->ffn * 2; break;
    case 8: *out_dev = w.act16; *out_bytes = (uint64_t)T * L->ffn * 2; break;
    case 9: *out_dev = w.d16; *out_bytes = T * H * 2; break;
    default: return fail(ctx, ATS_ERR_INVALID, "unknown buffer %u", which);
  }
  if (!*out_dev) return fail(ctx, ATS_ERR_INVALID, "buffer %u is not part of this layer", which);
  return ATS_OK;
}

int32_t ats_debug_fail_copies(ats_ctx* ctx, uint32_t n) {
  if (!ctx) return ATS_ERR_INVALID;
  ctx->fail_copies = n;
  return ATS_OK;
}

int32_t ats_debug_gemv_wait(ats_ctx* ctx, uint64_t limit_cycles, int32_t withhold_tile) {
  if (!ctx || withhold_tile < -1 || limit_cycles > (1ull << 40)) return ATS_ERR_INVALID;
  ctx->dbg_wait_limit = (long long)limit_cycles;
  ctx->dbg_withhold_plus1 = withhold_tile + 1;
  return ATS_OK;
}

int32_t ats_debug_skip_stages(ats_ctx* ctx, uint32_t mask) {
  if (!ctx || mask > 511u) return ATS_ERR_INVALID;
  ctx->dbg_skip = mask;
  return ATS_OK;
}

}  // extern "C"
