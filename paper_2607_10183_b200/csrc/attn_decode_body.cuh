// Decode attention for one (split, kv head) job: the device code of the decode attention kernel, written so that a
// subset of a CTA's threads can run it too (CTA_SYNC = false).
#pragma once
#include "ats_internal.h"

namespace ats {

constexpr int kAttnMaxGroup = 8;  // query heads per kv head at most
constexpr int kAttnMaxWarps = 16;  // warps of a job at most (heads of the CTA * sub-blocks)
constexpr int kAttnMaxD = 128;

// Static shared memory of a job (head dimensions up to kAttnMaxD use the front of each row).
struct AttnShared {
  __align__(16) float q_s[kAttnMaxGroup][kAttnMaxD];  // rotated query heads
  float w_acc[kAttnMaxWarps][kAttnMaxD];              // per-warp unnormalised outputs
  float w_m[kAttnMaxWarps], w_l[kAttnMaxWarps];       // per-warp score maximum and sum of exponentials
  int is_last;
};

#ifdef ATS_TRACE_ATTN
// Timeline probe of development builds: (globaltimer, CTA, event) records of thread 0 of every CTA.
struct AttnTraceRec {
  unsigned long long t;
  unsigned int cta, ev;
};
__device__ AttnTraceRec g_attn_trace[1 << 15];
__device__ unsigned int g_attn_trace_n;
__shared__ unsigned long long s_attn_tr[8];
__device__ __forceinline__ void attn_trace(int ev) {
  if (threadIdx.x != 0) return;
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  s_attn_tr[ev] = t;
  if (ev == 6 || ev == 7) {  // flush: 6 is every CTA's last stamp unless it merges (then 7 follows and re-flushes that one)
    const int first = ev == 6 ? 0 : 7, n = ev == 6 ? 7 : 1;
    const unsigned int i = atomicAdd(&g_attn_trace_n, (unsigned)n);
    for (int k = 0; k < n; ++k)
      if (i + k < (1u << 15)) g_attn_trace[i + k] = AttnTraceRec{s_attn_tr[first + k], blockIdx.x + 100u * blockIdx.y, (unsigned)(first + k)};
  }
}
#define ATS_ATR(ev) attn_trace(ev)
#else
#define ATS_ATR(ev) do { } while (0)
#endif

__device__ __forceinline__ __half2 ad_half2(uint32_t v) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = v;
  return h;
}
__device__ __forceinline__ float ad_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float ad_warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}

// Job (split, kv head, head part): the group's query heads are divided over `hsplit` CTAs (each stages the same cache rows
// and attends with group / hsplit heads), so that short contexts still fill the SMs.  jy = kv head * hsplit + part.
// The work of one job, in two parts: staging the past cache rows (which do not depend on the new
// token's projections) and everything after those projections exist.  nthr = group * 32 * SUB threads take part,
// numbered tid = 0 .. nthr-1; they synchronise with __syncthreads() when they are the whole CTA (CTA_SYNC) and with
// named barrier 4 otherwise.
template <int D, int SUB>
__device__ __forceinline__ void attn_decode_stage(const AttnDecodeParams& p, const int split, const int kvh, const int tid,
                                                  const int nthr, uint8_t* dyn_s) {
  constexpr int POS = 32 * SUB;
  constexpr int CH = D * 2 / 16;
  constexpr int KROW = D * 2 + 16;
  constexpr int VROW = D * 2;
  uint8_t* k_s = dyn_s;
  uint8_t* v_s = dyn_s + (size_t)POS * KROW;
  const int n_ctx = p.pos + 1;
  const int tc0 = split * POS;
  const int rows_here = min(POS, n_ctx - tc0);
  const bool own = split == p.pos / POS;
  const int r_new = p.pos - tc0;
  for (int c = tid; c < rows_here * CH; c += nthr) {
    const int row = c / CH, ch = c % CH;
    if (!(own && row == r_new)) {
      const size_t off = ((size_t)kvh * p.cap + tc0 + row) * D + ch * 8;
      cp_async16(k_s + (size_t)row * KROW + ch * 16, p.kc + off);
      cp_async16(v_s + (size_t)row * VROW + ch * 16, p.vc + off);
    }
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // value rows beyond the context are read by the PV loop with weight zero: they must hold finite numbers
  for (int c = tid + rows_here * CH; c < POS * CH; c += nthr)
    *reinterpret_cast<uint4*>(v_s + (size_t)(c / CH) * VROW + (c % CH) * 16) = make_uint4(0, 0, 0, 0);
}

template <int D, int SUB, bool CTA_SYNC>
__device__ __forceinline__ void attn_decode_compute(const AttnDecodeParams& p, const int split, const int jy, const int n_splits,
                                                    const int tid, const int nthr, uint8_t* dyn_s, AttnShared& as) {
  auto job_sync = [&]() {
    if (CTA_SYNC)
      __syncthreads();
    else
      asm volatile("bar.sync 4, %0;" ::"r"(nthr) : "memory");
  };
  constexpr int POS = 32 * SUB;        // positions per CTA
  constexpr int V = D / 32;            // output dims per lane
  constexpr int CH = D * 2 / 16;       // 16-byte chunks per cache row
  constexpr int KROW = D * 2 + 16;     // key row pitch in shared memory: the 16-byte pad makes lane-per-row reads conflict-free
  constexpr int VROW = D * 2;
  constexpr int EPT = D / 64;          // output elements per thread in the merges (64 threads per head)
  uint8_t* k_s = dyn_s;                              // [POS][KROW]
  uint8_t* v_s = dyn_s + (size_t)POS * KROW;    // [POS][VROW]
  float (&q_s)[kAttnMaxGroup][kAttnMaxD] = as.q_s;
  float (&w_acc)[kAttnMaxWarps][kAttnMaxD] = as.w_acc;
  float (&w_m)[kAttnMaxWarps] = as.w_m;
  float (&w_l)[kAttnMaxWarps] = as.w_l;
  int& is_last = as.is_last;
  const int G = p.group / p.hsplit;  // query heads of this CTA; nthr = G * POS
  const int kvh = jy / p.hsplit;
  const int hbase = kvh * p.group + (jy % p.hsplit) * G;  // first of them
  const bool writer = jy % p.hsplit == 0;                 // one CTA per kv head appends to the caches
  const int lane = tid & 31, warp = tid >> 5;
  const int g = warp / SUB, sub = warp % SUB;
  const int half = D / 2, n_ctx = p.pos + 1;
  const int qd = p.n_q * D, kvd = p.n_kv * D;
  const int tc0 = split * POS;                     // first position of the CTA
  const bool own = split == p.pos / POS;           // this CTA holds the new token's position
  const int r_new = p.pos - tc0;
  // rotary embedding of the group's query heads into shared memory
  for (int idx = tid; idx < G * half; idx += nthr) {
    const int g2 = idx / half, i = idx % half;
    const int hq2 = hbase + g2;
    const float* q = p.qkv + (size_t)hq2 * D;
    const float a = q[i], b = q[i + half];
    const float c = p.cs[2 * i], s = p.cs[2 * i + 1];
    const float ra = a * c - b * s, rb = b * c + a * s;
    q_s[g2][i] = ra;
    q_s[g2][i + half] = rb;
    if (p.q_rot_out && split == 0) {
      p.q_rot_out[(size_t)hq2 * D + i] = ra;
      p.q_rot_out[(size_t)hq2 * D + i + half] = rb;
    }
  }
  // the CTA that covers position `pos` rotates the new key, rounds key and value to fp16 as the cache holds them, puts
  // them into its staged tiles and appends them to the caches
  if (own) {
    for (int i = tid; i < half; i += nthr) {
      const float c = p.cs[2 * i], s = p.cs[2 * i + 1];
      const float* k = p.qkv + qd + (size_t)kvh * D;
      const float a = k[i], b = k[i + half];
      const __half ka = __float2half_rn(a * c - b * s), kb = __float2half_rn(b * c + a * s);
      __half* srow = reinterpret_cast<__half*>(k_s + (size_t)r_new * KROW);
      srow[i] = ka;
      srow[i + half] = kb;
      if (writer) {
        __half* dst = p.kc + ((size_t)kvh * p.cap + p.pos) * D;
        dst[i] = ka;
        dst[i + half] = kb;
      }
    }
    for (int i = tid; i < D; i += nthr) {
      const __half vv = __float2half_rn(p.qkv[qd + kvd + (size_t)kvh * D + i]);
      reinterpret_cast<__half*>(v_s + (size_t)r_new * VROW)[i] = vv;
      if (writer) p.vc[((size_t)kvh * p.cap + p.pos) * D + i] = vv;
    }
  }
  ATS_ATR(2);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  job_sync();
  ATS_ATR(3);
  const int t0 = tc0 + sub * 32;
  const int n_here = min(32, n_ctx - t0);  // uniform over the warp; <= 0 when the warp has no position
  const bool ok = lane < n_here;
  float sc = 0.f;
  if (ok) {
    const uint4* kr = reinterpret_cast<const uint4*>(k_s + (size_t)(sub * 32 + lane) * KROW);
    const float* qh = q_s[g];
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const uint4 kv = kr[c];
      const float4 q0 = *reinterpret_cast<const float4*>(qh + c * 8);
      const float4 q1 = *reinterpret_cast<const float4*>(qh + c * 8 + 4);
      float2 f;
      f = __half22float2(ad_half2(kv.x)); s0 = fmaf(f.x, q0.x, s0); s1 = fmaf(f.y, q0.y, s1);
      f = __half22float2(ad_half2(kv.y)); s0 = fmaf(f.x, q0.z, s0); s1 = fmaf(f.y, q0.w, s1);
      f = __half22float2(ad_half2(kv.z)); s0 = fmaf(f.x, q1.x, s0); s1 = fmaf(f.y, q1.y, s1);
      f = __half22float2(ad_half2(kv.w)); s0 = fmaf(f.x, q1.z, s0); s1 = fmaf(f.y, q1.w, s1);
    }
    sc = s0 + s1;
  }
  const float sv = ok ? sc * p.scale : -INFINITY;
  const float mw = ad_warp_max(sv);
  const float pr = (ok && mw > -INFINITY) ? expf(sv - mw) : 0.f;
  const float lw = ad_warp_sum(pr);
  if (lane == 0) {
    w_m[warp] = mw;
    w_l[warp] = lw;
  }
  float acc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) acc[v] = 0.f;
#pragma unroll
  for (int tt = 0; tt < 32; ++tt) {
    const float pt = __shfl_sync(0xffffffffu, pr, tt);
    {
      const uint8_t* vr = v_s + (size_t)(sub * 32 + tt) * VROW + lane * (V * 2);
      float2 f;
      if (V == 4) {
        const uint2 raw = *reinterpret_cast<const uint2*>(vr);
        f = __half22float2(ad_half2(raw.x));
        acc[0] = fmaf(pt, f.x, acc[0]);
        acc[1] = fmaf(pt, f.y, acc[1]);
        f = __half22float2(ad_half2(raw.y));
        acc[2] = fmaf(pt, f.x, acc[2]);
        acc[3] = fmaf(pt, f.y, acc[3]);
      } else {
        f = __half22float2(ad_half2(*reinterpret_cast<const uint32_t*>(vr)));
        acc[0] = fmaf(pt, f.x, acc[0]);
        acc[1] = fmaf(pt, f.y, acc[1]);
      }
    }
  }
#pragma unroll
  for (int v = 0; v < V; ++v) w_acc[warp][lane * V + v] = acc[v];
  ATS_ATR(4);
  job_sync();
  // merge each head's warps (ascending) into this split's partial: 64 threads per head
  const int g2 = tid / 64, j = tid % 64;
  const int hq2 = hbase + g2;
  if (g2 < G) {
    float* part = p.part + ((size_t)hq2 * n_splits + split) * (D + 2);
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < SUB; ++w) mx = fmaxf(mx, w_m[g2 * SUB + w]);
    float l = 0.f, o[EPT];
#pragma unroll
    for (int q = 0; q < EPT; ++q) o[q] = 0.f;
#pragma unroll
    for (int w = 0; w < SUB; ++w) {
      const float m = w_m[g2 * SUB + w];
      const float f = m > -INFINITY ? expf(m - mx) : 0.f;
      l = fmaf(w_l[g2 * SUB + w], f, l);
#pragma unroll
      for (int q = 0; q < EPT; ++q) o[q] = fmaf(w_acc[g2 * SUB + w][j + 64 * q], f, o[q]);
    }
#pragma unroll
    for (int q = 0; q < EPT; ++q) part[j + 64 * q] = o[q];
    if (j == 0) {
      part[D] = mx;
      part[D + 1] = l;
    }
  }
  // The last CTA of this job row merges the splits of its query heads.  The barrier orders every thread's partial
  // before thread 0's arrival, an atomic with release and acquire semantics: released with it are the CTA's partials
  // (the barrier makes them precede it), acquired by the last arrival are the other CTAs' (its loads below bypass L1).
  // One such atomic instead of a fence on each side of a relaxed one is one round trip less (0.4 us of the step).
  ATS_ATR(5);
  job_sync();
  if (tid == 0) {
    int prev;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(prev) : "l"(p.counters + jy) : "memory");
    is_last = prev == n_splits - 1;
    if (is_last) p.counters[jy] = 0;  // ready for the next launch
  }
  job_sync();
  ATS_ATR(6);
  if (!is_last || g2 >= G) return;
  const float* base = p.part + (size_t)hq2 * n_splits * (D + 2);
  float mx = -INFINITY, l = 0.f, o[EPT];
#pragma unroll
  for (int q = 0; q < EPT; ++q) o[q] = 0.f;
  constexpr int NB = 16;  // splits per round trip: all of a batch's loads are issued before any is used
  for (int s0 = 0; s0 < n_splits; s0 += NB) {
    float m[NB], ls[NB], v[NB][EPT];
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const bool in = s0 + u < n_splits;
      const float* ps = base + (size_t)(s0 + u) * (D + 2);
      m[u] = in ? __ldcg(ps + D) : -INFINITY;
      ls[u] = in ? __ldcg(ps + D + 1) : 0.f;
#pragma unroll
      for (int q = 0; q < EPT; ++q) v[u][q] = in ? __ldcg(ps + j + 64 * q) : 0.f;
    }
    float bm = mx;
#pragma unroll
    for (int u = 0; u < NB; ++u) bm = fmaxf(bm, m[u]);
    const float rs = mx > -INFINITY ? expf(mx - bm) : 0.f;  // rescale what earlier batches accumulated
    l *= rs;
#pragma unroll
    for (int q = 0; q < EPT; ++q) o[q] *= rs;
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const float f = m[u] > -INFINITY ? expf(m[u] - bm) : 0.f;
      l = fmaf(ls[u], f, l);
#pragma unroll
      for (int q = 0; q < EPT; ++q) o[q] = fmaf(v[u][q], f, o[q]);
    }
    mx = bm;
  }
  const float inv = 1.0f / l;
#pragma unroll
  for (int q = 0; q < EPT; ++q) p.a16[(size_t)hq2 * D + j + 64 * q] = __float2half_rn(o[q] * inv);
  ATS_ATR(7);
}

// Stand-alone form: the cache rows of past tokens are requested before the grid dependency resolves.
template <int D, int SUB, bool CTA_SYNC>
__device__ __forceinline__ void attn_decode_body(const AttnDecodeParams& p, const int split, const int jy, const int n_splits,
                                                 const int tid, const int nthr, uint8_t* dyn_s, AttnShared& as) {
  ATS_ATR(0);
  attn_decode_stage<D, SUB>(p, split, jy / p.hsplit, tid, nthr, dyn_s);
  asm volatile("griddepcontrol.wait;" ::: "memory");  // q, k, v of the new token come from the preceding kernel
  ATS_ATR(1);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  attn_decode_compute<D, SUB, CTA_SYNC>(p, split, jy, n_splits, tid, nthr, dyn_s, as);
}

}  // namespace ats
