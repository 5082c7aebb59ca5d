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
  // rotated query heads as the sum of two fp16 numbers (q = hi + lo to about 22 bits: the operands of the tensor-core
  // score products); rows past the group are zero
  __align__(16) __half q16_s[2][kAttnMaxGroup][kAttnMaxD + 8];
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

// Warp-level tensor-core pieces (mma.sync m16n8k16, fp16 operands, fp32 accumulation) and their operand loads.
__device__ __forceinline__ void ad_mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ad_ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
}
__device__ __forceinline__ void ad_ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(smem_row)));
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
  constexpr int VROW = D * 2 + 16;
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
  constexpr int CH = D * 2 / 16;       // 16-byte chunks per cache row
  constexpr int KROW = D * 2 + 16;     // row pitch in shared memory: the 16-byte pad spreads the eight rows of a matrix load over all banks
  constexpr int VROW = D * 2 + 16;
  constexpr int EPT = D / 64;          // output elements per thread in the merges (64 threads per head)
  constexpr int KS = D / 16;           // k-steps of a score product
  uint8_t* k_s = dyn_s;                              // [POS][KROW]
  uint8_t* v_s = dyn_s + (size_t)POS * KROW;    // [POS][VROW]
  __half (&q16_s)[2][kAttnMaxGroup][kAttnMaxD + 8] = as.q16_s;
  float (&w_acc)[kAttnMaxWarps][kAttnMaxD] = as.w_acc;
  float (&w_m)[kAttnMaxWarps] = as.w_m;
  float (&w_l)[kAttnMaxWarps] = as.w_l;
  int& is_last = as.is_last;
  const int G = p.group / p.hsplit;  // query heads of this CTA
  const int kvh = jy / p.hsplit;
  const int hbase = kvh * p.group + (jy % p.hsplit) * G;  // first of them
  const bool writer = jy % p.hsplit == 0;                 // one CTA per kv head appends to the caches
  const int lane = tid & 31, warp = tid >> 5;
  const int half = D / 2, n_ctx = p.pos + 1;
  const int qd = p.n_q * D, kvd = p.n_kv * D;
  const int tc0 = split * POS;                     // first position of the CTA
  const bool own = split == p.pos / POS;           // this CTA holds the new token's position
  const int r_new = p.pos - tc0;
  // Rotary embedding of the group's query heads into shared memory, each element split into two fp16 numbers
  // (hi = rn16(q), lo = rn16(q - hi)); rows of heads the group does not have are zero.
  for (int idx = tid; idx < kAttnMaxGroup * half; idx += nthr) {
    const int g2 = idx / half, i = idx % half;
    float ra = 0.f, rb = 0.f;
    if (g2 < G) {
      const int hq2 = hbase + g2;
      const float* q = p.qkv + (size_t)hq2 * D;
      const float a = q[i], b = q[i + half];
      const float c = p.cs[2 * i], s = p.cs[2 * i + 1];
      ra = a * c - b * s;
      rb = b * c + a * s;
      if (p.q_rot_out && split == 0) {
        p.q_rot_out[(size_t)hq2 * D + i] = ra;
        p.q_rot_out[(size_t)hq2 * D + i + half] = rb;
      }
    }
    const __half ha = __float2half_rn(ra), hb = __float2half_rn(rb);
    q16_s[0][g2][i] = ha;
    q16_s[0][g2][i + half] = hb;
    q16_s[1][g2][i] = __float2half_rn(ra - __half2float(ha));
    q16_s[1][g2][i + half] = __float2half_rn(rb - __half2float(hb));
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
  // Warp `sub` (< SUB) attends with ALL heads of the CTA to positions sub * 32 .. + 31 on the tensor cores.
  // Scores, transposed: S^T[head][pos] = Q[head][d] K^T[d][pos]; the heads are the 16 rows of the A operand (rows past the
  // group are zero), eight positions are the columns of an instruction.  A lane then holds, for head lane / 4, the scores
  // of positions 8 nt + 2 (lane % 4) + {0, 1} of the block, nt = 0..3.
  if (warp < SUB) {
    const int sub = warp;
    const int hh = lane >> 2, pq = (lane & 3) * 2;  // this lane's head row and position pair within an 8-column tile
    float sc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[nt][e] = 0.f;
    uint32_t qa[2][KS][2];  // [hi | lo][k-step][k, k + 8]
#pragma unroll
    for (int hl = 0; hl < 2; ++hl)
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[hl][ks][0] = *reinterpret_cast<const uint32_t*>(&q16_s[hl][hh][ks * 16 + pq]);
        qa[hl][ks][1] = *reinterpret_cast<const uint32_t*>(&q16_s[hl][hh][ks * 16 + 8 + pq]);
      }
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      // matrices of one load: d chunks (lane / 8) * 8 of two k-steps, rows = the tile's eight positions
      const uint8_t* krow = k_s + (size_t)(sub * 32 + nt * 8 + (lane & 7)) * KROW + (lane >> 3) * 16;
#pragma unroll
      for (int kp = 0; kp < KS / 2; ++kp) {
        uint32_t kb[4];
        ad_ldmatrix_x4(kb, krow + kp * 64);
        // the small halves first: both products are exact in the fp32 accumulator's terms, only the order of additions differs
        ad_mma16816(sc[nt], qa[1][2 * kp][0], 0u, qa[1][2 * kp][1], 0u, kb[0], kb[1]);
        ad_mma16816(sc[nt], qa[1][2 * kp + 1][0], 0u, qa[1][2 * kp + 1][1], 0u, kb[2], kb[3]);
        ad_mma16816(sc[nt], qa[0][2 * kp][0], 0u, qa[0][2 * kp][1], 0u, kb[0], kb[1]);
        ad_mma16816(sc[nt], qa[0][2 * kp + 1][0], 0u, qa[0][2 * kp + 1][1], 0u, kb[2], kb[3]);
      }
    }
    // softmax over the block's 32 positions per head: a head's scores sit in the four lanes of a quad
    const int rel0 = tc0 + sub * 32;  // first position of the block
    float mw = -INFINITY;
    float sv[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const bool ok = rel0 + nt * 8 + pq + e < n_ctx;
        sv[nt][e] = ok ? sc[nt][e] * p.scale : -INFINITY;
        mw = fmaxf(mw, sv[nt][e]);
      }
    mw = fmaxf(mw, __shfl_xor_sync(0xffffffffu, mw, 1));
    mw = fmaxf(mw, __shfl_xor_sync(0xffffffffu, mw, 2));
    // the weights enter the value products as the sum of two fp16 numbers as well (hi = rn16(p), lo = rn16(p - hi))
    uint32_t pb[2][4];
    float lw = 0.f;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const float p0 = (hh < G && sv[nt][0] > -INFINITY) ? expf(sv[nt][0] - mw) : 0.f;
      const float p1 = (hh < G && sv[nt][1] > -INFINITY) ? expf(sv[nt][1] - mw) : 0.f;
      const __half2 hi = __floats2half2_rn(p0, p1);
      const float2 hf = __half22float2(hi);
      const __half2 lo = __floats2half2_rn(p0 - hf.x, p1 - hf.y);
      pb[0][nt] = *reinterpret_cast<const uint32_t*>(&hi);
      pb[1][nt] = *reinterpret_cast<const uint32_t*>(&lo);
      lw += p0 + p1;
    }
    lw += __shfl_xor_sync(0xffffffffu, lw, 1);
    lw += __shfl_xor_sync(0xffffffffu, lw, 2);
    if ((lane & 3) == 0 && hh < G) {
      w_m[hh * SUB + sub] = mw;
      w_l[hh * SUB + sub] = lw;
    }
    // Outputs, transposed: O^T[d][head] = V^T[d][pos] P^T[pos][head]: the value rows, loaded transposed, are the A
    // operand (16 dims per instruction), the weights are the B operand straight from the score registers.
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
      float oc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        // matrices of one load: (positions 16 kk + 0..7, dims 16 mt + 0..7), (same positions, dims + 8), (positions + 8, dims),
        // (positions + 8, dims + 8)
        const uint8_t* vrow = v_s + (size_t)(sub * 32 + kk * 16 + (lane >> 4) * 8 + (lane & 7)) * VROW + (mt * 16 + ((lane >> 3) & 1) * 8) * 2;
        uint32_t va[4];
        ad_ldmatrix_x4_trans(va, vrow);
        ad_mma16816(oc, va[0], va[1], va[2], va[3], pb[1][2 * kk], pb[1][2 * kk + 1]);
        ad_mma16816(oc, va[0], va[1], va[2], va[3], pb[0][2 * kk], pb[0][2 * kk + 1]);
      }
      // oc[0], oc[1]: dim 16 mt + lane / 4, heads pq, pq + 1; oc[2], oc[3]: dim + 8
      if (pq < G) {
        w_acc[pq * SUB + sub][mt * 16 + hh] = oc[0];
        w_acc[pq * SUB + sub][mt * 16 + hh + 8] = oc[2];
      }
      if (pq + 1 < G) {
        w_acc[(pq + 1) * SUB + sub][mt * 16 + hh] = oc[1];
        w_acc[(pq + 1) * SUB + sub][mt * 16 + hh + 8] = oc[3];
      }
    }
  }
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
  // before thread 0's fence, and the fence is cumulative: one thread's fence on each side of the counter publishes the
  // CTA's partials and, in the last CTA, makes the others' visible to the loads below (which bypass L1).
  ATS_ATR(5);
  job_sync();
  if (tid == 0) {
    __threadfence();
    const int prev = atomicAdd(p.counters + jy, 1);
    is_last = prev == n_splits - 1;
    if (is_last) p.counters[jy] = 0;  // ready for the next launch
    __threadfence();
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
