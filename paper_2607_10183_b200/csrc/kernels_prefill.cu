// Prefill-side glue kernels (sm_100a): rotary embedding + KV append over T tokens, causal grouped-query attention
// over the cache, fp16 residual add and SwiGLU.  Every intermediate of the prefill path is stored as fp16 (the
// operands of the tensor-core GEMMs), so these kernels read and write fp16 and compute in fp32.
#include "ats_internal.h"

namespace ats {

__device__ __forceinline__ __half2 bits_as_half2(uint32_t v) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = v;
  return h;
}

__device__ __forceinline__ float wsum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float wmax(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// thread <-> (token, pair index i): one fp64 sincos per (token, i), reused over all heads.
__global__ void rope_append_prefill_kernel(const __half* __restrict__ qkv, int ld, __half* __restrict__ q_rot,
                                           __half* __restrict__ kc, __half* __restrict__ vc, int T, int n_q, int n_kv, int d,
                                           int cap, int pos0, float theta) {
  const int half = d / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * half) return;
  const int t = idx / half, i = idx % half;
  const int pos = pos0 + t;
  float c = 1.f, s = 0.f;
  if (theta != 0.f) {
    const double inv = pow((double)theta, -2.0 * (double)i / (double)d);
    double sd, cd;
    sincos((double)pos * inv, &sd, &cd);
    c = (float)cd;
    s = (float)sd;
  }
  const __half* row = qkv + (size_t)t * ld;
  const int qd = n_q * d, kvd = n_kv * d;
  for (int hq = 0; hq < n_q; ++hq) {
    const float a = __half2float(row[hq * d + i]), b = __half2float(row[hq * d + i + half]);
    q_rot[(size_t)t * qd + hq * d + i] = __float2half_rn(a * c - b * s);
    q_rot[(size_t)t * qd + hq * d + i + half] = __float2half_rn(b * c + a * s);
  }
  for (int kvh = 0; kvh < n_kv; ++kvh) {
    const float a = __half2float(row[qd + kvh * d + i]), b = __half2float(row[qd + kvh * d + i + half]);
    __half* dst = kc + ((size_t)kvh * cap + pos) * d;
    dst[i] = __float2half_rn(a * c - b * s);
    dst[i + half] = __float2half_rn(b * c + a * s);
    __half* vd = vc + ((size_t)kvh * cap + pos) * d;
    vd[i] = row[qd + kvd + kvh * d + i];
    vd[i + half] = row[qd + kvd + kvh * d + i + half];
  }
}

cudaError_t launch_rope_append_prefill(const __half* qkv16, int ld, __half* q_rot16, __half* kc, __half* vc, int T,
                                       int n_q, int n_kv, int d, int cap, int pos0, float theta, cudaStream_t st,
                                       uint64_t* n_launch) {
  const int total = T * (d / 2);
  rope_append_prefill_kernel<<<(total + 127) / 128, 128, 0, st>>>(qkv16, ld, q_rot16, kc, vc, T, n_q, n_kv, d, cap, pos0, theta);
  ++*n_launch;
  return cudaGetLastError();
}

// Causal attention: one warp per (token, query head); lanes take cache positions 32 at a time (each lane one whole
// key row), online softmax across chunks, then P.V with the probabilities broadcast by shuffles.
template <int D>
__global__ void __launch_bounds__(128) attn_prefill_kernel(const __half* __restrict__ q_rot, const __half* __restrict__ kc,
                                                           const __half* __restrict__ vc, __half* __restrict__ a16, int T,
                                                           int n_q, int group, int cap, int pos0, float scale) {
  constexpr int V = D / 32;
  __shared__ float q_s[4][D];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int hq = blockIdx.x * 4 + warp;  // 4 heads per CTA
  const int t = blockIdx.y;
  if (hq >= n_q) return;
  const int kvh = hq / group;
  const int n_ctx = pos0 + t + 1;
  for (int e = lane; e < D; e += 32) q_s[warp][e] = __half2float(q_rot[((size_t)t * n_q + hq) * D + e]);
  __syncwarp();
  float m_run = -INFINITY, l_run = 0.f;
  float acc[V];
#pragma unroll
  for (int v = 0; v < V; ++v) acc[v] = 0.f;
  for (int t0 = 0; t0 < n_ctx; t0 += 32) {
    const int tp = t0 + lane;
    const bool ok = tp < n_ctx;
    float sc = 0.f;
    if (ok) {
      const uint4* kr = reinterpret_cast<const uint4*>(kc + ((size_t)kvh * cap + tp) * D);
#pragma unroll 4
      for (int c = 0; c < D / 8; ++c) {
        const uint4 kv = __ldg(kr + c);
        const float* qg = q_s[warp] + c * 8;
        float2 f;
        f = __half22float2(bits_as_half2(kv.x)); sc = fmaf(f.x, qg[0], sc); sc = fmaf(f.y, qg[1], sc);
        f = __half22float2(bits_as_half2(kv.y)); sc = fmaf(f.x, qg[2], sc); sc = fmaf(f.y, qg[3], sc);
        f = __half22float2(bits_as_half2(kv.z)); sc = fmaf(f.x, qg[4], sc); sc = fmaf(f.y, qg[5], sc);
        f = __half22float2(bits_as_half2(kv.w)); sc = fmaf(f.x, qg[6], sc); sc = fmaf(f.y, qg[7], sc);
      }
    }
    const float s = ok ? sc * scale : -INFINITY;
    const float m_new = fmaxf(m_run, wmax(s));
    const float corr = m_run > -INFINITY ? expf(m_run - m_new) : 0.f;
    const float p = ok ? expf(s - m_new) : 0.f;
    l_run = l_run * corr + wsum(p);
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] *= corr;
    const int n_here = min(32, n_ctx - t0);
    for (int tt = 0; tt < n_here; ++tt) {
      const float pt = __shfl_sync(0xffffffffu, p, tt);
      const __half* vr = vc + ((size_t)kvh * cap + t0 + tt) * D + lane * V;
      if (V == 4) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(vr));
        float2 f;
        f = __half22float2(bits_as_half2(raw.x)); acc[0] = fmaf(pt, f.x, acc[0]); acc[1] = fmaf(pt, f.y, acc[1]);
        f = __half22float2(bits_as_half2(raw.y)); acc[2] = fmaf(pt, f.x, acc[2]); acc[3] = fmaf(pt, f.y, acc[3]);
      } else {
        const float2 f = __half22float2(bits_as_half2(__ldg(reinterpret_cast<const uint32_t*>(vr))));
        acc[0] = fmaf(pt, f.x, acc[0]);
        acc[1] = fmaf(pt, f.y, acc[1]);
      }
    }
    m_run = m_new;
  }
  __half* dst = a16 + ((size_t)t * n_q + hq) * D + lane * V;
#pragma unroll
  for (int v = 0; v < V; ++v) dst[v] = __float2half_rn(acc[v] / l_run);
}

cudaError_t launch_attn_prefill(const __half* q_rot16, const __half* kc, const __half* vc, __half* a16, int T, int n_q,
                                int n_kv, int d, int cap, int pos0, cudaStream_t st, uint64_t* n_launch) {
  dim3 grid((n_q + 3) / 4, T);
  const float scale = 1.0f / sqrtf((float)d);
  if (d == 128)
    attn_prefill_kernel<128><<<grid, 128, 0, st>>>(q_rot16, kc, vc, a16, T, n_q, n_q / n_kv, cap, pos0, scale);
  else if (d == 64)
    attn_prefill_kernel<64><<<grid, 128, 0, st>>>(q_rot16, kc, vc, a16, T, n_q, n_q / n_kv, cap, pos0, scale);
  else
    return cudaErrorInvalidValue;
  ++*n_launch;
  return cudaGetLastError();
}

__global__ void add16_kernel(const __half* __restrict__ a, const __half* __restrict__ b, __half* __restrict__ out, uint64_t n) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
    out[i] = __float2half_rn(__half2float(a[i]) + __half2float(b[i]));
}

cudaError_t launch_add16(const __half* a, const __half* b, __half* out, uint64_t n, cudaStream_t st, uint64_t* n_launch) {
  const int grid = (int)std::min<uint64_t>((n + 255) / 256, 148 * 8);
  add16_kernel<<<grid, 256, 0, st>>>(a, b, out, n);
  ++*n_launch;
  return cudaGetLastError();
}

// gu holds [T][ld] with gate in columns [0, ffn) and up in [ffn, 2 ffn): act = rn16(silu(g) * u)
__global__ void swiglu16_kernel(const __half* __restrict__ gu, int ld, int ffn, __half* __restrict__ act, uint64_t n) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t t = i / ffn, c = i % ffn;
    const float g = __half2float(gu[t * ld + c]), u = __half2float(gu[t * ld + ffn + c]);
    act[i] = __float2half_rn(g / (1.0f + expf(-g)) * u);
  }
}

cudaError_t launch_swiglu16(const __half* gu, int ld, int ffn, __half* act, int T, cudaStream_t st, uint64_t* n_launch) {
  const uint64_t n = (uint64_t)T * ffn;
  const int grid = (int)std::min<uint64_t>((n + 255) / 256, 148 * 8);
  swiglu16_kernel<<<grid, 256, 0, st>>>(gu, ld, ffn, act, n);
  ++*n_launch;
  return cudaGetLastError();
}

}  // namespace ats
