// Prefill-side glue kernels (sm_100a): rotary embedding + KV append over T tokens, causal grouped-query attention
// over the cache (tensor cores), fp16 residual add and SwiGLU.  Every intermediate of the prefill path is stored as fp16 (the
// operands of the tensor-core GEMMs), so these kernels read and write fp16 and compute in fp32.
#include "ats_internal.h"
#include "sm100_sync.cuh"

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

// One CTA per token.  The cos/sin table of the token's position (one fp64 sincos per pair index i) goes to shared memory;
// the threads then take (head, run of 8 pair indices) tasks with 16-byte loads and stores: rotate q into q_rot, rotate k
// into the key cache, copy v into the value cache.
__global__ void __launch_bounds__(256) rope_append_prefill_kernel(const __half* __restrict__ qkv, int ld, __half* __restrict__ q_rot,
                                                                  __half* __restrict__ kc, __half* __restrict__ vc, int n_q, int n_kv,
                                                                  int d, int cap, int pos0, float theta) {
  __shared__ float2 cs_s[128];  // d <= 256
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int half = d / 2, t = blockIdx.x, pos = pos0 + t;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    float c = 1.f, s = 0.f;
    if (theta != 0.f) {
      const double inv = pow((double)theta, -2.0 * (double)i / (double)d);
      double sd, cd;
      sincos((double)pos * inv, &sd, &cd);
      c = (float)cd;
      s = (float)sd;
    }
    cs_s[i] = make_float2(c, s);
  }
  __syncthreads();
  const __half* row = qkv + (size_t)t * ld;
  const int qd = n_q * d, kvd = n_kv * d;
  const int segs = half / 8;  // runs of 8 pair indices per head
  for (int task = threadIdx.x; task < (n_q + n_kv) * segs; task += blockDim.x) {
    const int head = task / segs, i0 = (task % segs) * 8;
    const bool is_q = head < n_q;
    const __half* src = row + (is_q ? head * d : qd + (head - n_q) * d);
    __half* dst = is_q ? q_rot + (size_t)t * qd + head * d : kc + ((size_t)(head - n_q) * cap + pos) * d;
    const uint4 a4 = *reinterpret_cast<const uint4*>(src + i0), b4 = *reinterpret_cast<const uint4*>(src + half + i0);
    const uint32_t aw[4] = {a4.x, a4.y, a4.z, a4.w}, bw[4] = {b4.x, b4.y, b4.z, b4.w};
    uint32_t ra[4], rb[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      __half2 ah, bh;
      *reinterpret_cast<uint32_t*>(&ah) = aw[q];
      *reinterpret_cast<uint32_t*>(&bh) = bw[q];
      const float2 a = __half22float2(ah), b = __half22float2(bh);
      const float2 cs0 = cs_s[i0 + 2 * q], cs1 = cs_s[i0 + 2 * q + 1];
      const __half2 oa = __floats2half2_rn(a.x * cs0.x - b.x * cs0.y, a.y * cs1.x - b.y * cs1.y);
      const __half2 ob = __floats2half2_rn(b.x * cs0.x + a.x * cs0.y, b.y * cs1.x + a.y * cs1.y);
      ra[q] = *reinterpret_cast<const uint32_t*>(&oa);
      rb[q] = *reinterpret_cast<const uint32_t*>(&ob);
    }
    *reinterpret_cast<uint4*>(dst + i0) = make_uint4(ra[0], ra[1], ra[2], ra[3]);
    *reinterpret_cast<uint4*>(dst + half + i0) = make_uint4(rb[0], rb[1], rb[2], rb[3]);
  }
  for (int task = threadIdx.x; task < n_kv * (d / 8); task += blockDim.x) {
    const int kvh = task / (d / 8), c = (task % (d / 8)) * 8;
    *reinterpret_cast<uint4*>(vc + ((size_t)kvh * cap + pos) * d + c) = *reinterpret_cast<const uint4*>(row + qd + kvd + kvh * d + c);
  }
}

cudaError_t launch_rope_append_prefill(const __half* qkv16, int ld, __half* q_rot16, __half* kc, __half* vc, int T,
                                       int n_q, int n_kv, int d, int cap, int pos0, float theta, cudaStream_t st,
                                       uint64_t* n_launch, int pdl) {
  // 16-byte accesses: head_dim a multiple of 16, rows and caches 16-byte aligned
  if (d % 16 != 0 || d > 256 || ld % 8 != 0 ||
      (((reinterpret_cast<uintptr_t>(qkv16) | reinterpret_cast<uintptr_t>(q_rot16) | reinterpret_cast<uintptr_t>(kc) |
         reinterpret_cast<uintptr_t>(vc)) & 15) != 0))
    return cudaErrorInvalidValue;
  ++*n_launch;
  return launch_dep(rope_append_prefill_kernel, dim3(T), dim3(256), 0, st, pdl, 1, qkv16, ld, q_rot16, kc, vc, n_q, n_kv, d, cap, pos0,
                    theta);
}

// Causal grouped-query attention over the cache on the tensor cores (mma.sync m16n8k16, fp16 operands, fp32 accumulate).
// CTA = 64 query tokens of one query head, 4 warps x 16 rows.  Key/value blocks of 64 cache rows are staged with 16-byte
// async copies into padded shared-memory rows (double buffered); S = Q K^T and O += P V use ldmatrix fragments; the softmax
// is the running-max form in fp32, with P rounded to fp16 as the operand of the second product.
constexpr int kFaQ = 64;   // query rows per CTA
constexpr int kFaK = 64;   // cache rows per block

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <int D>
__global__ void __launch_bounds__(128) attn_prefill_kernel(const __half* __restrict__ q_rot, const __half* __restrict__ kc,
                                                           const __half* __restrict__ vc, __half* __restrict__ a16, int T,
                                                           int n_q, int group, int cap, int pos0, float scale) {
  constexpr int PITCH = D + 8;          // halfs per shared-memory row (16-byte pad: conflict-free ldmatrix)
  constexpr int CH = D / 8;             // 16-byte chunks per row
  constexpr int KS = D / 16;            // k-steps of Q K^T
  constexpr int NT = D / 8;             // n-tiles of the output
  extern __shared__ __align__(16) __half fa_smem[];
  __half* q_s = fa_smem;                          // [kFaQ][PITCH]
  __half* k_s = q_s + kFaQ * PITCH;               // [2][kFaK][PITCH]
  __half* v_s = k_s + 2 * kFaK * PITCH;           // [2][kFaK][PITCH]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int qb = blockIdx.x, hq = blockIdx.y, kvh = hq / group;
  const int tq0 = qb * kFaQ;                      // first token of the CTA
  const int n_kb = (pos0 + min(T, tq0 + kFaQ) - 1) / kFaK + 1;  // cache blocks any row of the CTA attends to
  // ---- stage Q (zero rows beyond T) and the first K/V block
  for (int c = threadIdx.x; c < kFaQ * CH; c += 128) {
    const int row = c / CH, ch = c % CH;
    const int t = tq0 + row;
    if (t < T)
      cp_async_16(q_s + row * PITCH + ch * 8, q_rot + ((size_t)t * n_q + hq) * D + ch * 8);
    else
      *reinterpret_cast<uint4*>(q_s + row * PITCH + ch * 8) = make_uint4(0, 0, 0, 0);
  }
  auto stage_kv = [&](int kb, int buf) {
    for (int c = threadIdx.x; c < kFaK * CH; c += 128) {
      const int row = c / CH, ch = c % CH;
      const int key = min(kb * kFaK + row, cap - 1);  // rows past the context are masked below; keep the address legal
      cp_async_16(k_s + (buf * kFaK + row) * PITCH + ch * 8, kc + ((size_t)kvh * cap + key) * D + ch * 8);
      cp_async_16(v_s + (buf * kFaK + row) * PITCH + ch * 8, vc + ((size_t)kvh * cap + key) * D + ch * 8);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  stage_kv(0, 0);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  // ---- Q fragments of this warp's 16 rows
  uint32_t qf[KS][4];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
    ldsm_x4(qf[ks], q_s + (warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + ks * 16 + (lane >> 4) * 8);
  float o[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[n][e] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const int g = lane >> 2, tq = lane & 3;
  const int qpos[2] = {pos0 + tq0 + warp * 16 + g, pos0 + tq0 + warp * 16 + g + 8};  // absolute positions of this thread's rows
  for (int kb = 0; kb < n_kb; ++kb) {
    const int buf = kb & 1;
    if (kb + 1 < n_kb) stage_kv(kb + 1, buf ^ 1);  // next block in flight while this one is used
    const __half* kb_s = k_s + buf * kFaK * PITCH;
    const __half* vb_s = v_s + buf * kFaK * PITCH;
    // S = Q K^T for 16 rows x 64 keys
    float sacc[kFaK / 8][4];
#pragma unroll
    for (int n = 0; n < kFaK / 8; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) sacc[n][e] = 0.f;
#pragma unroll
    for (int n = 0; n < kFaK / 8; ++n) {
#pragma unroll
      for (int ks2 = 0; ks2 < KS / 2; ++ks2) {
        uint32_t b[4];  // b0,b1 of k-step 2*ks2 and of k-step 2*ks2+1 for keys 8n..8n+7
        ldsm_x4(b, kb_s + (n * 8 + (lane & 7)) * PITCH + ks2 * 32 + (lane >> 3) * 8);
        mma_16816(sacc[n], qf[2 * ks2], b[0], b[1]);
        mma_16816(sacc[n], qf[2 * ks2 + 1], b[2], b[3]);
      }
    }
    // scale, causal mask, running softmax (rows g and g+8 of the warp's 16)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int n = 0; n < kFaK / 8; ++n) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kb * kFaK + n * 8 + 2 * tq + (e & 1);
        const int r = e >> 1;
        const float v = key <= qpos[r] ? sacc[n][e] * scale : -INFINITY;
        sacc[n][e] = v;
        mx[r] = fmaxf(mx[r], v);
      }
    }
    float corr[2], m_new[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      m_new[r] = fmaxf(m_run[r], mx[r]);
      corr[r] = m_run[r] > -INFINITY ? expf(m_run[r] - m_new[r]) : 0.f;
      m_run[r] = m_new[r];
    }
    float ls[2] = {0.f, 0.f};
    uint32_t pf[kFaK / 16][4];  // P as A fragments (fp16)
#pragma unroll
    for (int n = 0; n < kFaK / 8; ++n) {
      float pv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = e >> 1;
        pv[e] = m_new[r] > -INFINITY ? expf(sacc[n][e] - m_new[r]) : 0.f;
        ls[r] += pv[e];
      }
      pf[n >> 1][(n & 1) * 2] = pack_h2(pv[0], pv[1]);
      pf[n >> 1][(n & 1) * 2 + 1] = pack_h2(pv[2], pv[3]);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      ls[r] += __shfl_xor_sync(0xffffffffu, ls[r], 1);
      ls[r] += __shfl_xor_sync(0xffffffffu, ls[r], 2);
      l_run[r] = l_run[r] * corr[r] + ls[r];
    }
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      o[n][0] *= corr[0];
      o[n][1] *= corr[0];
      o[n][2] *= corr[1];
      o[n][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < kFaK / 16; ++kk) {
#pragma unroll
      for (int n2 = 0; n2 < NT / 2; ++n2) {
        uint32_t b[4];  // (b0,b1) for dims 16 n2 .. +7 and for dims 16 n2 + 8 .. +15, keys 16 kk .. +15
        ldsm_x4_t(b, vb_s + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + n2 * 16 + (lane >> 4) * 8);
        mma_16816(o[2 * n2], pf[kk], b[0], b[1]);
        mma_16816(o[2 * n2 + 1], pf[kk], b[2], b[3]);
      }
    }
    if (kb + 1 < n_kb) asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // the next block has landed, and nobody still reads the buffer the block after it will overwrite
  }
  // ---- normalise and store
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int t = tq0 + warp * 16 + g + r * 8;
    if (t < T) {
      const float inv = 1.0f / l_run[r];
      __half* dst = a16 + ((size_t)t * n_q + hq) * D;
#pragma unroll
      for (int n = 0; n < NT; ++n)
        *reinterpret_cast<uint32_t*>(dst + n * 8 + 2 * tq) = pack_h2(o[n][2 * r] * inv, o[n][2 * r + 1] * inv);
    }
  }
}

cudaError_t launch_attn_prefill(const __half* q_rot16, const __half* kc, const __half* vc, __half* a16, int T, int n_q,
                                int n_kv, int d, int cap, int pos0, cudaStream_t st, uint64_t* n_launch, int pdl) {
  dim3 grid((T + kFaQ - 1) / kFaQ, n_q);
  const float scale = 1.0f / sqrtf((float)d);
  const size_t smem = (size_t)(kFaQ + 4 * kFaK) * (d + 8) * sizeof(__half);
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e1 = cudaFuncSetAttribute(attn_prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)((kFaQ + 4 * kFaK) * (128 + 8) * sizeof(__half)));
    cudaError_t e2 = cudaFuncSetAttribute(attn_prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)((kFaQ + 4 * kFaK) * (64 + 8) * sizeof(__half)));
    if (e1 != cudaSuccess) return e1;
    if (e2 != cudaSuccess) return e2;
  }
  ++*n_launch;
  if (d == 128)
    return launch_dep(attn_prefill_kernel<128>, grid, dim3(128), smem, st, pdl, 1, q_rot16, kc, vc, a16, T, n_q, n_q / n_kv, cap, pos0,
                      scale);
  if (d == 64)
    return launch_dep(attn_prefill_kernel<64>, grid, dim3(128), smem, st, pdl, 1, q_rot16, kc, vc, a16, T, n_q, n_q / n_kv, cap, pos0,
                      scale);
  return cudaErrorInvalidValue;
}

// gu holds [T][ld] with gate in columns [0, ffn) and up in [ffn, 2 ffn): act = rn16(silu(g) * u); 8 elements per thread
__global__ void swiglu16_kernel(const __half* __restrict__ gu, int ld, int ffn, __half* __restrict__ act, uint64_t n8) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int per_row = ffn / 8;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n8; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t t = i / per_row, c = (i % per_row) * 8;
    const uint4 gv = *reinterpret_cast<const uint4*>(gu + t * ld + c);
    const uint4 uv = *reinterpret_cast<const uint4*>(gu + t * ld + ffn + c);
    const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, uw[4] = {uv.x, uv.y, uv.z, uv.w};
    uint32_t ow[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 g = __half22float2(bits_as_half2(gw[q])), u = __half22float2(bits_as_half2(uw[q]));
      const __half2 r = __floats2half2_rn(g.x / (1.0f + expf(-g.x)) * u.x, g.y / (1.0f + expf(-g.y)) * u.y);
      ow[q] = *reinterpret_cast<const uint32_t*>(&r);
    }
    *reinterpret_cast<uint4*>(act + t * ffn + c) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
  }
}

cudaError_t launch_swiglu16(const __half* gu, int ld, int ffn, __half* act, int T, cudaStream_t st, uint64_t* n_launch, int pdl) {
  const uint64_t n8 = (uint64_t)T * ffn / 8;  // ffn is a multiple of 32
  const int grid = (int)std::min<uint64_t>((n8 + 255) / 256, 148 * 8);
  ++*n_launch;
  return launch_dep(swiglu16_kernel, dim3(grid), dim3(256), 0, st, pdl, 1, gu, ld, ffn, act, n8);
}

// MoE prefill: rows sorted by expert.  xs[r] = h[order[r] / k] (order[r] = the (token, slot) pair at sorted position r);
// 16 bytes per thread.
__global__ void moe_gather_rows_kernel(const __half* __restrict__ h, const int* __restrict__ order, int k, __half* __restrict__ xs,
                                       uint64_t n8, int H) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // h comes from the preceding kernel, order from a preceding copy
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int per_row = H / 8;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n8; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t r = i / per_row, c = (i % per_row) * 8;
    const int t = order[r] / k;
    *reinterpret_cast<uint4*>(xs + r * H + c) = *reinterpret_cast<const uint4*>(h + (uint64_t)t * H + c);
  }
}

cudaError_t launch_moe_gather_rows(const __half* h, const int* order, int k, __half* xs, int P, int H, cudaStream_t st,
                                   uint64_t* n_launch, int pdl) {
  const uint64_t n8 = (uint64_t)P * H / 8;  // H is a multiple of 32
  const int grid = (int)std::min<uint64_t>((n8 + 255) / 256, 148 * 8);
  ++*n_launch;
  return launch_dep(moe_gather_rows_kernel, dim3(grid), dim3(256), 0, st, pdl, 1, h, order, k, xs, n8, H);
}

// y[t] = rn16(res[t] + sum_j gates[t][j] * d[pos[t k + j]]) with the sum in slot order, fp32; pos[p] = sorted position
// of pair p.  8 columns per thread.
__global__ void moe_combine_sorted_kernel(const __half* __restrict__ res, const float* __restrict__ gates, const __half* __restrict__ d,
                                          const int* __restrict__ pos, __half* __restrict__ y, uint64_t n8, int k, int H) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int per_row = H / 8;
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n8; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t t = i / per_row, c = (i % per_row) * 8;
    float acc[8];
    {
      const uint4 rv = *reinterpret_cast<const uint4*>(res + t * H + c);
      const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __half22float2(bits_as_half2(rw[q]));
        acc[2 * q] = f.x;
        acc[2 * q + 1] = f.y;
      }
    }
    for (int j = 0; j < k; ++j) {
      const float gj = gates[t * k + j];
      const uint4 dv = *reinterpret_cast<const uint4*>(d + (uint64_t)pos[t * k + j] * H + c);
      const uint32_t dw[4] = {dv.x, dv.y, dv.z, dv.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __half22float2(bits_as_half2(dw[q]));
        acc[2 * q] = fmaf(gj, f.x, acc[2 * q]);
        acc[2 * q + 1] = fmaf(gj, f.y, acc[2 * q + 1]);
      }
    }
    uint32_t ow[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const __half2 r2 = __floats2half2_rn(acc[2 * q], acc[2 * q + 1]);
      ow[q] = *reinterpret_cast<const uint32_t*>(&r2);
    }
    *reinterpret_cast<uint4*>(y + t * H + c) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
  }
}

cudaError_t launch_moe_combine_sorted(const __half* res, const float* gates, const __half* d, const int* pos, __half* y, int T, int k,
                                      int H, cudaStream_t st, uint64_t* n_launch, int pdl) {
  const uint64_t n8 = (uint64_t)T * H / 8;
  const int grid = (int)std::min<uint64_t>((n8 + 255) / 256, 148 * 8);
  ++*n_launch;
  return launch_dep(moe_combine_sorted_kernel, dim3(grid), dim3(256), 0, st, pdl, 1, res, gates, d, pos, y, n8, k, H);
}

// ---------------------------------------------------------------------------------------------------------------
// Copy kernel for host-placed expert slices (the SM-driven transfer path of Sections 4.1 / 4.2.1): every chunk of the
// list is pulled from the mapped pinned store into shared memory with a bulk-async copy and pushed to its place in
// device memory with another; one thread per CTA keeps four chunks in flight.  One launch moves all the slices a call
// needs, so the per-copy cost of the DMA path (about a third of the time of a sub-megabyte copy) is not paid.
namespace {
constexpr int kCopyStages = 4;
constexpr int kCopyChunk = 32 * 1024;
}  // namespace

__global__ void __launch_bounds__(32, 1) host_gather_kernel(const CopyChunk* __restrict__ list, int n, int* status) {
  extern __shared__ __align__(128) uint8_t cp_s[];
  __shared__ uint64_t full[kCopyStages];
  if (threadIdx.x != 0) return;
  for (int s = 0; s < kCopyStages; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&full[s])));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the list was written by a copy that precedes this launch
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int first = blockIdx.x, gx = gridDim.x;
  const int n_my = first < n ? (n - first + gx - 1) / gx : 0;
  auto issue_load = [&](int j) {
    const int s = j % kCopyStages;
    const CopyChunk c = list[first + j * gx];
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&full[s])), "r"(c.bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(cp_s + (size_t)s * kCopyChunk)),
                 "l"(c.src), "r"(c.bytes), "r"(smem_u32(&full[s]))
                 : "memory");
  };
  for (int j = 0; j < min(kCopyStages, n_my); ++j) issue_load(j);
  for (int j = 0; j < n_my; ++j) {
    const int s = j % kCopyStages;
    if (!mbar_wait_suspending(&full[s], (uint32_t)(j / kCopyStages) & 1u, 2 * kWaitLimitCycles)  /* about two seconds: the source is across PCIe */) {
      raise_status(status, 5);
      break;
    }
    const CopyChunk c = list[first + j * gx];
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(c.dst), "r"(smem_u32(cp_s + (size_t)s * kCopyChunk)),
                 "r"(c.bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    if (j + kCopyStages < n_my) {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the store has read stage s: it may be refilled
      issue_load(j + kCopyStages);
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

cudaError_t launch_host_gather(const CopyChunk* list, int n, int* status, int sm_count, cudaStream_t st, uint64_t* n_launch, int pdl) {
  if (n <= 0) return cudaSuccess;
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e = cudaFuncSetAttribute(host_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCopyStages * kCopyChunk);
    if (e != cudaSuccess) return e;
  }
  ++*n_launch;
  return launch_dep(host_gather_kernel, dim3(std::min(n, sm_count)), dim3(32), (size_t)kCopyStages * kCopyChunk, st, pdl, 1, list, n, status);
}

}  // namespace ats
