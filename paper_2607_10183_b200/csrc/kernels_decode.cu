// Decode-side CUDA kernels (sm_100a): block dequantization, the dequantize-fused GEMV (dense and grouped-expert),
// RMSNorm, rotary embedding + KV append, split attention over the KV cache, router top-k and the MoE combine.
//
// The GEMV is memory-bound: 4.5 bits per weight must cross HBM once.  Every lane loads one quantization block per
// step with a single 128-bit load (32 codes) plus its fp16 scale, expands the nibbles to exact fp16 integers with
// two logic ops and one half2 op per pair, accumulates sum_k code*x in fp32 per block, and applies the block scale
// once: y += scale * sum.  No tensor cores, no atomics; reductions run in a fixed order so results are reproducible
// run to run and independent of where the weight bytes live (resident region or staging slot).
#include "ats_internal.h"
#include "sm100_sync.cuh"
#include "attn_decode_body.cuh"

namespace ats {

// ------------------------------------------------------------------------------------------- helpers
__device__ __forceinline__ __half2 u32_as_half2(uint32_t v) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = v;
  return h;
}

// One 32-bit word of the internal format -> 8 exact fp16 codes as the pairs (k0,k1) (k2,k3) (k4,k5) (k6,k7).
// Nibble u = code + 8.  (w & 0x000F000F) | 0x6400 is the fp16 pair 1024 + u; the 0x00F000F0 pair is 1024 + 16u.
__device__ __forceinline__ void unpack8(uint32_t w, __half2 (&c)[4]) {
  const uint32_t kMagic = 0x64006400u;
  const __half2 k1032 = u32_as_half2(0x64086408u);   // 1032
  const __half2 k16th = u32_as_half2(0x2C002C00u);   // 1/16
  const __half2 kM72 = u32_as_half2(0xD480D480u);    // -72 = -(1024/16 + 8)
  const uint32_t w8 = w >> 8;
  c[0] = __hsub2(u32_as_half2((w & 0x000F000Fu) | kMagic), k1032);
  c[1] = __hfma2(u32_as_half2((w & 0x00F000F0u) | kMagic), k16th, kM72);
  c[2] = __hsub2(u32_as_half2((w8 & 0x000F000Fu) | kMagic), k1032);
  c[3] = __hfma2(u32_as_half2((w8 & 0x00F000F0u) | kMagic), k16th, kM72);
}

// The microscaling 4-bit float (1 sign, 2 exponent bits with bias 1, 1 mantissa bit; exponent 0 is subnormal) in the same
// word layout.  The three magnitude bits placed at bits 11..9 of an fp16 (the two low exponent bits and the top mantissa
// bit) read as the element times 2^-14, subnormal case included, since both formats treat exponent field 0 the same way;
// one multiplication by 2^14 (exact) gives the element.  Pair j sits in nibbles j and j + 4.
__device__ __forceinline__ void unpack8_mx(uint32_t w, __half2 (&c)[4]) {
  const __half2 k2p14 = u32_as_half2(0x74007400u);  // 16384
  const uint32_t kMag = 0x0E000E00u, kSgn = 0x80008000u;
  c[0] = __hmul2(u32_as_half2(((w << 9) & kMag) | ((w << 12) & kSgn)), k2p14);
  c[1] = __hmul2(u32_as_half2(((w << 5) & kMag) | ((w << 8) & kSgn)), k2p14);
  c[2] = __hmul2(u32_as_half2(((w << 1) & kMag) | ((w << 4) & kSgn)), k2p14);
  c[3] = __hmul2(u32_as_half2(((w >> 3) & kMag) | (w & kSgn)), k2p14);
}
// 8 exact fp16 element values of one word in either 4-bit format (mx: uniform over the launch)
__device__ __forceinline__ void unpack8_any(uint32_t w, __half2 (&c)[4], int mx) {
  if (mx) unpack8_mx(w, c);
  else unpack8(w, c);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.0f + expf(-g)) * u; }

// ------------------------------------------------------------------------------------------- dequantize (a1)
template <bool F16>
__global__ void dequant_kernel(const uint8_t* __restrict__ slice, int n_rows, int K, void* __restrict__ out, int mx) {
  const uint64_t words = (uint64_t)n_rows * K / 8;
  const uint32_t* codes = reinterpret_cast<const uint32_t*>(slice);
  const __half* scales = reinterpret_cast<const __half*>(slice + (uint64_t)n_rows * K / 2);
  for (uint64_t w = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; w < words; w += (uint64_t)gridDim.x * blockDim.x) {
    __half2 c[4];
    unpack8_any(codes[w], c, mx);
    const __half s = scales[w / 4];  // 4 words per block of 32
    if (F16) {
      const __half2 s2 = __half2half2(s);
      uint4 o;
      __half2 r0 = __hmul2(c[0], s2), r1 = __hmul2(c[1], s2), r2 = __hmul2(c[2], s2), r3 = __hmul2(c[3], s2);
      o.x = *reinterpret_cast<uint32_t*>(&r0);
      o.y = *reinterpret_cast<uint32_t*>(&r1);
      o.z = *reinterpret_cast<uint32_t*>(&r2);
      o.w = *reinterpret_cast<uint32_t*>(&r3);
      reinterpret_cast<uint4*>(out)[w] = o;
    } else {
      const float sf = __half2float(s);
      float4 a, b;
      float2 f;
      f = __half22float2(c[0]); a.x = sf * f.x; a.y = sf * f.y;
      f = __half22float2(c[1]); a.z = sf * f.x; a.w = sf * f.y;
      f = __half22float2(c[2]); b.x = sf * f.x; b.y = sf * f.y;
      f = __half22float2(c[3]); b.z = sf * f.x; b.w = sf * f.y;
      reinterpret_cast<float4*>(out)[2 * w] = a;
      reinterpret_cast<float4*>(out)[2 * w + 1] = b;
    }
  }
}

// Embedding lookup: out[m] = rn16(scale * code) of row ids[m] of a Q4B32 table (the fp16 form ats_dequantize writes).
// One thread per code word; ids outside [0, n_rows) give a row of zeros and raise the status word.
__global__ void embed_rows_kernel(const uint8_t* __restrict__ slice, int n_rows, int K, const int32_t* __restrict__ ids, int M,
                                  __half* __restrict__ out, int* __restrict__ status, int mx) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the ids may come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int wpr = K / 8;  // words per row
  const uint32_t* codes = reinterpret_cast<const uint32_t*>(slice);
  const __half* scales = reinterpret_cast<const __half*>(slice + (uint64_t)n_rows * K / 2);
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < (uint64_t)M * wpr; i += (uint64_t)gridDim.x * blockDim.x) {
    const int m = (int)(i / wpr), w = (int)(i % wpr);
    const int row = ids[m];
    uint4 o = make_uint4(0, 0, 0, 0);
    if (row >= 0 && row < n_rows) {
      __half2 c[4];
      unpack8_any(codes[(uint64_t)row * wpr + w], c, mx);
      const __half2 s2 = __half2half2(scales[(uint64_t)row * (K / 32) + w / 4]);
      __half2 r0 = __hmul2(c[0], s2), r1 = __hmul2(c[1], s2), r2 = __hmul2(c[2], s2), r3 = __hmul2(c[3], s2);
      o.x = *reinterpret_cast<uint32_t*>(&r0);
      o.y = *reinterpret_cast<uint32_t*>(&r1);
      o.z = *reinterpret_cast<uint32_t*>(&r2);
      o.w = *reinterpret_cast<uint32_t*>(&r3);
    } else if (w == 0) {
      raise_status(status, 6);
    }
    reinterpret_cast<uint4*>(out)[i] = o;
  }
}

cudaError_t launch_embed_rows(const uint8_t* slice, int n_rows, int K, const int32_t* ids, int M, __half* out, int* status,
                              int mx, cudaStream_t st, uint64_t* n_launch, int pdl) {
  const uint64_t words = (uint64_t)M * K / 8;
  const int grid = (int)std::min<uint64_t>((words + 255) / 256, 148 * 8);
  ++*n_launch;
  return launch_dep(embed_rows_kernel, dim3(grid), dim3(256), 0, st, pdl, 1, slice, n_rows, K, ids, M, out, status, mx);
}

cudaError_t launch_dequant(const uint8_t* slice, int n_rows, int K, void* out, int out_f16, int mx, cudaStream_t st,
                           uint64_t* n_launch) {
  const uint64_t words = (uint64_t)n_rows * K / 8;
  const int block = 256;
  const int grid = (int)std::min<uint64_t>((words + block - 1) / block, 148 * 16);
  if (out_f16)
    dequant_kernel<true><<<grid, block, 0, st>>>(slice, n_rows, K, out, mx);
  else
    dequant_kernel<false><<<grid, block, 0, st>>>(slice, n_rows, K, out, mx);
  ++*n_launch;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------- fp16-weight GEMV
// The per-tensor operator for unquantized fp16 matrices W [N][K], M <= 8 rows of x, with the epilogues of the quantized
// GEMV (plain, + residual, SwiGLU of two matrices) and up to three matrices side by side (fused QKV).  HBM-bound at 2 bytes
// per weight: a warp owns two weight rows at a time (two outputs; for SwiGLU the gate row and the up row of one output), its
// lanes walk K in 16-byte pieces with eight weight loads in flight per thread (streaming loads: every weight is used once); x
// comes through L1.  Products of fp16 values are exact in fp32; sums in fp32, lanes combined by shuffles in fixed order.
struct W16Params {
  const __half* w[3];
  int n_rows[3];
  int n_seg, K, mode;
  const __half* x;
  int ldx;
  float* y32;
  __half* y16;
  int ldy;
  const float* res32;
  const __half* res16;
  int ldres;
  int ksplit;  // warps that share one pair of rows, each on its own part of K: 1, 2, 4 or 8
};
template <int M>
__global__ void __launch_bounds__(256) gemv_w16_kernel(const W16Params p) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  bool waited = false;  // x and the residual come from the preceding kernel; the first weight loads need not wait for it
  __shared__ float red_s[8][2][M];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int K = p.K, nch = K / 8;  // 16-byte pieces per row
  const bool sw = p.mode == GEMV_SWIGLU_F16;
  int n_rows = 0;  // weight rows side by side (SwiGLU: outputs, each fed by one gate row and one up row)
  if (sw) n_rows = p.n_rows[0];
  else n_rows = p.n_rows[0] + (p.n_seg > 1 ? p.n_rows[1] : 0) + (p.n_seg > 2 ? p.n_rows[2] : 0);
  auto row_ptr = [&](int r) {  // constant indices only: a runtime index would move the parameters to local memory
    const __half* base = p.w[0];
    if (p.n_seg > 1 && r >= p.n_rows[0]) {
      r -= p.n_rows[0];
      base = p.w[1];
      if (p.n_seg > 2 && r >= p.n_rows[1]) {
        r -= p.n_rows[1];
        base = p.w[2];
      }
    }
    return reinterpret_cast<const uint4*>(base + (size_t)r * K);
  };
  auto dot8 = [](const uint4& a, const uint4& b, float acc) {
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 fa = __half22float2(u32_as_half2(aw[q])), fb = __half22float2(u32_as_half2(bw[q]));
      acc = fmaf(fa.x, fb.x, acc);
      acc = fmaf(fa.y, fb.y, acc);
    }
    return acc;
  };
  // A unit is two weight rows: two neighbouring output rows, or the gate and up rows of one SwiGLU output.  `ksplit`
  // warps share a unit, each taking one contiguous part of K (few rows would otherwise leave every warp a long serial
  // walk with one batch of loads in flight at a time); the CTA's 8 warps hold 8 / ksplit units.
  const int n_units = sw ? n_rows : (n_rows + 1) / 2;
  const int ks = p.ksplit, upc = 8 / ks;  // units per CTA and round
  const int part = w % ks, slot = w / ks;
  const int per = (((nch + ks - 1) / ks) + 31) & ~31;  // pieces per part (whole 512-byte lines)
  const int c_lo = part * per, c_hi = min(nch, c_lo + per);
  for (int u0 = blockIdx.x * upc; u0 < n_units; u0 += gridDim.x * upc) {
    const int u = u0 + slot;
    const bool live = u < n_units;
    const int r0 = sw ? u : 2 * u, r1 = sw ? u : min(r0 + 1, n_rows - 1);
    float acc[2][M];
#pragma unroll
    for (int m = 0; m < M; ++m) acc[0][m] = acc[1][m] = 0.f;
    if (live) {
      const uint4* w0 = sw ? reinterpret_cast<const uint4*>(p.w[0] + (size_t)r0 * K) : row_ptr(r0);
      const uint4* w1 = sw ? reinterpret_cast<const uint4*>(p.w[1] + (size_t)r0 * K) : row_ptr(r1);
      for (int c0 = c_lo + lane; c0 < c_hi; c0 += 128) {
        uint4 a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = c0 + 32 * i;
          a[i] = c < c_hi ? __ldcs(w0 + c) : make_uint4(0, 0, 0, 0);
          b[i] = c < c_hi ? __ldcs(w1 + c) : make_uint4(0, 0, 0, 0);
        }
        if (!waited) {
          asm volatile("griddepcontrol.wait;" ::: "memory");
          waited = true;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = c0 + 32 * i;
          if (c < c_hi) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
              const uint4 xv = __ldg(reinterpret_cast<const uint4*>(p.x + (size_t)m * p.ldx) + c);
              acc[0][m] = dot8(a[i], xv, acc[0][m]);
              acc[1][m] = dot8(b[i], xv, acc[1][m]);
            }
          }
        }
      }
    }
    if (!waited) {  // no piece for this lane
      asm volatile("griddepcontrol.wait;" ::: "memory");
      waited = true;
    }
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const float s0 = warp_sum(acc[0][m]), s1 = warp_sum(acc[1][m]);
      if (lane == 0) {
        red_s[w][0][m] = s0;
        red_s[w][1][m] = s1;
      }
    }
    __syncthreads();
    // one thread per (unit, row of the pair, activation row) adds the parts in fixed order and writes the output
    if (threadIdx.x < upc * 2 * M) {
      const int m = threadIdx.x % M, h = (threadIdx.x / M) & 1, sl = threadIdx.x / (2 * M);
      const int uu = u0 + sl;
      float s = 0.f, s_up = 0.f;
      for (int q = 0; q < ks; ++q) {
        s += red_s[sl * ks + q][sw ? 0 : h][m];
        if (sw) s_up += red_s[sl * ks + q][1][m];
      }
      const int r = sw ? uu : 2 * uu + h;
      if (uu < n_units && r < n_rows && !(sw && h)) {
        const size_t o = (size_t)m * p.ldy + r, ro = (size_t)m * p.ldres + r;
        switch (p.mode) {
          case GEMV_OUT_F32: p.y32[o] = s; break;
          case GEMV_OUT_F16: p.y16[o] = __float2half_rn(s); break;
          case GEMV_RES16_OUT_F32: p.y32[o] = __half2float(p.res16[ro]) + s; break;
          case GEMV_RES32_OUT_F16: p.y16[o] = __float2half_rn(p.res32[ro] + s); break;
          case GEMV_RES16_OUT_F16: p.y16[o] = __float2half_rn(__half2float(p.res16[ro]) + s); break;
          case GEMV_SWIGLU_F16: p.y16[o] = __float2half_rn(silu_mul(s, s_up)); break;
          default: break;
        }
      }
    }
    __syncthreads();
  }
  if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
}

cudaError_t launch_gemv_w16(const GemvParams& g, cudaStream_t st, uint64_t* n_launch) {
  if (g.M < 1 || g.M > 8 || g.K % 8 || g.n_seg < 1 || g.n_seg > 3) return cudaErrorInvalidValue;
  W16Params p{};
  int n_out = 0;
  for (int s = 0; s < g.n_seg; ++s) {
    p.w[s] = reinterpret_cast<const __half*>(g.seg[s].base);
    p.n_rows[s] = g.seg[s].n_rows;
    n_out += g.seg[s].n_rows;
  }
  if (g.mode == GEMV_SWIGLU_F16) {
    if (g.n_seg != 2 || g.seg[0].n_rows != g.seg[1].n_rows) return cudaErrorInvalidValue;
    n_out = g.seg[0].n_rows;
  }
  p.n_seg = g.n_seg; p.K = g.K; p.mode = g.mode;
  p.x = g.x; p.ldx = g.ldx; p.y32 = g.y32; p.y16 = g.y16; p.ldy = g.ldy;
  p.res32 = g.res32; p.res16 = g.res16; p.ldres = g.ldres;
  const int n_units = g.mode == GEMV_SWIGLU_F16 ? n_out : (n_out + 1) / 2;
  // Split K while the units alone give fewer warps than the machine holds (4 CTAs of 8 warps per SM) and every part keeps
  // at least one full pass of a warp (128 pieces of 16 bytes).  A function of the shapes only.
  int ks = 1;
  while (ks < 8 && (long)n_units * ks <= 2 * 148L * 32 && (g.K / 8) / (ks * 2) >= 128) ks *= 2;
  p.ksplit = ks;
  const int upc = 8 / ks;
  const dim3 grid(std::max(1, std::min((n_units + upc - 1) / upc, 148 * 8))), block(256);
  ++*n_launch;
  switch (g.M) {
    case 1: return launch_dep(gemv_w16_kernel<1>, grid, block, 0, st, g.pdl, 1, p);
    case 2: return launch_dep(gemv_w16_kernel<2>, grid, block, 0, st, g.pdl, 1, p);
    case 3: return launch_dep(gemv_w16_kernel<3>, grid, block, 0, st, g.pdl, 1, p);
    case 4: return launch_dep(gemv_w16_kernel<4>, grid, block, 0, st, g.pdl, 1, p);
    case 5: return launch_dep(gemv_w16_kernel<5>, grid, block, 0, st, g.pdl, 1, p);
    case 6: return launch_dep(gemv_w16_kernel<6>, grid, block, 0, st, g.pdl, 1, p);
    case 7: return launch_dep(gemv_w16_kernel<7>, grid, block, 0, st, g.pdl, 1, p);
    default: return launch_dep(gemv_w16_kernel<8>, grid, block, 0, st, g.pdl, 1, p);
  }
}

// ------------------------------------------------------------------------------------------- GEMV core (a2, a5)
constexpr int kGemvMaxWarps = 8;
constexpr int kWR = 4;  // weight rows a CTA works on at once

// Accumulate WR weight rows against M activation rows over the blocks this thread owns.
// cptr[i]: row i's codes as uint4 (one per block of 32); sptr[i]: row i's scales.
template <int M>
__device__ __forceinline__ void gemv_accumulate(const uint4* const (&cptr)[kWR], const __half* const (&sptr)[kWR],
                                                const bool (&valid)[kWR], const __half* __restrict__ x, int ldx, int nblk,
                                                float (&acc)[kWR][M], int mx) {
  const int nthreads = blockDim.x;
  for (int blk = threadIdx.x; blk < nblk; blk += nthreads) {
    uint4 q[kWR];
    float s[kWR];
#pragma unroll
    for (int i = 0; i < kWR; ++i) {
      if (valid[i]) {
        q[i] = __ldg(cptr[i] + blk);
        s[i] = __half2float(sptr[i][blk]);
      } else {
        q[i] = mx ? make_uint4(0, 0, 0, 0) : make_uint4(0x88888888u, 0x88888888u, 0x88888888u, 0x88888888u);
        s[i] = 0.f;
      }
    }
    float part[kWR][M];
#pragma unroll
    for (int i = 0; i < kWR; ++i)
#pragma unroll
      for (int m = 0; m < M; ++m) part[i][m] = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float xf[M][8];
#pragma unroll
      for (int m = 0; m < M; ++m) {
        const uint4 xv = __ldg(reinterpret_cast<const uint4*>(x + (size_t)m * ldx + (size_t)blk * 32 + j * 8));
        float2 f;
        f = __half22float2(u32_as_half2(xv.x)); xf[m][0] = f.x; xf[m][1] = f.y;
        f = __half22float2(u32_as_half2(xv.y)); xf[m][2] = f.x; xf[m][3] = f.y;
        f = __half22float2(u32_as_half2(xv.z)); xf[m][4] = f.x; xf[m][5] = f.y;
        f = __half22float2(u32_as_half2(xv.w)); xf[m][6] = f.x; xf[m][7] = f.y;
      }
#pragma unroll
      for (int i = 0; i < kWR; ++i) {
        const uint32_t word = j == 0 ? q[i].x : j == 1 ? q[i].y : j == 2 ? q[i].z : q[i].w;
        __half2 c[4];
        unpack8_any(word, c, mx);
        float cf[8];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const float2 f = __half22float2(c[t]);
          cf[2 * t] = f.x;
          cf[2 * t + 1] = f.y;
        }
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
          for (int t = 0; t < 8; ++t) part[i][m] = fmaf(cf[t], xf[m][t], part[i][m]);
      }
    }
#pragma unroll
    for (int i = 0; i < kWR; ++i)
#pragma unroll
      for (int m = 0; m < M; ++m) acc[i][m] = fmaf(s[i], part[i][m], acc[i][m]);
  }
}

// Sum acc over the CTA in a fixed order (lanes by butterfly, warps ascending); the totals land in tot[] (shared).
template <int M>
__device__ __forceinline__ void gemv_reduce(float (&acc)[kWR][M], float* red /*[kGemvMaxWarps][kWR*M]*/, float* tot /*[kWR*M]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
#pragma unroll
  for (int i = 0; i < kWR; ++i)
#pragma unroll
    for (int m = 0; m < M; ++m) {
      const float v = warp_sum(acc[i][m]);
      if (lane == 0) red[warp * (kWR * M) + i * M + m] = v;
    }
  __syncthreads();
  if (threadIdx.x < kWR * M) {
    float t = 0.f;
    for (int w = 0; w < nwarps; ++w) t += red[w * (kWR * M) + threadIdx.x];
    tot[threadIdx.x] = t;
  }
  __syncthreads();
}

template <int M, bool SW>
__global__ void __launch_bounds__(kGemvMaxWarps * 32) gemv_kernel(const GemvParams p) {
  __shared__ float red[kGemvMaxWarps * kWR * M];
  __shared__ float tot[kWR * M];
  const int K = p.K, nblk = K / 32;
  const uint4* cptr[kWR];
  const __half* sptr[kWR];
  bool valid[kWR];
  int orow[kWR];  // output row (global, across segments)
#pragma unroll
  for (int i = 0; i < kWR; ++i) {
    int s, r;
    if (SW) {
      s = i & 1;
      r = blockIdx.x * (kWR / 2) + (i >> 1);
      valid[i] = r < p.seg[0].n_rows;
      orow[i] = r;
    } else {
      r = blockIdx.x * kWR + i;
      orow[i] = r;
      s = 0;
      while (s < p.n_seg - 1 && r >= p.seg[s].n_rows) {
        r -= p.seg[s].n_rows;
        ++s;
      }
      valid[i] = r < p.seg[s].n_rows;
    }
    const uint8_t* base = p.seg[s].base;
    cptr[i] = reinterpret_cast<const uint4*>(base + (size_t)r * (K / 2));
    sptr[i] = reinterpret_cast<const __half*>(base + (size_t)p.seg[s].n_rows * (K / 2)) + (size_t)r * nblk;
  }
  float acc[kWR][M];
#pragma unroll
  for (int i = 0; i < kWR; ++i)
#pragma unroll
    for (int m = 0; m < M; ++m) acc[i][m] = 0.f;
  gemv_accumulate<M>(cptr, sptr, valid, p.x, p.ldx, nblk, acc, p.mx);
  gemv_reduce<M>(acc, red, tot);

  if (SW) {
    if (threadIdx.x < (kWR / 2) * M) {
      const int i2 = threadIdx.x / M, m = threadIdx.x % M;
      const int row = blockIdx.x * (kWR / 2) + i2;
      if (row < p.seg[0].n_rows) {
        const float g = tot[(2 * i2) * M + m], u = tot[(2 * i2 + 1) * M + m];
        p.y16[(size_t)m * p.ldy + row] = __float2half_rn(silu_mul(g, u));
      }
    }
    return;
  }
  if (threadIdx.x < kWR * M) {
    const int i = threadIdx.x / M, m = threadIdx.x % M;
    // valid[]/orow[] are per-thread copies of the same values; recompute validity for row i
    int r = blockIdx.x * kWR + i, total = 0;
    for (int s = 0; s < p.n_seg; ++s) total += p.seg[s].n_rows;
    if (r < total) {
      const float v = tot[i * M + m];
      const size_t o = (size_t)m * p.ldy + r;
      switch (p.mode) {
        case GEMV_OUT_F32: p.y32[o] = v; break;
        case GEMV_OUT_F16: p.y16[o] = __float2half_rn(v); break;
        case GEMV_RES16_OUT_F32: p.y32[o] = __half2float(p.res16[(size_t)m * p.ldres + r]) + v; break;
        case GEMV_RES32_OUT_F16: p.y16[o] = __float2half_rn(p.res32[(size_t)m * p.ldres + r] + v); break;
        case GEMV_RES16_OUT_F16: p.y16[o] = __float2half_rn(__half2float(p.res16[(size_t)m * p.ldres + r]) + v); break;
        default: break;
      }
    }
  }
}

static int gemv_threads(int K) {
  const int nblk = K / 32;
  int warps = (nblk + 31) / 32;
  warps = std::max(1, std::min(warps, kGemvMaxWarps));
  return warps * 32;
}

template <int M>
static void launch_gemv_m(const GemvParams& p, int grid, int block, cudaStream_t st) {
  if (p.mode == GEMV_SWIGLU_F16)
    gemv_kernel<M, true><<<grid, block, 0, st>>>(p);
  else
    gemv_kernel<M, false><<<grid, block, 0, st>>>(p);
}

cudaError_t launch_gemv(const GemvParams& p, cudaStream_t st, uint64_t* n_launch) {
  int total = 0;
  for (int s = 0; s < p.n_seg; ++s) total += p.seg[s].n_rows;
  const bool sw = p.mode == GEMV_SWIGLU_F16;
  const int rows_per_cta = sw ? kWR / 2 : kWR;
  const int out_rows = sw ? p.seg[0].n_rows : total;
  const int grid = (out_rows + rows_per_cta - 1) / rows_per_cta;
  const int block = gemv_threads(p.K);
  switch (p.M) {
    case 1: launch_gemv_m<1>(p, grid, block, st); break;
    case 2: launch_gemv_m<2>(p, grid, block, st); break;
    case 3: launch_gemv_m<3>(p, grid, block, st); break;
    case 4: launch_gemv_m<4>(p, grid, block, st); break;
    case 5: launch_gemv_m<5>(p, grid, block, st); break;
    case 6: launch_gemv_m<6>(p, grid, block, st); break;
    case 7: launch_gemv_m<7>(p, grid, block, st); break;
    case 8: launch_gemv_m<8>(p, grid, block, st); break;
    default: return cudaErrorInvalidValue;
  }
  ++*n_launch;
  return cudaGetLastError();
}

// Grouped-expert GEMV: blockIdx.y = job (one (token, slot) pair), blockIdx.x = row group of that expert's matrix.
template <bool SW, bool EXPLICIT>
__global__ void __launch_bounds__(kGemvMaxWarps * 32)
    moe_gemv_kernel(const MoeGemvParams p, const __grid_constant__ MoeJobs jobs) {
  __shared__ float red[kGemvMaxWarps * kWR];
  __shared__ float tot[kWR];
  const int job = blockIdx.y;
  const uint8_t *b0, *b1;
  int xrow, out_row;
  if (EXPLICIT) {
    b0 = jobs.w0[job];
    b1 = jobs.w1[job];
    xrow = jobs.xrow[job];
    out_row = jobs.orow[job];
  } else {
    int e = p.ids[job];
    if ((unsigned)e >= (unsigned)p.n_experts) {  // an id that names no expert: expert 0 stands in and the status word says so
      if (threadIdx.x == 0 && blockIdx.x == 0) raise_status(p.status, 7);
      e = 0;
    }
    b0 = p.base0 + (size_t)e * p.stride;
    b1 = SW ? p.base1 + (size_t)e * p.stride : nullptr;
    xrow = job / p.x_div;
    out_row = job;
  }
  const int K = p.K, nblk = K / 32, N = p.n_rows;
  const uint4* cptr[kWR];
  const __half* sptr[kWR];
  bool valid[kWR];
#pragma unroll
  for (int i = 0; i < kWR; ++i) {
    const int r = SW ? blockIdx.x * (kWR / 2) + (i >> 1) : blockIdx.x * kWR + i;
    const uint8_t* base = (SW && (i & 1)) ? b1 : b0;
    valid[i] = r < N;
    cptr[i] = reinterpret_cast<const uint4*>(base + (size_t)r * (K / 2));
    sptr[i] = reinterpret_cast<const __half*>(base + (size_t)N * (K / 2)) + (size_t)r * nblk;
  }
  float acc[kWR][1];
#pragma unroll
  for (int i = 0; i < kWR; ++i) acc[i][0] = 0.f;
  gemv_accumulate<1>(cptr, sptr, valid, p.x + (size_t)xrow * p.ldx, p.ldx, nblk, acc, p.mx);
  gemv_reduce<1>(acc, red, tot);
  if (SW) {
    if (threadIdx.x < kWR / 2) {
      const int row = blockIdx.x * (kWR / 2) + threadIdx.x;
      if (row < N)
        p.y16[(size_t)out_row * p.ldy + row] = __float2half_rn(silu_mul(tot[2 * threadIdx.x], tot[2 * threadIdx.x + 1]));
    }
  } else if (threadIdx.x < kWR) {
    const int row = blockIdx.x * kWR + threadIdx.x;
    if (row < N) {
      if (p.mode == GEMV_OUT_F32)
        p.y32[(size_t)out_row * p.ldy + row] = tot[threadIdx.x];
      else
        p.y16[(size_t)out_row * p.ldy + row] = __float2half_rn(tot[threadIdx.x]);
    }
  }
}

cudaError_t launch_moe_gemv(const MoeGemvParams& p, const MoeJobs* jobs, cudaStream_t st, uint64_t* n_launch) {
  const bool sw = p.mode == GEMV_SWIGLU_F16;
  const int rows_per_cta = sw ? kWR / 2 : kWR;
  const int gx = (p.n_rows + rows_per_cta - 1) / rows_per_cta;
  const int block = gemv_threads(p.K);
  if (jobs) {
    dim3 grid(gx, jobs->n);
    if (sw)
      moe_gemv_kernel<true, true><<<grid, block, 0, st>>>(p, *jobs);
    else
      moe_gemv_kernel<false, true><<<grid, block, 0, st>>>(p, *jobs);
  } else {
    static const MoeJobs none{};
    dim3 grid(gx, p.P);
    if (sw)
      moe_gemv_kernel<true, false><<<grid, block, 0, st>>>(p, none);
    else
      moe_gemv_kernel<false, false><<<grid, block, 0, st>>>(p, none);
  }
  ++*n_launch;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------- RMSNorm (a6)
template <typename TIn>
__device__ __forceinline__ float load_f(const TIn* p, size_t i);
template <>
__device__ __forceinline__ float load_f<float>(const float* p, size_t i) { return p[i]; }
template <>
__device__ __forceinline__ float load_f<__half>(const __half* p, size_t i) { return __half2float(p[i]); }

template <typename TIn>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const TIn* __restrict__ x, const __half* __restrict__ gain,
                                                      __half* __restrict__ out, int H, float eps) {
  __shared__ float red[8];
  __shared__ float inv_s;
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const TIn* xr = x + (size_t)blockIdx.x * H;
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    const float v = load_f<TIn>(xr, i);
    ss = fmaf(v, v, ss);
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    inv_s = 1.0f / sqrtf(t / (float)H + eps);
  }
  __syncthreads();
  const float inv = inv_s;
  for (int i = threadIdx.x; i < H; i += blockDim.x)
    out[(size_t)blockIdx.x * H + i] = __float2half_rn(load_f<TIn>(xr, i) * __half2float(gain[i]) * inv);
}

// fp16 rows of up to 8192 elements, eight per 16-byte access, held in registers between the two passes
__global__ void __launch_bounds__(256) rmsnorm16_vec_kernel(const __half* __restrict__ x, const __half* __restrict__ gain,
                                                            __half* __restrict__ out, int H, float eps) {
  __shared__ float red[8];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n8 = H / 8;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)blockIdx.x * H);
  uint4 xv[4], gv[4];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = threadIdx.x + 256 * j;
    xv[j] = make_uint4(0, 0, 0, 0);
    gv[j] = make_uint4(0, 0, 0, 0);
    if (c < n8) {
      xv[j] = xr[c];
      gv[j] = __ldg(reinterpret_cast<const uint4*>(gain) + c);
    }
    const uint32_t w[4] = {xv[j].x, xv[j].y, xv[j].z, xv[j].w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 f = __half22float2(u32_as_half2(w[q]));
      ss = fmaf(f.x, f.x, ss);
      ss = fmaf(f.y, f.y, ss);
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) t += red[w];
  const float inv = 1.0f / sqrtf(t / (float)H + eps);
  uint4* orow = reinterpret_cast<uint4*>(out + (size_t)blockIdx.x * H);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = threadIdx.x + 256 * j;
    if (c < n8) {
      const uint32_t w[4] = {xv[j].x, xv[j].y, xv[j].z, xv[j].w}, g[4] = {gv[j].x, gv[j].y, gv[j].z, gv[j].w};
      uint32_t o[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 f = __half22float2(u32_as_half2(w[q])), gg = __half22float2(u32_as_half2(g[q]));
        const __half2 h = __floats2half2_rn(f.x * gg.x * inv, f.y * gg.y * inv);
        o[q] = *reinterpret_cast<const uint32_t*>(&h);
      }
      orow[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// The same for fp32 rows (the residual stream between the two halves of a decode layer): eight elements per thread and
// pass as two 16-byte loads, held in registers between the passes.
__global__ void __launch_bounds__(256) rmsnorm32_vec_kernel(const float* __restrict__ x, const __half* __restrict__ gain,
                                                            __half* __restrict__ out, int H, float eps) {
  __shared__ float red[8];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int n8 = H / 8;
  const float4* xr = reinterpret_cast<const float4*>(x + (size_t)blockIdx.x * H);
  float4 xa[4], xb[4];
  uint4 gv[4];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = threadIdx.x + 256 * j;
    xa[j] = xb[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    gv[j] = make_uint4(0, 0, 0, 0);
    if (c < n8) {
      xa[j] = xr[2 * c];
      xb[j] = xr[2 * c + 1];
      gv[j] = __ldg(reinterpret_cast<const uint4*>(gain) + c);
    }
    ss = fmaf(xa[j].x, xa[j].x, ss); ss = fmaf(xa[j].y, xa[j].y, ss); ss = fmaf(xa[j].z, xa[j].z, ss); ss = fmaf(xa[j].w, xa[j].w, ss);
    ss = fmaf(xb[j].x, xb[j].x, ss); ss = fmaf(xb[j].y, xb[j].y, ss); ss = fmaf(xb[j].z, xb[j].z, ss); ss = fmaf(xb[j].w, xb[j].w, ss);
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) t += red[w];
  const float inv = 1.0f / sqrtf(t / (float)H + eps);
  uint4* orow = reinterpret_cast<uint4*>(out + (size_t)blockIdx.x * H);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = threadIdx.x + 256 * j;
    if (c < n8) {
      const float f[8] = {xa[j].x, xa[j].y, xa[j].z, xa[j].w, xb[j].x, xb[j].y, xb[j].z, xb[j].w};
      const uint32_t g[4] = {gv[j].x, gv[j].y, gv[j].z, gv[j].w};
      uint32_t o[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 gg = __half22float2(u32_as_half2(g[q]));
        const __half2 h = __floats2half2_rn(f[2 * q] * gg.x * inv, f[2 * q + 1] * gg.y * inv);
        o[q] = *reinterpret_cast<const uint32_t*>(&h);
      }
      orow[c] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

cudaError_t launch_rmsnorm(const void* x, int x_is_f32, const __half* gain, __half* out, int M, int H, float eps,
                           cudaStream_t st, uint64_t* n_launch, int pdl) {
  ++*n_launch;
  if (!x_is_f32 && H % 8 == 0 && H <= 8192 &&
      (((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(gain) | reinterpret_cast<uintptr_t>(out)) & 15) == 0))
    return launch_dep(rmsnorm16_vec_kernel, dim3(M), dim3(256), 0, st, pdl, 1, (const __half*)x, gain, out, H, eps);
  if (x_is_f32 && H % 8 == 0 && H <= 8192 &&
      (((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(gain) | reinterpret_cast<uintptr_t>(out)) & 15) == 0))
    return launch_dep(rmsnorm32_vec_kernel, dim3(M), dim3(256), 0, st, pdl, 1, (const float*)x, gain, out, H, eps);
  if (x_is_f32) return launch_dep(rmsnorm_kernel<float>, dim3(M), dim3(256), 0, st, pdl, 1, (const float*)x, gain, out, H, eps);
  return launch_dep(rmsnorm_kernel<__half>, dim3(M), dim3(256), 0, st, pdl, 1, (const __half*)x, gain, out, H, eps);
}

// ------------------------------------------------------------------------------------------- fused decode attention
// One launch does the rotary embedding of q and of the new key (half-split pairs, angle pos * theta^(-2i/d), the
// cos/sin table for `pos` computed on the host in fp64 and passed by value), appends the new K/V row to the caches as
// fp16, attends over positions 0..pos split across CTAs, and merges the splits: the last CTA to finish a kv head
// (a counter in global memory, reset for the next launch) sums the partials in ascending split order, so the result
// does not depend on which CTA arrives last.
// CTA (split, kv head) covers 64 positions for ALL query heads of the group: the K and V rows are staged once in shared
// memory (16-byte async copies, issued before the grid dependency resolves) and every head's warps read them from
// there, so the cache crosses the L2-to-SM fabric once instead of once per query head; that traffic, not DRAM, bounds
// this kernel.  Warp (head, sub-block) owns 32 positions, one per lane.
// Positions per CTA: 64, or 128 for contexts beyond 1024 so that the final merge still reads all splits of a head in
// one round trip (16 splits) up to 2048 positions.  (64 positions up to 2048, with both kernels' registers capped so that
// a CTA of this kernel fits an SM beside a CTA of the streaming GEMV, was measured and lost: the GEMV slows down by 0.5 us
// per launch at 80 registers and this kernel by 2.9 us with 17 splits to merge, and nothing is gained back.)
// (A tensor-core form, scores as Q K^T and outputs as V^T P^T by mma.sync m16n8k16 with the group's heads as operand rows,
// was built and measured in the step: 7.6 us with the query and the weights rounded to fp16, which costs accuracy the
// layer's end-to-end gate does not have to spare, and 8.2 us with both split into hi + lo fp16 pairs that keep fp32
// accuracy, against 7.7 us for this form.  The launch is a chain of global round trips (query load, partial store and
// arrival counter, partial loads of the merge), each about a microsecond at one CTA per SM; the arithmetic between
// them is not what it waits for.)
int attn_decode_pos_per_cta(int n_ctx) { return n_ctx <= 1024 ? 64 : 128; }
int attn_decode_splits(int n_ctx) {
  const int pc = attn_decode_pos_per_cta(n_ctx);
  return (n_ctx + pc - 1) / pc;
}
size_t attn_decode_scratch_floats(int n_q, int d, int n_ctx) {
  return (size_t)n_q * ((n_ctx + 63) / 64 + 1) * (d + 2);  // enough for 64 positions per CTA at any context up to n_ctx
}

template <int D, int SUB>
__global__ void __launch_bounds__(512) attn_decode_fused_kernel(const AttnDecodeParams p) {
  extern __shared__ __align__(16) uint8_t dyn_s[];
  __shared__ AttnShared as;
  attn_decode_body<D, SUB, true>(p, (int)blockIdx.x, (int)blockIdx.y, (int)gridDim.x, (int)threadIdx.x, (int)blockDim.x, dyn_s, as);
}

cudaError_t launch_attn_decode_fused(AttnDecodeParams p, int d, int pdl, cudaStream_t st, uint64_t* n_launch) {
  if (p.group < 1 || p.group > kAttnMaxGroup || p.n_q != p.n_kv * p.group) return cudaErrorInvalidValue;
  int pc = attn_decode_pos_per_cta(p.pos + 1);
  if (p.group * pc > 512) pc = 64;  // large groups: 64 positions keep the CTA within 512 threads
  const int splits = (p.pos + 1 + pc - 1) / pc;
  // Short contexts give fewer jobs than SMs: the query heads of a group are then divided over 2 or 4 CTAs (each stages
  // the same cache rows out of L2), up to two CTAs per SM: the launch is a chain of latencies, and more, smaller CTAs
  // overlap more of them (config-2 step, 1025 positions: 37.3 us with 72 CTAs, 37.1 with 144, 36.6 with 288).
  int hsplit = 1;
  while (p.group % (2 * hsplit) == 0 && splits * p.n_kv * 2 * hsplit <= 2 * 148 && p.n_kv * 2 * hsplit <= kAttnMaxCounters) hsplit *= 2;
  p.hsplit = hsplit;
  p.scale = 1.0f / sqrtf((float)d);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(splits, p.n_kv * hsplit);
  cfg.blockDim = dim3(p.group / hsplit * pc);
  cfg.dynamicSmemBytes = (size_t)pc * (d * 4 + 16);
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e[4] = {
        cudaFuncSetAttribute(attn_decode_fused_kernel<128, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * (128 * 4 + 16)),
        cudaFuncSetAttribute(attn_decode_fused_kernel<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * (128 * 4 + 16)),
        cudaFuncSetAttribute(attn_decode_fused_kernel<64, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * (64 * 4 + 16)),
        cudaFuncSetAttribute(attn_decode_fused_kernel<64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * (64 * 4 + 16))};
    for (cudaError_t x : e)
      if (x != cudaSuccess) return x;
  }
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++*n_launch;
  if (d == 128 && pc == 64) return cudaLaunchKernelEx(&cfg, attn_decode_fused_kernel<128, 2>, p);
  if (d == 128) return cudaLaunchKernelEx(&cfg, attn_decode_fused_kernel<128, 4>, p);
  if (d == 64 && pc == 64) return cudaLaunchKernelEx(&cfg, attn_decode_fused_kernel<64, 2>, p);
  if (d == 64) return cudaLaunchKernelEx(&cfg, attn_decode_fused_kernel<64, 4>, p);
  return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------------------------------- router + top-k (a4)
// One CTA per token.  Thread (grp, e) sums h[i] * W_r[i][e] over i = grp, grp+G, ...; groups are added in ascending
// order; warp 0 then extracts the k largest logits (equal logits: lower index first) and the gates.
// Warp 0 extracts the k largest logits (equal logits: lower index first) and their gates from logit[Epad] in shared memory.
__device__ __forceinline__ void router_select(const float* logit, int m, int E, int Epad, int k, int renorm,
                                              int32_t* __restrict__ ids, float* __restrict__ gates) {
  const int lane = threadIdx.x;
  const int per = Epad / 32;  // candidates per lane: e = lane + 32*j
  uint32_t taken = 0;
  float sel_v = 0.f;  // lane j (< k) keeps the j-th selected logit
  int sel_i = 0;
  float total = 0.f, top = 0.f;
  // A NaN logit (a NaN activation or weight) compares false with everything: it takes part in the selection as -inf so
  // that the ids always lie in [0, E) (they index weight slices downstream), and every gate of the token becomes NaN.
  bool has_nan = false;
  for (int j = 0; j < per; ++j) {
    const float v = logit[lane + 32 * j];
    has_nan |= (lane + 32 * j < E) && (v != v);
  }
  has_nan = __any_sync(0xffffffffu, has_nan);
  if (!renorm) {
    float mx = -INFINITY;
    for (int j = 0; j < per; ++j) mx = fmaxf(mx, logit[lane + 32 * j]);
    mx = warp_max(mx);
    float s = 0.f;
    for (int j = 0; j < per; ++j) {
      const float v = logit[lane + 32 * j];
      s += v > -INFINITY ? expf(v - mx) : 0.f;
    }
    total = warp_sum(s);
    top = mx;
  }
  for (int r = 0; r < k; ++r) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int j = 0; j < per; ++j) {
      if (taken & (1u << j)) continue;
      const float vr = logit[lane + 32 * j];
      const float v = vr == vr ? vr : -INFINITY;
      const int idx = lane + 32 * j;
      if (idx < E && (v > bv || (v == bv && idx < bi))) {
        bv = v;
        bi = idx;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
      }
    }
    if ((bi & 31) == lane) taken |= 1u << (bi >> 5);
    if (lane == r) {
      sel_v = bv;
      sel_i = bi;
    }
  }
  float gate;
  if (renorm) {
    const float mx = __shfl_sync(0xffffffffu, sel_v, 0);
    const float ex = lane < k ? expf(sel_v - mx) : 0.f;
    const float s = warp_sum(ex);
    gate = ex / s;
  } else {
    gate = lane < k ? expf(sel_v - top) / total : 0.f;
  }
  if (has_nan) gate = __int_as_float(0x7FC00000);
  if (lane < k) {
    ids[(size_t)m * k + lane] = sel_i;
    gates[(size_t)m * k + lane] = gate;
  }
}

// The same selection for up to 256 experts by counting, all threads of the CTA at once: the rank of a logit is the number
// of logits that come before it in the order (larger value first, equal values: lower index first; NaN as -inf), so the
// expert of rank r < k is the r-th selection of router_select; warp 0 then forms the gates with router_select's own
// arithmetic.  sel_v / sel_i: k entries of shared memory.  Called by every thread of the CTA.
__device__ __forceinline__ void router_select_counting(const float* logit, int m, int E, int Epad, int k, int renorm,
                                                       int32_t* __restrict__ ids, float* __restrict__ gates, float* sel_v, int* sel_i) {
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    const float vr = logit[e];
    const float v = vr == vr ? vr : -INFINITY;
    int rank = 0;
    for (int j = 0; j < E; j += 4) {  // E is a multiple of 8 here
      const float4 o = *reinterpret_cast<const float4*>(logit + j);
      const float o0 = o.x == o.x ? o.x : -INFINITY, o1 = o.y == o.y ? o.y : -INFINITY;
      const float o2 = o.z == o.z ? o.z : -INFINITY, o3 = o.w == o.w ? o.w : -INFINITY;
      rank += (o0 > v || (o0 == v && j < e)) + (o1 > v || (o1 == v && j + 1 < e)) + (o2 > v || (o2 == v && j + 2 < e)) +
              (o3 > v || (o3 == v && j + 3 < e));
    }
    if (rank < k) {
      sel_v[rank] = v;
      sel_i[rank] = e;
    }
  }
  __syncthreads();
  if (threadIdx.x >= 32) return;
  const int lane = threadIdx.x;
  const int per = Epad / 32;
  bool has_nan = false;
  for (int j = 0; j < per; ++j) {
    const float v = logit[lane + 32 * j];
    has_nan |= (lane + 32 * j < E) && (v != v);
  }
  has_nan = __any_sync(0xffffffffu, has_nan);
  const float my_v = lane < k ? sel_v[lane] : 0.f;
  float gate;
  if (renorm) {
    const float mx = __shfl_sync(0xffffffffu, my_v, 0);
    const float ex = lane < k ? expf(my_v - mx) : 0.f;
    const float s = warp_sum(ex);
    gate = ex / s;
  } else {
    float mx = -INFINITY;
    for (int j = 0; j < per; ++j) mx = fmaxf(mx, logit[lane + 32 * j]);
    mx = warp_max(mx);
    float t = 0.f;
    for (int j = 0; j < per; ++j) {
      const float v = logit[lane + 32 * j];
      t += v > -INFINITY ? expf(v - mx) : 0.f;
    }
    const float total = warp_sum(t);
    gate = lane < k ? expf(my_v - mx) / total : 0.f;
  }
  if (has_nan) gate = __int_as_float(0x7FC00000);
  if (lane < k) {
    ids[(size_t)m * k + lane] = sel_i[lane];
    gates[(size_t)m * k + lane] = gate;
  }
}

constexpr int kRouterThreads = 1024;

__global__ void __launch_bounds__(kRouterThreads) router_topk_kernel(const __half* __restrict__ h, const __half* __restrict__ wr,
                                                                     int H, int E, int Epad, int k, int renorm,
                                                                     int32_t* __restrict__ ids, float* __restrict__ gates) {
  extern __shared__ float smem[];
  float* h_s = smem;             // [H]
  float* part = h_s + H;         // [G][Epad]
  float* logit = part + kRouterThreads;  // [Epad]
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int m = blockIdx.x;
  const int G = kRouterThreads / Epad;
  for (int i = threadIdx.x; i < H; i += blockDim.x) h_s[i] = __half2float(h[(size_t)m * H + i]);
  __syncthreads();
  const int e = threadIdx.x % Epad, grp = threadIdx.x / Epad;
  float acc = 0.f;
  if (e < E)
    for (int i = grp; i < H; i += G) acc = fmaf(h_s[i], __half2float(wr[(size_t)i * E + e]), acc);
  part[grp * Epad + e] = acc;
  __syncthreads();
  if (threadIdx.x < Epad) {
    float t = 0.f;
    for (int g = 0; g < G; ++g) t += part[g * Epad + threadIdx.x];
    logit[threadIdx.x] = threadIdx.x < E ? t : -INFINITY;
  }
  __syncthreads();
  if (threadIdx.x >= 32) return;
  router_select(logit, m, E, Epad, k, renorm, ids, gates);
}

// The same routing for hidden sizes and expert counts that are multiples of 8, spread over a cluster of 8 CTAs per
// token: CTA r of the cluster sums rows [r H/8, (r+1) H/8) of W_r (16-byte loads: a thread owns 8 consecutive experts of
// the rows i = row group, row group + R, ...), adds its row groups in ascending order, and writes its partial logits
// into CTA 0's shared memory (distributed shared memory); after the cluster barrier CTA 0 adds the 8 partials in rank
// order and selects.  A single token's router matrix then streams through 8 SMs instead of one.
constexpr int kRouterCluster = 8;
constexpr int kRouterClThreads = 256;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f32(const float* local_smem_ptr, uint32_t rank, float v) {
  uint32_t la = (uint32_t)__cvta_generic_to_shared(local_smem_ptr), ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}

// Optional RMSNorm prologue (gain != null): the token's row is xn (fp16 or fp32), every CTA of the cluster sums its
// squares itself (the whole row is a few kilobytes), normalises its own eighth, h = rn16(x * g / sqrt(mean(x^2) + eps)),
// uses it and writes it to h_out for the expert kernels that follow.
__global__ void __launch_bounds__(kRouterClThreads) router_topk_cluster_kernel(const __half* __restrict__ h,
                                                                               const __half* __restrict__ wr, int H, int E, int Epad,
                                                                               int k, int renorm, int32_t* __restrict__ ids,
                                                                               float* __restrict__ gates, const void* __restrict__ xn,
                                                                               int xn_f32, const __half* __restrict__ gain, float eps,
                                                                               __half* __restrict__ h_out) {
  extern __shared__ __align__(16) float smem[];
  const int Hc = H / kRouterCluster;          // rows of this CTA
  const int L = E / 8;                        // threads per row
  const int R = kRouterClThreads / L;         // row groups (L <= 128, so R >= 2)
  float* h_s = smem;                          // [Hc]
  float* part = h_s + Hc;                     // [R][E]
  float* cl = part + (size_t)R * E;           // [kRouterCluster][Epad]   (used in CTA 0)
  float* logit = cl + (size_t)kRouterCluster * Epad;  // [Epad]
  const int m = blockIdx.y;
  const uint32_t rank = cluster_ctarank();
  const int row0 = (int)rank * Hc;
  const int grp = threadIdx.x / L, e0 = (threadIdx.x % L) * 8;
  // The rows of a thread are fetched in batches of 16 loads that are all issued before the first is used: the matrix is
  // read once at memory latency (a token's 512 KB are 64 KB per CTA, one batch per thread), not once per row.  The
  // router matrix does not depend on the preceding kernel: the first batch is requested before waiting for it.
  constexpr int kBatch = 16;
  uint4 w[kBatch];
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int i = grp + b * R;
    w[b] = (grp < R && i < Hc) ? __ldg(reinterpret_cast<const uint4*>(wr + (size_t)(row0 + i) * E + e0)) : make_uint4(0, 0, 0, 0);
  }
  // the norm gains of this CTA's rows are parameters too (up to 8 per thread: hidden sizes up to 16384)
  float gain_pre[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int i = (int)threadIdx.x + q * kRouterClThreads;
    gain_pre[q] = (gain && i < Hc) ? __half2float(gain[row0 + i]) : 0.f;
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the token's row comes from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (gain) {
    // every CTA sums the squares of the whole row (a few kilobytes) and normalises its own eighth; the row is read once
    __shared__ float red[kRouterClThreads / 32];
    const __half* x16 = static_cast<const __half*>(xn) + (size_t)m * H;
    const float* x32 = static_cast<const float*>(xn) + (size_t)m * H;
    float ss = 0.f;
    for (int i = threadIdx.x; i < H; i += kRouterClThreads) {
      const float v = xn_f32 ? x32[i] : __half2float(x16[i]);
      if (i >= row0 && i < row0 + Hc) h_s[i - row0] = v;  // kept for the second pass
      ss = fmaf(v, v, ss);
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w2 = 0; w2 < kRouterClThreads / 32; ++w2) t += red[w2];
    const float inv = 1.0f / sqrtf(t / (float)H + eps);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = (int)threadIdx.x + q * kRouterClThreads;
      if (i < Hc) {
        const __half hv = __float2half_rn(h_s[i] * gain_pre[q] * inv);
        h_s[i] = __half2float(hv);
        h_out[(size_t)m * H + row0 + i] = hv;
      }
    }
  } else {
    for (int i = threadIdx.x; i < Hc; i += kRouterClThreads) h_s[i] = __half2float(h[(size_t)m * H + row0 + i]);
  }
  __syncthreads();
  float acc[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) acc[q] = 0.f;
  if (grp < R) {
    for (int i0 = grp; i0 < Hc; i0 += R * kBatch) {
      if (i0 != grp) {
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int i = i0 + b * R;
          w[b] = i < Hc ? __ldg(reinterpret_cast<const uint4*>(wr + (size_t)(row0 + i) * E + e0)) : make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int b = 0; b < kBatch; ++b) {
        const int i = i0 + b * R;
        const float x = i < Hc ? h_s[i] : 0.f;
        const uint32_t ws[4] = {w[b].x, w[b].y, w[b].z, w[b].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 f = __half22float2(u32_as_half2(ws[q]));
          acc[2 * q] = fmaf(x, f.x, acc[2 * q]);
          acc[2 * q + 1] = fmaf(x, f.y, acc[2 * q + 1]);
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) part[(size_t)grp * E + e0 + q] = acc[q];
  }
  __syncthreads();
  for (int e = threadIdx.x; e < Epad; e += kRouterClThreads) {
    float t = 0.f;
    if (e < E)
      for (int g = 0; g < R; ++g) t += part[(size_t)g * E + e];
    st_cluster_f32(cl + (size_t)rank * Epad + e, 0, t);  // into CTA 0's copy of cl
  }
  cluster_sync_all();
  if (rank != 0) return;
  for (int e = threadIdx.x; e < Epad; e += kRouterClThreads) {
    float t = 0.f;
#pragma unroll
    for (int r = 0; r < kRouterCluster; ++r) t += cl[(size_t)r * Epad + e];
    logit[e] = e < E ? t : -INFINITY;
  }
  __syncthreads();
  if (E <= 256) {
    __shared__ float sel_v[32];
    __shared__ int sel_i[32];
    router_select_counting(logit, m, E, Epad, k, renorm, ids, gates, sel_v, sel_i);
    return;
  }
  if (threadIdx.x >= 32) return;
  router_select(logit, m, E, Epad, k, renorm, ids, gates);
}

cudaError_t launch_router_topk(const __half* h, const __half* wr, int M, int H, int E, int k, int renorm, int32_t* ids,
                               float* gates, cudaStream_t st, uint64_t* n_launch, int pdl) {
  return launch_router_topk_norm(h, wr, M, H, E, k, renorm, ids, gates, nullptr, 0, nullptr, 0.f, st, n_launch, pdl);
}

// With norm_gain: h = RMSNorm(norm_x; norm_gain) is computed first and written to h (which the kernels after the router
// read); one launch where the cluster kernel takes the shape, else the stand-alone norm and then the router.
cudaError_t launch_router_topk_norm(const __half* h, const __half* wr, int M, int H, int E, int k, int renorm, int32_t* ids,
                                    float* gates, const void* norm_x, int norm_x_f32, const __half* norm_gain, float eps,
                                    cudaStream_t st, uint64_t* n_launch, int pdl) {
  int Epad = 32;
  while (Epad < E) Epad <<= 1;
  if (E % 8 == 0 && H % (8 * kRouterCluster) == 0 && H <= 8 * kRouterClThreads * kRouterCluster && (((uintptr_t)wr | (uintptr_t)h) & 15) == 0) {
    const int L = E / 8, R = kRouterClThreads / L;
    const size_t smem_cl = ((size_t)H / kRouterCluster + (size_t)R * E + (size_t)(kRouterCluster + 1) * Epad) * sizeof(float);
    if (smem_cl <= 160 * 1024) {
      if (smem_cl > 48 * 1024) {  // (cheap; set on every call because the size depends on the shape)
        cudaError_t e = cudaFuncSetAttribute(router_topk_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_cl);
        if (e != cudaSuccess) return e;
      }
      ++*n_launch;
      return launch_dep(router_topk_cluster_kernel, dim3(kRouterCluster, M), dim3(kRouterClThreads), smem_cl, st, pdl, kRouterCluster,
                        h, wr, H, E, Epad, k, renorm, ids, gates, norm_x, norm_x_f32, norm_gain, eps, const_cast<__half*>(h));
    }
  }
  if (norm_gain) {
    cudaError_t e = launch_rmsnorm(norm_x, norm_x_f32, norm_gain, const_cast<__half*>(h), M, H, eps, st, n_launch, pdl);
    if (e != cudaSuccess) return e;
  }
  const size_t smem = ((size_t)H + kRouterThreads + Epad) * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(router_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  ++*n_launch;
  return launch_dep(router_topk_kernel, dim3(M), dim3(kRouterThreads), smem, st, pdl, 1, h, wr, H, E, Epad, k, renorm, ids, gates);
}

// ------------------------------------------------------------------------------------------- MoE combine
template <typename TRes>
__global__ void moe_combine_kernel(const TRes* __restrict__ res, const float* __restrict__ gates, const float* __restrict__ d32,
                                   __half* __restrict__ y16, int k, int H) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // inputs come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int m = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= H) return;
  float acc = load_f<TRes>(res, (size_t)m * H + i);
  for (int j = 0; j < k; ++j) acc = fmaf(gates[m * k + j], d32[((size_t)m * k + j) * H + i], acc);
  y16[(size_t)m * H + i] = __float2half_rn(acc);
}

cudaError_t launch_moe_combine(const void* res, int res_is_f32, const float* gates, const float* d32, __half* y16, int M,
                               int k, int H, cudaStream_t st, uint64_t* n_launch, int pdl) {
  dim3 grid((H + 255) / 256, M);
  ++*n_launch;
  if (res_is_f32)
    return launch_dep(moe_combine_kernel<float>, grid, dim3(256), 0, st, pdl, 1, (const float*)res, gates, d32, y16, k, H);
  return launch_dep(moe_combine_kernel<__half>, grid, dim3(256), 0, st, pdl, 1, (const __half*)res, gates, d32, y16, k, H);
}

// ---------------------------------------------------------------- host-driven calls: completion word
// Completion word of a host-driven call: written (to mapped pinned host memory) once everything before it in the stream
// has completed and its writes are visible, so the host can poll the word instead of synchronising with the stream.
__global__ void signal_done_kernel(int* done, int seq) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  *reinterpret_cast<volatile int*>(done) = seq;
  __threadfence_system();
}
cudaError_t launch_signal_done(int* done_alias, int seq, int pdl, cudaStream_t st, uint64_t* n_launch) {
  ++*n_launch;
  return launch_dep(signal_done_kernel, dim3(1), dim3(1), 0, st, pdl, 1, done_alias, seq);
}

cudaError_t launch_fill(void* p, uint64_t bytes, uint8_t v, cudaStream_t st, uint64_t* n_launch) {
  (void)n_launch;
  return cudaMemsetAsync(p, v, bytes, st);
}

}  // namespace ats

#ifdef ATS_TRACE_ATTN
extern "C" int ats_attn_trace_read(void* out_host, int cap_records) {
  unsigned int n = 0;
  if (cudaMemcpyFromSymbol(&n, ats::g_attn_trace_n, sizeof n) != cudaSuccess) return -1;
  if (n > (1u << 15)) n = 1u << 15;
  if ((int)n > cap_records) n = cap_records;
  if (n && cudaMemcpyFromSymbol(out_host, ats::g_attn_trace, (size_t)n * sizeof(ats::AttnTraceRec)) != cudaSuccess) return -1;
  unsigned int zero = 0;
  cudaMemcpyToSymbol(ats::g_attn_trace_n, &zero, sizeof zero);
  return (int)n;
}
#endif
