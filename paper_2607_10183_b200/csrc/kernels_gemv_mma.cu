// Few-row GEMV for the two 4-bit block formats on the warp-level tensor-core instruction (mma.sync m16n8k16, fp16
// operands, fp32 accumulation): y[m][n] = sum_k w[n][k] x[m][k] for M <= 8 rows of x.
//
// The generic GEMV decodes every weight to fp32 and spends a fused multiply-add per weight and activation row: about five
// thread instructions per weight, which is what bounds it (not HBM) for the microscaling format and for several rows.
// Here a warp owns 16 weight rows; the weights of a 16 x 16 tile are the A operand, decoded straight into fp16 pairs in
// the fragment layout (each thread decodes only the pair the layout gives it: two shifts and two logic operations for the
// microscaling format, a shift, a logic operation and one fp16 subtraction for the integer codes), the M activation rows
// are the eight columns of the B operand, and one instruction does the 16 x 16 x 8 products.  Products of fp16 values are
// exact in fp32; the two k-steps of a 32-wide block accumulate in the instruction's fp32 accumulator, the block's scale
// is applied in fp32 and blocks are summed in fp32, so weights stay exact as in the generic kernel.  The layout:
//   A (16 x 16, row):  reg0 = (row g, k 2t..2t+1), reg1 = (row g+8, same k), reg2 = (row g, k 2t+8..2t+9), reg3 = (row g+8, ..)
//   B (16 x 8, col):   reg0 = (k 2t..2t+1, column g), reg1 = (k 2t+8..2t+9, column g)
//   C (16 x 8):        c0 c1 = (row g, columns 2t 2t+1), c2 c3 = (row g+8, columns 2t 2t+1)        g = lane / 4, t = lane % 4
// and a code word holds k = 0..7 of its row with the pair (2j, 2j+1) in nibbles j and j + 4, so thread t takes pair t of
// word 2s (reg0/1) and of word 2s+1 (reg2/3) in k-step s.
//
// A unit is 16 consecutive output rows (SwiGLU: 16 gate rows and the 16 up rows of the same outputs).  1, 2, 4 or 8 warps of
// the CTA share a unit, each on its own part of K; partial tiles meet in shared memory and are added in fixed order.
// Code loads are 16 bytes per thread and row; the four lanes that share a row pair load four consecutive blocks (64
// contiguous bytes per row) and hand the words round by shuffle, four such loads per row in flight (sixteen blocks), the
// first batch issued before the grid dependency resolves (weights do not depend on the preceding kernel).
#include "ats_internal.h"

namespace ats {

namespace {

struct MmaGemvParams {
  const uint8_t* base[3];
  int n_rows[3];
  int n_seg, K, M, mode, ksplit;
  const __half* x;
  int ldx;
  float* y32;
  __half* y16;
  int ldy;
  const float* res32;
  const __half* res16;
  int ldres;
};

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Pair t (nibbles t and t + 4) of a code word as two fp16 values.
//   MX = false: offset-binary integer codes u = c + 8: the fp16 pair 1024 + u minus 1032.
//   MX = true: microscaling floats: magnitude bits onto bits 11..9 of each half, sign onto bit 15: element * 2^-14.
template <bool MX>
__device__ __forceinline__ uint32_t decode_pair(uint32_t w, int t) {
  if (MX) {
    const uint32_t mag = __funnelshift_l(w, w, (9 - 4 * t) & 31) & 0x0E000E00u;
    return (__funnelshift_l(w, w, (12 - 4 * t) & 31) & 0x80008000u) | mag;
  } else {
    const uint32_t u = ((w >> (4 * t)) & 0x000F000Fu) | 0x64006400u;
    __half2 h, k1032;
    *reinterpret_cast<uint32_t*>(&h) = u;
    *reinterpret_cast<uint32_t*>(&k1032) = 0x64086408u;
    h = __hsub2(h, k1032);
    return *reinterpret_cast<uint32_t*>(&h);
  }
}

__device__ __forceinline__ uint32_t pick_word(const uint4& q, int j) { return j == 0 ? q.x : j == 1 ? q.y : j == 2 ? q.z : q.w; }

// N (4, 8 or 16) consecutive block scales of a row as packed fp16 pairs: one or two vector loads where the address allows,
// else scalar loads; blocks at or beyond b_hi read as zero.
template <int N>
__device__ __forceinline__ void load_scales(const __half* sp, int b0, int b_hi, bool live, uint32_t (&s)[N / 2]) {
  if (live && b0 + N <= b_hi && (reinterpret_cast<uintptr_t>(sp + b0) & (2 * N > 16 ? 15 : 2 * N - 1)) == 0) {
    if (N == 4) {
      const uint2 v = __ldg(reinterpret_cast<const uint2*>(sp + b0));
      s[0] = v.x; s[1] = v.y;
    } else {
#pragma unroll
      for (int i = 0; i < N / 8; ++i) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(sp + b0) + i);
        s[4 * i] = v.x; s[4 * i + 1] = v.y; s[4 * i + 2] = v.z; s[4 * i + 3] = v.w;
      }
    }
    return;
  }
#pragma unroll
  for (int j = 0; j < N / 2; ++j) {
    const unsigned short a = (live && b0 + 2 * j < b_hi) ? __half_as_ushort(__ldg(sp + b0 + 2 * j)) : (unsigned short)0;
    const unsigned short b = (live && b0 + 2 * j + 1 < b_hi) ? __half_as_ushort(__ldg(sp + b0 + 2 * j + 1)) : (unsigned short)0;
    s[j] = (uint32_t)a | ((uint32_t)b << 16);
  }
}
template <int N2>
__device__ __forceinline__ float scale_of(const uint32_t (&s)[N2], int j) {
  return __half2float(__ushort_as_half((unsigned short)(s[j >> 1] >> (16 * (j & 1)))));
}

template <bool MX, bool SW>
__global__ void __launch_bounds__(256) gemv_mma_kernel(const MmaGemvParams p) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  bool waited = false;  // x and the residual come from the preceding kernel; the first weight loads need not wait for it
  constexpr int NT = SW ? 2 : 1;   // weight tiles per unit
  constexpr int NB = SW ? 1 : 2;   // 16-byte loads in flight per thread and row: a batch covers 4 * NB blocks
  __shared__ float red_s[8][NT][16][8];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int K = p.K, nblk = K / 32, M = p.M;
  int n_rows = p.n_rows[0];  // rows side by side (SwiGLU: outputs)
  if (!SW) n_rows += (p.n_seg > 1 ? p.n_rows[1] : 0) + (p.n_seg > 2 ? p.n_rows[2] : 0);
  // codes and scales of weight row r of tile kind nt (SwiGLU: 0 = gate, 1 = up; otherwise rows run across the segments)
  auto row_ptrs = [&](int r, int nt, const uint4*& codes, const __half*& scales) {
    const uint8_t* base = p.base[0];
    int rows = p.n_rows[0];
    if (SW) {
      if (nt) base = p.base[1];
    } else if (p.n_seg > 1 && r >= p.n_rows[0]) {
      r -= p.n_rows[0];
      base = p.base[1];
      rows = p.n_rows[1];
      if (p.n_seg > 2 && r >= p.n_rows[1]) {
        r -= p.n_rows[1];
        base = p.base[2];
        rows = p.n_rows[2];
      }
    }
    codes = reinterpret_cast<const uint4*>(base + (size_t)r * (K / 2));
    scales = reinterpret_cast<const __half*>(base + (size_t)rows * (K / 2)) + (size_t)r * nblk;
  };
  const int n_units = (n_rows + 15) / 16;
  const int ks = p.ksplit, upc = 8 / ks;
  const int part = w % ks, slot = w / ks;
  const int per = (((nblk + ks - 1) / ks) + 15) & ~15;  // blocks per part: whole batches, so that scale loads stay aligned
  const int b_lo = part * per, b_hi = min(nblk, b_lo + per);
  const uint32_t zero_word = MX ? 0u : 0x88888888u;  // eight zeros in either format
  const __half* xrow = p.x + (size_t)min(g, M - 1) * p.ldx + 2 * t;
  const bool xlive = g < M;
  const int quad = lane & ~3;
  for (int u0 = blockIdx.x * upc; u0 < n_units; u0 += gridDim.x * upc) {
    const int u = u0 + slot;
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
    if (u < n_units) {
      const uint4* cp[NT][2];
      const __half* sp[NT][2];
      bool live[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = 16 * u + g + 8 * h;
        live[h] = r < n_rows;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) row_ptrs(live[h] ? r : 0, nt, cp[nt][h], sp[nt][h]);
      }
      for (int b0 = b_lo; b0 < b_hi; b0 += 4 * NB) {
        // The four lanes of a quad share their two rows: lane t loads blocks b0 + 4 i + t (64 contiguous bytes per row and
        // quad), and each block's words travel to the other three lanes by shuffle when the block is consumed.
        uint4 q[NB][NT][2];
        uint32_t sc[NT][2][2 * NB];
#pragma unroll
        for (int i = 0; i < NB; ++i) {
          const int b = b0 + 4 * i + t;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int h = 0; h < 2; ++h)
              q[i][nt][h] = (live[h] && b < b_hi) ? __ldcs(cp[nt][h] + b) : make_uint4(zero_word, zero_word, zero_word, zero_word);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int h = 0; h < 2; ++h) load_scales<4 * NB>(sp[nt][h], b0, b_hi, live[h], sc[nt][h]);
        if (!waited) {
          asm volatile("griddepcontrol.wait;" ::: "memory");
          waited = true;
        }
#pragma unroll
        for (int j = 0; j < 4 * NB; ++j) {
          const int b = b0 + j;
          if (b >= b_hi) break;  // uniform over the warp
          uint32_t xb[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) xb[e] = xlive ? __ldg(reinterpret_cast<const uint32_t*>(xrow + b * 32 + 8 * e)) : 0u;
          const int src = quad | (j & 3);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            uint32_t wd[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint4& v = q[j >> 2][nt][h];
              wd[h][0] = __shfl_sync(0xffffffffu, v.x, src);
              wd[h][1] = __shfl_sync(0xffffffffu, v.y, src);
              wd[h][2] = __shfl_sync(0xffffffffu, v.z, src);
              wd[h][3] = __shfl_sync(0xffffffffu, v.w, src);
            }
            float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int s = 0; s < 2; ++s) {
              uint32_t a[4];
              a[0] = decode_pair<MX>(wd[0][2 * s], t);
              a[1] = decode_pair<MX>(wd[1][2 * s], t);
              a[2] = decode_pair<MX>(wd[0][2 * s + 1], t);
              a[3] = decode_pair<MX>(wd[1][2 * s + 1], t);
              mma16816(c, a, xb[2 * s], xb[2 * s + 1]);
            }
            const float s0 = scale_of(sc[nt][0], j), s1 = scale_of(sc[nt][1], j);
            acc[nt][0] = fmaf(s0, c[0], acc[nt][0]);
            acc[nt][1] = fmaf(s0, c[1], acc[nt][1]);
            acc[nt][2] = fmaf(s1, c[2], acc[nt][2]);
            acc[nt][3] = fmaf(s1, c[3], acc[nt][3]);
          }
        }
      }
    }
    if (!waited) {  // no block for this warp
      asm volatile("griddepcontrol.wait;" ::: "memory");
      waited = true;
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float f = MX ? 16384.f : 1.f;  // the microscaling decode left a factor 2^-14 on every element
      red_s[w][nt][g][2 * t] = acc[nt][0] * f;
      red_s[w][nt][g][2 * t + 1] = acc[nt][1] * f;
      red_s[w][nt][g + 8][2 * t] = acc[nt][2] * f;
      red_s[w][nt][g + 8][2 * t + 1] = acc[nt][3] * f;
    }
    __syncthreads();
    // one thread per (unit, row of the tile, activation row) adds the K parts in fixed order and writes the output
    for (int e = threadIdx.x; e < upc * 16 * M; e += blockDim.x) {
      const int m = e % M, row = (e / M) % 16, sl = e / (16 * M);
      const int r = 16 * (u0 + sl) + row;
      if (r >= n_rows) continue;
      float s0 = 0.f, s1 = 0.f;
      for (int q2 = 0; q2 < ks; ++q2) {
        s0 += red_s[sl * ks + q2][0][row][m];
        if (SW) s1 += red_s[sl * ks + q2][NT - 1][row][m];
      }
      const size_t o = (size_t)m * p.ldy + r, ro = (size_t)m * p.ldres + r;
      switch (p.mode) {
        case GEMV_OUT_F32: p.y32[o] = s0; break;
        case GEMV_OUT_F16: p.y16[o] = __float2half_rn(s0); break;
        case GEMV_RES16_OUT_F32: p.y32[o] = __half2float(p.res16[ro]) + s0; break;
        case GEMV_RES32_OUT_F16: p.y16[o] = __float2half_rn(p.res32[ro] + s0); break;
        case GEMV_RES16_OUT_F16: p.y16[o] = __float2half_rn(__half2float(p.res16[ro]) + s0); break;
        case GEMV_SWIGLU_F16: p.y16[o] = __float2half_rn(s0 / (1.0f + expf(-s0)) * s1); break;
        default: break;
      }
    }
    __syncthreads();
  }
  if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace

bool gemv_mma_eligible(const GemvParams& g) {
  if (g.w16 || g.M < 1 || g.M > 8 || g.K % 32 || g.n_seg < 1 || g.n_seg > 3) return false;
  if ((g.ldx & 1) || (reinterpret_cast<uintptr_t>(g.x) & 3)) return false;  // activation pairs are read as 32-bit words
  if (g.mode == GEMV_SWIGLU_F16 && (g.n_seg != 2 || g.seg[0].n_rows != g.seg[1].n_rows)) return false;
  for (int s = 0; s < g.n_seg; ++s)
    if ((reinterpret_cast<uintptr_t>(g.seg[s].base) & 15) || (g.K / 2) % 16) return false;  // 16-byte code loads per block
  return true;
}

cudaError_t launch_gemv_mma(const GemvParams& g, cudaStream_t st, uint64_t* n_launch) {
  if (!gemv_mma_eligible(g)) return cudaErrorInvalidValue;
  MmaGemvParams p{};
  int n_rows = 0;
  for (int s = 0; s < g.n_seg; ++s) {
    p.base[s] = g.seg[s].base;
    p.n_rows[s] = g.seg[s].n_rows;
    n_rows += g.seg[s].n_rows;
  }
  const bool sw = g.mode == GEMV_SWIGLU_F16;
  if (sw) n_rows = g.seg[0].n_rows;
  p.n_seg = g.n_seg; p.K = g.K; p.M = g.M; p.mode = g.mode;
  p.x = g.x; p.ldx = g.ldx; p.y32 = g.y32; p.y16 = g.y16; p.ldy = g.ldy;
  p.res32 = g.res32; p.res16 = g.res16; p.ldres = g.ldres;
  const int n_units = (n_rows + 15) / 16, nblk = g.K / 32;
  // Split K while the units alone give fewer warps than about twice what the machine holds and every part keeps at least
  // one batch of sixteen blocks.  A function of the shapes only.
  int ks = 1;
  while (ks < 8 && (long)n_units * ks <= 2 * 148L * 24 && nblk / (ks * 2) >= 16) ks *= 2;
  p.ksplit = ks;
  const int upc = 8 / ks;
  const dim3 grid(std::max(1, std::min((n_units + upc - 1) / upc, 148 * 8))), block(256);
  ++*n_launch;
  if (g.mx) {
    return sw ? launch_dep(gemv_mma_kernel<true, true>, grid, block, 0, st, g.pdl, 1, p)
              : launch_dep(gemv_mma_kernel<true, false>, grid, block, 0, st, g.pdl, 1, p);
  }
  return sw ? launch_dep(gemv_mma_kernel<false, true>, grid, block, 0, st, g.pdl, 1, p)
            : launch_dep(gemv_mma_kernel<false, false>, grid, block, 0, st, g.pdl, 1, p);
}

}  // namespace ats
