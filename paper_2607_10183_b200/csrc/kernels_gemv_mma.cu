// Few-row GEMV for the two 4-bit block formats on the warp-level tensor-core instruction (mma.sync m16n8k16, fp16
// operands, fp32 accumulation): y[m][n] = sum_k w[n][k] x[m][k] for M <= 8 rows of x.
//
// The generic GEMV decodes every weight to fp32 and spends a fused multiply-add per weight and activation row: about five
// thread instructions per weight, which is what bounds it (not HBM) for the microscaling format and for several rows.
// Here a warp owns 16 weight rows; the weights of a 16 x 16 tile are the A operand, decoded straight into fp16 pairs in
// the fragment layout (two shifts and two logic operations per pair for the microscaling format, one logic
// operation and one fp16 operation for the integer codes), the M activation rows
// are the eight columns of the B operand, and one instruction does the 16 x 16 x 8 products.  Products of fp16 values are
// exact in fp32; the two k-steps of a 32-wide block accumulate in the instruction's fp32 accumulator, the block's scale
// is applied in fp32 and blocks are summed in fp32, so weights stay exact as in the generic kernel.  The layout:
//   A (16 x 16, row):  reg0 = (row g, kk 2t..2t+1), reg1 = (row g+8, same kk), reg2 = (row g, kk 2t+8..2t+9), reg3 = (row g+8, ..)
//   B (16 x 8, col):   reg0 = (kk 2t..2t+1, column g), reg1 = (kk 2t+8..2t+9, column g)
//   C (16 x 8):        c0 c1 = (row g, columns 2t 2t+1), c2 c3 = (row g+8, columns 2t 2t+1)        g = lane / 4, t = lane % 4
// The instruction sums over its sixteen kk whatever they stand for, so the k of a 32-wide block are dealt to the two
// instructions in the order that suits the data: lane t takes k = 8t .. 8t+7 of the block, that is ONE code word per row
// (word t of the block's four) and 16 contiguous bytes of x, with the word's pairs (2j, 2j+1), j = 0..3, as
// (instruction j / 2, reg 0/1 or 2/3 by j % 2) on both operands.  All shifts of the decode are compile-time constants.
//
// A unit is 16 consecutive output rows (SwiGLU: 16 gate rows and the 16 up rows of the same outputs).  1, 2, 4 or 8 warps of
// the CTA share a unit, each on its own part of K; partial tiles meet in shared memory and are added in fixed order.
// Code loads are 4 bytes per thread, row and block (the quad's four words are the block's 16 contiguous bytes), sixteen
// blocks in flight, the first batch issued before the grid dependency resolves (weights do not depend on the preceding
// kernel).
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

// The four pairs (k = 2j, 2j+1 in nibbles j and j + 4) of a code word as fp16 pairs.
//   MX = false: offset-binary integer codes u = c + 8.  (w & 0x000F000F) | 0x6400.. is the fp16 pair 1024 + u, the
//     0x00F000F0 pair is 1024 + 16 u: one subtraction or one multiply-add gives c exactly.
//   MX = true: microscaling floats: magnitude bits onto bits 11..9 of each half, sign onto bit 15: element * 2^-14.
template <bool MX>
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t (&a)[4]) {
  if (MX) {
    const uint32_t kMag = 0x0E000E00u, kSgn = 0x80008000u;
    a[0] = ((w << 9) & kMag) | ((w << 12) & kSgn);
    a[1] = ((w << 5) & kMag) | ((w << 8) & kSgn);
    a[2] = ((w << 1) & kMag) | ((w << 4) & kSgn);
    a[3] = ((w >> 3) & kMag) | (w & kSgn);
  } else {
    auto h2 = [](uint32_t v) { __half2 h; *reinterpret_cast<uint32_t*>(&h) = v; return h; };
    auto u32 = [](__half2 h) { return *reinterpret_cast<uint32_t*>(&h); };
    const uint32_t kMagic = 0x64006400u, w8 = w >> 8;
    const __half2 k1032 = h2(0x64086408u), k16th = h2(0x2C002C00u), kM72 = h2(0xD480D480u);
    a[0] = u32(__hsub2(h2((w & 0x000F000Fu) | kMagic), k1032));
    a[1] = u32(__hfma2(h2((w & 0x00F000F0u) | kMagic), k16th, kM72));
    a[2] = u32(__hsub2(h2((w8 & 0x000F000Fu) | kMagic), k1032));
    a[3] = u32(__hfma2(h2((w8 & 0x00F000F0u) | kMagic), k16th, kM72));
  }
}

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
  constexpr int NBK = SW ? 8 : 16;  // blocks in flight per thread and row
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
  const __half* xrow = p.x + (size_t)min(g, M - 1) * p.ldx + 8 * t;
  const bool xlive = g < M;
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
      for (int b0 = b_lo; b0 < b_hi; b0 += NBK) {
        // Lane t of a quad loads word t of every block of its two rows (the quad's four words are the block's 16 contiguous
        // bytes), NBK blocks in flight.
        uint32_t q[NBK][NT][2];
        uint32_t sc[NT][2][NBK / 2];
#pragma unroll
        for (int j = 0; j < NBK; ++j) {
          const int b = b0 + j;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int h = 0; h < 2; ++h)
              q[j][nt][h] = (live[h] && b < b_hi) ? __ldg(reinterpret_cast<const uint32_t*>(cp[nt][h] + b) + t) : zero_word;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int h = 0; h < 2; ++h) load_scales<NBK>(sp[nt][h], b0, b_hi, live[h], sc[nt][h]);
        if (!waited) {
          asm volatile("griddepcontrol.wait;" ::: "memory");
          waited = true;
        }
#pragma unroll
        for (int j = 0; j < NBK; ++j) {
          const int b = b0 + j;
          if (b >= b_hi) break;  // uniform over the warp
          // x[b * 32 + 8 t .. + 7]: the four pairs this lane's word multiplies, in instruction order
          const uint4 xv = xlive ? __ldg(reinterpret_cast<const uint4*>(xrow + b * 32)) : make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            uint32_t a0[4], a1[4];
            decode_word<MX>(q[j][nt][0], a0);
            decode_word<MX>(q[j][nt][1], a1);
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t f0[4] = {a0[0], a1[0], a0[1], a1[1]}, f1[4] = {a0[2], a1[2], a0[3], a1[3]};
            mma16816(c, f0, xv.x, xv.y);
            mma16816(c, f1, xv.z, xv.w);
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
  if ((g.ldx & 7) || (reinterpret_cast<uintptr_t>(g.x) & 15)) return false;  // a lane reads its eight activations as 16 bytes
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
