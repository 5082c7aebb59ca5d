// Dequantize-fused prefill GEMM on the 5th-generation tensor cores (sm_100a): Y[T][N] = X[T][K] * W^T, fp16 operands,
// fp32 accumulation in tensor memory, fp16 output.
//
// One CTA computes a tile of 256 tokens x 256 output features (or 128 x 128) over a K range (split-K when the tiles do
// not fill the GPU).  The activation tile is the MMA A operand (M = 128 tokens per instruction, two token blocks share
// one weight tile), loaded by TMA (cp.async.bulk.tensor, 128-byte swizzle, out-of-range rows zero-filled).  The weight
// tile is the B operand (N = features): sixteen warps read the packed 4-bit codes and fp16 scales straight from global
// memory (two threads per weight row, one 32-k block each per stage), expand them to fp16 (w = rn16(scale * code), a
// single rounding) and store them into shared memory in the canonical K-major 128-byte-swizzle layout the tensor core
// reads.  A single thread issues tcgen05.mma (K = 16 per instruction) into one accumulator per token block in TMEM;
// tcgen05.commit releases the stage to the producers through an mbarrier.  The dequantization warps then become the
// epilogue: tcgen05.ld brings the accumulator back with lane = token and columns = features, so each thread holds runs
// of consecutive features of one output row and writes Y (or an fp32 split-K partial that a second kernel sums in split
// order) in 16-byte pieces.
//
// Warp roles: 0 = TMA producer, 1 = TMEM allocation + MMA issue, 2.. = weight dequantization, then epilogue.
// One CTA per tile, no cluster launch.  Every mbarrier wait is bounded; on expiry the CTA raises the status word, skips
// the rest of its work, frees its tensor memory and returns.
#include <cuda.h>

#include "ats_internal.h"
#include "sm100_sync.cuh"

namespace ats {

namespace {

constexpr int BM = 128;         // tokens per MMA (M); also the granule of the feature tile
constexpr int BK = 64;          // k per stage: 64 fp16 = one 128-byte swizzle row
constexpr int BOXR = 64;        // activation rows per TMA box
constexpr int A_BYTES = BM * BK * 2;        // 16 KB per 128-row feature sub-tile
constexpr int kMaxStages = 6;
// Two tile configurations <FT, TT>: FT * 128 features x TT tokens per CTA (TT / 128 accumulators of FT * 128 columns).
//   <2, 256>: 256 x 256, 3 stages of 64 KB, all 512 TMEM columns
//   <1, 128>: 128 x 128, 6 stages of 32 KB, 128 TMEM columns
template <int FT, int TT>
struct TileCfg {
  static constexpr int BF = BM * FT;                      // features per CTA
  static constexpr int kDequantWarps = 2 * BF / 32;       // two threads per weight row: one 32-k block each per k-step
  static constexpr int kThreads = (2 + kDequantWarps) * 32;
  static constexpr int B_BYTES = TT * BK * 2;
  static constexpr int kStageBytes = FT * A_BYTES + B_BYTES;
  static constexpr int kStages = (FT == 2 ? 3 : 6);
  static constexpr int kTmemCols = FT * TT;               // 512 or 128: powers of two >= 32
};

struct GemmSeg {
  const uint8_t* base;
  int n_rows;
  int tile0;  // first feature tile of the segment
  int col0;   // first output column of the segment
};
struct GemmKParams {
  GemmSeg seg[3];
  int n_seg;
  int K, T;
  int total_ksteps, ksteps_per_split, splits;
  int bf;  // feature rows per CTA tile: a multiple of 32, at most the configuration's width (narrower tiles even out the waves)
  __half* y;
  int ldy;
  float* partial;  // [splits][T][ldy] when splits > 1
  int stages;
  int* status;
  const __half* res;  // optional residual: y2 = rn16(res + y)
  __half* y2;
  // grouped form (one weight slice per expert, blockIdx.z = expert; splits = 1): expert e multiplies the activation rows
  // grp_off[e] .. grp_off[e+1]-1 (rows sorted by expert) with slice e of every segment and writes the same rows of y
  int w16;  // the weights are an unquantized fp16 matrix (one segment): their tiles come by TMA, nothing is dequantized
  const int* grp_off;                 // DEVICE [n_experts + 1], null = the plain form
  unsigned long long grp_stride;      // bytes between the slices of consecutive experts (contiguous resident experts)
  const uint8_t* const* grp_tab[3];   // per segment: DEVICE table of slice addresses (device or mapped host memory), or null
};

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
// K-major operand tile with 128-byte rows in the 128-byte swizzle: rows at 128 B, groups of 8 rows at 1024 B.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                    // leading byte offset (not used by swizzled K-major layouts)
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}
// kind::f16, fp16 x fp16 -> fp32, both operands K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
      "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
        "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
        "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ __half2 u2h2(uint32_t v) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = v;
  return h;
}
// One code word (8 codes, internal nibble order) times the block scale -> 8 fp16 weights (k ascending) as one 16-byte chunk.
__device__ __forceinline__ uint4 dequant8(uint32_t w, __half2 s2) {
  const uint32_t kMagic = 0x64006400u;
  const __half2 k1032 = u2h2(0x64086408u), k16th = u2h2(0x2C002C00u), kM72 = u2h2(0xD480D480u);
  const uint32_t w8 = w >> 8;
  const __half2 c0 = __hmul2(__hsub2(u2h2((w & 0x000F000Fu) | kMagic), k1032), s2);
  const __half2 c1 = __hmul2(__hfma2(u2h2((w & 0x00F000F0u) | kMagic), k16th, kM72), s2);
  const __half2 c2 = __hmul2(__hsub2(u2h2((w8 & 0x000F000Fu) | kMagic), k1032), s2);
  const __half2 c3 = __hmul2(__hfma2(u2h2((w8 & 0x00F000F0u) | kMagic), k16th, kM72), s2);
  uint4 o;
  o.x = *reinterpret_cast<const uint32_t*>(&c0);
  o.y = *reinterpret_cast<const uint32_t*>(&c1);
  o.z = *reinterpret_cast<const uint32_t*>(&c2);
  o.w = *reinterpret_cast<const uint32_t*>(&c3);
  return o;
}

// The same for a word of microscaling 4-bit floats: the magnitude bits land on bits 11..9 of each fp16 (= element * 2^-14,
// exponent-0 subnormals included), 2^14 and the power-of-two block scale follow as two exact multiplications.
__device__ __forceinline__ uint4 dequant8_mx(uint32_t w, __half2 s2) {
  const __half2 k2p14 = u2h2(0x74007400u);
  const uint32_t kMag = 0x0E000E00u, kSgn = 0x80008000u;
  const __half2 c0 = __hmul2(__hmul2(u2h2(((w << 9) & kMag) | ((w << 12) & kSgn)), k2p14), s2);
  const __half2 c1 = __hmul2(__hmul2(u2h2(((w << 5) & kMag) | ((w << 8) & kSgn)), k2p14), s2);
  const __half2 c2 = __hmul2(__hmul2(u2h2(((w << 1) & kMag) | ((w << 4) & kSgn)), k2p14), s2);
  const __half2 c3 = __hmul2(__hmul2(u2h2(((w >> 3) & kMag) | (w & kSgn)), k2p14), s2);
  uint4 o;
  o.x = *reinterpret_cast<const uint32_t*>(&c0);
  o.y = *reinterpret_cast<const uint32_t*>(&c1);
  o.z = *reinterpret_cast<const uint32_t*>(&c2);
  o.w = *reinterpret_cast<const uint32_t*>(&c3);
  return o;
}

// MX: the code words hold microscaling 4-bit floats (a compile-time switch: the branch inside the dequantization loop
// costs the integer-code kernel 5 % when taken at run time).
template <int FT, int TT, bool MX>
__global__ void __launch_bounds__(TileCfg<FT, TT>::kThreads, FT == 1 ? 2 : 1) gemm_q4_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap, const GemmKParams p) {
  using Cfg = TileCfg<FT, TT>;
  constexpr int BF = Cfg::BF, TTILE = TT, MB = TT / BM, kStageBytes = Cfg::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_a[kMaxStages], full_b[kMaxStages], empty[kMaxStages], acc_full;
  __shared__ uint32_t tmem_base_s;
  __shared__ int fail_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int S = p.stages;
  // ---- which tile
  const int tile = blockIdx.x;
  int sg = 0;
  while (sg + 1 < p.n_seg && tile >= p.seg[sg + 1].tile0) ++sg;
  const int row0 = (tile - p.seg[sg].tile0) * p.bf;
  const int n_rows = p.seg[sg].n_rows;
  const int t0 = blockIdx.y * TTILE;
  // grouped form: the expert's rows and weight slice.  The row offsets were written by a copy that precedes this launch
  // in the stream, so every thread waits for the grid dependency before reading them.
  int T_ = p.T, rowoff = 0;
  const uint8_t* segbase = p.seg[sg].base;
  if (p.grp_off) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int e = blockIdx.z;
    rowoff = p.grp_off[e];
    T_ = p.grp_off[e + 1] - rowoff;
    if (t0 >= T_) return;  // this expert has fewer rows than the grid's token blocks cover (no barrier, no tensor memory yet)
    segbase = p.grp_tab[sg] ? p.grp_tab[sg][e] : segbase + (size_t)e * p.grp_stride;
  }
  const int Tt = min(TTILE, T_ - t0);
  const int nmma = min(p.bf, (n_rows - row0 + 15) / 16 * 16);  // MMA N: the features of this tile that hold real rows
  const int n_dq = (p.bf + 15) / 16;                           // dequantization warps with rows to fill (16 rows each)
  const int boxes = (Tt + BOXR - 1) / BOXR;                  // TMA boxes of 64 activation rows
  const int n_mb = (Tt + BM - 1) / BM;                       // 128-token blocks (MMA M) that hold real tokens
  const int split = p.grp_off ? 0 : blockIdx.z;
  const int ks0 = split * p.ksteps_per_split;
  const int nks = min(p.ksteps_per_split, p.total_ksteps - ks0);
  if (threadIdx.x == 0) {
    fail_s = 0;
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&full_a[s], n_dq);  // one arrival per dequantization warp that has rows
      mbar_init(&full_b[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(&acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const uint32_t tmem_cols = (uint32_t)Cfg::kTmemCols;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;
  // Only the activations come from the preceding kernel: the TMA producer waits for it, the weight path (parameters)
  // starts at once, and everything that touches other kernels' data (epilogue stores, the residual read) is ordered
  // behind the producer's wait through the pipeline's barriers.  Dependents are released after that wait, never before.
  if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (activation tile)
    if (lane == 0) {
      // fp16 weights: the weight tile of a stage is loaded like the activation tile (boxes of 64 rows x 64 k, rows past the
      // matrix read as zeros) and counted on the same barrier
      const int wboxes = p.w16 ? (nmma + BOXR - 1) / BOXR : 0;
      const uint32_t tx = (uint32_t)(boxes + wboxes) * BOXR * BK * 2;
      for (int i = 0; i < nks; ++i) {
        const int s = i % S;
        if (i >= S && !mbar_wait(&empty[s], ((i / S) - 1) & 1)) {
          fail_s = 1;
          break;
        }
        uint8_t* bdst = smem + (size_t)s * kStageBytes + FT * A_BYTES;
        mbar_expect_tx(&full_b[s], tx);
        for (int b = 0; b < boxes; ++b)
          tma_load_2d(bdst + (size_t)b * BOXR * BK * 2, &xmap, (ks0 + i) * BK, rowoff + t0 + b * BOXR, &full_b[s]);
        for (int b = 0; b < wboxes; ++b)
          tma_load_2d(smem + (size_t)s * kStageBytes + (size_t)b * BOXR * BK * 2, &wmap, (ks0 + i) * BK, row0 + b * BOXR, &full_b[s]);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issue
    if (lane == 0) {
      bool ok = true;
      const uint32_t idesc = umma_idesc(nmma);
      // Descriptors differ from stage to stage and from MMA to MMA only in the 14-bit start-address field, so each is
      // one 32-bit add on the low word: the loop stays a handful of instructions per MMA and the issuing thread keeps
      // the tensor pipe fed even when the other warps of its scheduler are busy.
      const uint64_t desc0 = umma_desc(smem_u32(smem));
      uint32_t accum = 0;
      int s = 0;
      uint32_t par = 0;
      for (int i = 0; i < nks; ++i) {
        if ((!p.w16 && !mbar_wait(&full_a[s], par)) || !mbar_wait(&full_b[s], par)) {
          fail_s = 1;
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t wdesc = desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kStageBytes >> 4));  // weight tile: the B operand
        const uint64_t xdesc = wdesc + (uint64_t)((FT * A_BYTES) >> 4);                         // activation tile: the A operand
        if (n_mb == MB) {
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
            for (int mb = 0; mb < MB; ++mb)
              umma_f16(tmem_base + (uint32_t)(mb * BF), xdesc + (uint64_t)(mb * (A_BYTES >> 4) + 2 * kk), wdesc + (uint64_t)(2 * kk), idesc,
                       kk > 0 ? 1u : accum);
          }
        } else {
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            umma_f16(tmem_base, xdesc + (uint64_t)(2 * kk), wdesc + (uint64_t)(2 * kk), idesc, kk > 0 ? 1u : accum);
        }
        accum = 1;
        umma_commit(&empty[s]);  // arrives when the MMAs reading stage s are done
        if (++s == S) {
          s = 0;
          par ^= 1;
        }
      }
      if (ok) umma_commit(&acc_full);
    }
  } else {
    // ------------------------------------------------------------ weight dequantization (A tiles): thread = (row, block)
    // Two adjacent lanes share a weight row (one 32-k block of the k-step each), so a warp's 16-byte loads touch 16
    // cache lines instead of 32: the L1 tag stage, which takes a cycle per distinct line, is the busiest unit here.
    const int w2 = warp - 2;                         // 0 .. kDequantWarps-1
    const int r = w2 * 16 + (lane >> 1);             // row of the CTA tile: sub-tile r / 128, row r % 128
    const int hb = lane & 1;                         // which of the two 32-k blocks of a k-step
    const int grow = row0 + r;
    const bool valid = grow < n_rows;
    const int K = p.K, nblk = K / 32;
    const uint8_t* crow = segbase + (size_t)(valid ? grow : 0) * (K / 2);
    const __half* srow = reinterpret_cast<const __half*>(segbase + (size_t)n_rows * (K / 2)) + (size_t)(valid ? grow : 0) * nblk;
    // Packed weights are fetched kPD k-steps ahead into registers: a k-step lasts about a thousand cycles, less than
    // the latency of a first-touch DRAM read under load.  Scales come as one 16-byte load per row for four k-steps
    // (eight blocks) when the row's scale array is 16-byte aligned, else one fp16 at a time.
    constexpr int kPD = 4;
    const bool vec_sc = (K % 256 == 0) && (ks0 % kPD == 0);
    uint4 qbuf[kPD];
    uint32_t sbuf[kPD];
    uint4 snext = make_uint4(0, 0, 0, 0);
    auto fetch_codes = [&](int ks, uint4& q) {
      const int kb = ks * 2 + hb;
      q = make_uint4(0, 0, 0, 0);
      if (valid && kb < nblk) q = __ldg(reinterpret_cast<const uint4*>(crow + (size_t)kb * 16));
    };
    auto fetch_scale1 = [&](int ks) -> uint32_t {
      const int kb = ks * 2 + hb;
      return (valid && kb < nblk) ? (uint32_t)__half_as_ushort(srow[kb]) : 0u;
    };
    auto fetch_scale8 = [&](int ks) -> uint4 {  // ks a multiple of kPD: blocks 2 ks .. 2 ks + 7
      return (valid && ks * 2 < nblk) ? __ldg(reinterpret_cast<const uint4*>(srow + ks * 2)) : make_uint4(0, 0, 0, 0);
    };
    auto pick = [&](const uint4& v, int d) -> uint32_t {  // the scale of block 2 d + hb of the eight
      const uint32_t w = d == 0 ? v.x : d == 1 ? v.y : d == 2 ? v.z : v.w;
      return (w >> (16 * hb)) & 0xFFFFu;
    };
    const int nks_dq = (w2 < n_dq && !p.w16) ? nks : 0;  // warps beyond the tile's width (and all of them with fp16 weights) have no rows to dequantize: they only take part in the epilogue
    if (vec_sc && nks_dq > 0) snext = fetch_scale8(ks0);
#pragma unroll
    for (int d = 0; d < kPD; ++d) {
      qbuf[d] = make_uint4(0, 0, 0, 0);
      sbuf[d] = 0;
      if (d < nks_dq) {
        fetch_codes(ks0 + d, qbuf[d]);
        sbuf[d] = vec_sc ? pick(snext, d) : fetch_scale1(ks0 + d);
      }
    }
    bool ok = true;
    int s = 0, round = 0;
    const int sw = r & 7, cb = hb * 4;
    for (int i0 = 0; i0 < nks_dq && ok; i0 += kPD) {
      if (vec_sc && i0 + kPD < nks) snext = fetch_scale8(ks0 + i0 + kPD);
#pragma unroll
      for (int d = 0; d < kPD; ++d) {
        const int i = i0 + d;
        if (i >= nks || !ok) break;
        const uint4 c0 = qbuf[d];
        const __half2 s0 = __half2half2(__ushort_as_half((unsigned short)sbuf[d]));
        if (i + kPD < nks) {
          fetch_codes(ks0 + i + kPD, qbuf[d]);
          if (!vec_sc) sbuf[d] = fetch_scale1(ks0 + i + kPD);
        }
        // the arithmetic needs no shared memory: do it before waiting for the stage to drain
        uint4 o0, o1, o2, o3;
        if constexpr (MX) {
          o0 = dequant8_mx(c0.x, s0), o1 = dequant8_mx(c0.y, s0), o2 = dequant8_mx(c0.z, s0), o3 = dequant8_mx(c0.w, s0);
        } else {
          o0 = dequant8(c0.x, s0), o1 = dequant8(c0.y, s0), o2 = dequant8(c0.z, s0), o3 = dequant8(c0.w, s0);
        }
        if (round > 0) {
          // one lane polls for the warp: hundreds of threads hammering the same mbarrier word slow its arrivals down
          int got = 1;
          if (lane == 0) got = mbar_wait(&empty[s], (uint32_t)(round - 1) & 1u) ? 1 : 0;
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) {
            fail_s = 1;
            ok = false;
            break;
          }
        }
        uint8_t* arow = smem + (size_t)s * kStageBytes + (size_t)r * 128;  // sub-tiles are contiguous: row r at r * 128
        *reinterpret_cast<uint4*>(arow + (((cb + 0) ^ sw) << 4)) = o0;
        *reinterpret_cast<uint4*>(arow + (((cb + 1) ^ sw) << 4)) = o1;
        *reinterpret_cast<uint4*>(arow + (((cb + 2) ^ sw) << 4)) = o2;
        *reinterpret_cast<uint4*>(arow + (((cb + 3) ^ sw) << 4)) = o3;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // make the stores visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive(&full_a[s]);  // one arrival per warp: an mbarrier retires only a few arrivals per cycle
        if (++s == S) {
          s = 0;
          ++round;
        }
      }
      if (vec_sc) {
#pragma unroll
        for (int d = 0; d < kPD; ++d) sbuf[d] = pick(snext, d);
      }
    }
    // ------------------------------------------------------------ epilogue: accumulator rows -> Y (transposed)
    int acc_ready = 0;
    if (ok && nks > 0) {
      if (lane == 0) acc_ready = mbar_wait(&acc_full, 0) ? 1 : 0;
      acc_ready = __shfl_sync(0xffffffffu, acc_ready, 0);
    }
    if (acc_ready) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // accumulator mb: lane = token of the 128-token block, columns = features, so a thread holds 32 consecutive
      // features of one token and writes them as 16-byte pieces
      const int q = warp & 3;               // TMEM lane quarter this warp may read
      const int mb = (w2 >> 2) % MB;        // token block = accumulator
      const int ch = w2 / (MB * 4);         // which half of the feature columns
      const int t = t0 + mb * BM + q * 32 + lane;
      const bool tvalid = t < T_;
      const int colbase = p.seg[sg].col0 + row0;
      const bool vec = (p.ldy % 8 == 0) && (colbase % 8 == 0) &&
                       (((reinterpret_cast<uintptr_t>(p.y) | reinterpret_cast<uintptr_t>(p.res) | reinterpret_cast<uintptr_t>(p.y2)) & 15) == 0);
      // Full rows of a 32 x 32 block are regrouped through shared memory (the pipeline stages are idle once the
      // accumulator is complete; each warp uses a private 4.5 KB piece) so that a store instruction writes whole 128-byte
      // lines (fp32 partials: 4 rows x 128 B; fp16 output: 8 rows x 64 B) instead of 32 scattered 16-byte pieces.
      uint8_t* stg = smem + (size_t)w2 * (32 * 144);
      const int tbase = t0 + mb * BM + q * 32;  // first token of this warp's rows
      if (mb < n_mb) {
        for (int c0 = ch * (BF / 2); c0 < min(nmma, (ch + 1) * (BF / 2)); c0 += 32) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mb * BF + c0), v);
          const int nf = min(32, min(p.bf, n_rows - row0) - c0);  // features of this chunk that exist and belong to this tile
          if (p.splits > 1) {
            if (vec && nf == 32) {
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<uint4*>(stg + lane * 144 + e * 4) = make_uint4(v[e], v[e + 1], v[e + 2], v[e + 3]);
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const int r = 4 * j + (lane >> 3), cq = lane & 7;
                const uint4 val = *reinterpret_cast<const uint4*>(stg + r * 144 + cq * 16);
                const int tt = tbase + r;
                if (tt < T_) *reinterpret_cast<uint4*>(p.partial + ((size_t)split * p.T + tt) * p.ldy + colbase + c0 + cq * 4) = val;
              }
              __syncwarp();
            } else if (tvalid) {
              float* dst = p.partial + ((size_t)split * p.T + t) * p.ldy + colbase + c0;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (e < nf) dst[e] = __uint_as_float(v[e]);
            }
          } else {
            if (vec && nf == 32) {
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const __half2 h = __floats2half2_rn(__uint_as_float(v[e + 2 * j]), __uint_as_float(v[e + 2 * j + 1]));
                  o[j] = *reinterpret_cast<const uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(stg + lane * 80 + e * 2) = make_uint4(o[0], o[1], o[2], o[3]);
              }
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int r = 8 * j + (lane >> 2), cq = lane & 3;
                const uint4 o4 = *reinterpret_cast<const uint4*>(stg + r * 80 + cq * 16);
                const int tt = tbase + r;
                if (tt < T_) {
                  const size_t off = (size_t)(rowoff + tt) * p.ldy + colbase + c0 + cq * 8;
                  *reinterpret_cast<uint4*>(p.y + off) = o4;
                  if (p.res) {
                    const uint4 r4 = *reinterpret_cast<const uint4*>(p.res + off);
                    const uint32_t oo[4] = {o4.x, o4.y, o4.z, o4.w}, rr[4] = {r4.x, r4.y, r4.z, r4.w};
                    uint32_t z[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                      const float2 a = __half22float2(u2h2(oo[u])), b = __half22float2(u2h2(rr[u]));
                      const __half2 h = __floats2half2_rn(b.x + a.x, b.y + a.y);
                      z[u] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(p.y2 + off) = make_uint4(z[0], z[1], z[2], z[3]);
                  }
                }
              }
              __syncwarp();
            } else if (tvalid) {
              __half* dst = p.y + (size_t)(rowoff + t) * p.ldy + colbase + c0;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (e < nf) {
                  const __half h = __float2half_rn(__uint_as_float(v[e]));
                  dst[e] = h;
                  if (p.res) {
                    const size_t off = (size_t)(rowoff + t) * p.ldy + colbase + c0 + e;
                    p.y2[off] = __float2half_rn(__half2float(p.res[off]) + __half2float(h));
                  }
                }
            }
          }
        }
      }
    } else if (nks > 0) {
      fail_s = 1;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (fail_s && threadIdx.x == 0) raise_status(p.status, 3);
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// y[t][c] = rn16(sum_s partial[s][t][c]) for c < n_cols, splits summed in ascending order; eight columns per thread when
// the row length allows 16-byte accesses
__global__ void gemm_splitk_reduce_kernel(const float* __restrict__ partial, __half* __restrict__ y, int T, int n_cols, int ldy,
                                          int splits, const __half* __restrict__ res, __half* __restrict__ y2) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const size_t plane = (size_t)T * ldy;
  if (n_cols % 8 == 0 && ldy % 8 == 0 &&
      (((reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(res) | reinterpret_cast<uintptr_t>(y2)) & 15) == 0)) {
    const int cg = n_cols / 8;
    const size_t total = (size_t)T * cg;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
      const size_t t = i / cg, c = (i % cg) * 8;
      const float* src = partial + t * ldy + c;
      float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
      for (int s = 1; s < splits; ++s) {
        const float4 a2 = *reinterpret_cast<const float4*>(src + s * plane), b2 = *reinterpret_cast<const float4*>(src + s * plane + 4);
        a.x += a2.x; a.y += a2.y; a.z += a2.z; a.w += a2.w;
        b.x += b2.x; b.y += b2.y; b.z += b2.z; b.w += b2.w;
      }
      const __half2 h0 = __floats2half2_rn(a.x, a.y), h1 = __floats2half2_rn(a.z, a.w), h2 = __floats2half2_rn(b.x, b.y),
                    h3 = __floats2half2_rn(b.z, b.w);
      uint4 o;
      o.x = *reinterpret_cast<const uint32_t*>(&h0);
      o.y = *reinterpret_cast<const uint32_t*>(&h1);
      o.z = *reinterpret_cast<const uint32_t*>(&h2);
      o.w = *reinterpret_cast<const uint32_t*>(&h3);
      *reinterpret_cast<uint4*>(y + t * ldy + c) = o;
      if (res) {
        const uint4 r4 = *reinterpret_cast<const uint4*>(res + t * ldy + c);
        const uint32_t oo[4] = {o.x, o.y, o.z, o.w}, rr[4] = {r4.x, r4.y, r4.z, r4.w};
        uint32_t z[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 p0 = __half22float2(u2h2(oo[j])), p1 = __half22float2(u2h2(rr[j]));
          const __half2 h = __floats2half2_rn(p1.x + p0.x, p1.y + p0.y);
          z[j] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(y2 + t * ldy + c) = make_uint4(z[0], z[1], z[2], z[3]);
      }
    }
    return;
  }
  const size_t total = (size_t)T * n_cols;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t t = i / n_cols, c = i % n_cols;
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += partial[(size_t)s * plane + t * ldy + c];
    const __half h = __float2half_rn(acc);
    y[t * ldy + c] = h;
    if (res) y2[t * ldy + c] = __float2half_rn(__half2float(res[t * ldy + c]) + __half2float(h));
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tile configuration and split-K factor for one launch, picked by a small cost model (SM cycles): the CTAs run in
// waves of sm_count; a wide k-step (256 x 256 x 64) costs about 1250 cycles and a narrow one (128 x 128 x 64) about 1150,
// both bound by the L2 traffic of the activation tile rather than by the tensor pipe, which is why few wide CTAs with
// split-K beat many narrow ones; split-K adds the fp32 partial traffic and a second launch.
struct GemmPlan {
  bool wide;
  int splits;
  int bf;  // feature rows per tile
};
// Cost model in SM cycles.  CTAs run in waves of sm_count.  A k-step (64 k) of a 256-token x w-feature tile is bound by
// shared-memory traffic: about 1250 cycles at w = 256, of which the part that scales with w (weight-tile stores and the
// tensor core's reads of them) is 60 %; a 128 x 128 k-step costs about 1150.  Narrower tiles than the configuration's
// full width are considered because they can even out the waves (28672 features at 512 tokens: 224 tiles of 256 take
// two waves of which the second is half empty; 276 tiles of 208 fill both).  Split-K adds the fp32 partial traffic and
// a second launch.
GemmPlan choose_plan(const int* seg_rows, int n_seg, int T, int n_cols, int total_ksteps, int sm_count, uint64_t scratch_bytes) {
  GemmPlan best{false, 1, 128};
  double best_cost = 1e30;
  for (int w = 0; w < 2; ++w) {
    const int tt = w ? 256 : 128, full = w ? 256 : 128;
    const int tchunks = (T + tt - 1) / tt;
    for (int bf = full; bf >= (w ? 160 : 128); bf -= 32) {  // multiples of 32: whole 32-column epilogue chunks
      int tiles = 0;
      for (int i = 0; i < n_seg; ++i) tiles += (seg_rows[i] + bf - 1) / bf;
      const int ctas = tiles * tchunks;
      const double kstep = w ? 1250.0 * (0.4 + 0.6 * bf / 256.0) : 1150.0;
      for (int s = 1; s <= 8; ++s) {
        if (s > 1 && (total_ksteps / s < 8 || (uint64_t)s * T * n_cols * 4 > scratch_bytes)) break;
        const int per = (total_ksteps + s - 1) / s;
        if ((s - 1) * per >= total_ksteps) continue;  // the last split would be empty
        const int waves = (ctas * s + sm_count - 1) / sm_count;
        double cost = (double)waves * (per * kstep + 9000.0);
        if (s > 1) cost += 8000.0 + (double)(s + 1) * T * n_cols * 4.0 / 2000.0;  // second launch + partials at ~2 KB per cycle
        if (cost < best_cost * 0.97 || (cost < best_cost && bf == full)) {  // a narrower tile has to pay for itself
          if (cost < best_cost) best_cost = cost;
          best = GemmPlan{w != 0, s, bf};
        }
      }
    }
  }
  return best;
}

}  // namespace

uint64_t gemm_scratch_bytes(int T, int n_total, int K) {
  // fp32 partials of the plan this shape gets with unlimited scratch (the launcher re-plans within the buffer it is given)
  const int total_ksteps = (K + BK - 1) / BK;
  const GemmPlan pl = choose_plan(&n_total, 1, T, n_total, total_ksteps, 148, ~0ull);
  return pl.splits > 1 ? (uint64_t)pl.splits * T * n_total * 4 + 256 : 256;
}

cudaError_t launch_gemm(const GemmParams& g, cudaStream_t st, uint64_t* n_launch, std::string* err) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) {
    if (err) *err = "cuTensorMapEncodeTiled is not available from the driver";
    return cudaErrorNotSupported;
  }
  if (((uintptr_t)g.x & 15) || (g.ldx % 8)) {
    if (err) *err = "GEMM activations must be 16-byte aligned with a leading dimension that is a multiple of 8";
    return cudaErrorInvalidValue;
  }
  CUtensorMap xmap;
  const cuuint64_t dims[2] = {(cuuint64_t)g.K, (cuuint64_t)g.T};
  const cuuint64_t strides[1] = {(cuuint64_t)g.ldx * 2};
  const cuuint32_t box[2] = {BK, BOXR};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(g.x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled failed for the activation tile";
    return cudaErrorInvalidValue;
  }
  CUtensorMap wmap = xmap;  // only read by the kernel when the weights are fp16
  if (g.w16) {
    if (g.n_seg != 1 || g.grp_off || ((uintptr_t)g.seg[0].base & 15) || (g.K % 8)) {
      if (err) *err = "fp16 weights: one 16-byte aligned matrix with K a multiple of 8";
      return cudaErrorInvalidValue;
    }
    const cuuint64_t wdims[2] = {(cuuint64_t)g.K, (cuuint64_t)g.seg[0].n_rows};
    const cuuint64_t wstrides[1] = {(cuuint64_t)g.K * 2};
    if (enc(&wmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint8_t*>(g.seg[0].base), wdims, wstrides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      if (err) *err = "cuTensorMapEncodeTiled failed for the weight tile";
      return cudaErrorInvalidValue;
    }
  }
  int sm_count = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  int n_total = 0;
  for (int i = 0; i < g.n_seg; ++i) n_total += g.seg[i].n_rows;
  int seg_rows[3] = {0, 0, 0};
  for (int i = 0; i < g.n_seg; ++i) seg_rows[i] = g.seg[i].n_rows;
  const int total_ksteps = (g.K + BK - 1) / BK;
  GemmPlan pl = choose_plan(seg_rows, g.n_seg, g.T, g.ldy, total_ksteps, sm_count, g.scratch ? g.scratch_bytes : 0);
  if (g.grp_off) {
    // per-expert row counts are small next to the tile: 128-token tiles unless an expert holds several of them
    if (g.res || g.n_groups <= 0 || g.grp_max_rows <= 0) return cudaErrorInvalidValue;
    pl = GemmPlan{g.grp_max_rows > 256, 1, g.grp_max_rows > 256 ? 256 : 128};
  }
  const bool wide = pl.wide;
  const int bf = pl.bf, tt = wide ? 256 : 128;
  GemmKParams p{};
  p.n_seg = g.n_seg;
  p.bf = bf;
  int tiles = 0, col = 0;
  for (int i = 0; i < g.n_seg; ++i) {
    p.seg[i] = GemmSeg{g.seg[i].base, g.seg[i].n_rows, tiles, col};
    tiles += (g.seg[i].n_rows + bf - 1) / bf;
    col += g.seg[i].n_rows;
  }
  const int tchunks = g.grp_off ? (g.grp_max_rows + tt - 1) / tt : (g.T + tt - 1) / tt;
  p.K = g.K;
  p.T = g.T;
  p.total_ksteps = total_ksteps;
  p.splits = pl.splits;
  p.ksteps_per_split = (p.total_ksteps + p.splits - 1) / p.splits;
  p.y = g.y;
  p.ldy = g.ldy;
  p.partial = (float*)g.scratch;
  p.status = g.status;
  p.res = g.res;
  p.y2 = g.y2;
  p.w16 = g.w16;
  p.grp_off = g.grp_off;
  p.grp_stride = g.grp_stride;
  for (int i = 0; i < 3; ++i) p.grp_tab[i] = g.grp_tab[i];
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e1 = cudaFuncSetAttribute(gemm_q4_kernel<2, 256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaError_t e2 = cudaFuncSetAttribute(gemm_q4_kernel<1, 128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaError_t e3 = cudaFuncSetAttribute(gemm_q4_kernel<2, 256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaError_t e4 = cudaFuncSetAttribute(gemm_q4_kernel<1, 128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e1 != cudaSuccess) return e1;
    if (e2 != cudaSuccess) return e2;
    if (e3 != cudaSuccess) return e3;
    if (e4 != cudaSuccess) return e4;
  }
  dim3 grid(tiles, tchunks, g.grp_off ? g.n_groups : p.splits);
  ++*n_launch;
  cudaError_t e;
  if (wide) {
    using Cfg = TileCfg<2, 256>;
    p.stages = Cfg::kStages;
    const size_t smem = (size_t)Cfg::kStages * Cfg::kStageBytes + 1024;
    e = g.mx ? launch_dep(gemm_q4_kernel<2, 256, true>, grid, dim3(Cfg::kThreads), smem, st, g.pdl, 1, xmap, wmap, p)
             : launch_dep(gemm_q4_kernel<2, 256, false>, grid, dim3(Cfg::kThreads), smem, st, g.pdl, 1, xmap, wmap, p);
  } else {
    using Cfg = TileCfg<1, 128>;
    // Grouped form: every CTA streams its own expert's weights once and has few real rows, so what counts is how many
    // weight loads are in flight per SM: three stages let two CTAs share an SM (registers are capped for that).
    p.stages = g.grp_off ? 3 : Cfg::kStages;
    const size_t smem = (size_t)p.stages * Cfg::kStageBytes + 1024;
    e = g.mx ? launch_dep(gemm_q4_kernel<1, 128, true>, grid, dim3(Cfg::kThreads), smem, st, g.pdl, 1, xmap, wmap, p)
             : launch_dep(gemm_q4_kernel<1, 128, false>, grid, dim3(Cfg::kThreads), smem, st, g.pdl, 1, xmap, wmap, p);
  }
  if (e != cudaSuccess) return e;
  if (p.splits > 1) {
    const size_t total = (size_t)g.T * col;
    const int blocks = (int)std::min<size_t>((total / 8 + 255) / 256 + 1, (size_t)sm_count * 8);
    ++*n_launch;
    e = launch_dep(gemm_splitk_reduce_kernel, dim3(blocks), dim3(256), 0, st, g.pdl, 1, (const float*)p.partial, g.y, g.T, col, g.ldy,
                   p.splits, g.res, g.y2);
  }
  return e;
}

// The split-K sum as a launch of its own, for the other GEMM kernels of the library.
cudaError_t launch_gemm_splitk_reduce(const float* partial, __half* y, int T, int n_cols, int ldy, int splits, const __half* res, __half* y2,
                                      int pdl, cudaStream_t st, uint64_t* n_launch) {
  int sm_count = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  const size_t total = (size_t)T * n_cols;
  const int blocks = (int)std::min<size_t>((total / 8 + 255) / 256 + 1, (size_t)sm_count * 8);
  ++*n_launch;
  return launch_dep(gemm_splitk_reduce_kernel, dim3(blocks), dim3(256), 0, st, pdl, 1, partial, y, T, n_cols, ldy, splits, res, y2);
}

// ---------------------------------------------------------------------------------------------------------------
// Split-K scratch that needs no allocation: a fixed array in the library's own device image.
// Every GPU that loads the library carries these 8 MiB from load until exit.
constexpr uint64_t kStaticScratchBytes = 8ull << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

uint64_t gemm_static_scratch_capacity() { return kStaticScratchBytes; }

// Device address of the array for the CURRENT device.  In host code the symbol's name is only a handle, not an address a
// kernel could use, so the address is asked from the runtime once per device and cached.
cudaError_t gemm_static_scratch(void** out) {
  static void* cached[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!cached[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return cudaSuccess;
}

}  // namespace ats
