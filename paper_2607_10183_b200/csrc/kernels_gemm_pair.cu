// fp16-weight GEMM as a pair of CTAs on two SMs (tcgen05 cta_group::2): Y[T][N] = X[T][K] * W^T, W an unquantized fp16 matrix.
//
// A single CTA that computes 256 tokens x 256 features reads 96 bytes of operands per cycle from shared memory while
// the tensor pipe is busy and refills 64 more: above the SM's 128.  As a pair, the instruction computes 256 tokens
// (128 from each CTA's shared memory) x 256 features (128 weight rows from each CTA's shared memory), so every CTA
// reads 64 bytes per cycle and refills 47.  Pair tile: 512 tokens (two 128-token blocks per CTA, one accumulator each,
// all 512 tensor-memory columns of both SMs) x 256 features.
//
// Roles in each CTA: warp 0 = TMA producer (activations of its 256 tokens and its 128 weight rows, boxes of 64 rows x 64 k,
// 128-byte swizzle), warp 1 = tensor-memory allocation (both CTAs, cta_group::2) and, in the leader (even rank) only,
// MMA issue; warps 2..9 = epilogue (tcgen05.ld of the CTA's own accumulators, fp16 stores).
// Barriers: the loads of BOTH CTAs complete on the leader's full barrier (loads carry cta_group::2 and name that barrier:
// the own barrier's address with the peer bit cleared), for which the leader posts the byte count of both; the leader's
// tcgen05.commit releases a stage in both CTAs (one commit per CTA: its own barrier, then the peer's through mapa).
// Every mbarrier wait is bounded; a CTA that gives up raises the status word and skips its work, but every thread still
// reaches the closing cluster barrier, so that no CTA leaves while its partner may still signal it.
#include <cuda.h>

#include "ats_internal.h"
#include "sm100_sync.cuh"

namespace ats {

namespace {

constexpr int BM = 128, BK = 64, BOXR = 64;
constexpr int kTokPerCta = 256, kFeatPerCta = 128;           // per CTA: two token blocks, half of the pair's 256 features
constexpr int kXBytes = kTokPerCta * BK * 2;                 // 32 KB
constexpr int kWBytes = kFeatPerCta * BK * 2;                // 16 KB
constexpr int kStageBytes = kXBytes + kWBytes;               // 48 KB
constexpr int kStages = 4;
constexpr int kThreads = 10 * 32;
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;               // clears the CTA-rank bit of a shared::cluster address

struct PairParams {
  int K, T, N;
  int ksteps;
  __half* y;
  int ldy;
  int* status;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the load of one 64-row x 64-k box; its bytes complete on the pair leader's barrier
__device__ __forceinline__ void tma_load_pair(void* dst, const CUtensorMap* map, int x, int y, uint64_t* own_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(own_bar) & kPeerBitMask)
      : "memory");
}
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;  // 128-byte swizzle
  return d;
}
// kind::f16, fp16 x fp16 -> fp32, both operands K-major, M = 256 over the pair, N = 256
__device__ __forceinline__ uint32_t umma_idesc_pair() { return (1u << 4) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24); }
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at shared::cluster address `bar_addr` when the pair's MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_addr) : "memory");
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

__global__ void __launch_bounds__(kThreads, 1)
    gemm_w16_pair_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap, const PairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full[kStages], empty[kStages], acc_full;
  __shared__ uint32_t tmem_base_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t rank = cluster_rank();     // 0 = leader
  const int pair = blockIdx.x >> 1;          // feature tile of the pair
  const int n0 = pair * 256 + (int)rank * kFeatPerCta;             // first weight row this CTA loads
  const int t0 = blockIdx.y * 512 + (int)rank * kTokPerCta;        // first token of this CTA
  const int nks = p.ksteps;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);   // the leader's own arrive.expect_tx; the bytes of both CTAs' loads complete on it
      mbar_init(&empty[s], 1);  // one commit from the leader's MMA thread
    }
    mbar_init(&acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // one warp of each CTA, same shared-memory offset and column count in both
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();  // both CTAs' barriers are initialised and their tensor memory allocated before anyone signals the other
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;
  if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");  // the activations come from the preceding kernel
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  bool failed = false;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < nks; ++i) {
        const int s = i % kStages;
        if (i >= kStages && !mbar_wait(&empty[s], ((i / kStages) - 1) & 1)) {
          failed = true;
          break;
        }
        uint8_t* st = smem + (size_t)s * kStageBytes;
        if (rank == 0) mbar_expect_tx(&full[s], 2u * kStageBytes);
        for (int b = 0; b < kTokPerCta / BOXR; ++b) tma_load_pair(st + kWBytes + (size_t)b * BOXR * BK * 2, &xmap, i * BK, t0 + b * BOXR, &full[s]);
        for (int b = 0; b < kFeatPerCta / BOXR; ++b) tma_load_pair(st + (size_t)b * BOXR * BK * 2, &wmap, i * BK, n0 + b * BOXR, &full[s]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_pair();
      const uint64_t desc0 = umma_desc(smem_u32(smem));
      uint32_t empty_peer[kStages];
#pragma unroll
      for (int s = 0; s < kStages; ++s) empty_peer[s] = map_to_cta(smem_u32(&empty[s]), 1);
      uint32_t accum = 0, par = 0;
      int s = 0;
      bool ok = true;
      for (int i = 0; i < nks; ++i) {
        if (!mbar_wait(&full[s], par)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t wdesc = desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kStageBytes >> 4));  // weight rows: the B operand (N)
        const uint64_t xdesc = wdesc + (uint64_t)(kWBytes >> 4);                                // activation rows: the A operand (M)
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
          for (int mb = 0; mb < 2; ++mb)
            umma_f16_pair(tmem_base + (uint32_t)(mb * 256), xdesc + (uint64_t)(mb * ((BM * BK * 2) >> 4) + 2 * kk), wdesc + (uint64_t)(2 * kk),
                          idesc, kk > 0 ? 1u : accum);
        }
        accum = 1;
        umma_commit_pair(smem_u32(&empty[s]));  // this CTA's producer may refill the stage ...
        umma_commit_pair(empty_peer[s]);        // ... and so may the partner's
        if (++s == kStages) {
          s = 0;
          par ^= 1;
        }
      }
      if (ok) {
        umma_commit_pair(smem_u32(&acc_full));
        umma_commit_pair(map_to_cta(smem_u32(&acc_full), 1));
      } else {
        failed = true;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's 256 tokens x 256 features
    const int w2 = warp - 2;           // 0..7
    const int q = warp & 3;            // tensor-memory lane quarter this warp may read
    const int half = w2 >> 2;          // which half of the 256 feature columns
    int ready = 0;
    if (nks > 0) {
      if (lane == 0) ready = mbar_wait(&acc_full, 0) ? 1 : 0;
      ready = __shfl_sync(0xffffffffu, ready, 0);
    }
    if (ready) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int nbase = pair * 256;
#pragma unroll 1
      for (int mb = 0; mb < 2; ++mb) {
        const int t = t0 + mb * BM + q * 32 + lane;
#pragma unroll 1
        for (int c0 = half * 128; c0 < half * 128 + 128; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mb * 256 + c0), v);
          if (t < p.T) {
            __half* dst = p.y + (size_t)t * p.ldy + nbase + c0;
            if (nbase + c0 + 32 <= p.N && (p.ldy % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.y) & 15) == 0)) {
#pragma unroll
              for (int e = 0; e < 32; e += 8) {
                uint32_t o[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                  const __half2 hh = __floats2half2_rn(__uint_as_float(v[e + 2 * h]), __uint_as_float(v[e + 2 * h + 1]));
                  o[h] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                *reinterpret_cast<uint4*>(dst + e) = make_uint4(o[0], o[1], o[2], o[3]);
              }
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (nbase + c0 + e < p.N) dst[e] = __float2half_rn(__uint_as_float(v[e]));
            }
          }
        }
      }
    } else if (nks > 0) {
      failed = true;
    }
  }
  if (failed && p.status) raise_status(p.status, 2);
  // nobody leaves, frees tensor memory or lets its shared memory go while the partner may still read or signal it
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

// ------------------------------------------------------------------------------------------- the dequantizing form
// The same pair for the 4-bit formats: the activation tiles come by TMA as above; each CTA's weight half-tile (128 rows x
// 64 k per stage) is written by its own sixteen dequantization warps (four threads per weight row, 16 k each, codes
// prefetched four k-steps ahead) in the canonical K-major 128-byte-swizzle layout.  A
// stage is full when the leader's barrier has seen the leader's expect_tx arrival, the bytes of both CTAs' activation
// loads and one arrival per dequantization warp of BOTH CTAs; the peer's warps arrive through mapa with the plain
// mbarrier.arrive (after the proxy fence that makes their stores visible to the tensor core).  With
// mbarrier.arrive.release.cluster instead, every arrival took about as long as a k-step and the kernel ran at 0.65 of the
// single-CTA kernel's rate.  Per pair and k-step each CTA dequantizes half of what a single CTA would for the same
// 512 x 256 outputs.  Measured against the single-CTA kernel: 6 to 12 % faster for long reductions (K >= 8192) from 128
// CTAs on (with few tiles: K split over blockIdx.z into fp32 partials that a second launch sums, 5 to 9 % faster from 1024
// tokens on), within +-4 % otherwise, which is where the launcher uses it.
struct PairSeg {
  const uint8_t* base;
  int n_rows;
  int tile0;  // first pair tile of the segment
  int col0;   // first output column of the segment
};
struct PairQParams {
  PairSeg seg[3];
  int n_seg;
  int K, T;
  int ksteps;
  __half* y;
  int ldy;
  const __half* res;  // optional residual: y2 = rn16(res + y)
  __half* y2;
  int* status;
  int splits, ksteps_per_split;  // split-K over blockIdx.z: fp32 partials [splits][T][ldy], summed by a second launch
  float* partial;
};
constexpr int kQStageBytes = kXBytes + kWBytes;  // weight half-tile first, then the activations (same layout as above)

__device__ __forceinline__ __half2 u2h2(uint32_t v) {
  __half2 h;
  *reinterpret_cast<uint32_t*>(&h) = v;
  return h;
}
// One code word (8 codes, internal nibble order) times the block scale -> 8 fp16 weights (k ascending) as one 16-byte chunk.
template <bool MX>
__device__ __forceinline__ uint4 dequant8_any(uint32_t w, __half2 s2) {
  __half2 c0, c1, c2, c3;
  if (MX) {
    const __half2 k2p14 = u2h2(0x74007400u);
    const uint32_t kMag = 0x0E000E00u, kSgn = 0x80008000u;
    c0 = __hmul2(__hmul2(u2h2(((w << 9) & kMag) | ((w << 12) & kSgn)), k2p14), s2);
    c1 = __hmul2(__hmul2(u2h2(((w << 5) & kMag) | ((w << 8) & kSgn)), k2p14), s2);
    c2 = __hmul2(__hmul2(u2h2(((w << 1) & kMag) | ((w << 4) & kSgn)), k2p14), s2);
    c3 = __hmul2(__hmul2(u2h2(((w >> 3) & kMag) | (w & kSgn)), k2p14), s2);
  } else {
    const uint32_t kMagic = 0x64006400u, w8 = w >> 8;
    const __half2 k1032 = u2h2(0x64086408u), k16th = u2h2(0x2C002C00u), kM72 = u2h2(0xD480D480u);
    c0 = __hmul2(__hsub2(u2h2((w & 0x000F000Fu) | kMagic), k1032), s2);
    c1 = __hmul2(__hfma2(u2h2((w & 0x00F000F0u) | kMagic), k16th, kM72), s2);
    c2 = __hmul2(__hsub2(u2h2((w8 & 0x000F000Fu) | kMagic), k1032), s2);
    c3 = __hmul2(__hfma2(u2h2((w8 & 0x00F000F0u) | kMagic), k16th, kM72), s2);
  }
  uint4 o;
  o.x = *reinterpret_cast<const uint32_t*>(&c0);
  o.y = *reinterpret_cast<const uint32_t*>(&c1);
  o.z = *reinterpret_cast<const uint32_t*>(&c2);
  o.w = *reinterpret_cast<const uint32_t*>(&c3);
  return o;
}
__device__ __forceinline__ void mbar_arrive_local(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// arrival on a barrier of another CTA of the cluster (address from mapa)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

constexpr int kQThreads = 18 * 32;
template <bool MX>
__global__ void __launch_bounds__(kQThreads, 1) gemm_q4_pair_kernel(const __grid_constant__ CUtensorMap xmap, const PairQParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full[kStages], empty[kStages], acc_full;
  __shared__ uint32_t tmem_base_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t rank = cluster_rank();
  const int pair = blockIdx.x >> 1;
  int sg = 0;
  while (sg + 1 < p.n_seg && pair >= p.seg[sg + 1].tile0) ++sg;
  const int prow0 = (pair - p.seg[sg].tile0) * 256;        // first row of the pair's tile within its segment
  const int row0 = prow0 + (int)rank * kFeatPerCta;        // first weight row this CTA dequantizes
  const int n_rows = p.seg[sg].n_rows;
  const int t0 = blockIdx.y * 512 + (int)rank * kTokPerCta;
  const int ks0 = (int)blockIdx.z * p.ksteps_per_split;
  const int nks = min(p.ksteps_per_split, p.ksteps - ks0);
  constexpr int kDqWarps = 16;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1 + 2 * kDqWarps);  // leader's expect_tx + one arrival per dequantization warp of both CTAs
      mbar_init(&empty[s], 1);
    }
    mbar_init(&acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;
  if (warp == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  bool failed = false;
  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < nks; ++i) {
        const int s = i % kStages;
        if (i >= kStages && !mbar_wait(&empty[s], ((i / kStages) - 1) & 1)) {
          failed = true;
          break;
        }
        uint8_t* st = smem + (size_t)s * kQStageBytes;
        if (rank == 0) mbar_expect_tx(&full[s], 2u * kXBytes);
        for (int b = 0; b < kTokPerCta / BOXR; ++b)
          tma_load_pair(st + kWBytes + (size_t)b * BOXR * BK * 2, &xmap, (ks0 + i) * BK, t0 + b * BOXR, &full[s]);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_pair();
      const uint64_t desc0 = umma_desc(smem_u32(smem));
      uint32_t empty_peer[kStages];
#pragma unroll
      for (int s = 0; s < kStages; ++s) empty_peer[s] = map_to_cta(smem_u32(&empty[s]), 1);
      uint32_t accum = 0, par = 0;
      int s = 0;
      bool ok = true;
      for (int i = 0; i < nks; ++i) {
        if (!mbar_wait(&full[s], par)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t wdesc = desc0 + (uint64_t)((uint32_t)s * (uint32_t)(kQStageBytes >> 4));
        const uint64_t xdesc = wdesc + (uint64_t)(kWBytes >> 4);
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
          for (int mb = 0; mb < 2; ++mb)
            umma_f16_pair(tmem_base + (uint32_t)(mb * 256), xdesc + (uint64_t)(mb * ((BM * BK * 2) >> 4) + 2 * kk), wdesc + (uint64_t)(2 * kk),
                          idesc, kk > 0 ? 1u : accum);
        }
        accum = 1;
        umma_commit_pair(smem_u32(&empty[s]));
        umma_commit_pair(empty_peer[s]);
        if (++s == kStages) {
          s = 0;
          par ^= 1;
        }
      }
      if (ok) {
        umma_commit_pair(smem_u32(&acc_full));
        umma_commit_pair(map_to_cta(smem_u32(&acc_full), 1));
      } else {
        failed = true;
      }
    }
  } else {
    // ------------------------------------------------------------ weight dequantization: thread = (row, 16 k of the k-step)
    // Sixteen warps for 128 rows: four adjacent lanes share a weight row, each expands two code words (16 k) per k-step.
    const int w2 = warp - 2;                 // 0..15
    const int r = w2 * 8 + (lane >> 2);      // row of this CTA's half-tile
    const int qd = lane & 3;                 // which 16-k quarter of the k-step: block qd / 2, words 2 (qd % 2) .. + 1 of it
    const int grow = row0 + r;
    const bool valid = grow < n_rows;
    const int K = p.K, nblk = K / 32;
    const uint8_t* segbase = p.seg[sg].base;
    const uint8_t* crow = segbase + (size_t)(valid ? grow : 0) * (K / 2);
    const __half* srow = reinterpret_cast<const __half*>(segbase + (size_t)n_rows * (K / 2)) + (size_t)(valid ? grow : 0) * nblk;
    uint32_t full_leader[kStages];
#pragma unroll
    for (int i = 0; i < kStages; ++i) full_leader[i] = map_to_cta(smem_u32(&full[i]), 0);
    constexpr int kPD = 4;
    uint2 qbuf[kPD];
    uint32_t sbuf[kPD];
    auto fetch = [&](int ks, uint2& q, uint32_t& sc) {
      const int kb = (ks0 + ks) * 2 + (qd >> 1);
      q = make_uint2(0, 0);
      sc = 0;
      if (valid && kb < nblk) {
        q = __ldg(reinterpret_cast<const uint2*>(crow + (size_t)kb * 16) + (qd & 1));
        sc = (uint32_t)__half_as_ushort(__ldg(srow + kb));
      }
    };
#pragma unroll
    for (int d = 0; d < kPD; ++d) {
      qbuf[d] = make_uint2(0, 0);
      sbuf[d] = 0;
      if (d < nks) fetch(d, qbuf[d], sbuf[d]);
    }
    bool ok = true;
    int s = 0, round = 0;
    const int sw = r & 7, cb = qd * 2;  // 16-byte chunks cb, cb + 1 of the row's 128 bytes
    for (int i0 = 0; i0 < nks && ok; i0 += kPD) {
#pragma unroll
      for (int d = 0; d < kPD; ++d) {
        const int i = i0 + d;
        if (i >= nks || !ok) break;
        const uint2 c0 = qbuf[d];
        const __half2 s0 = __half2half2(__ushort_as_half((unsigned short)sbuf[d]));
        if (i + kPD < nks) fetch(i + kPD, qbuf[d], sbuf[d]);
        const uint4 o0 = dequant8_any<MX>(c0.x, s0), o1 = dequant8_any<MX>(c0.y, s0);
        if (round > 0) {
          int got = 1;
          if (lane == 0) got = mbar_wait(&empty[s], (uint32_t)(round - 1) & 1u) ? 1 : 0;
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) {
            failed = true;
            ok = false;
            break;
          }
        }
        uint8_t* arow = smem + (size_t)s * kQStageBytes + (size_t)r * 128;
        *reinterpret_cast<uint4*>(arow + (((cb + 0) ^ sw) << 4)) = o0;
        *reinterpret_cast<uint4*>(arow + (((cb + 1) ^ sw) << 4)) = o1;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the stores become visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) {
          if (rank == 0) mbar_arrive_local(&full[s]);
          else mbar_arrive_cluster(full_leader[s]);
        }
        if (++s == kStages) {
          s = 0;
          ++round;
        }
      }
    }
    // ------------------------------------------------------------ epilogue: this CTA's 256 tokens x the pair's 256 features
    const int q = warp & 3;        // tensor-memory lane quarter this warp may read
    const int cq = w2 >> 2;        // which quarter (64 columns) of the 256 feature columns
    int ready = 0;
    if (ok && nks > 0) {
      if (lane == 0) ready = mbar_wait(&acc_full, 0) ? 1 : 0;
      ready = __shfl_sync(0xffffffffu, ready, 0);
    }
    if (ready) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int colbase = p.seg[sg].col0 + prow0;
      const bool vec = (p.ldy % 8 == 0) && (colbase % 8 == 0) &&
                       (((reinterpret_cast<uintptr_t>(p.y) | reinterpret_cast<uintptr_t>(p.res) | reinterpret_cast<uintptr_t>(p.y2)) & 15) == 0);
#pragma unroll 1
      for (int mb = 0; mb < 2; ++mb) {
        const int t = t0 + mb * BM + q * 32 + lane;
#pragma unroll 1
        for (int c0 = cq * 64; c0 < cq * 64 + 64; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(mb * 256 + c0), v);
          if (t >= p.T) continue;
          const int nf = min(32, n_rows - prow0 - c0);  // features of this chunk that exist
          if (nf <= 0) continue;
          if (p.splits > 1) {  // fp32 partial of this K range; the sum over the splits runs as a second launch
            float* pd = p.partial + ((size_t)blockIdx.z * p.T + t) * p.ldy + colbase + c0;
            if (nf == 32 && (p.ldy % 4 == 0) && (colbase % 4 == 0)) {
#pragma unroll
              for (int e = 0; e < 32; e += 4) *reinterpret_cast<uint4*>(pd + e) = make_uint4(v[e], v[e + 1], v[e + 2], v[e + 3]);
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (e < nf) pd[e] = __uint_as_float(v[e]);
            }
            continue;
          }
          __half* dst = p.y + (size_t)t * p.ldy + colbase + c0;
          const __half* rs = p.res ? p.res + (size_t)t * p.ldy + colbase + c0 : nullptr;
          __half* d2 = p.y2 ? p.y2 + (size_t)t * p.ldy + colbase + c0 : nullptr;
          if (vec && nf == 32) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint32_t o[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const __half2 hh = __floats2half2_rn(__uint_as_float(v[e + 2 * h]), __uint_as_float(v[e + 2 * h + 1]));
                o[h] = *reinterpret_cast<const uint32_t*>(&hh);
              }
              *reinterpret_cast<uint4*>(dst + e) = make_uint4(o[0], o[1], o[2], o[3]);
              if (rs) {
                const uint4 rv = *reinterpret_cast<const uint4*>(rs + e);
                const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
                uint32_t o2[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                  const float2 a = __half22float2(u2h2(o[h])), b = __half22float2(u2h2(rw[h]));
                  const __half2 hh = __floats2half2_rn(a.x + b.x, a.y + b.y);
                  o2[h] = *reinterpret_cast<const uint32_t*>(&hh);
                }
                *reinterpret_cast<uint4*>(d2 + e) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
              }
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (e < nf) {
                const __half hv = __float2half_rn(__uint_as_float(v[e]));
                dst[e] = hv;
                if (rs) d2[e] = __float2half_rn(__half2float(rs[e]) + __half2float(hv));
              }
          }
        }
      }
    } else if (nks > 0) {
      failed = true;
    }
  }
  if (failed && p.status) raise_status(p.status, 2);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster_sync_all();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace

// Shapes the pair kernels take: no grouping, operands aligned for TMA, and enough tiles to occupy three quarters of the SMs
// (they have no split-K: with fewer tiles the single-CTA kernel, which splits K, is faster; measured cross-over for fp16
// weights: 112 CTAs even, 128 and more 8 to 17 % faster, 64 and fewer slower).  fp16 weights: one matrix, no residual.
static long pair_ctas(const GemmParams& g) {
  long pairs = 0;
  for (int i = 0; i < g.n_seg; ++i) pairs += (g.seg[i].n_rows + 255) / 256;
  return 2L * pairs * ((g.T + 511) / 512);
}
// Split-K factor of the dequantizing pair kernel: enough K ranges to bring the grid to about one CTA per SM, each at
// least 16 k-steps long, as far as the scratch holds the fp32 partials.
static int pair_splits(const GemmParams& g) {
  const long ctas = pair_ctas(g);
  if (g.w16 || ctas >= 112) return 1;
  const int ksteps = (g.K + BK - 1) / BK;
  int n_cols = 0;
  for (int i = 0; i < g.n_seg; ++i) n_cols += g.seg[i].n_rows;
  int s = 1;
  while (s < 8 && ctas * s < 128 && ksteps / (s * 2) >= 16 && (uint64_t)(s * 2) * g.T * g.ldy * 4 <= (g.scratch ? g.scratch_bytes : 0)) s *= 2;
  return s;
}
bool gemm_pair_eligible(const GemmParams& g) {
  if (g.grp_off || g.n_seg < 1 || g.n_seg > 3) return false;
  if (g.T < 384 || g.ldx % 8 || g.K < BK || (reinterpret_cast<uintptr_t>(g.x) & 15)) return false;
  if (g.w16) {
    if (g.n_seg != 1 || g.res || g.y2 || g.K % 8 || (reinterpret_cast<uintptr_t>(g.seg[0].base) & 15)) return false;
    return pair_ctas(g) >= 112;
  }
  // 4-bit formats: only where the pair measured faster than the single-CTA kernel (see the comment at the kernel)
  if (g.K % 32 || g.K < 8192) return false;
  for (int i = 0; i < g.n_seg; ++i)
    if (reinterpret_cast<uintptr_t>(g.seg[i].base) & 15) return false;
  if ((g.res != nullptr) != (g.y2 != nullptr)) return false;
  const int splits = pair_splits(g);
  if (splits > 1 && g.T < 1024) return false;  // split over K the pair gains 5-9 % from 1024 tokens on, nothing at 512
  return pair_ctas(g) * splits >= 128;
}

cudaError_t launch_gemm_pair(const GemmParams& g, cudaStream_t st, uint64_t* n_launch, std::string* err) {
  if (!gemm_pair_eligible(g)) return cudaErrorInvalidValue;
  EncodeTiledFn enc = encode_fn();
  if (!enc) {
    if (err) *err = "cuTensorMapEncodeTiled is not available from the driver";
    return cudaErrorNotSupported;
  }
  CUtensorMap xmap, wmap;
  const cuuint32_t box[2] = {BK, BOXR}, estr[2] = {1, 1};
  const cuuint64_t xdims[2] = {(cuuint64_t)g.K, (cuuint64_t)g.T}, xstr[1] = {(cuuint64_t)g.ldx * 2};
  if (enc(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(g.x), xdims, xstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
    if (err) *err = "cuTensorMapEncodeTiled failed for the activation tile";
    return cudaErrorInvalidValue;
  }
  const size_t smem = (size_t)kStages * kStageBytes + 1024;
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e1 = cudaFuncSetAttribute(gemm_w16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaError_t e2 = cudaFuncSetAttribute(gemm_q4_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaError_t e3 = cudaFuncSetAttribute(gemm_q4_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e1 != cudaSuccess) return e1;
    if (e2 != cudaSuccess) return e2;
    if (e3 != cudaSuccess) return e3;
  }
  const int tchunks = (g.T + 511) / 512;
  ++*n_launch;
  if (g.w16) {
    const int N = g.seg[0].n_rows;
    const cuuint64_t wdims[2] = {(cuuint64_t)g.K, (cuuint64_t)N}, wstr[1] = {(cuuint64_t)g.K * 2};
    if (enc(&wmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint8_t*>(g.seg[0].base), wdims, wstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      if (err) *err = "cuTensorMapEncodeTiled failed for the weight tile";
      return cudaErrorInvalidValue;
    }
    PairParams p{};
    p.K = g.K;
    p.T = g.T;
    p.N = N;
    p.ksteps = (g.K + BK - 1) / BK;
    p.y = g.y;
    p.ldy = g.ldy;
    p.status = g.status;
    const dim3 grid(2 * ((N + 255) / 256), tchunks);
    return launch_dep(gemm_w16_pair_kernel, grid, dim3(kThreads), smem, st, g.pdl, 2, xmap, wmap, p);
  }
  PairQParams p{};
  p.n_seg = g.n_seg;
  int tiles = 0, col = 0;
  for (int i = 0; i < g.n_seg; ++i) {
    p.seg[i] = PairSeg{g.seg[i].base, g.seg[i].n_rows, tiles, col};
    tiles += (g.seg[i].n_rows + 255) / 256;
    col += g.seg[i].n_rows;
  }
  p.K = g.K;
  p.T = g.T;
  p.ksteps = (g.K + BK - 1) / BK;
  p.y = g.y;
  p.ldy = g.ldy;
  p.res = g.res;
  p.y2 = g.y2;
  p.status = g.status;
  p.splits = pair_splits(g);
  p.ksteps_per_split = (p.ksteps + p.splits - 1) / p.splits;
  while (p.splits > 1 && (p.splits - 1) * p.ksteps_per_split >= p.ksteps) {  // no empty K range
    --p.splits;
    p.ksteps_per_split = (p.ksteps + p.splits - 1) / p.splits;
  }
  p.partial = (float*)g.scratch;
  const dim3 grid(2 * tiles, tchunks, p.splits);
  cudaError_t e = g.mx ? launch_dep(gemm_q4_pair_kernel<true>, grid, dim3(kQThreads), smem, st, g.pdl, 2, xmap, p)
                       : launch_dep(gemm_q4_pair_kernel<false>, grid, dim3(kQThreads), smem, st, g.pdl, 2, xmap, p);
  if (e != cudaSuccess || p.splits == 1) return e;
  return launch_gemm_splitk_reduce(p.partial, g.y, g.T, col, g.ldy, p.splits, g.res, g.y2, g.pdl, st, n_launch);
}

}  // namespace ats
