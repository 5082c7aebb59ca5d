// Streaming decode GEMV for one token (sm_100a): the memory-bound hot kernel of the decode path.  Device code shared by
// the dense and the grouped-expert kernels: a producer function and a consumer function over a ring in shared memory.
//
// Structure: one persistent CTA per SM: 16 consumer warps in two groups of 8 + kProducerWarps producer warps.  The
// producers stream row tiles of the packed weights (codes and scales, contiguous byte ranges) into a ring of 8
// shared-memory stages with 1-D bulk-async copies (TMA) that complete on mbarriers; tiles alternate between the consumer
// groups; consumers never touch global memory for weights.  Several producer warps, because the bulk copies of ONE thread
// are served at about 30 GB/s however many of them are in flight (measured: a thread gets one 16 KB copy through per
// 0.5 us), less than an SM's share of the HBM stream, while copies issued from different warps proceed side by side:
// with one producer thread the ring took 4 us to request and the tile loop ran at the producer's pace.  Every lane owns
// up to two quantization blocks (32 k each) of a k-part of the row and keeps the activation for them in registers for the
// whole kernel, so a weight byte is read once from shared memory and an activation never again.
//
// Arithmetic: the activation block is re-expressed once per CTA as 16-bit block fixed point, x_k ~ xi_k * 2^-sh with
// sh chosen from the block's largest exponent (exact for every element within 2^-4 of the block maximum, rounded at
// 2^-16 of it otherwise: 32 times finer than fp16 resolves the maximum itself).  Pairs of xi meet pairs of masked 4-bit
// codes in dp2a: block dot products are exact integers; one fp32 multiply-add per block applies the scale, and blocks
// are accumulated in fp32.  sum_k (u_k - 8) x_k = sum_k u_k x_k - 8 sum_k x_k with the second term precomputed per
// block.  All integer instructions issue at half rate on this part and the dot-product pipe is the one that fills, so
// the instruction count per block (16 dp2a, 8 masks, 2 to combine) is what the format allows: the high nibbles are
// used in place as 16 * code and their sum shifted back once per block.  Lane partials are reduced by warp shuffles,
// k-parts through shared memory, both in fixed order.  A block that holds an Inf or a NaN activation yields NaN (the
// fixed-point form cannot carry it; the plain definition gives Inf or NaN there).
//
// Optional prologue: RMSNorm of the input row (fp16 or fp32) with an fp16 gain, rounded to fp16 (the operand edge of
// the numerics contract), computed once per CTA by all 512 consumer threads while the first weight tiles are in flight.
// All waits on mbarriers are bounded; on expiry the kernel raises a status word and returns.
#pragma once
#include "ats_internal.h"
#include "sm100_sync.cuh"

namespace ats {

namespace {

constexpr int kMaxStages = 8;
constexpr int kGroups = 2;         // consumer groups per CTA, each with its own stream of tiles
constexpr int kGroupWarps = 8;
constexpr int kConsumerWarps = kGroups * kGroupWarps;
constexpr int kConsumerThreads = kConsumerWarps * 32;
#ifndef ATS_PRODUCER_WARPS
#define ATS_PRODUCER_WARPS 2
#endif
constexpr int kProducerWarps = ATS_PRODUCER_WARPS;  // must not exceed the number of ring stages (see stream_produce)
constexpr int kThreads = kConsumerThreads + 32 * kProducerWarps;
constexpr int kRPW = 2;      // rows per consumer warp per tile
constexpr int kJ = 2;        // quantization blocks per lane per row
constexpr int kMaxDynSmem = 216 * 1024;  // ring + quantized activation row; 7 KB of static shared memory on top
// Stages requested before the consumers have issued their activation loads.  Measured on the config-2 step with two
// producer warps: 1 -> 38.1 us, 2 -> 37.4, 3 -> 37.2, 4 -> 37.4, 6 -> 37.8, 8 (no gating) -> 38.0: a few tiles must be on
// their way when the prologue ends, but a full ring of requests ahead of the activation loads delays those.
constexpr int kEarlyStages = 3;
constexpr int kMaxIt = 48;   // tiles of a CTA whose partial sums are buffered before a flush (at kRPW rows per warp)
// Short rows (K <= 1024: at most one quantization block per lane): a tile of the default geometry is a few kilobytes and
// the per-copy cost of the producers, not the memory, sets the pace.  Such shapes take twice the rows per tile, one block
// per lane, and four producer warps.
constexpr int kRPWShort = 4, kJShort = 1, kProducerWarpsShort = 4;
constexpr int kShortK = 1024;
constexpr int kThreadsShort = kConsumerThreads + 32 * kProducerWarpsShort;

#ifdef ATS_TRACE
// Timeline probe of development builds (-DATS_TRACE): stamps are collected in shared memory (cheap) and written out as
// (globaltimer, CTA, event, kernel tag) records when the CTA's consumers are done.
struct TraceRec {
  unsigned long long t;
  uint32_t cta;
  uint16_t ev, tag;
};
constexpr int kTraceCap = 1 << 16;
constexpr int kTraceLocal = 192;
__device__ TraceRec g_trace[kTraceCap];
__device__ unsigned int g_trace_n;
__shared__ unsigned long long tr_t[kTraceLocal];
__shared__ unsigned short tr_ev[kTraceLocal];
__shared__ unsigned int tr_n;
__device__ __forceinline__ void trace(int ev) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  const unsigned int i = atomicAdd(&tr_n, 1u);
  if (i < kTraceLocal) {
    tr_t[i] = t;
    tr_ev[i] = (unsigned short)ev;
  }
}
__device__ __forceinline__ void trace_flush(int tag) {
  const unsigned int n = min(tr_n, (unsigned)kTraceLocal);
  const unsigned int base = atomicAdd(&g_trace_n, n);
  for (unsigned int i = 0; i < n && base + i < kTraceCap; ++i)
    g_trace[base + i] = TraceRec{tr_t[i], blockIdx.x + 1000u * blockIdx.y, tr_ev[i], (uint16_t)tag};
}
#define ATS_TR(ev) do { if (threadIdx.x == 0 || threadIdx.x == 512) trace((ev)); } while (0)
#define ATS_TR_FLUSH() do { if (threadIdx.x == 0) trace_flush(p.K / 256 + 100 * p.mode); } while (0)
#define ATS_TR_INIT() do { if (threadIdx.x == 0) tr_n = 0; } while (0)
#else
#define ATS_TR(ev) do { } while (0)
#define ATS_TR_FLUSH() do { } while (0)
#define ATS_TR_INIT() do { } while (0)
#endif

// Weights are read once per call: the copies carry an evict-first L2 policy so that a step's 100+ MB of weights do not
// push the activations, the KV cache and the kernels' own instructions out of the L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol)
               : "memory");
}
// d = c + a.lo16 * b.byte0 + a.hi16 * b.byte1 (dp2a_lo) or with bytes 2, 3 (dp2a_hi): signed halves, unsigned bytes
__device__ __forceinline__ int dp2a_lo(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp2a.lo.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ int dp2a_hi(uint32_t a, uint32_t b, int c) {
  int d;
  asm("dp2a.hi.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// named barriers: 1 and 2 = the two consumer groups (256 threads each), 3 = all consumers (512); 0 is __syncthreads,
// which the producer warps would have to join
__device__ __forceinline__ void group_sync(int grp) {
  if (grp == 0)
    asm volatile("bar.sync 1, 256;" ::: "memory");
  else
    asm volatile("bar.sync 2, 256;" ::: "memory");
}
__device__ __forceinline__ void consumer_sync_all() { asm volatile("bar.sync 3, 512;" ::: "memory"); }

__device__ __forceinline__ float silu_mul_f(float g, float u) { return g / (1.0f + expf(-g)) * u; }

// rn(x * up) as an integer for |x * up| < 2^22 (up a power of two, so the product is exact): adding 1.5 * 2^23 leaves the
// rounded integer in the low mantissa bits.  One FMA and one integer add instead of a conversion instruction, which
// issues at a quarter of their rate.
__device__ __forceinline__ int f2i_magic(float x, float up) {
  return (int)__float_as_uint(fmaf(x, up, 12582912.0f)) - 0x4B400000;
}

// Layout of a quantized activation block (kXqWords words): the block's 32 activations as 16-bit block fixed point,
// xi_k = rn(x_k * 2^sh) with sh = 29 - E for the block's largest biased fp16 exponent E, so |xi| <= 32752: exact for
// every element within 2^-4 of the block maximum, rounded at 2^-16 of the maximum otherwise (32 times finer than
// fp16's own resolution at the maximum).  Code word w of a block holds codes k = 8w..8w+7 at nibble positions
// (0,2,4,6,1,3,5,7); (word & 0x0F0F0F0F) therefore carries k = 8w + {0,4,1,5} in its bytes and (word & 0xF0F0F0F0)
// carries 16 times the codes of k = 8w + {2,6,3,7}.  Words 4w..4w+3 of the block hold the pairs (xi_{8w+0}, xi_{8w+4}),
// (xi_{8w+1}, xi_{8w+5}), (xi_{8w+2}, xi_{8w+6}), (xi_{8w+3}, xi_{8w+7}) as two signed 16-bit halves (first in the
// low half): the operands of dp2a.lo / dp2a.hi against the two masked words.  Words 16 and 17 hold mul = 2^-sh and
// corr = -8 * sum(xi) * mul; both are NaN when the block holds an Inf or a NaN (fp32 exponent field 255), so that the
// block's term, and with it the output, is NaN.
//
// Microscaling 4-bit floats (MX): twice an element is an integer in [-12, 12]; the kernel looks the biased byte
// 2 e + 16 up per nibble (see mx_bytes) and uses the same unsigned dot products: sum xi (2 e + 16) = 2 sum xi e + 16 sum xi,
// so mul is halved and the correction stays -8 * sum(xi) * mul.  The lookup yields the bytes of a word's even k
// (0,2,4,6) and odd k (1,3,5,7), so for this format words 4w..4w+3 hold the pairs (xi_0, xi_2), (xi_4, xi_6), (xi_1, xi_3),
// (xi_5, xi_7) of the run.
constexpr int kXqWords = 20;  // 18 used; the 80-byte pitch keeps the 128-bit reads of consecutive blocks conflict-free

// The shift of a block from the largest fp32 exponent field m among its (fp16-valued) elements.
// fp16 exponent field E = m - 112 (normals); subnormal fp16 values have fp32 fields <= 112 -> E = 1.  sh = 29 - E: the
// largest fp16 magnitude with field E, (2 - 2^-10) 2^(E-15), maps to 32752.
__device__ __forceinline__ void block_scale(uint32_t m, float& up, float& mul) {
  const int E = max((int)m - 112, 1);
  const int sh = 29 - E;
  up = __uint_as_float((uint32_t)(sh + 127) << 23);
  mul = m == 255u ? __uint_as_float(0x7FC00000u) : __uint_as_float((uint32_t)(127 - sh) << 23);
}

// One run of 8 consecutive elements (one code word's worth) -> its four words of the block.
template <bool MX>
__device__ __forceinline__ uint4 pack_run(const int (&xi)[8]) {
  uint4 o;
  if (MX) {
    o.x = __byte_perm((uint32_t)xi[0], (uint32_t)xi[2], 0x5410u);
    o.y = __byte_perm((uint32_t)xi[4], (uint32_t)xi[6], 0x5410u);
    o.z = __byte_perm((uint32_t)xi[1], (uint32_t)xi[3], 0x5410u);
    o.w = __byte_perm((uint32_t)xi[5], (uint32_t)xi[7], 0x5410u);
  } else {
    o.x = __byte_perm((uint32_t)xi[0], (uint32_t)xi[4], 0x5410u);
    o.y = __byte_perm((uint32_t)xi[1], (uint32_t)xi[5], 0x5410u);
    o.z = __byte_perm((uint32_t)xi[2], (uint32_t)xi[6], 0x5410u);
    o.w = __byte_perm((uint32_t)xi[3], (uint32_t)xi[7], 0x5410u);
  }
  return o;
}

// Four adjacent lanes each hold one run of a 32-element block; exponent maximum and integer sum are shared by two
// butterfly shuffles.  Lane w of the group writes words 4w..4w+3 (and lane 0 the two scalars).
template <bool MX>
__device__ __forceinline__ void quantize_run4(const float (&x)[8], int w, uint32_t* blk) {
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) m = max(m, (__float_as_uint(x[i]) >> 23) & 0xFFu);  // fp32 exponent field of an fp16-valued number
  m = max(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = max(m, __shfl_xor_sync(0xffffffffu, m, 2));
  float up, mul;
  block_scale(m, up, mul);
  int xi[8];
  int sx = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    xi[i] = f2i_magic(x[i], up);
    sx += xi[i];
  }
  sx += __shfl_xor_sync(0xffffffffu, sx, 1);
  sx += __shfl_xor_sync(0xffffffffu, sx, 2);
  *reinterpret_cast<uint4*>(blk + 4 * w) = pack_run<MX>(xi);
  if (w == 0) *reinterpret_cast<float2*>(blk + 16) = make_float2(MX ? 0.5f * mul : mul, -8.0f * (float)sx * mul);
}

// Four nibbles (the low 16 bits of sel: sign bit, three magnitude bits each) -> the bytes 2 e + 16 of their elements.
// Twice the magnitudes are v = 0 1 2 3 4 6 8 12.  Two eight-byte tables for prmt: 16 - v, looked up with the sign bits
// masked out, and 2 v, looked up with the sign bit left in the selector, where prmt returns the sign of the table byte
// (0: every entry is positive) instead of the byte.  Their sum is 16 + v for a non-negative element and 16 - v for a
// negative one; no byte exceeds 40, so one 32-bit addition adds the four bytes without carries.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));  // generic form: selector bit 3 = replicate the byte's sign
  return d;
}
__device__ __forceinline__ uint32_t mx_bytes(uint32_t sel) {
  return prmt(0x0D0E0F10u, 0x04080A0Cu, sel & 0x7777u) + prmt(0x06040200u, 0x18100C08u, sel);
}

struct StreamSeg {
  const uint8_t* base;
  int n_rows;
  int tile0;  // first tile index of the segment
};

struct StreamParams {
  StreamSeg seg[3];
  int n_seg;
  int n_tiles;
  int K;
  int mode;
  int n_stages;  // ring stages of this launch (<= kMaxStages), chosen by the host from the shared-memory budget
  // activation source: x16 (already the operand), or a row to RMS-normalise first
  const __half* x16;
  const __half* norm_in16;
  const float* norm_in32;
  const __half* gain;
  float eps;
  __half* h_out;  // optional copy of the normalised operand (written by CTA 0)
  float* y32;
  __half* y16;
  const float* res32;
  const __half* res16;
  int* status;
  // test hooks (0 / -1 in production): limit of the bounded waits in SM cycles, and a tile whose copies the producer
  // leaves out, so that a test can make a wait run out without anything faulting
  long long wait_limit;
  int withhold_tile;
};

// Shared state of a CTA's ring; lives in static shared memory.
struct StreamShared {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t xbar;  // consumers -> producers: the activation loads have been issued
  float part_s[kGroups][kMaxIt * kGroupWarps * kRPW];
  float red_s[kConsumerWarps];
  int fail_g[kGroups];  // a warp of the group gave up a bounded wait (written and read by that group only)
};

__device__ __forceinline__ void stream_init(StreamShared& sh, int n_stages) {
  ATS_TR_INIT();
  if (threadIdx.x == 0) {
    for (int g = 0; g < kGroups; ++g) sh.fail_g[g] = 0;
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&sh.full[s], 1);
      mbar_init(&sh.empty[s], kGroupWarps);
    }
    mbar_init(&sh.xbar, kConsumerWarps);
    mbar_fence_init();
  }
  __syncthreads();
}

// (stage, ring cycle) of an iteration -> those of the iteration `step` later (step <= n_stages)
__device__ __forceinline__ void stream_advance(int& s, int& cyc, int step, int n_stages) {
  s += step;
  if (s >= n_stages) {
    s -= n_stages;
    ++cyc;
  }
}

__device__ __forceinline__ int stream_n_it(const StreamParams& p, int bx, int gx) {
  return bx < p.n_tiles ? (p.n_tiles - bx + gx - 1) / gx : 0;
}

// One elected thread of each producer warp requests tiles; producer warp w of the kProducerWarps takes the CTA's
// iterations it = w, w + kProducerWarps, ...  Before it refills a stage a producer waits for the PARITY of the phase in
// which the consumers released the stage's previous content; that test is only unambiguous while no producer runs a whole
// ring cycle ahead of the consumers, which holds as long as the number of producer warps (PW) <= n_stages (a producer's previous iteration
// waited for a release at most one ring cycle older).  bx / gx: index of this CTA among the gx CTAs that share the work described by p.  The weights do not depend
// on the preceding kernel, so nothing here waits for it (callers whose weight ADDRESSES come from the preceding kernel
// wait before they call).  Returns false after a bounded wait ran out (status word raised).
template <int PARTS, bool SW, int RPW = kRPW, int PW = kProducerWarps>
__device__ __forceinline__ bool stream_produce(const StreamParams& p, const int bx, const int gx, const int pw, StreamShared& sh,
                                               uint8_t* stages, const uint64_t pol) {
  constexpr int ROWS = kGroupWarps / PARTS * RPW;     // weight rows per tile
  constexpr int OUT_ROWS = SW ? ROWS / 2 : ROWS;       // output rows per tile
  const int row_codes = p.K / 2, row_scales = p.K / 16;
  const int stage_bytes = ROWS * (row_codes + row_scales);
  const int n_it = stream_n_it(p, bx, gx);
  const int n_stages = p.n_stages;
  const long long limit = p.wait_limit ? p.wait_limit : kWaitLimitCycles;
  ATS_TR(7);
  bool x_issued = false;
  // stage and ring cycle of iteration it, kept incrementally (the ring size is a run-time value)
  int s = pw % n_stages, cyc = pw / n_stages;
  for (int it = pw; it < n_it; it += PW) {
    // Weight copies queued ahead of the consumers' activation loads delay them (the row is a cache hit that then waits
    // behind megabytes of misses): kEarlyStages stages go out at once, the rest after those loads have been issued.
    if (it >= kEarlyStages && !x_issued) {
      if (!mbar_wait_suspending(&sh.xbar, 0, limit)) {
        raise_status(p.status, 3);
        return false;
      }
      x_issued = true;
    }
    if (cyc > 0 && !mbar_wait_suspending(&sh.empty[s], (cyc - 1) & 1, limit)) {
      raise_status(p.status, 2);
      return false;
    }
    const int tile = bx + it * gx;
    uint8_t* dst = stages + (size_t)s * stage_bytes;
    mbar_expect_tx(&sh.full[s], (uint32_t)stage_bytes);
    if (pw == 0) ATS_TR(300 + it);
    if (tile == p.withhold_tile) {  // test hook: this stage never fills
      stream_advance(s, cyc, PW, n_stages);
      continue;
    }
    if (SW) {
      // gate rows land in stage rows [0, ROWS/2), up rows in [ROWS/2, ROWS)
      const size_t r0 = (size_t)tile * OUT_ROWS;
      const uint8_t *g = p.seg[0].base, *u = p.seg[1].base;
      const size_t n = (size_t)p.seg[0].n_rows;
      bulk_g2s(dst, g + r0 * row_codes, OUT_ROWS * row_codes, &sh.full[s], pol);
      bulk_g2s(dst + OUT_ROWS * row_codes, u + r0 * row_codes, OUT_ROWS * row_codes, &sh.full[s], pol);
      uint8_t* sd = dst + ROWS * row_codes;
      bulk_g2s(sd, g + n * row_codes + r0 * row_scales, OUT_ROWS * row_scales, &sh.full[s], pol);
      bulk_g2s(sd + OUT_ROWS * row_scales, u + n * row_codes + r0 * row_scales, OUT_ROWS * row_scales, &sh.full[s], pol);
    } else {
      int sg = 0;
      while (sg + 1 < p.n_seg && tile >= p.seg[sg + 1].tile0) ++sg;
      const size_t r0 = (size_t)(tile - p.seg[sg].tile0) * ROWS;
      const uint8_t* b = p.seg[sg].base;
      bulk_g2s(dst, b + r0 * row_codes, ROWS * row_codes, &sh.full[s], pol);
      bulk_g2s(dst + ROWS * row_codes, b + (size_t)p.seg[sg].n_rows * row_codes + r0 * row_scales, ROWS * row_scales, &sh.full[s], pol);
    }
    stream_advance(s, cyc, PW, n_stages);
  }
  ATS_TR(9);
  return true;
}

__device__ __forceinline__ void unpack_h8(const uint4 a, float (&xv)[8]) {
  const uint32_t w4[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    __half2 h2;
    *reinterpret_cast<uint32_t*>(&h2) = w4[q];
    const float2 f = __half22float2(h2);
    xv[2 * q] = f.x;
    xv[2 * q + 1] = f.y;
  }
}

// The 16 consumer warps of a CTA: wait for the preceding kernel, activation prologue, the CTA's tiles, the epilogue.
// Two groups of 8 warps; the CTA's tiles alternate between the groups, each group with its own partial-sum buffer and
// barrier, so the tile loop is that of two independent 8-warp CTAs; what they share is the ring and the activation
// prologue: all 512 consumer threads load, normalise and quantise the row ONCE per SM.
// dep_resolved: the caller has already executed griddepcontrol.wait.  The dependent launch is released after the prologue.  Returns false after a bounded wait ran out (status word raised).
template <int PARTS, bool SW, bool MX, int RPW = kRPW, int J = kJ>
__device__ __forceinline__ bool stream_consume(const StreamParams& p, const int bx, const int gx, StreamShared& sh, const uint8_t* stages,
                                               uint32_t* xq_s, const bool dep_resolved) {
  constexpr int ROWS = kGroupWarps / PARTS * RPW;     // weight rows per tile
  constexpr int MAXIT = kMaxIt * kRPW / RPW;           // tiles whose partial sums fit the buffer
  constexpr int OUT_ROWS = SW ? ROWS / 2 : ROWS;       // output rows per tile
  const int K = p.K, nblk = K / 32;
  const int row_codes = K / 2, row_scales = K / 16;
  const int stage_bytes = ROWS * (row_codes + row_scales);
  const int n_it = stream_n_it(p, bx, gx);
  const int n_stages = p.n_stages;
  const long long limit = p.wait_limit ? p.wait_limit : kWaitLimitCycles;
  const int tid = threadIdx.x;  // 0..511
  const int lane = tid & 31, warp = tid >> 5;
  const int grp = warp / kGroupWarps;         // which of the two tile streams
  const int wg = warp % kGroupWarps;          // warp within the group
  const int tg = tid % (kGroupWarps * 32);    // thread within the group
  const int part = wg % PARTS, rsub = wg / PARTS;
  const int pblk = (nblk + PARTS - 1) / PARTS;
  const int b0 = part * pblk, b1 = min(nblk, b0 + pblk);
  uint32_t xr[J][16];
  float xm[J], xc[J];
  ATS_TR(0);
  {
    // Thread t owns the runs of 8 consecutive elements r = t + 512 j (one run when K <= 4096, up to four for K = 16384);
    // four adjacent lanes hold one 32-element block.  The optional RMSNorm (h = rn16(x * g / sqrt(mean(x^2) + eps)),
    // K <= 4096) and the block quantization work on those registers; the quantized blocks go to shared memory once
    // per CTA and every lane then fetches the blocks of its k-part.
    if (p.gain) {
      // The norm gains are parameters, not products of the preceding kernel: fetch them before waiting for it.
      const int i0 = tid * 8;
      const bool has = i0 < K;
      const uint4 graw = has ? __ldg(reinterpret_cast<const uint4*>(p.gain + i0)) : make_uint4(0, 0, 0, 0);
      if (!dep_resolved) asm volatile("griddepcontrol.wait;" ::: "memory");
      float xv[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) xv[q] = 0.f;
      if (has) {
        if (p.norm_in32) {
          const float4 a = *reinterpret_cast<const float4*>(p.norm_in32 + i0);
          const float4 b = *reinterpret_cast<const float4*>(p.norm_in32 + i0 + 4);
          xv[0] = a.x; xv[1] = a.y; xv[2] = a.z; xv[3] = a.w;
          xv[4] = b.x; xv[5] = b.y; xv[6] = b.z; xv[7] = b.w;
        } else {
          unpack_h8(*reinterpret_cast<const uint4*>(p.norm_in16 + i0), xv);
        }
      }
      ATS_TR(1);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.xbar);
      float ss = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) ss = fmaf(xv[q], xv[q], ss);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (lane == 0) sh.red_s[warp] = ss;
      consumer_sync_all();
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < kConsumerWarps; ++w) tot += sh.red_s[w];
      const float inv = 1.0f / sqrtf(tot / (float)K + p.eps);
      if (has) {
        const uint32_t gw[4] = {graw.x, graw.y, graw.z, graw.w};
        uint32_t o4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          __half2 g2;
          *reinterpret_cast<uint32_t*>(&g2) = gw[q];
          const float2 gf = __half22float2(g2);
          const __half2 h2 = __floats2half2_rn(xv[2 * q] * gf.x * inv, xv[2 * q + 1] * gf.y * inv);
          o4[q] = *reinterpret_cast<const uint32_t*>(&h2);
          const float2 f = __half22float2(h2);  // the operand is the fp16-rounded value
          xv[2 * q] = f.x;
          xv[2 * q + 1] = f.y;
        }
        if (p.h_out && bx == 0) *reinterpret_cast<uint4*>(p.h_out + i0) = make_uint4(o4[0], o4[1], o4[2], o4[3]);
        quantize_run4<MX>(xv, tid & 3, xq_s + (size_t)(tid >> 2) * kXqWords);
      }
    } else {
      if (!dep_resolved) asm volatile("griddepcontrol.wait;" ::: "memory");
      uint4 raw[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = tid + kConsumerThreads * j;  // run index; block r / 4, word r % 4.  All four lanes of a block are in range together.
        if (r * 8 < K) raw[j] = *reinterpret_cast<const uint4*>(p.x16 + r * 8);
      }
      ATS_TR(1);
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.xbar);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = tid + kConsumerThreads * j;
        if (r * 8 < K) {
          float xv[8];
          unpack_h8(raw[j], xv);
          quantize_run4<MX>(xv, r & 3, xq_s + (size_t)(r >> 2) * kXqWords);
        }
      }
    }
    ATS_TR(2);
    consumer_sync_all();
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const int b = b0 + lane + 32 * j;
      if (b < b1) {
        const uint4* src = reinterpret_cast<const uint4*>(xq_s + (size_t)b * kXqWords);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 v = src[q];
          xr[j][4 * q] = v.x;
          xr[j][4 * q + 1] = v.y;
          xr[j][4 * q + 2] = v.z;
          xr[j][4 * q + 3] = v.w;
        }
        const float2 mc = *reinterpret_cast<const float2*>(xq_s + (size_t)b * kXqWords + 16);
        xm[j] = mc.x;
        xc[j] = mc.y;
      } else {
#pragma unroll
        for (int q = 0; q < 16; ++q) xr[j][q] = 0;
        xm[j] = 0.f;
        xc[j] = 0.f;
      }
    }
  }
  ATS_TR(3);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // this group's tiles: it = grp, grp + 2, ...; li counts them.  The cross-lane reduction of a tile's row sums is
  // deferred into the next tile's iteration, where its shuffle latencies hide behind that tile's integer work.
  const int n_li = n_it > grp ? (n_it - grp + kGroups - 1) / kGroups : 0;
  float* my_part = sh.part_s[grp];
  bool failed = false;
  int s = grp % n_stages, cyc = grp / n_stages;  // stage and ring cycle of the group's next tile
  auto reduce_store = [&](float (&a)[RPW], int slot) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int r = 0; r < RPW; ++r) a[r] += __shfl_xor_sync(0xffffffffu, a[r], o);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < RPW; ++r) my_part[(slot * ROWS + r * (ROWS / RPW) + rsub) * PARTS + part] = a[r];
    }
  };
  for (int li0 = 0; li0 < n_li; li0 += MAXIT) {
    const int li1 = min(n_li, li0 + MAXIT);
    float prev[RPW];
    bool have_prev = false;
    for (int li = li0; li < li1; ++li) {
      [[maybe_unused]] const int it = grp + kGroups * li;
      if (!__all_sync(0xffffffffu, mbar_wait_suspending(&sh.full[s], cyc & 1, limit))) {
        failed = true;
        break;
      }
      if (li == 0) ATS_TR(4);
      ATS_TR(100 + it);
      const uint8_t* st = stages + (size_t)s * stage_bytes;
      uint4 cw[RPW][J];
      float sc[RPW][J];
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        const int row = r * (ROWS / RPW) + rsub;  // stage row of this warp's r-th row
        const uint4* codes = reinterpret_cast<const uint4*>(st + (size_t)row * row_codes);
        const __half* scp = reinterpret_cast<const __half*>(st + (size_t)ROWS * row_codes + (size_t)row * row_scales);
#pragma unroll
        for (int j = 0; j < J; ++j) {
          const int b = b0 + lane + 32 * j;
          const bool in = b < b1;
          cw[r][j] = in ? codes[b] : make_uint4(0, 0, 0, 0);
          sc[r][j] = in ? __half2float(scp[b]) : 0.f;
        }
      }
      // The stage is released as soon as its words are in registers, not after the arithmetic on them: a stage that is
      // held while it is being computed on is a stage that is not in flight, and the ring is what keeps HBM busy.  The
      // fold below makes the release wait for every load (an instruction issues only when its operands have arrived).
      {
        uint32_t fold = 0;
#pragma unroll
        for (int r = 0; r < RPW; ++r)
#pragma unroll
          for (int j = 0; j < J; ++j) fold ^= cw[r][j].x ^ cw[r][j].y ^ cw[r][j].z ^ cw[r][j].w ^ __float_as_uint(sc[r][j]);
        asm volatile("" ::"r"(fold) : "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
      }
      if (have_prev) reduce_store(prev, li - 1 - li0);
      float acc[RPW];
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        acc[r] = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
          const uint32_t ws[4] = {cw[r][j].x, cw[r][j].y, cw[r][j].z, cw[r][j].w};
          int dl = 0, dh = 0;
#pragma unroll
          for (int w = 0; w < 4; ++w) {
            if (MX) {
              const uint32_t ev = mx_bytes(ws[w]), od = mx_bytes(ws[w] >> 16);  // k = 0 2 4 6 and k = 1 3 5 7 of the word
              dl = dp2a_lo(xr[j][4 * w], ev, dl);
              dl = dp2a_hi(xr[j][4 * w + 1], ev, dl);
              dh = dp2a_lo(xr[j][4 * w + 2], od, dh);
              dh = dp2a_hi(xr[j][4 * w + 3], od, dh);
            } else {
              const uint32_t lo = ws[w] & 0x0F0F0F0Fu, hi = ws[w] & 0xF0F0F0F0u;  // hi carries 16 * code
              dl = dp2a_lo(xr[j][4 * w], lo, dl);
              dl = dp2a_hi(xr[j][4 * w + 1], lo, dl);
              dh = dp2a_lo(xr[j][4 * w + 2], hi, dh);
              dh = dp2a_hi(xr[j][4 * w + 3], hi, dh);
            }
          }
          // integer codes: dh is a multiple of 16; either way |dot| < 2^24: exact
          const float dot = MX ? (float)(dl + dh) : (float)(dl + (dh >> 4));
          acc[r] = fmaf(sc[r][j], fmaf(dot, xm[j], xc[j]), acc[r]);
        }
      }
      ATS_TR(200 + it);
      stream_advance(s, cyc, kGroups, n_stages);
#pragma unroll
      for (int r = 0; r < RPW; ++r) prev[r] = acc[r];
      have_prev = true;
    }
    if (have_prev && !failed) reduce_store(prev, li1 - 1 - li0);
    ATS_TR(5);
    if (failed) sh.fail_g[grp] = 1;
    group_sync(grp);
    if (sh.fail_g[grp]) {  // a warp of this group gave up; every thread of the group reads the same flag and leaves here
      if (tg == 0) raise_status(p.status, 1);
      return false;
    }
    // flush: sum the k-parts (ascending) and run the epilogue
    const int n_out = (li1 - li0) * OUT_ROWS;
    for (int i = tg; i < n_out; i += kGroupWarps * 32) {
      const int itl = i / OUT_ROWS, j = i % OUT_ROWS;
      const int tile = bx + (grp + kGroups * (li0 + itl)) * gx;
      float v[2];
#pragma unroll
      for (int h = 0; h < (SW ? 2 : 1); ++h) {
        const float* ps = my_part + ((size_t)itl * ROWS + j + h * OUT_ROWS) * PARTS;
        float t = 0.f;
#pragma unroll
        for (int q = 0; q < PARTS; ++q) t += ps[q];
        v[h] = t;
      }
      if (SW) {
        p.y16[(size_t)tile * OUT_ROWS + j] = __float2half_rn(silu_mul_f(v[0], v[1]));
      } else {
        // output index: rows of the segments lie side by side
        int sg = 0;
        while (sg + 1 < p.n_seg && tile >= p.seg[sg + 1].tile0) ++sg;
        int row = (tile - p.seg[sg].tile0) * ROWS + j;
        for (int q = 0; q < sg; ++q) row += p.seg[q].n_rows;
        switch (p.mode) {
          case GEMV_OUT_F32: p.y32[row] = v[0]; break;
          case GEMV_OUT_F16: p.y16[row] = __float2half_rn(v[0]); break;
          case GEMV_RES16_OUT_F32: p.y32[row] = __half2float(p.res16[row]) + v[0]; break;
          case GEMV_RES32_OUT_F16: p.y16[row] = __float2half_rn(p.res32[row] + v[0]); break;
          case GEMV_RES16_OUT_F16: p.y16[row] = __float2half_rn(__half2float(p.res16[row]) + v[0]); break;
          default: break;
        }
      }
    }
    group_sync(grp);
  }
  ATS_TR(6);
  ATS_TR_FLUSH();
  return true;
}

// ------------------------------------------------------------------ host side: shapes the kernel takes, its parameters
inline int stream_parts_for(int K) { return K <= 2048 ? 1 : K <= 4096 ? 2 : K <= 8192 ? 4 : 8; }
inline bool stream_short(int K) { return K <= kShortK; }                       // the wide-tile geometry applies
inline int stream_rpw_for(int K) { return stream_short(K) ? kRPWShort : kRPW; }
inline int stream_producers_for(int K) { return stream_short(K) ? kProducerWarpsShort : kProducerWarps; }

inline bool stream_shape_ok(const GemvParams& p) {
  if (p.M != 1 || p.K % 256 != 0 || p.K > 16384) return false;
  const int parts = stream_parts_for(p.K);
  const int rows = kGroupWarps / parts * stream_rpw_for(p.K);
  if (p.mode == GEMV_SWIGLU_F16) {
    if (p.n_seg != 2 || p.seg[0].n_rows != p.seg[1].n_rows || p.seg[0].n_rows % (rows / 2)) return false;
  } else {
    for (int s = 0; s < p.n_seg; ++s)
      if (p.seg[s].n_rows % rows) return false;
  }
  if (p.norm_gain && p.K > 4096) return false;  // the fused norm prologue covers hidden sizes up to 4096
  return true;
}

// Bytes of one ring stage and of the quantized activation row, and the number of stages that fit the SM.
inline size_t stream_stage_bytes(int K) { return (size_t)(kGroupWarps / stream_parts_for(K) * stream_rpw_for(K)) * (K / 2 + K / 16); }
inline size_t stream_xq_bytes(int K) { return (size_t)(K / 32) * (kXqWords * 4); }
inline int stream_n_stages(int K) {
  const size_t n = ((size_t)kMaxDynSmem - stream_xq_bytes(K)) / stream_stage_bytes(K);
  return (int)std::min<size_t>(n, kMaxStages);
}

inline StreamParams stream_params_from(const GemvParams& g, int* status) {
  const int rows = kGroupWarps / stream_parts_for(g.K) * stream_rpw_for(g.K);
  const bool sw = g.mode == GEMV_SWIGLU_F16;
  StreamParams p{};
  p.n_seg = g.n_seg;
  int tiles = 0;
  if (sw) {
    p.seg[0] = StreamSeg{g.seg[0].base, g.seg[0].n_rows, 0};
    p.seg[1] = StreamSeg{g.seg[1].base, g.seg[1].n_rows, 0};
    tiles = g.seg[0].n_rows / (rows / 2);
  } else {
    for (int s = 0; s < g.n_seg; ++s) {
      p.seg[s] = StreamSeg{g.seg[s].base, g.seg[s].n_rows, tiles};
      tiles += g.seg[s].n_rows / rows;
    }
  }
  p.n_tiles = tiles;
  p.K = g.K;
  p.mode = g.mode;
  p.n_stages = stream_n_stages(g.K);
  p.x16 = g.x;
  p.norm_in16 = g.norm_x16;
  p.norm_in32 = g.norm_x32;
  p.gain = g.norm_gain;
  p.eps = g.norm_eps;
  p.h_out = g.norm_out;
  p.y32 = g.y32;
  p.y16 = g.y16;
  p.res32 = g.res32;
  p.res16 = g.res16;
  p.status = status;
  p.wait_limit = 0;
  p.withhold_tile = -1;
  return p;
}

}  // namespace

}  // namespace ats
