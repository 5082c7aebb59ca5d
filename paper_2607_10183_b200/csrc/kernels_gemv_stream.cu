// Stand-alone launches of the streaming decode GEMV (sm_100a): the dense single-token GEMV and its grouped-expert form.
// The device code of a phase (producer, consumers, arithmetic) is in gemv_stream_body.cuh.
#include "gemv_stream_body.cuh"

namespace ats {

namespace {

// One CTA: ring set-up, then the producer warp and the consumer warps go their ways.  dep_resolved: the caller has already
// waited for the preceding kernel (its weight addresses come from that kernel's output).
// SHORT: the wide-tile geometry of short rows (K <= 1024; one k-part): four rows per warp, one block per lane, four
// producer warps.
template <int PARTS, bool SW, bool MX, bool SHORT>
__device__ __forceinline__ void gemv_stream_body(const StreamParams& p, const int bx, const int gx, const bool dep_resolved) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ StreamShared sh;
  constexpr int RPW = SHORT ? kRPWShort : kRPW, J = SHORT ? kJShort : kJ, PW = SHORT ? kProducerWarpsShort : kProducerWarps;
  constexpr int ROWS = kGroupWarps / PARTS * RPW;
  const int stage_bytes = ROWS * (p.K / 2 + p.K / 16);
  stream_init(sh, p.n_stages);
  if ((threadIdx.x >> 5) >= kConsumerWarps) {
    // weights do not depend on the preceding kernel, so their copies start before the grid dependency is resolved
    if ((threadIdx.x & 31) == 0)
      stream_produce<PARTS, SW, RPW, PW>(p, bx, gx, (int)(threadIdx.x >> 5) - kConsumerWarps, sh, smem, l2_evict_first_policy());
    return;
  }
  stream_consume<PARTS, SW, MX, RPW, J>(p, bx, gx, sh, smem, reinterpret_cast<uint32_t*>(smem + (size_t)p.n_stages * stage_bytes), dep_resolved);
}

template <int PARTS, bool SW, bool MX, bool SHORT = false>
__global__ void __launch_bounds__(SHORT ? kThreadsShort : kThreads, 1) gemv_stream_kernel(const StreamParams p) {
  gemv_stream_body<PARTS, SW, MX, SHORT>(p, (int)blockIdx.x, (int)gridDim.x, false);
}

// Grouped-expert variant: blockIdx.y selects the job (a (token, slot) pair), whose expert slices, activation row and
// output row come from the expert ids on the device (all experts resident and contiguous) or from a job table passed
// by value (resident and streamed experts mixed); the gridDim.x CTAs of a job then run the same body.
struct MoeSel {
  const uint8_t* base0;
  const uint8_t* base1;
  unsigned long long stride;
  const int32_t* ids;  // null: use the job table
  const uint8_t* const* tab0;  // with ids: per-expert slice addresses (device memory or mapped pinned host memory)
  const uint8_t* const* tab1;
  int x_div;
  int ldx, ldy;
  int n_experts;
};
template <int PARTS, bool SW, bool MX, bool SHORT = false>
__global__ void __launch_bounds__(SHORT ? kThreadsShort : kThreads, 1) gemv_stream_moe_kernel(const StreamParams p0, const MoeSel m, const MoeJobs jobs) {
  StreamParams p = p0;
  const int job = blockIdx.y;
  int xrow, orow;
  if (m.ids) {
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the ids come from the router kernel (every thread waits: the consumers skip their own wait)
    size_t e = (size_t)(unsigned)m.ids[job];
    if (e >= (size_t)m.n_experts) {  // an id that names no expert: expert 0 stands in and the status word says so
      if (threadIdx.x == 0 && blockIdx.x == 0) raise_status(p0.status, 7);
      e = 0;
    }
    p.seg[0].base = m.tab0 ? m.tab0[e] : m.base0 + e * m.stride;
    if (SW) p.seg[1].base = m.tab1 ? m.tab1[e] : m.base1 + e * m.stride;
    xrow = job / m.x_div;
    orow = job;
  } else {
    p.seg[0].base = jobs.w0[job];
    if (SW) p.seg[1].base = jobs.w1[job];
    xrow = jobs.xrow[job];
    orow = jobs.orow[job];
  }
  p.x16 = p0.x16 + (size_t)xrow * m.ldx;
  if (p0.y32) p.y32 = p0.y32 + (size_t)orow * m.ldy;
  if (p0.y16) p.y16 = p0.y16 + (size_t)orow * m.ldy;
  gemv_stream_body<PARTS, SW, MX, SHORT>(p, (int)blockIdx.x, (int)gridDim.x, m.ids != nullptr);
}

int parts_for(int K) { return stream_parts_for(K); }

// The kernels take nearly all of an SM's shared memory for the ring.
cudaError_t set_stream_kernel_attributes(const void* kern) {
  return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
}

}  // namespace

bool gemv_stream_eligible(const GemvParams& p) { return !p.w16 && stream_shape_ok(p); }  // the two 4-bit formats

cudaError_t launch_gemv_stream(const GemvParams& g, int* status, int sm_count, cudaStream_t st, uint64_t* n_launch) {
  const int parts = parts_for(g.K);
  const bool sw = g.mode == GEMV_SWIGLU_F16;
  StreamParams p = stream_params_from(g, status);
  p.wait_limit = g.dbg_wait_limit;
  p.withhold_tile = g.dbg_withhold_tile_plus1 - 1;
  const int tiles = p.n_tiles;
  const size_t stage_bytes = stream_stage_bytes(g.K);
  const size_t smem = p.n_stages * stage_bytes + stream_xq_bytes(g.K);
  const int grid = std::max(1, std::min(tiles, sm_count));
  void (*kern)(const StreamParams) = nullptr;
  const bool shrt = stream_short(g.K);
  const int producers = stream_producers_for(g.K);
  if (shrt) {
    if (g.mx) kern = sw ? gemv_stream_kernel<1, true, true, true> : gemv_stream_kernel<1, false, true, true>;
    else kern = sw ? gemv_stream_kernel<1, true, false, true> : gemv_stream_kernel<1, false, false, true>;
  } else if (g.mx) {
    switch (parts) {
      case 1: kern = sw ? gemv_stream_kernel<1, true, true> : gemv_stream_kernel<1, false, true>; break;
      case 2: kern = sw ? gemv_stream_kernel<2, true, true> : gemv_stream_kernel<2, false, true>; break;
      case 4: kern = sw ? gemv_stream_kernel<4, true, true> : gemv_stream_kernel<4, false, true>; break;
      default: kern = sw ? gemv_stream_kernel<8, true, true> : gemv_stream_kernel<8, false, true>; break;
    }
  } else {
    switch (parts) {
      case 1: kern = sw ? gemv_stream_kernel<1, true, false> : gemv_stream_kernel<1, false, false>; break;
      case 2: kern = sw ? gemv_stream_kernel<2, true, false> : gemv_stream_kernel<2, false, false>; break;
      case 4: kern = sw ? gemv_stream_kernel<4, true, false> : gemv_stream_kernel<4, false, false>; break;
      default: kern = sw ? gemv_stream_kernel<8, true, false> : gemv_stream_kernel<8, false, false>; break;
    }
  }
  static uint64_t attr_done[20] = {};
  const int ki = ((shrt ? 4 : parts == 1 ? 0 : parts == 2 ? 1 : parts == 4 ? 2 : 3) * 2 + (sw ? 1 : 0)) * 2 + (g.mx ? 1 : 0);
  if (first_use_on_device(&attr_done[ki])) {
    cudaError_t e = set_stream_kernel_attributes(reinterpret_cast<const void*>(kern));
    if (e != cudaSuccess) return e;
  }
  if (smem > kMaxDynSmem || p.n_stages < producers) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(shrt ? kThreadsShort : kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = g.pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++*n_launch;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

bool moe_gemv_stream_eligible(const MoeGemvParams& p) {
  if (p.K % 256 != 0 || p.K > 16384) return false;
  const int rows = kGroupWarps / parts_for(p.K) * stream_rpw_for(p.K);
  if (p.mode == GEMV_SWIGLU_F16) return p.n_rows % (rows / 2) == 0;
  return (p.mode == GEMV_OUT_F32 || p.mode == GEMV_OUT_F16) && p.n_rows % rows == 0;
}

cudaError_t launch_moe_gemv_stream(const MoeGemvParams& g, const MoeJobs* jobs, int* status, int sm_count, int pdl, cudaStream_t st,
                                   uint64_t* n_launch) {
  const int parts = parts_for(g.K);
  const int rows = kGroupWarps / parts * stream_rpw_for(g.K);
  const bool sw = g.mode == GEMV_SWIGLU_F16;
  const bool shrt = stream_short(g.K);
  const int n_jobs = jobs ? jobs->n : g.P;
  if (n_jobs <= 0) return cudaSuccess;
  StreamParams p{};
  p.n_seg = sw ? 2 : 1;
  p.seg[0] = StreamSeg{nullptr, g.n_rows, 0};
  p.seg[1] = StreamSeg{nullptr, g.n_rows, 0};
  p.n_tiles = sw ? g.n_rows / (rows / 2) : g.n_rows / rows;
  p.K = g.K;
  p.mode = g.mode;
  p.n_stages = stream_n_stages(g.K);
  p.x16 = g.x;
  p.y32 = g.y32;
  p.y16 = g.y16;
  p.status = status;
  p.withhold_tile = -1;
  MoeSel m{};
  m.base0 = g.base0;
  m.base1 = g.base1;
  m.stride = g.stride;
  m.ids = jobs ? nullptr : g.ids;
  m.tab0 = g.tab0;
  m.tab1 = g.tab1;
  m.x_div = g.x_div;
  m.ldx = g.ldx;
  m.ldy = g.ldy;
  m.n_experts = g.n_experts;
  MoeJobs none;
  none.n = 0;
  const size_t smem = p.n_stages * stream_stage_bytes(g.K) + stream_xq_bytes(g.K);
  if (smem > kMaxDynSmem || p.n_stages < stream_producers_for(g.K)) return cudaErrorInvalidValue;
  const int per_job = std::max(1, std::min(p.n_tiles, sm_count / n_jobs));  // one wave: a CTA fills its SM
  void (*kern)(const StreamParams, const MoeSel, const MoeJobs) = nullptr;
  if (shrt) {
    if (g.mx) kern = sw ? gemv_stream_moe_kernel<1, true, true, true> : gemv_stream_moe_kernel<1, false, true, true>;
    else kern = sw ? gemv_stream_moe_kernel<1, true, false, true> : gemv_stream_moe_kernel<1, false, false, true>;
  } else if (g.mx) {
    switch (parts) {
      case 1: kern = sw ? gemv_stream_moe_kernel<1, true, true> : gemv_stream_moe_kernel<1, false, true>; break;
      case 2: kern = sw ? gemv_stream_moe_kernel<2, true, true> : gemv_stream_moe_kernel<2, false, true>; break;
      case 4: kern = sw ? gemv_stream_moe_kernel<4, true, true> : gemv_stream_moe_kernel<4, false, true>; break;
      default: kern = sw ? gemv_stream_moe_kernel<8, true, true> : gemv_stream_moe_kernel<8, false, true>; break;
    }
  } else {
    switch (parts) {
      case 1: kern = sw ? gemv_stream_moe_kernel<1, true, false> : gemv_stream_moe_kernel<1, false, false>; break;
      case 2: kern = sw ? gemv_stream_moe_kernel<2, true, false> : gemv_stream_moe_kernel<2, false, false>; break;
      case 4: kern = sw ? gemv_stream_moe_kernel<4, true, false> : gemv_stream_moe_kernel<4, false, false>; break;
      default: kern = sw ? gemv_stream_moe_kernel<8, true, false> : gemv_stream_moe_kernel<8, false, false>; break;
    }
  }
  static uint64_t attr_done[20] = {};
  const int ki = ((shrt ? 4 : parts == 1 ? 0 : parts == 2 ? 1 : parts == 4 ? 2 : 3) * 2 + (sw ? 1 : 0)) * 2 + (g.mx ? 1 : 0);
  if (first_use_on_device(&attr_done[ki])) {
    cudaError_t e = set_stream_kernel_attributes(reinterpret_cast<const void*>(kern));
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(per_job, n_jobs);
  cfg.blockDim = dim3(shrt ? kThreadsShort : kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++*n_launch;
  return cudaLaunchKernelEx(&cfg, kern, p, m, jobs ? *jobs : none);
}

// ------------------------------------------------------------------------------------------ read-only HBM probe
// What this GPU delivers to a kernel that only reads, with the access pattern of the streaming GEMV (bulk-async copies of
// 16 KB into shared memory, four issuing warps per SM, nothing done with the data): the third denominator next to the
// nominal figure and the measured copy bandwidth (a copy also writes, and reaches less).
namespace {
constexpr int kProbeWarps = 4, kProbeDepth = 2, kProbeChunk = 16 * 1024;
__global__ void __launch_bounds__(kProbeWarps * 32) hbm_read_probe_kernel(const uint8_t* __restrict__ src, unsigned long long n_chunks,
                                                                          int* status) {
  extern __shared__ __align__(128) uint8_t probe_s[];
  __shared__ uint64_t bar[kProbeWarps * kProbeDepth];
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) != 0) return;
  uint64_t* mybar = bar + warp * kProbeDepth;
  uint8_t* mysm = probe_s + (size_t)warp * kProbeDepth * kProbeChunk;
  for (int s = 0; s < kProbeDepth; ++s) mbar_init(&mybar[s], 1);
  mbar_fence_init();
  const unsigned long long issuers = (unsigned long long)gridDim.x * kProbeWarps;
  const unsigned long long first = (unsigned long long)blockIdx.x * kProbeWarps + warp;
  const long long per = (long long)((n_chunks + issuers - 1) / issuers);
  const uint64_t pol = l2_evict_first_policy();
  for (long long it = 0; it < per + kProbeDepth; ++it) {
    const int s = (int)(it % kProbeDepth);
    if (it >= kProbeDepth && !mbar_wait(&mybar[s], (uint32_t)(((it / kProbeDepth) - 1) & 1))) {
      raise_status(status, 8);
      return;
    }
    if (it < per) {
      const unsigned long long chunk = first + (unsigned long long)it * issuers;
      if (chunk < n_chunks) {
        mbar_expect_tx(&mybar[s], kProbeChunk);
        bulk_g2s(mysm + (size_t)s * kProbeChunk, src + chunk * kProbeChunk, kProbeChunk, &mybar[s], pol);
      } else {
        mbar_arrive(&mybar[s]);
      }
    }
  }
}
}  // namespace

cudaError_t launch_hbm_read_probe(const uint8_t* src, uint64_t bytes, int* status, int sm_count, cudaStream_t st) {
  const size_t smem = (size_t)kProbeWarps * kProbeDepth * kProbeChunk;
  static uint64_t attr_done = 0;
  if (first_use_on_device(&attr_done)) {
    cudaError_t e = cudaFuncSetAttribute(hbm_read_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  hbm_read_probe_kernel<<<sm_count, kProbeWarps * 32, smem, st>>>(src, bytes / kProbeChunk, status);
  return cudaGetLastError();
}

}  // namespace ats

#ifdef ATS_TRACE
// Development builds only: read and clear the timeline probe (see gemv_stream_body.cuh).
extern "C" int ats_trace_read(void* out_host, int cap_records) {
  unsigned int n = 0;
  if (cudaMemcpyFromSymbol(&n, ats::g_trace_n, sizeof n) != cudaSuccess) return -1;
  if (n > (unsigned)ats::kTraceCap) n = ats::kTraceCap;
  if ((int)n > cap_records) n = cap_records;
  if (n && cudaMemcpyFromSymbol(out_host, ats::g_trace, (size_t)n * sizeof(ats::TraceRec)) != cudaSuccess) return -1;
  unsigned int zero = 0;
  cudaMemcpyToSymbol(ats::g_trace_n, &zero, sizeof zero);
  return (int)n;
}
#endif
