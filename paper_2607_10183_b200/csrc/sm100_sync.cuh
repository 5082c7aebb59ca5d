// Shared-memory barrier (mbarrier) and address helpers used by every kernel of the library that moves data with
// asynchronous copies (sm_100a).  All waits are bounded: a wait that runs out returns false and the caller raises the
// context's status word, releases what it holds and returns, so that a lost completion never hangs the device.
#pragma once
#include <stdint.h>

namespace ats {
namespace {

// Default limit of a bounded wait in SM clock cycles: about a second at 2 GHz.
constexpr long long kWaitLimitCycles = 2000000000ll;

// Raise the context's status word (any non-zero code: a bounded wait ran out, an id was out of range).  The word may live
// in pinned host memory that the device addresses directly, where atomics are not available on every system: a plain
// store made visible system-wide is enough, since every writer stores a non-zero value and any of them may win.
__device__ __forceinline__ void raise_status(int* status, int code) {
  if (!status) return;
  *reinterpret_cast<volatile int*>(status) = code;
  __threadfence_system();
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
// Makes the initialised barriers visible to the asynchronous proxy (and to the other CTAs of a cluster).
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Non-blocking poll of a phase parity.
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Poll that may suspend the thread for a hardware-chosen time (waking up afterwards can cost on the order of a
// microsecond: use it where the wait is long anyway, test_wait where a pipeline step is short).
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded spin on test_wait.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, long long limit = kWaitLimitCycles) {
  if (mbar_test_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_test_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}
// Bounded wait on try_wait (the thread may be suspended between polls).
__device__ __forceinline__ bool mbar_wait_suspending(uint64_t* bar, uint32_t parity, long long limit = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > limit) return false;
  }
}

}  // namespace
}  // namespace ats
