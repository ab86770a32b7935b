// Bounded waits on mbarrier phases, shared by the GEMM kernels and by the wait-limit self-test.
#pragma once

#include "ptx.cuh"

namespace qb {

constexpr long long kWaitLimitCycles = 4000000000ll;  // default bound of a wait: about 2 s at 2 GHz

// Bounded wait on an mbarrier phase.  Returns false if the wait expired (more than `limit` SM cycles) or
// another role raised the abort flag.  The bound is counted in SM clock cycles (clock64 is a cheap
// register read; the global nanosecond timer costs about a microsecond per read and would dominate short
// waits).
// kSleep: the waiter is not on the critical path (it runs several stages ahead) and must not compete
// for issue slots with the MMA issuer that shares its scheduler: it uses the form of try_wait that
// takes a suspend-time hint.  A warp that polls in a tight loop is always "ready", and a handful of
// them starve the one thread that feeds the tensor cores.
template <bool kSleep>
__device__ __forceinline__ bool wait_barrier_t(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               long long limit = kWaitLimitCycles) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t spin = 1;; ++spin) {
    if (kSleep) {
      // suspended by the hardware until the phase completes or about a microsecond has passed: no issue
      // slots are spent while waiting and the wake-up does not wait for a sleep interval to end
      if (ptx::mbar_try_wait_suspend(bar, parity, 1000u)) return true;
    } else {
      if (ptx::mbar_try_wait(bar, parity)) return true;
    }
    if ((spin & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
}
__device__ __forceinline__ bool wait_barrier(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             long long limit = kWaitLimitCycles) {
  return wait_barrier_t<false>(bar, parity, abort_flag, limit);
}
__device__ __forceinline__ bool wait_barrier_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                     long long limit = kWaitLimitCycles) {
  return wait_barrier_t<true>(bar, parity, abort_flag, limit);
}

// Whole-warp wait: only lane 0 polls the barrier (hundreds of threads polling the same shared-memory
// word would flood the shared-memory pipeline that the stores and the other roles' waits also use);
// the outcome is broadcast, and the shuffle orders the other lanes' later accesses after the wait.
__device__ __forceinline__ bool wait_barrier_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  long long limit = kWaitLimitCycles) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = wait_barrier_relaxed(bar, parity, abort_flag, limit) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

}  // namespace qb
