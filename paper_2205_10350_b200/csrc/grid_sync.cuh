// Grid-wide barrier for persistent kernels whose CTAs are all resident at once (one CTA per SM, launched
// cooperatively or with a grid no larger than what the device holds at a time).
//
// One monotonically increasing arrival counter in global memory: every CTA adds 1 per barrier, and barrier number
// g (1, 2, ...) is passed once the counter has reached g * gridDim.  The counter is never reset inside a launch, so
// there is no second phase word and no ABA problem; the host (or the kernel before) zeroes it between launches.
// Every wait is bounded by time: on expiry the caller latches AD_ERR_TIMEOUT and the kernel winds down.
#pragma once

#include "ad_common.cuh"

namespace ad {
namespace gs {

__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Adds v to *ctr with release semantics at GPU scope: everything this thread observed or wrote before (including,
// through the preceding CTA barrier, the other threads' writes) is visible to whoever acquires the new value.
__device__ __forceinline__ void arrive_release(unsigned int* ctr, unsigned int v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(ctr), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int load_acquire(const unsigned int* ctr) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
  return v;
}

// Spins until *ctr >= target (wrap-safe comparison) or budget_ns have passed.  One thread per CTA calls this.
__device__ __forceinline__ bool wait_reached(const unsigned int* ctr, unsigned int target, unsigned long long budget_ns) {
  for (int i = 0; i < 32; ++i)
    if ((int)(load_acquire(ctr) - target) >= 0) return true;
  const unsigned long long t0 = now_ns();
  for (;;) {
    for (int i = 0; i < 32; ++i)
      if ((int)(load_acquire(ctr) - target) >= 0) return true;
    if (now_ns() - t0 > budget_ns) return false;
  }
}

// Full barrier of all CTAs of the grid; call from every thread.  Returns false in every thread of a CTA whose wait
// ran out.  `generation` counts this CTA's barriers (starts at 0, incremented here).
__device__ __forceinline__ bool grid_barrier(unsigned int* ctr, unsigned int& generation, unsigned int n_ctas,
                                             unsigned long long budget_ns, int* shared_flag) {
  __syncthreads();
  generation += 1;
  if (threadIdx.x == 0) {
    arrive_release(ctr, 1u);
    *shared_flag = wait_reached(ctr, generation * n_ctas, budget_ns) ? 1 : 0;
  }
  __syncthreads();
  return *shared_flag != 0;
}

}  // namespace gs
}  // namespace ad
