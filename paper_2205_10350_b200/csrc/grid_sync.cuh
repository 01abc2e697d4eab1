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

__device__ __forceinline__ unsigned int load_relaxed(const unsigned int* ctr) {
  unsigned int v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
  return v;
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

// Spins until *ctr >= target (wrap-safe comparison) or budget_ns have passed.  One thread per CTA calls this.
// Every poll is an acquire load: measured on a B200 over one CTA per SM, 1.26 us per barrier against 1.42 us for
// relaxed polls followed by one acquire fence (the fence alone costs about half a microsecond).
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
// The variant with relaxed polls and one fence (kept for the timing probe).
__device__ __forceinline__ bool wait_reached_relaxed_polls(const unsigned int* ctr, unsigned int target, unsigned long long budget_ns) {
  bool ok = false;
  for (int i = 0; i < 32 && !ok; ++i) ok = (int)(load_relaxed(ctr) - target) >= 0;
  if (!ok) {
    const unsigned long long t0 = now_ns();
    while (!ok) {
      for (int i = 0; i < 32 && !ok; ++i) ok = (int)(load_relaxed(ctr) - target) >= 0;
      if (!ok && now_ns() - t0 > budget_ns) return false;
    }
  }
  fence_acq_rel_gpu();
  return true;
}

// Full barrier of all CTAs of the grid; call from every thread.  Returns false in every thread of a CTA whose wait
// ran out.  `generation` counts this CTA's barriers (starts at 0, incremented here).
__device__ __forceinline__ bool grid_barrier(unsigned int* ctr, unsigned int& generation, unsigned int n_ctas,
                                             unsigned long long budget_ns, int* shared_flag, bool relaxed_polls = false) {
  __syncthreads();
  generation += 1;
  if (threadIdx.x == 0) {
    arrive_release(ctr, 1u);
    *shared_flag = (relaxed_polls ? wait_reached_relaxed_polls(ctr, generation * n_ctas, budget_ns)
                                  : wait_reached(ctr, generation * n_ctas, budget_ns)) ? 1 : 0;
  }
  __syncthreads();
  return *shared_flag != 0;
}

}  // namespace gs
}  // namespace ad
