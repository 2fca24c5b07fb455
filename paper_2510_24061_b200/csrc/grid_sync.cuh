// A grid-wide barrier for kernels whose CTAs are all resident (cooperative launches): two counters in device memory
// that start at zero and are put back to zero by the last CTA to leave, so that the same words serve the next launch.
// Every CTA must arrive AND depart exactly once, whatever happened to it; the wait is bounded by wall time and a wait
// that runs out is reported through the status word.
#pragma once

#include <cstdint>

#include "ptx.cuh"

namespace falqon {

struct GridSync {
  unsigned int arrive;
  unsigned int depart;
};

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// One thread of the CTA, after the CTA's earlier global writes were made visible to it (a CTA-wide barrier): publishes
// them, arrives and waits for the whole grid.  failed: this CTA has already given up (it arrives and does not wait).
// Returns whether the whole grid arrived in time.
__device__ __forceinline__ bool grid_arrive_and_wait(GridSync* sync, int* status, bool failed) {
  bool ok = !failed;
  if (!ok) atomicExch(status, kStatusTimeout);
  __threadfence();
  atomicAdd(&sync->arrive, 1u);
  if (ok && ld_acquire_gpu(&sync->arrive) < gridDim.x) {
    const uint64_t t0 = global_timer_ns();
    for (;;) {
      if (ld_acquire_gpu(&sync->arrive) >= gridDim.x) break;
      __nanosleep(40);
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        ok = false;
        atomicExch(status, kStatusTimeout);
        break;
      }
    }
  }
  return ok;
}

// One thread of the CTA, as the CTA's last action.
__device__ __forceinline__ void grid_depart(GridSync* sync) {
  const unsigned int prev = atomicAdd(&sync->depart, 1u);
  if (prev == gridDim.x - 1) {
    sync->arrive = 0u;
    sync->depart = 0u;
    __threadfence();
  }
}

}  // namespace falqon
