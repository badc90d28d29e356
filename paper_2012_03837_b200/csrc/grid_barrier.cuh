// Grid-wide barrier for kernels started with a cooperative launch (all blocks co-resident), with a bounded wait.
// counter[0] counts arrivals, counter[1] the blocks that have left the kernel; both are zero between launches:
// the last block to leave puts them back.  Barrier number i (i = 1, 2, ...) of a launch waits for
// i * gridDim.x arrivals.
#pragma once
#include "lp_kernels.h"

namespace lp {

constexpr long long GRID_BARRIER_LIMIT_NS = 2000000000ll;

__device__ __forceinline__ long long gb_now_ns() {
  long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Every thread of every block calls it.  Returns false if the wait was given up (about two seconds, or another
// block has already given up): ST_TIMEOUT is raised in *status and the caller leaves its kernel through
// grid_barrier_leave.
__device__ __forceinline__ bool grid_barrier(unsigned long long* counter, unsigned long long target, int* status) {
  __shared__ int ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(counter, 1ull);
    const long long t0 = gb_now_ns();
    int good = 1;
    while (*(volatile unsigned long long*)counter < target) {
      if ((*(volatile int*)status & ST_TIMEOUT) || gb_now_ns() - t0 > GRID_BARRIER_LIMIT_NS) {
        atomicOr(status, ST_TIMEOUT);
        good = 0;
        break;
      }
    }
    __threadfence();
    ok = good;
  }
  __syncthreads();
  return ok != 0;
}

// The last statement of the kernel, reached by every block on every path.
__device__ __forceinline__ void grid_barrier_leave(unsigned long long* counter) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(counter + 1, 1ull) == (unsigned long long)gridDim.x - 1) {
      counter[0] = 0ull;
      counter[1] = 0ull;
      __threadfence();
    }
  }
}

}  // namespace lp
