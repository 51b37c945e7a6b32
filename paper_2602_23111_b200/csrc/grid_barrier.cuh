// A barrier over all CTAs of a cooperative launch (every CTA resident), with a bounded wait.
// The CTAs count arrivals in a global word that is zeroed before the launch and never reset
// inside it: barrier number b (1, 2, ...) is complete when the count reaches b * gridDim.x.
// A CTA that has polled `poll_limit` times without seeing that raises `abort`, which releases
// every other waiter too; the caller then leaves its kernel through the normal exit.  Nothing
// asynchronous is in flight while a CTA waits here, so giving up is clean.
#pragma once
#include <cuda_runtime.h>

namespace prac {

struct GridBarrierState {
  unsigned arrivals;   // arrivals so far
  int abort;           // a wait gave up
};

constexpr unsigned GRID_BARRIER_POLLS = 1u << 22;   // default poll limit (seconds of polling)

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Returns false when this or another CTA gave up.  All threads of the CTA must call it.
__device__ __forceinline__ bool grid_barrier(GridBarrierState* gb, unsigned target, unsigned poll_limit) {
  __shared__ int ok_sh;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(&gb->arrivals, 1u);
    int ok = 1;
    unsigned polls = 0;
    while (ld_acquire_u32(&gb->arrivals) < target) {
      if (++polls >= poll_limit) { atomicExch(&gb->abort, 1); ok = 0; break; }
      if ((polls & 63u) == 0u && *reinterpret_cast<volatile int*>(&gb->abort)) { ok = 0; break; }
    }
    if (ok && *reinterpret_cast<volatile int*>(&gb->abort)) ok = 0;
    __threadfence();
    ok_sh = ok;
  }
  __syncthreads();
  return ok_sh != 0;
}

}  // namespace prac
