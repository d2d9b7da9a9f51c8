// Self-test of the bounded-wait scheme every tensor-core kernel relies on: a kernel whose
// only job is to let one bounded mbarrier wait run out, so that the path "wait gives up ->
// abort word -> global error word -> mtla_check" can be exercised without disturbing the GPU.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mtla {

// One CTA of 64 threads.  Thread 0 initialises an mbarrier that expects one arrival which
// never comes; every thread then waits on it with the same bounded wait the product kernels
// use, with `budget_ns` in place of their two-second budget.  All threads return false from the
// wait (the first to time out raises the CTA's abort word, the others see it), nothing traps,
// and the kernel exits normally with `code` in the error word.
__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(int* error_word, int code,
                                                                    unsigned long long budget_ns,
                                                                    int* gave_up) {
  __shared__ unsigned long long bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_word = 0;
    ptx::mbar_fence_init();
  }
  __syncthreads();
  const bool ok = ptx::mbar_wait_for(ptx::smem_u32(&bar), 0, &abort_word, error_word, code, budget_ns);
  if (!ok) atomicAdd(gave_up, 1);
}

}  // namespace mtla
