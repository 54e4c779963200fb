// Test-only kernel: a bounded mbarrier wait that nothing ever satisfies.
//
// The library's kernels wait on mbarriers with mbar_wait_bounded(); when a wait runs out they set the timeout bit of an
// error word and leave through their ordinary exit. This kernel takes exactly that path in isolation: it initialises
// an mbarrier that nobody arrives on, with no copy, no TMA and no tensor-core work in flight, waits with the short
// drain limit, records that the wait gave up and returns. It is built by the test that uses it and is not part of
// libadore.so.
#include <cuda_runtime.h>

#include "../../paper_2407_02328_b200/csrc/mbarrier.cuh"

using namespace adore;

__global__ void wait_that_runs_out_kernel(unsigned* err_word, unsigned* reached_end) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // phase 0 of `bar` never completes: no thread arrives, no transaction is pending
  const bool ok = mbar_wait_bounded(&bar, 0u, kDrainPolls);
  if (!ok && threadIdx.x == 0) set_error(err_word, ERRW_TIMEOUT);
  __syncthreads();
  if (threadIdx.x == 0) atomicAdd(reached_end, 1u);
}

// err_word, reached_end: device pointers to zero-initialised 32-bit words. Returns the CUDA error of the launch.
extern "C" int wait_probe_run(unsigned* err_word, unsigned* reached_end, int ctas, void* cuda_stream) {
  wait_that_runs_out_kernel<<<ctas, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(err_word, reached_end);
  return int(cudaGetLastError());
}

extern "C" unsigned wait_probe_timeout_bit() { return ERRW_TIMEOUT; }
