// Diagnostic: makes a bounded device-side wait run out on purpose, so that the path every kernel of the
// library uses to report a stuck wait (status word, detail words, normal return) can be tested without
// anything being stuck.  One CTA, one mbarrier that nobody ever arrives on; no copy or MMA is in flight.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace sparsp {

constexpr int kSelftestWhere = 99;  // the `where` code this kernel reports

__global__ void __launch_bounds__(32) wait_timeout_kernel(int32_t* __restrict__ status, long long limit_cycles,
                                                          int32_t* __restrict__ waited_cycles) {
  __shared__ uint64_t bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    ptx::mbar_init_fence();
    s_abort = 0;
  }
  __syncwarp();
  const long long t0 = clock64();
  // phase 0 of a freshly initialised barrier never completes without an arrival: the wait runs out
  if (threadIdx.x == 0) ptx::mbar_wait_bounded(&bar, 0, &s_abort, status, kSelftestWhere, limit_cycles);
  __syncwarp();
  // every later wait of the CTA falls through at once (the abort flag is up)
  ptx::mbar_wait_bounded(&bar, 0, &s_abort, status, kSelftestWhere + 1, limit_cycles);
  if (threadIdx.x == 0 && waited_cycles) *waited_cycles = (int32_t)min(clock64() - t0, (long long)0x7fffffff);
}

int launch_wait_timeout(char* ws, const WsLayout& L, long long limit_cycles, cudaStream_t st) {
  int32_t* status = (int32_t*)(ws + L.status);
  wait_timeout_kernel<<<1, 32, 0, st>>>(status, limit_cycles, status + 4);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

}  // namespace sparsp
