// Diagnostic entry point for the bounded device-side waits: every mbarrier wait in the tcgen05
// kernels gives up after a fixed number of polls, records LOCRET_ERR_DEVICE_TIMEOUT in a status
// word and lets the kernel run to its end.  The self-test makes one such wait run out on purpose
// (a barrier that nothing ever arrives at, with a short limit) so that the status path can be
// checked without faulting, trapping or hanging the GPU.
#include "../../include/locret.h"
#include "tc_common.cuh"

using namespace locret;
using namespace locret::tc;

namespace {

__global__ void wait_timeout_kernel(int *status, unsigned limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    bool done = false;
    for (unsigned i = 0; i < limit && !done; i++) done = mbar_try_wait(&bar, 0);
    if (!done) atomicExch(status, ERR_TIMEOUT);  // the same record the production waits leave
  }
}

}  // namespace

extern "C" int locret_selftest_wait_timeout(void *stream) {
  cudaStream_t st = (cudaStream_t)stream;
  int *d = nullptr;
  if (cudaMalloc(&d, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_ALLOC; }
  int host = 0;
  cudaError_t e = cudaMemsetAsync(d, 0, sizeof(int), st);
  if (e == cudaSuccess) {
    wait_timeout_kernel<<<1, 32, 0, st>>>(d, 1u << 12);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&host, d, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d);
  if (e != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; }
  return host;
}
