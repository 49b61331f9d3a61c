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

// The production wait run out: warp 0 gives up after `short_limit` polls, warp 1 waits with the
// production limit and has to be stopped by the abort flag warp 0 sets.
__global__ void wait_abort_kernel(int *status, long long *report, unsigned short_limit) {
  __shared__ uint64_t bars[2];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    const long long t0 = clock64();
    const bool done = mbar_wait(&bars[warp], 0, &abort_flag, status, warp == 0 ? short_limit : WAIT_LIMIT);
    const long long t1 = clock64();
    report[2 + warp] = t1 - t0;
    if (warp == 1) report[1] = done ? 0 : 1;
  }
}

}  // namespace

extern "C" int locret_selftest_wait_abort(void *stream, int64_t *report) {
  if (!report) return LOCRET_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  int *d_status = nullptr;
  long long *d_rep = nullptr;
  if (cudaMalloc(&d_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_ALLOC; }
  if (cudaMalloc(&d_rep, 4 * sizeof(long long)) != cudaSuccess) { cudaGetLastError(); cudaFree(d_status); return LOCRET_ERR_ALLOC; }
  int host_status = 0;
  long long host_rep[4] = {0, 0, 0, 0};
  cudaError_t e = cudaMemsetAsync(d_status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaMemsetAsync(d_rep, 0, 4 * sizeof(long long), st);
  if (e == cudaSuccess) {
    wait_abort_kernel<<<1, 64, 0, st>>>(d_status, d_rep, 1u << 12);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(&host_status, d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(host_rep, d_rep, sizeof(host_rep), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d_status);
  cudaFree(d_rep);
  if (e != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; }
  report[0] = host_status;
  for (int i = 1; i < 4; i++) report[i] = host_rep[i];
  return LOCRET_OK;
}

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
