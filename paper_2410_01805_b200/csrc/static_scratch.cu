// Retaining-head scores for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc on the path where they need scores: code
// running inside a memory pool that owns every byte of the device, a serving loop whose
// allocator is locked while a request is in flight, or a plug-in that is only handed
// buffers.  locret_rh_scores_static runs the same two kernels as the layer's step (c) but keeps
// the per-tile partial sums in a fixed array that is part of the library image, so the call
// needs nothing beyond the caller's own input and output buffers.
#include "../../include/locret.h"
#include "common.cuh"

using namespace locret;

namespace {

// Scratch for the partial scores [N-tiles of the GEMM (at most ceil(d_R / 64))][n_tok][h_kv] (fp32).  It lives in every
// GPU context that loads the library until the process exits.
static __device__ __align__(256) float g_static_partial[LOCRET_STATIC_SCRATCH_FLOATS];

float *g_partial_ptr[MAX_DEVICES] = {nullptr};

// In host code `g_static_partial` is only a stand-in for the symbol, never a device address:
// the address a kernel may use has to be asked for, once per device, with that device current.
int static_partial_for_current_device(float **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    cudaGetLastError();
    return LOCRET_ERR_CUDA;
  }
  if (!g_partial_ptr[dev]) {
    float *p = nullptr;
    if (cudaGetSymbolAddress((void **)&p, g_static_partial) != cudaSuccess || !p) {
      cudaGetLastError();
      return LOCRET_ERR_CUDA;
    }
    g_partial_ptr[dev] = p;
  }
  *out = g_partial_ptr[dev];
  return LOCRET_OK;
}

}  // namespace

extern "C" int locret_rh_scores_static(const void *z, int32_t n_tok, int32_t d_in, const void *w1_t,
                                       int32_t d_retain, const float *w2, int32_t n_kv_heads,
                                       int32_t act, float *scores, int32_t *status, void *stream) {
  if (!z || !w1_t || !w2 || !scores) return LOCRET_ERR_INVALID;
  if (n_tok < 1 || d_in < 64 || d_in % 64 != 0 || d_retain < 32 || d_retain % 32 != 0)
    return LOCRET_ERR_INVALID;
  if (n_kv_heads < 1 || n_kv_heads > 32 || act < 0 || act > 2) return LOCRET_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(z) & 15u) || (reinterpret_cast<uintptr_t>(w1_t) & 15u))
    return LOCRET_ERR_INVALID;
  const long long need = (long long)rh_tc_num_tiles(d_retain) * n_tok * n_kv_heads;
  if (need > (long long)LOCRET_STATIC_SCRATCH_FLOATS) return LOCRET_ERR_CAPACITY;
  if (!gemm_tc_supported(n_tok, d_retain, d_in, d_in, d_in)) return LOCRET_ERR_INVALID;

  float *partial = nullptr;
  int rc = static_partial_for_current_device(&partial);
  if (rc != LOCRET_OK) return rc;

  cudaStream_t st = (cudaStream_t)stream;
  int n_tiles = 0;
  // Every partial this call reads is written by this call first, so nothing has to be cleared.
  if (launch_rh_gemm_tc((const bf16 *)z, d_in, (const bf16 *)w1_t, w2, partial, n_tok, d_retain, d_in,
                        n_kv_heads, act, &n_tiles, status, st) != cudaSuccess) {
    cudaGetLastError();
    return LOCRET_ERR_CUDA;
  }
  if (launch_rh_reduce(partial, n_tiles, n_tok, n_kv_heads, scores, n_tok, 0, st) != cudaSuccess) {
    cudaGetLastError();
    return LOCRET_ERR_CUDA;
  }
  return LOCRET_OK;
}
