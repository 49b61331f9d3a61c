// Kernels of the step when the KV heads (with their query groups) are divided over several GPUs.
// Heads attend and evict independently (Algorithm 1 runs per head); the retaining head reads every
// head's [Q, K, V] (Section 3.3), so each GPU forms the product of its own columns of z with its
// own rows of W1, the products are summed across the GPUs, and each GPU finishes with the
// activation and its own columns of W2.
#include "common.cuh"

namespace locret {

namespace {

// partial first product for shapes the tensor-core GEMM does not take (tiny test shapes)
__global__ void preact_naive_kernel(const bf16 *__restrict__ z, const bf16 *__restrict__ W1t,
                                    float *__restrict__ pre, int n_tok, int d_R, int d_in) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x, t = blockIdx.y;
  if (r >= d_R || t >= n_tok) return;
  float acc = 0.f;
  for (int k = 0; k < d_in; k++)
    acc = fmaf(__bfloat162float(z[(size_t)t * d_in + k]), __bfloat162float(W1t[(size_t)r * d_in + k]), acc);
  pre[(size_t)t * d_R + r] = acc;
}

// one warp per token: s[m][slot0 + t] = sum_r act(pre[t][r]) W2[r][m], h_kv <= 32
__global__ void rh_finish_kernel(const float *__restrict__ pre, const float *__restrict__ w2,
                                 float *__restrict__ s, int score_stride, int slot0, int n_tok, int d_R,
                                 int h_kv, int act) {
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= n_tok) return;
  float acc[32];
#pragma unroll
  for (int m = 0; m < 32; m++) acc[m] = 0.f;
  for (int r = lane; r < d_R; r += 32) {
    const float a = apply_act(pre[(size_t)t * d_R + r], act);
#pragma unroll
    for (int m = 0; m < 32; m++)
      if (m < h_kv) acc[m] = fmaf(a, w2[(size_t)r * h_kv + m], acc[m]);
  }
#pragma unroll
  for (int m = 0; m < 32; m++) {
    if (m < h_kv) {
      float v = acc[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) s[(size_t)m * score_stride + slot0 + t] = v;
    }
  }
}

__global__ void add_to_peers_kernel(const float *__restrict__ src, float *const *__restrict__ peers, int n_peers,
                                    size_t count) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float v = src[i];
  for (int p = 0; p < n_peers; p++)
    asm volatile("red.relaxed.sys.global.add.f32 [%0], %1;" ::"l"(peers[p] + i), "f"(v) : "memory");
}

}  // namespace

cudaError_t launch_add_to_peers(const float *src, float *const *peers, int n_peers, size_t count, cudaStream_t st) {
  add_to_peers_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(src, peers, n_peers, count);
  return cudaGetLastError();
}

cudaError_t launch_preact_naive(const bf16 *z, const bf16 *W1t, float *pre, int n_tok, int d_R, int d_in,
                                cudaStream_t st) {
  preact_naive_kernel<<<dim3((d_R + 127) / 128, n_tok), 128, 0, st>>>(z, W1t, pre, n_tok, d_R, d_in);
  return cudaGetLastError();
}

cudaError_t launch_rh_finish(const float *pre, const float *w2, float *s, int score_stride, int slot0,
                             int n_tok, int d_R, int h_kv, int act, cudaStream_t st) {
  if (h_kv > 32) return cudaErrorInvalidValue;
  rh_finish_kernel<<<(n_tok + 7) / 8, 256, 0, st>>>(pre, w2, s, score_stride, slot0, n_tok, d_R, h_kv, act);
  return cudaGetLastError();
}

}  // namespace locret
