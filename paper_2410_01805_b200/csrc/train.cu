// Training of the retaining head (Eq. 2, Eq. 3): loss and gradients of W1, W2 for one sequence,
// backbone frozen.  The two large contractions (z W1 and z^T dpre) run on the tcgen05 GEMM with
// fp32 results; the rest is element-wise work around the thin W2.
#include "../../include/locret.h"
#include "common.cuh"

using namespace locret;

namespace {

__device__ __forceinline__ float sigmoidf_(float x) { return 1.0f / (1.0f + __expf(-x)); }

// one warp per token: s[t][m] = sum_r silu(pre[t][r]) W2[r][m]
__global__ void rh_scores_f32_kernel(const float *__restrict__ pre, const float *__restrict__ w2,
                                     float *__restrict__ s, int n, int d_R, int h_kv) {
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= n) return;
  float acc[32];
#pragma unroll
  for (int m = 0; m < 32; m++) acc[m] = 0.f;
  for (int r = lane; r < d_R; r += 32) {
    const float p = pre[(size_t)t * d_R + r];
    const float a = p * sigmoidf_(p);
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
      if (lane == 0) s[(size_t)t * h_kv + m] = v;
    }
  }
}

// Eq. 3 per (token, head): Smooth-L1 (threshold 1) to the label plus alpha (s[t] - s[t+1])^2;
// ds = its derivative; the loss is summed with one atomic per block
__global__ void rh_loss_kernel(const float *__restrict__ s, const float *__restrict__ labels, float *__restrict__ ds,
                               float *__restrict__ loss, int n, int h_kv, float alpha) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  float l = 0.f;
  if (i < n * h_kv) {
    const int t = i / h_kv, m = i - t * h_kv;
    const float v = s[i], diff = v - labels[(size_t)m * n + t];
    const float ad = fabsf(diff);
    l = ad < 1.0f ? 0.5f * diff * diff : ad - 0.5f;
    float g = fminf(fmaxf(diff, -1.0f), 1.0f);
    if (t + 1 < n) {
      const float adj = v - s[i + h_kv];
      l = fmaf(alpha * adj, adj, l);
      g = fmaf(2.0f * alpha, adj, g);
    }
    if (t > 0) g -= 2.0f * alpha * (s[i - h_kv] - v);
    ds[i] = g;
  }
  __shared__ float red[32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = l;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (threadIdx.x == 0) atomicAdd(loss, v);
  }
}

// dW2[r][m] += sum over a slab of tokens of silu(pre[t][r]) ds[t][m]; thread = r
__global__ void rh_dw2_kernel(const float *__restrict__ pre, const float *__restrict__ ds, float *__restrict__ dw2,
                              int n, int d_R, int h_kv, int slab) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  const int t0 = blockIdx.y * slab, t1 = min(n, t0 + slab);
  if (r >= d_R) return;
  float acc[32];
#pragma unroll
  for (int m = 0; m < 32; m++) acc[m] = 0.f;
  for (int t = t0; t < t1; t++) {
    const float p = pre[(size_t)t * d_R + r];
    const float a = p * sigmoidf_(p);
#pragma unroll
    for (int m = 0; m < 32; m++)
      if (m < h_kv) acc[m] = fmaf(a, ds[(size_t)t * h_kv + m], acc[m]);
  }
#pragma unroll
  for (int m = 0; m < 32; m++)
    if (m < h_kv) atomicAdd(dw2 + (size_t)r * h_kv + m, acc[m]);
}

// dpreT[r][t] = bf16( (sum_m ds[t][m] W2[r][m]) * silu'(pre[t][r]) ), written transposed through a
// shared-memory tile so that the second contraction finds its K dimension (tokens) contiguous
__global__ void rh_dpre_t_kernel(const float *__restrict__ pre, const float *__restrict__ ds,
                                 const float *__restrict__ w2, bf16 *__restrict__ dpre_t, int n, int d_R, int h_kv) {
  __shared__ float tile[32][33];
  const int r = blockIdx.x * 32 + threadIdx.x;
  for (int y = threadIdx.y; y < 32; y += 8) {
    const int t = blockIdx.y * 32 + y;
    float v = 0.f;
    if (t < n && r < d_R) {
      float da = 0.f;
      for (int m = 0; m < h_kv; m++) da = fmaf(ds[(size_t)t * h_kv + m], w2[(size_t)r * h_kv + m], da);
      const float p = pre[(size_t)t * d_R + r], sg = sigmoidf_(p);
      v = da * (sg * (1.0f + p * (1.0f - sg)));
    }
    tile[y][threadIdx.x] = v;
  }
  __syncthreads();
  const int t = blockIdx.y * 32 + threadIdx.x;
  for (int y = threadIdx.y; y < 32; y += 8) {
    const int rr = blockIdx.x * 32 + y;
    if (t < n && rr < d_R) dpre_t[(size_t)rr * n + t] = __float2bfloat16_rn(tile[threadIdx.x][y]);
  }
}

__device__ int g_train_status;

// workspace from the stream-ordered allocator: after the first call the pool serves it without a
// device synchronisation
struct Scratch {
  cudaStream_t st = nullptr;
  void *p[8] = {};
  ~Scratch() { for (void *q : p) if (q) cudaFreeAsync(q, st); }
};

}  // namespace

#define TCK(call)                                                            \
  do {                                                                       \
    cudaError_t e__ = (call);                                                \
    if (e__ != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; }  \
  } while (0)

extern "C" int locret_rh_loss_grad(const void *z, const float *labels, const void *w1, const void *w2, int32_t n,
                                   int32_t d_in, int32_t d_R, int32_t h_kv, float alpha, float *loss,
                                   float *d_w1, float *d_w2, void *stream) {
  if (!z || !labels || !w1 || !w2 || !loss || !d_w1 || !d_w2) return LOCRET_ERR_INVALID;
  if (n < 64 || n % 64 || d_in < 64 || d_in % 64 || d_R < 32 || d_R % 32 || h_kv < 1 || h_kv > 32 || alpha < 0.f)
    return LOCRET_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(z) | reinterpret_cast<uintptr_t>(w1) | reinterpret_cast<uintptr_t>(d_w1)) & 15u)
    return LOCRET_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  Scratch sc;  // freed on every return path
  sc.st = st;
  bf16 *w1_t, *z_t, *dpre_t;
  float *pre, *w2f, *s, *ds;
  auto alloc = [&](int slot, void **out, size_t bytes) {
    if (cudaMallocAsync(out, bytes, st) != cudaSuccess) { cudaGetLastError(); return false; }
    sc.p[slot] = *out;
    return true;
  };
  if (!alloc(0, (void **)&w1_t, (size_t)d_R * d_in * sizeof(bf16)) || !alloc(1, (void **)&z_t, (size_t)d_in * n * sizeof(bf16)) ||
      !alloc(2, (void **)&dpre_t, (size_t)d_R * n * sizeof(bf16)) || !alloc(3, (void **)&pre, (size_t)n * d_R * sizeof(float)) ||
      !alloc(4, (void **)&w2f, (size_t)d_R * h_kv * sizeof(float)) || !alloc(5, (void **)&s, (size_t)n * h_kv * sizeof(float)) ||
      !alloc(6, (void **)&ds, (size_t)n * h_kv * sizeof(float)))
    return LOCRET_ERR_ALLOC;
  int *d_status = nullptr;
  TCK(cudaGetSymbolAddress((void **)&d_status, g_train_status));
  TCK(cudaMemsetAsync(d_status, 0, sizeof(int), st));
  TCK(cudaMemsetAsync(loss, 0, sizeof(float), st));
  TCK(cudaMemsetAsync(d_w2, 0, (size_t)d_R * h_kv * sizeof(float), st));
  TCK(launch_transpose_bf16((const bf16 *)w1, w1_t, d_in, d_R, st));   // [d_in x d_R] -> [d_R x d_in]
  TCK(launch_transpose_bf16((const bf16 *)z, z_t, n, d_in, st));       // [n x d_in]  -> [d_in x n]
  TCK(launch_bf16_to_f32((const bf16 *)w2, w2f, d_R * h_kv, st));
  // pre = z W1 (fp32)
  TCK(launch_gemm_tc_f32((const bf16 *)z, d_in, w1_t, d_in, pre, d_R, n, d_R, d_in, d_status, st));
  rh_scores_f32_kernel<<<(n + 7) / 8, 256, 0, st>>>(pre, w2f, s, n, d_R, h_kv);
  TCK(cudaGetLastError());
  rh_loss_kernel<<<(n * h_kv + 255) / 256, 256, 0, st>>>(s, labels, ds, loss, n, h_kv, alpha);
  TCK(cudaGetLastError());
  const int slab = 256;
  rh_dw2_kernel<<<dim3((d_R + 127) / 128, (n + slab - 1) / slab), 128, 0, st>>>(pre, ds, d_w2, n, d_R, h_kv, slab);
  TCK(cudaGetLastError());
  rh_dpre_t_kernel<<<dim3((d_R + 31) / 32, (n + 31) / 32), dim3(32, 8), 0, st>>>(pre, ds, w2f, dpre_t, n, d_R, h_kv);
  TCK(cudaGetLastError());
  // dW1 [d_in x d_R] = z^T dpre: both operands with the tokens as their contiguous K dimension
  TCK(launch_gemm_tc_f32(z_t, n, dpre_t, n, d_w1, d_R, d_in, d_R, n, d_status, st));
  int status = 0;
  TCK(cudaMemcpyAsync(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  TCK(cudaStreamSynchronize(st));
  return status ? LOCRET_ERR_DEVICE_TIMEOUT : LOCRET_OK;
}

// ---------------------------------------------------------------- AdamW (Appendix A, training)
namespace {
__global__ void adamw_kernel(float *__restrict__ p, bf16 *__restrict__ p_bf16, const float *__restrict__ g,
                             float *__restrict__ m, float *__restrict__ v, size_t n, float lr, float beta1,
                             float beta2, float eps, float wd, float bc1, float bc2) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float gi = g[i];
  const float mi = beta1 * m[i] + (1.0f - beta1) * gi;
  const float vi = beta2 * v[i] + (1.0f - beta2) * gi * gi;
  m[i] = mi;
  v[i] = vi;
  const float pi = p[i] * (1.0f - lr * wd) - lr * (mi / bc1) / (sqrtf(vi / bc2) + eps);
  p[i] = pi;
  if (p_bf16) p_bf16[i] = __float2bfloat16_rn(pi);
}
}  // namespace

extern "C" int locret_adamw_step(float *param, void *param_bf16, const float *grad, float *m, float *v, int64_t n,
                                 int32_t step, float lr, float beta1, float beta2, float eps, float weight_decay,
                                 void *stream) {
  if (!param || !grad || !m || !v || n < 1 || step < 1) return LOCRET_ERR_INVALID;
  if (!(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f) || eps <= 0.f) return LOCRET_ERR_INVALID;
  const float bc1 = 1.0f - powf(beta1, (float)step), bc2 = 1.0f - powf(beta2, (float)step);
  adamw_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(param, (bf16 *)param_bf16, grad, m, v,
                                                                             (size_t)n, lr, beta1, beta2, eps,
                                                                             weight_decay, bc1, bc2);
  TCK(cudaGetLastError());
  return LOCRET_OK;
}
