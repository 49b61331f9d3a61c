// The rest of the decoder layer around the attention block: RMSNorm, W_o with its residual, gated
// SiLU FFN with its residual.  The three projections run on the tcgen05 GEMM (residual add and
// silu(gate) * up in its epilogues); shapes that GEMM does not take fall back to the mma.sync
// GEMM plus element-wise kernels.
#include <map>
#include <mutex>
#include <new>

#include "../../include/locret.h"
#include "common.cuh"

using namespace locret;

namespace {

// ---- RMSNorm: one warp per row, fp32 statistics, bf16 in and out
__global__ void rmsnorm_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ gain, bf16 *__restrict__ y,
                               int rows, int D, float eps) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)row * D);
  const uint4 *gv = reinterpret_cast<const uint4 *>(gain);
  uint4 *dst = reinterpret_cast<uint4 *>(y + (size_t)row * D);
  float ss = 0.f;
  for (int v = lane; v < D / 8; v += 32) {
    const uint4 q = src[v];
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float a = __uint_as_float(w[e] << 16), b = __uint_as_float(w[e] & 0xffff0000u);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float inv = rsqrtf(ss / (float)D + eps);
  for (int v = lane; v < D / 8; v += 32) {
    const uint4 q = src[v], g = gv[v];
    const uint32_t w[4] = {q.x, q.y, q.z, q.w}, gw[4] = {g.x, g.y, g.z, g.w};
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float a = __uint_as_float(w[e] << 16) * inv * __uint_as_float(gw[e] << 16);
      const float b = __uint_as_float(w[e] & 0xffff0000u) * inv * __uint_as_float(gw[e] & 0xffff0000u);
      o[e] = pack_bf16(a, b);
    }
    dst[v] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---- fallbacks for shapes the tcgen05 GEMM does not take
__global__ void add_rows_kernel(bf16 *__restrict__ c, const bf16 *__restrict__ r, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) c[i] = __float2bfloat16_rn(__bfloat162float(c[i]) + __bfloat162float(r[i]));
}
// gu [rows x 2F] in the interleaved layout (blocks of 128 gate then 128 up) -> act [rows x F]
__global__ void swiglu_kernel(const float *__restrict__ gu, bf16 *__restrict__ act, int rows, int F) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * F) return;
  const int row = (int)(i / F), c = (int)(i - (size_t)row * F);
  const size_t base = (size_t)row * 2 * F + (size_t)(c / 128) * 256 + (c % 128);
  const float g = gu[base], u = gu[base + 128];
  act[i] = __float2bfloat16_rn(g / (1.0f + __expf(-g)) * u);
}
// dst[n][k] for the gated layout: row t*256 + j (j < 128) = column t*128 + j of W_gate, row
// t*256 + 128 + j = the same column of W_up;  W_* are [K x F] row-major
__global__ void repack_gate_up_kernel(const bf16 *__restrict__ wg, const bf16 *__restrict__ wu,
                                      bf16 *__restrict__ dst, int K, int F) {
  __shared__ bf16 tile[32][33];
  const int which = blockIdx.z;  // 0 gate, 1 up
  const bf16 *src = which ? wu : wg;
  const int c = blockIdx.x * 32 + threadIdx.x;  // column of W (output index)
  for (int r = threadIdx.y; r < 32; r += 8) {
    const int k = blockIdx.y * 32 + r;
    if (k < K && c < F) tile[r][threadIdx.x] = src[(size_t)k * F + c];
  }
  __syncthreads();
  const int k = blockIdx.y * 32 + threadIdx.x;
  for (int r = threadIdx.y; r < 32; r += 8) {
    const int cc = blockIdx.x * 32 + r;
    if (k < K && cc < F) {
      const size_t row = (size_t)(cc / 128) * 256 + (which ? 128 : 0) + (cc % 128);
      dst[row * K + k] = tile[threadIdx.x][r];
    }
  }
}

// general-shape GEMM with fp32 output, for the fallback of the gated projection only (tiny shapes)
__global__ void gemm_f32_naive_kernel(const bf16 *__restrict__ A, const bf16 *__restrict__ Bt,
                                      float *__restrict__ C, int M, int N, int K) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x, m = blockIdx.y;
  if (n >= N || m >= M) return;
  float acc = 0.f;
  for (int k = 0; k < K; k++) acc = fmaf(__bfloat162float(A[(size_t)m * K + k]), __bfloat162float(Bt[(size_t)n * K + k]), acc);
  C[(size_t)m * N + n] = acc;
}
__global__ void gemm_resid_naive_kernel(const bf16 *__restrict__ A, const bf16 *__restrict__ Bt,
                                        const bf16 *__restrict__ R, bf16 *__restrict__ C, int M, int N, int K) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x, m = blockIdx.y;
  if (n >= N || m >= M) return;
  float acc = 0.f;
  for (int k = 0; k < K; k++) acc = fmaf(__bfloat162float(A[(size_t)m * K + k]), __bfloat162float(Bt[(size_t)n * K + k]), acc);
  C[(size_t)m * N + n] = __float2bfloat16_rn(acc + __bfloat162float(R[(size_t)m * N + n]));
}

// scratch shared by the blocks of one stream (one block's step is in flight at a time)
struct BlockScratch {
  int refs = 0;
  bf16 *h = nullptr, *att = nullptr, *x1 = nullptr, *act = nullptr;
  float *gu = nullptr;  // fallback only
  size_t h_b = 0, att_b = 0, x1_b = 0, act_b = 0, gu_b = 0;
};
std::mutex b_mu;
// keyed by (device, stream): the default stream has the same handle on every device
std::map<std::pair<int, cudaStream_t>, BlockScratch *> b_pools;

bool grow_b(void **p, size_t *have, size_t want, cudaStream_t st) {
  if (want <= *have) return true;
  void *np_ = nullptr;
  if (cudaMalloc(&np_, want) != cudaSuccess) { cudaGetLastError(); return false; }
  if (*p) { cudaStreamSynchronize(st); cudaFree(*p); }
  *p = np_;
  *have = want;
  return true;
}

}  // namespace

struct locret_block {
  locret_layer *attn;
  cudaStream_t st;
  int D, hd, F, chunk;
  float eps;
  bf16 *wo_t, *wgu_t, *wd_t, *g1, *g2;  // repacked: [D x hd], [2F x D] gated layout, [D x F]
  int *d_status;
  BlockScratch *pool;
  int device;
};

#define BCK(call)                                                            \
  do {                                                                       \
    cudaError_t e__ = (call);                                                \
    if (e__ != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; }  \
  } while (0)

extern "C" {

void locret_block_destroy(locret_block *B) {
  if (!B) return;
  if (B->attn) { locret_sync_status(B->attn); locret_destroy(B->attn); }
  cudaFree(B->wo_t); cudaFree(B->wgu_t); cudaFree(B->wd_t); cudaFree(B->g1); cudaFree(B->g2);
  cudaFree(B->d_status);
  if (B->pool) {
    std::lock_guard<std::mutex> lk(b_mu);
    if (--B->pool->refs == 0) {
      BlockScratch *p = B->pool;
      cudaFree(p->h); cudaFree(p->att); cudaFree(p->x1); cudaFree(p->act); cudaFree(p->gu);
      b_pools.erase(std::make_pair(B->device, B->st));
      delete p;
    }
  }
  delete B;
}

int locret_block_create(const locret_block_cfg *cfg, int32_t budget, int32_t chunk, int32_t n_stab,
                        locret_block **out) {
  if (out) *out = nullptr;
  if (!cfg || !out || !cfg->w_o || !cfg->w_gate || !cfg->w_up || !cfg->w_down || !cfg->g1 || !cfg->g2)
    return LOCRET_ERR_INVALID;
  if (cfg->d_ff < 128 || cfg->d_ff % 128 || cfg->attn.d_model % 8) return LOCRET_ERR_INVALID;
  locret_block *B = new (std::nothrow) locret_block();
  if (!B) return LOCRET_ERR_ALLOC;
  *B = locret_block{};
  int rc = locret_create(&cfg->attn, budget, chunk, n_stab, &B->attn);
  if (rc != LOCRET_OK) { delete B; return rc; }
  B->st = (cudaStream_t)cfg->attn.stream;
  B->D = cfg->attn.d_model; B->hd = cfg->attn.n_q_heads * cfg->attn.head_dim; B->F = cfg->d_ff;
  B->chunk = chunk;
  B->eps = cfg->rms_eps > 0.f ? cfg->rms_eps : 1e-5f;
  const int D = B->D, hd = B->hd, F = B->F;
  bool ok = cudaMalloc(&B->wo_t, (size_t)D * hd * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&B->wgu_t, (size_t)2 * F * D * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&B->wd_t, (size_t)D * F * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&B->g1, (size_t)D * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&B->g2, (size_t)D * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&B->d_status, sizeof(int)) == cudaSuccess;
  if (ok) {
    std::lock_guard<std::mutex> lk(b_mu);
    if (cudaGetDevice(&B->device) != cudaSuccess) { cudaGetLastError(); B->device = 0; }
    BlockScratch *&p = b_pools[std::make_pair(B->device, B->st)];
    if (!p) p = new (std::nothrow) BlockScratch();
    if (p) {
      p->refs++;
      B->pool = p;
      ok = grow_b((void **)&p->h, &p->h_b, (size_t)chunk * D * sizeof(bf16), B->st) &&
           grow_b((void **)&p->att, &p->att_b, (size_t)chunk * hd * sizeof(bf16), B->st) &&
           grow_b((void **)&p->x1, &p->x1_b, (size_t)chunk * D * sizeof(bf16), B->st) &&
           grow_b((void **)&p->act, &p->act_b, (size_t)chunk * F * sizeof(bf16), B->st);
    } else {
      ok = false;
    }
  }
  if (!ok) { cudaGetLastError(); locret_block_destroy(B); return LOCRET_ERR_ALLOC; }
  cudaError_t e = launch_transpose_bf16((const bf16 *)cfg->w_o, B->wo_t, hd, D, B->st);       // [hd x D] -> [D x hd]
  if (e == cudaSuccess) e = launch_transpose_bf16((const bf16 *)cfg->w_down, B->wd_t, F, D, B->st);  // [F x D] -> [D x F]
  if (e == cudaSuccess) {
    dim3 grid((F + 31) / 32, (D + 31) / 32, 2);
    repack_gate_up_kernel<<<grid, dim3(32, 8), 0, B->st>>>((const bf16 *)cfg->w_gate, (const bf16 *)cfg->w_up,
                                                            B->wgu_t, D, F);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(B->g1, cfg->g1, (size_t)D * sizeof(bf16), cudaMemcpyDeviceToDevice, B->st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(B->g2, cfg->g2, (size_t)D * sizeof(bf16), cudaMemcpyDeviceToDevice, B->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(B->d_status, 0, sizeof(int), B->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(B->st);
  if (e != cudaSuccess) { cudaGetLastError(); locret_block_destroy(B); return LOCRET_ERR_CUDA; }
  *out = B;
  return LOCRET_OK;
}

locret_layer *locret_block_attention(locret_block *B) { return B ? B->attn : nullptr; }

int locret_block_prefill_chunk(locret_block *B, const void *x_in, int32_t n_tok, uint32_t flags, void *y_out) {
  if (!B || !x_in || !y_out) return LOCRET_ERR_INVALID;
  if (n_tok < 1 || n_tok > B->chunk) return LOCRET_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(x_in) | reinterpret_cast<uintptr_t>(y_out)) & 15u) return LOCRET_ERR_INVALID;
  BlockScratch *P = B->pool;
  const int D = B->D, hd = B->hd, F = B->F;
  const bf16 *x = (const bf16 *)x_in;
  bf16 *y = (bf16 *)y_out;
  const int rows_per_blk = 8;
  const dim3 nblk((n_tok + rows_per_blk - 1) / rows_per_blk);
  // h1 = RMSNorm(x; g1)
  rmsnorm_kernel<<<nblk, rows_per_blk * 32, 0, B->st>>>(x, B->g1, P->h, n_tok, D, B->eps);
  BCK(cudaGetLastError());
  // the attention block (projection, RoPE, attention, retaining head, eviction)
  int rc = locret_prefill_chunk(B->attn, P->h, n_tok, flags, P->att);
  if (rc != LOCRET_OK) return rc;
  // x1 = x + attn_out W_o
  const bool tc = n_tok >= 32;
  if (tc && gemm_tc_supported(n_tok, D, hd, hd, hd)) {
    BCK(launch_gemm_tc_resid(P->att, hd, B->wo_t, hd, P->x1, D, n_tok, D, hd, x, D, B->d_status, B->st));
  } else if (n_tok == 1 && hd % 8 == 0) {  // one token: bandwidth-bound GEMV
    BCK(launch_gemv_resid(P->att, B->wo_t, D, hd, x, P->x1, B->st));
  } else {
    gemm_resid_naive_kernel<<<dim3((D + 127) / 128, n_tok), 128, 0, B->st>>>(P->att, B->wo_t, x, P->x1, n_tok, D, hd);
    BCK(cudaGetLastError());
  }
  // h2 = RMSNorm(x1; g2)
  rmsnorm_kernel<<<nblk, rows_per_blk * 32, 0, B->st>>>(P->x1, B->g2, P->h, n_tok, D, B->eps);
  BCK(cudaGetLastError());
  // act = silu(h2 W_gate) * (h2 W_up)
  if (tc && gemm_tc_gated_supported(n_tok, 2 * F, D, D, D)) {
    BCK(launch_gemm_tc_gated(P->h, D, B->wgu_t, D, P->act, F, n_tok, 2 * F, D, B->d_status, B->st));
  } else if (n_tok == 1) {
    BCK(launch_gemv_gated(P->h, B->wgu_t, F, D, P->act, B->st));
  } else {
    {
      std::lock_guard<std::mutex> lk(b_mu);
      if (!grow_b((void **)&P->gu, &P->gu_b, (size_t)B->chunk * 2 * F * sizeof(float), B->st)) return LOCRET_ERR_ALLOC;
    }
    gemm_f32_naive_kernel<<<dim3((2 * F + 127) / 128, n_tok), 128, 0, B->st>>>(P->h, B->wgu_t, P->gu, n_tok, 2 * F, D);
    BCK(cudaGetLastError());
    const size_t n = (size_t)n_tok * F;
    swiglu_kernel<<<(unsigned)((n + 255) / 256), 256, 0, B->st>>>(P->gu, P->act, n_tok, F);
    BCK(cudaGetLastError());
  }
  // y = x1 + act W_down
  if (tc && gemm_tc_supported(n_tok, D, F, F, F)) {
    BCK(launch_gemm_tc_resid(P->act, F, B->wd_t, F, y, D, n_tok, D, F, P->x1, D, B->d_status, B->st));
  } else if (n_tok == 1) {
    BCK(launch_gemv_resid(P->act, B->wd_t, D, F, P->x1, y, B->st));
  } else {
    gemm_resid_naive_kernel<<<dim3((D + 127) / 128, n_tok), 128, 0, B->st>>>(P->act, B->wd_t, P->x1, y, n_tok, D, F);
    BCK(cudaGetLastError());
  }
  return LOCRET_OK;
}

}  // extern "C"

// ---------------------------------------------------------------- training labels (Section 3.3)
namespace {
__global__ void fill_f32_kernel(float *p, size_t n, float v) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}
__device__ int g_cis_status;
}  // namespace

extern "C" int locret_cis_labels(const void *q_ans, const void *k_prompt, int32_t n_a, int32_t n_q, int32_t h,
                                 int32_t h_kv, int32_t d, float scale, float *labels, void *stream) {
  if (!q_ans || !k_prompt || !labels) return LOCRET_ERR_INVALID;
  if (n_a < 1 || n_q < 1 || h < 1 || h_kv < 1 || h % h_kv || (d != 64 && d != 96 && d != 128) || !(scale > 0.f))
    return LOCRET_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(q_ans) | reinterpret_cast<uintptr_t>(k_prompt)) & 15u) return LOCRET_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  int *d_status = nullptr;
  BCK(cudaGetSymbolAddress((void **)&d_status, g_cis_status));
  BCK(cudaMemsetAsync(d_status, 0, sizeof(int), st));
  const size_t n = (size_t)h_kv * n_q;
  fill_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(labels, n, -INFINITY);
  BCK(cudaGetLastError());
  const bf16 *q = (const bf16 *)q_ans, *k = (const bf16 *)k_prompt;
  const int g = h / h_kv;
  for (int j = 0; j < h; j++) {  // one contraction per query head: keys of its KV head x its answer queries
    const int m = j / g;
    BCK(launch_gemm_tc_rowmax(k + (size_t)m * d, h_kv * d, q + (size_t)j * d, h * d, labels + (size_t)m * n_q, n_q,
                              n_a, d, scale, d_status, st));
  }
  int status = 0;
  BCK(cudaMemcpyAsync(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  BCK(cudaStreamSynchronize(st));
  return status ? LOCRET_ERR_DEVICE_TIMEOUT : LOCRET_OK;
}
