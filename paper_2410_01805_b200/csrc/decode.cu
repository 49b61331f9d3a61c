// Decoding (the B = 1 case of Eq. 1): one token per step, so every kernel is bound by the bytes
// it must read once: the weights for the two projections, the retained keys and values for
// attention.  Plain CUDA cores, 16-byte loads, no tensor cores (there is no contraction to tile).
#include "common.cuh"

namespace locret {

namespace {

__device__ __forceinline__ float dot8(const uint4 &a, const uint4 &b) {
  const __nv_bfloat162 *x = reinterpret_cast<const __nv_bfloat162 *>(&a);
  const __nv_bfloat162 *y = reinterpret_cast<const __nv_bfloat162 *>(&b);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const float2 xf = __bfloat1622float2(x[i]), yf = __bfloat1622float2(y[i]);
    s = fmaf(xf.x, yf.x, s);
    s = fmaf(xf.y, yf.y, s);
  }
  return s;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

constexpr int GV_THREADS = 256;

// y[n] = sum_k Wt[n][k] x[k]; one warp per output row, rows strided over the grid.
// MODE 0: bf16 store.  MODE 1 (retaining head): hidden = act(y[n]); every warp keeps
// sum_n hidden * W2[n][m] and the block writes one partial score per KV head.
template <int MODE>
__global__ void __launch_bounds__(GV_THREADS)
gemv_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ Wt, int N, int K, bf16 *__restrict__ y,
            const float *__restrict__ W2, float *__restrict__ partial, int h_kv, int act) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *sx = reinterpret_cast<uint4 *>(smem_raw);  // K / 8 vectors
  float *swarp = reinterpret_cast<float *>(sx + K / 8);  // [8 warps][32]
  for (int i = threadIdx.x; i < K / 8; i += GV_THREADS) sx[i] = reinterpret_cast<const uint4 *>(x)[i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (GV_THREADS / 32) + warp, nw = gridDim.x * (GV_THREADS / 32);
  float score = 0.f;  // MODE 1: lane m < h_kv accumulates head m
  for (int n = gw; n < N; n += nw) {
    const uint4 *row = reinterpret_cast<const uint4 *>(Wt + (size_t)n * K);
    float s = 0.f;
    for (int v = lane; v < K / 8; v += 32) s += dot8(row[v], sx[v]);
    s = warp_sum(s);
    if (MODE == 0) {
      if (lane == 0) y[n] = __float2bfloat16_rn(s);
    } else {
      const float hdn = apply_act(s, act);
      if (lane < h_kv) score = fmaf(hdn, W2[(size_t)n * h_kv + lane], score);
    }
  }
  if (MODE == 1) {
    swarp[warp * 32 + lane] = score;
    __syncthreads();
    if (warp == 0 && lane < h_kv) {
      float t = 0.f;
      for (int w = 0; w < GV_THREADS / 32; w++) t += swarp[w * 32 + lane];
      partial[(size_t)blockIdx.x * h_kv + lane] = t;  // layout [block][token 0][head]
    }
  }
}

// ---- decode attention: grid (h_kv, splits, head groups of <= 8).  128 threads: in the score
// phase thread = key of a 128-key tile, in the value phase thread = column of the head vector.
constexpr int DA_THREADS = 128, DA_MAXG = 8;

__global__ void __launch_bounds__(DA_THREADS)
attn_decode_kernel(const bf16 *__restrict__ q_rot, const bf16 *__restrict__ k_rot,
                   const bf16 *__restrict__ v, float *__restrict__ part_o, float *__restrict__ part_ml,
                   int h, int h_kv, int d, int cap, int n, int n_splits, float scale_log2) {
  __shared__ __align__(16) bf16 sq[DA_MAXG][128];
  __shared__ float sp[DA_MAXG][DA_THREADS];
  __shared__ float sred[DA_MAXG][4];
  const int g = h / h_kv;
  const int m = blockIdx.x, split = blockIdx.y, hg = blockIdx.z;
  const int h0 = m * g + hg * DA_MAXG;
  const int gh = min(DA_MAXG, g - hg * DA_MAXG);  // heads handled here
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < gh * d; i += DA_THREADS) sq[i / d][i % d] = q_rot[(size_t)(h0 + i / d) * d + i % d];
  __syncthreads();
  const int per = (n + n_splits - 1) / n_splits;
  const int k0 = split * per, k1 = min(n, k0 + per);
  const bf16 *kb = k_rot + (size_t)m * cap * d, *vb = v + (size_t)m * cap * d;

  float mrun[DA_MAXG], lrun[DA_MAXG], acc[DA_MAXG];
#pragma unroll
  for (int i = 0; i < DA_MAXG; i++) { mrun[i] = -INFINITY; lrun[i] = 0.f; acc[i] = 0.f; }

  for (int t0 = k0; t0 < k1; t0 += DA_THREADS) {
    const int key = t0 + tid;
    float s[DA_MAXG];
#pragma unroll
    for (int i = 0; i < DA_MAXG; i++) s[i] = -INFINITY;
    if (key < k1) {
#pragma unroll
      for (int i = 0; i < DA_MAXG; i++) s[i] = 0.f;
      const uint4 *kr = reinterpret_cast<const uint4 *>(kb + (size_t)key * d);
      for (int c = 0; c < d / 8; c++) {
        const uint4 kv = kr[c];
#pragma unroll
        for (int i = 0; i < DA_MAXG; i++)
          if (i < gh) s[i] += dot8(kv, reinterpret_cast<const uint4 *>(&sq[i][0])[c]);
      }
#pragma unroll
      for (int i = 0; i < DA_MAXG; i++) s[i] = (i < gh) ? s[i] * scale_log2 : -INFINITY;
    }
    // tile maximum per head
#pragma unroll
    for (int i = 0; i < DA_MAXG; i++) {
      float mx = warp_max(s[i]);
      if (lane == 0) sred[i][warp] = mx;
    }
    __syncthreads();
    float alpha[DA_MAXG];
#pragma unroll
    for (int i = 0; i < DA_MAXG; i++) {
      const float tmax = fmaxf(fmaxf(sred[i][0], sred[i][1]), fmaxf(sred[i][2], sred[i][3]));
      const float mnew = fmaxf(mrun[i], tmax);
      const float muse = (mnew == -INFINITY) ? 0.f : mnew;
      alpha[i] = exp2f(mrun[i] - muse);
      mrun[i] = mnew;
      const float p = exp2f(s[i] - muse);
      sp[i][tid] = p;
      s[i] = p;
    }
    __syncthreads();  // sred is reused below, sp is complete
#pragma unroll
    for (int i = 0; i < DA_MAXG; i++) {
      float sm = warp_sum(s[i]);
      if (lane == 0) sred[i][warp] = sm;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < DA_MAXG; i++)
      lrun[i] = lrun[i] * alpha[i] + (sred[i][0] + sred[i][1]) + (sred[i][2] + sred[i][3]);
    // values: thread = column
    if (tid < d) {
#pragma unroll
      for (int i = 0; i < DA_MAXG; i++) acc[i] *= alpha[i];
      const int cnt = min(DA_THREADS, k1 - t0);
      for (int kk = 0; kk < cnt; kk++) {
        const float vv = __bfloat162float(vb[(size_t)(t0 + kk) * d + tid]);
#pragma unroll
        for (int i = 0; i < DA_MAXG; i++)
          if (i < gh) acc[i] = fmaf(sp[i][kk], vv, acc[i]);
      }
    }
    __syncthreads();
  }
  // partial results: o [h][split][d], (m, l) [h][split][2]
#pragma unroll
  for (int i = 0; i < DA_MAXG; i++) {
    if (i < gh) {
      const size_t hs = (size_t)(h0 + i) * n_splits + split;
      if (tid < d) part_o[hs * d + tid] = acc[i];
      if (tid == 0) { part_ml[hs * 2] = mrun[i]; part_ml[hs * 2 + 1] = lrun[i]; }
    }
  }
}

__global__ void attn_decode_combine_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                                           bf16 *__restrict__ out, int h, int d, int n_splits) {
  const int head = blockIdx.x, c = threadIdx.x;
  float mx = -INFINITY;
  for (int s = 0; s < n_splits; s++) mx = fmaxf(mx, part_ml[((size_t)head * n_splits + s) * 2]);
  float l = 0.f, o = 0.f;
  for (int s = 0; s < n_splits; s++) {
    const size_t hs = (size_t)head * n_splits + s;
    const float ms = part_ml[hs * 2];
    const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - mx);
    l += w * part_ml[hs * 2 + 1];
    if (c < d) o += w * part_o[hs * d + c];
  }
  if (c < d) out[(size_t)head * d + c] = __float2bfloat16_rn(o / l);
}

}  // namespace

cudaError_t launch_gemv(const bf16 *x, const bf16 *Wt, int N, int K, bf16 *y, cudaStream_t st) {
  if (K % 8) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = min((N + 7) / 8, 148 * 4);
  gemv_kernel<0><<<blocks, GV_THREADS, smem, st>>>(x, Wt, N, K, y, nullptr, nullptr, 0, 0);
  return cudaGetLastError();
}

int rh_gemv_blocks(int d_R) { return min((d_R + 7) / 8, 148 * 2); }

cudaError_t launch_rh_gemv(const bf16 *z, const bf16 *W1t, const float *W2, float *partial, int d_R, int K,
                           int h_kv, int act, int *n_blocks, cudaStream_t st) {
  if (K % 8 || h_kv > 32) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = rh_gemv_blocks(d_R);
  *n_blocks = blocks;
  gemv_kernel<1><<<blocks, GV_THREADS, smem, st>>>(z, W1t, d_R, K, nullptr, W2, partial, h_kv, act);
  return cudaGetLastError();
}

int decode_attn_splits(int h_kv, int n) {
  int s = (148 * 2 + h_kv - 1) / h_kv;          // about two CTAs per SM in total
  const int max_s = (n + 127) / 128;            // at least one 128-key tile per split
  if (s > max_s) s = max_s;
  if (s > 64) s = 64;
  return s < 1 ? 1 : s;
}

cudaError_t launch_attention_decode(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out,
                                    float *part_o, float *part_ml, int h, int h_kv, int d, int cap, int n,
                                    int n_splits, cudaStream_t st) {
  const int g = h / h_kv;
  dim3 grid(h_kv, n_splits, (g + DA_MAXG - 1) / DA_MAXG);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  attn_decode_kernel<<<grid, DA_THREADS, 0, st>>>(q_rot, k_rot, v, part_o, part_ml, h, h_kv, d, cap, n,
                                                  n_splits, scale_log2);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  attn_decode_combine_kernel<<<h, 128, 0, st>>>(part_o, part_ml, out, h, d, n_splits);
  return cudaGetLastError();
}

}  // namespace locret
