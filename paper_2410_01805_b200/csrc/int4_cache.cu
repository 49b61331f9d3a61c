// The 4-bit cache variant (the paper's Appendix H combines a 4-bit KV cache with the method).
// Format: symmetric codes in [-8, 7], two per byte (even element in the low nibble), one fp16
// scale per head vector: scale = fp16(absmax / 7) (1 if that is zero),
// code = clamp(rint(x / scale), -8, 7), decided in fp32.  Units are quantised when they enter
// the cache; the keys are stored pre-RoPE.  Before attention a pre-pass expands the retained
// units into bf16 scratch (keys rotated at the unit's position in temporal order, its rank), so
// the attention kernels are the same as for a bf16 cache; eviction moves codes and scales unchanged.
#include "common.cuh"

namespace locret {

namespace {

__device__ __forceinline__ float code_lo(uint32_t byte) { return (float)((int)(byte << 28) >> 28); }
__device__ __forceinline__ float code_hi(uint32_t byte) { return (float)((int)(byte << 24) >> 28); }

// 8 consecutive elements from 4 bytes of codes
__device__ __forceinline__ void dequant8(uint32_t w, float s, float (&x)[8]) {
#pragma unroll
  for (int b = 0; b < 4; b++) {
    const uint32_t byte = (w >> (8 * b)) & 0xFFu;
    x[2 * b] = code_lo(byte) * s;
    x[2 * b + 1] = code_hi(byte) * s;
  }
}
__device__ __forceinline__ uint4 to_bf16x8(const float (&x)[8]) {
  uint4 o;
  o.x = pack_bf16(x[0], x[1]); o.y = pack_bf16(x[2], x[3]);
  o.z = pack_bf16(x[4], x[5]); o.w = pack_bf16(x[6], x[7]);
  return o;
}

// One thread: elements [c, c+8) and [c+half, c+half+8) of one (head, slot) vector of K and V.
__global__ void dequant_rope_kernel(Int4Half q, bf16 *__restrict__ k_rot, bf16 *__restrict__ v_out,
                                    const float2 *__restrict__ cs, int h_kv, int d, int cap, int len,
                                    int rotate, const int32_t *__restrict__ rank, int ranked_len) {
  const int row = blockIdx.x * blockDim.y + threadIdx.y;
  if (row >= h_kv * len) return;
  const int m = row / len, i = row - m * len;
  const int half = d / 2, c = threadIdx.x * 8;
  const size_t u = (size_t)m * cap + i;
  const uint8_t *kc = q.kq + u * half, *vc = q.vq + u * half;
  const float ks = __half2float(q.ks[u]), vs = __half2float(q.vs[u]);
  float a[8], b[8];
  dequant8(*reinterpret_cast<const uint32_t *>(kc + c / 2), ks, a);
  dequant8(*reinterpret_cast<const uint32_t *>(kc + (c + half) / 2), ks, b);
  if (rotate) {
    const int pos = i < ranked_len ? rank[u] : i;
    const float2 *t = cs + (size_t)pos * half + c;
#pragma unroll
    for (int e = 0; e < 8; e++) {
      const float x1 = a[e], x2 = b[e];
      a[e] = x1 * t[e].x - x2 * t[e].y;
      b[e] = x2 * t[e].x + x1 * t[e].y;
    }
  }
  *reinterpret_cast<uint4 *>(k_rot + u * d + c) = to_bf16x8(a);
  *reinterpret_cast<uint4 *>(k_rot + u * d + c + half) = to_bf16x8(b);
  dequant8(*reinterpret_cast<const uint32_t *>(vc + c / 2), vs, a);
  dequant8(*reinterpret_cast<const uint32_t *>(vc + (c + half) / 2), vs, b);
  *reinterpret_cast<uint4 *>(v_out + u * d + c) = to_bf16x8(a);
  *reinterpret_cast<uint4 *>(v_out + u * d + c + half) = to_bf16x8(b);
}

// One warp per (token, kv head, K|V) vector of the chunk: quantise from bf16 rows and append.
// src row stride and head offsets describe where the vectors live (staging of the chunk, or a
// plain [h_kv][n][d] array on import).
__global__ void quantize_kernel(const bf16 *__restrict__ k_src, const bf16 *__restrict__ v_src,
                                long long tok_stride, long long head_stride, Int4Half q, int n_tok,
                                int h_kv, int d, int cap, int slot0) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= n_tok * h_kv * 2) return;
  const int t = warp / (2 * h_kv), rem = warp - t * 2 * h_kv;
  const bool is_v = rem >= h_kv;
  const int m = is_v ? rem - h_kv : rem;
  const bf16 *src = (is_v ? v_src : k_src) + (size_t)t * tok_stride + (size_t)m * head_stride;
  float x0[2], x1[2];
  float amax = 0.f;
#pragma unroll
  for (int k = 0; k < 2; k++) {
    const int p = lane + 32 * k;  // pair index: elements 2p, 2p+1
    x0[k] = x1[k] = 0.f;
    if (2 * p < d) {
      const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162 *>(src + 2 * p);
      x0[k] = __bfloat162float(v2.x);
      x1[k] = __bfloat162float(v2.y);
      amax = fmaxf(amax, fmaxf(fabsf(x0[k]), fabsf(x1[k])));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __half sh = __float2half_rn(__fdiv_rn(amax, 7.0f));
  if (__half2float(sh) == 0.f) sh = __float2half_rn(1.0f);
  const float sf = __half2float(sh);
  const size_t u = (size_t)m * cap + slot0 + t;
  uint8_t *dst = (is_v ? q.vq : q.kq) + u * (d / 2);
#pragma unroll
  for (int k = 0; k < 2; k++) {
    const int p = lane + 32 * k;
    if (2 * p < d) {
      const int q0 = (int)fminf(fmaxf(rintf(__fdiv_rn(x0[k], sf)), -8.f), 7.f);
      const int q1 = (int)fminf(fmaxf(rintf(__fdiv_rn(x1[k], sf)), -8.f), 7.f);
      dst[p] = (uint8_t)((q0 & 0xF) | ((q1 & 0xF) << 4));
    }
  }
  if (lane == 0) (is_v ? q.vs : q.ks)[u] = sh;
}

// Eviction in place: the units that come from another slot bring their codes, scales, score and
// token id along (src_of[m][i] is the slot whose unit ends up in slot i; sources lie at or above
// budget, destinations below).
__global__ void compact_int4_kernel(Int4Half q, float *__restrict__ s, int64_t *__restrict__ t,
                                    const int32_t *__restrict__ src_of, int h_kv, int d, int cap, int budget) {
  const int row = blockIdx.x * blockDim.y + threadIdx.y;
  if (row >= h_kv * budget) return;
  const int m = row / budget, i = row - m * budget;
  const int from = src_of[(size_t)m * budget + i];
  if (from == i) return;
  const size_t us = (size_t)m * cap + from, ud = (size_t)m * cap + i;
  const int vecs = d / 32;  // 16-byte vectors per code row (d/2 bytes)
  const int x = threadIdx.x;
  if (x < vecs)
    reinterpret_cast<uint4 *>(q.kq + ud * (d / 2))[x] = reinterpret_cast<const uint4 *>(q.kq + us * (d / 2))[x];
  else if (x < 2 * vecs)
    reinterpret_cast<uint4 *>(q.vq + ud * (d / 2))[x - vecs] =
        reinterpret_cast<const uint4 *>(q.vq + us * (d / 2))[x - vecs];
  if (x == 0) {
    q.ks[ud] = q.ks[us];
    q.vs[ud] = q.vs[us];
    s[ud] = s[us];
    t[ud] = t[us];
  }
}

}  // namespace

cudaError_t launch_dequant(const Int4Half &q, bf16 *k_out, bf16 *v_out, const float2 *cs, int h_kv, int d,
                           int cap, int len, bool rotate, const int32_t *rank, int ranked_len, cudaStream_t st) {
  if (len == 0) return cudaSuccess;
  const int tx = d / 16, ty = 256 / tx;
  const int rows = h_kv * len;
  dequant_rope_kernel<<<(rows + ty - 1) / ty, dim3(tx, ty), 0, st>>>(q, k_out, v_out, cs, h_kv, d, cap, len,
                                                                    rotate ? 1 : 0, rank, rank ? ranked_len : 0);
  return cudaGetLastError();
}

cudaError_t launch_quantize(const bf16 *k_src, const bf16 *v_src, long long tok_stride,
                            long long head_stride, const Int4Half &q, int n_tok, int h_kv, int d, int cap,
                            int slot0, cudaStream_t st) {
  if (n_tok == 0) return cudaSuccess;
  const long long warps = (long long)n_tok * h_kv * 2;
  const int wpb = 8;
  quantize_kernel<<<(unsigned)((warps + wpb - 1) / wpb), wpb * 32, 0, st>>>(
      k_src, v_src, tok_stride, head_stride, q, n_tok, h_kv, d, cap, slot0);
  return cudaGetLastError();
}

cudaError_t launch_compact_int4(const Int4Half &q, float *s, int64_t *t, const int32_t *src_of, int h_kv, int d,
                                int cap, int budget, cudaStream_t st) {
  const int tx = 2 * (d / 32), ty = 256 / tx;
  const int rows = h_kv * budget;
  compact_int4_kernel<<<(rows + ty - 1) / ty, dim3(tx, ty), 0, st>>>(q, s, t, src_of, h_kv, d, cap, budget);
  return cudaGetLastError();
}

}  // namespace locret
