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
// The block that finishes last (counted with a wrapping atomic, so the counter is zero again
// afterwards) adds the per-block partials in block order: deterministic, and no second launch.
template <int MODE>
__global__ void __launch_bounds__(GV_THREADS)
gemv_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ Wt, int N, int K, bf16 *__restrict__ y,
            const float *__restrict__ W2, float *__restrict__ partial, int h_kv, int act,
            unsigned *__restrict__ counter, float *__restrict__ score_out, int score_stride) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *sx = reinterpret_cast<uint4 *>(smem_raw);  // K / 8 vectors
  float *swarp = reinterpret_cast<float *>(sx + K / 8);  // [8 warps][32]
  for (int i = threadIdx.x; i < K / 8; i += GV_THREADS) sx[i] = reinterpret_cast<const uint4 *>(x)[i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (GV_THREADS / 32) + warp, nw = gridDim.x * (GV_THREADS / 32);
  float score = 0.f;  // MODE 1: lane m < h_kv accumulates head m
  if (MODE == 0) {
    for (int n = gw; n < N; n += nw) {
      const uint4 *row = reinterpret_cast<const uint4 *>(Wt + (size_t)n * K);
      float s = 0.f;
#pragma unroll 8
      for (int v = lane; v < K / 8; v += 32) s += dot8(__ldg(row + v), sx[v]);
      s = warp_sum(s);
      if (lane == 0) y[n] = __float2bfloat16_rn(s);
    }
  } else {
    // two warps per row (halves of K), four rows per block at a time: d_R rows are too few to
    // keep enough loads in flight with one warp per row
    __shared__ float shalf[GV_THREADS / 32];
    const int kv2 = K / 16;  // vectors per half row
    for (int n0 = blockIdx.x * 4; n0 < N; n0 += gridDim.x * 4) {
      const int n = n0 + (warp >> 1), hf = warp & 1;
      float s = 0.f;
      if (n < N) {
        const uint4 *row = reinterpret_cast<const uint4 *>(Wt + (size_t)n * K) + hf * kv2;
        const uint4 *xs = sx + hf * kv2;
#pragma unroll 4
        for (int v = lane; v < kv2; v += 32) s += dot8(__ldg(row + v), xs[v]);
      }
      s = warp_sum(s);
      if (lane == 0) shalf[warp] = s;
      __syncthreads();
      if (hf == 0 && n < N) {
        const float hdn = apply_act(shalf[warp] + shalf[warp + 1], act);
        if (lane < h_kv) score = fmaf(hdn, W2[(size_t)n * h_kv + lane], score);
      }
      __syncthreads();
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
    if (counter) {
      __shared__ bool last;
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) last = atomicInc(counter, gridDim.x - 1) == gridDim.x - 1;
      __syncthreads();
      if (last) {
        __threadfence();
        // warp w sums heads w, w + 8, ...: lanes stride over the blocks, then a shuffle tree
        // (a fixed order, so the sum does not depend on which block came last)
        for (int m = warp; m < h_kv; m += GV_THREADS / 32) {
          float t = 0.f;
          for (unsigned b = lane; b < gridDim.x; b += 32) t += __ldcg(partial + (size_t)b * h_kv + m);
          t = warp_sum(t);
          if (lane == 0) score_out[(size_t)m * score_stride] = t;
        }
      }
    }
  }
}

// Projection of one token with positions, RoPE and cache append: a warp computes the two rows
// (i, i + d/2) of one head, so it holds a whole rotation pair.  The rotation starts from the
// bf16-rounded projection, the value the pre-RoPE cache stores.
__global__ void __launch_bounds__(GV_THREADS)
gemv_rope_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ Wt, int K, bf16 *__restrict__ staging,
                 RopeAppendArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *sx = reinterpret_cast<uint4 *>(smem_raw);  // K / 8 vectors
  for (int i = threadIdx.x; i < K / 8; i += GV_THREADS) sx[i] = reinterpret_cast<const uint4 *>(x)[i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (GV_THREADS / 32) + warp, nw = gridDim.x * (GV_THREADS / 32);
  const int half = a.d / 2, heads = a.h + 2 * a.h_kv;
  for (int it = gw; it < heads * half; it += nw) {
    const int hd = it / half, i = it - hd * half;
    const int n0 = hd * a.d + i, n1 = n0 + half;
    const uint4 *r0 = reinterpret_cast<const uint4 *>(Wt + (size_t)n0 * K);
    const uint4 *r1 = reinterpret_cast<const uint4 *>(Wt + (size_t)n1 * K);
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int v = lane; v < K / 8; v += 32) {
      const uint4 xv = sx[v];
      s0 += dot8(__ldg(r0 + v), xv);
      s1 += dot8(__ldg(r1 + v), xv);
    }
    s0 = warp_sum(s0);
    s1 = warp_sum(s1);
    if (lane != 0) continue;
    const bf16 b0 = __float2bfloat16_rn(s0), b1 = __float2bfloat16_rn(s1);
    staging[n0] = b0;
    staging[n1] = b1;
    const int slot = a.len;
    if (hd < a.h + a.h_kv) {
      const float2 t = a.cs[(size_t)slot * half + i];
      const float x0 = __bfloat162float(b0), x1 = __bfloat162float(b1);
      // lower half: x1 cos − x2 sin ; upper half: x2 cos + x1 sin
      const bf16 q0 = __float2bfloat16_rn(x0 * t.x - x1 * t.y), q1 = __float2bfloat16_rn(x1 * t.x + x0 * t.y);
      if (hd < a.h) {
        a.q_rot[n0] = q0;
        a.q_rot[n1] = q1;
      } else {
        const int m = hd - a.h;
        const size_t off = ((size_t)m * a.cap + slot) * a.d + i;
        if (a.k_pre) { a.k_pre[off] = b0; a.k_pre[off + half] = b1; }  // null for a 4-bit cache
        a.k_rot[off] = q0;
        a.k_rot[off + half] = q1;
        if (i == 0) a.tid[(size_t)m * a.cap + slot] = a.seen;
      }
      if (a.z_post) { a.z_post[n0] = q0; a.z_post[n1] = q1; }
    } else {
      const int m = hd - a.h - a.h_kv;
      const size_t off = ((size_t)m * a.cap + slot) * a.d + i;
      a.v[off] = b0;
      a.v[off + half] = b1;
      if (a.z_post) { a.z_post[n0] = b0; a.z_post[n1] = b1; }
    }
  }
}

// ---- decode attention: grid (h_kv, splits, head groups of <= 8).  128 threads: a tile of 128
// keys and values is brought into shared memory with 16-byte loads (all of a thread's loads in
// flight together; key rows rotated by their index so that thread = key reads without bank
// conflicts); in the score phase thread = key, in the value phase thread = column.
constexpr int DA_THREADS = 128, DA_MAXG = 8;

// G: query heads per block (a power of two up to DA_MAXG; the launcher picks the GQA group size);
// D: head_dim (= d), compile-time so that the tile indexing needs no divisions
template <int G, int D>
__global__ void __launch_bounds__(DA_THREADS)
attn_decode_kernel(const bf16 *__restrict__ q_rot, const bf16 *__restrict__ k_rot,
                   const bf16 *__restrict__ v, float *__restrict__ part_o, float *__restrict__ part_ml,
                   int h, int h_kv, int d, int cap, int n, int n_splits, float scale_log2,
                   unsigned *__restrict__ counters, bf16 *__restrict__ out) {
  extern __shared__ uint4 da_smem[];  // K tile [128][d/8], V tile [128][d/8]
  __shared__ __align__(16) float sq[DA_MAXG][128];
  __shared__ __align__(16) float sp[DA_THREADS * DA_MAXG];  // p[key][head]; reused for the final column sums
  __shared__ float sred[DA_MAXG][4];
  const int g = h / h_kv;
  const int m = blockIdx.x, split = blockIdx.y, hg = blockIdx.z;
  const int h0 = m * g + hg * G;
  const int gh = min(G, g - hg * G);  // heads handled here
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < gh * D; i += DA_THREADS) sq[i / D][i % D] = __bfloat162float(q_rot[(size_t)(h0 + i / D) * D + i % D]);
  __syncthreads();
  const int per = (n + n_splits - 1) / n_splits;
  const int k0 = split * per, k1 = min(n, k0 + per);
  const bf16 *kb = k_rot + (size_t)m * cap * D, *vb = v + (size_t)m * cap * D;
  constexpr int vpr = D / 8;  // 16-byte vectors per row: 8, 12 or 16
  constexpr int HC = D / 2;   // value phase: thread = column pair, two key halves of the tile
  const int cp = tid % HC, kh = tid / HC;
  uint4 *sK = da_smem, *sV = da_smem + DA_THREADS * vpr;

  float mrun[G], lrun[G], acc[G][2];
#pragma unroll
  for (int i = 0; i < G; i++) { mrun[i] = -INFINITY; lrun[i] = 0.f; acc[i][0] = acc[i][1] = 0.f; }

  for (int t0 = k0; t0 < k1; t0 += DA_THREADS) {
    {  // the tile: row r of K at vectors (c + r) % vpr, V row-major
      uint4 kreg[16], vreg[16];
#pragma unroll
      for (int it = 0; it < 16; it++) {
        const int idx = tid + it * DA_THREADS, r = idx / vpr, c = idx - r * vpr;
        if (it < vpr && t0 + r < k1) {
          kreg[it] = __ldg(reinterpret_cast<const uint4 *>(kb + (size_t)(t0 + r) * D) + c);
          vreg[it] = __ldg(reinterpret_cast<const uint4 *>(vb + (size_t)(t0 + r) * D) + c);
        }
      }
#pragma unroll
      for (int it = 0; it < 16; it++) {
        const int idx = tid + it * DA_THREADS, r = idx / vpr, c = idx - r * vpr;
        if (it < vpr && t0 + r < k1) {
          int cr = c + r % vpr;
          if (cr >= vpr) cr -= vpr;
          sK[r * vpr + cr] = kreg[it];
          sV[idx] = vreg[it];
        }
      }
    }
    __syncthreads();
    const int key = t0 + tid;
    float s[G];
#pragma unroll
    for (int i = 0; i < G; i++) s[i] = -INFINITY;
    if (key < k1) {
#pragma unroll
      for (int i = 0; i < G; i++) s[i] = 0.f;
      const uint4 *kr = sK + tid * vpr;
      const int rot = tid % vpr;
      for (int c = 0; c < vpr; c++) {
        int cr = c + rot;
        if (cr >= vpr) cr -= vpr;
        const uint4 kv = kr[cr];
        float kf[8];
        {
          const __nv_bfloat162 *kp = reinterpret_cast<const __nv_bfloat162 *>(&kv);
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const float2 f = __bfloat1622float2(kp[e]);
            kf[2 * e] = f.x; kf[2 * e + 1] = f.y;
          }
        }
#pragma unroll
        for (int i = 0; i < G; i++) {
          if (i < gh) {
            const float4 q0 = *reinterpret_cast<const float4 *>(&sq[i][c * 8]);
            const float4 q1 = *reinterpret_cast<const float4 *>(&sq[i][c * 8 + 4]);
            s[i] = fmaf(kf[0], q0.x, s[i]); s[i] = fmaf(kf[1], q0.y, s[i]);
            s[i] = fmaf(kf[2], q0.z, s[i]); s[i] = fmaf(kf[3], q0.w, s[i]);
            s[i] = fmaf(kf[4], q1.x, s[i]); s[i] = fmaf(kf[5], q1.y, s[i]);
            s[i] = fmaf(kf[6], q1.z, s[i]); s[i] = fmaf(kf[7], q1.w, s[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < G; i++) s[i] = (i < gh) ? s[i] * scale_log2 : -INFINITY;
    }
    // tile maximum per head
#pragma unroll
    for (int i = 0; i < G; i++) {
      float mx = warp_max(s[i]);
      if (lane == 0) sred[i][warp] = mx;
    }
    __syncthreads();
    float alpha[G];
#pragma unroll
    for (int i = 0; i < G; i++) {
      const float tmax = fmaxf(fmaxf(sred[i][0], sred[i][1]), fmaxf(sred[i][2], sred[i][3]));
      const float mnew = fmaxf(mrun[i], tmax);
      const float muse = (mnew == -INFINITY) ? 0.f : mnew;
      alpha[i] = exp2f(mrun[i] - muse);
      mrun[i] = mnew;
      const float p = exp2f(s[i] - muse);
      sp[tid * G + i] = p;
      s[i] = p;
    }
    __syncthreads();  // sred is reused below, sp is complete
#pragma unroll
    for (int i = 0; i < G; i++) {
      float sm = warp_sum(s[i]);
      if (lane == 0) sred[i][warp] = sm;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < G; i++)
      lrun[i] = lrun[i] * alpha[i] + (sred[i][0] + sred[i][1]) + (sred[i][2] + sred[i][3]);
    // values: thread = column pair cp, keys [64 kh, 64 kh + 64) of the tile
    if (kh < 2) {
#pragma unroll
      for (int i = 0; i < G; i++) { acc[i][0] *= alpha[i]; acc[i][1] *= alpha[i]; }
      const int cnt = min(DA_THREADS, k1 - t0);
      const uint32_t *sv = reinterpret_cast<const uint32_t *>(sV);
      const int kend = min(cnt, kh * 64 + 64);
#pragma unroll 4
      for (int kk = kh * 64; kk < kend; kk++) {
        const uint32_t v2 = sv[kk * HC + cp];
        const float v0 = __uint_as_float(v2 << 16), v1 = __uint_as_float(v2 & 0xffff0000u);
        float pr[G];
        if (G % 4 == 0) {
#pragma unroll
          for (int i4 = 0; i4 < G / 4; i4++) {
            const float4 t = *reinterpret_cast<const float4 *>(&sp[kk * G + 4 * i4]);
            pr[4 * i4] = t.x; pr[4 * i4 + 1] = t.y; pr[4 * i4 + 2] = t.z; pr[4 * i4 + 3] = t.w;
          }
        } else {
#pragma unroll
          for (int i = 0; i < G; i++) pr[i] = sp[kk * G + i];
        }
#pragma unroll
        for (int i = 0; i < G; i++) {
          acc[i][0] = fmaf(pr[i], v0, acc[i][0]);
          acc[i][1] = fmaf(pr[i], v1, acc[i][1]);
        }
      }
    }
    __syncthreads();
  }
  // the two key halves of every column pair meet in shared memory
  if (kh == 1) {
#pragma unroll
    for (int i = 0; i < G; i++) { sp[(i * HC + cp) * 2] = acc[i][0]; sp[(i * HC + cp) * 2 + 1] = acc[i][1]; }
  }
  __syncthreads();
  // partial results: o [h][split][d], (m, l) [h][split][2]
#pragma unroll
  for (int i = 0; i < G; i++) {
    if (i < gh) {
      const size_t hs = (size_t)(h0 + i) * n_splits + split;
      if (kh == 0) {
        part_o[hs * D + 2 * cp] = acc[i][0] + sp[(i * HC + cp) * 2];
        part_o[hs * D + 2 * cp + 1] = acc[i][1] + sp[(i * HC + cp) * 2 + 1];
      }
      if (tid == 0) { part_ml[hs * 2] = mrun[i]; part_ml[hs * 2 + 1] = lrun[i]; }
    }
  }
  // the split that finishes last for this (KV head, head group) merges the partial results, in
  // split order; the wrapping atomic leaves the counter at zero for the next step
  __shared__ bool last;
  __threadfence();
  __syncthreads();
  if (tid == 0) last = atomicInc(&counters[m * gridDim.z + hg], n_splits - 1) == (unsigned)(n_splits - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  // sm / sl: running maximum and sum of every split; then one thread per head turns them into
  // weights; then thread = column adds the weighted partial outputs, four loads in flight
  __shared__ float sm[DA_MAXG][64], sl[DA_MAXG][64], sinv[DA_MAXG];
  for (int idx = tid; idx < gh * n_splits; idx += DA_THREADS) {
    const int i = idx / n_splits, s2 = idx - i * n_splits;
    const size_t hs = (size_t)(h0 + i) * n_splits + s2;
    sm[i][s2] = __ldcg(part_ml + hs * 2);
    sl[i][s2] = __ldcg(part_ml + hs * 2 + 1);
  }
  __syncthreads();
  if (tid < gh) {
    float mx = -INFINITY;
    for (int s2 = 0; s2 < n_splits; s2++) mx = fmaxf(mx, sm[tid][s2]);
    float l = 0.f;
    for (int s2 = 0; s2 < n_splits; s2++) {
      const float ms = sm[tid][s2];
      const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - mx);
      l += w * sl[tid][s2];
      sm[tid][s2] = w;
    }
    sinv[tid] = 1.0f / l;
  }
  __syncthreads();
  if (tid < D) {
    // all heads of this column together, four splits at a time: 4 G loads in flight per thread
    float o[G];
#pragma unroll
    for (int i = 0; i < G; i++) o[i] = 0.f;
    const float *po = part_o + (size_t)h0 * n_splits * D + tid;
    for (int s2 = 0; s2 < n_splits; s2 += 4) {
      float a[G][4];
#pragma unroll
      for (int i = 0; i < G; i++)
#pragma unroll
        for (int u = 0; u < 4; u++)
          a[i][u] = (i < gh && s2 + u < n_splits) ? __ldcg(po + ((size_t)i * n_splits + s2 + u) * D) : 0.f;
#pragma unroll
      for (int i = 0; i < G; i++)
#pragma unroll
        for (int u = 0; u < 4; u++)
          if (s2 + u < n_splits) o[i] = fmaf(sm[i][s2 + u], a[i][u], o[i]);
    }
#pragma unroll
    for (int i = 0; i < G; i++)
      if (i < gh) out[(size_t)(h0 + i) * D + tid] = __float2bfloat16_rn(o[i] * sinv[i]);
  }
}

}  // namespace

cudaError_t launch_gemv(const bf16 *x, const bf16 *Wt, int N, int K, bf16 *y, cudaStream_t st) {
  if (K % 8) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = min((N + 7) / 8, 148 * 4);
  gemv_kernel<0><<<blocks, GV_THREADS, smem, st>>>(x, Wt, N, K, y, nullptr, nullptr, 0, 0, nullptr, nullptr, 0);
  return cudaGetLastError();
}

int rh_gemv_blocks(int d_R) { return min((d_R + 3) / 4, 148 * 4); }

cudaError_t launch_gemv_rope(const bf16 *x, const bf16 *Wt, int K, bf16 *staging, const RopeAppendArgs &a,
                             cudaStream_t st) {
  if (K % 8 || a.d % 2) return cudaErrorInvalidValue;
  const int items = (a.h + 2 * a.h_kv) * (a.d / 2);
  const int blocks = min((items + 7) / 8, 148 * 4);
  gemv_rope_kernel<<<blocks, GV_THREADS, K * 2, st>>>(x, Wt, K, staging, a);
  return cudaGetLastError();
}

// score_out: where the token's scores go (element m * score_stride for KV head m); counter: one
// zero-initialised word that the kernel leaves at zero
cudaError_t launch_rh_gemv(const bf16 *z, const bf16 *W1t, const float *W2, float *partial, int d_R, int K,
                           int h_kv, int act, unsigned *counter, float *score_out, int score_stride,
                           cudaStream_t st) {
  if (K % 16 || h_kv > 32) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = rh_gemv_blocks(d_R);
  gemv_kernel<1><<<blocks, GV_THREADS, smem, st>>>(z, W1t, d_R, K, nullptr, W2, partial, h_kv, act, counter,
                                                  score_out, score_stride);
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
                                    float *part_o, float *part_ml, unsigned *counters, int h, int h_kv, int d,
                                    int cap, int n, int n_splits, cudaStream_t st) {
  const int g = h / h_kv;
  const int G = g >= 8 ? 8 : (g > 2 ? (g == 4 ? 4 : 8) : g);  // 1, 2, 4 exactly; otherwise blocks of 8
  dim3 grid(h_kv, n_splits, (g + G - 1) / G);
  if ((int)grid.x * (int)grid.z > 32 * 16) return cudaErrorInvalidValue;  // counters: one per (x, z)
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  const int smem = 2 * DA_THREADS * d * (int)sizeof(bf16);
  auto launch = [&](auto kern) -> cudaError_t {
    static bool attr_set[4][3] = {};  // per (G, d) instantiation: the kernels share one pointer type
    bool &done = attr_set[G == 1 ? 0 : (G == 2 ? 1 : (G == 4 ? 2 : 3))][d == 64 ? 0 : (d == 96 ? 1 : 2)];
    if (!done) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           2 * DA_THREADS * 128 * (int)sizeof(bf16));
      if (e != cudaSuccess) return e;
      done = true;
    }
    kern<<<grid, DA_THREADS, smem, st>>>(q_rot, k_rot, v, part_o, part_ml, h, h_kv, d, cap, n, n_splits,
                                         scale_log2, counters, out);
    return cudaGetLastError();
  };
#define LOCRET_DA_CASE(GG)                                           \
  switch (d) {                                                       \
    case 64: return launch(attn_decode_kernel<GG, 64>);              \
    case 96: return launch(attn_decode_kernel<GG, 96>);              \
    case 128: return launch(attn_decode_kernel<GG, 128>);            \
    default: return cudaErrorInvalidValue;                           \
  }
  switch (G) {
    case 1: LOCRET_DA_CASE(1)
    case 2: LOCRET_DA_CASE(2)
    case 4: LOCRET_DA_CASE(4)
    default: LOCRET_DA_CASE(8)
  }
#undef LOCRET_DA_CASE
}

}  // namespace locret
