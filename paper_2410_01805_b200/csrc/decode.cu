// Decoding (the B = 1 case of Eq. 1): one token per step, so every kernel is bound by the bytes
// it must read once: the weights for the two projections, the retained keys and values for
// attention.  Plain CUDA cores, 16-byte loads, no tensor cores (there is no contraction to tile).
#include <stdlib.h>

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
            unsigned *__restrict__ counter, float *__restrict__ score_out, int score_stride,
            const bf16 *__restrict__ resid) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *sx = reinterpret_cast<uint4 *>(smem_raw);  // K / 8 vectors
  float *swarp = reinterpret_cast<float *>(sx + K / 8);  // [8 warps][32]
  // MODE 1 in a one-token step's chain: the input is the projection's output, complete since the
  // attention kernel before this one passed its own wait, so nothing is waited for here; the next
  // layer's projection may start (and request its weights) at once
  if (MODE == 1) pdl_launch_dependents();
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
      if (lane == 0) y[n] = __float2bfloat16_rn(resid ? s + __bfloat162float(resid[n]) : s);
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
#pragma unroll 12
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
    // the attention kernel of this step must have finished before the next layer's projection (which
    // waits for THIS kernel) overwrites the buffers attention reads
    pdl_wait();
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
  pdl_wait();
  pdl_launch_dependents();
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

// The same projection for K <= 4096 laid out for bandwidth: a block of 512 threads owns a contiguous
// range of rotation pairs, thread t holds element group t of x in registers (no staging step before
// the first weight load) and reads group t of both rows of four pairs at a time, so a block has
// 64 KB of weights in flight and two blocks per SM cover each other's reductions.  The eight
// partial sums of a batch are reduced with one butterfly that halves the number of values at each
// step (9 shuffles instead of 40), then across the warps through shared memory.
constexpr int GW_THREADS = 512, GW_PB = 4;

__global__ void __launch_bounds__(GW_THREADS, 2)
gemv_rope_wide_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ Wt, int K, bf16 *__restrict__ staging,
                      RopeAppendArgs a) {
  __shared__ float red[2][GW_THREADS / 32][2 * GW_PB];
  __shared__ float res[2][2 * GW_PB];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int kv = K / 8;
  const bool act = tid < kv;
  const int half = a.d / 2, heads = a.h + 2 * a.h_kv;
  const int n_pairs = heads * half;
  const int p_lo = (int)((long long)blockIdx.x * n_pairs / gridDim.x);
  const int p_hi = (int)((long long)(blockIdx.x + 1) * n_pairs / gridDim.x);
  const uint4 *W4 = reinterpret_cast<const uint4 *>(Wt);
  // the first batch of weights is requested before x
  uint4 w[2 * GW_PB];
  auto load_batch = [&](int p0) {
#pragma unroll
    for (int j = 0; j < GW_PB; j++) {
      const int it = min(p0 + j, n_pairs - 1);
      const int hd = it / half, i = it - hd * half;
      const size_t n0 = (size_t)hd * a.d + i;
      w[2 * j] = act ? __ldg(W4 + n0 * kv + tid) : make_uint4(0, 0, 0, 0);
      w[2 * j + 1] = act ? __ldg(W4 + (n0 + half) * kv + tid) : make_uint4(0, 0, 0, 0);
    }
  };
  load_batch(p_lo);
  // the weights do not depend on anything before this kernel: the first batch is in flight while the
  // kernel waits for the step before it (whose buffers it is about to overwrite).  The attention
  // kernel may start only after that wait: it requests retained keys before its own, and an
  // eviction of the previous step may still be rewriting them until then.
  pdl_wait();
  pdl_launch_dependents();
  const uint4 xv = act ? __ldg(reinterpret_cast<const uint4 *>(x) + tid) : make_uint4(0, 0, 0, 0);
  int par = 0;
  for (int p0 = p_lo; p0 < p_hi; p0 += GW_PB, par ^= 1) {
    float v[2 * GW_PB];
#pragma unroll
    for (int e = 0; e < 2 * GW_PB; e++) v[e] = dot8(w[e], xv);
    if (p0 + GW_PB < p_hi) load_batch(p0 + GW_PB);  // in flight during the reduction
    // eight values across 32 lanes: exchange half of them at each of three steps
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float send = (lane & 16) ? v[e] : v[e + 4], keep = (lane & 16) ? v[e + 4] : v[e];
      v[e] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int e = 0; e < 2; e++) {
      const float send = (lane & 8) ? v[e] : v[e + 2], keep = (lane & 8) ? v[e + 2] : v[e];
      v[e] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    {
      const float send = (lane & 4) ? v[0] : v[1], keep = (lane & 4) ? v[1] : v[0];
      v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], 2);
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
    if ((lane & 3) == 0) red[par][warp][((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1)] = v[0];
    __syncthreads();
    if (tid < 2 * GW_PB) {
      float t = 0.f;
#pragma unroll
      for (int q = 0; q < GW_THREADS / 32; q++) t += red[par][q][tid];
      res[par][tid] = t;
    }
    __syncthreads();
    if (tid < GW_PB && p0 + tid < p_hi) {
      const int it = p0 + tid;
      const int hd = it / half, i = it - hd * half;
      const int n0 = hd * a.d + i, n1 = n0 + half;
      const bf16 b0 = __float2bfloat16_rn(res[par][2 * tid]), b1 = __float2bfloat16_rn(res[par][2 * tid + 1]);
      staging[n0] = b0;
      staging[n1] = b1;
      const int slot = a.len;
      if (hd < a.h + a.h_kv) {
        const float2 t = a.cs[(size_t)slot * half + i];
        const float x0 = __bfloat162float(b0), x1 = __bfloat162float(b1);
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
}

// 4-bit codes -> floats, the arithmetic of the cache's expansion pre-pass (two codes per byte, even
// element in the low nibble, value = code * scale)
__device__ __forceinline__ void dequant8(uint32_t w, float s, float (&x)[8]) {
#pragma unroll
  for (int b = 0; b < 4; b++) {
    const uint32_t byte = (w >> (8 * b)) & 0xFFu;
    x[2 * b] = (float)((int)(byte << 28) >> 28) * s;
    x[2 * b + 1] = (float)((int)(byte << 24) >> 28) * s;
  }
}
__device__ __forceinline__ uint4 to_bf16x8(const float (&x)[8]) {
  uint4 o;
  o.x = pack_bf16(x[0], x[1]); o.y = pack_bf16(x[2], x[3]);
  o.z = pack_bf16(x[4], x[5]); o.w = pack_bf16(x[6], x[7]);
  return o;
}

// ---- decode attention on warp-level tensor-core instructions.  grid (h_kv, splits, head groups
// of <= 16).  The rows of the m16n8k16 tiles are the query heads of one GQA group (all of them read
// the same keys), padded to 16; keys and values of the split stream through shared memory in
// tiles of 64 (cp.async, two stages).  Each of the four warps takes 16 keys of a tile and keeps
// its own running maximum, sum and output, so the tile loop has no block-wide reduction; the
// four states meet in shared memory at the end, the block writes one partial result per head,
// and the split that finishes last for its (KV head, head group) merges all splits in split
// order (a wrapping atomic counter, left at zero for the next step).
constexpr int DA_THREADS = 128, DA_G = 16, DA_KT = 64;

// INT4: keys [0, n - 1) come from the 4-bit cache (codes and scales expanded, keys rotated at the
// unit's position in temporal order, with the arithmetic of the expansion pre-pass, as the tile is brought into shared
// memory); key n - 1, the token of this step, comes from the bf16 arrays k_rot / v like every key of
// a bf16 cache.
template <int D, bool INT4>
__global__ void __launch_bounds__(DA_THREADS)
attn_decode_kernel(const bf16 *__restrict__ q_rot, const bf16 *__restrict__ k_rot,
                   const bf16 *__restrict__ v, float *__restrict__ part_o, float *__restrict__ part_ml,
                   int h, int h_kv, int cap, int n, int n_splits, float scale_log2,
                   unsigned *__restrict__ counters, bf16 *__restrict__ out, Int4Half q4,
                   const float2 *__restrict__ cs, const int32_t *__restrict__ rank, int ranked_len,
                   const bf16 *__restrict__ tok_k, const bf16 *__restrict__ tok_v) {
  constexpr int LD = D + 8;
  constexpr int VPR = D / 8;  // 16-byte vectors per row
  extern __shared__ __align__(16) unsigned char da_smem[];
  bf16 *sQ = reinterpret_cast<bf16 *>(da_smem);  // [16][LD]
  bf16 *sK = sQ + DA_G * LD;                     // [2][64][LD]
  bf16 *sV = sK + 2 * DA_KT * LD;                // [2][64][LD]
  __shared__ float wm[4][DA_G], wl[4][DA_G];     // per-warp running maximum and sum of every head
  __shared__ float sm[DA_G][64], sl[DA_G][64], sinv[DA_G];
  __shared__ bool last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g4 = lane >> 2, q = lane & 3;
  const int g = h / h_kv;
  const int m = blockIdx.x, split = blockIdx.y, hg = blockIdx.z;
  const int h0 = m * g + hg * DA_G;
  const int gh = min(DA_G, g - hg * DA_G);  // heads handled here
  const int per = (n + n_splits - 1) / n_splits;
  const int k0 = split * per, k1 = min(n, k0 + per);
  const int NKT = k1 > k0 ? (k1 - k0 + DA_KT - 1) / DA_KT : 0;
  const bf16 *kbase = k_rot + (size_t)m * cap * D;
  const bf16 *vbase = v + (size_t)m * cap * D;

  auto load_kv = [&](int buf, int kt) {
    for (int x = tid; x < DA_KT * VPR; x += DA_THREADS) {
      const int r = x / VPR, c = (x - r * VPR) * 8;
      const int key = k0 + kt * DA_KT + r;
      const bool ok = key < k1;
      const size_t off = (size_t)min(key, n - 1) * D + c;
      cp_async16(sK + (buf * DA_KT + r) * LD + c, kbase + off, ok);
      cp_async16(sV + (buf * DA_KT + r) * LD + c, vbase + off, ok);
    }
  };
  // 4-bit cache: one thread expands elements [c, c+8) and [c+half, c+half+8) of K and V of one key.
  // In two steps, so that a tile's codes, scales and ranks are already on their way while the
  // previous tile is multiplied: fetch_q4 requests them into registers (one tile ahead), expand_q4
  // reads the (cos, sin) rows of the units' positions, expands, rotates and fills the shared tile.
  constexpr int Q4_ITER = DA_KT * (D / 16) / DA_THREADS;
  static_assert(Q4_ITER * DA_THREADS == DA_KT * (D / 16), "whole iterations");
  struct Q4Pre { uint32_t kw0, kw1, vw0, vw1; float ks, vs; int pos; };  // pos < 0: not a unit of the 4-bit cache
  Q4Pre pre[INT4 ? Q4_ITER : 1];
  auto fetch_q4 = [&](int kt) {
    constexpr int HALF = D / 2, HV = D / 16;
#pragma unroll
    for (int i = 0; i < Q4_ITER; i++) {
      const int x = tid + i * DA_THREADS;
      const int r = x / HV, c = (x - r * HV) * 8;
      const int key = k0 + kt * DA_KT + r;
      pre[i].pos = -1;
      if (key < n - 1) {
        const size_t u = (size_t)m * cap + key;
        const uint8_t *kc = q4.kq + u * HALF, *vc = q4.vq + u * HALF;
        pre[i].kw0 = *reinterpret_cast<const uint32_t *>(kc + c / 2);
        pre[i].kw1 = *reinterpret_cast<const uint32_t *>(kc + (c + HALF) / 2);
        pre[i].vw0 = *reinterpret_cast<const uint32_t *>(vc + c / 2);
        pre[i].vw1 = *reinterpret_cast<const uint32_t *>(vc + (c + HALF) / 2);
        pre[i].ks = __half2float(q4.ks[u]);
        pre[i].vs = __half2float(q4.vs[u]);
        pre[i].pos = key < ranked_len ? rank[u] : key;  // the unit's place in temporal order
      }
    }
  };
  auto expand_q4 = [&](int buf, int kt) {
    constexpr int HALF = D / 2, HV = D / 16;
    float4 t4[Q4_ITER][4];   // 8 (cos, sin) pairs per item, all requested before any is used
#pragma unroll
    for (int i = 0; i < Q4_ITER; i++) {
      const int x = tid + i * DA_THREADS;
      const int c = (x - (x / HV) * HV) * 8;
      if (pre[i].pos >= 0) {
        const float4 *t = reinterpret_cast<const float4 *>(cs + (size_t)pre[i].pos * HALF + c);
#pragma unroll
        for (int e = 0; e < 4; e++) t4[i][e] = __ldg(t + e);
      }
    }
#pragma unroll
    for (int i = 0; i < Q4_ITER; i++) {
      const int x = tid + i * DA_THREADS;
      const int r = x / HV, c = (x - r * HV) * 8;
      const int key = k0 + kt * DA_KT + r;
      bf16 *kd = sK + (buf * DA_KT + r) * LD, *vd = sV + (buf * DA_KT + r) * LD;
      uint4 ka = make_uint4(0, 0, 0, 0), kb = ka, va = ka, vb = ka;
      if (pre[i].pos >= 0) {
        float a[8], b[8];
        dequant8(pre[i].kw0, pre[i].ks, a);
        dequant8(pre[i].kw1, pre[i].ks, b);
        const float2 *t = reinterpret_cast<const float2 *>(&t4[i][0]);
#pragma unroll
        for (int e = 0; e < 8; e++) {
          const float x1 = a[e], x2 = b[e];
          a[e] = x1 * t[e].x - x2 * t[e].y;
          b[e] = x2 * t[e].x + x1 * t[e].y;
        }
        ka = to_bf16x8(a); kb = to_bf16x8(b);
        dequant8(pre[i].vw0, pre[i].vs, a);
        dequant8(pre[i].vw1, pre[i].vs, b);
        va = to_bf16x8(a); vb = to_bf16x8(b);
      } else if (key >= n - 1 && key < k1) {  // the token of this step
        const size_t off = ((size_t)m * cap + key) * D + c;
        ka = *reinterpret_cast<const uint4 *>(k_rot + off); kb = *reinterpret_cast<const uint4 *>(k_rot + off + HALF);
        va = *reinterpret_cast<const uint4 *>(v + off); vb = *reinterpret_cast<const uint4 *>(v + off + HALF);
      }
      *reinterpret_cast<uint4 *>(kd + c) = ka; *reinterpret_cast<uint4 *>(kd + c + HALF) = kb;
      *reinterpret_cast<uint4 *>(vd + c) = va; *reinterpret_cast<uint4 *>(vd + c + HALF) = vb;
    }
  };
  // The retained keys and values were written by earlier steps: a first tile that does not reach
  // the token of this step is requested before the wait for this step's projection.
  const bool early = !INT4 && NKT > 0 && k0 + DA_KT <= n - 1;
  if (early) load_kv(0, 0);
  if (INT4 && NKT > 0) fetch_q4(0);   // (the token of this step is not among them: it is read in bf16, after the wait)
  pdl_wait();
  pdl_launch_dependents();  // the retaining head reads only what the projection wrote: it may run beside this kernel
  if (INT4 && tok_k && split == 0 && hg == 0 && warp < 2) {
    // The token of this step enters the 4-bit cache (this step still reads it in bf16): one warp
    // quantises its pre-RoPE key, one its value, with the arithmetic of the chunk kernel.
    const bf16 *src = (warp == 0 ? tok_k : tok_v) + (size_t)m * D;
    float x0[2], x1[2], amax = 0.f;
#pragma unroll
    for (int k = 0; k < 2; k++) {
      const int p = lane + 32 * k;
      x0[k] = x1[k] = 0.f;
      if (2 * p < D) {
        const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162 *>(src + 2 * p);
        x0[k] = __bfloat162float(v2.x);
        x1[k] = __bfloat162float(v2.y);
        amax = fmaxf(amax, fmaxf(fabsf(x0[k]), fabsf(x1[k])));
      }
    }
    amax = warp_max(amax);
    __half sh = __float2half_rn(__fdiv_rn(amax, 7.0f));
    if (__half2float(sh) == 0.f) sh = __float2half_rn(1.0f);
    const float sf = __half2float(sh);
    const size_t u = (size_t)m * cap + (n - 1);
    uint8_t *dst = (warp == 0 ? q4.kq : q4.vq) + u * (D / 2);
#pragma unroll
    for (int k = 0; k < 2; k++) {
      const int p = lane + 32 * k;
      if (2 * p < D) {
        const int c0 = (int)fminf(fmaxf(rintf(__fdiv_rn(x0[k], sf)), -8.f), 7.f);
        const int c1 = (int)fminf(fmaxf(rintf(__fdiv_rn(x1[k], sf)), -8.f), 7.f);
        dst[p] = (uint8_t)((c0 & 0xF) | ((c1 & 0xF) << 4));
      }
    }
    if (lane == 0) (warp == 0 ? q4.ks : q4.vs)[u] = sh;
  }
  for (int x = tid; x < DA_G * VPR; x += DA_THREADS) {
    const int r = x / VPR, c = (x - r * VPR) * 8;
    cp_async16(sQ + r * LD + c, q_rot + (size_t)(h0 + min(r, gh - 1)) * D + c, r < gh);
  }
  if (!INT4 && NKT > 0 && !early) load_kv(0, 0);
  cp_async_commit();

  uint32_t qf[D / 16][4];
  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; i++)
#pragma unroll
    for (int e = 0; e < 4; e++) o[i][e] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};  // heads g4 and g4 + 8

  for (int kt = 0; kt < NKT; kt++) {
    if (INT4) {
      expand_q4(kt & 1, kt);   // (the other buffer may still be read by a slower warp)
      if (kt + 1 < NKT) fetch_q4(kt + 1);
      cp_async_wait<0>();
    } else {
      if (kt + 1 < NKT) load_kv((kt + 1) & 1, kt + 1);
      cp_async_commit();
      cp_async_wait<1>();
    }
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int kk = 0; kk < D / 16; kk++)
        ldmatrix_x4(qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3],
                    sQ + (lane & 15) * LD + kk * 16 + (lane >> 4) * 8);
    }
    const bf16 *k_s = sK + ((kt & 1) * DA_KT + warp * 16) * LD;  // this warp's 16 keys
    const bf16 *v_s = sV + ((kt & 1) * DA_KT + warp * 16) * LD;

    float s[2][4];
#pragma unroll
    for (int i = 0; i < 2; i++)
#pragma unroll
      for (int e = 0; e < 4; e++) s[i][e] = 0.f;
#pragma unroll
    for (int kk = 0; kk < D / 16; kk++) {
      uint32_t b0, b1, b2, b3;
      const int id = lane >> 3;
      const int r = (id >> 1) * 8 + (lane & 7);
      const int c = kk * 16 + (id & 1) * 8;
      ldmatrix_x4(b0, b1, b2, b3, k_s + r * LD + c);
      mma_bf16_16816(s[0], qf[kk], b0, b1);
      mma_bf16_16816(s[1], qf[kk], b2, b3);
    }

    // scale, mask the keys past the split's end, online softmax of this warp's 16 keys
    const int key0 = k0 + kt * DA_KT + warp * 16;
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 2; i++)
#pragma unroll
      for (int e = 0; e < 4; e++) {
        float val = s[i][e] * scale_log2;
        if (key0 + i * 8 + q * 2 + (e & 1) >= k1) val = -INFINITY;
        s[i][e] = val;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], val);
      }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; r++) {
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
      const float mnew = fmaxf(mrow[r], tmax[r]);
      const float muse = (mnew == -INFINITY) ? 0.f : mnew;
      alpha[r] = exp2f(mrow[r] - muse);
      mrow[r] = mnew;
      float psum = 0.f;
#pragma unroll
      for (int i = 0; i < 2; i++) {
        const float p0 = exp2f(s[i][2 * r] - muse), p1 = exp2f(s[i][2 * r + 1] - muse);
        s[i][2 * r] = p0;
        s[i][2 * r + 1] = p1;
        psum += p0 + p1;
      }
      lrow[r] = lrow[r] * alpha[r] + psum;
    }
#pragma unroll
    for (int i = 0; i < D / 8; i++) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[0];
      o[i][2] *= alpha[1]; o[i][3] *= alpha[1];
    }
    // O += P V over this warp's 16 keys
    uint32_t pf[4];
    pf[0] = pack_bf16(s[0][0], s[0][1]);
    pf[1] = pack_bf16(s[0][2], s[0][3]);
    pf[2] = pack_bf16(s[1][0], s[1][1]);
    pf[3] = pack_bf16(s[1][2], s[1][3]);
#pragma unroll
    for (int dn = 0; dn < D / 16; dn++) {
      uint32_t b0, b1, b2, b3;
      const int id = lane >> 3;
      const int r = (id & 1) * 8 + (lane & 7);
      const int c = dn * 16 + (id >> 1) * 8;
      ldmatrix_x4_trans(b0, b1, b2, b3, v_s + r * LD + c);
      mma_bf16_16816(o[2 * dn], pf, b0, b1);
      mma_bf16_16816(o[2 * dn + 1], pf, b2, b3);
    }
    // bf16 cache: the next iteration's cp.async refills the buffer read here.  4-bit cache: the next
    // expansion fills the other buffer, and the one after it comes behind the next iteration's barrier.
    if (!INT4) __syncthreads();
  }
  cp_async_wait<0>();

  // ---- the four warps' states meet: fo[warp][head][column] in the tile buffers
#pragma unroll
  for (int r = 0; r < 2; r++) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
    if (q == 0) { wm[warp][g4 + 8 * r] = mrow[r]; wl[warp][g4 + 8 * r] = lrow[r]; }
  }
  float *fo = reinterpret_cast<float *>(sK);  // [4][16][D] floats = 32 KB at D = 128 <= the tile buffers
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; r++)
#pragma unroll
    for (int i = 0; i < D / 8; i++) {
      float2 val = make_float2(o[i][2 * r], o[i][2 * r + 1]);
      *reinterpret_cast<float2 *>(fo + ((size_t)(warp * DA_G + g4 + 8 * r)) * D + i * 8 + q * 2) = val;
    }
  __syncthreads();
  // partial result of this split: o [h][split][D] (not normalised), (m, l) [h][split][2]
  for (int idx = tid; idx < gh * D; idx += DA_THREADS) {
    const int i = idx / D, c = idx - i * D;
    const float mx = fmaxf(fmaxf(wm[0][i], wm[1][i]), fmaxf(wm[2][i], wm[3][i]));
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < 4; w++) {
      const float wgt = (wm[w][i] == -INFINITY) ? 0.f : exp2f(wm[w][i] - mx);
      acc = fmaf(wgt, fo[((size_t)(w * DA_G + i)) * D + c], acc);
      l = fmaf(wgt, wl[w][i], l);
    }
    const size_t hs = (size_t)(h0 + i) * n_splits + split;
    part_o[hs * D + c] = acc;
    if (c == 0) { part_ml[hs * 2] = mx; part_ml[hs * 2 + 1] = l; }
  }

  // ---- the split that finishes last merges the partial results of all splits
  __threadfence();
  __syncthreads();
  if (tid == 0) last = atomicInc(&counters[m * gridDim.z + hg], n_splits - 1) == (unsigned)(n_splits - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  for (int idx = tid; idx < gh * n_splits; idx += DA_THREADS) {
    const int i = idx / n_splits, s2 = idx - i * n_splits;
    const size_t hs = (size_t)(h0 + i) * n_splits + s2;
    sm[i][s2] = __ldcg(part_ml + hs * 2);
    sl[i][s2] = __ldcg(part_ml + hs * 2 + 1);
  }
  __syncthreads();
  // weights of the splits: one warp per head at a time, the splits across its lanes
  for (int i = warp; i < gh; i += DA_THREADS / 32) {
    float mx = -INFINITY;
    for (int s2 = lane; s2 < n_splits; s2 += 32) mx = fmaxf(mx, sm[i][s2]);
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));
    float l = 0.f;
    for (int s2 = lane; s2 < n_splits; s2 += 32) {
      const float ms = sm[i][s2];
      const float w = (ms == -INFINITY) ? 0.f : exp2f(ms - mx);
      l = fmaf(w, sl[i][s2], l);
      sm[i][s2] = w;
    }
    // (fixed order of the partial sums: lanes, then the butterfly)
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o2);
    if (lane == 0) sinv[i] = 1.0f / l;
  }
  __syncthreads();
  // thread = (head, four columns); sixteen splits in flight as 16-byte loads
  for (int item = tid; item < gh * (D / 4); item += DA_THREADS) {
    const int i = item / (D / 4), c = (item - i * (D / 4)) * 4;
    const float *po = part_o + (size_t)(h0 + i) * n_splits * D + c;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s2 = 0; s2 < n_splits; s2 += 16) {
      float4 a[16];
#pragma unroll
      for (int u = 0; u < 16; u++)
        a[u] = (s2 + u < n_splits) ? __ldcg(reinterpret_cast<const float4 *>(po + (size_t)(s2 + u) * D))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 16; u++)
        if (s2 + u < n_splits) {
          const float w = sm[i][s2 + u];
          acc.x = fmaf(w, a[u].x, acc.x); acc.y = fmaf(w, a[u].y, acc.y);
          acc.z = fmaf(w, a[u].z, acc.z); acc.w = fmaf(w, a[u].w, acc.w);
        }
    }
    const float inv = sinv[i];
    uint2 o2;
    o2.x = pack_bf16(acc.x * inv, acc.y * inv);
    o2.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(out + (size_t)(h0 + i) * D + c) = o2;
  }
}

}  // namespace

cudaError_t launch_gemv(const bf16 *x, const bf16 *Wt, int N, int K, bf16 *y, cudaStream_t st) {
  if (K % 8) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = min((N + 7) / 8, 148 * 4);
  gemv_kernel<0><<<blocks, GV_THREADS, smem, st>>>(x, Wt, N, K, y, nullptr, nullptr, 0, 0, nullptr, nullptr, 0,
                                                   nullptr);
  return cudaGetLastError();
}

// y[n] = x . Wt[n] + r[n]: a projection of one token with its residual connection
cudaError_t launch_gemv_resid(const bf16 *x, const bf16 *Wt, int N, int K, const bf16 *r, bf16 *y,
                              cudaStream_t st) {
  if (K % 8) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = min((N + 7) / 8, 148 * 4);
  gemv_kernel<0><<<blocks, GV_THREADS, smem, st>>>(x, Wt, N, K, y, nullptr, nullptr, 0, 0, nullptr, nullptr, 0, r);
  return cudaGetLastError();
}

// Gated FFN, first half, for one token: Wt [2F x K] holds, per block of 128 outputs, the 128
// rows of W_gate^T followed by the 128 rows of W_up^T; a warp computes one gate row and the
// matching up row and stores silu(gate) * up.
__global__ void __launch_bounds__(GV_THREADS)
gemv_gated_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ Wt, int F, int K, bf16 *__restrict__ act) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4 *sx = reinterpret_cast<uint4 *>(smem_raw);
  for (int i = threadIdx.x; i < K / 8; i += GV_THREADS) sx[i] = reinterpret_cast<const uint4 *>(x)[i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (GV_THREADS / 32) + warp, nw = gridDim.x * (GV_THREADS / 32);
  for (int c = gw; c < F; c += nw) {
    const size_t row = (size_t)(c / 128) * 256 + (c % 128);
    const uint4 *r0 = reinterpret_cast<const uint4 *>(Wt + row * K);
    const uint4 *r1 = reinterpret_cast<const uint4 *>(Wt + (row + 128) * K);
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int v = lane; v < K / 8; v += 32) {
      const uint4 xv = sx[v];
      s0 += dot8(__ldg(r0 + v), xv);
      s1 += dot8(__ldg(r1 + v), xv);
    }
    s0 = warp_sum(s0);
    s1 = warp_sum(s1);
    if (lane == 0) act[c] = __float2bfloat16_rn(s0 / (1.0f + __expf(-s0)) * s1);
  }
}
cudaError_t launch_gemv_gated(const bf16 *x, const bf16 *Wt, int F, int K, bf16 *act, cudaStream_t st) {
  if (K % 8) return cudaErrorInvalidValue;
  const int blocks = min((F + 7) / 8, 148 * 8);
  gemv_gated_kernel<<<blocks, GV_THREADS, K * 2, st>>>(x, Wt, F, K, act);
  return cudaGetLastError();
}

int rh_gemv_blocks(int d_R) { return min((d_R + 3) / 4, 148 * 4); }

cudaError_t launch_gemv_rope(const bf16 *x, const bf16 *Wt, int K, bf16 *staging, const RopeAppendArgs &a,
                             cudaStream_t st, bool pdl) {
  if (K % 8 || a.d % 2) return cudaErrorInvalidValue;
  const int items = (a.h + 2 * a.h_kv) * (a.d / 2);
  if (K / 8 <= GW_THREADS) {
    const int blocks = min((items + GW_PB - 1) / GW_PB, 148 * 2);
    return launch_kernel(gemv_rope_wide_kernel, dim3(blocks), dim3(GW_THREADS), 0, st, pdl, x, Wt, K, staging, a);
  }
  const int blocks = min((items + 7) / 8, 148 * 4);
  return launch_kernel(gemv_rope_kernel, dim3(blocks), dim3(GV_THREADS), (size_t)K * 2, st, pdl, x, Wt, K, staging, a);
}

// score_out: where the token's scores go (element m * score_stride for KV head m); counter: one
// zero-initialised word that the kernel leaves at zero
cudaError_t launch_rh_gemv(const bf16 *z, const bf16 *W1t, const float *W2, float *partial, int d_R, int K,
                           int h_kv, int act, unsigned *counter, float *score_out, int score_stride,
                           cudaStream_t st, bool pdl) {
  if (K % 16 || h_kv > 32) return cudaErrorInvalidValue;
  const int smem = K * 2 + 8 * 32 * 4;
  const int blocks = rh_gemv_blocks(d_R);
  return launch_kernel(gemv_kernel<1>, dim3(blocks), dim3(GV_THREADS), (size_t)smem, st, pdl, z, W1t, d_R, K,
                       (bf16 *)nullptr, W2, partial, h_kv, act, counter, score_out, score_stride,
                       (const bf16 *)nullptr);
}

// Splits of the key range per KV head.  Measured at the Llama shape (8 KV heads, 6000 keys, 256 steps through
// 32 layers): with a bf16 cache 64 / 96 / 120 / 148 / 200 / 296 / 444 CTAs in total give 914 / 1058 / 1130 /
// 1152 / 1224 / 1133 / 1052 tokens/s (more splits shorten each CTA's chain of tiles, but the last split of a
// head merges them all); a 4-bit cache, whose CTAs also expand and rotate the codes (and load a tile's codes
// without overlapping the previous tile's arithmetic), wants more: 96 / 148 / 296 / 444 CTAs give 501 / 639 /
// 825 / 700 tokens/s.
int decode_attn_splits(int h_kv, int n, bool int4) {
  static int forced = -1;
  if (forced < 0) { const char *e = getenv("LOCRET_DEC_CTAS"); forced = e ? atoi(e) : 0; if (forced < 0 || forced > 2048) forced = 0; }
  const int sms = sm_count_of_current_device();
  const int total = forced ? forced : (int4 ? 2 * sms : (sms * 27) / 20);
  int s = (total + h_kv - 1) / h_kv;
  const int max_s = (n + 127) / 128;            // at least one 128-key tile per split
  if (s > max_s) s = max_s;
  if (s > 64) s = 64;
  return s < 1 ? 1 : s;
}

cudaError_t launch_attention_decode(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out,
                                    float *part_o, float *part_ml, unsigned *counters, int h, int h_kv, int d,
                                    int cap, int n, int n_splits, const Int4Half *q4, const float2 *cs,
                                    const int32_t *rank, int ranked_len, const bf16 *tok_k, const bf16 *tok_v,
                                    cudaStream_t st, bool pdl) {
  const int g = h / h_kv;
  dim3 grid(h_kv, n_splits, (g + DA_G - 1) / DA_G);
  if ((int)grid.x * (int)grid.z > 32 * 16 || n_splits > 64) return cudaErrorInvalidValue;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  const Int4Half qq = q4 ? *q4 : Int4Half{nullptr, nullptr, nullptr, nullptr};
  auto launch = [&](auto kern, int smem, PerDeviceFlag &attr_set) -> cudaError_t {
    if (cudaError_t e = allow_dynamic_smem(kern, smem, attr_set); e != cudaSuccess) return e;
    return launch_kernel(kern, grid, dim3(DA_THREADS), (size_t)smem, st, pdl, q_rot, k_rot, v, part_o, part_ml, h, h_kv,
                         cap, n, n_splits, scale_log2, counters, out, qq, cs, rank, rank ? ranked_len : 0, tok_k, tok_v);
  };
  static PerDeviceFlag set_done[2][3];
  const int qi = q4 ? 1 : 0;
  switch (d) {
    case 64:
      return q4 ? launch(attn_decode_kernel<64, true>, (DA_G + 4 * DA_KT) * (64 + 8) * 2, set_done[qi][0])
                : launch(attn_decode_kernel<64, false>, (DA_G + 4 * DA_KT) * (64 + 8) * 2, set_done[qi][0]);
    case 96:
      return q4 ? launch(attn_decode_kernel<96, true>, (DA_G + 4 * DA_KT) * (96 + 8) * 2, set_done[qi][1])
                : launch(attn_decode_kernel<96, false>, (DA_G + 4 * DA_KT) * (96 + 8) * 2, set_done[qi][1]);
    case 128:
      return q4 ? launch(attn_decode_kernel<128, true>, (DA_G + 4 * DA_KT) * (128 + 8) * 2, set_done[qi][2])
                : launch(attn_decode_kernel<128, false>, (DA_G + 4 * DA_KT) * (128 + 8) * 2, set_done[qi][2]);
  }
  return cudaErrorInvalidValue;
}

}  // namespace locret
