// Memory-bound kernels of the step: position assignment + RoPE + append, per-head
// top-b selection, gather/compaction with re-RoPE, and small utilities.
#include "common.cuh"

namespace locret {

namespace {

// ---------------------------------------------------------------- RoPE helpers
// One thread holds 8 consecutive elements [c, c+8) of a head vector and the 8 partner
// elements at c ± d/2.  Rotate-half pairing: (i, i + d/2), angle pos · theta^(−2i/d).
struct Vec8 {
  uint4 raw;
  __device__ __forceinline__ float get(int i) const {
    const bf16 *p = reinterpret_cast<const bf16 *>(&raw);
    return __bfloat162float(p[i]);
  }
};

__device__ __forceinline__ uint4 rope8(const Vec8 &self, const Vec8 &partner, const float2 *cs_row,
                                       int c, int half) {
  // cs_row: (cos, sin) of this position for pair index 0..half-1
  const bool lower = c < half;
  const int p0 = lower ? c : c - half;
  uint4 out;
  bf16 *o = reinterpret_cast<bf16 *>(&out);
#pragma unroll
  for (int i = 0; i < 8; i++) {
    float2 t = cs_row[p0 + i];
    float x = self.get(i), y = partner.get(i);
    // lower half: x1 cos − x2 sin ; upper half: x2 cos + x1 sin
    float r = lower ? (x * t.x - y * t.y) : (x * t.x + y * t.y);
    o[i] = __float2bfloat16_rn(r);
  }
  return out;
}

// ---------------------------------------------------------------- rope + append
// grid: (n_tok, h + 2 h_kv) rows of d elements; blockDim = d / 8 threads per row, several rows
// per block through threadIdx.y.
__global__ void rope_append_kernel(RopeAppendArgs a) {
  const int vpr = a.d / 8;
  const int row = blockIdx.x * blockDim.y + threadIdx.y;  // over n_tok * (h + 2 h_kv)
  const int heads = a.h + 2 * a.h_kv;
  if (row >= a.n_tok * heads) return;
  const int t = row / heads, hd = row - t * heads;
  const int c = threadIdx.x * 8;
  const int half = a.d / 2;
  const int d_in = heads * a.d;
  const bf16 *src = a.staging + (size_t)t * d_in + (size_t)hd * a.d;
  Vec8 self, partner;
  self.raw = *reinterpret_cast<const uint4 *>(src + c);
  const int slot = a.len + t;
  const float2 *cs_row = a.cs + (size_t)slot * half;
  if (hd < a.h + a.h_kv) {
    partner.raw = *reinterpret_cast<const uint4 *>(src + (c < half ? c + half : c - half));
    uint4 rot = rope8(self, partner, cs_row, c, half);
    if (hd < a.h) {
      *reinterpret_cast<uint4 *>(a.q_rot + (size_t)t * a.h * a.d + (size_t)hd * a.d + c) = rot;
    } else {
      const int m = hd - a.h;
      size_t off = ((size_t)m * a.cap + slot) * a.d + c;
      if (a.k_pre) *reinterpret_cast<uint4 *>(a.k_pre + off) = self.raw;  // null for a 4-bit cache
      *reinterpret_cast<uint4 *>(a.k_rot + off) = rot;
      if (threadIdx.x == 0) a.tid[(size_t)m * a.cap + slot] = a.seen + t;
    }
    if (a.z_post) *reinterpret_cast<uint4 *>(a.z_post + (size_t)t * d_in + (size_t)hd * a.d + c) = rot;
  } else {
    const int m = hd - a.h - a.h_kv;
    *reinterpret_cast<uint4 *>(a.v + ((size_t)m * a.cap + slot) * a.d + c) = self.raw;
    if (a.z_post)
      *reinterpret_cast<uint4 *>(a.z_post + (size_t)t * d_in + (size_t)hd * a.d + c) = self.raw;
  }
  (void)vpr;
}

// ---------------------------------------------------------------- compaction
// One row group (d/8 threads) per (head, new slot i): src = keep[m][i].
__global__ void compact_kernel(CompactArgs a) {
  const int row = blockIdx.x * blockDim.y + threadIdx.y;
  if (row >= a.h_kv * a.budget) return;
  const int m = row / a.budget, i = row - m * a.budget;
  const int src = a.keep[(size_t)m * a.budget + i];
  const int c = threadIdx.x * 8;
  const int half = a.d / 2;
  const size_t so = ((size_t)m * a.cap + src) * a.d, dof = ((size_t)m * a.cap + i) * a.d;
  Vec8 self, partner;
  self.raw = *reinterpret_cast<const uint4 *>(a.k_src + so + c);
  uint4 vv = *reinterpret_cast<const uint4 *>(a.v_src + so + c);
  *reinterpret_cast<uint4 *>(a.k_dst + dof + c) = self.raw;
  *reinterpret_cast<uint4 *>(a.v_dst + dof + c) = vv;
  if (src != i) {  // an unmoved unit keeps its position, so its rotated key is already right
    partner.raw = *reinterpret_cast<const uint4 *>(a.k_src + so + (c < half ? c + half : c - half));
    *reinterpret_cast<uint4 *>(a.k_rot + dof + c) =
        rope8(self, partner, a.cs + (size_t)i * half, c, half);
  }
  if (threadIdx.x == 0) {
    a.s_dst[(size_t)m * a.cap + i] = a.s_src[(size_t)m * a.cap + src];
    a.t_dst[(size_t)m * a.cap + i] = a.t_src[(size_t)m * a.cap + src];
  }
}

__global__ void rerope_kernel(const bf16 *k_pre, bf16 *k_rot, const float2 *cs, int h_kv, int d,
                              int cap, int len) {
  const int row = blockIdx.x * blockDim.y + threadIdx.y;
  if (row >= h_kv * len) return;
  const int m = row / len, i = row - m * len;
  const int c = threadIdx.x * 8, half = d / 2;
  const size_t off = ((size_t)m * cap + i) * d;
  Vec8 self, partner;
  self.raw = *reinterpret_cast<const uint4 *>(k_pre + off + c);
  partner.raw = *reinterpret_cast<const uint4 *>(k_pre + off + (c < half ? c + half : c - half));
  *reinterpret_cast<uint4 *>(k_rot + off + c) = rope8(self, partner, cs + (size_t)i * half, c, half);
}

// ---------------------------------------------------------------- top-b selection
// One CTA per KV head.  Candidates: slots [0, n); the last n_prot are kept unconditionally;
// among rest = [0, n − n_prot) keep the k = budget − n_prot best by (score desc, slot desc).
// Radix select (4 passes of 8 bits) on an order-preserving 32-bit image of the score finds
// the k-th largest value tau; everything above tau is kept, and of the units equal to tau the
// most recent ones fill the remainder.  Kept slots are written in ascending order.
constexpr int TK_THREADS = 1024;

__device__ __forceinline__ uint32_t score_key(float x) {
  if (x != x) x = -INFINITY;   // NaN ranks as −inf
  if (x == 0.f) x = 0.f;       // −0 and +0 are the same score
  uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ int block_exclusive_scan(int val, int *warp_sums, int *total) {
  // blockDim.x == TK_THREADS; returns exclusive prefix of val over threads
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = val;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  __syncthreads();  // warp_sums may still be read from a previous call
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    warp_sums[lane] = winc - w;  // exclusive prefix of warp sums
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *total = warp_sums[32];
  return warp_sums[warp] + inc - val;
}

__global__ void __launch_bounds__(TK_THREADS)
topk_kernel(const float *__restrict__ scores, int score_stride, int n, int budget, int n_prot, int n_pre,
            int32_t *__restrict__ keep, int smem_keys) {
  extern __shared__ uint32_t skeys[];  // [rest] when it fits (smem_keys != 0)
  __shared__ int hist[256];
  __shared__ int warp_sums[33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;

  const int m = blockIdx.x;
  const float *sc = scores + (size_t)m * score_stride;
  int32_t *out = keep + (size_t)m * budget;
  const int tid = threadIdx.x;
  const int rest = n - n_prot;
  // slots [0, n_pre) and [rest, n) are kept unconditionally; k of the slots between them are chosen
  const int k = budget - n_prot - n_pre;  // 0 <= k < rest - n_pre (the caller guarantees n > budget)

  auto key_at = [&](int i) -> uint32_t { return smem_keys ? skeys[i] : score_key(sc[i]); };

  if (smem_keys)
    for (int i = tid; i < rest; i += TK_THREADS) skeys[i] = score_key(sc[i]);

  // ---- radix select of the k-th largest key among rest (k >= 1)
  uint32_t prefix = 0, mask = 0;
  int need = k;
  if (k > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      // warp-aggregated histogram: lanes that hit the same bin elect one atomic
      for (int i0 = 0; i0 < rest; i0 += TK_THREADS) {
        const int i = i0 + tid;
        uint32_t key = 0;
        bool in = false;
        if (i < rest) {
          key = key_at(i);
          in = i >= n_pre && (key & mask) == prefix;
        }
        const unsigned active = __ballot_sync(0xffffffffu, in);
        if (in) {
          const uint32_t bin = (key >> shift) & 255u;
          const unsigned peers = __match_any_sync(active, bin);
          if ((tid & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
        }
      }
      __syncthreads();
      if (tid < 32) {
        // lane l owns bins [8l, 8l+8); suffix sums over lanes locate the bin of the need-th key
        int loc[8], sum = 0;
#pragma unroll
        for (int b = 0; b < 8; b++) { loc[b] = hist[tid * 8 + b]; sum += loc[b]; }
        int above = 0;  // keys in the bins of higher lanes
#pragma unroll
        for (int l2 = 0; l2 < 32; l2++) {
          const int v = __shfl_sync(0xffffffffu, sum, l2);
          if (l2 > (int)tid) above += v;
        }
        const bool mine = (above < need) && (above + sum >= need);
        if (mine) {
          int acc = above, b = 7;
          for (; b > 0; b--) {
            if (acc + loc[b] >= need) break;
            acc += loc[b];
          }
          s_prefix = prefix | ((uint32_t)(tid * 8 + b) << shift);
          s_need = need - acc;
        }
      }
      __syncthreads();
      prefix = s_prefix;
      need = s_need;
      mask |= 255u << shift;
      __syncthreads();
    }
  }
  const uint32_t tau = prefix;  // need = how many units equal to tau are kept (the most recent)

  // ---- contiguous segment per thread, so that output order is slot order
  const int per = (n + TK_THREADS - 1) / TK_THREADS;
  const int lo = min(tid * per, n), hi = min(lo + per, n);
  int cnt_eq = 0;
  if (k > 0)
    for (int i = max(lo, n_pre); i < hi && i < rest; i++) cnt_eq += (key_at(i) == tau);
  int total_eq;
  int eq_before = block_exclusive_scan(cnt_eq, warp_sums, &total_eq);
  const int eq_skip = total_eq - need;  // equal units with rank-from-start < eq_skip are dropped

  int cnt_keep = 0;
  {
    int eqr = eq_before;
    for (int i = lo; i < hi; i++) {
      bool kp;
      if (i >= rest || i < n_pre) kp = true;
      else if (k == 0) kp = false;
      else {
        uint32_t key = key_at(i);
        kp = key > tau;
        if (key == tau) { kp = eqr >= eq_skip; eqr++; }
      }
      cnt_keep += kp;
    }
  }
  int total_keep;
  int pos = block_exclusive_scan(cnt_keep, warp_sums, &total_keep);
  {
    int eqr = eq_before;
    for (int i = lo; i < hi; i++) {
      bool kp;
      if (i >= rest || i < n_pre) kp = true;
      else if (k == 0) kp = false;
      else {
        uint32_t key = key_at(i);
        kp = key > tau;
        if (key == tau) { kp = eqr >= eq_skip; eqr++; }
      }
      if (kp) { if (pos < budget) out[pos] = i; pos++; }
    }
  }
}

// ---------------------------------------------------------------- utilities
__global__ void transpose_bf16_kernel(const bf16 *__restrict__ src, bf16 *__restrict__ dst, int rows,
                                      int cols) {
  __shared__ bf16 tile[32][33];
  int c = blockIdx.x * 32 + threadIdx.x;
  for (int r = threadIdx.y; r < 32; r += 8) {
    int rr = blockIdx.y * 32 + r;
    if (rr < rows && c < cols) tile[r][threadIdx.x] = src[(size_t)rr * cols + c];
  }
  __syncthreads();
  int rr = blockIdx.y * 32 + threadIdx.x;
  for (int r = threadIdx.y; r < 32; r += 8) {
    int cc = blockIdx.x * 32 + r;
    if (rr < rows && cc < cols) dst[(size_t)cc * rows + rr] = tile[threadIdx.x][r];
  }
}

__global__ void bf16_to_f32_kernel(const bf16 *src, float *dst, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = __bfloat162float(src[i]);
}

inline dim3 row_block(int d, int *rows_per_block) {
  int vpr = d / 8;
  int rpb = 256 / vpr;
  *rows_per_block = rpb;
  return dim3(vpr, rpb);
}

}  // namespace

cudaError_t launch_rope_append(const RopeAppendArgs &a, cudaStream_t st) {
  int rpb;
  dim3 blk = row_block(a.d, &rpb);
  int rows = a.n_tok * (a.h + 2 * a.h_kv);
  rope_append_kernel<<<(rows + rpb - 1) / rpb, blk, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_compact(const CompactArgs &a, cudaStream_t st) {
  int rpb;
  dim3 blk = row_block(a.d, &rpb);
  int rows = a.h_kv * a.budget;
  compact_kernel<<<(rows + rpb - 1) / rpb, blk, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_rerope(const bf16 *k_pre, bf16 *k_rot, const float2 *cs, int h_kv, int d, int cap,
                          int len, cudaStream_t st) {
  if (len == 0) return cudaSuccess;
  int rpb;
  dim3 blk = row_block(d, &rpb);
  int rows = h_kv * len;
  rerope_kernel<<<(rows + rpb - 1) / rpb, blk, 0, st>>>(k_pre, k_rot, cs, h_kv, d, cap, len);
  return cudaGetLastError();
}

cudaError_t launch_topk(const float *scores, int score_stride, int h_kv, int n, int budget,
                        int n_prot, int n_pre, int32_t *keep, cudaStream_t st) {
  const int rest = n - n_prot;
  const size_t bytes = (size_t)rest * 4;
  const size_t max_dyn = 200 * 1024;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(topk_kernel, (int)max_dyn, attr_set); e != cudaSuccess) return e;
  int use_smem = bytes <= max_dyn;
  topk_kernel<<<h_kv, TK_THREADS, use_smem ? bytes : 0, st>>>(scores, score_stride, n, budget, n_prot,
                                                              n_pre, keep, use_smem);
  return cudaGetLastError();
}

cudaError_t launch_transpose_bf16(const bf16 *src, bf16 *dst, int rows, int cols, cudaStream_t st) {
  dim3 grid((cols + 31) / 32, (rows + 31) / 32);
  transpose_bf16_kernel<<<grid, dim3(32, 8), 0, st>>>(src, dst, rows, cols);
  return cudaGetLastError();
}

cudaError_t launch_bf16_to_f32(const bf16 *src, float *dst, int n, cudaStream_t st) {
  bf16_to_f32_kernel<<<(n + 255) / 256, 256, 0, st>>>(src, dst, n);
  return cudaGetLastError();
}

}  // namespace locret
