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
  // the head's own cache length when the heads have budgets of their own (a query head uses its KV head's)
  const int kvh = hd < a.h ? hd / (a.h / a.h_kv) : (hd < a.h + a.h_kv ? hd - a.h : hd - a.h - a.h_kv);
  const int slot = (a.per_head ? a.len_m.v[kvh] : a.len) + t;
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
// Eviction leaves every kept unit in its slot and refills the freed slots below `budget` with the
// kept units that sit above it (Algorithm 1's gather, done in place): src_of[m][i] is the slot
// whose unit ends up in slot i (i itself for a unit that stays), rank_new[m][i] its position in
// temporal order afterwards.  One row group (d/8 threads) per (head, slot i < budget): a unit
// that comes from another slot is copied (K, V, score, token id); the rotated key is rewritten
// where the unit is new in the slot or its position has changed (Section 3.4: positions are
// re-assigned from the beginning).  Sources lie at or above `budget`, destinations below: no
// slot is both read and written by different rows.
// One thread holds the two halves of 8 rotation pairs: elements [c, c + 8) and [c + d/2, c + d/2 + 8)
// (each key element and each (cos, sin) is then loaded once per row; the table is as large as the
// keys it rotates).
__device__ __forceinline__ void rope_pairs8(const uint4 &lo, const uint4 &hi, const float2 *cs_pairs, uint4 &out_lo,
                                            uint4 &out_hi) {
  const bf16 *x1 = reinterpret_cast<const bf16 *>(&lo), *x2 = reinterpret_cast<const bf16 *>(&hi);
  bf16 *o1 = reinterpret_cast<bf16 *>(&out_lo), *o2 = reinterpret_cast<bf16 *>(&out_hi);
  const float4 *t4 = reinterpret_cast<const float4 *>(cs_pairs);  // two (cos, sin) per load
#pragma unroll
  for (int q = 0; q < 4; q++) {
    const float4 t = __ldg(t4 + q);
    const float a0 = __bfloat162float(x1[2 * q]), b0 = __bfloat162float(x2[2 * q]);
    const float a1 = __bfloat162float(x1[2 * q + 1]), b1 = __bfloat162float(x2[2 * q + 1]);
    o1[2 * q] = __float2bfloat16_rn(a0 * t.x - b0 * t.y);
    o2[2 * q] = __float2bfloat16_rn(b0 * t.x + a0 * t.y);
    o1[2 * q + 1] = __float2bfloat16_rn(a1 * t.z - b1 * t.w);
    o2[2 * q + 1] = __float2bfloat16_rn(b1 * t.z + a1 * t.w);
  }
}

// blockDim.x = d / 16 threads per row, blockDim.y rows per block.
__global__ void compact_kernel(CompactArgs a) {
  const int row = blockIdx.x * blockDim.y + threadIdx.y;
  if (row >= a.h_kv * a.src_stride) return;
  const int m = row / a.src_stride, i = row - m * a.src_stride;
  if (a.per_head ? (!a.evict_m.v[m] || i >= a.budget_m.v[m]) : i >= a.budget) return;
  const int ranked_len = a.per_head ? a.ranked_m.v[m] : a.ranked_len;
  const int rcur = a.per_head ? a.rcur_m.v[m] : a.rcur;
  const size_t u = (size_t)m * a.cap + i;
  const int src = a.src_of[(size_t)m * a.src_stride + i];
  const int pos = a.rank[rcur ^ 1][u];
  const int pos_old = i < ranked_len ? a.rank[rcur][u] : i;
  if (src == i && pos == pos_old) return;  // stays, and stays where it was in the order
  const int c = threadIdx.x * 8;
  const int half = a.d / 2;
  const size_t so = ((size_t)m * a.cap + src) * a.d, dof = u * a.d;
  const uint4 k_lo = *reinterpret_cast<const uint4 *>(a.k + so + c);
  const uint4 k_hi = *reinterpret_cast<const uint4 *>(a.k + so + c + half);
  if (src != i) {
    const uint4 v_lo = *reinterpret_cast<const uint4 *>(a.v + so + c);
    const uint4 v_hi = *reinterpret_cast<const uint4 *>(a.v + so + c + half);
    *reinterpret_cast<uint4 *>(a.k + dof + c) = k_lo;
    *reinterpret_cast<uint4 *>(a.k + dof + c + half) = k_hi;
    *reinterpret_cast<uint4 *>(a.v + dof + c) = v_lo;
    *reinterpret_cast<uint4 *>(a.v + dof + c + half) = v_hi;
    if (threadIdx.x == 0) {
      a.s[u] = a.s[(size_t)m * a.cap + src];
      a.t[u] = a.t[(size_t)m * a.cap + src];
    }
  }
  uint4 r_lo, r_hi;
  rope_pairs8(k_lo, k_hi, a.cs + (size_t)pos * half + c, r_lo, r_hi);
  *reinterpret_cast<uint4 *>(a.k_rot + dof + c) = r_lo;
  *reinterpret_cast<uint4 *>(a.k_rot + dof + c + half) = r_hi;
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
// One CTA per KV head.  Candidates: the units in slots [0, n).  A unit's place in temporal order is
// its rank (rank_old[slot] for slot < ranked_len, the slot itself above: units appended since the
// last eviction are in order).  Kept unconditionally: ranks [0, n_pre) (the protected prefix of
// the query-aware variant) and ranks [n - n_prot, n) (the stabilizers of Algorithm 1); among the
// rest the k = budget - n_prot - n_pre best by (score descending, rank descending).
//   1. radix select (4 passes of 8 bits) on an order-preserving 32-bit image of the score finds
//      the k-th largest value tau; only if more units equal tau than may stay, a second radix
//      select over their ranks finds the rank from which on they stay (the most recent ones);
//   2. a bitmap of the kept slots and a bitmap of the evicted RANKS; prefix sums over their words;
//   3. every kept unit's new rank is its old one minus the evicted ranks below it; kept units in
//      slots >= budget go, in slot order, to the freed slots below budget, in slot order.
// Output: src_of[m][i] and rank_new[m][i] for every slot i < budget (see compact_kernel).
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

// The need-th largest value of val(i) over the slots i < n with in(i): 4 passes of 8 bits, most
// significant first.  Returns the value; *need_out = how many units EQUAL to it belong to the
// `need` largest.  Requires 1 <= need <= number of units with in(i).
template <typename In, typename Val>
__device__ __forceinline__ uint32_t radix_select(int n, int need, In in, Val val, int *hist2, uint32_t *s_prefix,
                                                 int *s_need, int *need_out) {
  // hist2: two histograms of 256 bins used alternately; the idle one is cleared while warp 0 locates
  // the bin of the current one, so a pass costs two block-wide barriers.  Both are clear on entry
  // and on return.
  const int tid = threadIdx.x;
  uint32_t prefix = 0, mask = 0;
  int pass = 0;
  for (int shift = 24; shift >= 0; shift -= 8, pass++) {
    int *hist = hist2 + (pass & 1) * 256, *other = hist2 + ((pass & 1) ^ 1) * 256;
    // warp-aggregated histogram: lanes that hit the same bin elect one atomic
    for (int i0 = 0; i0 < n; i0 += TK_THREADS) {
      const int i = i0 + tid;
      uint32_t key = 0;
      bool hit = false;
      if (i < n && in(i)) {
        key = val(i);
        hit = (key & mask) == prefix;
      }
      const unsigned active = __ballot_sync(0xffffffffu, hit);
      if (hit) {
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
        *s_prefix = prefix | ((uint32_t)(tid * 8 + b) << shift);
        *s_need = need - acc;
      }
#pragma unroll
      for (int b = 0; b < 8; b++) hist[tid * 8 + b] = 0;  // (read above by this lane only)
    } else if (tid >= 256 && tid < 512) {
      other[tid - 256] = 0;
    }
    __syncthreads();
    prefix = *s_prefix;
    need = *s_need;
    mask |= 255u << shift;
  }
  __syncthreads();  // s_prefix / s_need may be overwritten by the next call only after everybody has read them
  *need_out = need;
  return prefix;
}

// Exclusive prefix sums of three counters at once (one pass of the block scan for all three).
__device__ __forceinline__ void block_exclusive_scan3(int (&val)[3], int (*warp_sums3)[33]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc[3] = {val[0], val[1], val[2]};
#pragma unroll
  for (int o = 1; o < 32; o <<= 1)
#pragma unroll
    for (int q = 0; q < 3; q++) {
      const int y = __shfl_up_sync(0xffffffffu, inc[q], o);
      if (lane >= o) inc[q] += y;
    }
  __syncthreads();
  if (lane == 31)
#pragma unroll
    for (int q = 0; q < 3; q++) warp_sums3[q][warp] = inc[q];
  __syncthreads();
  if (warp < 3) {
    const int w = warp_sums3[warp][lane];
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    warp_sums3[warp][lane] = winc - w;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 3; q++) val[q] = warp_sums3[q][warp] + inc[q] - val[q];
}

__global__ void __launch_bounds__(TK_THREADS)
topk_kernel(TopkArgs a, int cache_in_smem) {
  // dynamic shared memory: five bitmap / prefix arrays of W = ceil(n / 32) words, then (when it
  // fits) the keys and ranks of all n slots
  extern __shared__ uint32_t tk_smem[];
  __shared__ int hist[512];
  __shared__ int warp_sums[33];
  __shared__ int warp_sums3[3][33];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;
  __shared__ int s_total_eq;

  const int m = blockIdx.x, tid = threadIdx.x;
  const int n = a.per_head ? a.n_m.v[m] : a.n, budget = a.per_head ? a.budget_m.v[m] : a.budget;
  if (n <= budget) return;  // (a budget per head: this head keeps everything in this step)
  const int W = (n + 31) / 32;
  uint32_t *keptbits = tk_smem;          // bit s: slot s is kept
  uint32_t *evbits = tk_smem + W;        // bit r: the unit of rank r is evicted
  int *kept_pref = reinterpret_cast<int *>(tk_smem + 2 * W);   // per word: freed slots below budget before it
  int *ev_pref = reinterpret_cast<int *>(tk_smem + 3 * W);     // per word: evicted ranks before it
  uint32_t *skeys = tk_smem + 5 * W;
  int32_t *sranks = reinterpret_cast<int32_t *>(tk_smem + 5 * W + n);

  const float *sc = a.scores + (size_t)m * a.stride;
  const int rcur = a.per_head ? a.rcur_m.v[m] : a.rcur;
  const int32_t *rk = a.rank[rcur] + (size_t)m * a.stride;
  int32_t *src_of = a.src_of + (size_t)m * a.src_stride;
  int32_t *rank_new = a.rank[rcur ^ 1] + (size_t)m * a.stride;
  const int ranked_len = a.per_head ? a.ranked_m.v[m] : a.ranked_len;
  const int n_prot = a.per_head ? a.nprot_m.v[m] : a.n_prot;
  const int lo_rank = a.n_pre, hi_rank = n - n_prot;   // ranks [lo_rank, hi_rank) compete
  const int k = budget - n_prot - a.n_pre;              // 0 <= k < hi_rank - lo_rank (n > budget)

  auto key_at = [&](int i) -> uint32_t { return cache_in_smem ? skeys[i] : score_key(sc[i]); };
  auto rank_at = [&](int i) -> int { return cache_in_smem ? sranks[i] : (i < ranked_len ? rk[i] : i); };
  auto competes = [&](int i) -> bool { const int r = rank_at(i); return r >= lo_rank && r < hi_rank; };

  if (cache_in_smem)
    for (int i = tid; i < n; i += TK_THREADS) {
      skeys[i] = score_key(sc[i]);
      sranks[i] = i < ranked_len ? rk[i] : i;
    }
  for (int w = tid; w < W; w += TK_THREADS) evbits[w] = 0;
  if (tid < 512) hist[tid] = 0;
  if (tid == 0) s_total_eq = 0;
  __syncthreads();

  // ---- 1. the cut: tau, and the rank from which on units equal to tau stay
  uint32_t tau = 0, rank_cut = 0;
  if (k > 0) {
    int need_eq;
    tau = radix_select(n, k, competes, key_at, hist, &s_prefix, &s_need, &need_eq);
    int cnt = 0;
    for (int i = tid; i < n; i += TK_THREADS) cnt += competes(i) && key_at(i) == tau;
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if ((tid & 31) == 0 && cnt) atomicAdd(&s_total_eq, cnt);
    __syncthreads();
    const int total_eq = s_total_eq;
    if (total_eq > need_eq) {  // (uniform over the block) ties at the cut: the most recent stay
      int dummy;
      rank_cut = radix_select(n, need_eq, [&](int i) { return competes(i) && key_at(i) == tau; },
                              [&](int i) { return (uint32_t)rank_at(i); }, hist, &s_prefix, &s_need, &dummy);
    }
  }

  // ---- 2. kept slots and evicted ranks
  for (int i0 = 0; i0 < W * 32; i0 += TK_THREADS) {
    const int i = i0 + tid;
    bool kp = false;
    if (i < n) {
      const int r = rank_at(i);
      if (r < lo_rank || r >= hi_rank) kp = true;
      else if (k > 0) {
        const uint32_t key = key_at(i);
        kp = key > tau || (key == tau && (uint32_t)r >= rank_cut);
      }
      if (!kp) atomicOr(&evbits[r >> 5], 1u << (r & 31));
    }
    const unsigned b = __ballot_sync(0xffffffffu, kp);
    if ((tid & 31) == 0 && (i >> 5) < W) keptbits[i >> 5] = b;
  }
  __syncthreads();

  // per word: evicted ranks before it; freed slots below budget before it
  auto hole_bits = [&](int w) -> uint32_t {   // evicted slots of word w that lie below budget
    const int s0 = w * 32;
    if (s0 >= budget) return 0u;
    uint32_t valid = budget - s0 >= 32 ? 0xffffffffu : ((1u << (budget - s0)) - 1u);
    return ~keptbits[w] & valid;
  };
  auto mover_bits = [&](int w) -> uint32_t {  // kept slots of word w at or above budget
    const int s0 = w * 32;
    if (s0 + 32 <= budget) return 0u;
    uint32_t valid = s0 >= budget ? 0xffffffffu : ~((1u << (budget - s0)) - 1u);
    return keptbits[w] & valid;
  };
  int *mover_pref = reinterpret_cast<int *>(keptbits) + 4 * W;  // (a fifth array of W words, see the launcher)
  {
    const int per = (W + TK_THREADS - 1) / TK_THREADS;
    const int w0 = min(tid * per, W), w1 = min(w0 + per, W);
    int c3[3] = {0, 0, 0};
    for (int w = w0; w < w1; w++) {
      c3[0] += __popc(evbits[w]); c3[1] += __popc(hole_bits(w)); c3[2] += __popc(mover_bits(w));
    }
    block_exclusive_scan3(c3, warp_sums3);
    for (int w = w0; w < w1; w++) {
      ev_pref[w] = c3[0]; c3[0] += __popc(evbits[w]);
      kept_pref[w] = c3[1]; c3[1] += __popc(hole_bits(w));
      mover_pref[w] = c3[2]; c3[2] += __popc(mover_bits(w));
    }
  }
  __syncthreads();
  // the freed slots below budget, in slot order, parked in rank_new[budget ...) (slots the step leaves unused)
  int32_t *holes = rank_new + budget;
  for (int w = tid; w < W; w += TK_THREADS) {
    uint32_t hb = hole_bits(w);
    int at = kept_pref[w];
    while (hb) {
      const int b = __ffs(hb) - 1;
      hb &= hb - 1;
      holes[at++] = w * 32 + b;
    }
  }
  __syncthreads();   // (block-wide: the holes were written to global memory by other threads of this block)

  // ---- 3. where every kept unit ends up, and at which position
  int moved = 0, rotated = 0;
  for (int i = tid; i < n; i += TK_THREADS) {
    const int w = i >> 5, bit = i & 31;
    if (!((keptbits[w] >> bit) & 1u)) continue;
    const int r = rank_at(i);
    const int below = ev_pref[r >> 5] + __popc(evbits[r >> 5] & ((1u << (r & 31)) - 1u));
    const int r_new = r - below;
    int dst = i;
    if (i >= budget) {
      const int idx = mover_pref[w] + __popc(mover_bits(w) & ((1u << bit) - 1u));
      dst = __ldcg(holes + idx);
      moved++;
    }
    src_of[dst] = i;
    // (rank_new[dst] for dst < budget; the parked hole list lies at or above budget)
    rank_new[dst] = r_new;
    rotated += (dst != i) || (r_new != r);
  }
  if (a.counters) {
    moved = __reduce_add_sync(0xffffffffu, moved);
    rotated = __reduce_add_sync(0xffffffffu, rotated);
    if ((tid & 31) == 0) {
      if (moved) atomicAdd(&a.counters[0], (unsigned long long)moved);
      if (rotated) atomicAdd(&a.counters[1], (unsigned long long)rotated);
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
  const int tpr = a.d / 16, rpb = 256 / tpr;  // threads per row, rows per block
  const int rows = a.h_kv * a.src_stride;
  compact_kernel<<<(rows + rpb - 1) / rpb, dim3(tpr, rpb), 0, st>>>(a);
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

size_t topk_smem_bytes(int n, bool cached) {
  const size_t W = (size_t)(n + 31) / 32;
  return (5 * W + (cached ? 2 * (size_t)n : 0)) * 4;
}

cudaError_t launch_topk(const TopkArgs &a, int h_kv, cudaStream_t st) {
  const size_t max_dyn = 200 * 1024;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(topk_kernel, (int)max_dyn, attr_set); e != cudaSuccess) return e;
  int n_max = a.n;
  if (a.per_head) {
    n_max = 0;
    for (int m = 0; m < h_kv; m++) n_max = a.n_m.v[m] > n_max ? a.n_m.v[m] : n_max;
  }
  const int cached = topk_smem_bytes(n_max, true) <= max_dyn;
  const size_t bytes = topk_smem_bytes(n_max, cached);
  if (bytes > max_dyn || n_max > a.stride) return cudaErrorInvalidValue;
  topk_kernel<<<h_kv, TK_THREADS, bytes, st>>>(a, cached);
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
