// Eq. 1 on tcgen05 tensor cores with TMEM accumulators, head_dim 64, 96 or 128 (tiles are laid
// out for 128 columns; narrower heads load and multiply only their own columns).
//
// One CTA owns two 128-row query tiles that share a KV head (two query heads of one GQA
// group over the same rows, or two consecutive row blocks of one head) and streams the
// keys/values of that head in tiles of 128 through shared memory with TMA.  Roles:
//   warps 0-7        softmax, one query tile at a time (tile 0 and tile 1 alternately, so one
//                    tile's softmax runs while the other tile's MMAs execute).  A warp may only
//                    touch TMEM lanes 32 (w % 4) .. +31, so warps q and 4 + q share the 32 rows of
//                    quarter q and split the tile's 128 keys in halves: each thread reads half a
//                    row of S = Q K^T from TMEM, the pair exchanges its half maxima through shared
//                    memory, and each writes P = exp2(S - max) as bf16 back into TMEM over S (the
//                    first half releases the first four k-steps of P V, the second the rest).
//                    The accumulator is rescaled in TMEM only when the maximum has grown by more
//                    than 2^100.
//   warp 8           TMA producer: Q once, then K and V tiles (two stages each), walking the
//                    unmasked key tiles in a per-CTA rotated order, with an L2 prefetch ahead;
//   warps 9 / 10     issue S_t = Q_t K_j^T (both operands in shared memory) and O_t += P_t V_j
//                    (P from TMEM, V from shared memory) for tile 0 / 1.  The tensor pipe accepts
//                    only about two instructions ahead of execution, so each issuer builds its
//                    descriptors once and advances them by constants, and the other issuer's MMAs
//                    cover the time one spends polling a barrier.
// TMEM columns: S0/P0 [0,128), S1/P1 [128,256), O0 [256,384), O1 [384,512).
// Query row t sees keys [0, len + t]: the retained cache unmasked, the chunk causally.
#include <stdlib.h>

#include "tc_common.cuh"

namespace locret {

namespace {

using namespace tc;

constexpr int AT_THREADS = 384;  // 3 warpgroups: softmax (two), {TMA, 2 MMA issuers, 1 idle warp}
constexpr int TILE = 128;               // query rows per tile and keys per tile
constexpr int HD = 128;                 // column pitch of a head in shared and tensor memory
constexpr int HALF_BYTES = TILE * 128;  // one 64-column swizzled box of 128 rows: 16 KB
constexpr int TILE_BYTES = 2 * HALF_BYTES;
constexpr int AT_SMEM = 1024 + 6 * TILE_BYTES + 256 + 2048 + 256;  // Q0,Q1,K0,K1,V0,V1 + barriers + softmax exchange + work-list state
// The accumulator is rescaled only when a row's maximum has grown by more than 2^100 since the
// scale in use was fixed.  P is stored as bf16 and O, l accumulate in fp32, both with an 8-bit
// exponent, so P <= 2^100 and O <= keys * 2^100 * |v| (< 2^122 for 2^14 keys, |v| < 2^8) stay
// finite, and relative precision does not depend on the common scale.  A small threshold would
// trigger a rescale (a TMEM round trip on the critical path) at almost every tile that holds one
// of the workload's 20x-norm outlier keys.
constexpr float RESCALE_LOG2 = 100.0f;
constexpr int PF = 6;       // key tiles prefetched into L2 ahead of the shared-memory pipeline

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

struct AttnParams {
  bf16 *out;
  int n_tok, h, h_kv, d, len, pair_heads;
  float scale_log2;
  int *status;
  // ---- division of the work (see the kernel's comment)
  int n_groups;        // groups of items with the same number of key tiles, longest first
  int group_items;     // items per group
  int n_items;
  int total_steps;     // sum over all items of their key tiles
  float *part_o;       // [2 * units][2 tiles][TILE rows][D]  unnormalised partial outputs
  float *part_ml;      // [2 * units][2 tiles][2][TILE rows]  their running maximum (log2 scale) and sum
  unsigned *item_cnt;  // [n_items] finished pieces of a divided item; zero between launches
};

// ---- the work list.  An ITEM is what one CTA of an undivided launch would do: two 128-row query
// tiles that share a KV head, against all the key tiles they see.  Items of one row block form a
// GROUP (same number of key tiles); groups are ordered longest first.  Key steps of all items,
// in item order, form one line of `total_steps` steps, and CTA u of U takes the steps
// [u S / U, (u + 1) S / U): a few SEGMENTS, each a range [k0, k1) of one item's key steps.  With U
// a multiple of the number of SMs every SM gets the same number of key steps, whatever the
// lengths of the items (a launch of whole items leaves 13 % of the SM time idle at 24 row
// blocks of 48..71 key tiles on 148 SMs, and 14 % with 128 items).  A segment that is not a
// whole item leaves its unnormalised accumulator, running maximum and sum in scratch; the CTA
// that finishes an item's last missing piece merges the pieces in segment order (a fixed order:
// the result does not depend on which CTA comes last) and writes the output rows.  No CTA ever
// waits for another.
__host__ __device__ __forceinline__ int group_key_tiles(const AttnParams &p, int g) {
  const int n_rb = (p.n_tok + TILE - 1) / TILE;
  const int top_row0 = p.pair_heads ? (n_rb - 1 - g) * TILE : (((n_rb + 1) / 2 - 1 - g) * 2 + 1) * TILE;
  const int nk = (p.len + top_row0 + TILE + TILE - 1) / TILE;
  const int all = (p.len + p.n_tok + TILE - 1) / TILE;
  return nk < all ? nk : all;
}
__host__ __device__ __forceinline__ int unit_start(const AttnParams &p, int u, int n_units) {
  return (int)(((long long)u * p.total_steps) / n_units);
}
// The pieces of one item: its first global step, and the first and last CTA whose range meets it.
__host__ __device__ __forceinline__ void item_pieces(const AttnParams &p, int item, int nk, int n_units,
                                                     int &base, int &ua, int &ub) {
  base = 0;
  for (int g = 0; g < item / p.group_items; g++) base += group_key_tiles(p, g) * p.group_items;
  base += (item % p.group_items) * nk;
  ua = (int)(((long long)base * n_units) / p.total_steps);
  while (ua + 1 < n_units && unit_start(p, ua + 1, n_units) <= base) ua++;
  while (ua > 0 && unit_start(p, ua, n_units) > base) ua--;
  const int last_step = base + nk - 1;
  ub = ua;
  while (ub + 1 < n_units && unit_start(p, ub + 1, n_units) <= last_step) ub++;
}
// Scratch slot of the piece of an item (first global step `base`, first CTA `ua`) that CTA u holds:
// its first segment, unless the item begins inside u's range.
__host__ __device__ __forceinline__ int piece_slot(const AttnParams &p, int u, int ua, int base, int n_units) {
  return 2 * u + ((u == ua && base > unit_start(p, u, n_units)) ? 1 : 0);
}

struct Item {
  int row0[2], head[2], kvh, NK, NF, rot;
  __host__ __device__ __forceinline__ void set(const AttnParams &p, int item, int nk) {
    const int n_rb = (p.n_tok + TILE - 1) / TILE;
    const int g = item / p.group_items, idx = item - g * p.group_items;
    if (p.pair_heads) {
      row0[0] = row0[1] = (n_rb - 1 - g) * TILE;
      head[0] = 2 * idx; head[1] = 2 * idx + 1;
    } else {
      row0[0] = ((n_rb + 1) / 2 - 1 - g) * 2 * TILE; row0[1] = row0[0] + TILE;
      head[0] = head[1] = idx;
    }
    kvh = head[0] / (p.h / p.h_kv);
    NK = nk;
    // The softmax is order independent, so every item walks the key tiles that need no mask in
    // its own rotated order: CTAs of one KV head work at the same time, and in a common order
    // they would all ask the L2 for the same K and V lines at the same moment (measured: 1.4x
    // slower).  The tiles that cross the causal boundary come last.
    NF = (p.len + row0[0] + 1) / TILE;  // tiles fully visible to every row
    if (NF > NK) NF = NK;
    rot = NF > 0 ? (int)(((unsigned)item * 29u + 7u) % (unsigned)NF) : 0;
  }
  __host__ __device__ __forceinline__ int tile_of(int j) const {
    const int x = j + rot;
    return j < NF ? (x >= NF ? x - NF : x) : j;
  }
};

struct Segment { int item, k0, k1, nk, first; };

// Walks the segments of one CTA's range of steps.  Every role of the CTA runs its own walker over
// the same list.
struct Walker {
  int g, item, base, nk, s, s1, seg;
  __host__ __device__ __forceinline__ void init(const AttnParams &p, int unit, int n_units) {
    s = unit_start(p, unit, n_units);
    s1 = unit_start(p, unit + 1, n_units);
    base = 0; nk = 1;
    for (g = 0; g < p.n_groups; g++) {
      nk = group_key_tiles(p, g);
      const int span = nk * p.group_items;
      if (s < base + span) break;
      base += span;
    }
    const int idx = (s - base) / nk;
    item = g * p.group_items + idx;
    base += idx * nk;
    seg = 0;
  }
  __host__ __device__ __forceinline__ bool next(const AttnParams &p, Segment &o) {
    if (s >= s1 || g >= p.n_groups) return false;
    o.item = item; o.nk = nk; o.k0 = s - base; o.k1 = nk < s1 - base ? nk : s1 - base; o.first = seg == 0;
    s = base + o.k1;
    seg++;
    if (o.k1 == nk) {
      base += nk;
      item++;
      if (item - g * p.group_items == p.group_items) {
        g++;
        if (g < p.n_groups) nk = group_key_tiles(p, g);
      }
    }
    return true;
  }
};

template <int D>
__global__ void __launch_bounds__(AT_THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char *sQ = smem;                   // [2][TILE_BYTES]
  unsigned char *sK = smem + 2 * TILE_BYTES;  // [2 stages][TILE_BYTES]
  unsigned char *sV = smem + 4 * TILE_BYTES;  // [2 stages][TILE_BYTES]
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + 6 * TILE_BYTES);
  uint64_t *q_full = bars;          // 1
  uint64_t *k_full = bars + 1;      // 2
  uint64_t *v_full = bars + 3;      // 2
  uint64_t *k_empty = bars + 5;     // 2
  uint64_t *v_empty = bars + 7;     // 2
  uint64_t *s_full = bars + 9;      // 2
  uint64_t *p_full = bars + 11;     // 2
  uint64_t *o_full = bars + 13;     // 2
  uint64_t *p_half = bars + 15;     // 2: first 64 keys of P_t written (p_full: all 128)
  uint64_t *q_empty = bars + 17;    // 1: every S = Q K^T of the segment has executed (Q may be replaced)
  uint64_t *o_empty = bars + 18;    // 2: the segment's accumulator O_t has been read out
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 20);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_units = (int)gridDim.x;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_empty, 2);  // both MMA issuers
    for (int s = 0; s < 2; s++) {
      mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1);
      mbar_init(&k_empty[s], 2); mbar_init(&v_empty[s], 2);  // released by both MMA issuers
      mbar_init(&s_full[s], 1); mbar_init(&p_full[s], 4); mbar_init(&o_full[s], 1);
      mbar_init(&p_half[s], 4);
      mbar_init(&o_empty[s], 8);  // the eight softmax warps
    }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
  }
  if (warp == 9) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Each role walks the CTA's list of segments on its own; the walkers live in shared memory
  // (one per role, touched by that role's leading thread at segment boundaries only) so that they
  // cost no registers in the loops.
  Walker *walkers = reinterpret_cast<Walker *>(smem + 6 * TILE_BYTES + 256 + 2048);  // [4]
  Segment *crew_seg = reinterpret_cast<Segment *>(walkers + 4);
  Segment sg;
  Item it;

  if (warp >= 8) {
    setmaxnreg_dec<56>();
  if (warp == 11) {
    // idle warp of the third warpgroup
  } else if (warp == 8) {
    // ------------------------------------------------------------ TMA producer.  K and V tiles of
    // consecutive segments follow one another through the same two stages; Q is replaced as soon
    // as the last S = Q K^T of the previous segment has executed.
    if (lane == 0) {
      constexpr int nbox = (D + 63) / 64;  // 64-column boxes per head vector
      uint32_t gs = 0, nseg = 0;           // key steps / segments so far in this CTA
      bool ok = true;
      Walker &walk = walkers[0];
      walk.init(p, (int)blockIdx.x, n_units);
      while (ok && walk.next(p, sg)) {
        it.set(p, sg.item, sg.nk);
        // L2 prefetch PF tiles ahead: the cache of a layer is not L2 resident when its chunk step
        // starts, and two stages of shared memory do not cover an HBM miss.
        auto prefetch_tile = [&](int j) {
          const int row = it.tile_of(j) * TILE;
          for (int hh = 0; hh < nbox; hh++) {
            tma_prefetch_3d(&map_k, hh * 64, row, it.kvh);
            tma_prefetch_3d(&map_v, hh * 64, row, it.kvh);
          }
        };
        for (int j = sg.k0; j < min(sg.k0 + PF, sg.k1); j++) prefetch_tile(j);
        if (!mbar_wait(q_empty, (nseg & 1) ^ 1, abort_flag, p.status)) break;
        mbar_expect_tx(q_full, 2 * nbox * HALF_BYTES);
        for (int t = 0; t < 2; t++)
          for (int hh = 0; hh < nbox; hh++)
            tma_load_2d(sQ + t * TILE_BYTES + hh * HALF_BYTES, &map_q, it.head[t] * D + hh * 64, it.row0[t],
                        q_full);
        for (int j = sg.k0; j < sg.k1; j++, gs++) {
          const int s = gs & 1;
          const uint32_t ph = (gs >> 1) & 1;
          if (j + PF < sg.k1) prefetch_tile(j + PF);
          if (!mbar_wait(&k_empty[s], ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&k_full[s], nbox * HALF_BYTES);
          for (int hh = 0; hh < nbox; hh++)
            tma_load_3d(sK + s * TILE_BYTES + hh * HALF_BYTES, &map_k, hh * 64, it.tile_of(j) * TILE, it.kvh, &k_full[s]);
          if (!mbar_wait(&v_empty[s], ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&v_full[s], nbox * HALF_BYTES);
          for (int hh = 0; hh < nbox; hh++)
            tma_load_3d(sV + s * TILE_BYTES + hh * HALF_BYTES, &map_v, hh * 64, it.tile_of(j) * TILE, it.kvh, &v_full[s]);
        }
        nseg++;
      }
    }
  } else {
    // ------------------------------------------------------------ MMA issuers: warp 9 for query
    // tile 0, warp 10 for tile 1.  The tensor pipe's queue is only a couple of instructions deep,
    // so an issuer that stops to poll a barrier starves the pipe; with one issuer per tile the
    // other tile's MMAs cover each wait.  Descriptors are built once and advanced by constants.
    if (lane == 0) {
      const int t = warp - 9;
      constexpr uint32_t idesc_qk = idesc_bf16(TILE, TILE, 0, 0);
      constexpr uint32_t idesc_pv = idesc_bf16(TILE, D, 0, 1);
      constexpr int ksteps = D / 16;
      const uint64_t dq = desc_kmajor_sw128(sQ + t * TILE_BYTES);
      const uint64_t dk0 = desc_kmajor_sw128(sK), dk1 = desc_kmajor_sw128(sK + TILE_BYTES);
      const uint64_t dv0 = desc_mnmajor_sw128(sV, HALF_BYTES), dv1 = desc_mnmajor_sw128(sV + TILE_BYTES, HALF_BYTES);
      const uint32_t s_tmem = tmem_base + t * TILE, o_tmem = tmem_base + 2 * TILE + t * HD;
      // `last`: no further S of this segment follows, so Q may be replaced once these have executed
      auto issue_s = [&](int ks, bool last) {
        const uint64_t b = ks ? dk1 : dk0;
#pragma unroll
        for (int kk = 0; kk < ksteps; kk++) {
          const uint64_t off = (uint64_t)(((kk >> 2) * HALF_BYTES + (kk & 3) * 32) >> 4);
          if (kk == 0) mma_ss_first(s_tmem, dq + off, b + off, idesc_qk);
          else mma_ss_acc(s_tmem, dq + off, b + off, idesc_qk);
        }
        mma_commit(&s_full[t]);
        mma_commit(&k_empty[ks]);
        if (last) mma_commit(q_empty);
      };
      // the first four k-steps (keys 0..63) only need the first half of P
      auto issue_pv = [&](int vs, bool acc, int half) {
        const uint64_t b = vs ? dv1 : dv0;
#pragma unroll
        for (int kk = 0; kk < TILE / 16; kk++) {
          if ((kk >> 2) != half) continue;
          const uint64_t off = (uint64_t)((kk * 16 * 128) >> 4);
          if (kk == 0) mma_ts(o_tmem, s_tmem, b, idesc_pv, acc);
          else mma_ts_acc(o_tmem, s_tmem + kk * 8, b + off, idesc_pv);
        }
        if (half == 1) {
          mma_commit(&o_full[t]);
          mma_commit(&v_empty[vs]);
        }
      };
      uint32_t gs = 0, nseg = 0;
      bool ok = true;
      Walker &walk = walkers[1 + t];
      walk.init(p, (int)blockIdx.x, n_units);
      while (ok && walk.next(p, sg)) {
        ok = mbar_wait(q_full, nseg & 1, abort_flag, p.status);
        ok = ok && mbar_wait(&k_full[gs & 1], (gs >> 1) & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        // (the previous segment's last P V was issued by this thread before, and the pipe
        // executes in order: S may overwrite the columns that P occupied)
        issue_s(gs & 1, sg.k0 + 1 == sg.k1);
        for (int j = sg.k0; j < sg.k1 && ok; j++, gs++) {
          const int sv = gs & 1, sk = (gs + 1) & 1;
          // The tiles from memory arrive long before P does: poll them first, so that nothing but
          // the MMAs themselves stands between P and the next S.
          ok = mbar_wait(&v_full[sv], (gs >> 1) & 1, abort_flag, p.status);
          if (j + 1 < sg.k1) ok = ok && mbar_wait(&k_full[sk], ((gs + 1) >> 1) & 1, abort_flag, p.status);
          // the accumulator of the previous segment must have been read out before it is overwritten
          if (j == sg.k0 && nseg > 0) ok = ok && mbar_wait(&o_empty[t], (nseg - 1) & 1, abort_flag, p.status);
          // O_t += P_t V_j
          ok = ok && mbar_wait(&p_half[t], gs & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(sv, j > sg.k0, 0);
          ok = mbar_wait(&p_full[t], gs & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(sv, j > sg.k0, 1);
          // S_t = Q_t K_{j+1}^T
          if (j + 1 < sg.k1) issue_s(sk, j + 2 == sg.k1);
        }
        nseg++;
      }
    }
  }
  } else {
    // ------------------------------------------------------------ softmax: all eight warps work
    // on one query tile at a time, tile 0 and tile 1 alternately.  Warp w may only touch TMEM
    // lanes 32 (w % 4) .. +31, so warps q and 4 + q share the 32 rows of quarter q and split
    // the tile's 128 keys in halves: two warps per scheduler interleave their exponentials,
    // while the other tile's MMAs run.  The pair exchanges its half maxima through shared
    // memory around a 64-thread named barrier; that barrier also orders the first warp's read
    // of S columns [32, 64) before the second warp's P (keys 64..127) overwrites them.
    setmaxnreg_inc<224>();
    const int hf = warp >> 2, quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    float *xch = reinterpret_cast<float *>(smem + 6 * TILE_BYTES + 256);  // [tile][half][128 rows]
    const float c = p.scale_log2;
    bool ok = true;
    uint32_t gs = 0, nseg = 0;
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quarter) : "memory"); };
    auto crew_sync = [&]() { asm volatile("bar.sync 5, 256;" ::: "memory"); };

    // (no early exit anywhere below: after a timed-out wait the warps still meet at their named barriers)
    if (threadIdx.x == 0) walkers[3].init(p, (int)blockIdx.x, n_units);
    while (true) {
      // the crew's leading thread advances the walker; everybody reads the segment it found
      if (threadIdx.x == 0) {
        Segment nx;
        if (!walkers[3].next(p, nx)) nx.item = -1;
        *crew_seg = nx;
      }
      crew_sync();
      sg = *crew_seg;
      crew_sync();
      if (sg.item < 0) break;
      it.set(p, sg.item, sg.nk);
      float m_used[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
      const int seg_k0 = sg.k0, seg_k1 = sg.k1;
      for (int j = seg_k0; j < seg_k1; j++, gs++) {
#pragma unroll
        for (int t = 0; t < 2; t++) {
          const int row = it.row0[t] + r;
          const int limit = p.len + row;  // last visible key
          const uint32_t s_addr = tmem_base + lane_off + t * TILE;
          const uint32_t o_addr = tmem_base + lane_off + 2 * TILE + t * HD;
          if (ok) ok = mbar_wait(&s_full[t], gs & 1, abort_flag, p.status);
          tc_fence_after();
          uint32_t s[64];
          tmem_ld32(s_addr + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
          tmem_ld32(s_addr + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
          tmem_wait_ld();

          const int key0 = it.tile_of(j) * TILE;
          float tmax;
          if (key0 + TILE - 1 > p.len + it.row0[t]) {  // a tile that crosses the causal boundary
            tmax = -INFINITY;
#pragma unroll
            for (int i = 0; i < 64; i++) {
              float x = (key0 + hf * 64 + i <= limit) ? __uint_as_float(s[i]) : -INFINITY;
              s[i] = __float_as_uint(x);
              tmax = fmaxf(tmax, x);
            }
          } else {
            float tm[8];
#pragma unroll
            for (int a = 0; a < 8; a++) tm[a] = fmaxf(__uint_as_float(s[2 * a]), __uint_as_float(s[2 * a + 1]));
#pragma unroll
            for (int i = 16; i < 64; i += 16)
#pragma unroll
              for (int a = 0; a < 8; a++)
                tm[a] = fmaxf(tm[a], fmaxf(__uint_as_float(s[i + 2 * a]), __uint_as_float(s[i + 2 * a + 1])));
            tmax = fmaxf(fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])), fmaxf(fmaxf(tm[4], tm[5]), fmaxf(tm[6], tm[7])));
          }
          xch[(t * 2 + hf) * TILE + r] = tmax;
          pair_sync();
          // A piece of an item may begin with a tile in which this row sees no key at all (the
          // other query tile of the pair lies one row block lower): a finite floor keeps
          // (-inf) - (-inf) out of the exponent; such a tile contributes exact zeros.
          tmax = fmaxf(fmaxf(tmax, xch[(t * 2 + (hf ^ 1)) * TILE + r]) * c, -1e30f);

          if (j == seg_k0) {
            m_used[t] = tmax;
          } else {
            // both warps of the pair see the same maxima, hence take the same branch
            const bool need = tmax > m_used[t] + RESCALE_LOG2;
            if (__any_sync(0xffffffffu, need)) {
              // the accumulator must hold every product issued so far before it is rescaled
              if (ok) ok = mbar_wait(&o_full[t], (gs - 1) & 1, abort_flag, p.status);
              tc_fence_after();
              float alpha = 1.0f;
              if (need) { alpha = exp2f(m_used[t] - tmax); m_used[t] = tmax; }
              l[t] *= alpha;
#pragma unroll 1
              for (int q = hf; q < D / 32; q += 2) {  // the pair shares the accumulator's columns
                uint32_t o[32];
                tmem_ld32(o_addr + q * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i++) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                tmem_st32(o_addr + q * 32, o);
              }
              tmem_wait_st();
              // the next product touches every column: both halves must be rescaled before either
              // warp hands over its P
              pair_sync();
            }
          }

          const uint64_t c2 = pack_f32x2(c, c), nm2 = pack_f32x2(-m_used[t], -m_used[t]);
          uint64_t la = pack_f32x2(0.f, 0.f), lb = la;
          uint32_t pk[32];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float x0, x1, x2, x3;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, nm2), x0, x1);
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[2 * i + 2]), __uint_as_float(s[2 * i + 3])), c2, nm2), x2, x3);
            const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
            la = add_f32x2(la, pack_f32x2(p0, p1));
            lb = add_f32x2(lb, pack_f32x2(p2, p3));
            pk[i] = pack_bf16(p0, p1);
            pk[i + 1] = pack_bf16(p2, p3);
          }
          tmem_st32(s_addr + hf * 32, pk);
          {
            float a0, a1, b0, b1;
            unpack_f32x2(la, a0, a1);
            unpack_f32x2(lb, b0, b1);
            l[t] += (a0 + a1) + (b0 + b1);
          }
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(hf == 0 ? &p_half[t] : &p_full[t]);
        }
      }

      // ---- end of the segment: a whole item is normalised and written; a piece goes to scratch
      // (the segment is read again from shared memory: what only this part needs does not occupy
      // registers during the loop above)
      sg = *crew_seg;
      it.set(p, sg.item, sg.nk);
      const bool whole = sg.k0 == 0 && sg.k1 == sg.nk;
      const int slot = 2 * (int)blockIdx.x + (sg.first ? 0 : 1);
#pragma unroll
      for (int t = 0; t < 2; t++) {
        const int row = it.row0[t] + r;
        const uint32_t o_addr = tmem_base + lane_off + 2 * TILE + t * HD;
        if (ok) ok = mbar_wait(&o_full[t], (gs - 1) & 1, abort_flag, p.status);
        tc_fence_after();
        xch[(t * 2 + hf) * TILE + r] = l[t];
        pair_sync();
        const float l_row = l[t] + xch[(t * 2 + (hf ^ 1)) * TILE + r];
        if (whole) {
          const float inv = 1.0f / l_row;
          bf16 *dst = p.out + (size_t)row * p.h * D + (size_t)it.head[t] * D;
#pragma unroll 1
          for (int q = hf; q < D / 32; q += 2) {
            uint32_t o[32];
            tmem_ld32(o_addr + q * 32, o);
            tmem_wait_ld();
            if (ok && row < p.n_tok) {
#pragma unroll
              for (int v = 0; v < 4; v++) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                w.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                w.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                w.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                *reinterpret_cast<uint4 *>(dst + q * 32 + v * 8) = w;
              }
            }
          }
        } else {
          float *po = p.part_o + ((size_t)(slot * 2 + t) * TILE + r) * D;
          if (hf == 0 && ok) {
            float *pml = p.part_ml + (size_t)(slot * 2 + t) * 2 * TILE;
            pml[r] = m_used[t];
            pml[TILE + r] = l_row;
          }
#pragma unroll 1
          for (int q = hf; q < D / 32; q += 2) {
            uint32_t o[32];
            tmem_ld32(o_addr + q * 32, o);
            tmem_wait_ld();
            if (ok) {
#pragma unroll
              for (int v = 0; v < 8; v++)
                *reinterpret_cast<uint4 *>(po + q * 32 + v * 4) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
            }
          }
        }
        // this warp has read its part of O_t: the next segment's first product may overwrite it
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_empty[t]);
      }
      nseg++;

      if (!whole) {
        // The piece is in scratch.  Whoever completes the item merges all its pieces.
        __threadfence();
        crew_sync();
        if (threadIdx.x == 0) {
          // pieces of this item: one per CTA whose range meets the item's steps
          int base, ua, ub;
          item_pieces(p, sg.item, sg.nk, n_units, base, ua, ub);
          const unsigned pieces = (unsigned)(ub - ua + 1);
          unsigned done = ok ? atomicAdd(&p.item_cnt[sg.item], 1u) : 0u;
          int lastf = 0;
          if (ok && done + 1 == pieces) {
            p.item_cnt[sg.item] = 0;  // every piece has arrived: leave the counter at zero for the next launch
            lastf = 1;
          }
          reinterpret_cast<volatile int *>(xch)[0] = lastf;
          reinterpret_cast<volatile int *>(xch)[1] = ua;
          reinterpret_cast<volatile int *>(xch)[2] = ub;
          reinterpret_cast<volatile int *>(xch)[3] = base;
        }
        crew_sync();
        const int lastf = reinterpret_cast<volatile int *>(xch)[0];
        const int ua = reinterpret_cast<volatile int *>(xch)[1], ub = reinterpret_cast<volatile int *>(xch)[2];
        const int base = reinterpret_cast<volatile int *>(xch)[3];
        crew_sync();  // xch is reused by the next segment
        if (lastf) {
          __threadfence();
          auto slot_of = [&](int u) { return piece_slot(p, u, ua, base, n_units); };
          // Every thread owns D / 8 float4 of the tile and folds the pieces in one after the other,
          // in segment order (the same sums whoever merges), with all of a piece's loads in flight
          // at once: the pieces come from the L2, and a loop with one load at a time would take
          // longer than forty key steps.
          constexpr int V4 = D / 4;    // float4 per row
          constexpr int EPT = D / 8;   // float4 per thread: TILE * V4 / 256
          for (int t = 0; t < 2; t++) {
            float4 acc[EPT];
            float mx[EPT], lsum[EPT];
#pragma unroll
            for (int i = 0; i < EPT; i++) { acc[i] = make_float4(0.f, 0.f, 0.f, 0.f); mx[i] = -INFINITY; lsum[i] = 0.f; }
            for (int u = ua; u <= ub; u++) {
              const size_t sl = (size_t)(slot_of(u) * 2 + t);
              const float *ml = p.part_ml + sl * 2 * TILE;
              const float4 *po = reinterpret_cast<const float4 *>(p.part_o + sl * TILE * D);
              float m_u[EPT], l_u[EPT];
              float4 o_u[EPT];
#pragma unroll
              for (int i = 0; i < EPT; i++) {
                const int e = (int)threadIdx.x + 256 * i, rr = e / V4;
                m_u[i] = __ldcg(ml + rr);
                l_u[i] = __ldcg(ml + TILE + rr);
                o_u[i] = __ldcg(po + e);
              }
#pragma unroll
              for (int i = 0; i < EPT; i++) {
                const float nm = fmaxf(mx[i], m_u[i]);
                const float a = exp2f(mx[i] - nm), w = exp2f(m_u[i] - nm);  // (-inf) - finite = -inf: a = 0 at the first piece
                mx[i] = nm;
                lsum[i] = lsum[i] * a + w * l_u[i];
                acc[i].x = acc[i].x * a + w * o_u[i].x; acc[i].y = acc[i].y * a + w * o_u[i].y;
                acc[i].z = acc[i].z * a + w * o_u[i].z; acc[i].w = acc[i].w * a + w * o_u[i].w;
              }
            }
#pragma unroll
            for (int i = 0; i < EPT; i++) {
              const int e = (int)threadIdx.x + 256 * i, rr = e / V4, c4 = e - rr * V4;
              const int row = it.row0[t] + rr;
              if (row >= p.n_tok) continue;
              const float inv = 1.0f / lsum[i];
              uint2 w2;
              w2.x = pack_bf16(acc[i].x * inv, acc[i].y * inv);
              w2.y = pack_bf16(acc[i].z * inv, acc[i].w * inv);
              *reinterpret_cast<uint2 *>(p.out + (size_t)row * p.h * D + (size_t)it.head[t] * D + c4 * 4) = w2;
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 9) {
    __syncwarp();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool attention_tc_supported(int n_tok, int h, int h_kv, int d) {
  return (d == 64 || d == 96 || d == 128) && n_tok >= 64 && h % h_kv == 0;
}

// Most CTAs a launch may use on the current device: one per SM by default.  A multiple of the SM
// count keeps the SMs' shares equal; LOCRET_ATTN_WAVES = k makes it k per SM (smaller ranges,
// handed out by the hardware as SMs free up), LOCRET_ATTN_UNITS = n forces exactly n (tests).
// Read when a layer is created.
int attention_tc_max_units() {
  const char *e = getenv("LOCRET_ATTN_UNITS");
  const int forced = e ? atoi(e) : 0;
  if (forced > 0) return forced < 4096 ? forced : 4096;
  const char *w = getenv("LOCRET_ATTN_WAVES");
  int waves = w ? atoi(w) : 1;
  if (waves < 1 || waves > 8) waves = 1;
  return waves * sm_count_of_current_device();
}
size_t attention_tc_part_o_floats(int units, int d) { return (size_t)2 * units * 2 * TILE * d; }
size_t attention_tc_part_ml_floats(int units) { return (size_t)2 * units * 2 * 2 * TILE; }
int attention_tc_max_items(int chunk, int h) { return ((chunk + TILE - 1) / TILE) * h; }

// map_k / map_v: 3-D maps {d, cap, h_kv} with box {64, 128, 1}; map_q: 2-D {h*d, rows} box {64, 128}.
template <int D>
static cudaError_t launch_attn_d(const CUtensorMap *map_q, const CUtensorMap *map_k, const CUtensorMap *map_v,
                                 const AttnParams &p, int grid, cudaStream_t st) {
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(attn_tc_kernel<D>, AT_SMEM, attr_set); e != cudaSuccess) return e;
  attn_tc_kernel<D><<<grid, AT_THREADS, AT_SMEM, st>>>(*map_q, *map_k, *map_v, p);
  return cudaGetLastError();
}

// The work list of a launch and its number of CTAs (0 if the step count does not fit an int).
static int plan_attention(AttnParams &p, int n_tok, int h, int h_kv, int d, int len, int max_units) {
  p.n_tok = n_tok; p.h = h; p.h_kv = h_kv; p.d = d; p.len = len;
  p.pair_heads = ((h / h_kv) % 2 == 0) ? 1 : 0;
  const int n_rb = (n_tok + TILE - 1) / TILE;
  p.n_groups = p.pair_heads ? n_rb : (n_rb + 1) / 2;
  p.group_items = p.pair_heads ? h / 2 : h;
  p.n_items = p.n_groups * p.group_items;
  long long total = 0;
  for (int g = 0; g < p.n_groups; g++) total += (long long)group_key_tiles(p, g) * p.group_items;
  if (total > 0x7fffffffll) return 0;
  p.total_steps = (int)total;
  // at least MIN_STEPS key steps per CTA; never more CTAs than the scratch was sized for
  constexpr int MIN_STEPS = 4;
  int grid = max_units;
  if ((long long)grid * MIN_STEPS > total) grid = (int)(total / MIN_STEPS);
  return grid < 1 ? 1 : grid;
}

// Host-side replay of the division of a launch's work, for tests: the segments every CTA would
// walk, in order, as rows (unit, item, k0, k1, key tiles of the item, scratch slot or -1 for a
// whole item, first CTA of the item, last CTA of the item).  Returns the number of rows (also
// when more than `cap` exist; only `cap` are written), or -1 for arguments the kernel does not take.
int attention_tc_replay_split(int n_tok, int h, int h_kv, int d, int len, int max_units, int32_t *rows,
                              int cap, int32_t *n_units_out, int32_t *total_steps_out) {
  if (!attention_tc_supported(n_tok, h, h_kv, d) || max_units < 1 || len < 0) return -1;
  AttnParams p{};
  const int units = plan_attention(p, n_tok, h, h_kv, d, len, max_units);
  if (units < 1) return -1;
  if (n_units_out) *n_units_out = units;
  if (total_steps_out) *total_steps_out = p.total_steps;
  int n = 0;
  for (int u = 0; u < units; u++) {
    Walker w;
    w.init(p, u, units);
    Segment sg;
    while (w.next(p, sg)) {
      if (n < cap && rows) {
        int base, ua, ub;
        item_pieces(p, sg.item, sg.nk, units, base, ua, ub);
        const bool whole = sg.k0 == 0 && sg.k1 == sg.nk;
        int32_t *r = rows + (size_t)n * 8;
        r[0] = u; r[1] = sg.item; r[2] = sg.k0; r[3] = sg.k1; r[4] = sg.nk;
        r[5] = whole ? -1 : 2 * u + (sg.first ? 0 : 1);
        r[6] = ua; r[7] = ub;
        // the merging CTA must look for this piece where its writer put it
        if (!whole && piece_slot(p, u, ua, base, units) != r[5]) return -2;
      }
      n++;
    }
  }
  return n;
}

cudaError_t launch_attention_tc(const CUtensorMap *map_q, const CUtensorMap *map_k,
                                const CUtensorMap *map_v, bf16 *out, int n_tok, int h, int h_kv, int d,
                                int len, const AttnWork &work, int *status, cudaStream_t st) {
  AttnParams p;
  const int grid = plan_attention(p, n_tok, h, h_kv, d, len, work.max_units);
  if (grid < 1 || p.n_items > work.max_items) return cudaErrorInvalidValue;
  p.out = out;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  p.status = status;
  p.part_o = work.part_o; p.part_ml = work.part_ml; p.item_cnt = work.item_cnt;
  switch (d) {
    case 64: return launch_attn_d<64>(map_q, map_k, map_v, p, grid, st);
    case 96: return launch_attn_d<96>(map_q, map_k, map_v, p, grid, st);
    case 128: return launch_attn_d<128>(map_q, map_k, map_v, p, grid, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace locret
