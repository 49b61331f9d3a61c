// Eq. 1 on tcgen05 tensor cores with a pair of CTAs per instruction (cta_group::2), head_dim 128.
//
// A cluster of two CTAs (two SMs) owns two 128-row query tiles that share a KV head (two query
// heads of one GQA group over the same rows, or two consecutive row blocks of one head): CTA c
// holds query tile c, its accumulator and its softmax.  Every tcgen05.mma covers both tiles
// (M = 256: rows 0..127 in CTA 0's tensor memory, 128..255 in CTA 1's); its B operand is split
// between the two CTAs' shared memories, so each CTA loads only half of every key tile (64 of
// the 128 keys for S = Q K^T) and half of every value tile (64 of the 128 columns for O += P V).
// One SM then reads 6 KB of shared memory per instruction instead of 8 KB, and has the tensor
// memory of ONE query tile to fill: three S/P buffers of 128 columns and the accumulator, so S of
// key tiles j + 1 and j + 2 exist before P of key tile j is consumed.
// Roles in each CTA:
//   warps 0-3 / 4-7  softmax of the even / odd key tiles: thread = query row, 128 keys in
//                    registers, P = exp2(S - m) written as bf16 over S.  The two groups run
//                    independently (two warps per scheduler in different phases); what they share is
//                    the row's scale m: the warp that handles key tile j waits for the value its
//                    partner published for tile j - 1, decides (m grows only when the maximum
//                    exceeds it by 2^100, then the warp rescales the accumulator once every earlier
//                    product has completed) and publishes m for tile j before its exponentials.
//                    Each group keeps its own partial row sum.
//   warp 8           TMA producer of this CTA's halves (Q once, then K three tiles ahead of V);
//                    the loads of both CTAs complete on CTA 0's barriers;
//   warp 9           CTA 0 only: issues every MMA of the pair: S for the first three key tiles,
//                    then per key tile O += P_j V_j (first half of P, second half) and S_{j+3}
//                    into the buffer P_j leaves; commits are multicast to both CTAs' barriers.
// TMEM columns per CTA: S/P buffers [0,128) [128,256) [256,384), O [384,512).
// Query row t sees keys [0, len + t]: the retained cache unmasked, the chunk causally.
#include "tc_common.cuh"

namespace locret {

namespace {

using namespace tc;

constexpr int A2_THREADS = 384;
constexpr int TILE = 128;
constexpr int D = 128;
constexpr int NBUF = 3;                 // S/P buffers per CTA
constexpr int NSTK = 4, NSTV = 4;       // shared-memory stages of key halves / value halves
constexpr int Q_BYTES = TILE * D * 2;   // 32 KB: two 64-column swizzled boxes of 128 rows
constexpr int QBOX = TILE * 128;        // 16 KB
constexpr int KBOX = 64 * 128;          // 64 keys x 64 columns: 8 KB
constexpr int K_STAGE = 2 * KBOX;       // this CTA's 64 keys x 128 columns
constexpr int V_STAGE = TILE * 128;     // 128 keys x this CTA's 64 columns
constexpr int A2_BAR_BYTES = 512;
constexpr int A2_SMEM = 1024 + Q_BYTES + NSTK * K_STAGE + NSTV * V_STAGE + A2_BAR_BYTES + 2 * TILE * 4 + 2 * TILE * 4;
constexpr float RESCALE_LOG2 = 100.0f;  // see attn_tc.cu: P and O stay finite, precision is scale free
constexpr int PF = 3;       // key tiles prefetched into L2 ahead of the shared-memory stages (0 / 3 / 6 / 10 measured: 3 is best by about 1 % of the step)

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

// ---- cluster and cta_group::2 forms
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  // (no cluster-scope release: what the arrival publishes lives in tensor memory and is ordered by
  // tcgen05.wait::st + tcgen05.fence::before_thread_sync; a cluster-scope fence here cost ~25 % of the kernel)
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// loads by either CTA of the pair; completion is counted on the barrier at `bar_cluster`
__device__ __forceinline__ void tma2_load_2d(void *dst, const CUtensorMap *map, int c0, int c1,
                                             uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2,
                                             uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem2_alloc(uint32_t *dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tmem2_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem2_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the barrier at this offset in both CTAs arrives when every MMA issued so far has completed
__device__ __forceinline__ void mma2_commit_both(uint64_t *bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"((uint16_t)3)
      : "memory");
}

struct Attn2Params {
  bf16 *out;
  int n_tok, h, h_kv, len, pair_heads;
  float scale_log2;
  int *status;
  int per_head;
  PerHead len_m;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(A2_THREADS, 1)
attn_tc2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const Attn2Params p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char *sQ = smem;
  unsigned char *sK = sQ + Q_BYTES;              // [NSTK][K_STAGE]
  unsigned char *sV = sK + NSTK * K_STAGE;       // [NSTV][V_STAGE]
  uint64_t *bars = reinterpret_cast<uint64_t *>(sV + NSTV * V_STAGE);
  uint64_t *q_full = bars;                    // 1        (used in CTA 0)
  uint64_t *k_full = q_full + 1;              // NSTK     (CTA 0)
  uint64_t *v_full = k_full + NSTK;           // NSTV     (CTA 0)
  uint64_t *k_empty = v_full + NSTV;          // NSTK     (each CTA)
  uint64_t *v_empty = k_empty + NSTK;         // NSTV     (each CTA)
  uint64_t *s_full = v_empty + NSTV;          // NBUF     (each CTA)
  uint64_t *p_half = s_full + NBUF;           // NBUF     (CTA 0: 4 warps of each CTA)
  uint64_t *p_full = p_half + NBUF;           // NBUF     (CTA 0)
  uint64_t *pv_done = p_full + NBUF;          // NBUF     (each CTA)
  uint64_t *m_ready = pv_done + NBUF;         // [4 quarters][2]  (each CTA)
  uint64_t *o_final = m_ready + 8;            // 1        (each CTA): every product of the pair is complete
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(o_final + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  static_assert((1 + 2 * NSTK + 2 * NSTV + 4 * NBUF + 8 + 1) * 8 + 8 <= A2_BAR_BYTES, "barrier area");
  float *m_pub = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(bars) + A2_BAR_BYTES);  // [2][128]
  float *xch = m_pub + 2 * TILE;                                                                     // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t cta = cluster_ctarank();
  const int pair = (int)blockIdx.x >> 1;
  const int g = p.h / p.h_kv;
  const int n_rb = (p.n_tok + TILE - 1) / TILE;

  int row0[2], head[2];
  if (p.pair_heads) {
    const int hp = p.h / 2;
    const int rb = n_rb - 1 - pair / hp;
    const int hq = pair % hp;
    row0[0] = row0[1] = rb * TILE;
    head[0] = 2 * hq; head[1] = 2 * hq + 1;
  } else {
    const int n_rp = (n_rb + 1) / 2;
    const int rp = n_rp - 1 - pair / p.h;
    row0[0] = rp * 2 * TILE; row0[1] = row0[0] + TILE;
    head[0] = head[1] = pair % p.h;
  }
  const int my_row0 = row0[cta], my_head = head[cta];
  const int kvh = head[0] / g;
  const int len = p.per_head ? p.len_m.v[kvh] : p.len;
  const int n = len + p.n_tok;
  int NK = (len + row0[1] + TILE + TILE - 1) / TILE;
  NK = min(NK, (n + TILE - 1) / TILE);
  const int NF = min(NK, (len + row0[0] + 1) / TILE);  // key tiles fully visible to every row of the pair
  const int rot = NF > 0 ? (int)(((unsigned)pair * 29u + 7u) % (unsigned)NF) : 0;
  auto tile_of = [&](int j) { int x = j + rot; return j < NF ? (x >= NF ? x - NF : x) : j; };

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < NSTK; s++) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
    for (int s = 0; s < NSTV; s++) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int s = 0; s < NBUF; s++) {
      mbar_init(&s_full[s], 1); mbar_init(&p_half[s], 8); mbar_init(&p_full[s], 8); mbar_init(&pv_done[s], 1);
    }
    for (int s = 0; s < 8; s++) mbar_init(&m_ready[s], 1);
    mbar_init(o_final, 1);
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
  }
  if (warp == 9) {
    tmem2_alloc(tmem_slot, 512);
    tmem2_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the partner's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp >= 8) {
    setmaxnreg_dec<56>();
    if (warp == 8) {
      // ------------------------------------------------------------ TMA producer (both CTAs)
      if (lane == 0) {
        const uint32_t q_full0 = map_to_cta(smem_u32(q_full), 0);
        if (cta == 0) mbar_expect_tx(q_full, 2 * Q_BYTES);
        for (int hh = 0; hh < 2; hh++)
          tma2_load_2d(sQ + hh * QBOX, &map_q, my_head * D + hh * 64, my_row0, q_full0);
        auto prefetch_tile = [&](int j) {
          const int row = tile_of(j) * TILE;
          tma_prefetch_3d(&map_k, 0, row + (int)cta * 64, kvh);
          tma_prefetch_3d(&map_k, 64, row + (int)cta * 64, kvh);
          tma_prefetch_3d(&map_v, (int)cta * 64, row, kvh);
        };
        auto load_k = [&](int j) -> bool {
          const int s = j % NSTK;
          if (!mbar_wait(&k_empty[s], ((j / NSTK) & 1) ^ 1, abort_flag, p.status)) return false;
          if (cta == 0) mbar_expect_tx(&k_full[s], 2 * K_STAGE);
          const uint32_t bar0 = map_to_cta(smem_u32(&k_full[s]), 0);
          for (int hh = 0; hh < 2; hh++)
            tma2_load_3d(sK + s * K_STAGE + hh * KBOX, &map_k, hh * 64, tile_of(j) * TILE + (int)cta * 64, kvh, bar0);
          return true;
        };
        auto load_v = [&](int j) -> bool {
          const int s = j % NSTV;
          if (!mbar_wait(&v_empty[s], ((j / NSTV) & 1) ^ 1, abort_flag, p.status)) return false;
          if (cta == 0) mbar_expect_tx(&v_full[s], 2 * V_STAGE);
          const uint32_t bar0 = map_to_cta(smem_u32(&v_full[s]), 0);
          tma2_load_3d(sV + s * V_STAGE, &map_v, (int)cta * 64, tile_of(j) * TILE, kvh, bar0);
          return true;
        };
        for (int j = 0; j < min(PF, NK); j++) prefetch_tile(j);
        bool ok = true;
        for (int j = 0; j < min(NBUF, NK) && ok; j++) ok = load_k(j);
        for (int j = 0; j < NK && ok; j++) {
          if (j + PF < NK) prefetch_tile(j + PF);
          ok = load_v(j);
          if (ok && j + NBUF < NK) ok = load_k(j + NBUF);
        }
        // Drain: the completions of the last uses of every stage are multicast to both CTAs and nobody
        // else waits for them; the CTA must not end (and its shared memory pass to another kernel's
        // CTA) while such an arrival is still on its way.  This thread has nothing else left to do.
#ifndef A2_NO_DRAIN
        for (int j = max(NK - NSTK, 0); j < NK && ok; j++)
          ok = mbar_wait(&k_empty[j % NSTK], (j / NSTK) & 1, abort_flag, p.status);
        for (int j = max(NK - NSTV, 0); j < NK && ok; j++)
          ok = mbar_wait(&v_empty[j % NSTV], (j / NSTV) & 1, abort_flag, p.status);
        for (int j = max(NK - NBUF, 0); j < NK && ok; j++)
          ok = mbar_wait(&pv_done[j % NBUF], (j / NBUF) & 1, abort_flag, p.status);
        if (ok && NK > 0) ok = mbar_wait(o_final, 0, abort_flag, p.status);
#endif
      }
    } else if (warp == 9 && cta == 0) {
      // ------------------------------------------------------------ issuer of O += P_j V_j (pair)
      if (lane == 0) {
        constexpr uint32_t idesc_pv = idesc_bf16(2 * TILE, D, 0, 1);
        const uint64_t dv = desc_mnmajor_sw128(sV, V_STAGE);
        const uint32_t o_tmem = tmem_base + NBUF * TILE;
        auto issue_pv = [&](int j, int half) {   // keys [64 half, 64 half + 64) of key tile j
          const uint32_t p_tmem = tmem_base + (uint32_t)(j % NBUF) * TILE;
          const uint64_t b = dv + (uint64_t)(((j % NSTV) * V_STAGE) >> 4);
#pragma unroll
          for (int kk = 4 * half; kk < 4 * half + 4; kk++)
            mma2_ts(o_tmem, p_tmem + kk * 8, b + (uint64_t)((kk * 16 * 128) >> 4), idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
          if (half == 1) {
            mma2_commit_both(&pv_done[j % NBUF]);
            mma2_commit_both(&v_empty[j % NSTV]);
          }
        };
        bool ok = true;
        for (int j = 0; j < NK && ok; j++) {
          const int buf = j % NBUF;
          const uint32_t ph = (j / NBUF) & 1;
          ok = mbar_wait(&v_full[j % NSTV], (j / NSTV) & 1, abort_flag, p.status);
          ok = ok && mbar_wait(&p_half[buf], ph, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(j, 0);
          ok = mbar_wait(&p_full[buf], ph, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(j, 1);
          // (a barrier of its own: pv_done completes once per use of a buffer, and a warp that is done
          // early could be two phases ahead of it, which a parity cannot tell from none)
          if (j == NK - 1) mma2_commit_both(o_final);
        }
      }
    } else if (warp == 10 && cta == 0) {
      // ------------------------------------------------------------ issuer of S_j = Q K_j^T (pair):
      // a thread of its own, so that its polling is covered by the other issuer's instructions
      if (lane == 0) {
        constexpr uint32_t idesc_qk = idesc_bf16(2 * TILE, TILE, 0, 0);
        const uint64_t dq = desc_kmajor_sw128(sQ);
        const uint64_t dk = desc_kmajor_sw128(sK);
        auto issue_s = [&](int j) {   // into buffer j % NBUF
          const uint32_t s_tmem = tmem_base + (uint32_t)(j % NBUF) * TILE;
          const uint64_t b = dk + (uint64_t)(((j % NSTK) * K_STAGE) >> 4);
#pragma unroll
          for (int kk = 0; kk < D / 16; kk++) {
            const uint64_t offq = (uint64_t)(((kk >> 2) * QBOX + (kk & 3) * 32) >> 4);
            const uint64_t offk = (uint64_t)(((kk >> 2) * KBOX + (kk & 3) * 32) >> 4);
            mma2_ss(s_tmem, dq + offq, b + offk, idesc_qk, kk > 0);
          }
          mma2_commit_both(&s_full[j % NBUF]);
          mma2_commit_both(&k_empty[j % NSTK]);
        };
        bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
        for (int j = 0; j < NK && ok; j++) {
          ok = mbar_wait(&k_full[j % NSTK], (j / NSTK) & 1, abort_flag, p.status);
          // the buffer is free once the product that read P_{j-3} from it has completed
          if (ok && j >= NBUF) ok = mbar_wait(&pv_done[j % NBUF], ((j - NBUF) / NBUF) & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_s(j);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax: group G = warp / 4
    // takes the key tiles j = G, G + 2, ...; thread = query row.
    setmaxnreg_inc<224>();
    const int G = warp >> 2, quarter = warp & 3;
    const int r = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t o_addr = tmem_base + lane_off + NBUF * TILE;
    const float c = p.scale_log2;
    const int row = my_row0 + r;
    const int limit = len + row;  // last visible key
    const uint32_t p_half0 = map_to_cta(smem_u32(p_half), 0), p_full0 = map_to_cta(smem_u32(p_full), 0);
    float m_mine = -INFINITY, l = 0.f;
    bool ok = true;

    for (int j = G; j < NK; j += 2) {
      const int buf = j % NBUF;
      const uint32_t s_addr = tmem_base + lane_off + (uint32_t)buf * TILE;
      if (ok) ok = mbar_wait(&s_full[buf], (j / NBUF) & 1, abort_flag, p.status);
      tc_fence_after();
      uint32_t s[128];
#pragma unroll
      for (int q = 0; q < 4; q++) tmem_ld32(s_addr + q * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32 * q]));
      tmem_wait_ld();

      const int key0 = tile_of(j) * TILE;
      float tmax;
      if (key0 + TILE - 1 > len + my_row0) {  // a tile that crosses this query tile's causal boundary
        tmax = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; i++) {
          float x = (key0 + i <= limit) ? __uint_as_float(s[i]) : -INFINITY;
          s[i] = __float_as_uint(x);
          tmax = fmaxf(tmax, x);
        }
      } else {
        float tm[8];
#pragma unroll
        for (int a = 0; a < 8; a++) tm[a] = fmaxf(__uint_as_float(s[2 * a]), __uint_as_float(s[2 * a + 1]));
#pragma unroll
        for (int i = 16; i < 128; i += 16)
#pragma unroll
          for (int a = 0; a < 8; a++)
            tm[a] = fmaxf(tm[a], fmaxf(__uint_as_float(s[i + 2 * a]), __uint_as_float(s[i + 2 * a + 1])));
        tmax = fmaxf(fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])), fmaxf(fmaxf(tm[4], tm[5]), fmaxf(tm[6], tm[7])));
      }
      tmax *= c;

      // the row's scale: the value published for tile j - 1, unless this tile's maximum is far above it
      float m_prev = tmax;
      bool need = false;
      if (j > 0) {
        if (ok) ok = mbar_wait(&m_ready[quarter * 2 + ((j - 1) & 1)], ((j - 1) >> 1) & 1, abort_flag, p.status);
        m_prev = m_pub[((j - 1) & 1) * TILE + r];
        need = tmax > m_prev + RESCALE_LOG2;
      }
      const float m_new = need ? tmax : m_prev;
      m_pub[(j & 1) * TILE + r] = m_new;
      __syncwarp();
      if (lane == 0) mbar_arrive(&m_ready[quarter * 2 + (j & 1)]);
      if (m_new != m_mine) {
        l = (l == 0.f) ? 0.f : l * exp2f(m_mine - m_new);
        m_mine = m_new;
      }
      if (__any_sync(0xffffffffu, need)) {
        // every product up to tile j - 1 is in the accumulator; none of tile j or later is issued
        // before this warp hands over its P
        if (ok) ok = mbar_wait(&pv_done[(j - 1) % NBUF], ((j - 1) / NBUF) & 1, abort_flag, p.status);
        tc_fence_after();
        const float alpha = need ? exp2f(m_prev - m_new) : 1.0f;
#pragma unroll 1
        for (int q = 0; q < D / 32; q++) {
          uint32_t o[32];
          tmem_ld32(o_addr + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; i++) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
          tmem_st32(o_addr + q * 32, o);
        }
        tmem_wait_st();
      }

      const uint64_t c2 = pack_f32x2(c, c), nm2 = pack_f32x2(-m_mine, -m_mine);
      uint64_t la = pack_f32x2(0.f, 0.f), lb = la;
#pragma unroll
      for (int hf = 0; hf < 2; hf++) {
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const int e = 64 * hf + 2 * i;
          float x0, x1, x2, x3;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), c2, nm2), x0, x1);
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[e + 2]), __uint_as_float(s[e + 3])), c2, nm2), x2, x3);
          const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
          la = add_f32x2(la, pack_f32x2(p0, p1));
          lb = add_f32x2(lb, pack_f32x2(p2, p3));
          pk[i] = pack_bf16(p0, p1);
          pk[i + 1] = pack_bf16(p2, p3);
        }
        tmem_st32(s_addr + hf * 32, pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote((hf == 0 ? p_half0 : p_full0) + (uint32_t)buf * 8u);
      }
      {
        float a0, a1, b0, b1;
        unpack_f32x2(la, a0, a1);
        unpack_f32x2(lb, b0, b1);
        l += (a0 + a1) + (b0 + b1);
      }
    }

    // the last tile's scale is the row's final one
    if (NK > 0) {
      const int last = NK - 1;
      if ((last & 1) != G) {
        if (ok) ok = mbar_wait(&m_ready[quarter * 2 + (last & 1)], (last >> 1) & 1, abort_flag, p.status);
        const float m_fin = m_pub[(last & 1) * TILE + r];
        if (m_fin != m_mine) { l = (l == 0.f) ? 0.f : l * exp2f(m_mine - m_fin); m_mine = m_fin; }
      }
      if (ok) ok = mbar_wait(o_final, 0, abort_flag, p.status);
    }
    tc_fence_after();
    xch[G * TILE + r] = l;
    asm volatile("bar.sync %0, 64;" ::"r"(1 + quarter) : "memory");
    const float inv = 1.0f / (l + xch[(G ^ 1) * TILE + r]);
    if (ok) {
      bf16 *dst = p.out + (size_t)row * p.h * D + (size_t)my_head * D;
#pragma unroll 1
      for (int q = G; q < D / 32; q += 2) {
        uint32_t o[32];
        tmem_ld32(o_addr + q * 32, o);
        tmem_wait_ld();
        if (row < p.n_tok) {
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
    }
  }

  // Neither CTA may leave (or free tensor memory the pair's instructions use) before both are done.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  if (warp == 9) {
    __syncwarp();
    tmem2_dealloc(tmem_base, 512);
  }
  // Neither CTA leaves before BOTH have released the pair's tensor memory: if one SM were handed to
  // another kernel's CTA while the partner's release (a cta_group::2 operation) is still to come,
  // that release could reach the newcomer's allocation.
  cluster_sync_all();
}

}  // namespace

bool attention_tc2_supported(int n_tok, int h, int h_kv, int d) {
  return d == 128 && n_tok >= 64 && h % h_kv == 0;
}

// map_q: 2-D {h*d, rows}, box {64, 128}; map_k: 3-D {d, cap, h_kv}, box {64, 64, 1};
// map_v: 3-D {d, cap, h_kv}, box {64, 128, 1}.
cudaError_t launch_attention_tc2(const CUtensorMap *map_q, const CUtensorMap *map_k, const CUtensorMap *map_v,
                                 bf16 *out, int n_tok, int h, int h_kv, int d, int len, int *status,
                                 cudaStream_t st, const PerHead *len_m) {
  if (d != D) return cudaErrorInvalidValue;
  Attn2Params p;
  p.out = out; p.n_tok = n_tok; p.h = h; p.h_kv = h_kv; p.len = len;
  p.per_head = len_m ? 1 : 0;
  p.len_m = len_m ? *len_m : PerHead{};
  p.pair_heads = ((h / h_kv) % 2 == 0) ? 1 : 0;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  p.status = status;
  const int n_rb = (n_tok + TILE - 1) / TILE;
  const int pairs = p.pair_heads ? n_rb * (h / 2) : ((n_rb + 1) / 2) * h;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(attn_tc2_kernel, A2_SMEM, attr_set); e != cudaSuccess) return e;
  attn_tc2_kernel<<<2 * pairs, A2_THREADS, A2_SMEM, st>>>(*map_q, *map_k, *map_v, p);
  return cudaGetLastError();
}

}  // namespace locret
