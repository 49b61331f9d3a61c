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
#include "tc_common.cuh"


namespace locret {

namespace {

using namespace tc;

constexpr int AT_THREADS = 384;  // 3 warpgroups: softmax (two), {TMA, 2 MMA issuers, 1 idle warp}
constexpr int TILE = 128;               // query rows per tile and keys per tile
constexpr int HD = 128;                 // column pitch of a head in shared and tensor memory
constexpr int HALF_BYTES = TILE * 128;  // one 64-column swizzled box of 128 rows: 16 KB
constexpr int TILE_BYTES = 2 * HALF_BYTES;
constexpr int AT_SMEM = 1024 + 6 * TILE_BYTES + 256 + 2048;  // Q0,Q1,K0,K1,V0,V1 + barriers + softmax exchange
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
  int per_head;   // a budget per head: KV head m holds len_m.v[m] retained units
  PerHead len_m;
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
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 17);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = p.h / p.h_kv;
  const int n_rb = (p.n_tok + TILE - 1) / TILE;

  // which two query tiles; longest key ranges first
  int row0[2], head[2];
  if (p.pair_heads) {
    const int hp = p.h / 2;
    const int rb = n_rb - 1 - (int)blockIdx.x / hp;
    const int hq = (int)blockIdx.x % hp;
    row0[0] = row0[1] = rb * TILE;
    head[0] = 2 * hq; head[1] = 2 * hq + 1;
  } else {
    const int n_rp = (n_rb + 1) / 2;
    const int rp = n_rp - 1 - (int)blockIdx.x / p.h;
    row0[0] = rp * 2 * TILE; row0[1] = row0[0] + TILE;
    head[0] = head[1] = (int)blockIdx.x % p.h;
  }
  const int kvh = head[0] / g;
  const int len = p.per_head ? p.len_m.v[kvh] : p.len;   // retained units of this KV head
  const int n = len + p.n_tok;
  int NK = (len + row0[1] + TILE + TILE - 1) / TILE;
  NK = min(NK, (n + TILE - 1) / TILE);
  // The softmax is order independent, so every CTA walks the key tiles that need no mask in its
  // own rotated order: CTAs of one KV head start together, and in a common order they would all
  // ask the L2 for the same K and V lines at the same moment (measured: 1.4x slower).
  const int NF = min(NK, (len + row0[0] + 1) / TILE);  // tiles fully visible to every row
  const int rot = NF > 0 ? (int)((blockIdx.x * 29u + 7u) % (unsigned)NF) : 0;
  auto tile_of = [&](int j) { int x = j + rot; return j < NF ? (x >= NF ? x - NF : x) : j; };

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; s++) {
      mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1);
      mbar_init(&k_empty[s], 2); mbar_init(&v_empty[s], 2);  // released by both MMA issuers
      mbar_init(&s_full[s], 1); mbar_init(&p_full[s], 4); mbar_init(&o_full[s], 1);
      mbar_init(&p_half[s], 4);
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

  if (warp >= 8) {
    setmaxnreg_dec<56>();
  if (warp == 11) {
    // idle warp of the third warpgroup
  } else if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      constexpr int nbox = (D + 63) / 64;  // 64-column boxes per head vector
      mbar_expect_tx(q_full, 2 * nbox * HALF_BYTES);
      for (int t = 0; t < 2; t++)
        for (int hh = 0; hh < nbox; hh++)
          tma_load_2d(sQ + t * TILE_BYTES + hh * HALF_BYTES, &map_q, head[t] * D + hh * 64, row0[t],
                      q_full);
      // L2 prefetch PF tiles ahead: the cache of a layer is not L2 resident when its chunk step
      // starts, and two stages of shared memory do not cover an HBM miss.
      auto prefetch_tile = [&](int j) {
        const int row = tile_of(j) * TILE;
        for (int hh = 0; hh < nbox; hh++) {
          tma_prefetch_3d(&map_k, hh * 64, row, kvh);
          tma_prefetch_3d(&map_v, hh * 64, row, kvh);
        }
      };
      for (int j = 0; j < min(PF, NK); j++) prefetch_tile(j);
      for (int j = 0; j < NK; j++) {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (j + PF < NK) prefetch_tile(j + PF);
        if (!mbar_wait(&k_empty[s], ph ^ 1, abort_flag, p.status)) break;
        mbar_expect_tx(&k_full[s], nbox * HALF_BYTES);
        for (int hh = 0; hh < nbox; hh++)
          tma_load_3d(sK + s * TILE_BYTES + hh * HALF_BYTES, &map_k, hh * 64, tile_of(j) * TILE, kvh, &k_full[s]);
        if (!mbar_wait(&v_empty[s], ph ^ 1, abort_flag, p.status)) break;
        mbar_expect_tx(&v_full[s], nbox * HALF_BYTES);
        for (int hh = 0; hh < nbox; hh++)
          tma_load_3d(sV + s * TILE_BYTES + hh * HALF_BYTES, &map_v, hh * 64, tile_of(j) * TILE, kvh, &v_full[s]);
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
      auto issue_s = [&](int ks) {
        const uint64_t b = ks ? dk1 : dk0;
#pragma unroll
        for (int kk = 0; kk < ksteps; kk++) {
          const uint64_t off = (uint64_t)(((kk >> 2) * HALF_BYTES + (kk & 3) * 32) >> 4);
          if (kk == 0) mma_ss_first(s_tmem, dq + off, b + off, idesc_qk);
          else mma_ss_acc(s_tmem, dq + off, b + off, idesc_qk);
        }
        mma_commit(&s_full[t]);
        mma_commit(&k_empty[ks]);
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
      bool ok = mbar_wait(q_full, 0, abort_flag, p.status);
      ok = ok && mbar_wait(&k_full[0], 0, abort_flag, p.status);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; j < NK && ok; j++) {
        const int sv = j & 1, sk = (j + 1) & 1;
        // The tiles from memory arrive long before P does: poll them first, so that nothing but
        // the MMAs themselves stands between P and the next S.
        ok = mbar_wait(&v_full[sv], (j >> 1) & 1, abort_flag, p.status);
        if (j + 1 < NK) ok = ok && mbar_wait(&k_full[sk], ((j + 1) >> 1) & 1, abort_flag, p.status);
        // O_t += P_t V_j
        ok = ok && mbar_wait(&p_half[t], j & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        issue_pv(sv, j > 0, 0);
        ok = mbar_wait(&p_full[t], j & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        issue_pv(sv, j > 0, 1);
        // S_t = Q_t K_{j+1}^T
        if (j + 1 < NK) {
          issue_s(sk);
        }
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
    float m_used[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    bool ok = true;
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quarter) : "memory"); };

    for (int j = 0; j < NK; j++) {
      // (no early exit: after a timed-out wait the pair still meets at its named barrier)
#pragma unroll
      for (int t = 0; t < 2; t++) {
        const int row = row0[t] + r;
        const int limit = len + row;  // last visible key
        const uint32_t s_addr = tmem_base + lane_off + t * TILE;
        const uint32_t o_addr = tmem_base + lane_off + 2 * TILE + t * HD;
        if (ok) ok = mbar_wait(&s_full[t], j & 1, abort_flag, p.status);
        tc_fence_after();
        uint32_t s[64];
        tmem_ld32(s_addr + hf * 64, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tmem_ld32(s_addr + hf * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tmem_wait_ld();

        const int key0 = tile_of(j) * TILE;
        float tmax;
        if (key0 + TILE - 1 > len + row0[t]) {  // a tile that crosses the causal boundary
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
        tmax = fmaxf(tmax, xch[(t * 2 + (hf ^ 1)) * TILE + r]) * c;

        if (j == 0) {
          m_used[t] = tmax;
        } else {
          // both warps of the pair see the same maxima, hence take the same branch
          const bool need = tmax > m_used[t] + RESCALE_LOG2;
          if (__any_sync(0xffffffffu, need)) {
            // the accumulator must hold every product issued so far before it is rescaled
            if (ok) ok = mbar_wait(&o_full[t], (j - 1) & 1, abort_flag, p.status);
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

#pragma unroll
    for (int t = 0; t < 2; t++) {
      const int row = row0[t] + r;
      const uint32_t o_addr = tmem_base + lane_off + 2 * TILE + t * HD;
      if (ok && NK > 0) ok = mbar_wait(&o_full[t], (NK - 1) & 1, abort_flag, p.status);
      tc_fence_after();
      xch[(t * 2 + hf) * TILE + r] = l[t];
      pair_sync();
      const float inv = 1.0f / (l[t] + xch[(t * 2 + (hf ^ 1)) * TILE + r]);
      if (ok) {
        bf16 *dst = p.out + (size_t)row * p.h * D + (size_t)head[t] * D;
#pragma unroll 1
        for (int q = hf; q < D / 32; q += 2) {
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

// map_k / map_v: 3-D maps {d, cap, h_kv} with box {64, 128, 1}; map_q: 2-D {h*d, rows} box {64, 128}.
template <int D>
static cudaError_t launch_attn_d(const CUtensorMap *map_q, const CUtensorMap *map_k, const CUtensorMap *map_v,
                                 const AttnParams &p, int grid, cudaStream_t st) {
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(attn_tc_kernel<D>, AT_SMEM, attr_set); e != cudaSuccess) return e;
  attn_tc_kernel<D><<<grid, AT_THREADS, AT_SMEM, st>>>(*map_q, *map_k, *map_v, p);
  return cudaGetLastError();
}

cudaError_t launch_attention_tc(const CUtensorMap *map_q, const CUtensorMap *map_k,
                                const CUtensorMap *map_v, bf16 *out, int n_tok, int h, int h_kv, int d,
                                int len, int *status, cudaStream_t st, const PerHead *len_m) {
  AttnParams p;
  p.out = out; p.n_tok = n_tok; p.h = h; p.h_kv = h_kv; p.d = d; p.len = len;
  p.per_head = len_m ? 1 : 0;
  p.len_m = len_m ? *len_m : PerHead{};
  p.pair_heads = ((h / h_kv) % 2 == 0) ? 1 : 0;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  p.status = status;
  const int n_rb = (n_tok + TILE - 1) / TILE;
  const int grid = p.pair_heads ? n_rb * (h / 2) : ((n_rb + 1) / 2) * h;
  switch (d) {
    case 64: return launch_attn_d<64>(map_q, map_k, map_v, p, grid, st);
    case 96: return launch_attn_d<96>(map_q, map_k, map_v, p, grid, st);
    case 128: return launch_attn_d<128>(map_q, map_k, map_v, p, grid, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace locret
