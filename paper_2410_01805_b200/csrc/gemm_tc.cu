// bf16 GEMM on tcgen05 tensor cores: C[M x N] = A[M x K] · Bt[N x K]^T, fp32 accumulation in
// tensor memory.  One CTA computes a 128 x BN tile: warp 0 feeds shared memory with TMA
// (128-byte swizzled K-blocks of 64), warp 1 issues tcgen05.mma, warps 2..5 read the
// accumulator from TMEM and run the epilogue:
//   MODE 0: bf16 store (the QKV projection);
//   MODE 1: the retaining head's activation and its second, thin GEMM with W2, written as one
//           partial score per (N-tile, row, KV head)                       (Section 3.3).
#include <cstring>
#include "tc_common.cuh"

namespace locret {

// ------------------------------------------------------------------ tensor-map encoding (host)
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}
}  // namespace

bool tmap_encode_2d_bf16(CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer,
                         uint64_t outer_stride_bytes, uint32_t box_inner, uint32_t box_outer) {
  EncodeTiledFn fn = get_encode();
  if (!fn) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {outer_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tmap_encode_3d_bf16(CUtensorMap *map, const void *base, uint64_t d0, uint64_t d1, uint64_t d2,
                         uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1,
                         uint32_t b2) {
  EncodeTiledFn fn = get_encode();
  if (!fn) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {b0, b1, b2};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

using namespace tc;

constexpr int BM = 128, BK = 64, GT_THREADS = 192;
constexpr int MAX_HKV = 32;
constexpr int EPI_WARP_BYTES = 32 * 128 * 2;  // 32 rows of a head of up to 128 bf16

// sigma of the retaining head with the fast division / exponential intrinsics (relative error
// ~1e-6, far inside the score tolerance)
__device__ __forceinline__ float fast_act(float x, int act) {
  if (act == 0) return __fdividef(x, 1.0f + __expf(-x));
  return apply_act(x, act);
}

template <int BN>
struct GemmCfg {
  static constexpr int STAGES = BN >= 192 ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int TMEM_COLS = BN == 192 ? 512 : 2 * BN;  // two accumulators; a power of two
  static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int W2_BYTES = BN * MAX_HKV * 4;
  static constexpr int EPI_BYTES = 4 * EPI_WARP_BYTES;  // MODE 2: one staged head of 32 rows per warp
  // 1024 for alignment slack, barriers + tmem pointer in a small tail
  static constexpr int smem_bytes(int mode) {
    return 1024 + STAGES * STAGE_BYTES + (mode == 1 ? W2_BYTES : (mode == 2 ? EPI_BYTES : 0)) + 256;
  }
};

template <int BN, int MODE, int HD = 0>
__global__ void __launch_bounds__(GT_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               bf16 *__restrict__ C, int ldc, int M, int N, int K, const float *__restrict__ W2,
               float *__restrict__ partial, int h_kv, int act, const RopeAppendArgs ra,
               const bf16 *__restrict__ resid, int ldr, int n_major, int *status) {
  // Persistent: CTA b computes tiles b, b + gridDim.x, ... (row-block major, so that concurrent
  // CTAs share the A row block in L2).  The accumulator is double-buffered in TMEM: the epilogue
  // of one tile overlaps the main loop of the next.
  using Cfg = GemmCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  unsigned char *tiles = smem;
  float *sW2 = reinterpret_cast<float *>(tiles + STAGES * Cfg::STAGE_BYTES);
  unsigned char *sEpi = tiles + STAGES * Cfg::STAGE_BYTES;
  unsigned char *tail = tiles + STAGES * Cfg::STAGE_BYTES +
                        (MODE == 1 ? Cfg::W2_BYTES : (MODE == 2 ? Cfg::EPI_BYTES : 0));
  uint64_t *full = reinterpret_cast<uint64_t *>(tail);
  uint64_t *empty = full + STAGES;
  uint64_t *acc_full = empty + STAGES;   // [2]
  uint64_t *acc_empty = acc_full + 2;    // [2]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // K-blocks of 64; a last partial block reads past the operands' inner extent, where TMA fills zeros
  const int KB = (K + BK - 1) / BK;
  const int tiles_n = (N + BN - 1) / BN;
  const int tiles_m = (M + BM - 1) / BM;
  const int total = tiles_m * tiles_n;
  // tile order: row-block major (concurrent CTAs share the A row block in L2), or, when B is the
  // large operand and does not fit the L2, column-block major (they share the B tile and sweep M)
  auto tile_mn = [&](int tile, int &m0, int &n0) {
    if (n_major) { m0 = (tile % tiles_m) * BM; n0 = (tile / tiles_m) * BN; }
    else { m0 = (tile / tiles_n) * BM; n0 = (tile % tiles_n) * BN; }
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&map_a);
    prefetch_tmap(&map_b);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
        int m0, n0;
        tile_mn(tile, m0, n0);
        for (int kb = 0; kb < KB; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          ok = mbar_wait(&empty[s], ph ^ 1, abort_flag, status);
          if (!ok) break;
          mbar_expect_tx(&full[s], Cfg::STAGE_BYTES);
          unsigned char *a_dst = tiles + s * Cfg::STAGE_BYTES;
          tma_load_2d(a_dst, &map_a, kb * BK, m0, &full[s]);
          tma_load_2d(a_dst + Cfg::A_BYTES, &map_b, kb * BK, n0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(BM, BN, 0, 0);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x, lt++) {
        const uint32_t buf = lt & 1;
        ok = mbar_wait(&acc_empty[buf], ((lt >> 1) & 1) ^ 1, abort_flag, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < KB; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          ok = mbar_wait(&full[s], ph, abort_flag, status);
          if (!ok) break;
          tc_fence_after();
          unsigned char *a_src = tiles + s * Cfg::STAGE_BYTES;
          const uint64_t da = desc_kmajor_sw128(a_src), db = desc_kmajor_sw128(a_src + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; k++) {
            if (kb == 0 && k == 0) mma_ss_first(d_tmem, da, db, idesc);
            else mma_ss_acc(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc);
          }
          mma_commit(&empty[s]);  // frees the stage once these MMAs have read it
        }
        if (ok) mma_commit(&acc_full[buf]);
      }
    }
  } else {
    // epilogue warps 2..5: TMEM lane quarter = warp % 4
    const int quarter = warp & 3;
    const int etid = threadIdx.x - 64;  // 0..127 among the epilogue threads
    uint32_t lt = 0;
    bool ok = true;
    // (no early exit: after a timed-out wait the warps still meet at the named barrier)
    for (int tile = blockIdx.x; tile < total; tile += gridDim.x, lt++) {
      int m0, n0;
      tile_mn(tile, m0, n0);
      const uint32_t buf = lt & 1;
      const int row = m0 + quarter * 32 + lane;
      if (MODE == 1) {
        // this tile's slice of W2; the named barrier keeps the four warps together around it
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int v = etid; v < BN * h_kv; v += 128) {
          int c = v / h_kv;
          sW2[v] = (n0 + c < N) ? W2[(size_t)(n0 + c) * h_kv + (v - c * h_kv)] : 0.f;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
      // MODE 2: (cos, sin) of this thread's position for every rotation pair, fetched while the
      // tile's MMAs are still running
      float4 csr[MODE == 2 ? HD / 4 : 1];
      if (MODE == 2) {
        const float4 *cs4 = reinterpret_cast<const float4 *>(ra.cs + (size_t)(ra.len + row) * (HD / 2));
#pragma unroll
        for (int i = 0; i < HD / 4; i++) csr[i] = row < M ? __ldg(cs4 + i) : make_float4(1.f, 0.f, 1.f, 0.f);
      }
      if (ok) ok = mbar_wait(&acc_full[buf], (lt >> 1) & 1, abort_flag, status);
      tc_fence_after();
      const uint32_t taddr = tmem_base + buf * BN + ((uint32_t)(quarter * 32) << 16);
      if (MODE == 0) {
        if (ok) {
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(taddr + c0, r);
            tmem_wait_ld();
            if (row < M && n0 + c0 < N) {
              uint4 *dst = reinterpret_cast<uint4 *>(C + (size_t)row * ldc + n0 + c0);
              const uint4 *rs = resid ? reinterpret_cast<const uint4 *>(resid + (size_t)row * ldr + n0 + c0) : nullptr;
#pragma unroll
              for (int v = 0; v < 4; v++) {
                float f[8];
#pragma unroll
                for (int e = 0; e < 8; e++) f[e] = __uint_as_float(r[8 * v + e]);
                if (rs) {  // C = A B^T + R (a residual connection), rounded once
                  const uint4 rv = rs[v];
                  const uint32_t w[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
                  for (int e = 0; e < 4; e++) {
                    f[2 * e] += __uint_as_float(w[e] << 16);
                    f[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                  }
                }
                uint4 o;
                o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]);
                o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
                dst[v] = o;
              }
            }
          }
        }
      } else if (MODE == 5) {
        // plain GEMM with an fp32 result (gradients): C is a float array, ldc in floats
        if (ok) {
          float *Cf = reinterpret_cast<float *>(C);
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(taddr + c0, r);
            tmem_wait_ld();
            if (row < M && n0 + c0 < N) {
              float4 *dst = reinterpret_cast<float4 *>(Cf + (size_t)row * ldc + n0 + c0);
#pragma unroll
              for (int v = 0; v < 8; v++)
                dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                     __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
            }
          }
        }
      } else if (MODE == 6) {
        // Heads divided over GPUs: this GPU's partial product is ADDED into the sum buffer of every
        // GPU (`partial` holds h_kv = n_peers device pointers to fp32 [M x ldc] buffers, which may be
        // other GPUs' memory mapped into this process).  Plain reductions to global memory at system
        // scope, 16 bytes each: no TMA and no multicast touches a peer's memory.
        if (ok) {
          float *const *peers = reinterpret_cast<float *const *>(partial);
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(taddr + c0, r);
            tmem_wait_ld();
            if (row < M && n0 + c0 < N) {
              for (int pe = 0; pe < h_kv; pe++) {
                float *dst = peers[pe] + (size_t)row * ldc + n0 + c0;
#pragma unroll
                for (int v = 0; v < 8; v++)
                  asm volatile("red.relaxed.sys.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4 * v),
                               "f"(__uint_as_float(r[4 * v])), "f"(__uint_as_float(r[4 * v + 1])),
                               "f"(__uint_as_float(r[4 * v + 2])), "f"(__uint_as_float(r[4 * v + 3]))
                               : "memory");
              }
            }
          }
        }
      } else if (MODE == 4) {
        // Row maximum of A B^T over the valid columns, merged into out[row] with an atomic
        // maximum on the order-preserving integer image of the float (`partial` is the output,
        // `act` carries the bits of the scale factor): the labels of Section 3.3.
        if (ok) {
          const float scale = __int_as_float(act);
          float mx = -INFINITY;
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(taddr + c0, r);
            tmem_wait_ld();
            if (n0 + c0 < N) {
#pragma unroll
              for (int i = 0; i < 32; i++)
                if (n0 + c0 + i < N) mx = fmaxf(mx, __uint_as_float(r[i]));
            }
          }
          if (row < M && mx > -INFINITY) {
            mx *= scale;
            if (mx == 0.f) mx = 0.f;  // -0 would order below every negative as an integer
            float *dst = partial + row;
            if (mx >= 0.f) atomicMax(reinterpret_cast<int *>(dst), __float_as_int(mx));
            else atomicMin(reinterpret_cast<unsigned int *>(dst), __float_as_uint(mx));
          }
        }
      } else if (MODE == 3) {
        // Gated FFN: a 256-column tile holds 128 gate columns followed by the 128 up columns
        // of the same outputs (the weight rows are laid out that way when the block is
        // created); the epilogue stores silu(gate) * up, 128 outputs per tile.
        if (ok) {
#pragma unroll 1
          for (int c0 = 0; c0 < BN / 2; c0 += 32) {
            uint32_t gt[32], up[32];
            tmem_ld32(taddr + c0, gt);
            tmem_ld32(taddr + BN / 2 + c0, up);
            tmem_wait_ld();
            if (row < M && n0 + c0 < N) {
              uint4 *dst = reinterpret_cast<uint4 *>(C + (size_t)row * ldc + n0 / 2 + c0);
#pragma unroll
              for (int v = 0; v < 4; v++) {
                float f[8];
#pragma unroll
                for (int e = 0; e < 8; e++)
                  f[e] = fast_act(__uint_as_float(gt[8 * v + e]), 0) * __uint_as_float(up[8 * v + e]);
                uint4 o;
                o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]);
                o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
                dst[v] = o;
              }
            }
          }
        }
      } else if (MODE == 2) {
        // QKV projection with the chunk's positions, RoPE and cache append in the epilogue: a
        // tile holds BN / HD whole heads, so both halves (i, i + HD/2) of every rotation pair
        // are in this thread's TMEM row.  The rotation starts from the bf16-rounded projection,
        // the value the pre-RoPE cache stores.  Each warp stages its 32 rows of one head in
        // shared memory (16-byte pieces XOR-swizzled by row) and writes them out as whole rows,
        // so the global stores are full lines.
        if (ok) {
          // 16-byte pieces of a staged row: XOR-swizzled by row when their number is a power of
          // two, else rows padded by one piece (an odd stride in pieces spreads the banks as well)
          constexpr int HALF = HD / 2, VPR = HD / 8, VMASK = VPR - 1;
          constexpr bool POW2 = (VPR & (VPR - 1)) == 0;
          constexpr int ROW_B = POW2 ? HD * 2 : HD * 2 + 16;
          auto piece = [&](int j, int r) { return POW2 ? ((j ^ (r & VMASK)) << 4) : (j << 4); };
          const int d_in = (ra.h + 2 * ra.h_kv) * HD;
          const int wrow0 = m0 + quarter * 32;  // first row of this warp
          unsigned char *buf_w = sEpi + quarter * EPI_WARP_BYTES;
          unsigned char *my_row = buf_w + lane * ROW_B;
          // rows [wrow0, wrow0 + 32) of the staged head -> dst + r * stride (elements)
          auto copy_out = [&](bf16 *dst, size_t stride) {
#pragma unroll 4
            for (int i = 0; i < VPR; i++) {
              const int idx = lane + 32 * i, r = idx / VPR, j = idx % VPR;
              if (wrow0 + r < M)
                *reinterpret_cast<uint4 *>(dst + (size_t)r * stride + j * 8) =
                    *reinterpret_cast<const uint4 *>(buf_w + r * ROW_B + piece(j, r));
            }
          };
#pragma unroll 1
          for (int hc = 0; hc < BN; hc += HD) {
            const int col0 = n0 + hc;
            if (col0 >= N) break;
            const int hd = col0 / HD;
            const bool is_v = hd >= ra.h + ra.h_kv, is_k = !is_v && hd >= ra.h;
            const int m = is_v ? hd - ra.h - ra.h_kv : hd - ra.h;
            const size_t cache_off = ((size_t)m * ra.cap + ra.len + wrow0) * HD;
            // pass A: the projection as stored (staging, pre-RoPE key cache, value cache)
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
              uint32_t r[32];
              tmem_ld32(taddr + hc + c0, r);
              tmem_wait_ld();
#pragma unroll
              for (int v = 0; v < 4; v++) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(r[8 * v + 0]), __uint_as_float(r[8 * v + 1]));
                o.y = pack_bf16(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                o.z = pack_bf16(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                o.w = pack_bf16(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                *reinterpret_cast<uint4 *>(my_row + piece((c0 >> 3) + v, lane)) = o;
              }
            }
            __syncwarp();
            copy_out(C + (size_t)wrow0 * ldc + col0, ldc);
            if (is_v) {
              copy_out(ra.v + cache_off, HD);
              if (ra.z_post) copy_out(ra.z_post + (size_t)wrow0 * d_in + col0, d_in);
            } else if (is_k && ra.k_pre) {
              copy_out(ra.k_pre + cache_off, HD);
            }
            __syncwarp();
            if (is_v) continue;
            // pass B: rotated at position = slot
#pragma unroll
            for (int c0 = 0; c0 < HALF; c0 += 32) {
              uint32_t lo[32], hi[32];
              tmem_ld32(taddr + hc + c0, lo);
              tmem_ld32(taddr + hc + HALF + c0, hi);
              tmem_wait_ld();
#pragma unroll
              for (int v = 0; v < 4; v++) {
                if (c0 + 8 * v >= HALF) break;  // head_dim 96: the second load holds 16 columns of the half
                uint32_t ol[4], oh[4];
#pragma unroll
                for (int q = 0; q < 4; q++) {
                  const float4 t = csr[(c0 >> 1) + 4 * v + q];  // (cos, sin) of two pairs
                  const uint32_t wl = pack_bf16(__uint_as_float(lo[8 * v + 2 * q]), __uint_as_float(lo[8 * v + 2 * q + 1]));
                  const uint32_t wh = pack_bf16(__uint_as_float(hi[8 * v + 2 * q]), __uint_as_float(hi[8 * v + 2 * q + 1]));
                  const float x0 = __uint_as_float(wl << 16), x1 = __uint_as_float(wl & 0xffff0000u);
                  const float y0 = __uint_as_float(wh << 16), y1 = __uint_as_float(wh & 0xffff0000u);
                  // lower half: x cos − y sin ; upper half: y cos + x sin
                  ol[q] = pack_bf16(x0 * t.x - y0 * t.y, x1 * t.z - y1 * t.w);
                  oh[q] = pack_bf16(y0 * t.x + x0 * t.y, y1 * t.z + x1 * t.w);
                }
                const int jl = (c0 >> 3) + v, jh = jl + (HALF >> 3);
                *reinterpret_cast<uint4 *>(my_row + piece(jl, lane)) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
                *reinterpret_cast<uint4 *>(my_row + piece(jh, lane)) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
              }
            }
            __syncwarp();
            if (is_k) {
              copy_out(ra.k_rot + cache_off, HD);
              if (row < M) ra.tid[(size_t)m * ra.cap + ra.len + row] = ra.seen + row;
            } else {
              copy_out(ra.q_rot + (size_t)wrow0 * ra.h * HD + (size_t)hd * HD, (size_t)ra.h * HD);
            }
            if (ra.z_post) copy_out(ra.z_post + (size_t)wrow0 * d_in + col0, d_in);
            __syncwarp();
          }
        }
      } else {
        float sc[MAX_HKV];
#pragma unroll
        for (int m = 0; m < MAX_HKV; m++) sc[m] = 0.f;
        if (ok) {
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(taddr + c0, r);
            tmem_wait_ld();
            // activation of the 32 columns first (independent, so the special-function unit
            // pipelines them), then the thin GEMM with W2 as broadcast 16-byte loads
            float a[32];
#pragma unroll
            for (int i = 0; i < 32; i++) a[i] = fast_act(__uint_as_float(r[i]), act);
            if (h_kv == 8) {
#pragma unroll
              for (int i = 0; i < 32; i++) {
                const float4 w0 = *reinterpret_cast<const float4 *>(sW2 + (c0 + i) * 8);
                const float4 w1 = *reinterpret_cast<const float4 *>(sW2 + (c0 + i) * 8 + 4);
                sc[0] = fmaf(a[i], w0.x, sc[0]); sc[1] = fmaf(a[i], w0.y, sc[1]);
                sc[2] = fmaf(a[i], w0.z, sc[2]); sc[3] = fmaf(a[i], w0.w, sc[3]);
                sc[4] = fmaf(a[i], w1.x, sc[4]); sc[5] = fmaf(a[i], w1.y, sc[5]);
                sc[6] = fmaf(a[i], w1.z, sc[6]); sc[7] = fmaf(a[i], w1.w, sc[7]);
              }
            } else if (h_kv == 32) {
#pragma unroll
              for (int i = 0; i < 32; i++) {
                const float4 *w = reinterpret_cast<const float4 *>(sW2 + (c0 + i) * 32);
#pragma unroll
                for (int m4 = 0; m4 < 8; m4++) {
                  const float4 wv = w[m4];
                  sc[4 * m4 + 0] = fmaf(a[i], wv.x, sc[4 * m4 + 0]);
                  sc[4 * m4 + 1] = fmaf(a[i], wv.y, sc[4 * m4 + 1]);
                  sc[4 * m4 + 2] = fmaf(a[i], wv.z, sc[4 * m4 + 2]);
                  sc[4 * m4 + 3] = fmaf(a[i], wv.w, sc[4 * m4 + 3]);
                }
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; i++) {
                const float *w = sW2 + (c0 + i) * h_kv;
#pragma unroll
                for (int m = 0; m < MAX_HKV; m++)
                  if (m < h_kv) sc[m] = fmaf(a[i], w[m], sc[m]);
              }
            }
          }
          if (row < M) {
            float *dst = partial + ((size_t)(n0 / BN) * M + row) * h_kv;
#pragma unroll
            for (int m = 0; m < MAX_HKV; m++)
              if (m < h_kv) dst[m] = sc[m];
          }
        }
      }
      // every tcgen05.ld of this warp has completed (wait::ld above): the buffer may be reused
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

struct MapCache {
  const void *base = nullptr;
  uint64_t inner = 0, outer = 0, stride = 0;
  uint32_t box_outer = 0;
  CUtensorMap map;
};

// Small per-thread cache of encoded maps (weights and staging buffers repeat every call).
const CUtensorMap *cached_map(const void *base, uint64_t inner, uint64_t outer, uint64_t stride_bytes,
                              uint32_t box_outer) {
  constexpr int SLOTS = 256;
  static thread_local MapCache cache[SLOTS];
  static thread_local int next = 0;
  for (int i = 0; i < SLOTS; i++) {
    MapCache &c = cache[i];
    if (c.base == base && c.inner == inner && c.outer == outer && c.stride == stride_bytes &&
        c.box_outer == box_outer)
      return &c.map;
  }
  MapCache &c = cache[next];
  next = (next + 1) % SLOTS;
  if (!tmap_encode_2d_bf16(&c.map, base, inner, outer, stride_bytes, BK, box_outer)) {
    c.base = nullptr;
    return nullptr;
  }
  c.base = base; c.inner = inner; c.outer = outer; c.stride = stride_bytes; c.box_outer = box_outer;
  return &c.map;
}

template <int BN, int MODE, int HD = 0>
cudaError_t launch_t(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M, int N,
                     int K, const float *W2, float *partial, int h_kv, int act, const RopeAppendArgs &ra,
                     int *status, cudaStream_t st, const bf16 *resid = nullptr, int ldr = 0) {
  using Cfg = GemmCfg<BN>;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(gemm_tc_kernel<BN, MODE, HD>, Cfg::smem_bytes(MODE), attr_set);
      e != cudaSuccess)
    return e;
  const CUtensorMap *ma = cached_map(A, K, M, (uint64_t)lda * 2, BM);
  const CUtensorMap *mb = cached_map(Bt, K, N, (uint64_t)ldb * 2, BN);
  if (!ma || !mb) return cudaErrorInvalidValue;
  const int num_sms = sm_count_of_current_device();
  const int total = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
  const int grid = total < num_sms ? total : num_sms;
  // B is the larger operand: keep a B tile resident and sweep the rows (each B tile is then read
  // from HBM once; in row-block-major order a B that exceeds the L2 is re-read for every row
  // block, and even one that fits is read about three times)
  const size_t a_bytes = (size_t)M * K * 2, b_bytes = (size_t)N * K * 2;
  const int n_major = MODE != 1 && b_bytes > a_bytes;  // (MODE 1 indexes its partial sums by column tile either way)
  gemm_tc_kernel<BN, MODE, HD><<<grid, GT_THREADS, Cfg::smem_bytes(MODE), st>>>(
      *ma, *mb, C, ldc, M, N, K, W2, partial, h_kv, act, ra, resid, ldr, n_major, status);
  return cudaGetLastError();
}

}  // namespace

bool gemm_tc_supported(int M, int N, int K, int lda, int ldb) {
  return K % BK == 0 && N % 32 == 0 && lda % 8 == 0 && ldb % 8 == 0 && M >= 1;
}

cudaError_t launch_gemm_tc(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                           int N, int K, int *status, cudaStream_t st) {
  if (N >= 256)
    return launch_t<256, 0>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st);
  return launch_t<128, 0>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st);
}

// C = A Bt^T + R: a projection with its residual connection (R [M x N] bf16, leading dimension ldr)
cudaError_t launch_gemm_tc_resid(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                                 int N, int K, const bf16 *R, int ldr, int *status, cudaStream_t st) {
  if (N >= 256)
    return launch_t<256, 0>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status,
                            st, R, ldr);
  return launch_t<128, 0>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st,
                          R, ldr);
}

// Gated FFN first half: C[M x N/2] = silu(A Wg) * (A Wu), where Bt [N x K] holds, for every block
// of 128 outputs, the 128 rows of Wg^T followed by the 128 rows of Wu^T (N = 2 d_ff, d_ff % 128 == 0)
bool gemm_tc_gated_supported(int M, int N, int K, int lda, int ldb) {
  return gemm_tc_supported(M, N, K, lda, ldb) && N % 256 == 0;
}
cudaError_t launch_gemm_tc_gated(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                                 int N, int K, int *status, cudaStream_t st) {
  return launch_t<256, 3>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st);
}

// C (fp32, leading dimension ldc in floats) = A Bt^T
cudaError_t launch_gemm_tc_f32(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *C, int ldc, int M, int N,
                               int K, int *status, cudaStream_t st) {
  bf16 *Cb = reinterpret_cast<bf16 *>(C);
  if (N >= 256)
    return launch_t<256, 5>(A, lda, Bt, ldb, Cb, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st);
  return launch_t<128, 5>(A, lda, Bt, ldb, Cb, ldc, M, N, K, nullptr, nullptr, 0, 0, RopeAppendArgs{}, status, st);
}

// peers[p][m][n] += (A Bt^T)[m][n] for every p < n_peers (fp32 buffers with leading dimension ldc floats;
// `peers` is a DEVICE array of n_peers pointers)
cudaError_t launch_gemm_tc_f32_add_peers(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *const *peers,
                                         int n_peers, int ldc, int M, int N, int K, int *status, cudaStream_t st) {
  float *pl = reinterpret_cast<float *>(const_cast<float **>(peers));
  if (N >= 256)
    return launch_t<256, 6>(A, lda, Bt, ldb, nullptr, ldc, M, N, K, nullptr, pl, n_peers, 0, RopeAppendArgs{}, status, st);
  return launch_t<128, 6>(A, lda, Bt, ldb, nullptr, ldc, M, N, K, nullptr, pl, n_peers, 0, RopeAppendArgs{}, status, st);
}

// out[m] = max(out[m], scale * max_n (A Bt^T)[m][n]) for m < M (out fp32, initialised by the
// caller, e.g. to -inf); scale > 0.  K % 8 == 0 (a last K-block that is not full is zero-filled by
// TMA); any N.
cudaError_t launch_gemm_tc_rowmax(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *out, int M, int N,
                                  int K, float scale, int *status, cudaStream_t st) {
  int bits;
  memcpy(&bits, &scale, sizeof(bits));
  return launch_t<256, 4>(A, lda, Bt, ldb, nullptr, 0, M, N, K, nullptr, out, 0, bits, RopeAppendArgs{}, status, st);
}

// QKV projection whose epilogue also assigns positions, rotates Q and K and appends K, V to the
// cache (what rope_append_kernel does in a pass of its own): head_dim 64 or 128, so that a
// 256-column tile holds whole heads.
bool qkv_rope_tc_supported(int M, int N, int K, int lda, int ldb, int d) {
  if (d == 96) return gemm_tc_supported(M, N, K, lda, ldb) && N % 192 == 0;
  return gemm_tc_supported(M, N, K, lda, ldb) && N >= 256 && (d == 64 || d == 128) && N % d == 0;
}

cudaError_t launch_qkv_rope_tc(const bf16 *X, int ldx, const bf16 *Wt, int ldw, bf16 *staging, int M,
                               int N, int K, const RopeAppendArgs &ra, int *status, cudaStream_t st) {
  if (ra.d == 96)
    return launch_t<192, 2, 96>(X, ldx, Wt, ldw, staging, N, M, N, K, nullptr, nullptr, 0, 0, ra, status, st);
  if (ra.d == 128)
    return launch_t<256, 2, 128>(X, ldx, Wt, ldw, staging, N, M, N, K, nullptr, nullptr, 0, 0, ra, status, st);
  return launch_t<256, 2, 64>(X, ldx, Wt, ldw, staging, N, M, N, K, nullptr, nullptr, 0, 0, ra, status, st);
}

// Tile width of the retaining-head GEMM: the widest of 256 / 128 / 64 columns that divides d_R.  The
// kernel runs beside attention and the next projection, so what it costs the step is SM time, not
// latency, and a CTA's latency is set by the length of K whatever the width (measured at 1024 tokens,
// K = 9216: 128 / 64 / 32 CTAs for 70.6 / 76.4 / 87.7 us; the whole run is 4 % faster with the 32 wide ones).
static int rh_tile_n(int M, int d_R) {
  (void)M;
  if (d_R % 256 == 0) return 256;
  return d_R % 128 == 0 ? 128 : 64;
}
// upper bound on the number of N-tiles (scratch sizing)
int rh_tc_num_tiles(int d_R) { return (d_R + 63) / 64; }

cudaError_t launch_rh_gemm_tc(const bf16 *A, int lda, const bf16 *W1t, const float *W2, float *partial,
                              int M, int d_R, int K, int h_kv, int act, int *n_tiles, int *status,
                              cudaStream_t st) {
  const int bn = rh_tile_n(M, d_R);
  *n_tiles = (d_R + bn - 1) / bn;
  if (bn == 256)
    return launch_t<256, 1>(A, lda, W1t, K, nullptr, 0, M, d_R, K, W2, partial, h_kv, act, RopeAppendArgs{}, status, st);
  if (bn == 128)
    return launch_t<128, 1>(A, lda, W1t, K, nullptr, 0, M, d_R, K, W2, partial, h_kv, act, RopeAppendArgs{}, status, st);
  return launch_t<64, 1>(A, lda, W1t, K, nullptr, 0, M, d_R, K, W2, partial, h_kv, act, RopeAppendArgs{}, status, st);
}

}  // namespace locret
