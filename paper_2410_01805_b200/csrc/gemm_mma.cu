// General-shape bf16 GEMM on warp-level tensor-core instructions (mma.sync m16n8k16),
// used for shapes the tcgen05 kernels do not take (small or ragged problems, decode).
//   MODE 0: C = A · Bt^T, bf16 store                       (QKV projection)
//   MODE 1: retaining head: act(A · W1t^T) · W2 summed over this CTA's 128 columns,
//           written as one partial score per (N-tile, row, KV head)   (Section 3.3)
#include "common.cuh"

namespace locret {

namespace {

constexpr int BM = 128, BN = 128, BK = 32, STAGES = 3, PAD = 8;
constexpr int LDS = BK + PAD;  // shared-memory row pitch in elements (80 bytes)
constexpr int THREADS = 256;
constexpr int PIPE_BYTES = STAGES * (BM + BN) * LDS * 2;
constexpr int ACT_LD = BN + 1;
constexpr int MAX_HKV = 32;

template <int MODE>
__global__ void __launch_bounds__(THREADS)
gemm_mma_kernel(const bf16 *__restrict__ A, int lda, const bf16 *__restrict__ Bt, int ldb,
                bf16 *__restrict__ C, int ldc, int M, int N, int K,
                const float *__restrict__ W2, float *__restrict__ partial, int h_kv, int act) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16 *sA = reinterpret_cast<bf16 *>(smem_raw);
  bf16 *sB = sA + STAGES * BM * LDS;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = warp >> 2, wn = warp & 3;  // 2 x 4 warps, warp tile 64 x 32
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;

  float acc[4][4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++)
#pragma unroll
      for (int k = 0; k < 4; k++) acc[i][j][k] = 0.f;

  const int KT = K / BK;

  auto load_stage = [&](int stage, int kt) {
    // 128 rows x 32 elements = 128 x 4 vectors of 16 bytes per operand; 256 threads x 2
#pragma unroll
    for (int it = 0; it < 2; it++) {
      int v = tid + it * THREADS;
      int r = v >> 2, c = (v & 3) * 8;
      int gr = m0 + r;
      cp_async16(sA + (stage * BM + r) * LDS + c, A + (size_t)min(gr, M - 1) * lda + kt * BK + c,
                 gr < M);
      int gn = n0 + r;
      cp_async16(sB + (stage * BN + r) * LDS + c, Bt + (size_t)min(gn, N - 1) * ldb + kt * BK + c,
                 gn < N);
    }
  };

#pragma unroll
  for (int s = 0; s < STAGES - 1; s++) {
    if (s < KT) load_stage(s, s);
    cp_async_commit();
  }

  for (int kt = 0; kt < KT; kt++) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    {
      int nk = kt + STAGES - 1;
      if (nk < KT) load_stage(nk % STAGES, nk);
      cp_async_commit();
    }
    const bf16 *a_s = sA + (kt % STAGES) * BM * LDS;
    const bf16 *b_s = sB + (kt % STAGES) * BN * LDS;
#pragma unroll
    for (int kk = 0; kk < BK; kk += 16) {
      uint32_t af[4][4], bfr[4][2];
#pragma unroll
      for (int i = 0; i < 4; i++) {
        int r = wm * 64 + i * 16 + (lane & 15);
        int c = kk + (lane >> 4) * 8;
        ldmatrix_x4(af[i][0], af[i][1], af[i][2], af[i][3], a_s + r * LDS + c);
      }
#pragma unroll
      for (int j = 0; j < 2; j++) {
        int id = lane >> 3;
        int r = wn * 32 + j * 16 + (id >> 1) * 8 + (lane & 7);
        int c = kk + (id & 1) * 8;
        ldmatrix_x4(bfr[2 * j][0], bfr[2 * j][1], bfr[2 * j + 1][0], bfr[2 * j + 1][1],
                    b_s + r * LDS + c);
      }
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) mma_bf16_16816(acc[i][j], af[i], bfr[j][0], bfr[j][1]);
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  const int g = lane >> 2, q = lane & 3;
  if (MODE == 0) {
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) {
        int col = n0 + wn * 32 + j * 8 + q * 2;
#pragma unroll
        for (int hh = 0; hh < 2; hh++) {
          int row = m0 + wm * 64 + i * 16 + g + hh * 8;
          if (row < M) {
            float v0 = acc[i][j][hh * 2], v1 = acc[i][j][hh * 2 + 1];
            if (col + 1 < N && (ldc & 1) == 0) {
              *reinterpret_cast<uint32_t *>(C + (size_t)row * ldc + col) = pack_bf16(v0, v1);
            } else {
              if (col < N) C[(size_t)row * ldc + col] = __float2bfloat16_rn(v0);
              if (col + 1 < N) C[(size_t)row * ldc + col + 1] = __float2bfloat16_rn(v1);
            }
          }
        }
      }
  } else {
    // activation tile to shared memory (fp32), then row x head dot products with W2
    float *sAct = reinterpret_cast<float *>(smem_raw);
    float *sW2 = sAct + BM * ACT_LD;  // [BN][h_kv]
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int j = 0; j < 4; j++)
#pragma unroll
        for (int e = 0; e < 4; e++) {
          int r = wm * 64 + i * 16 + g + (e >> 1) * 8;
          int c = wn * 32 + j * 8 + q * 2 + (e & 1);
          sAct[r * ACT_LD + c] = (n0 + c < N) ? apply_act(acc[i][j][e], act) : 0.f;
        }
    for (int v = tid; v < BN * h_kv; v += THREADS) {
      int c = v / h_kv;
      sW2[v] = (n0 + c < N) ? W2[(size_t)(n0 + c) * h_kv + (v - c * h_kv)] : 0.f;
    }
    __syncthreads();
    const int row = tid & (BM - 1), half = tid >> 7;
    const int per = (h_kv + 1) / 2;
    const int mb = half * per;
    const int cnt = min(per, h_kv - mb);
    float s[MAX_HKV / 2];
#pragma unroll
    for (int m = 0; m < MAX_HKV / 2; m++) s[m] = 0.f;
    for (int c = 0; c < BN; c++) {
      float a = sAct[row * ACT_LD + c];
#pragma unroll
      for (int m = 0; m < MAX_HKV / 2; m++)
        if (m < cnt) s[m] += a * sW2[c * h_kv + mb + m];
    }
    if (m0 + row < M) {
      float *dst = partial + ((size_t)blockIdx.x * M + (m0 + row)) * h_kv + mb;
#pragma unroll
      for (int m = 0; m < MAX_HKV / 2; m++)
        if (m < cnt) dst[m] = s[m];
    }
  }
}

__global__ void rh_reduce_kernel(const float *__restrict__ partial, int n_tiles, int M, int h_kv,
                                 float *__restrict__ scores, int score_stride, int slot0, int per_head,
                                 PerHead slot0_m) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= M * h_kv) return;
  int t = i / h_kv, m = i - t * h_kv;
  float s = 0.f;
  for (int nt = 0; nt < n_tiles; nt++) s += partial[((size_t)nt * M + t) * h_kv + m];
  scores[(size_t)m * score_stride + (per_head ? slot0_m.v[m] : slot0) + t] = s;
}

constexpr int rh_smem_bytes(int h_kv) {
  return (BM * ACT_LD + BN * h_kv) * 4 > PIPE_BYTES ? (BM * ACT_LD + BN * h_kv) * 4 : PIPE_BYTES;
}

}  // namespace

int rh_num_tiles(int d_R) { return (d_R + BN - 1) / BN; }

cudaError_t launch_gemm_bf16(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc,
                             int M, int N, int K, cudaStream_t st) {
  if (K % BK != 0 || (lda % 8) || (ldb % 8)) return cudaErrorInvalidValue;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(gemm_mma_kernel<0>, PIPE_BYTES, attr_set); e != cudaSuccess) return e;
  dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM);
  gemm_mma_kernel<0><<<grid, THREADS, PIPE_BYTES, st>>>(A, lda, Bt, ldb, C, ldc, M, N, K, nullptr,
                                                         nullptr, 0, 0);
  return cudaGetLastError();
}

cudaError_t launch_rh_gemm(const bf16 *A, int lda, const bf16 *W1t, const float *W2, float *partial,
                           int M, int d_R, int K, int h_kv, int act, int *n_tiles, cudaStream_t st) {
  if (K % BK != 0 || (lda % 8) || h_kv > MAX_HKV) return cudaErrorInvalidValue;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(gemm_mma_kernel<1>, rh_smem_bytes(MAX_HKV), attr_set); e != cudaSuccess)
    return e;
  dim3 grid((d_R + BN - 1) / BN, (M + BM - 1) / BM);
  *n_tiles = grid.x;
  gemm_mma_kernel<1><<<grid, THREADS, rh_smem_bytes(MAX_HKV), st>>>(
      A, lda, W1t, K, nullptr, 0, M, d_R, K, W2, partial, h_kv, act);
  return cudaGetLastError();
}

cudaError_t launch_rh_reduce(const float *partial, int n_tiles, int M, int h_kv, float *scores,
                             int score_stride, int slot0, cudaStream_t st, const PerHead *slot0_m) {
  int total = M * h_kv;
  rh_reduce_kernel<<<(total + 255) / 256, 256, 0, st>>>(partial, n_tiles, M, h_kv, scores, score_stride, slot0,
                                                        slot0_m ? 1 : 0, slot0_m ? *slot0_m : PerHead{});
  return cudaGetLastError();
}

}  // namespace locret
