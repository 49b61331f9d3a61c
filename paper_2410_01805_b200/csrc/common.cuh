// Shared device helpers and the launcher declarations of the library's kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace locret {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- small device helpers

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte async copy global -> shared; when !pred the destination is zero-filled.
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool pred) {
  uint32_t s = smem_u32(smem);
  int sz = pred ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3,
                                            const void *smem) {
  uint32_t s = smem_u32(smem);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(s));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2,
                                                  uint32_t &r3, const void *smem) {
  uint32_t s = smem_u32(smem);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(s));
}

// D (16x8 fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4],
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ float apply_act(float x, int act) {
  if (act == 0) return x / (1.0f + __expf(-x));  // SiLU
  if (act == 1) {                                // GELU, tanh form
    float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
    return 0.5f * x * (1.0f + tanhf(u));
  }
  return fmaxf(x, 0.0f);                         // ReLU
}

// ---------------------------------------------------------------- programmatic dependent launch
// Consecutive kernels of one stream launched with `pdl` may overlap: the later one starts once every
// CTA of the earlier one has called pdl_launch_dependents() (or exited) and runs up to its
// pdl_wait(), which returns when the earlier grid has completed and its writes are visible.  In a
// kernel launched the ordinary way both calls do nothing.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 bool pdl, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------- per-device launch state (host)
// cudaFuncSetAttribute acts on the current device only, so "already done" is remembered per
// device: one process may drive several GPUs.
constexpr int MAX_DEVICES = 64;
struct PerDeviceFlag { bool done[MAX_DEVICES] = {}; };

inline cudaError_t current_device_index(int *dev) {
  cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return e;
  return (*dev < 0 || *dev >= MAX_DEVICES) ? cudaErrorInvalidDevice : cudaSuccess;
}

// Raise a kernel's dynamic shared-memory limit once per device.
template <typename Kernel>
inline cudaError_t allow_dynamic_smem(Kernel kernel, int bytes, PerDeviceFlag &flag) {
  int dev = 0;
  cudaError_t e = current_device_index(&dev);
  if (e != cudaSuccess) return e;
  if (flag.done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) flag.done[dev] = true;
  return e;
}

// Number of SMs of the current device (148 if it cannot be read), looked up once per device.
inline int sm_count_of_current_device() {
  static int count[MAX_DEVICES] = {};
  int dev = 0;
  if (current_device_index(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
  if (count[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = 148;
    }
    count[dev] = n;
  }
  return count[dev];
}

// One value per KV head, handed to kernels by value (a layer has at most 32 KV heads).  Used when the
// heads have budgets of their own (Appendix H: heads evict independently): cache lengths, and with
// them append slots and positions, then differ from head to head.
struct PerHead { int v[32]; };

// ---------------------------------------------------------------- launchers (host)
// Every launcher enqueues on `st` and returns the cudaError_t of the launch.

// C[M x N] (bf16, row-major, leading dimension ldc) = A[M x K] · Bt[N x K]^T, both K-major bf16.
cudaError_t launch_gemm_bf16(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc,
                             int M, int N, int K, cudaStream_t st);

// Retaining head: partial[nt][M][h_kv] = sum over the N-tile nt of act(A·W1t^T)[:, n] * W2[n][:]
// A [M x K] bf16 (K = d_in), W1t [d_R x K] bf16, W2 [d_R x h_kv] fp32.  Returns the number of
// N-tiles through *n_tiles.
cudaError_t launch_rh_gemm(const bf16 *A, int lda, const bf16 *W1t, const float *W2, float *partial,
                           int M, int d_R, int K, int h_kv, int act, int *n_tiles, cudaStream_t st);
int rh_num_tiles(int d_R);

// The same two GEMMs on tcgen05 tensor cores (TMA-fed, TMEM accumulators); `status` is the
// layer's device status word (set if a bounded wait gives up).
bool gemm_tc_supported(int M, int N, int K, int lda, int ldb);
// the same GEMM with a residual added before the one rounding: C = A Bt^T + R
cudaError_t launch_gemm_tc_resid(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                                 int N, int K, const bf16 *R, int ldr, int *status, cudaStream_t st);
// first half of a gated FFN: C[M x N/2] = silu(A Wg) * (A Wu); Bt [N x K] interleaves, per block of
// 128 outputs, 128 rows of Wg^T and 128 rows of Wu^T
// out[m] = max(out[m], scale * max_n (A Bt^T)[m][n]): row maxima merged with atomics (out fp32,
// initialised by the caller); K % 64 == 0, lda / ldb multiples of 8, scale > 0
cudaError_t launch_gemm_tc_rowmax(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *out, int M, int N,
                                  int K, float scale, int *status, cudaStream_t st);
// C (fp32, leading dimension ldc in floats) = A Bt^T
// heads divided over GPUs: this GPU's partial first product of the retaining head (fallback for
// shapes the tensor-core GEMM does not take), and scores from the summed product
cudaError_t launch_preact_naive(const bf16 *z, const bf16 *W1t, float *pre, int n_tok, int d_R, int d_in,
                                cudaStream_t st);
cudaError_t launch_rh_finish(const float *pre, const float *w2, float *s, int score_stride, int slot0,
                             int n_tok, int d_R, int h_kv, int act, cudaStream_t st);
cudaError_t launch_gemm_tc_f32(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *C, int ldc, int M, int N,
                               int K, int *status, cudaStream_t st);
// the same product ADDED into n_peers fp32 buffers (device array of device pointers; the buffers may be
// other GPUs' memory): reductions to global memory at system scope, no TMA on peer memory
cudaError_t launch_gemm_tc_f32_add_peers(const bf16 *A, int lda, const bf16 *Bt, int ldb, float *const *peers,
                                         int n_peers, int ldc, int M, int N, int K, int *status, cudaStream_t st);
// peers[p][i] += src[i] for i < count (the fallback beside the GEMM above)
cudaError_t launch_add_to_peers(const float *src, float *const *peers, int n_peers, size_t count, cudaStream_t st);
bool gemm_tc_gated_supported(int M, int N, int K, int lda, int ldb);
cudaError_t launch_gemm_tc_gated(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                                 int N, int K, int *status, cudaStream_t st);
cudaError_t launch_gemm_tc(const bf16 *A, int lda, const bf16 *Bt, int ldb, bf16 *C, int ldc, int M,
                           int N, int K, int *status, cudaStream_t st);
cudaError_t launch_rh_gemm_tc(const bf16 *A, int lda, const bf16 *W1t, const float *W2, float *partial,
                              int M, int d_R, int K, int h_kv, int act, int *n_tiles, int *status,
                              cudaStream_t st);
int rh_tc_num_tiles(int d_R);

// scores[m][slot0 + t] = sum_nt partial[nt][t][m]
cudaError_t launch_rh_reduce(const float *partial, int n_tiles, int M, int h_kv, float *scores,
                             int score_stride, int slot0, cudaStream_t st, const PerHead *slot0_m = nullptr);

struct RopeAppendArgs {
  const bf16 *staging;  // [n_tok x d_in]  pre-RoPE Q | K | V
  bf16 *q_rot;          // [n_tok x h*d]
  bf16 *z_post;         // [n_tok x d_in] or nullptr: post-RoPE Q | K, V (retaining-head input variant)
  bf16 *k_pre;          // [h_kv][cap][d]
  bf16 *k_rot;          // [h_kv][cap][d]
  bf16 *v;              // [h_kv][cap][d]
  int64_t *tid;         // [h_kv][cap]
  const float2 *cs;     // [cap][d/2] (cos, sin)
  int n_tok, h, h_kv, d, cap, len;
  int64_t seen;
  int per_head;    // the chunk is appended at slot len_m.v[m] + t of KV head m (query heads use their KV head's)
  PerHead len_m;   // (read by rope_append_kernel only: the fused epilogue and the one-token kernel take `len`)
};
cudaError_t launch_rope_append(const RopeAppendArgs &a, cudaStream_t st);
// The projection GEMM with rope_append's work done in its epilogue (a.staging is written, not read).
bool qkv_rope_tc_supported(int M, int N, int K, int lda, int ldb, int d);
cudaError_t launch_qkv_rope_tc(const bf16 *X, int ldx, const bf16 *Wt, int ldw, bf16 *staging, int M,
                               int N, int K, const RopeAppendArgs &a, int *status, cudaStream_t st);

// Attention (Eq. 1): query row t of head j sees keys [0, len + t] of KV head j / g.
cudaError_t launch_attention_mma(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out,
                                 int n_tok, int h, int h_kv, int d, int cap, int len,
                                 cudaStream_t st, const PerHead *len_m = nullptr);

// Eviction in place.  Kept units stay in their slots and freed slots below `budget` are refilled, so
// slot order is not temporal order: a unit's position in temporal order is its RANK, stored per slot
// for slots below `ranked_len`; slots from there on (appended since the last eviction) are in order,
// rank = slot.
struct TopkArgs {
  const float *scores;      // [h_kv][stride]
  int32_t *rank[2];         // [h_kv][stride] each: rank[rcur] holds the ranks, the other receives the new ones
  int rcur;                 //   (for slots < budget; its entries from budget on are used as scratch)
  int stride, ranked_len;
  int n, budget, n_prot, n_pre;   // candidates: slots [0, n); ranks [0, n_pre) and [n - n_prot, n) protected
  int32_t *src_of;          // [h_kv][src_stride]  out: the slot whose unit ends up in slot i
  int src_stride;
  unsigned long long *counters;  // [2] or null: units moved to another slot, rotated keys rewritten (added to)
  // a budget per head: head m has n_m candidates, budget_m, nprot_m protected at the end, ranks valid
  // below ranked_m, its ranks in rank[rcur_m]; a head with n_m <= budget_m keeps everything and is skipped
  int per_head;
  PerHead n_m, budget_m, nprot_m, ranked_m, rcur_m;
};
cudaError_t launch_topk(const TopkArgs &a, int h_kv, cudaStream_t st);

struct CompactArgs {
  bf16 *k, *v, *k_rot;      // [h_kv][cap][d]
  float *s;                 // [h_kv][cap]
  int64_t *t;
  const int32_t *src_of;    // [h_kv][src_stride]
  const int32_t *rank[2];   // [h_kv][cap]: rank[rcur] before the eviction, the other after
  int rcur;
  const float2 *cs;
  int h_kv, d, cap, budget, ranked_len, src_stride;
  int per_head;             // (see TopkArgs) evict_m: 1 where head m evicts in this step
  PerHead budget_m, ranked_m, rcur_m, evict_m;
};
cudaError_t launch_compact(const CompactArgs &a, cudaStream_t st);

// k_rot[m][i] = RoPE(k_pre[m][i], i) for i < len (used after an import).
cudaError_t launch_rerope(const bf16 *k_pre, bf16 *k_rot, const float2 *cs, int h_kv, int d, int cap,
                          int len, cudaStream_t st);

// ---- 4-bit cache (int4_cache.cu).  One half of the ping-pong pair:
struct Int4Half {
  uint8_t *kq, *vq;  // [h_kv][cap][d/2] two codes per byte, even element in the low nibble
  __half *ks, *vs;   // [h_kv][cap] one scale per head vector
};
// Expand slots [0, len) into bf16: keys rotated at the unit's position in temporal order when `rotate`
// (rank[m * cap + slot] for slot < ranked_len, the slot itself above; rank may be null: position = slot),
// values plain.
cudaError_t launch_dequant(const Int4Half &q, bf16 *k_out, bf16 *v_out, const float2 *cs, int h_kv, int d,
                           int cap, int len, bool rotate, const int32_t *rank, int ranked_len, cudaStream_t st);
// Quantise n_tok vectors per KV head into slots [slot0, slot0 + n_tok).  Vector (t, m) of K is at
// k_src + t * tok_stride + m * head_stride (elements), likewise V.
cudaError_t launch_quantize(const bf16 *k_src, const bf16 *v_src, long long tok_stride,
                            long long head_stride, const Int4Half &q, int n_tok, int h_kv, int d, int cap,
                            int slot0, cudaStream_t st);
cudaError_t launch_compact_int4(const Int4Half &q, float *s, int64_t *t, const int32_t *src_of, int h_kv, int d,
                                int cap, int budget, cudaStream_t st);

// ---- decoding (decode.cu): one token
cudaError_t launch_gemv(const bf16 *x, const bf16 *Wt, int N, int K, bf16 *y, cudaStream_t st);
// y = x Wt^T + r (one token; the residual is added before the one rounding)
cudaError_t launch_gemv_resid(const bf16 *x, const bf16 *Wt, int N, int K, const bf16 *r, bf16 *y,
                              cudaStream_t st);
// act[c] = silu(x . Wg[:, c]) * (x . Wu[:, c]) for one token; Wt [2F x K] in the interleaved
// layout of launch_gemm_tc_gated
cudaError_t launch_gemv_gated(const bf16 *x, const bf16 *Wt, int F, int K, bf16 *act, cudaStream_t st);
// projection + positions + RoPE + cache append of one token (a.staging is not used: `staging` is written)
cudaError_t launch_gemv_rope(const bf16 *x, const bf16 *Wt, int K, bf16 *staging, const RopeAppendArgs &a,
                             cudaStream_t st, bool pdl = false);
// retaining head of one token; the last block sums the per-block partials into
// score_out[m * score_stride]; counter: one zeroed word, left at zero
// pdl: the kernel is the third of a one-token step's chain (projection, attention, retaining head)
// launched with programmatic dependent launch; it needs only the projection's output, so it runs beside
// the attention kernel and waits for that kernel just before it ends (which keeps the chain ordered)
cudaError_t launch_rh_gemv(const bf16 *z, const bf16 *W1t, const float *W2, float *partial, int d_R, int K,
                           int h_kv, int act, unsigned *counter, float *score_out, int score_stride,
                           cudaStream_t st, bool pdl = false);
int rh_gemv_blocks(int d_R);
int decode_attn_splits(int h_kv, int n, bool int4);
// part_o: fp32 [h][n_splits][d]; part_ml: fp32 [h][n_splits][2]; counters: one zeroed word per
// (KV head, group of 16 query heads), left at zero (the last split merges the partial results).
// q4 != nullptr: keys [0, n - 1) are read from the 4-bit cache (expanded and rotated with `cs` on the
// way into shared memory, at position rank[m * cap + slot] for slot < ranked_len and slot above) and only
// key n - 1, the token of this step, from k_rot / v.  tok_k / tok_v (4-bit cache only, may be null): the
// token's pre-RoPE keys and values [h_kv][d], which the kernel quantises into slot n - 1 of the cache.
struct Int4Half;
cudaError_t launch_attention_decode(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out,
                                    float *part_o, float *part_ml, unsigned *counters, int h, int h_kv, int d,
                                    int cap, int n, int n_splits, const Int4Half *q4, const float2 *cs,
                                    const int32_t *rank, int ranked_len, const bf16 *tok_k, const bf16 *tok_v,
                                    cudaStream_t st, bool pdl = false);

// dst[c][r] = src[r][c]  (weight repack at create)
cudaError_t launch_transpose_bf16(const bf16 *src, bf16 *dst, int rows, int cols, cudaStream_t st);
cudaError_t launch_bf16_to_f32(const bf16 *src, float *dst, int n, cudaStream_t st);

}  // namespace locret
