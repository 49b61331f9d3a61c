// Eq. 1 on warp-level tensor-core instructions (mma.sync), general shapes:
// any n_tok (decode included), head_dim 64 / 96 / 128.  One CTA = 64 query rows of one
// query head; keys/values of KV head j / g stream through shared memory in tiles of 64
// with an online softmax.  Query row t sees keys [0, len + t]: the retained cache
// unmasked, the chunk causally.
#include "common.cuh"

namespace locret {

namespace {

constexpr int QT = 64, KT_ = 64, ATHREADS = 128;

template <int D>
__global__ void __launch_bounds__(ATHREADS)
attn_mma_kernel(const bf16 *__restrict__ q_rot, const bf16 *__restrict__ k_rot,
                const bf16 *__restrict__ v, bf16 *__restrict__ out, int n_tok, int h, int h_kv,
                int cap, int len_all, float scale_log2, int per_head, PerHead len_m) {
  constexpr int LD = D + 8;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16 *sQ = reinterpret_cast<bf16 *>(smem_raw);
  bf16 *sK = sQ + QT * LD;          // [2][64][LD]
  bf16 *sV = sK + 2 * KT_ * LD;     // [2][64][LD]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  const int qtile = gridDim.x - 1 - blockIdx.x;  // longest tiles first
  const int q0 = qtile * QT;
  const int j = blockIdx.y;
  const int m = j / (h / h_kv);
  const int len = per_head ? len_m.v[m] : len_all;  // (a budget per head: this KV head's cache length)
  const int n = len + n_tok;
  const int n_keys = min(n, len + q0 + QT);
  const int NKT = (n_keys + KT_ - 1) / KT_;
  const bf16 *kbase = k_rot + (size_t)m * cap * D;
  const bf16 *vbase = v + (size_t)m * cap * D;

  constexpr int VPR = D / 8;  // 16-byte vectors per row
  auto load_kv = [&](int buf, int kt) {
    for (int x = tid; x < KT_ * VPR; x += ATHREADS) {
      int r = x / VPR, c = (x - r * VPR) * 8;
      int key = kt * KT_ + r;
      bool ok = key < n;
      size_t off = (size_t)min(key, n - 1) * D + c;
      cp_async16(sK + (buf * KT_ + r) * LD + c, kbase + off, ok);
      cp_async16(sV + (buf * KT_ + r) * LD + c, vbase + off, ok);
    }
  };

  for (int x = tid; x < QT * VPR; x += ATHREADS) {
    int r = x / VPR, c = (x - r * VPR) * 8;
    int row = q0 + r;
    cp_async16(sQ + r * LD + c, q_rot + (size_t)min(row, n_tok - 1) * h * D + (size_t)j * D + c,
               row < n_tok);
  }
  load_kv(0, 0);
  cp_async_commit();

  uint32_t qf[D / 16][4];
  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; i++)
#pragma unroll
    for (int e = 0; e < 4; e++) o[i][e] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const int row_lo = q0 + warp * 16 + g;  // rows row_lo and row_lo + 8

  for (int kt = 0; kt < NKT; kt++) {
    if (kt + 1 < NKT) load_kv((kt + 1) & 1, kt + 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int kk = 0; kk < D / 16; kk++)
        ldmatrix_x4(qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3],
                    sQ + (warp * 16 + (lane & 15)) * LD + kk * 16 + (lane >> 4) * 8);
    }
    const bf16 *k_s = sK + (kt & 1) * KT_ * LD;
    const bf16 *v_s = sV + (kt & 1) * KT_ * LD;

    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
      for (int e = 0; e < 4; e++) s[i][e] = 0.f;
#pragma unroll
    for (int kk = 0; kk < D / 16; kk++) {
#pragma unroll
      for (int jn = 0; jn < 4; jn++) {
        uint32_t b0, b1, b2, b3;
        int id = lane >> 3;
        int r = jn * 16 + (id >> 1) * 8 + (lane & 7);
        int c = kk * 16 + (id & 1) * 8;
        ldmatrix_x4(b0, b1, b2, b3, k_s + r * LD + c);
        mma_bf16_16816(s[2 * jn], qf[kk], b0, b1);
        mma_bf16_16816(s[2 * jn + 1], qf[kk], b2, b3);
      }
    }

    // scale, mask, online softmax
    const int key0 = kt * KT_;
    const bool need_mask = key0 + KT_ - 1 > len + q0 + warp * 16;
    float tmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
      for (int e = 0; e < 4; e++) {
        float val = s[i][e] * scale_log2;
        if (need_mask) {
          int key = key0 + i * 8 + q * 2 + (e & 1);
          int row = row_lo + (e >> 1) * 8;
          if (key > len + row) val = -INFINITY;
        }
        s[i][e] = val;
        tmax[e >> 1] = fmaxf(tmax[e >> 1], val);
      }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; r++) {
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 1));
      tmax[r] = fmaxf(tmax[r], __shfl_xor_sync(0xffffffffu, tmax[r], 2));
      float mnew = fmaxf(mrow[r], tmax[r]);
      float muse = (mnew == -INFINITY) ? 0.f : mnew;
      alpha[r] = exp2f(mrow[r] - muse);
      mrow[r] = mnew;
      float psum = 0.f;
#pragma unroll
      for (int i = 0; i < 8; i++) {
        float p0 = exp2f(s[i][2 * r] - muse), p1 = exp2f(s[i][2 * r + 1] - muse);
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

    // O += P · V
#pragma unroll
    for (int k2 = 0; k2 < KT_ / 16; k2++) {
      uint32_t pf[4];
      pf[0] = pack_bf16(s[2 * k2][0], s[2 * k2][1]);
      pf[1] = pack_bf16(s[2 * k2][2], s[2 * k2][3]);
      pf[2] = pack_bf16(s[2 * k2 + 1][0], s[2 * k2 + 1][1]);
      pf[3] = pack_bf16(s[2 * k2 + 1][2], s[2 * k2 + 1][3]);
#pragma unroll
      for (int dn = 0; dn < D / 16; dn++) {
        uint32_t b0, b1, b2, b3;
        int id = lane >> 3;
        int r = k2 * 16 + (id & 1) * 8 + (lane & 7);
        int c = dn * 16 + (id >> 1) * 8;
        ldmatrix_x4_trans(b0, b1, b2, b3, v_s + r * LD + c);
        mma_bf16_16816(o[2 * dn], pf, b0, b1);
        mma_bf16_16816(o[2 * dn + 1], pf, b2, b3);
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int r = 0; r < 2; r++) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; r++) {
    int row = row_lo + r * 8;
    if (row < n_tok) {
      float inv = 1.0f / lrow[r];
      bf16 *dst = out + (size_t)row * h * D + (size_t)j * D;
#pragma unroll
      for (int i = 0; i < D / 8; i++)
        *reinterpret_cast<uint32_t *>(dst + i * 8 + q * 2) =
            pack_bf16(o[i][2 * r] * inv, o[i][2 * r + 1] * inv);
    }
  }
}

template <int D>
cudaError_t launch_d(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out, int n_tok, int h,
                     int h_kv, int cap, int len, cudaStream_t st, const PerHead *len_m) {
  constexpr int smem = (QT + 4 * KT_) * (D + 8) * 2;
  static PerDeviceFlag attr_set;
  if (cudaError_t e = allow_dynamic_smem(attn_mma_kernel<D>, smem, attr_set); e != cudaSuccess) return e;
  dim3 grid((n_tok + QT - 1) / QT, h);
  float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  attn_mma_kernel<D><<<grid, ATHREADS, smem, st>>>(q_rot, k_rot, v, out, n_tok, h, h_kv, cap, len,
                                                   scale_log2, len_m ? 1 : 0, len_m ? *len_m : PerHead{});
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention_mma(const bf16 *q_rot, const bf16 *k_rot, const bf16 *v, bf16 *out,
                                 int n_tok, int h, int h_kv, int d, int cap, int len,
                                 cudaStream_t st, const PerHead *len_m) {
  switch (d) {
    case 64: return launch_d<64>(q_rot, k_rot, v, out, n_tok, h, h_kv, cap, len, st, len_m);
    case 96: return launch_d<96>(q_rot, k_rot, v, out, n_tok, h, h_kv, cap, len, st, len_m);
    case 128: return launch_d<128>(q_rot, k_rot, v, out, n_tok, h, h_kv, cap, len, st, len_m);
  }
  return cudaErrorInvalidValue;
}

}  // namespace locret
