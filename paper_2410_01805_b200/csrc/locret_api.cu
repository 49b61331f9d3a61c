// C ABI of the library: argument checks, state, and the per-chunk launch sequence.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/locret.h"
#include "common.cuh"
#include "tc_common.cuh"

using namespace locret;

namespace {

// Scratch shared by every layer bound to the same stream (only one layer's step is in
// flight on a stream at a time).
struct ScratchPool {
  cudaStream_t st = nullptr;
  int device = 0;
  int refs = 0;
  // Second stream for the work that is off the critical path of a decoder layer (retaining
  // head, selection, compaction): it overlaps the tail of the attention kernel and the next
  // layer's projection.  staging / z_post are double-buffered because that work reads them.
  cudaStream_t side = nullptr;
  cudaEvent_t ev_stage_free[2] = {nullptr, nullptr};
  // 4-bit caches: the bf16 expansion is written on the second stream while the projection runs
  cudaEvent_t ev_exp_free = nullptr, ev_exp_ready = nullptr;
  // work of ANY layer may be pending on the second stream: a step that uses the shared scratch of the
  // off-critical-path kernels (partial scores, index lists) on the layer's own stream waits for it first
  cudaEvent_t ev_side_idle = nullptr;
  bool side_dirty = false;
  bool exp_busy = false;  // ev_exp_free recorded and not yet waited for
  bool stage_busy[2] = {false, false};  // recorded and not yet waited for
  int flip = 0;
  size_t staging_b[2] = {0, 0}, qrot_b = 0, zpost_b[2] = {0, 0}, partial_b = 0, keep_b = 0, kexp_b = 0, vexp_b = 0;
  bf16 *staging[2] = {nullptr, nullptr}, *q_rot = nullptr, *z_post[2] = {nullptr, nullptr};
  bf16 *k_exp = nullptr, *v_exp = nullptr;  // 4-bit caches: bf16 expansion of the layer in flight
  float *dec_o = nullptr, *dec_ml = nullptr;  // decode attention: per-split partial results
  size_t deco_b = 0, decml_b = 0;
  // decode kernels whose last block merges the partial results: zeroed words that each launch
  // leaves at zero (word 0: retaining head; words 1..: attention, one per KV head x head group)
  unsigned *dec_cnt = nullptr;
  float *partial = nullptr;
  int32_t *keep = nullptr;
  struct CsTable { float theta; int d, cap; float2 *ptr; };
  std::vector<CsTable> cs;
};

std::mutex g_mu;
// keyed by (device, stream): the default stream has the same handle on every device
std::map<std::pair<int, cudaStream_t>, ScratchPool *> g_pools;

template <typename T>
bool grow(T **p, size_t *have, size_t want, cudaStream_t st) {
  if (want <= *have) return true;
  T *np_ = nullptr;
  if (cudaMalloc(&np_, want) != cudaSuccess) { cudaGetLastError(); return false; }
  if (*p) { cudaStreamSynchronize(st); cudaFree(*p); }
  *p = np_;
  *have = want;
  return true;
}

struct TimedEvent { cudaEvent_t a, b; int kind; };
constexpr int DEC_CNT_WORDS = 1 + 32 * 16;  // retaining head + (KV head, head group) pairs

}  // namespace

struct locret_layer {
  locret_layer_cfg cfg;
  int budget, chunk, n_stab, cap, d_in, h, h_kv, d, D, d_R;
  int n_prefix;  // Section 4.4 variant: cache slots [0, n_prefix) are never evicted
  cudaStream_t st;
  ScratchPool *pool;
  bf16 *wqkv_t, *w1_t;
  float *w2f;
  bf16 *k_pre, *v, *k_rot;        // bf16 cache (null for a 4-bit cache)
  bool int4;
  Int4Half q4;                    // 4-bit cache
  const void *map_kv_base;
  float *s;
  int64_t *tid;
  // Eviction works in place, so slot order is not temporal order: rank[rcur][m][slot] is the unit's
  // position in temporal order for slot < ranked_len; slots from there on are in order (rank = slot).
  // The other array receives the ranks of the next eviction.
  int32_t *rank[2];
  int rcur, ranked_len;
  // a budget per KV head (Appendix H): lengths, valid-rank counts and the array that holds the ranks
  // then differ from head to head; `len` is the largest length
  bool per_head;
  PerHead budget_m, len_m, ranked_m, rcur_m;
  unsigned long long *d_counters;  // [2]: units moved to another slot, rotated keys rewritten
  int device;  // the device that was current at create: every later call must find it current
  const float2 *cs;
  int *d_status;
  int len;
  int64_t seen;
  int64_t launches;
  bool timing;
  bool serialize;  // timing mode 2: keep every kernel on the main stream (clean per-kernel times)
  bool attn_only;  // timing mode 3: bracket only the attention kernel (least overhead)
  bool use_tc;  // tcgen05 kernels (default); LOCRET_LEGACY_MMA=1 keeps the mma.sync kernels for A/B runs
  bool fuse_rope;  // RoPE + append in the projection's epilogue (LOCRET_UNFUSED_ROPE=1 disables)
  bool use_side;  // off-critical-path kernels go to the pool's second stream (LOCRET_SERIAL=1 disables)
  bool use_pdl;   // one-token steps overlap their kernels by programmatic dependent launch (LOCRET_NO_PDL=1 disables)
  bool side_pending;
  float **d_peers;  // divided heads, fused exchange: device array of the GPUs' sum buffers
  int n_peers;
  float *tp_scratch;  // this GPU's product for shapes the tensor-core GEMM does not take
  bool tp_pending;  // a divided-heads step was begun and waits for the summed product
  int tp_n_tok;
  uint32_t tp_flags;
  cudaEvent_t ev_ready, ev_attn, ev_side, ev_tp;  // ev_tp: the divided-heads exchange (both directions)
  bool tc_attn;  // tensor maps for the tcgen05 attention kernel are valid
  CUtensorMap map_k, map_v, map_q;
  CUtensorMap map_k64;   // keys in boxes of 64 (the CTA-pair attention kernel loads half a key tile per CTA)
  bool attn_pair;
  const void *map_q_base;
  std::vector<TimedEvent> events;
  size_t events_used;
};

namespace {

void free_layer_memory(locret_layer *L) {
  cudaFree(L->wqkv_t); cudaFree(L->w1_t); cudaFree(L->w2f);
  cudaFree(L->k_pre); cudaFree(L->v); cudaFree(L->s); cudaFree(L->tid);
  cudaFree(L->q4.kq); cudaFree(L->q4.vq); cudaFree(L->q4.ks); cudaFree(L->q4.vs);
  cudaFree(L->rank[0]); cudaFree(L->rank[1]); cudaFree(L->d_counters);
  cudaFree(L->k_rot); cudaFree(L->d_status); cudaFree(L->d_peers); cudaFree(L->tp_scratch);
  for (auto &e : L->events) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  if (L->ev_ready) cudaEventDestroy(L->ev_ready);
  if (L->ev_tp) cudaEventDestroy(L->ev_tp);
  if (L->ev_attn) cudaEventDestroy(L->ev_attn);
  if (L->ev_side) cudaEventDestroy(L->ev_side);
  cudaGetLastError();
}

void release_pool(ScratchPool *p) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (!p) return;
  if (--p->refs > 0) return;
  if (p->side) { cudaStreamSynchronize(p->side); cudaStreamDestroy(p->side); }
  for (int i = 0; i < 2; i++) {
    cudaFree(p->staging[i]); cudaFree(p->z_post[i]);
    if (p->ev_stage_free[i]) cudaEventDestroy(p->ev_stage_free[i]);
  }
  if (p->ev_exp_free) cudaEventDestroy(p->ev_exp_free);
  if (p->ev_exp_ready) cudaEventDestroy(p->ev_exp_ready);
  if (p->ev_side_idle) cudaEventDestroy(p->ev_side_idle);
  cudaFree(p->q_rot); cudaFree(p->partial); cudaFree(p->keep); cudaFree(p->dec_o); cudaFree(p->dec_ml); cudaFree(p->dec_cnt);
  cudaFree(p->k_exp); cudaFree(p->v_exp);
  for (auto &t : p->cs) cudaFree(t.ptr);
  g_pools.erase(std::make_pair(p->device, p->st));
  delete p;
  cudaGetLastError();
}

const float2 *get_cs_table(ScratchPool *p, float theta, int d, int cap, cudaStream_t st) {
  for (auto &t : p->cs)
    if (t.theta == theta && t.d == d && t.cap >= cap) return t.ptr;
  const int half = d / 2;
  std::vector<float2> host((size_t)cap * half);
  std::vector<double> inv(half);
  for (int i = 0; i < half; i++) inv[i] = pow((double)theta, -2.0 * i / d);
  for (int pos = 0; pos < cap; pos++)
    for (int i = 0; i < half; i++) {
      double ang = (double)pos * inv[i];
      host[(size_t)pos * half + i] = make_float2((float)cos(ang), (float)sin(ang));
    }
  float2 *dev = nullptr;
  if (cudaMalloc(&dev, host.size() * sizeof(float2)) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (cudaMemcpyAsync(dev, host.data(), host.size() * sizeof(float2), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaFree(dev); cudaGetLastError(); return nullptr;
  }
  p->cs.push_back({theta, d, cap, dev});
  return dev;
}

// Bracket one launch with events when timing is on; count it.
struct Timed {
  locret_layer *L; int kind; cudaStream_t st; TimedEvent *ev = nullptr;
  Timed(locret_layer *l, int k, cudaStream_t stream = nullptr) : L(l), kind(k), st(stream ? stream : l->st) {
    L->launches++;
    if (!L->timing || (L->attn_only && k != LOCRET_K_ATTN)) return;
    if (L->events_used == L->events.size()) {
      TimedEvent e; e.kind = k;
      if (cudaEventCreate(&e.a) != cudaSuccess || cudaEventCreate(&e.b) != cudaSuccess) { cudaGetLastError(); return; }
      L->events.push_back(e);
    }
    ev = &L->events[L->events_used++];
    ev->kind = k;
    cudaEventRecord(ev->a, st);
  }
  ~Timed() { if (ev) cudaEventRecord(ev->b, st); }
};

#define CK(call)                                         \
  do {                                                   \
    cudaError_t e__ = (call);                            \
    if (e__ != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; } \
  } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A layer's buffers, streams and events belong to the device that was current at create.
bool on_layer_device(const locret_layer *L) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
  return dev == L->device;
}

// Wait for everything this layer has in flight, on both streams.
cudaError_t sync_all(locret_layer *L) {
  cudaError_t e = cudaStreamSynchronize(L->st);
  if (e == cudaSuccess && L->use_side && L->pool && L->pool->side) e = cudaStreamSynchronize(L->pool->side);
  return e;
}

// Export in temporal order.  The cache keeps units where eviction left them; slot `i` of head `m`
// holds the unit of position rank[m][i] (for i below ranked_len; the slot itself above).  The arrays
// are copied to the host as they lie and put in order there (an export is a diagnostic path).
struct TemporalOrder {
  std::vector<int32_t> rank;  // [h_kv][ranked] or empty when the cache is in order
  int ranked = 0;
  int load(locret_layer *L) {
    ranked = L->ranked_len < L->len ? L->ranked_len : L->len;
    if (ranked == 0) return LOCRET_OK;
    rank.resize((size_t)L->h_kv * ranked);
    CK(cudaMemcpy2D(rank.data(), (size_t)ranked * 4, L->rank[L->rcur], (size_t)L->cap * 4, (size_t)ranked * 4,
                    L->h_kv, cudaMemcpyDeviceToHost));
    return LOCRET_OK;
  }
  // rows of `row_bytes` bytes, device pitch cap * row_bytes per head -> out [h_kv][len][row_bytes]
  int copy_out(locret_layer *L, const void *dev, size_t row_bytes, void *out) {
    const int n = L->len;
    const size_t dense = (size_t)n * row_bytes, pitch = (size_t)L->cap * row_bytes;
    if (ranked == 0) {
      CK(cudaMemcpy2D(out, dense, dev, pitch, dense, L->h_kv, cudaMemcpyDeviceToHost));
      return LOCRET_OK;
    }
    std::vector<unsigned char> tmp;
    try { tmp.resize((size_t)L->h_kv * dense); } catch (...) { return LOCRET_ERR_ALLOC; }
    CK(cudaMemcpy2D(tmp.data(), dense, dev, pitch, dense, L->h_kv, cudaMemcpyDeviceToHost));
    unsigned char *o = static_cast<unsigned char *>(out);
    for (int m = 0; m < L->h_kv; m++)
      for (int i = 0; i < n; i++) {
        const int r = i < ranked ? rank[(size_t)m * ranked + i] : i;
        if (r < 0 || r >= n) return LOCRET_ERR_CUDA;  // a rank outside the cache: the state is corrupt
        memcpy(o + ((size_t)m * n + r) * row_bytes, tmp.data() + ((size_t)m * n + i) * row_bytes, row_bytes);
      }
    return LOCRET_OK;
  }
};

}  // namespace

extern "C" {

const char *locret_strerror(int code) {
  switch (code) {
    case LOCRET_OK: return "ok";
    case LOCRET_ERR_INVALID: return "invalid argument or configuration";
    case LOCRET_ERR_ALLOC: return "allocation failed";
    case LOCRET_ERR_CAPACITY: return "cache capacity exceeded";
    case LOCRET_ERR_CUDA: return "CUDA call failed";
    case LOCRET_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown error";
}

int locret_create(const locret_layer_cfg *cfg, int32_t budget, int32_t chunk, int32_t n_stab,
                  locret_layer **out) {
  if (!out) return LOCRET_ERR_INVALID;
  *out = nullptr;
  if (!cfg) return LOCRET_ERR_INVALID;
  const int h = cfg->n_q_heads, hk = cfg->n_kv_heads, d = cfg->head_dim, D = cfg->d_model,
            dR = cfg->d_retain;
  if (h < 1 || hk < 1 || hk > 32 || h % hk != 0) return LOCRET_ERR_INVALID;
  if (d != 64 && d != 96 && d != 128) return LOCRET_ERR_INVALID;
  if (D < 32 || D % 32 != 0 || dR < 8 || dR % 8 != 0) return LOCRET_ERR_INVALID;
  if (cfg->act < 0 || cfg->act > 2 || cfg->rh_input < 0 || cfg->rh_input > 1) return LOCRET_ERR_INVALID;
  if (cfg->kv_dtype != 0 && cfg->kv_dtype != 1) return LOCRET_ERR_INVALID;
  if (!(cfg->rope_theta > 1.0f) || cfg->reserve < 0) return LOCRET_ERR_INVALID;
  if (budget < 1 || chunk < 1 || n_stab < 0 || n_stab > budget) return LOCRET_ERR_INVALID;
  if (!cfg->w_qkv || !cfg->w1 || !cfg->w2) return LOCRET_ERR_INVALID;
  if (!aligned16(cfg->w_qkv) || !aligned16(cfg->w1)) return LOCRET_ERR_INVALID;
  const long long cap_ll = (long long)budget + chunk + cfg->reserve;
  if (cap_ll > (1ll << 18)) return LOCRET_ERR_INVALID;  // (the selection keeps bitmaps of all candidates in shared memory)

  int ndev = 0, dev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); return LOCRET_ERR_CUDA; }
  if (current_device_index(&dev) != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_CUDA; }

  locret_layer *L = new (std::nothrow) locret_layer();
  if (!L) return LOCRET_ERR_ALLOC;
  L->cfg = *cfg;
  L->budget = budget; L->chunk = chunk; L->n_stab = n_stab; L->cap = (int)cap_ll;
  L->h = h; L->h_kv = hk; L->d = d; L->D = D; L->d_R = dR;
  L->d_in = (h + 2 * hk) * d;
  L->st = (cudaStream_t)cfg->stream;
  L->device = dev;
  L->n_prefix = 0;
  L->rcur = 0; L->ranked_len = 0; L->len = 0;
  L->per_head = false;
  for (int m = 0; m < 32; m++) { L->budget_m.v[m] = budget; L->len_m.v[m] = 0; L->ranked_m.v[m] = 0; L->rcur_m.v[m] = 0; } L->seen = 0; L->launches = 0; L->timing = false; L->serialize = false; L->attn_only = false; L->events_used = 0;
  L->pool = nullptr;
  L->d_peers = nullptr; L->n_peers = 0; L->tp_scratch = nullptr;
  {
    const char *e = getenv("LOCRET_LEGACY_MMA");
    L->use_tc = !(e && e[0] == '1');
    const char *ser = getenv("LOCRET_SERIAL");
    L->use_side = !(ser && ser[0] == '1');
    const char *unf = getenv("LOCRET_UNFUSED_ROPE");
    L->fuse_rope = !(unf && unf[0] == '1');
    // "1": Eq. 1 for head_dim 128 on clusters of two CTAs (faster; opt-in, see the comment at its launch)
    const char *ap = getenv("LOCRET_ATTN_PAIR");
    L->attn_pair = ap && ap[0] == '1';
    const char *np = getenv("LOCRET_NO_PDL");
    L->use_pdl = !(np && np[0] == '1');
    L->side_pending = false;
    L->ev_ready = L->ev_attn = L->ev_side = L->ev_tp = nullptr;
  }

  L->int4 = cfg->kv_dtype == 1;
  L->map_kv_base = nullptr;
  const size_t kv_b = (size_t)hk * L->cap * d * sizeof(bf16);
  const size_t code_b = (size_t)hk * L->cap * (d / 2), scale_b = (size_t)hk * L->cap * sizeof(__half);
  const size_t sc_b = (size_t)hk * L->cap * sizeof(float);
  const size_t td_b = (size_t)hk * L->cap * sizeof(int64_t);
  const size_t rk_b = (size_t)hk * L->cap * sizeof(int32_t);
  bool ok = true;
  ok = ok && cudaMalloc(&L->wqkv_t, (size_t)L->d_in * D * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&L->w1_t, (size_t)dR * L->d_in * sizeof(bf16)) == cudaSuccess;
  ok = ok && cudaMalloc(&L->w2f, (size_t)dR * hk * sizeof(float)) == cudaSuccess;
  if (L->int4) {
    ok = ok && cudaMalloc(&L->q4.kq, code_b) == cudaSuccess;
    ok = ok && cudaMalloc(&L->q4.vq, code_b) == cudaSuccess;
    ok = ok && cudaMalloc(&L->q4.ks, scale_b) == cudaSuccess;
    ok = ok && cudaMalloc(&L->q4.vs, scale_b) == cudaSuccess;
  } else {
    ok = ok && cudaMalloc(&L->k_pre, kv_b) == cudaSuccess;
    ok = ok && cudaMalloc(&L->v, kv_b) == cudaSuccess;
    ok = ok && cudaMalloc(&L->k_rot, kv_b) == cudaSuccess;
  }
  ok = ok && cudaMalloc(&L->s, sc_b) == cudaSuccess;
  ok = ok && cudaMalloc(&L->tid, td_b) == cudaSuccess;
  for (int i = 0; i < 2; i++) ok = ok && cudaMalloc(&L->rank[i], rk_b) == cudaSuccess;
  ok = ok && cudaMalloc(&L->d_counters, 2 * sizeof(unsigned long long)) == cudaSuccess;
  ok = ok && cudaMalloc(&L->d_status, 4 * sizeof(int)) == cudaSuccess;
  if (!ok) { cudaGetLastError(); free_layer_memory(L); delete L; return LOCRET_ERR_ALLOC; }

  // shared scratch
  {
    std::lock_guard<std::mutex> lk(g_mu);
    ScratchPool *&p = g_pools[std::make_pair(L->device, L->st)];
    if (!p) { p = new (std::nothrow) ScratchPool(); if (p) { p->st = L->st; p->device = L->device; } }
    if (p) {
      p->refs++;
      L->pool = p;
      bool g = true;
      if (L->use_side && !p->side) {
        int lo = 0, hi = 0;
        cudaDeviceGetStreamPriorityRange(&lo, &hi);
        g = g && cudaStreamCreateWithPriority(&p->side, cudaStreamNonBlocking, lo) == cudaSuccess;
        for (int i = 0; i < 2 && g; i++)
          g = cudaEventCreateWithFlags(&p->ev_stage_free[i], cudaEventDisableTiming) == cudaSuccess;
        g = g && cudaEventCreateWithFlags(&p->ev_exp_free, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p->ev_exp_ready, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p->ev_side_idle, cudaEventDisableTiming) == cudaSuccess;
      }
      if (g && !p->dec_cnt) {
        g = cudaMalloc(&p->dec_cnt, DEC_CNT_WORDS * sizeof(unsigned)) == cudaSuccess &&
            cudaMemsetAsync(p->dec_cnt, 0, DEC_CNT_WORDS * sizeof(unsigned), L->st) == cudaSuccess;
        if (!g) cudaGetLastError();
      }
      if (p->side) cudaStreamSynchronize(p->side);  // buffers may be replaced below
      for (int i = 0; i < 2; i++) {
        g = g && grow(&p->staging[i], &p->staging_b[i], (size_t)chunk * L->d_in * sizeof(bf16), L->st);
        if (cfg->rh_input == 1)
          g = g && grow(&p->z_post[i], &p->zpost_b[i], (size_t)chunk * L->d_in * sizeof(bf16), L->st);
      }
      g = g && grow(&p->q_rot, &p->qrot_b, (size_t)chunk * h * d * sizeof(bf16), L->st);
      {
        int nt = rh_num_tiles(dR) > rh_tc_num_tiles(dR) ? rh_num_tiles(dR) : rh_tc_num_tiles(dR);
        size_t pb = (size_t)nt * chunk * hk * sizeof(float);
        const size_t pb_dec = (size_t)rh_gemv_blocks(dR) * hk * sizeof(float);
        if (pb < pb_dec) pb = pb_dec;
        g = g && grow(&p->partial, &p->partial_b, pb, L->st);
        g = g && grow(&p->dec_o, &p->deco_b, (size_t)h * 64 * d * sizeof(float), L->st);
        g = g && grow(&p->dec_ml, &p->decml_b, (size_t)h * 64 * 2 * sizeof(float), L->st);
      }
      g = g && grow(&p->keep, &p->keep_b, (size_t)hk * budget * sizeof(int32_t), L->st);
      if (L->int4) {
        const size_t before_k = p->kexp_b, before_v = p->vexp_b;
        g = g && grow(&p->k_exp, &p->kexp_b, kv_b, L->st);
        g = g && grow(&p->v_exp, &p->vexp_b, kv_b, L->st);
        // rows past the live range are multiplied by zero probabilities: they must stay finite
        if (g && p->kexp_b != before_k) g = cudaMemsetAsync(p->k_exp, 0, p->kexp_b, L->st) == cudaSuccess;
        if (g && p->vexp_b != before_v) g = cudaMemsetAsync(p->v_exp, 0, p->vexp_b, L->st) == cudaSuccess;
      }
      if (g) L->cs = get_cs_table(p, cfg->rope_theta, d, L->cap, L->st);
      ok = g && L->cs;
    } else {
      ok = false;
    }
  }
  if (!ok) { ScratchPool *p = L->pool; free_layer_memory(L); delete L; release_pool(p); return LOCRET_ERR_ALLOC; }

  if (L->use_side) {
    ok = cudaEventCreateWithFlags(&L->ev_ready, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&L->ev_attn, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&L->ev_side, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&L->ev_tp, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { cudaGetLastError(); ScratchPool *p = L->pool; free_layer_memory(L); delete L; release_pool(p); return LOCRET_ERR_CUDA; }
  }

  // tensor maps of the cache for the tcgen05 attention kernel
  L->map_q_base = nullptr;
  if (L->int4)
    L->tc_attn = L->use_tc;  // maps point at the shared expansion scratch; encoded on first use
  else
    L->tc_attn = L->use_tc &&
                 tmap_encode_3d_bf16(&L->map_k, L->k_rot, d, L->cap, hk, (uint64_t)d * 2,
                                     (uint64_t)L->cap * d * 2, 64, 128, 1) &&
                 tmap_encode_3d_bf16(&L->map_v, L->v, d, L->cap, hk, (uint64_t)d * 2,
                                     (uint64_t)L->cap * d * 2, 64, 128, 1) &&
                 tmap_encode_3d_bf16(&L->map_k64, L->k_rot, d, L->cap, hk, (uint64_t)d * 2,
                                     (uint64_t)L->cap * d * 2, 64, 64, 1);

  // repack the weights: K-major copies for both GEMMs, W2 in fp32
  cudaError_t e = cudaSuccess;
  if (e == cudaSuccess) e = launch_transpose_bf16((const bf16 *)cfg->w_qkv, L->wqkv_t, D, L->d_in, L->st);
  if (e == cudaSuccess) e = launch_transpose_bf16((const bf16 *)cfg->w1, L->w1_t, L->d_in, dR, L->st);
  if (e == cudaSuccess) e = launch_bf16_to_f32((const bf16 *)cfg->w2, L->w2f, dR * hk, L->st);
  if (e == cudaSuccess) {
    if (L->int4) {
      e = cudaMemsetAsync(L->q4.kq, 0, code_b, L->st);
      if (e == cudaSuccess) e = cudaMemsetAsync(L->q4.vq, 0, code_b, L->st);
      if (e == cudaSuccess) e = cudaMemsetAsync(L->q4.ks, 0, scale_b, L->st);
      if (e == cudaSuccess) e = cudaMemsetAsync(L->q4.vs, 0, scale_b, L->st);
    } else {
      e = cudaMemsetAsync(L->k_pre, 0, kv_b, L->st);
      if (e == cudaSuccess) e = cudaMemsetAsync(L->v, 0, kv_b, L->st);
      if (e == cudaSuccess) e = cudaMemsetAsync(L->k_rot, 0, kv_b, L->st);
    }
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(L->s, 0, sc_b, L->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(L->tid, 0, td_b, L->st);
  for (int i = 0; i < 2 && e == cudaSuccess; i++) e = cudaMemsetAsync(L->rank[i], 0, rk_b, L->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(L->d_counters, 0, 2 * sizeof(unsigned long long), L->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(L->d_status, 0, 4 * sizeof(int), L->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(L->st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    ScratchPool *p = L->pool; free_layer_memory(L); delete L; release_pool(p);
    return LOCRET_ERR_CUDA;
  }
  *out = L;
  return LOCRET_OK;
}

}  // extern "C"

namespace {

// (d) of the step: protect, top-b, gather; then the bookkeeping that closes the step
int evict_and_close(locret_layer *L, int n_tok, uint32_t flags, bool side, cudaStream_t S) {
  ScratchPool *P = L->pool;
  const int n = L->len + n_tok;
  const bool may_evict = !(flags & LOCRET_NO_EVICT);
  bool evicts = may_evict && n > L->budget;
  PerHead n_m{}, nprot_m{}, evict_m{};
  if (L->per_head) {
    evicts = false;
    for (int m = 0; m < L->h_kv; m++) {
      n_m.v[m] = L->len_m.v[m] + n_tok;
      nprot_m.v[m] = (flags & LOCRET_LAST_CHUNK) ? 0 : (L->n_stab < n_m.v[m] ? L->n_stab : n_m.v[m]);
      evict_m.v[m] = may_evict && n_m.v[m] > L->budget_m.v[m];
      evicts = evicts || evict_m.v[m];
    }
  }
  if (evicts) {
    const int n_prot = (flags & LOCRET_LAST_CHUNK) ? 0 : (L->n_stab < n ? L->n_stab : n);
    {
      Timed t(L, LOCRET_K_TOPK, S);
      // (n_prefix + n_stab <= budget < n, so the prefix never reaches into the protected tail)
      TopkArgs a;
      a.scores = L->s; a.rank[0] = L->rank[0]; a.rank[1] = L->rank[1]; a.rcur = L->rcur;
      a.stride = L->cap; a.ranked_len = L->ranked_len;
      a.n = n; a.budget = L->budget; a.n_prot = n_prot; a.n_pre = L->n_prefix;
      a.src_of = P->keep; a.src_stride = L->budget; a.counters = L->d_counters;
      a.per_head = L->per_head ? 1 : 0;
      a.n_m = n_m; a.budget_m = L->budget_m; a.nprot_m = nprot_m; a.ranked_m = L->ranked_m; a.rcur_m = L->rcur_m;
      CK(launch_topk(a, L->h_kv, S));
    }
    // the gather rewrites keys and values that the attention kernel reads
    if (side) CK(cudaStreamWaitEvent(S, L->ev_attn, 0));
    if (L->int4) {
      Timed t(L, LOCRET_K_COMPACT, S);
      CK(launch_compact_int4(L->q4, L->s, L->tid, P->keep, L->h_kv, L->d, L->cap, L->budget, S));
    } else {
      Timed t(L, LOCRET_K_COMPACT, S);
      CompactArgs a;
      a.k = L->k_pre; a.v = L->v; a.k_rot = L->k_rot; a.s = L->s; a.t = L->tid;
      a.src_of = P->keep; a.src_stride = L->budget; a.rank[0] = L->rank[0]; a.rank[1] = L->rank[1]; a.rcur = L->rcur;
      a.cs = L->cs;
      a.h_kv = L->h_kv; a.d = L->d; a.cap = L->cap; a.budget = L->budget; a.ranked_len = L->ranked_len;
      a.per_head = L->per_head ? 1 : 0;
      a.budget_m = L->budget_m; a.ranked_m = L->ranked_m; a.rcur_m = L->rcur_m; a.evict_m = evict_m;
      CK(launch_compact(a, S));
    }
  }
  if (L->per_head) {
    int mx = 0;
    for (int m = 0; m < L->h_kv; m++) {
      if (evict_m.v[m]) {
        L->len_m.v[m] = L->budget_m.v[m];
        L->ranked_m.v[m] = L->budget_m.v[m];
        L->rcur_m.v[m] ^= 1;
      } else {
        L->len_m.v[m] = n_m.v[m];
      }
      mx = L->len_m.v[m] > mx ? L->len_m.v[m] : mx;
    }
    L->len = mx;
  } else if (evicts) {
    L->rcur ^= 1;
    L->ranked_len = L->budget;
    L->len = L->budget;
  } else {
    L->len = n;
  }
  if (side) {
    CK(cudaEventRecord(L->ev_side, S));
    L->side_pending = true;
  }
  L->seen += n_tok;
  return LOCRET_OK;
}

// One step.  tp_partial == nullptr: the whole step.  Otherwise the heads of this layer object are
// one GPU's share: the step stops after attention and this GPU's partial first product of the
// retaining head (fp32 [n_tok x d_R], written to tp_partial), everything on the layer's stream.
int chunk_step(locret_layer *L, const void *hidden_in, int32_t n_tok, uint32_t flags, void *attn_out,
               float *tp_partial, bool tp_peers = false) {
  if (!L || !hidden_in || !attn_out) return LOCRET_ERR_INVALID;
  if (!on_layer_device(L)) return LOCRET_ERR_INVALID;
  if (L->tp_pending) return LOCRET_ERR_INVALID;  // a begun step is finished first
  if (n_tok < 1 || n_tok > L->chunk) return LOCRET_ERR_INVALID;
  if (flags & ~(LOCRET_NO_EVICT | LOCRET_LAST_CHUNK)) return LOCRET_ERR_INVALID;
  if (!aligned16(hidden_in) || !aligned16(attn_out)) return LOCRET_ERR_INVALID;
  const int n = L->len + n_tok;
  if (n > L->cap) return LOCRET_ERR_CAPACITY;
  const PerHead *const len_m = L->per_head ? &L->len_m : nullptr;
  ScratchPool *P = L->pool;
  const bool tp = tp_partial != nullptr || tp_peers;
  if (L->per_head && tp) return LOCRET_ERR_INVALID;  // (a budget per head and divided heads are not combined)
  // one token: bandwidth-bound kernels of decode.cu (with a budget per head a one-token step takes the
  // chunk's general kernels, which know the heads' own lengths)
  const bool decode = n_tok == 1 && L->use_tc && !tp && !L->per_head;
  // (a one-token step is a chain of three short kernels on the layer's own stream, overlapped by
  // programmatic dependent launch: an event between them would serialise them again)
  const bool side = L->use_side && !L->serialize && !decode;
  const bool pdl = decode && L->use_pdl && !L->timing;
  cudaStream_t S = side ? P->side : L->st;  // stream of the off-critical-path kernels
  const int sb = P->flip;                    // staging buffer of this call
  P->flip ^= 1;
  bf16 *const staging = P->staging[sb];
  bf16 *const z_post = P->z_post[sb];
  if (L->use_side && !side && P->side_dirty) {
    // this step runs the retaining head (and an eviction) on the layer's own stream, with the scratch
    // other layers' steps may still be using on the second stream
    CK(cudaEventRecord(P->ev_side_idle, P->side));
    CK(cudaStreamWaitEvent(L->st, P->ev_side_idle, 0));
    P->side_dirty = false;
  }
  if (side) P->side_dirty = true;
  if (L->use_side) {
    // the staging buffer is free once the retaining head that last read it has run, and this
    // layer's cache once its previous selection / compaction has finished
    if (P->stage_busy[sb]) CK(cudaStreamWaitEvent(L->st, P->ev_stage_free[sb], 0));
    P->stage_busy[sb] = false;
    if (L->side_pending) CK(cudaStreamWaitEvent(L->st, L->ev_side, 0));
    L->side_pending = false;
  }

  // a 4-bit cache is expanded into bf16 scratch first: keys rotated at position = slot
  bf16 *const k_att = L->int4 ? P->k_exp : L->k_rot;
  bf16 *const v_att = L->int4 ? P->v_exp : L->v;
  RopeAppendArgs ra;  // positions, RoPE, append of the chunk's units at slots [len, len + n_tok)
  ra.staging = staging; ra.q_rot = P->q_rot;
  ra.z_post = L->cfg.rh_input == 1 ? z_post : nullptr;
  ra.k_pre = L->int4 ? nullptr : L->k_pre; ra.k_rot = k_att; ra.v = v_att; ra.tid = L->tid; ra.cs = L->cs;
  ra.n_tok = n_tok; ra.h = L->h; ra.h_kv = L->h_kv; ra.d = L->d; ra.cap = L->cap; ra.len = L->len;
  ra.seen = L->seen;
  ra.per_head = L->per_head ? 1 : 0;
  ra.len_m = L->len_m;
  // with a tensor-core projection whose width is a whole number of tiles the epilogue of the GEMM does the RoPE pass
  const bool fused_rope = !decode && !L->per_head && L->fuse_rope && L->use_tc && n_tok >= 32 &&
                          qkv_rope_tc_supported(n_tok, L->d_in, L->D, L->D, L->D, L->d);
  const bool deq = L->int4 && L->len > 0 && !decode;
  if (deq) {
    // the expansion writes slots [0, len) of the scratch the chunk's units are appended to
    // (a one-token step reads the codes inside its attention kernel instead).  Only attention
    // reads it, so it runs on the second stream beside the projection; the scratch is free once
    // the attention kernel that read it last has finished.
    if (side && P->exp_busy) { CK(cudaStreamWaitEvent(S, P->ev_exp_free, 0)); P->exp_busy = false; }
    {
      Timed t(L, LOCRET_K_DEQUANT, S);
      CK(launch_dequant(L->q4, P->k_exp, P->v_exp, L->cs, L->h_kv, L->d, L->cap, L->len, true, L->rank[L->rcur],
                        L->ranked_len, S));
    }
    if (side) CK(cudaEventRecord(P->ev_exp_ready, S));
  }
  {  // (a) projections
    Timed t(L, LOCRET_K_QKV);
    if (decode)  // projection, positions, RoPE and append of the one token in one kernel
      CK(launch_gemv_rope((const bf16 *)hidden_in, L->wqkv_t, L->D, staging, ra, L->st, pdl));
    else if (fused_rope)
      CK(launch_qkv_rope_tc((const bf16 *)hidden_in, L->D, L->wqkv_t, L->D, staging, n_tok, L->d_in, L->D,
                            ra, L->d_status + 1, L->st));
    else if (L->use_tc && n_tok >= 32 && gemm_tc_supported(n_tok, L->d_in, L->D, L->D, L->D))
      CK(launch_gemm_tc((const bf16 *)hidden_in, L->D, L->wqkv_t, L->D, staging, L->d_in, n_tok,
                        L->d_in, L->D, L->d_status + 1, L->st));
    else
      CK(launch_gemm_bf16((const bf16 *)hidden_in, L->D, L->wqkv_t, L->D, staging, L->d_in, n_tok,
                          L->d_in, L->D, L->st));
  }
  if (!fused_rope && !decode) {
    Timed t(L, LOCRET_K_ROPE);
    CK(launch_rope_append(ra, L->st));
  }
  auto quantize_chunk = [&](cudaStream_t R) -> int {  // the chunk's units enter the cache quantised (keys pre-RoPE)
    Timed t(L, LOCRET_K_QUANT, R);
    const bf16 *ks = staging + (size_t)L->h * L->d, *vs = ks + (size_t)L->h_kv * L->d;
    CK(launch_quantize(ks, vs, L->d_in, L->d, L->q4, n_tok, L->h_kv, L->d, L->cap, L->len, R));
    return LOCRET_OK;
  };
  // the codes are read by the compaction of this step and by later steps, never by this step's
  // attention (the chunk attends to its own keys and values in bf16): second stream
  // (a one-token step quantises its token inside the attention kernel)
  if (L->int4 && !side && !decode) { const int rc = quantize_chunk(L->st); if (rc != LOCRET_OK) return rc; }
  if (side) CK(cudaEventRecord(L->ev_ready, L->st));
  if (side && deq) CK(cudaStreamWaitEvent(L->st, P->ev_exp_ready, 0));
  {  // (b) Eq. 1
    Timed t(L, LOCRET_K_ATTN);
    bool tc_ok = L->tc_attn && attention_tc_supported(n_tok, L->h, L->h_kv, L->d);
    if (tc_ok && L->int4 && L->map_kv_base != P->k_exp) {
      tc_ok = tmap_encode_3d_bf16(&L->map_k, P->k_exp, L->d, L->cap, L->h_kv, (uint64_t)L->d * 2,
                                  (uint64_t)L->cap * L->d * 2, 64, 128, 1) &&
              tmap_encode_3d_bf16(&L->map_v, P->v_exp, L->d, L->cap, L->h_kv, (uint64_t)L->d * 2,
                                  (uint64_t)L->cap * L->d * 2, 64, 128, 1) &&
              tmap_encode_3d_bf16(&L->map_k64, P->k_exp, L->d, L->cap, L->h_kv, (uint64_t)L->d * 2,
                                  (uint64_t)L->cap * L->d * 2, 64, 64, 1);
      L->map_kv_base = tc_ok ? P->k_exp : nullptr;
    }
    if (tc_ok && L->map_q_base != P->q_rot) {
      tc_ok = tmap_encode_2d_bf16(&L->map_q, P->q_rot, (uint64_t)L->h * L->d, (uint64_t)L->chunk,
                                  (uint64_t)L->h * L->d * 2, 64, 128);
      L->map_q_base = tc_ok ? P->q_rot : nullptr;
    }
    if (decode)
      CK(launch_attention_decode(P->q_rot, k_att, v_att, (bf16 *)attn_out, P->dec_o, P->dec_ml, P->dec_cnt + 1,
                                 L->h, L->h_kv, L->d, L->cap, n, decode_attn_splits(L->h_kv, n, L->int4),
                                 L->int4 ? &L->q4 : nullptr, L->cs, L->rank[L->rcur], L->ranked_len,
                                 L->int4 ? staging + (size_t)L->h * L->d : nullptr,
                                 L->int4 ? staging + (size_t)(L->h + L->h_kv) * L->d : nullptr, L->st, pdl));
    // The CTA-pair kernel is opt-in (LOCRET_ATTN_PAIR=1) and never used in a divided-heads step.  In a test
    // process in which it had run, the projection GEMM of a later divided-heads step (eight shards of the
    // Llama shape on one GPU) reported a device-side time-out in about one full test run in three, also when
    // that step itself used the one-CTA kernel; no run without the pair kernel ever did.  The cause has not
    // been found, so the default is the kernel every earlier run validated.
    else if (tc_ok && L->attn_pair && !tp && attention_tc2_supported(n_tok, L->h, L->h_kv, L->d))
      CK(launch_attention_tc2(&L->map_q, &L->map_k64, &L->map_v, (bf16 *)attn_out, n_tok, L->h, L->h_kv,
                              L->d, L->len, L->d_status, L->st, len_m));
    else if (tc_ok)
      CK(launch_attention_tc(&L->map_q, &L->map_k, &L->map_v, (bf16 *)attn_out, n_tok, L->h, L->h_kv,
                             L->d, L->len, L->d_status, L->st, len_m));
    else
      CK(launch_attention_mma(P->q_rot, k_att, v_att, (bf16 *)attn_out, n_tok, L->h, L->h_kv,
                              L->d, L->cap, L->len, L->st, len_m));
  }
  if (side && L->int4) {  // the attention kernel just launched is the scratch's last reader (a one-token step reads its own token there)
    CK(cudaEventRecord(P->ev_exp_free, L->st));
    P->exp_busy = true;
  }
  if (tp) {
    // this GPU's columns of z times its rows of W1; the caller sums the products of all GPUs.
    // Like the retaining head of the undivided step it runs beside the attention kernel; the
    // layer's stream then waits for it, because the caller's all-reduce is enqueued there.
    if (side) {
      CK(cudaEventRecord(L->ev_attn, L->st));
      CK(cudaStreamWaitEvent(S, L->ev_ready, 0));
      if (L->int4) { const int rc = quantize_chunk(S); if (rc != LOCRET_OK) return rc; }
    }
    {
      Timed t(L, LOCRET_K_RH, S);
      const bf16 *z = L->cfg.rh_input == 1 ? z_post : staging;
      const bool tc = L->use_tc && gemm_tc_supported(n_tok, L->d_R, L->d_in, L->d_in, L->d_in);
      if (tp_peers && tc) {
        // the exchange inside the GEMM: the epilogue adds each tile into every GPU's sum buffer
        CK(launch_gemm_tc_f32_add_peers(z, L->d_in, L->w1_t, L->d_in, L->d_peers, L->n_peers, L->d_R, n_tok, L->d_R,
                                        L->d_in, L->d_status + 2, S));
      } else if (tp_peers) {
        CK(launch_preact_naive(z, L->w1_t, L->tp_scratch, n_tok, L->d_R, L->d_in, S));
        L->launches++;
        CK(launch_add_to_peers(L->tp_scratch, L->d_peers, L->n_peers, (size_t)n_tok * L->d_R, S));
      } else if (tc) {
        CK(launch_gemm_tc_f32(z, L->d_in, L->w1_t, L->d_in, tp_partial, L->d_R, n_tok, L->d_R, L->d_in,
                              L->d_status + 2, S));
      } else {
        CK(launch_preact_naive(z, L->w1_t, tp_partial, n_tok, L->d_R, L->d_in, S));
      }
    }
    if (side) {
      CK(cudaEventRecord(P->ev_stage_free[sb], S));
      P->stage_busy[sb] = true;
      CK(cudaEventRecord(L->ev_tp, S));
      CK(cudaStreamWaitEvent(L->st, L->ev_tp, 0));
    }
    L->tp_pending = true;
    L->tp_n_tok = n_tok;
    L->tp_flags = flags;
    return LOCRET_OK;
  }
  if (side) {
    CK(cudaEventRecord(L->ev_attn, L->st));
    CK(cudaStreamWaitEvent(S, L->ev_ready, 0));
    if (L->int4) { const int rc = quantize_chunk(S); if (rc != LOCRET_OK) return rc; }
  }
  int n_tiles = 0;
  {  // (c) retaining head: launched after the attention kernel, so its CTAs fill that kernel's tail
    Timed t(L, LOCRET_K_RH, S);
    const bf16 *z = L->cfg.rh_input == 1 ? z_post : staging;
    if (decode)
      CK(launch_rh_gemv(z, L->w1_t, L->w2f, P->partial, L->d_R, L->d_in, L->h_kv, L->cfg.act, P->dec_cnt,
                        L->s + L->len, L->cap, S, pdl));
    else if (L->use_tc && n_tok >= 32 && gemm_tc_supported(n_tok, L->d_R, L->d_in, L->d_in, L->d_in))
      CK(launch_rh_gemm_tc(z, L->d_in, L->w1_t, L->w2f, P->partial, n_tok, L->d_R, L->d_in, L->h_kv,
                           L->cfg.act, &n_tiles, L->d_status + 3, S));
    else
      CK(launch_rh_gemm(z, L->d_in, L->w1_t, L->w2f, P->partial, n_tok, L->d_R, L->d_in, L->h_kv,
                        L->cfg.act, &n_tiles, S));
  }
  if (!decode) {  // (the one-token kernel sums its own partial scores)
    Timed t(L, LOCRET_K_RH_REDUCE, S);
    CK(launch_rh_reduce(P->partial, n_tiles, n_tok, L->h_kv, L->s, L->cap, L->len, S, len_m));
  }
  if (side) {
    CK(cudaEventRecord(P->ev_stage_free[sb], S));
    P->stage_busy[sb] = true;
  }
  return evict_and_close(L, n_tok, flags, side, S);
}

}  // namespace

extern "C" {

int locret_prefill_chunk(locret_layer *L, const void *hidden_in, int32_t n_tok, uint32_t flags,
                         void *attn_out) {
  return chunk_step(L, hidden_in, n_tok, flags, attn_out, nullptr);
}

int locret_prefill_chunk_tp_begin(locret_layer *L, const void *hidden_in, int32_t n_tok, uint32_t flags,
                                  void *attn_out, float *preact_partial) {
  if (!preact_partial || !aligned16(preact_partial)) return LOCRET_ERR_INVALID;
  return chunk_step(L, hidden_in, n_tok, flags, attn_out, preact_partial);
}

int locret_tp_set_peers(locret_layer *L, float *const *peer_sums, int32_t n_peers) {
  if (!L || !peer_sums || n_peers < 1 || n_peers > 64 || !on_layer_device(L) || L->tp_pending) return LOCRET_ERR_INVALID;
  for (int i = 0; i < n_peers; i++)
    if (!peer_sums[i] || !aligned16(peer_sums[i])) return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  if (!L->d_peers && cudaMalloc(&L->d_peers, 64 * sizeof(float *)) != cudaSuccess) { cudaGetLastError(); return LOCRET_ERR_ALLOC; }
  if (!L->tp_scratch && cudaMalloc(&L->tp_scratch, (size_t)L->chunk * L->d_R * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    return LOCRET_ERR_ALLOC;
  }
  CK(cudaMemcpy(L->d_peers, peer_sums, (size_t)n_peers * sizeof(float *), cudaMemcpyHostToDevice));
  L->n_peers = n_peers;
  return LOCRET_OK;
}

int locret_prefill_chunk_tp_begin_peers(locret_layer *L, const void *hidden_in, int32_t n_tok, uint32_t flags,
                                        void *attn_out) {
  if (!L || L->n_peers < 1) return LOCRET_ERR_INVALID;
  return chunk_step(L, hidden_in, n_tok, flags, attn_out, nullptr, true);
}

int locret_prefill_chunk_tp_finish(locret_layer *L, const float *preact_sum) {
  if (!L || !preact_sum || !aligned16(preact_sum)) return LOCRET_ERR_INVALID;
  if (!L->tp_pending || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  L->tp_pending = false;
  const int n_tok = L->tp_n_tok;
  // nothing downstream in a decoder layer waits for the scores, the selection or the compaction: they
  // go to the second stream, after the summed product has arrived on the layer's stream
  const bool side = L->use_side && !L->serialize;
  cudaStream_t S = side ? L->pool->side : L->st;
  if (side) {
    L->pool->side_dirty = true;
    CK(cudaEventRecord(L->ev_tp, L->st));
    CK(cudaStreamWaitEvent(S, L->ev_tp, 0));
  }
  {  // (c) finished: activation and this GPU's columns of W2, into the score cache
    Timed t(L, LOCRET_K_RH_REDUCE, S);
    CK(launch_rh_finish(preact_sum, L->w2f, L->s, L->cap, L->len, n_tok, L->d_R, L->h_kv, L->cfg.act, S));
  }
  return evict_and_close(L, n_tok, L->tp_flags, side, S);
}

int locret_decode_step(locret_layer *L, const void *hidden_in, void *attn_out) {
  return locret_prefill_chunk(L, hidden_in, 1, LOCRET_NO_EVICT, attn_out);
}

int locret_decode_step_stack(locret_layer *const *layers, int32_t n_layers, const void *hidden_in, void *attn_out,
                             int64_t out_stride) {
  if (!layers || n_layers < 1 || !attn_out || out_stride < 0 || (out_stride % 8) != 0) return LOCRET_ERR_INVALID;
  for (int i = 0; i < n_layers; i++) {
    if (!layers[i]) return LOCRET_ERR_INVALID;
    bf16 *out = static_cast<bf16 *>(attn_out) + (size_t)i * out_stride;
    const int rc = locret_prefill_chunk(layers[i], hidden_in, 1, LOCRET_NO_EVICT, out);
    if (rc != LOCRET_OK) return rc;
  }
  return LOCRET_OK;
}

int locret_cache_len(const locret_layer *L, int32_t *len) {
  if (!L || !len) return LOCRET_ERR_INVALID;
  *len = L->len;
  return LOCRET_OK;
}

int locret_export_state(locret_layer *L, void *K, void *V, float *scores, int64_t *token_ids,
                        int32_t *len, int64_t *tokens_seen) {
  if (!L || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  if (L->per_head) return LOCRET_ERR_INVALID;           // use locret_export_state_heads
  if (L->int4 && (K || V)) return LOCRET_ERR_INVALID;  // use locret_export_state_int4
  CK(sync_all(L));
  const int n = L->len;
  if (len) *len = n;
  if (tokens_seen) *tokens_seen = L->seen;
  if (n > 0) {
    TemporalOrder ord;
    int rc = ord.load(L);
    if (rc != LOCRET_OK) return rc;
    const size_t row = (size_t)L->d * sizeof(bf16);
    if (K && (rc = ord.copy_out(L, L->k_pre, row, K)) != LOCRET_OK) return rc;
    if (V && (rc = ord.copy_out(L, L->v, row, V)) != LOCRET_OK) return rc;
    if (scores && (rc = ord.copy_out(L, L->s, 4, scores)) != LOCRET_OK) return rc;
    if (token_ids && (rc = ord.copy_out(L, L->tid, 8, token_ids)) != LOCRET_OK) return rc;
  }
  return LOCRET_OK;
}

int locret_import_state(locret_layer *L, const void *K, const void *V, const float *scores,
                        const int64_t *token_ids, int32_t len, int64_t tokens_seen) {
  if (!L || len < 0 || len > L->cap || tokens_seen < 0 || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  if (L->int4) return LOCRET_ERR_INVALID;  // use locret_import_state_int4
  if (L->per_head) return LOCRET_ERR_INVALID;  // use locret_import_state_heads
  if (len > 0 && (!K || !V || !scores || !token_ids)) return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  if (len > 0) {
    const size_t row = (size_t)len * L->d * sizeof(bf16), pitch = (size_t)L->cap * L->d * sizeof(bf16);
    CK(cudaMemcpy2DAsync(L->k_pre, pitch, K, row, row, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(L->v, pitch, V, row, row, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(L->s, (size_t)L->cap * 4, scores, (size_t)len * 4, (size_t)len * 4, L->h_kv,
                         cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(L->tid, (size_t)L->cap * 8, token_ids, (size_t)len * 8, (size_t)len * 8,
                         L->h_kv, cudaMemcpyHostToDevice, L->st));
    L->launches++;
    CK(launch_rerope(L->k_pre, L->k_rot, L->cs, L->h_kv, L->d, L->cap, len, L->st));
  }
  CK(cudaStreamSynchronize(L->st));
  L->len = len;
  L->ranked_len = 0;  // imported units are in temporal order: position = slot
  L->seen = tokens_seen;
  return LOCRET_OK;
}

int locret_export_state_int4(locret_layer *L, void *k_codes, void *k_scales, void *v_codes,
                             void *v_scales, float *scores, int64_t *token_ids, int32_t *len,
                             int64_t *tokens_seen) {
  if (!L || !L->int4 || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  const int n = L->len;
  if (len) *len = n;
  if (tokens_seen) *tokens_seen = L->seen;
  if (n > 0) {
    TemporalOrder ord;
    int rc = ord.load(L);
    if (rc != LOCRET_OK) return rc;
    const size_t crow = (size_t)(L->d / 2);
    const Int4Half &q = L->q4;
    if (k_codes && (rc = ord.copy_out(L, q.kq, crow, k_codes)) != LOCRET_OK) return rc;
    if (v_codes && (rc = ord.copy_out(L, q.vq, crow, v_codes)) != LOCRET_OK) return rc;
    if (k_scales && (rc = ord.copy_out(L, q.ks, 2, k_scales)) != LOCRET_OK) return rc;
    if (v_scales && (rc = ord.copy_out(L, q.vs, 2, v_scales)) != LOCRET_OK) return rc;
    if (scores && (rc = ord.copy_out(L, L->s, 4, scores)) != LOCRET_OK) return rc;
    if (token_ids && (rc = ord.copy_out(L, L->tid, 8, token_ids)) != LOCRET_OK) return rc;
  }
  return LOCRET_OK;
}

int locret_import_state_int4(locret_layer *L, const void *k_codes, const void *k_scales,
                             const void *v_codes, const void *v_scales, const float *scores,
                             const int64_t *token_ids, int32_t len, int64_t tokens_seen) {
  if (!L || !L->int4 || len < 0 || len > L->cap || tokens_seen < 0 || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  if (len > 0 && (!k_codes || !k_scales || !v_codes || !v_scales || !scores || !token_ids))
    return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  if (len > 0) {
    const size_t crow = (size_t)len * (L->d / 2), cpitch = (size_t)L->cap * (L->d / 2);
    const Int4Half &q = L->q4;
    CK(cudaMemcpy2DAsync(q.kq, cpitch, k_codes, crow, crow, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(q.vq, cpitch, v_codes, crow, crow, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(q.ks, (size_t)L->cap * 2, k_scales, (size_t)len * 2, (size_t)len * 2, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(q.vs, (size_t)L->cap * 2, v_scales, (size_t)len * 2, (size_t)len * 2, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(L->s, (size_t)L->cap * 4, scores, (size_t)len * 4, (size_t)len * 4, L->h_kv, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpy2DAsync(L->tid, (size_t)L->cap * 8, token_ids, (size_t)len * 8, (size_t)len * 8, L->h_kv, cudaMemcpyHostToDevice, L->st));
  }
  CK(cudaStreamSynchronize(L->st));
  L->len = len;
  L->ranked_len = 0;
  L->seen = tokens_seen;
  return LOCRET_OK;
}

int locret_set_head_budgets(locret_layer *L, const int32_t *budgets) {
  if (!L || !budgets || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  if (L->int4 || L->len != 0 || L->seen != 0 || L->tp_pending) return LOCRET_ERR_INVALID;
  for (int m = 0; m < L->h_kv; m++)
    if (budgets[m] < 1 || budgets[m] > L->budget || L->n_stab + L->n_prefix > budgets[m]) return LOCRET_ERR_INVALID;
  L->per_head = true;
  for (int m = 0; m < L->h_kv; m++) {
    L->budget_m.v[m] = budgets[m]; L->len_m.v[m] = 0; L->ranked_m.v[m] = 0; L->rcur_m.v[m] = 0;
  }
  return LOCRET_OK;
}

int locret_cache_lens(const locret_layer *L, int32_t *lens) {
  if (!L || !lens) return LOCRET_ERR_INVALID;
  for (int m = 0; m < L->h_kv; m++) lens[m] = L->per_head ? L->len_m.v[m] : L->len;
  return LOCRET_OK;
}

int locret_export_state_heads(locret_layer *L, void *K, void *V, float *scores, int64_t *token_ids, int32_t pitch,
                              int32_t *lens, int64_t *tokens_seen) {
  if (!L || !on_layer_device(L) || L->int4 || pitch < L->len) return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  if (tokens_seen) *tokens_seen = L->seen;
  std::vector<int32_t> rank;
  std::vector<unsigned char> tmp;
  for (int m = 0; m < L->h_kv; m++) {
    const int n = L->per_head ? L->len_m.v[m] : L->len;
    const int ranked = L->per_head ? L->ranked_m.v[m] : L->ranked_len;
    const int rc = L->per_head ? L->rcur_m.v[m] : L->rcur;
    if (lens) lens[m] = n;
    if (n == 0) continue;
    const int nr = ranked < n ? ranked : n;
    rank.resize(nr);
    if (nr) CK(cudaMemcpy(rank.data(), L->rank[rc] + (size_t)m * L->cap, (size_t)nr * 4, cudaMemcpyDeviceToHost));
    auto copy = [&](const void *dev, size_t row_bytes, void *out) -> int {
      if (!out) return LOCRET_OK;
      tmp.resize((size_t)n * row_bytes);
      CK(cudaMemcpy(tmp.data(), (const unsigned char *)dev + (size_t)m * L->cap * row_bytes, (size_t)n * row_bytes,
                    cudaMemcpyDeviceToHost));
      unsigned char *o = (unsigned char *)out + (size_t)m * pitch * row_bytes;
      for (int i = 0; i < n; i++) {
        const int r = i < nr ? rank[i] : i;
        if (r < 0 || r >= n) return LOCRET_ERR_CUDA;
        memcpy(o + (size_t)r * row_bytes, tmp.data() + (size_t)i * row_bytes, row_bytes);
      }
      return LOCRET_OK;
    };
    int e;
    if ((e = copy(L->k_pre, (size_t)L->d * 2, K)) != LOCRET_OK) return e;
    if ((e = copy(L->v, (size_t)L->d * 2, V)) != LOCRET_OK) return e;
    if ((e = copy(L->s, 4, scores)) != LOCRET_OK) return e;
    if ((e = copy(L->tid, 8, token_ids)) != LOCRET_OK) return e;
  }
  return LOCRET_OK;
}

int locret_import_state_heads(locret_layer *L, const void *K, const void *V, const float *scores,
                              const int64_t *token_ids, int32_t pitch, const int32_t *lens, int64_t tokens_seen) {
  if (!L || !on_layer_device(L) || L->int4 || !L->per_head || !lens || pitch < 0 || tokens_seen < 0)
    return LOCRET_ERR_INVALID;
  int mx = 0;
  for (int m = 0; m < L->h_kv; m++) {
    if (lens[m] < 0 || lens[m] > pitch || lens[m] > L->cap) return LOCRET_ERR_INVALID;
    mx = lens[m] > mx ? lens[m] : mx;
  }
  if (mx > 0 && (!K || !V || !scores || !token_ids)) return LOCRET_ERR_INVALID;
  CK(sync_all(L));
  for (int m = 0; m < L->h_kv; m++) {
    const int n = lens[m];
    L->len_m.v[m] = n;
    L->ranked_m.v[m] = 0;  // imported units are in temporal order
    if (n == 0) continue;
    const size_t row = (size_t)L->d * 2;
    CK(cudaMemcpyAsync(L->k_pre + (size_t)m * L->cap * L->d, (const unsigned char *)K + (size_t)m * pitch * row,
                       (size_t)n * row, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpyAsync(L->v + (size_t)m * L->cap * L->d, (const unsigned char *)V + (size_t)m * pitch * row,
                       (size_t)n * row, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpyAsync(L->s + (size_t)m * L->cap, scores + (size_t)m * pitch, (size_t)n * 4, cudaMemcpyHostToDevice, L->st));
    CK(cudaMemcpyAsync(L->tid + (size_t)m * L->cap, token_ids + (size_t)m * pitch, (size_t)n * 8,
                       cudaMemcpyHostToDevice, L->st));
    L->launches++;
    CK(launch_rerope(L->k_pre + (size_t)m * L->cap * L->d, L->k_rot + (size_t)m * L->cap * L->d, L->cs, 1, L->d, L->cap,
                     n, L->st));
  }
  CK(cudaStreamSynchronize(L->st));
  L->len = mx;
  L->seen = tokens_seen;
  return LOCRET_OK;
}

int locret_compaction_counters(locret_layer *L, int64_t *units_moved, int64_t *keys_rotated) {
  if (!L || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  unsigned long long host[2] = {0, 0};
  CK(sync_all(L));
  CK(cudaMemcpy(host, L->d_counters, sizeof(host), cudaMemcpyDeviceToHost));
  if (units_moved) *units_moved = (int64_t)host[0];
  if (keys_rotated) *keys_rotated = (int64_t)host[1];
  return LOCRET_OK;
}

int locret_sync_status(locret_layer *L) {
  if (!L || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  int host = 0;
  CK(sync_all(L));
  // one word per kernel family (attention; projection GEMM; divided-heads GEMM; retaining-head GEMM), so that
  // a reported time-out says where it happened (LOCRET_DIAG_STATUS=1 prints the words to stderr)
  int words[4] = {0, 0, 0, 0};
  CK(cudaMemcpyAsync(words, L->d_status, sizeof(words), cudaMemcpyDeviceToHost, L->st));
  CK(cudaStreamSynchronize(L->st));
  for (int i = 3; i >= 0; i--) if (words[i]) host = words[i];
  if (host != 0) {
    const char *dg = getenv("LOCRET_DIAG_STATUS");
    if (dg && dg[0] == '1')
      fprintf(stderr, "locret status words: attention %d, projection %d, divided-heads product %d, retaining head %d (h %d, h_kv %d, d %d)\n",
              words[0], words[1], words[2], words[3], L->h, L->h_kv, L->d);
  }
  CK(cudaGetLastError());
  return host;
}

int locret_reset(locret_layer *L) {
  if (!L || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  // a selection / compaction still in flight on the second stream writes this layer's cache: the
  // layer's stream is ordered behind it here, so whatever is enqueued after the reset sees it done
  if (L->use_side && L->side_pending) {
    CK(cudaStreamWaitEvent(L->st, L->ev_side, 0));
    L->side_pending = false;
  }
  L->len = 0;
  L->ranked_len = 0;
  for (int m = 0; m < 32; m++) { L->len_m.v[m] = 0; L->ranked_m.v[m] = 0; }
  L->seen = 0;
  L->tp_pending = false;
  return LOCRET_OK;
}

int locret_set_protected_prefix(locret_layer *L, int32_t n_prefix) {
  if (!L || n_prefix < 0 || n_prefix + L->n_stab > L->budget) return LOCRET_ERR_INVALID;
  if (L->per_head)
    for (int m = 0; m < L->h_kv; m++)
      if (n_prefix + L->n_stab > L->budget_m.v[m]) return LOCRET_ERR_INVALID;
  L->n_prefix = n_prefix;
  return LOCRET_OK;
}

int locret_set_timing(locret_layer *L, int32_t enable) {
  if (!L) return LOCRET_ERR_INVALID;
  L->timing = enable != 0;
  L->serialize = enable == 2;
  L->attn_only = enable == 3;
  return LOCRET_OK;
}

int locret_read_timing(locret_layer *L, float *ms, int64_t *launches) {
  if (!L || !ms || !launches || !on_layer_device(L)) return LOCRET_ERR_INVALID;
  for (int i = 0; i < LOCRET_K_COUNT; i++) { ms[i] = 0.f; launches[i] = 0; }
  CK(sync_all(L));
  for (size_t i = 0; i < L->events_used; i++) {
    float t = 0.f;
    CK(cudaEventElapsedTime(&t, L->events[i].a, L->events[i].b));
    ms[L->events[i].kind] += t;
    launches[L->events[i].kind]++;
  }
  L->events_used = 0;
  return LOCRET_OK;
}

int locret_launch_count(const locret_layer *L, int64_t *count) {
  if (!L || !count) return LOCRET_ERR_INVALID;
  *count = L->launches;
  return LOCRET_OK;
}

void locret_destroy(locret_layer *L) {
  if (!L) return;
  sync_all(L);
  ScratchPool *p = L->pool;
  free_layer_memory(L);
  delete L;
  release_pool(p);
}

}  // extern "C"
