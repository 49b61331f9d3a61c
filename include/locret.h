/*
 * locret.h — C ABI of the B200 (sm_100a) library for the per-layer chunked-prefill
 * step with retaining-head eviction (Locret, arXiv 2410.01805).
 *
 * One `locret_layer` holds the state of one decoder layer's attention block: the
 * retained cache units (pre-RoPE K, V), their causal importance scores, their token
 * ids, and scratch.  One `locret_prefill_chunk` call is one iteration of the loop
 * body of Algorithm 1 for that layer:
 *
 *   (a) [Q ‖ K ‖ V] = hidden_in · W_qkv                                  (Section 3.1)
 *   (b) attention of the chunk's queries over the retained cache plus the causal
 *       chunk, positions re-assigned contiguously from 0                 (Eq. 1, Section 3.4)
 *   (c) retaining head  S~ = sigma([Q ‖ K ‖ V] W1) W2, one score per KV head per
 *       token, W1 of size (h + 2 h_kv) d × d_R                           (Section 3.3)
 *   (d) concatenate cache and chunk, protect the last n_stab units, keep the
 *       top-`budget` per KV head, gather K, V, scores in temporal order  (Algorithm 1)
 *
 * Conventions
 *   - Every function returns 0 (LOCRET_OK) or a negative LOCRET_ERR_* code; nothing
 *     throws, aborts or exits.  Arguments are validated before anything is launched.
 *   - "device" pointers are CUDA device memory of the current device, 16-byte aligned;
 *     "host" pointers are ordinary host memory.  The caller owns every buffer it
 *     passes; the library owns the cache, scores, token ids, scratch and its own
 *     repacked copy of the weights (taken at create; the caller's weights may be
 *     freed afterwards).
 *   - All device work of a layer is enqueued without host synchronisation unless stated:
 *     projection, RoPE/append and attention (everything attn_out depends on) on the stream
 *     given at create; the retaining head, selection and compaction, which nothing downstream
 *     in a decoder layer waits for, on a second stream owned by the library, ordered against
 *     the first by events (set LOCRET_SERIAL=1 to keep everything on one stream).  Every call
 *     that reads or replaces state waits for both.  A handle is bound to its stream and is
 *     not thread-safe.  Layers created on the same stream of the same device share scratch.
 *   - A handle belongs to the device that was current when it was created (one process may
 *     create layers on several devices).  Every call that takes the handle must be made with
 *     that device current, else it returns LOCRET_ERR_INVALID and launches nothing
 *     (locret_destroy, locret_cache_len and the other host-only calls work from any device).
 *   - There is no CPU fallback: without a CUDA device every call that needs one
 *     returns LOCRET_ERR_CUDA.
 *   - Kernel selection, read from the environment when a layer is created (for A/B measurements;
 *     results agree within the stated tolerances): LOCRET_ATTN_PAIR=1 runs Eq. 1 for head_dim 128
 *     on a cluster of two CTAs per pair of query tiles (tcgen05 cta_group::2) instead of one CTA;
 *     it is faster and opt-in (bench.py sets it), and a divided-heads step never uses it.
 *     LOCRET_LEGACY_MMA=1 keeps every product on mma.sync kernels; LOCRET_UNFUSED_ROPE=1 runs
 *     positions, RoPE and the cache append as a pass of their own; LOCRET_NO_PDL=1 launches the
 *     one-token kernels without programmatic dependent launch; LOCRET_DIAG_STATUS=1 makes
 *     locret_sync_status print which kernel family recorded a device-side time-out.
 */
#ifndef LOCRET_H_
#define LOCRET_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LOCRET_OK                  0
#define LOCRET_ERR_INVALID        (-1)  /* bad argument or configuration                    */
#define LOCRET_ERR_ALLOC          (-2)  /* device or host allocation failed                 */
#define LOCRET_ERR_CAPACITY       (-3)  /* len + n_tok exceeds budget + chunk + reserve     */
#define LOCRET_ERR_CUDA           (-4)  /* a CUDA runtime/driver call failed                */
#define LOCRET_ERR_DEVICE_TIMEOUT (-5)  /* a bounded device-side wait gave up (sticky)      */

/* flags of locret_prefill_chunk */
#define LOCRET_NO_EVICT    1u  /* append only (Algorithm 1's n_loc tail pass and decode)     */
#define LOCRET_LAST_CHUNK  2u  /* evict without protecting stabilizers (Algorithm 1's
                                  "if chunk is not the last chunk" test, negated)            */

/* kernel families, indices into locret_read_timing's arrays */
enum {
  LOCRET_K_QKV = 0,     /* (a) projection GEMM (positions, RoPE and append in the   */
                        /*     same kernel)                                        */
  LOCRET_K_ROPE,        /* position assignment + RoPE + append of the chunk, where */
                        /*     it is a kernel of its own (fallback shapes)         */
  LOCRET_K_ATTN,        /* (b) attention                                          */
  LOCRET_K_RH,          /* (c) retaining head GEMM -> activation -> GEMM          */
  LOCRET_K_RH_REDUCE,   /* (c) sum of the retaining head's partial scores (a      */
                        /*     one-token step sums them inside LOCRET_K_RH)        */
  LOCRET_K_TOPK,        /* (d) per-head selection                                 */
  LOCRET_K_COMPACT,     /* (d) gather in place + re-RoPE of keys whose position   */
                        /*     changed                                            */
  LOCRET_K_DEQUANT,     /* 4-bit cache: expansion of the retained units to bf16   */
  LOCRET_K_QUANT,       /* 4-bit cache: quantisation of the chunk's units         */
  LOCRET_K_COUNT
};

typedef struct locret_layer locret_layer;   /* opaque */

typedef struct {
  int32_t d_model;      /* D: width of hidden_in                                              */
  int32_t n_q_heads;    /* h                                                                  */
  int32_t n_kv_heads;   /* h_kv = h / g; h must be a multiple of it                           */
  int32_t head_dim;     /* d_m in the paper: 64, 96 or 128                                    */
  int32_t d_retain;     /* d_R, hidden size of the retaining head (Section 4.1: 1024)         */
  int32_t act;          /* sigma: 0 SiLU, 1 GELU (tanh form), 2 ReLU (Appendix A: the
                           backbone's own non-linearity)                                      */
  float   rope_theta;   /* RoPE base                                                          */
  int32_t rh_input;     /* 0: retaining head reads pre-RoPE [Q ‖ K ‖ V]; 1: post-RoPE Q, K    */
  int32_t kv_dtype;     /* 0: bf16 cache; 1: int4 codes + one fp16 scale per head vector      */
  int32_t reserve;      /* cache slots beyond budget + chunk, for NO_EVICT appends            */
  const void *w_qkv;    /* device bf16 [d_model × (h + 2 h_kv) d] row-major; columns: the h
                           query heads, then the h_kv key heads, then the h_kv value heads    */
  const void *w1;       /* device bf16 [(h + 2 h_kv) d × d_R] row-major                       */
  const void *w2;       /* device bf16 [d_R × h_kv] row-major                                 */
  void *stream;         /* cudaStream_t; NULL = the legacy default stream                     */
} locret_layer_cfg;

/*
 * Create one layer's state for chunked prefill with a fixed cache budget (Section 3.4;
 * hyper-parameters b, B, n_s of Table 4).  Requires 1 <= chunk, 1 <= budget,
 * 0 <= n_stab <= budget, budget + chunk + reserve <= 262144.  Allocates device memory (cache
 * for budget + chunk + reserve units per KV head; scratch), repacks the weights, and
 * synchronises the stream once.  On failure *out is NULL and nothing stays allocated.
 */
int locret_create(const locret_layer_cfg *cfg, int32_t budget, int32_t chunk, int32_t n_stab,
                  locret_layer **out);

/*
 * One chunked-prefill step (loop body of Algorithm 1; attention per Eq. 1; scores per
 * Section 3.3).  hidden_in: device bf16 [n_tok × d_model], row-major, 1 <= n_tok <= chunk.
 * attn_out: device bf16 [n_tok × h·d] (concatenated heads, before W^O).
 * With flags = 0 the last min(n_stab, len + n_tok) units are protected and the cache is
 * cut to `budget` units per KV head; afterwards len = min(budget, len + n_tok).
 * Asynchronous on the layer's stream.  LOCRET_ERR_CAPACITY if a NO_EVICT append does
 * not fit.
 */
int locret_prefill_chunk(locret_layer *layer, const void *hidden_in, int32_t n_tok,
                         uint32_t flags, void *attn_out);

/*
 * Decoding: the B = 1 case of Eq. 1 (Algorithm 1's generate).  hidden_in: device bf16
 * [d_model]; attn_out: device bf16 [h·d].  Scores the new unit and appends it without
 * eviction (uses a `reserve` slot).
 */
int locret_decode_step(locret_layer *layer, const void *hidden_in, void *attn_out);

/*
 * locret_decode_step for several layers in one call, in order: every layer receives the same
 * hidden_in and layer i writes attn_out + i * out_stride elements (out_stride a multiple of 8; 0:
 * all layers write the same buffer).  For harnesses that drive the attention blocks of a stack
 * alone, where the cost of crossing into the library once per layer is comparable to a layer-step
 * on the device; in a model the caller computes the next layer's input in between and calls
 * locret_decode_step per layer.  Stops at the first layer that returns an error and returns it.
 */
int locret_decode_step_stack(locret_layer *const *layers, int32_t n_layers, const void *hidden_in,
                             void *attn_out, int64_t out_stride);

/*
 * The same step with the KV heads (and the query heads of their groups) divided over several
 * GPUs, one layer object per GPU.  Heads attend and evict independently (Algorithm 1 runs per
 * head) and only the retaining head reads every head's [Q, K, V] (Section 3.3), so the GPUs
 * exchange one thing per step: the sum of their partial first products z_local · W1_local.
 *
 * A GPU's layer object is created by locret_create with its share of the heads: n_q_heads and
 * n_kv_heads are the local counts, w_qkv holds the columns of its query, key and value heads
 * (in that order), w1 the matching rows [(h_local + 2 h_kv_local)·d x d_R], w2 the columns of
 * its KV heads [d_R x h_kv_local].  budget, chunk and n_stab are the same on every GPU, so
 * cache lengths and positions agree without communication.
 *
 * locret_prefill_chunk_tp_begin: steps (a), (b) as in locret_prefill_chunk for the local heads
 *   (attn_out: device bf16 [n_tok x h_local·d]), then preact_partial (device fp32
 *   [n_tok x d_R], 16-byte aligned, caller-owned) = z_local · W1_local.  Work enqueued on the
 *   layer's stream after the call returns sees the finished product.  The caller sums
 *   preact_partial over the GPUs on that stream (an all-reduce) and passes the sum to
 * locret_prefill_chunk_tp_finish: scores = act(preact_sum) · W2_local for the chunk's units, then
 *   step (d) as in locret_prefill_chunk (with the flags given to _begin).  preact_sum may be the
 *   buffer given to _begin.  It is read asynchronously (what was enqueued on the layer's stream
 *   before the call is seen): leave it unchanged until this layer's next call or
 *   locret_sync_status.
 * Between the two calls the layer accepts no other step (LOCRET_ERR_INVALID); locret_reset
 * abandons a begun step.  _finish without _begin returns LOCRET_ERR_INVALID.
 */
int locret_prefill_chunk_tp_begin(locret_layer *layer, const void *hidden_in, int32_t n_tok,
                                  uint32_t flags, void *attn_out, float *preact_partial);
int locret_prefill_chunk_tp_finish(locret_layer *layer, const float *preact_sum);

/*
 * The exchange of the divided step done by the GEMM itself (Section 3.3: the retaining head reads
 * every head).  locret_tp_set_peers registers, once, the sum buffers of all n_peers GPUs, this GPU's
 * among them: peer_sums is a HOST array of n_peers device pointers, each fp32 [chunk x d_R], 16-byte
 * aligned; a buffer of another GPU must be mapped into this process (peer access or an IPC handle).
 * Synchronises the layer's streams; allocates a few hundred bytes (and a [chunk x d_R] scratch).
 * locret_prefill_chunk_tp_begin_peers is locret_prefill_chunk_tp_begin whose first product is not
 * written to a buffer of the caller but ADDED, tile by tile in the GEMM's epilogue, into rows
 * [0, n_tok) of EVERY registered buffer, with plain reductions to global memory at system scope (no
 * TMA and no multicast ever touches a peer's memory).  The caller provides the two orderings an
 * all-reduce would: every buffer is zero before any GPU starts adding, and every GPU has finished
 * adding (its begin call's work on the layer's stream is complete) before any GPU's
 * locret_prefill_chunk_tp_finish reads its own buffer.  Each GPU sends its product n_peers - 1 times
 * over the links; sums may differ from an all-reduce's in the last bits (the order of the additions is
 * not fixed).  Not run on more than one GPU by the tests of this library: there all the buffers live on
 * one device.
 */
int locret_tp_set_peers(locret_layer *layer, float *const *peer_sums, int32_t n_peers);
int locret_prefill_chunk_tp_begin_peers(locret_layer *layer, const void *hidden_in, int32_t n_tok, uint32_t flags,
                                        void *attn_out);

/* Number of retained units per KV head (the same for every head).  No device work. */
int locret_cache_len(const locret_layer *layer, int32_t *len);

/*
 * Copy the retained state to HOST buffers (any may be NULL to skip it): K and V as bf16
 * [h_kv × len × d] (K pre-RoPE), scores fp32 [h_kv × len], token_ids int64 [h_kv × len]
 * (index of the token in the stream), *len, *tokens_seen.  Units come in temporal order (the
 * order of Algorithm 1's gather), whatever slots they occupy on the device.  Synchronises the stream.
 * A layer with a 4-bit cache returns LOCRET_ERR_INVALID if K or V is asked for (its state
 * is exchanged exactly through locret_export_state_int4).
 */
int locret_export_state(locret_layer *layer, void *K, void *V, float *scores,
                        int64_t *token_ids, int32_t *len, int64_t *tokens_seen);

/*
 * Replace the retained state from HOST buffers laid out as in locret_export_state
 * (all four required), 0 <= len <= budget + chunk + reserve.  Rebuilds the rotated-key
 * scratch at positions 0..len-1.  LOCRET_ERR_INVALID for a layer with a 4-bit cache.
 * Synchronises the stream.
 */
int locret_import_state(locret_layer *layer, const void *K, const void *V, const float *scores,
                        const int64_t *token_ids, int32_t len, int64_t tokens_seen);

/*
 * The same two calls for a layer created with kv_dtype = 1 (the 4-bit cache that Appendix H
 * combines with the method): codes uint8 [h_kv × len × d/2], two symmetric 4-bit codes in
 * [-8, 7] per byte with the even element in the low nibble; scales IEEE half [h_kv × len], one
 * per head vector (scale = half(absmax / 7), 1 if that is zero; element = code · scale).
 * HOST buffers; both synchronise the stream.
 */
int locret_export_state_int4(locret_layer *layer, void *k_codes, void *k_scales, void *v_codes,
                             void *v_scales, float *scores, int64_t *token_ids, int32_t *len,
                             int64_t *tokens_seen);
int locret_import_state_int4(locret_layer *layer, const void *k_codes, const void *k_scales,
                             const void *v_codes, const void *v_scales, const float *scores,
                             const int64_t *token_ids, int32_t len, int64_t tokens_seen);

/* Synchronise the stream; return the sticky device status (0, or LOCRET_ERR_*). */
int locret_sync_status(locret_layer *layer);

/*
 * Self-test of the bounded device-side waits: launches a one-warp kernel whose mbarrier wait
 * can never complete, with a limit of a few thousand polls, and returns the status word that
 * kernel leaves.  The expected return value is LOCRET_ERR_DEVICE_TIMEOUT; the context stays
 * usable.  (Diagnostic only; nothing on the hot path calls it.)  Synchronises `stream`.
 */
int locret_selftest_wait_timeout(void *stream);

/*
 * Self-test of the give-up path of the production wait itself (the routine every tcgen05 kernel
 * of the library polls its mbarriers with).  Two warps of one CTA wait on barriers nothing ever
 * arrives at: warp 0 with a limit of a few thousand polls, warp 1 with the production limit.
 * Warp 0 gives up, sets the CTA's abort flag and the status word; warp 1 must notice the flag
 * and stop long before its own limit.  report (HOST, 4 x int64): [0] the status word the kernel
 * left (expected LOCRET_ERR_DEVICE_TIMEOUT), [1] 1 if warp 1's wait returned "abandoned",
 * [2] clock cycles warp 0 waited, [3] clock cycles warp 1 waited.  Returns 0, or
 * LOCRET_ERR_ALLOC / LOCRET_ERR_CUDA.  Nothing faults, traps or hangs; the context stays usable.
 * Synchronises `stream`.
 */
int locret_selftest_wait_abort(void *stream, int64_t *report);

/* Forget all units: len = 0, tokens_seen = 0.  Asynchronous: nothing is launched; the layer's
 * stream is ordered behind any selection / compaction of this layer still in flight on the
 * library's second stream, so work enqueued after the reset finds the cache quiescent. */
int locret_reset(locret_layer *layer);

/*
 * Query-aware variant (Section 4.4; Appendix "Evaluating Locret-Q on RULER"): the query is
 * placed at the start of the sequence and has to stay visible across every eviction.  After
 * this call every evicting step keeps cache slots [0, n_prefix) besides the last n_stab
 * units, and chooses budget - n_stab - n_prefix units among the slots between them (with
 * LOCRET_LAST_CHUNK: budget - n_prefix).  Slots are in temporal order, so set before the
 * first evicting step the prefix is tokens 0 .. n_prefix-1 for the life of the stream; set
 * later it is whatever then occupies the first slots.  n_prefix = 0 (the default, and the
 * state after create) is Algorithm 1 unchanged.  Host-side state only: nothing is launched
 * and nothing on the device changes.  Requires 0 <= n_prefix and n_prefix + n_stab <= budget,
 * else LOCRET_ERR_INVALID and the previous value stays.  locret_reset keeps the value.
 */
int locret_set_protected_prefix(locret_layer *layer, int32_t n_prefix);

/*
 * A budget per KV head (Appendix H, the combination with head-wise budget allocation: "Locret evicts
 * cache units across the attention heads independently", so budgets may differ between heads; a budget
 * per layer is simply the `budget` each layer is created with).  budgets: HOST int32 [n_kv_heads], each
 * 1 <= b_m <= the budget given at create (which sizes the cache) and >= n_stab + protected prefix.
 * Allowed only while the layer is empty (right after create or locret_reset); LOCRET_ERR_INVALID for a
 * 4-bit cache.  From then on head m keeps min(b_m, tokens seen) units: its cache slot i sits at position i
 * and the chunk's token t at len_m + t (Section 3.4), its query heads use those positions, and it is cut
 * to b_m by every evicting step in which it holds more; the retaining head still reads all heads'
 * [Q, K, V].  Steps with head budgets use the general kernels (projection, then positions / RoPE / append
 * in a pass of their own; one-token steps take the chunk kernels); the divided-heads calls are refused.
 * locret_cache_len then returns the largest length; locret_cache_lens all of them (HOST int32
 * [n_kv_heads]; also valid without head budgets).  State is exchanged with the _heads calls below:
 * arrays as in locret_export_state but with `pitch` rows per head (pitch >= the largest length), head
 * m's first lens[m] rows valid, in temporal order; the plain export / import calls are refused.
 */
int locret_set_head_budgets(locret_layer *layer, const int32_t *budgets);
int locret_cache_lens(const locret_layer *layer, int32_t *lens);
int locret_export_state_heads(locret_layer *layer, void *K, void *V, float *scores, int64_t *token_ids,
                              int32_t pitch, int32_t *lens, int64_t *tokens_seen);
int locret_import_state_heads(locret_layer *layer, const void *K, const void *V, const float *scores,
                              const int64_t *token_ids, int32_t pitch, const int32_t *lens, int64_t tokens_seen);

/*
 * Per-kernel timing.  With enable != 0 every kernel launched for this layer is
 * bracketed by CUDA events on the stream it runs on (kernels on the two streams overlap, so
 * the per-kernel times of a step add up to more than its duration); enable = 2 also keeps
 * every kernel on the layer's own stream, which gives each kernel's time when it runs alone;
 * enable = 3 brackets only the attention kernel (the dominant one), for the least overhead.  locret_read_timing synchronises the
 * stream, adds up the elapsed time and the number of launches per kernel family since
 * the last read into ms[LOCRET_K_COUNT] and launches[LOCRET_K_COUNT] (host arrays), and
 * clears the record.
 */
int locret_set_timing(locret_layer *layer, int32_t enable);
int locret_read_timing(locret_layer *layer, float *ms, int64_t *launches);

/* Total number of this library's kernels launched for the layer since create. */
int locret_launch_count(const locret_layer *layer, int64_t *count);

/*
 * How much the evictions of this layer have moved since create (Algorithm 1's gather, done in place:
 * kept units stay in their slots, units kept from the chunk refill the freed slots, and a rotated key
 * is rewritten only where the unit's position in temporal order changed, Section 3.4).  *units_moved:
 * units (one token of one KV head) copied to another slot; *keys_rotated: rotated keys rewritten.
 * Either pointer may be NULL.  Synchronises the layer's streams.
 */
int locret_compaction_counters(locret_layer *layer, int64_t *units_moved, int64_t *keys_rotated);

/*
 * ---- The rest of the decoder layer (beyond the scope of the chunk step itself) ----
 *
 * Section 3.1 writes a layer as A = [A_1 .. A_h] W^O followed by H = FFN(A) and leaves
 * normalisation, residual connections and the form of the FFN to the backbone; both backbones
 * of the paper are pre-norm decoders with a gated SiLU FFN, which is what a block computes:
 *     h1 = RMSNorm(x; g1)   ->   the attention block above (hidden_in = h1), with eviction
 *     x1 = x + attn_out W_o
 *     h2 = RMSNorm(x1; g2)
 *     y  = x1 + (silu(h2 W_gate) * (h2 W_up)) W_down
 * so that a stack of blocks can be fed real hidden states, layer after layer.  bf16 storage of
 * h1, attn_out, x1, h2, the gated product and y; fp32 accumulation everywhere.
 */
typedef struct locret_block locret_block;

typedef struct {
  locret_layer_cfg attn;  /* the attention block (its w_qkv multiplies h1)                       */
  int32_t d_ff;           /* FFN hidden size; a multiple of 128                                   */
  float   rms_eps;        /* epsilon of both RMSNorms (1e-5 if <= 0)                              */
  const void *w_o;        /* device bf16 [h·d × d_model] row-major; borrowed until create returns */
  const void *w_gate;     /* device bf16 [d_model × d_ff]                                         */
  const void *w_up;       /* device bf16 [d_model × d_ff]                                         */
  const void *w_down;     /* device bf16 [d_ff × d_model]                                         */
  const void *g1, *g2;    /* device bf16 [d_model]: gains of the two RMSNorms                     */
} locret_block_cfg;

/*
 * Create a block: the attention layer (locret_create with the same budget, chunk, n_stab) plus
 * repacked copies of the four weight matrices and scratch shared by the blocks of one stream.
 * On failure *out is NULL and nothing stays allocated.
 */
int locret_block_create(const locret_block_cfg *cfg, int32_t budget, int32_t chunk, int32_t n_stab,
                        locret_block **out);

/*
 * One chunk through the whole layer.  x_in, y_out: device bf16 [n_tok × d_model], 16-byte
 * aligned, 1 <= n_tok <= chunk; they may be the same buffer.  flags as for
 * locret_prefill_chunk.  Asynchronous on the stream of cfg.attn.
 */
int locret_block_prefill_chunk(locret_block *block, const void *x_in, int32_t n_tok, uint32_t flags,
                               void *y_out);

/* The block's attention layer, for state export/import, status, timing (owned by the block). */
locret_layer *locret_block_attention(locret_block *block);

void locret_block_destroy(locret_block *block);

/*
 * Training labels of the retaining heads (Section 3.3): for prompt token k and KV head m the
 * causal importance score is the largest attention score before the softmax that any answer
 * token gives to k, over the query heads of the group:
 *     labels[m][k] = scale * max over p < n_a, j in group m of  q_ans[p][j] . k_prompt[k][m].
 * q_ans: device bf16 [n_a × h × d] (queries of the answer tokens as they enter the scores, i.e.
 * after RoPE); k_prompt: device bf16 [n_q × h_kv × d]; labels: device fp32 [h_kv × n_q]
 * (overwritten).  The passage prints the product without the 1/sqrt(d) of Eq. 1: scale = 1
 * reproduces it as printed; scale must be > 0.  head_dim 64, 96 or 128; pointers 16-byte aligned.
 * One tensor-core contraction per query head whose epilogue keeps only row maxima (the
 * n_q × n_a score matrix is never written).  Synchronises the stream before it returns.
 */
int locret_cis_labels(const void *q_ans, const void *k_prompt, int32_t n_a, int32_t n_q, int32_t h,
                      int32_t h_kv, int32_t d, float scale, float *labels, void *stream);

/*
 * Training objective of the retaining head for one sequence (Eq. 2, Eq. 3), backbone frozen:
 *     s~ = silu(z W1) W2,   L = sum_{k,m} SmoothL1(s~[k][m] - labels[m][k]) + alpha sum_{k<n-1,m} (s~[k][m] - s~[k+1][m])^2
 * and its gradients dL/dW1, dL/dW2.  Readings where the text is silent: Smooth-L1 threshold 1,
 * the L2 term as the plain square, sums rather than means; SiLU only.
 * z: device bf16 [n × d_in] (the tokens' [Q ‖ K ‖ V]); labels: device fp32 [h_kv × n] (e.g. from
 * locret_cis_labels); w1: device bf16 [d_in × d_R]; w2: device bf16 [d_R × h_kv]; outputs on the
 * device: loss (one fp32), d_w1 fp32 [d_in × d_R], d_w2 fp32 [d_R × h_kv] (all overwritten).
 * Requires n, d_in multiples of 64, d_R a multiple of 32, h_kv <= 32, alpha >= 0.  The two
 * large contractions take bf16 operands (dpre is rounded to bf16) and accumulate in fp32.
 * Allocates and frees its workspace (about n·(4 d_R + 2 d_in + 2 d_R) bytes) inside the call and
 * synchronises the stream before it returns.
 */
int locret_rh_loss_grad(const void *z, const float *labels, const void *w1, const void *w2, int32_t n,
                        int32_t d_in, int32_t d_R, int32_t h_kv, float alpha, float *loss, float *d_w1,
                        float *d_w2, void *stream);

/*
 * One AdamW update of a parameter array (Appendix A: AdamW, learning rate 5e-4 with a linear
 * warm-up schedule; the schedule is the caller's).  param: device fp32 master copy [n], updated
 * in place; param_bf16: device bf16 [n] that receives the rounded parameters, or NULL; grad: device
 * fp32 [n]; m, v: device fp32 [n] moment estimates (zero before the first step), updated in place.
 * step counts from 1 (bias correction).  Decoupled weight decay: p <- p (1 - lr wd) - lr m^/(sqrt(v^) + eps).
 * Asynchronous on the stream.
 */
int locret_adamw_step(float *param, void *param_bf16, const float *grad, float *m, float *v, int64_t n,
                      int32_t step, float lr, float beta1, float beta2, float eps, float weight_decay,
                      void *stream);

/*
 * Retaining-head scores without any allocation.  (The paper has no counterpart: this entry
 * point exists for hosts that may not allocate device memory where they need scores, e.g. code
 * that runs inside a pool owning the whole device, or under an allocator that is locked while
 * a request is in flight.)
 *
 * Computes scores[m][t] = sum_r act( sum_c z[t][c] * w1_t[r][c] ) * w2[r][m], the same
 * arithmetic, kernels and summation order as step (c) of locret_prefill_chunk.
 *   z       device bf16 [n_tok x d_in], row-major: the tokens' concatenated [Q ‖ K ‖ V]
 *   w1_t    device bf16 [d_retain x d_in], row-major: W1 TRANSPOSED (the layer API repacks W1
 *           into this form at create; here the caller supplies it, since repacking allocates)
 *   w2      device fp32 [d_retain x n_kv_heads], row-major
 *   scores  device fp32 [n_kv_heads x n_tok], written entirely
 * Requires d_in % 64 == 0, d_retain % 32 == 0, 1 <= n_kv_heads <= 32, act in {0,1,2}, z and w1_t
 * 16-byte aligned.  The per-tile partial sums live in a fixed array inside the library image of
 * LOCRET_STATIC_SCRATCH_FLOATS floats (4 MiB, present on every GPU that loads the library until
 * the process exits); a call needs ceil(d_retain / 64) * n_tok * n_kv_heads of them and returns
 * LOCRET_ERR_CAPACITY, launching nothing, if that is more.
 * status: device int32 that receives LOCRET_ERR_DEVICE_TIMEOUT if a bounded wait inside the kernel
 * gives up (the caller clears and reads it), or NULL: then such a give-up goes unreported and the
 * scores of that call are garbage.
 * The call makes no cudaMalloc/cudaFree and uses no allocating library routine.  Its first call on
 * a device looks up the array's device address (cudaGetSymbolAddress, with that device current);
 * make that first call outside of any stream capture.  All calls share the one array, which
 * keeps the previous call's contents (nothing in it needs clearing: a call writes every value it
 * later reads); two calls whose kernels overlap on the GPU (different streams, no dependency)
 * race on it.  Asynchronous on `stream` (cudaStream_t; NULL = legacy default stream).
 */
#define LOCRET_STATIC_SCRATCH_FLOATS (1 << 20)
int locret_rh_scores_static(const void *z, int32_t n_tok, int32_t d_in, const void *w1_t,
                            int32_t d_retain, const float *w2, int32_t n_kv_heads, int32_t act,
                            float *scores, int32_t *status, void *stream);

/* Free everything the layer owns.  Synchronises the stream.  NULL is allowed. */
void locret_destroy(locret_layer *layer);

const char *locret_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LOCRET_H_ */
