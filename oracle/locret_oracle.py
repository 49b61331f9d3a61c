"""CPU oracle for the per-layer chunked-prefill step with retaining-head eviction.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain fp64 restatement of the
method that the CUDA library is checked against.  It shares no code with the
CUDA path and must never be imported by the product package; only the tests,
the smoke check and the benchmark's CPU-baseline leg may use it.

What each function follows:

* ``project_qkv``          – the per-layer projection [Q, K, V] = H · [W^Q, W^K, W^V]
                             (Section 3.1, "Transformer Architecture").
* ``rope``                 – rotary embedding at re-assigned contiguous positions
                             (Section 3.4: the cache is kept pre-RoPE and positions are
                             re-assigned from the beginning at every step).
* ``attention_rows``       – Eq. 1: chunk queries over retained cache + causal chunk,
                             GQA map ceil(j/g), scale 1/sqrt(d_m).
* ``retaining_scores``     – S~ = sigma([Q, K, V] W1) W2 (Section 3.3).
* ``select_keep``          – Algorithm 1: last n_s scores set to +inf, top-b, gather
                            (+ the protected prefix of the query-aware variant, Section 4.4)
                             (stated without infinities: protected ∪ top-(b − n_prot) of the rest).
* ``OracleLayer.prefill_chunk`` – one iteration of Algorithm 1's loop body for one layer.
* ``shard_by_kv_head`` / ``OracleLayer.partial_preact`` / ``tp_prefill_chunk`` – the same step
                             with the KV heads (and their query groups) divided over several
                             workers: heads attend and evict independently (Algorithm 1 runs
                             per head), the retaining head reads every head's [Q, K, V]
                             (Section 3.3), so the workers exchange one thing, the sum of
                             their partial products z_local · W1_local, before the activation.
* ``OracleLayerHeadBudgets`` – the same step with one budget per KV head (Appendix H: heads evict
                             independently, so budgets may differ between them).
* ``quantize_int4`` / ``dequantize_int4`` – the 4-bit cache variant (Appendix H combines
                             a 4-bit KV cache with the method; the number format is the
                             workload's: symmetric, one fp16 scale per head vector).

Readings taken where the paper is silent are listed in the design notes of the
repository; the ones that matter here: W1 has (h + 2 h_kv)·d rows (all heads
concatenated, order Q heads, K heads, V heads); the activation is SiLU by
default; the retaining head sees the pre-RoPE projections by default; kept
units stay in temporal order; ties prefer the more recent unit; NaN scores rank
as −inf; the protected units are the last min(n_s, n) entries of cache ‖ chunk.

Two modes.  ``mirror=False``: no rounding anywhere (used for the pins).
``mirror=True``: values are rounded to bfloat16 exactly where the CUDA path
stores them (Q, K, V after projection; Q, K after RoPE; dequantised int4
values); everything else stays fp64.
"""

from __future__ import annotations

import numpy as np

NO_EVICT = 1
LAST_CHUNK = 2


class CapacityError(RuntimeError):
    pass


# --------------------------------------------------------------------------- rounding

def _round_sig(x, sig_bits: int, min_frexp_exp: int):
    """Round fp64 to a binary format with `sig_bits` significant bits (ties to even)."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    e = np.maximum(e, min_frexp_exp)
    q = np.ldexp(1.0, e - sig_bits)
    with np.errstate(invalid="ignore"):
        r = np.rint(x / q) * q
    return np.where(np.isfinite(x), r, x)


def round_bf16(x):
    """Nearest bfloat16 (8 significant bits), returned as fp64."""
    return _round_sig(x, 8, -125)


def round_fp16(x):
    """Nearest IEEE half (11 significant bits, subnormals below 2^-14), as fp64."""
    return _round_sig(x, 11, -13)


# --------------------------------------------------------------------------- steps

def project_qkv(X, w_qkv, h: int, h_kv: int, d: int):
    """[Q ‖ K ‖ V] = X · W_qkv; columns: h query heads, h_kv key heads, h_kv value heads."""
    qkv = np.asarray(X, np.float64) @ np.asarray(w_qkv, np.float64)
    return qkv


def split_qkv(qkv, h: int, h_kv: int, d: int):
    n = qkv.shape[0]
    Q = qkv[:, : h * d].reshape(n, h, d)
    K = qkv[:, h * d: (h + h_kv) * d].reshape(n, h_kv, d)
    V = qkv[:, (h + h_kv) * d:].reshape(n, h_kv, d)
    return Q, K, V


def rope(x, pos, theta: float):
    """Rotate-half rotary embedding: pairs (i, i + d/2), angle pos · theta^(−2i/d).

    x: [..., d]; pos broadcastable to x.shape[:-1].
    """
    x = np.asarray(x, np.float64)
    d = x.shape[-1]
    half = d // 2
    inv_freq = np.float64(theta) ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(pos, np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def attention_rows(Qr, Kr_cache, V_cache, Kr_chunk, V_chunk, group: int, rows=None, abs_out=None,
                   flip_sens=None):
    """Eq. 1 for the chunk's query rows.

    Qr [n, h, d] (roped); Kr_cache/V_cache [h_kv, len, d]; Kr_chunk/V_chunk [n, h_kv, d].
    Query t attends to every cache unit and to chunk units u <= t.
    Returns out [n, h*d]; rows not listed in `rows` are NaN.
    If `abs_out` (same shape) is given it receives sum_i p_i |V_i|, the magnitude of the
    terms the output sums, which error bounds of reduced-precision kernels scale with.
    If `flip_sens` (same shape) is given it receives the first-order change of the output when
    every key has one stored element moved by one bf16 ulp at its most influential position:
    sum_i p_i delta_i |V_i - out|, delta_i = 2^-7 max_c |q_c k_ic| / sqrt(d).
    """
    n, h, d = Qr.shape
    ln = Kr_cache.shape[1]
    rows = np.arange(n) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.full((n, h * d), np.nan)
    scale = 1.0 / np.sqrt(np.float64(d))
    u = np.arange(n)
    for j in range(h):
        m = j // group                      # 0-based form of ceil(j/g)
        Kall = np.concatenate([Kr_cache[m], Kr_chunk[:, m, :]], axis=0)
        Vall = np.concatenate([V_cache[m], V_chunk[:, m, :]], axis=0)
        logits = (Qr[rows, j, :] @ Kall.T) * scale
        masked = u[None, :] > rows[:, None]              # chunk unit after the query
        logits[:, ln:][masked] = -np.inf
        logits -= logits.max(axis=1, keepdims=True)
        p = np.exp(logits)
        p /= p.sum(axis=1, keepdims=True)
        out[rows, j * d:(j + 1) * d] = p @ Vall
        if abs_out is not None:
            abs_out[rows, j * d:(j + 1) * d] = p @ np.abs(Vall)
        if flip_sens is not None:
            o = out[rows, j * d:(j + 1) * d]
            for a, t in enumerate(rows):
                delta = 2.0 ** -7 * np.max(np.abs(Qr[t, j, :][None, :] * Kall), axis=1) * scale
                flip_sens[t, j * d:(j + 1) * d] = (p[a] * delta) @ np.abs(Vall - o[a][None, :])
    return out


def activation(x, act: int):
    if act == 0:      # SiLU
        return x / (1.0 + np.exp(-x))
    if act == 1:      # GELU, tanh form
        return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))
    if act == 2:
        return np.maximum(x, 0.0)
    raise ValueError(act)


def retaining_scores(z, w1, w2, act: int = 0):
    """S~ = sigma(z W1) W2, one score per KV head per token; z = [Q ‖ K ‖ V] of the token."""
    hidden = activation(np.asarray(z, np.float64) @ np.asarray(w1, np.float64), act)
    return hidden @ np.asarray(w2, np.float64)


def select_keep(scores, budget: int, n_prot: int, n_prefix: int = 0):
    """Slots kept by one head: the last n_prot, plus the best (budget − n_prot) of the rest.

    Order among the rest: higher score first; equal scores: more recent slot first;
    NaN ranks as −inf.  Returns ascending slot indices (temporal order).

    n_prefix > 0 (the query-aware variant of Section 4.4: the query sits at the start of the
    sequence and has to stay visible across every eviction) also keeps slots [0, n_prefix);
    the choice is then among the slots between the two protected ends.
    """
    s = np.array(scores, dtype=np.float64)
    n = s.shape[0]
    if n <= budget:
        return np.arange(n, dtype=np.int64)
    n_prot = min(n_prot, n, budget)
    n_prefix = min(n_prefix, budget - n_prot)
    rest = n - n_prot
    sr = np.where(np.isnan(s[n_prefix:rest]), -np.inf, s[n_prefix:rest])
    idx = np.arange(n_prefix, rest, dtype=np.int64)
    order = np.lexsort((-idx, -sr))          # primary: score desc; secondary: slot desc
    chosen = idx[order[: budget - n_prot - n_prefix]]
    keep = np.concatenate([np.arange(n_prefix, dtype=np.int64), chosen, np.arange(rest, n, dtype=np.int64)])
    return np.sort(keep)


def quantize_int4(x):
    """Symmetric 4-bit codes for one group per leading index: x [..., d] -> (codes int8, scale).

    scale = fp16(absmax / 7) (1 if the vector is all zero); code = clamp(rne(x / scale), −8, 7).
    The division that decides the code is taken in float32, the precision the
    CUDA kernel decides it in.
    """
    xf = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(xf), axis=-1, keepdims=True)
    scale = (amax / np.float32(7.0)).astype(np.float16)
    scale = np.where(scale == 0, np.float16(1.0), scale)
    q = np.rint(xf / scale.astype(np.float32))
    codes = np.clip(q, -8, 7).astype(np.int8)
    return codes, scale[..., 0].astype(np.float64)


def dequantize_int4(codes, scale):
    return codes.astype(np.float64) * np.asarray(scale, np.float64)[..., None]


# --------------------------------------------------------------------------- layer

class OracleLayer:
    """State and step of one decoder layer's attention block under Algorithm 1."""

    def __init__(self, shape, w_qkv, w1, w2, budget: int, chunk: int, n_stab: int,
                 reserve: int = 0, mirror: bool = False):
        if n_stab > budget or budget < 1 or chunk < 1 or n_stab < 0:
            raise ValueError("need 0 <= n_stab <= budget, budget >= 1, chunk >= 1")
        if shape.n_q_heads % shape.n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        self.s = shape
        self.h, self.hk, self.d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
        self.g = self.h // self.hk
        self.w_qkv = np.asarray(w_qkv, np.float64)
        self.w1 = np.asarray(w1, np.float64)
        self.w2 = np.asarray(w2, np.float64)
        self.budget, self.chunk, self.n_stab = budget, chunk, n_stab
        self.cap = budget + chunk + reserve
        self.mirror = mirror
        self.want_flip_sens = False   # tests switch this on: an error-propagation aid, not part of the method
        self.int4 = shape.kv_dtype == 1
        self.n_prefix = 0             # Section 4.4 variant: slots [0, n_prefix) are never evicted
        self.reset()

    def set_protected_prefix(self, n_prefix: int):
        """Section 4.4 variant: the first n_prefix slots of the cache (the query placed at the start
        of the sequence) are kept by every eviction, besides the last n_stab."""
        if n_prefix < 0 or n_prefix + self.n_stab > self.budget:
            raise ValueError("need 0 <= n_prefix and n_prefix + n_stab <= budget")
        self.n_prefix = int(n_prefix)

    # ---- state
    def reset(self):
        hk, d = self.hk, self.d
        self.K = np.zeros((hk, 0, d))          # pre-RoPE keys (dequantised if int4)
        self.V = np.zeros((hk, 0, d))
        self.S = np.zeros((hk, 0))
        self.T = np.zeros((hk, 0), dtype=np.int64)   # absolute token index of each unit
        if self.int4:
            self.Kc = np.zeros((hk, 0, d), np.int8); self.Ks = np.zeros((hk, 0))
            self.Vc = np.zeros((hk, 0, d), np.int8); self.Vs = np.zeros((hk, 0))
        self.seen = 0
        self.last_scores = None
        self.last_keep = None
        self.last_abs_out = None
        self.last_flip_sens = None

    @property
    def len(self) -> int:
        return self.K.shape[1]

    def export_state(self):
        st = dict(K=self.K.copy(), V=self.V.copy(), S=self.S.copy(), T=self.T.copy(),
                  seen=self.seen)
        if self.int4:
            st.update(Kc=self.Kc.copy(), Ks=self.Ks.copy(), Vc=self.Vc.copy(), Vs=self.Vs.copy())
        return st

    def import_state(self, st):
        self.K, self.V = st["K"].copy(), st["V"].copy()
        self.S, self.T = st["S"].copy(), st["T"].copy()
        self.seen = int(st["seen"])
        if self.int4:
            self.Kc, self.Ks = st["Kc"].copy(), st["Ks"].copy()
            self.Vc, self.Vs = st["Vc"].copy(), st["Vs"].copy()

    def _r(self, x):
        return round_bf16(x) if self.mirror else x

    # ---- one chunk
    def _rh_input(self, X):
        """z of the chunk's tokens, [n_tok, (h + 2 h_kv) d]: what the retaining head reads."""
        n_tok = X.shape[0]
        qkv = self._r(project_qkv(X, self.w_qkv, self.h, self.hk, self.d))
        if self.s.rh_input == 0:
            return qkv
        Q, K, V = split_qkv(qkv, self.h, self.hk, self.d)
        pos_chunk = (self.len + np.arange(n_tok))[:, None]
        Qr = self._r(rope(Q, pos_chunk, self.s.rope_theta))
        Kr = self._r(rope(K, pos_chunk, self.s.rope_theta))
        return np.concatenate([Qr.reshape(n_tok, -1), Kr.reshape(n_tok, -1), V.reshape(n_tok, -1)], axis=1)

    def partial_preact(self, X):
        """This worker's share of the retaining head's first product, z_local · W1_local
        [n_tok, d_R]: summed over the workers it is z · W1 of the whole layer."""
        return self._rh_input(np.asarray(X, np.float64)) @ self.w1

    def prefill_chunk(self, X, flags: int = 0, rows=None, preact=None):
        """One loop iteration of Algorithm 1 for this layer.  Returns attn_out [n_tok, h·d].
        preact: the summed first product of the retaining head when the heads are divided over
        workers (this worker's own product alone is not the layer's)."""
        X = np.asarray(X, np.float64)
        n_tok = X.shape[0]
        h, hk, d, g = self.h, self.hk, self.d, self.g
        ln = self.len
        if n_tok < 1 or n_tok > self.chunk:
            raise ValueError("n_tok must be in [1, chunk]")
        if ln + n_tok > self.cap:
            raise CapacityError("cache capacity exceeded")

        # (a) projections; the staging buffer is a storage point
        qkv = self._r(project_qkv(X, self.w_qkv, h, hk, d))
        Q, K, V = split_qkv(qkv, h, hk, d)

        # positions: cache slot i -> i, chunk token t -> len + t
        pos_chunk = (ln + np.arange(n_tok))[:, None]
        Qr = self._r(rope(Q, pos_chunk, self.s.rope_theta))
        Kr_chunk = self._r(rope(K, pos_chunk, self.s.rope_theta))
        Kr_cache = self._r(rope(self.K, np.arange(ln)[None, :], self.s.rope_theta))
        V_cache = self._r(self.V) if self.int4 else self.V

        # (b) Eq. 1
        self.last_abs_out = np.full((n_tok, h * d), np.nan)
        self.last_flip_sens = np.full((n_tok, h * d), np.nan) if self.want_flip_sens else None
        out = attention_rows(Qr, Kr_cache, V_cache, Kr_chunk, V, g, rows, self.last_abs_out,
                             self.last_flip_sens)

        # (c) retaining head on the token's concatenated [Q ‖ K ‖ V]
        if self.s.rh_input == 0:
            z = qkv
        else:
            z = np.concatenate([Qr.reshape(n_tok, -1), Kr_chunk.reshape(n_tok, -1),
                                V.reshape(n_tok, -1)], axis=1)
        if preact is None:
            s_chunk = retaining_scores(z, self.w1, self.w2, self.s.act)     # [n_tok, h_kv]
        else:
            s_chunk = activation(np.asarray(preact, np.float64), self.s.act) @ self.w2
        self.last_scores = s_chunk

        # (d) concat, protect, top-b, gather
        Kn = np.transpose(K, (1, 0, 2))
        Vn = np.transpose(V, (1, 0, 2))
        if self.int4:
            kc, ks = quantize_int4(Kn)
            vc, vs = quantize_int4(Vn)
            self.Kc = np.concatenate([self.Kc, kc], axis=1); self.Ks = np.concatenate([self.Ks, ks], axis=1)
            self.Vc = np.concatenate([self.Vc, vc], axis=1); self.Vs = np.concatenate([self.Vs, vs], axis=1)
            Kn, Vn = dequantize_int4(kc, ks), dequantize_int4(vc, vs)
        self.K = np.concatenate([self.K, Kn], axis=1)
        self.V = np.concatenate([self.V, Vn], axis=1)
        self.S = np.concatenate([self.S, s_chunk.T], axis=1)
        tid = np.broadcast_to(self.seen + np.arange(n_tok, dtype=np.int64), (hk, n_tok))
        self.T = np.concatenate([self.T, tid], axis=1)
        n = ln + n_tok
        self.seen += n_tok

        self.last_keep = None
        if not (flags & NO_EVICT) and n > self.budget:
            n_prot = 0 if (flags & LAST_CHUNK) else min(self.n_stab, n)
            keep = np.stack([select_keep(self.S[m], self.budget, n_prot, self.n_prefix) for m in range(hk)])
            self.last_keep = keep
            take = lambda a: np.stack([a[m][keep[m]] for m in range(hk)])
            self.K, self.V, self.S, self.T = take(self.K), take(self.V), take(self.S), take(self.T)
            if self.int4:
                self.Kc, self.Ks = take(self.Kc), take(self.Ks)
                self.Vc, self.Vs = take(self.Vc), take(self.Vs)
        return out

    def decode_step(self, x):
        """The B = 1 case of Eq. 1: append without eviction."""
        return self.prefill_chunk(np.asarray(x, np.float64).reshape(1, -1), NO_EVICT)


# --------------------------------------------------------------------------- a budget per head
#
# Appendix H (the combination with head-wise budget allocation): "Locret evicts cache units across the
# attention heads independently", so the budget may differ from head to head.  Every KV head m then has
# its own cache length len_m = min(b_m, tokens seen), its own re-assigned positions (cache slot i of head
# m sits at position i, the chunk's token t at len_m + t, Section 3.4) and its own eviction; the
# retaining head still reads the token's [Q, K, V] of all heads (Section 3.3).  Reading: stabilizers and
# the protected prefix are the same for every head; the query heads of a group use their KV head's
# positions.

class OracleLayerHeadBudgets(OracleLayer):
    """OracleLayer with one budget per KV head.  State per head: Kh[m] [len_m, d], Vh[m], Sh[m] [len_m],
    Th[m] [len_m]."""

    def __init__(self, shape, w_qkv, w1, w2, head_budgets, chunk: int, n_stab: int, reserve: int = 0,
                 mirror: bool = False):
        budgets = [int(b) for b in head_budgets]
        if len(budgets) != shape.n_kv_heads or min(budgets) < 1 or n_stab > min(budgets):
            raise ValueError("need one budget >= max(1, n_stab) per KV head")
        super().__init__(shape, w_qkv, w1, w2, max(budgets), chunk, n_stab, reserve=reserve, mirror=mirror)
        if self.int4:
            raise ValueError("per-head budgets are defined for the bf16 cache only")
        self.budgets = budgets
        self.reset()

    def set_protected_prefix(self, n_prefix: int):
        if n_prefix < 0 or n_prefix + self.n_stab > min(self.budgets):
            raise ValueError("need 0 <= n_prefix and n_prefix + n_stab <= every head's budget")
        self.n_prefix = int(n_prefix)

    def reset(self):
        super().reset()
        hk, d = self.hk, self.d
        self.Kh = [np.zeros((0, d)) for _ in range(hk)]
        self.Vh = [np.zeros((0, d)) for _ in range(hk)]
        self.Sh = [np.zeros(0) for _ in range(hk)]
        self.Th = [np.zeros(0, dtype=np.int64) for _ in range(hk)]

    @property
    def lens(self):
        return [k.shape[0] for k in self.Kh]

    @property
    def len(self) -> int:
        return max(self.lens) if hasattr(self, "Kh") else 0

    def export_state(self):
        return dict(K=[a.copy() for a in self.Kh], V=[a.copy() for a in self.Vh], S=[a.copy() for a in self.Sh],
                    T=[a.copy() for a in self.Th], seen=self.seen)

    def import_state(self, st):
        self.Kh = [np.array(a, np.float64) for a in st["K"]]
        self.Vh = [np.array(a, np.float64) for a in st["V"]]
        self.Sh = [np.array(a, np.float64) for a in st["S"]]
        self.Th = [np.array(a, np.int64) for a in st["T"]]
        self.seen = int(st["seen"])

    def prefill_chunk(self, X, flags: int = 0, rows=None, preact=None):
        X = np.asarray(X, np.float64)
        n_tok = X.shape[0]
        h, hk, d, g = self.h, self.hk, self.d, self.g
        lens = self.lens
        if n_tok < 1 or n_tok > self.chunk:
            raise ValueError("n_tok must be in [1, chunk]")
        for m in range(hk):
            if lens[m] + n_tok > self.budgets[m] + self.chunk + (self.cap - self.budget - self.chunk):
                raise CapacityError("cache capacity exceeded")

        # (a) projections; the staging buffer is a storage point
        qkv = self._r(project_qkv(X, self.w_qkv, h, hk, d))
        Q, K, V = split_qkv(qkv, h, hk, d)

        # (b) Eq. 1, head by head: head m's cache slot i sits at position i, the chunk's token t at len_m + t
        out = np.full((n_tok, h * d), np.nan)
        self.last_abs_out = np.full((n_tok, h * d), np.nan)
        self.last_flip_sens = np.full((n_tok, h * d), np.nan) if self.want_flip_sens else None
        Qr_all = np.zeros_like(Q)
        Kr_all = np.zeros_like(K)
        for m in range(hk):
            pos = (lens[m] + np.arange(n_tok))[:, None]
            js = slice(m * g, (m + 1) * g)
            Qr = self._r(rope(Q[:, js, :], pos, self.s.rope_theta))
            Kr_chunk = self._r(rope(K[:, m:m + 1, :], pos, self.s.rope_theta))
            Kr_cache = self._r(rope(self.Kh[m][None], np.arange(lens[m])[None, :], self.s.rope_theta))
            Qr_all[:, js, :], Kr_all[:, m:m + 1, :] = Qr, Kr_chunk
            cols = slice(m * g * d, (m + 1) * g * d)
            ab = np.full((n_tok, g * d), np.nan)
            fs = np.full((n_tok, g * d), np.nan) if self.want_flip_sens else None
            out[:, cols] = attention_rows(Qr, Kr_cache, self.Vh[m][None], Kr_chunk, V[:, m:m + 1, :], g, rows, ab, fs)
            self.last_abs_out[:, cols] = ab
            if fs is not None:
                self.last_flip_sens[:, cols] = fs

        # (c) retaining head on the token's concatenated [Q ‖ K ‖ V] of all heads
        if self.s.rh_input == 0:
            z = qkv
        else:
            z = np.concatenate([Qr_all.reshape(n_tok, -1), Kr_all.reshape(n_tok, -1), V.reshape(n_tok, -1)], axis=1)
        s_chunk = retaining_scores(z, self.w1, self.w2, self.s.act)     # [n_tok, h_kv]
        self.last_scores = s_chunk

        # (d) per head: concat, protect, top-b_m, gather
        tid = self.seen + np.arange(n_tok, dtype=np.int64)
        self.last_keep = [None] * hk
        for m in range(hk):
            Km = np.concatenate([self.Kh[m], K[:, m, :]], axis=0)
            Vm = np.concatenate([self.Vh[m], V[:, m, :]], axis=0)
            Sm = np.concatenate([self.Sh[m], s_chunk[:, m]])
            Tm = np.concatenate([self.Th[m], tid])
            n = Km.shape[0]
            if not (flags & NO_EVICT) and n > self.budgets[m]:
                n_prot = 0 if (flags & LAST_CHUNK) else min(self.n_stab, n)
                keep = select_keep(Sm, self.budgets[m], n_prot, self.n_prefix)
                self.last_keep[m] = keep
                Km, Vm, Sm, Tm = Km[keep], Vm[keep], Sm[keep], Tm[keep]
            self.Kh[m], self.Vh[m], self.Sh[m], self.Th[m] = Km, Vm, Sm, Tm
        self.seen += n_tok
        return out


# --------------------------------------------------------------------------- heads divided over workers
def shard_by_kv_head(w_qkv, w1, w2, h: int, h_kv: int, d: int, rank: int, world: int):
    """Worker rank's slices when KV heads [rank·h_kv/world, (rank+1)·h_kv/world) and the query
    heads of their groups live on it: the matching columns of W_qkv, the matching rows of W1
    (same order: local Q heads, local K heads, local V heads), the matching columns of W2."""
    if h_kv % world or not 0 <= rank < world:
        raise ValueError("n_kv_heads must divide evenly over the workers")
    g, hk_l = h // h_kv, h_kv // world
    q_heads = np.arange(rank * hk_l * g, (rank + 1) * hk_l * g)
    kv_heads = np.arange(rank * hk_l, (rank + 1) * hk_l)
    cols = np.concatenate([
        (q_heads[:, None] * d + np.arange(d)[None, :]).ravel(),
        ((h + kv_heads)[:, None] * d + np.arange(d)[None, :]).ravel(),
        ((h + h_kv + kv_heads)[:, None] * d + np.arange(d)[None, :]).ravel()])
    return (np.asarray(w_qkv)[:, cols], np.asarray(w1)[cols, :], np.asarray(w2)[:, kv_heads])


def tp_prefill_chunk(shards, X, flags: int = 0, rows=None):
    """One step of Algorithm 1 with the heads divided over len(shards) workers (OracleLayer
    objects built from shard_by_kv_head slices).  The only exchange is the sum of the partial
    products before the activation.  Returns the workers' attn_out side by side, which is the
    undivided layer's attn_out because query heads are dealt out in order."""
    total = sum(sh.partial_preact(X) for sh in shards)
    return np.concatenate([sh.prefill_chunk(X, flags, rows, preact=total) for sh in shards], axis=1)


# --------------------------------------------------------------------------- the rest of the decoder layer
#
# Section 3.1 writes the layer as A = [A_1 .. A_h] W^O followed by H = FFN(A) and leaves the
# normalisation, the residual connections and the form of the FFN to the backbone.  Both
# backbones of the paper (Llama-3.1, Phi-3) are pre-norm decoders with a gated SiLU FFN, which
# is the reading taken here:
#     h1 = RMSNorm(x; g1)            -> the attention block above (its hidden_in is h1)
#     x1 = x + attn_out W_o
#     h2 = RMSNorm(x1; g2)
#     y  = x1 + (silu(h2 W_gate) * (h2 W_up)) W_down

RMS_EPS = 1e-5


def rmsnorm(x, gain, eps: float = RMS_EPS):
    """Row-wise x / sqrt(mean(x^2) + eps) * gain."""
    x = np.asarray(x, np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, np.float64)


def gated_ffn(h, w_gate, w_up, w_down, rnd=None):
    """(silu(h W_gate) * (h W_up)) W_down; `rnd` rounds the gated product where it is stored."""
    h = np.asarray(h, np.float64)
    a = activation(h @ np.asarray(w_gate, np.float64), 0) * (h @ np.asarray(w_up, np.float64))
    if rnd is not None:
        a = rnd(a)
    return a @ np.asarray(w_down, np.float64)


class OracleBlock:
    """One decoder layer: RMSNorm -> attention block with eviction (OracleLayer) -> W_o + residual
    -> RMSNorm -> gated FFN + residual.  In mirror mode values are rounded to bf16 where the CUDA
    path stores them: h1, x1, h2, the gated product, y."""

    def __init__(self, attn: "OracleLayer", w_o, w_gate, w_up, w_down, g1, g2):
        self.attn = attn
        self.w_o = np.asarray(w_o, np.float64)
        self.w_gate, self.w_up = np.asarray(w_gate, np.float64), np.asarray(w_up, np.float64)
        self.w_down = np.asarray(w_down, np.float64)
        self.g1, self.g2 = np.asarray(g1, np.float64), np.asarray(g2, np.float64)
        self.last_h1 = None

    def _r(self, x):
        return round_bf16(x) if self.attn.mirror else x

    def prefill_chunk(self, X, flags: int = 0, rows=None):
        X = np.asarray(X, np.float64)
        h1 = self._r(rmsnorm(X, self.g1))
        self.last_h1 = h1
        att = self.attn.prefill_chunk(h1, flags, rows=rows)        # NaN rows where not computed
        # everything after attention is row-wise: with `rows` only those rows are computed
        sel = np.arange(X.shape[0]) if rows is None else np.asarray(rows, dtype=np.int64)
        a = self._r(att[sel])
        x1 = self._r(X[sel] + a @ self.w_o)
        h2 = self._r(rmsnorm(x1, self.g2))
        y = np.full((X.shape[0], X.shape[1]), np.nan)
        y[sel] = self._r(x1 + gated_ffn(h2, self.w_gate, self.w_up, self.w_down, rnd=self._r))
        return y


# --------------------------------------------------------------------------- training labels
#
# Section 3.3: the ground truth for the retaining head of a layer is, for prompt token k and
# head j, the largest attention score before the softmax that any answer token gives to k:
#     S[k]_j = max_p (Q_j K_j^T)[p, k],   n_q < p <= n_q + n_a,
# and for grouped-query attention the maximum is also taken over the query heads that share
# the KV head.  The passage prints the product without the 1/sqrt(d) factor of Eq. 1; `scale`
# is left to the caller (1 = as printed).

def cis_labels(q_ans, k_prompt, n_kv_heads: int, scale: float = 1.0):
    """q_ans [n_a, h, d] (queries of the answer tokens, as they enter the attention scores),
    k_prompt [n_q, h_kv, d] (keys of the prompt tokens) -> labels [h_kv, n_q]."""
    q = np.asarray(q_ans, np.float64)
    k = np.asarray(k_prompt, np.float64)
    n_a, h, d = q.shape
    n_q = k.shape[0]
    g = h // n_kv_heads
    out = np.full((n_kv_heads, n_q), -np.inf)
    for m in range(n_kv_heads):
        for j in range(m * g, (m + 1) * g):
            s = (q[:, j, :] @ k[:, m, :].T) * scale          # [n_a, n_q]
            out[m] = np.maximum(out[m], s.max(axis=0))
    return out


# --------------------------------------------------------------------------- training objective
#
# Eq. 3: per (token k, KV head m) Smooth-L1 between the predicted and the true score, plus
# alpha times the squared difference of adjacent predictions; Eq. 2 sums it over heads and
# prompt tokens.  Readings where the text is silent: Smooth-L1 with the usual threshold 1
# (0.5 x^2 for |x| < 1, |x| - 0.5 beyond), the L2 term as the plain square (s~[k] - s~[k+1])^2
# for k < n - 1, summed like the rest (no mean); alpha = 2.5e-3 (Section 4.1).  SiLU only.

def smooth_l1(x):
    ax = np.abs(x)
    return np.where(ax < 1.0, 0.5 * x * x, ax - 0.5)


def rh_loss_and_grads(z, labels, w1, w2, alpha: float = 2.5e-3):
    """z [n, d_in] (the tokens' [Q ‖ K ‖ V]), labels [h_kv, n] -> (loss, dL/dW1 [d_in, d_R],
    dL/dW2 [d_R, h_kv]); the backbone is frozen, only the retaining head gets gradients."""
    z = np.asarray(z, np.float64)
    w1 = np.asarray(w1, np.float64)
    w2 = np.asarray(w2, np.float64)
    tgt = np.asarray(labels, np.float64).T                 # [n, h_kv]
    pre = z @ w1
    sig = 1.0 / (1.0 + np.exp(-pre))
    a = pre * sig                                          # SiLU
    s = a @ w2                                             # [n, h_kv]
    diff = s - tgt
    adj = s[:-1] - s[1:]
    loss = float(smooth_l1(diff).sum() + alpha * (adj * adj).sum())
    ds = np.clip(diff, -1.0, 1.0)                          # derivative of Smooth-L1
    ds[:-1] += 2.0 * alpha * adj
    ds[1:] -= 2.0 * alpha * adj
    dw2 = a.T @ ds
    da = ds @ w2.T
    dpre = da * (sig * (1.0 + pre * (1.0 - sig)))          # d SiLU / d pre
    dw1 = z.T @ dpre
    return loss, dw1, dw2


# --------------------------------------------------------------------------- optimiser
#
# Appendix A (training): AdamW, learning rate 5e-4, linear schedule with 2000 warm-up steps, 3000
# steps, batch size 1.  Where the text is silent the usual defaults are taken: betas (0.9,
# 0.999), eps 1e-8, decoupled weight decay 0.01, bias correction on.

def adamw_step(param, grad, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
               eps: float = 1e-8, weight_decay: float = 0.01):
    """One decoupled-weight-decay Adam update (step counts from 1).  Returns (param, m, v)."""
    p = np.asarray(param, np.float64) * (1.0 - lr * weight_decay)
    g = np.asarray(grad, np.float64)
    m = beta1 * np.asarray(m, np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, np.float64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    return p - lr * mhat / (np.sqrt(vhat) + eps), m, v


def linear_schedule(step: int, peak_lr: float = 5e-4, warmup: int = 2000, total: int = 3000):
    """Learning rate of update number `step` (from 1): linear warm-up, then linear decay to 0."""
    k = step - 1
    if k < warmup:
        return peak_lr * k / max(1, warmup)
    return peak_lr * max(0.0, (total - k) / max(1, total - warmup))
