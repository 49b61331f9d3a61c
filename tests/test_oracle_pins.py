"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests needs a GPU and none touches the CUDA path.
"""

import itertools
import math
import os
import types

import numpy as np
import pytest
import torch

from oracle import locret_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def shape(**kw):
    base = dict(d_model=16, n_q_heads=4, n_kv_heads=2, head_dim=8, d_retain=12,
                rope_theta=10000.0, act=0, rh_input=0, kv_dtype=0)
    base.update(kw)
    return types.SimpleNamespace(**base)


def rand_layer(sh, budget, chunk, n_stab, seed=0, **kw):
    g = np.random.default_rng(seed)
    d_in = (sh.n_q_heads + 2 * sh.n_kv_heads) * sh.head_dim
    wqkv = g.standard_normal((sh.d_model, d_in)) / math.sqrt(sh.d_model)
    w1 = g.standard_normal((d_in, sh.d_retain)) / math.sqrt(d_in)
    w2 = g.standard_normal((sh.d_retain, sh.n_kv_heads)) / math.sqrt(sh.d_retain)
    return O.OracleLayer(sh, wqkv, w1, w2, budget, chunk, n_stab, **kw), (wqkv, w1, w2)


def run_chunks(layer, X, B, flags=0):
    outs = []
    for s in range(0, X.shape[0], B):
        outs.append(layer.prefill_chunk(X[s:s + B], flags))
    return np.concatenate(outs, axis=0)


# ------------------------------------------------------------------ rounding

def test_round_bf16_matches_library_conversion():
    g = np.random.default_rng(1)
    x = np.concatenate([g.standard_normal(20000) * 10.0 ** g.integers(-6, 6, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, 1e-30]])
    # inputs restricted to float32 so the library conversion is a single rounding
    x32 = x.astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x32.astype(np.float64)), want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert O.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6


def test_round_fp16_matches_library_conversion():
    g = np.random.default_rng(2)
    x = (g.standard_normal(20000) * 10.0 ** g.integers(-7, 4, 20000)).astype(np.float32)
    want = x.astype(np.float16).astype(np.float64)
    assert np.array_equal(O.round_fp16(x.astype(np.float64)), want)


# ------------------------------------------------------------------ RoPE

def test_rope_is_complex_rotation_of_half_split_pairs():
    g = np.random.default_rng(3)
    d, theta = 16, 500000.0
    x = g.standard_normal((5, 3, d))
    pos = np.array([0, 1, 7, 100, 5000])[:, None]
    got = O.rope(x, pos, theta)
    # independent statement: z_i = x_i + i x_{i+d/2}; z_i <- z_i * exp(i pos theta^(-2i/d))
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    w = np.exp(1j * pos[..., None] * theta ** (-2.0 * np.arange(d // 2) / d))
    zr = z * w
    want = np.concatenate([zr.real, zr.imag], axis=-1)
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    assert np.array_equal(got[0], x[0])                     # position 0 is the identity
    assert np.allclose(np.linalg.norm(got, axis=-1), np.linalg.norm(x, axis=-1))


def test_rope_inner_product_depends_on_relative_position_only():
    g = np.random.default_rng(4)
    q, k = g.standard_normal(32), g.standard_normal(32)
    a = O.rope(q, 17, 1e4) @ O.rope(k, 5, 1e4)
    b = O.rope(q, 1017, 1e4) @ O.rope(k, 1005, 1e4)
    assert abs(a - b) < 1e-9


# ------------------------------------------------------------------ Pin 1: budget >= context

def brute_force_causal_attention(X, wqkv, sh):
    """One-shot causal GQA attention with RoPE at true positions, in explicit loops."""
    h, hk, d = sh.n_q_heads, sh.n_kv_heads, sh.head_dim
    g = h // hk
    n = X.shape[0]
    out = np.zeros((n, h * d))
    half = d // 2
    freq = [sh.rope_theta ** (-2.0 * i / d) for i in range(half)]

    def rot(v, p):
        r = np.zeros(d)
        for i in range(half):
            c, s = math.cos(p * freq[i]), math.sin(p * freq[i])
            r[i] = v[i] * c - v[i + half] * s
            r[i + half] = v[i + half] * c + v[i] * s
        return r

    proj = X @ wqkv
    for j in range(h):
        m = j // g
        q = [rot(proj[t, j * d:(j + 1) * d], t) for t in range(n)]
        k = [rot(proj[t, (h + m) * d:(h + m + 1) * d], t) for t in range(n)]
        v = [proj[t, (h + hk + m) * d:(h + hk + m + 1) * d] for t in range(n)]
        for t in range(n):
            lg = np.array([q[t] @ k[u] / math.sqrt(d) for u in range(t + 1)])
            p = np.exp(lg - lg.max())
            p /= p.sum()
            out[t, j * d:(j + 1) * d] = sum(p[u] * v[u] for u in range(t + 1))
    return out


@pytest.mark.parametrize("B", [1, 5, 16, 37])
@pytest.mark.parametrize("heads", [(4, 2), (4, 4), (6, 1)])
def test_chunked_equals_full_attention_when_budget_covers_context(B, heads):
    sh = shape(n_q_heads=heads[0], n_kv_heads=heads[1])
    ctx = 37
    layer, (wqkv, _, _) = rand_layer(sh, budget=ctx, chunk=max(B, 1), n_stab=3, seed=5)
    X = np.random.default_rng(6).standard_normal((ctx, sh.d_model))
    got = run_chunks(layer, X, B)
    want = brute_force_causal_attention(X, wqkv, sh)
    assert np.allclose(got, want, rtol=0, atol=1e-11)
    assert layer.len == ctx and np.array_equal(layer.T[0], np.arange(ctx))


def test_full_attention_matches_library_sdpa():
    sh = shape(n_q_heads=4, n_kv_heads=2, head_dim=16, d_model=24)
    ctx = 50
    layer, (wqkv, _, _) = rand_layer(sh, budget=64, chunk=7, n_stab=0, seed=7)
    X = np.random.default_rng(8).standard_normal((ctx, sh.d_model))
    got = run_chunks(layer, X, 7)
    h, hk, d = 4, 2, 16
    proj = torch.from_numpy(X @ wqkv)
    pos = np.arange(ctx)[:, None]
    Q = torch.from_numpy(O.rope(proj[:, : h * d].reshape(ctx, h, d).numpy(), pos, sh.rope_theta))
    K = torch.from_numpy(O.rope(proj[:, h * d:(h + hk) * d].reshape(ctx, hk, d).numpy(), pos, sh.rope_theta))
    V = proj[:, (h + hk) * d:].reshape(ctx, hk, d)
    K = K.repeat_interleave(h // hk, dim=1)
    V = V.repeat_interleave(h // hk, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        Q.permute(1, 0, 2)[None], K.permute(1, 0, 2)[None], V.permute(1, 0, 2)[None], is_causal=True)
    ref = ref[0].permute(1, 0, 2).reshape(ctx, h * d).numpy()
    assert np.allclose(got, ref, rtol=0, atol=1e-11)


def test_decode_step_is_chunk_of_one():
    sh = shape()
    ctx = 20
    layer, (wqkv, _, _) = rand_layer(sh, budget=8, chunk=6, n_stab=2, reserve=40, seed=9)
    X = np.random.default_rng(10).standard_normal((ctx, sh.d_model))
    outs = [layer.decode_step(X[t]) for t in range(ctx)]
    want = brute_force_causal_attention(X, wqkv, sh)
    assert np.allclose(np.concatenate(outs), want, atol=1e-11)
    assert layer.len == ctx          # decode never evicts


# ------------------------------------------------------------------ attention with an evicted cache

def test_attention_over_evicted_cache_uses_reassigned_positions():
    """After eviction the kept units sit at positions 0..len-1 and the chunk follows."""
    sh = shape(n_q_heads=2, n_kv_heads=1)
    layer, (wqkv, w1, w2) = rand_layer(sh, budget=6, chunk=5, n_stab=2, seed=11)
    X = np.random.default_rng(12).standard_normal((15, sh.d_model))
    layer.prefill_chunk(X[:5]); layer.prefill_chunk(X[5:10])
    kept = layer.T[0].copy()
    assert len(kept) == 6
    out = layer.prefill_chunk(X[10:15])
    # explicit: gather kept tokens + the chunk, positions 0..10, causal inside the chunk
    h, d = 2, 8
    proj = X @ wqkv
    toks = list(kept) + list(range(10, 15))
    pos = np.arange(len(toks))
    Kr = O.rope(proj[toks, h * d:(h + 1) * d], pos, sh.rope_theta)
    Vv = proj[toks, (h + 1) * d:]
    for j in range(h):
        for t in range(5):
            q = O.rope(proj[10 + t, j * d:(j + 1) * d], 6 + t, sh.rope_theta)
            lg = Kr[: 6 + t + 1] @ q / math.sqrt(d)
            p = np.exp(lg - lg.max()); p /= p.sum()
            assert np.allclose(out[t, j * d:(j + 1) * d], p @ Vv[: 6 + t + 1], atol=1e-12)


# ------------------------------------------------------------------ retaining head (Pin 4)

@pytest.mark.parametrize("act", [0, 1, 2])
def test_retaining_head_matches_library_mlp(act):
    g = np.random.default_rng(13)
    z, w1, w2 = g.standard_normal((9, 20)), g.standard_normal((20, 7)), g.standard_normal((7, 3))
    tz, t1, t2 = map(torch.from_numpy, (z, w1, w2))
    F = torch.nn.functional
    fn = {0: F.silu, 1: lambda v: F.gelu(v, approximate="tanh"), 2: F.relu}[act]
    want = (fn(tz @ t1) @ t2).numpy()
    assert np.allclose(O.retaining_scores(z, w1, w2, act), want, atol=1e-12)


def test_retaining_head_hand_case():
    # W1 picks input columns 0 and 2; W2 maps hidden 0 -> head 0 (x2) and hidden 1 -> head 1 (x-1)
    z = np.array([[1.0, 5.0, -2.0]])
    w1 = np.array([[1.0, 0.0], [0.0, 0.0], [0.0, 1.0]])
    w2 = np.array([[2.0, 0.0], [0.0, -1.0]])
    silu = lambda v: v / (1 + math.exp(-v))
    got = O.retaining_scores(z, w1, w2, 0)
    assert np.allclose(got, [[2 * silu(1.0), -silu(-2.0)]], atol=1e-15)


def test_retaining_head_sees_all_heads_in_q_k_v_order():
    sh = shape()
    layer, (wqkv, w1, w2) = rand_layer(sh, budget=50, chunk=10, n_stab=0, seed=14)
    X = np.random.default_rng(15).standard_normal((10, sh.d_model))
    layer.prefill_chunk(X)
    z = X @ wqkv                       # all Q heads, then K heads, then V heads
    t = torch.from_numpy
    want = (torch.nn.functional.silu(t(z) @ t(w1)) @ t(w2)).numpy()
    assert np.allclose(layer.last_scores, want, atol=1e-12)
    assert np.allclose(layer.S, want.T, atol=1e-12)
    # a per-head-sized W1 (the other reading of the printed dimension) does not even fit
    with pytest.raises(ValueError):
        O.retaining_scores(z, w1[: 3 * sh.head_dim], w2)


# ------------------------------------------------------------------ selection

def literal_algorithm1_selection(scores, b, n_s, last_chunk):
    """Algorithm 1 as printed: overwrite the last n_s scores with +inf, then top-b."""
    s = np.array(scores, dtype=np.float64)
    n = len(s)
    if not last_chunk and n_s > 0:
        s[max(0, n - n_s):] = np.inf
    order = sorted(range(n), key=lambda i: (-s[i], -i))
    return sorted(order[:b])


def test_select_keep_equals_literal_algorithm1_bruteforce():
    g = np.random.default_rng(16)
    for n, b, n_s in itertools.product([1, 2, 5, 9, 14], [1, 3, 5, 8], [0, 1, 3, 5]):
        if n_s > b:
            continue
        for trial in range(4):
            s = g.standard_normal(n)
            if trial == 1:
                s = np.round(s)                       # many ties
            want = literal_algorithm1_selection(s, b, n_s, False)
            got = O.select_keep(s, b, n_s)
            assert list(got) == want, (n, b, n_s, s)
            assert list(O.select_keep(s, b, 0)) == literal_algorithm1_selection(s, b, n_s, True)


def test_select_keep_ties_prefer_recent_and_nan_ranks_last():
    assert list(O.select_keep([1.0, 1.0, 1.0, 1.0], 2, 0)) == [2, 3]
    assert list(O.select_keep([np.nan, 0.0, -5.0, np.nan], 2, 0)) == [1, 2]
    assert list(O.select_keep([np.nan, np.nan, -np.inf], 2, 0)) == [1, 2]


def literal_selection_with_prefix(scores, b, n_s, n_q):
    """The same overwrite-and-sort statement with both protected ends at +inf."""
    s = np.array(scores, dtype=np.float64)
    n = len(s)
    s = np.where(np.isnan(s), -np.inf, s)
    if n_s > 0:
        s[max(0, n - n_s):] = np.inf
    s[:min(n_q, n)] = np.inf
    order = sorted(range(n), key=lambda i: (-s[i], -i))
    return sorted(order[:b])


def test_protected_prefix_equals_overwrite_and_sort_bruteforce():
    """Section 4.4 (query at the start of the sequence, visible across every eviction)."""
    g = np.random.default_rng(160)
    for n, b, n_s, n_q in itertools.product([6, 9, 14, 23], [3, 5, 8], [0, 1, 3], [0, 1, 2, 4]):
        if n_s + n_q > b or n <= b:
            continue
        for trial in range(4):
            s = g.standard_normal(n)
            if trial == 1:
                s = np.round(s)                       # many ties
            if trial == 2:
                s[g.integers(0, n, 2)] = np.nan
            got = list(O.select_keep(s, b, n_s, n_q))
            assert got == literal_selection_with_prefix(s, b, n_s, n_q), (n, b, n_s, n_q, s)
            assert len(got) == b and got[:n_q] == list(range(n_q))
            assert got[b - n_s:] == list(range(n - n_s, n))
    # no prefix: the statement of Algorithm 1 itself
    s = g.standard_normal(12)
    assert list(O.select_keep(s, 5, 2, 0)) == list(O.select_keep(s, 5, 2))


@pytest.mark.parametrize("n_stab,n_q", [(0, 4), (6, 3), (9, 11)])
def test_protected_prefix_closed_form_and_chunk_size_invariance(n_stab, n_q):
    """With a protected prefix the final cache is Prefix ∪ Last_{n_s} ∪ Top_{b − n_s − l_q}(between),
    whatever the chunk size: the induction of the cache-problem argument (Appendix N) with both
    ends fixed."""
    sh = shape()
    b, ctx = 30, 131
    X = np.random.default_rng(190).standard_normal((ctx, sh.d_model))
    finals = []
    for B in [1, 7, 30, 50]:
        layer, (wqkv, w1, w2) = rand_layer(sh, budget=b, chunk=B, n_stab=n_stab, seed=200)
        layer.set_protected_prefix(n_q)
        run_chunks(layer, X, B)
        t = torch.from_numpy
        s_all = (torch.nn.functional.silu(t(X @ wqkv) @ t(w1)) @ t(w2)).numpy()   # [ctx, hk]
        for m in range(sh.n_kv_heads):
            mid = list(range(n_q, ctx - n_stab))
            order = sorted(mid, key=lambda i: (-s_all[i, m], -i))
            want = sorted(list(range(n_q)) + order[: b - n_stab - n_q] + list(range(ctx - n_stab, ctx)))
            assert list(layer.T[m]) == want
        finals.append(layer.T.copy())
    for f in finals[1:]:
        assert np.array_equal(f, finals[0])
    with pytest.raises(ValueError):
        layer.set_protected_prefix(b - n_stab + 1)


# ------------------------------------------------------------------ Pin 2 / Pin 3

@pytest.mark.parametrize("n_stab", [0, 3, 11, 40])
@pytest.mark.parametrize("B", [4, 16, 25])
def test_size_and_stabilizer_invariants_and_cache_problem_condition(n_stab, B):
    sh = shape()
    b = 40
    layer, _ = rand_layer(sh, budget=b, chunk=B, n_stab=n_stab, seed=17)
    X = np.random.default_rng(18).standard_normal((203, sh.d_model))
    prev = [set() for _ in range(sh.n_kv_heads)]
    for s in range(0, 203, B):
        n_tok = min(B, 203 - s)
        layer.prefill_chunk(X[s:s + B])
        seen = s + n_tok
        for m in range(sh.n_kv_heads):
            T = layer.T[m]
            assert len(T) == min(b, seen)                                  # size
            assert np.all(np.diff(T) > 0)                                  # temporal order
            ns = min(n_stab, seen)
            assert set(range(seen - ns, seen)) <= set(T)                   # stabilizers kept
            assert set(T) - prev[m] <= set(range(s, seen))                 # cache-problem cond. 2
            prev[m] = set(T)


@pytest.mark.parametrize("n_stab", [0, 7, 30])
def test_final_retained_set_has_closed_form(n_stab):
    """Scores depend on the token alone, so after any chunking the cache is
    Last_{n_s} ∪ Top_{b − n_s}(all earlier tokens)."""
    sh = shape()
    b, ctx = 30, 157
    X = np.random.default_rng(19).standard_normal((ctx, sh.d_model))
    finals = []
    for B in [1, 5, 30, 64]:
        layer, (wqkv, w1, w2) = rand_layer(sh, budget=b, chunk=B, n_stab=n_stab, seed=20)
        run_chunks(layer, X, B)
        t = torch.from_numpy
        s_all = (torch.nn.functional.silu(t(X @ wqkv) @ t(w1)) @ t(w2)).numpy()   # [ctx, hk]
        for m in range(sh.n_kv_heads):
            rest = ctx - n_stab
            order = sorted(range(rest), key=lambda i: (-s_all[i, m], -i))
            want = sorted(order[: b - n_stab] + list(range(rest, ctx)))
            assert list(layer.T[m]) == want
            assert np.allclose(layer.S[m], s_all[want, m], atol=1e-12)
        finals.append(layer.T.copy())
    for f in finals[1:]:
        assert np.array_equal(f, finals[0])           # chunk-size invariance


def test_last_chunk_flag_drops_protection_and_no_evict_appends():
    sh = shape(n_kv_heads=1, n_q_heads=2)
    layer, _ = rand_layer(sh, budget=5, chunk=8, n_stab=5, reserve=8, seed=21)
    X = np.random.default_rng(22).standard_normal((24, sh.d_model))
    layer.prefill_chunk(X[:8])
    assert list(layer.T[0]) == [3, 4, 5, 6, 7]                 # all five slots are stabilizers
    layer.prefill_chunk(X[8:16], O.LAST_CHUNK)
    s = layer.S[0]
    assert len(s) == 5
    layer.prefill_chunk(X[16:24], O.NO_EVICT)
    assert layer.len == 13 and list(layer.T[0][5:]) == list(range(16, 24))
    with pytest.raises(O.CapacityError):
        layer.prefill_chunk(X[:8], O.NO_EVICT)
        layer.prefill_chunk(X[:8], O.NO_EVICT)


# ------------------------------------------------------------------ Pin 5: arithmetic the paper prints

def read_golden():
    rows = {}
    with open(os.path.join(GOLDEN, "paper_arithmetic.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val, tol, _ = [p.strip() for p in line.split("|")]
            rows[name] = (float(val), float(tol))
    return rows


def test_paper_printed_arithmetic_fixes_shapes():
    gold = read_golden()

    def near(name, x):
        v, tol = gold[name]
        assert abs(x - v) <= tol * v + 1e-12, (name, x, v)

    # retaining-head size under the all-heads reading of W1: (h + 2 h_kv) d x d_R, d_R x h_kv
    def rh_params(h, hk, d, dR, layers):
        z = np.zeros((1, (h + 2 * hk) * d))
        w1, w2 = np.zeros(((h + 2 * hk) * d, dR)), np.zeros((dR, hk))
        assert O.retaining_scores(z, w1, w2).shape == (1, hk)
        return layers * (w1.size + w2.size)

    near("llama_retaining_param_share", rh_params(32, 8, 128, 1024, 32) / 8.03e9)
    near("phi3_retaining_param_share", rh_params(32, 32, 96, 1024, 32) / 3.82e9)
    # a cache unit is one token of one KV head of one layer, K and V, 16-bit
    unit_bytes = 2 * 96 * 2
    near("phi3_full_kv_128k_gb", 131072 * 32 * 32 * unit_bytes / 2 ** 30)
    near("phi3_2bit_kv_128k_gb", 131072 * 32 * 32 * unit_bytes / 8 / 2 ** 30)
    # the budget counts units per head: compression = context / budget
    near("compression_10m", 10 * 2 ** 20 / 6000)
    near("compression_phi3", 131072 / 6000)
    near("compression_llama", 131072 / 16384)


# ------------------------------------------------------------------ Pin 6: int4 cache

def test_int4_roundtrip_properties():
    g = np.random.default_rng(23)
    x = O.round_bf16(g.standard_normal((4, 50, 128)) * 3)
    codes, scale = O.quantize_int4(x)
    assert codes.min() >= -8 and codes.max() <= 7
    assert np.array_equal(scale, O.round_fp16(scale))                 # scales are fp16 values
    deq = O.dequantize_int4(codes, scale)
    assert np.all(np.abs(deq - x) <= scale[..., None] * 0.5 * (1 + 1e-6) + 1e-12)
    # exact multiples of the scale survive
    sc = 0.25
    y = np.arange(-7, 8).astype(np.float64) * sc
    y = np.concatenate([y, np.zeros(128 - 15)])[None]
    c2, s2 = O.quantize_int4(y)
    assert s2[0] == sc and np.array_equal(O.dequantize_int4(c2, s2), y)
    # all-zero vector: scale 1, codes 0
    c3, s3 = O.quantize_int4(np.zeros((1, 128)))
    assert s3[0] == 1.0 and not c3.any()


def test_int4_layer_quantises_on_append_and_moves_codes_unchanged():
    sh = shape(kv_dtype=1, head_dim=8)
    layer, (wqkv, _, _) = rand_layer(sh, budget=10, chunk=6, n_stab=2, seed=24, mirror=True)
    X = O.round_bf16(np.random.default_rng(25).standard_normal((18, sh.d_model)))
    layer.prefill_chunk(X[:6]); layer.prefill_chunk(X[6:12])
    before = layer.export_state()
    layer.prefill_chunk(X[12:18])
    # every cached unit is codes * scale, and kept units carry identical codes
    assert np.array_equal(layer.K, O.dequantize_int4(layer.Kc, layer.Ks))
    for m in range(sh.n_kv_heads):
        for slot, tok in enumerate(layer.T[m]):
            if tok < 12:
                old = list(before["T"][m]).index(tok)
                assert np.array_equal(layer.Kc[m, slot], before["Kc"][m, old])
                assert layer.Vs[m, slot] == before["Vs"][m, old]


def test_last_chunk_through_the_chunk_step_keeps_plain_top_b_by_hand():
    """Algorithm 1's last iteration: no score is overwritten with +inf, so the retained set is the
    plain top-b of cache ‖ chunk.  Scores are forced through hand-made weights: the retaining
    head reads V's first column (W1 picks it, ReLU, W2 = 1), so score(token) = max(0, V[t, 0])."""
    sh = shape(n_q_heads=1, n_kv_heads=1, head_dim=2, d_model=6, d_retain=1, act=2)
    wqkv = np.eye(6)                         # [Q ‖ K ‖ V] = the hidden state itself
    w1 = np.zeros((6, 1)); w1[4, 0] = 1.0    # first element of V
    w2 = np.ones((1, 1))
    b, n_s = 6, 4
    layer = O.OracleLayer(sh, wqkv, w1, w2, budget=b, chunk=8, n_stab=n_s)
    score = np.array([5., 1., 9., 2., 8., 3., 7., 4.,            # chunk 0: tokens 0..7
                      0.5, 6., 0.25, 10., 0.1, 0.2, 0.3, 0.4])   # chunk 1: tokens 8..15
    X = np.random.default_rng(40).standard_normal((16, 6))
    X[:, 4] = score
    layer.prefill_chunk(X[:8])               # protected: tokens 4..7; best two of 0..3: tokens 0 (5) and 2 (9)
    assert list(layer.T[0]) == [0, 2, 4, 5, 6, 7]
    assert np.allclose(layer.S[0], score[[0, 2, 4, 5, 6, 7]])
    layer.prefill_chunk(X[8:], O.LAST_CHUNK)
    # candidates: tokens {0,2,4,5,6,7} ∪ {8..15}; the six best scores are 10, 9, 8, 7, 6, 5
    assert list(layer.T[0]) == [0, 2, 4, 6, 9, 11]
    # the same step with protection would have kept the last four tokens whatever their scores
    prot = O.OracleLayer(sh, wqkv, w1, w2, budget=b, chunk=8, n_stab=n_s)
    prot.prefill_chunk(X[:8]); prot.prefill_chunk(X[8:])
    assert list(prot.T[0]) == [2, 11, 12, 13, 14, 15]


def test_abs_out_is_the_probability_weighted_magnitude_by_explicit_loops():
    g = np.random.default_rng(41)
    n, h, hk, d, ln = 5, 4, 2, 6, 7
    Qr, Kc, Vc = g.standard_normal((n, h, d)), g.standard_normal((hk, ln, d)), g.standard_normal((hk, ln, d)) * 3
    Kn, Vn = g.standard_normal((n, hk, d)), g.standard_normal((n, hk, d)) * 3
    abs_out = np.full((n, h * d), np.nan)
    out = O.attention_rows(Qr, Kc, Vc, Kn, Vn, h // hk, abs_out=abs_out)
    for t in range(n):
        for j in range(h):
            m = j // (h // hk)
            keys = [Kc[m, i] for i in range(ln)] + [Kn[u, m] for u in range(t + 1)]
            vals = [Vc[m, i] for i in range(ln)] + [Vn[u, m] for u in range(t + 1)]
            lg = np.array([Qr[t, j] @ k / math.sqrt(d) for k in keys])
            p = np.exp(lg - lg.max()); p /= p.sum()
            for c in range(d):
                assert abs(abs_out[t, j * d + c] - sum(p[i] * abs(vals[i][c]) for i in range(len(keys)))) < 1e-12
                assert abs(out[t, j * d + c] - sum(p[i] * vals[i][c] for i in range(len(keys)))) < 1e-12
    assert np.all(abs_out >= np.abs(out) - 1e-12)           # triangle inequality


def test_flip_sens_is_the_first_order_effect_of_one_flipped_key_element_by_brute_force():
    """flip_sens = sum_i p_i delta_i |V_i - out|, delta_i = 2^-7 max_c |q_c k_ic| / sqrt(d): the change of
    the output when key i's most influential element moves by 2^-7 of itself, summed over the keys
    in absolute value.  Brute force: move that one element of one key, recompute the softmax exactly,
    and add up the absolute output changes over the keys."""
    g = np.random.default_rng(42)
    n, h, hk, d, ln = 3, 2, 1, 8, 9
    Qr, Kc, Vc = g.standard_normal((n, h, d)), g.standard_normal((hk, ln, d)), g.standard_normal((hk, ln, d))
    Kn, Vn = g.standard_normal((n, hk, d)), g.standard_normal((n, hk, d))
    fs = np.full((n, h * d), np.nan)
    out = O.attention_rows(Qr, Kc, Vc, Kn, Vn, h, flip_sens=fs)

    def softmax_out(q, keys, vals):
        lg = keys @ q / math.sqrt(d)
        p = np.exp(lg - lg.max()); p /= p.sum()
        return p @ vals

    for t in range(n):
        for j in range(h):
            keys = np.concatenate([Kc[0], Kn[: t + 1, 0]])
            vals = np.concatenate([Vc[0], Vn[: t + 1, 0]])
            base = softmax_out(Qr[t, j], keys, vals)
            assert np.allclose(base, out[t, j * d:(j + 1) * d], atol=1e-13)
            total = np.zeros(d)
            for i in range(len(keys)):
                c = int(np.argmax(np.abs(Qr[t, j] * keys[i])))
                moved = keys.copy()
                moved[i, c] *= 1.0 + 2.0 ** -7
                total += np.abs(softmax_out(Qr[t, j], moved, vals) - base)
            got = fs[t, j * d:(j + 1) * d]
            # first order in 2^-7: the two agree to a few per cent; a factor of two (let alone ten)
            # in delta, a dropped p_i or |V_i| in place of |V_i - out| would not
            assert np.allclose(got, total, rtol=0.05, atol=1e-9), (got, total)


def _mirror_reference(X, wqkv, sh, Kc, Vc, skip=None):
    """The chunk step's attention with bf16 rounding at the storage points, written with the
    library's conversions (torch.bfloat16) and its attention routine.  `skip` leaves one point
    unrounded.  Points: 'staging' (projected Q, K, V), 'q_rot', 'k_rot_chunk', 'k_rot_cache'."""
    def r(x, name):
        if name == skip:
            return x
        return torch.from_numpy(np.asarray(x)).to(torch.bfloat16).to(torch.float64).numpy()
    h, hk, d = sh.n_q_heads, sh.n_kv_heads, sh.head_dim
    n, ln = X.shape[0], Kc.shape[1]
    qkv = r(X @ wqkv, "staging")
    Q = qkv[:, : h * d].reshape(n, h, d)
    K = qkv[:, h * d:(h + hk) * d].reshape(n, hk, d)
    V = qkv[:, (h + hk) * d:].reshape(n, hk, d)
    pos = (ln + np.arange(n))[:, None]
    Qr = r(O.rope(Q, pos, sh.rope_theta), "q_rot")
    Kr = r(O.rope(K, pos, sh.rope_theta), "k_rot_chunk")
    Kcr = r(O.rope(Kc, np.arange(ln)[None, :], sh.rope_theta), "k_rot_cache")
    out = np.zeros((n, h * d))
    g = h // hk
    for j in range(h):
        m = j // g
        keys = torch.from_numpy(np.concatenate([Kcr[m], Kr[:, m]]))
        vals = torch.from_numpy(np.concatenate([Vc[m], V[:, m]]))
        mask = torch.ones((n, ln + n), dtype=torch.bool)
        mask[:, ln:] = torch.tril(torch.ones((n, n), dtype=torch.bool))
        o = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Qr[:, j])[None], keys[None], vals[None],
                                                             attn_mask=mask[None])
        out[:, j * d:(j + 1) * d] = o[0].numpy()
    return out, K, V


@pytest.mark.parametrize("point", ["staging", "q_rot", "k_rot_chunk", "k_rot_cache"])
def test_each_mirror_rounding_point_is_where_the_stored_value_is_rounded(point):
    """Mirror mode rounds to bf16 exactly at the four storage points of the step.  With every point
    rounded, a restatement on the library's conversions reproduces the oracle to rounding error of
    fp64; with any one point left out it does not (so a point dropped from the oracle, or added
    elsewhere, is seen)."""
    sh = shape(n_q_heads=4, n_kv_heads=2, head_dim=8, d_model=16)
    layer, (wqkv, w1, w2) = rand_layer(sh, budget=32, chunk=12, n_stab=0, seed=43, mirror=True)
    g = np.random.default_rng(44)
    X0 = O.round_bf16(g.standard_normal((12, sh.d_model)))
    X1 = O.round_bf16(g.standard_normal((12, sh.d_model)))
    layer.prefill_chunk(X0)
    Kc, Vc = layer.K.copy(), layer.V.copy()
    got = layer.prefill_chunk(X1)
    want, K, V = _mirror_reference(X1, wqkv, sh, Kc, Vc)
    assert np.max(np.abs(got - want)) < 1e-12
    # what enters the cache is the staged (rounded) projection, pre-RoPE
    assert np.array_equal(layer.K[:, 12:], np.transpose(K, (1, 0, 2)))
    assert np.array_equal(layer.V[:, 12:], np.transpose(V, (1, 0, 2)))
    without, K2, _ = _mirror_reference(X1, wqkv, sh, Kc, Vc, skip=point)
    assert np.max(np.abs(got - without)) > 1e-6, f"rounding at {point} does not reach the output"
    if point == "staging":
        assert not np.array_equal(layer.K[:, 12:], np.transpose(K2, (1, 0, 2)))


# ------------------------------------------------------------------ a budget per head (Appendix H)

def rand_head_layer(sh, budgets, chunk, n_stab, seed=0, **kw):
    g = np.random.default_rng(seed)
    d_in = (sh.n_q_heads + 2 * sh.n_kv_heads) * sh.head_dim
    wqkv = g.standard_normal((sh.d_model, d_in)) / math.sqrt(sh.d_model)
    w1 = g.standard_normal((d_in, sh.d_retain)) / math.sqrt(d_in)
    w2 = g.standard_normal((sh.d_retain, sh.n_kv_heads)) / math.sqrt(sh.d_retain)
    return O.OracleLayerHeadBudgets(sh, wqkv, w1, w2, budgets, chunk, n_stab, **kw), (wqkv, w1, w2)


@pytest.mark.parametrize("mirror", [False, True])
def test_equal_head_budgets_reproduce_the_single_budget_layer(mirror):
    sh = shape(n_q_heads=6, n_kv_heads=3)
    lh, (wqkv, w1, w2) = rand_head_layer(sh, [9, 9, 9], 5, 2, seed=50, mirror=mirror)
    lu = O.OracleLayer(sh, wqkv, w1, w2, 9, 5, 2, mirror=mirror)
    X = np.random.default_rng(51).standard_normal((23, sh.d_model))
    for s0 in range(0, 23, 5):
        a, b = lh.prefill_chunk(X[s0:s0 + 5]), lu.prefill_chunk(X[s0:s0 + 5])
        assert np.array_equal(a, b)
        for m in range(3):
            assert np.array_equal(lh.Th[m], lu.T[m]) and np.array_equal(lh.Kh[m], lu.K[m])
            assert np.array_equal(lh.Sh[m], lu.S[m]) and np.array_equal(lh.Vh[m], lu.V[m])


@pytest.mark.parametrize("B", [3, 8, 16])
def test_head_budgets_closed_form_per_head_and_sizes(B):
    """Scores depend on the token alone, so head m ends with Last_{n_s} ∪ Top_{b_m - n_s} of the earlier
    tokens whatever the chunking and whatever the other heads keep; its size is min(b_m, seen) throughout."""
    sh = shape(n_q_heads=4, n_kv_heads=4, head_dim=4, d_model=12)
    budgets, n_stab, ctx = [5, 11, 40, 7], 3, 37
    layer, (wqkv, w1, w2) = rand_head_layer(sh, budgets, 16, n_stab, seed=52)
    X = np.random.default_rng(53).standard_normal((ctx, sh.d_model))
    seen = 0
    for s0 in range(0, ctx, B):
        layer.prefill_chunk(X[s0:s0 + B])
        seen = min(ctx, s0 + B)
        assert layer.lens == [min(b, seen) for b in budgets]
        for m in range(4):
            assert np.all(np.diff(layer.Th[m]) > 0)
    s_all = O.retaining_scores(X @ wqkv, w1, w2)
    for m, b in enumerate(budgets):
        if b >= ctx:
            assert list(layer.Th[m]) == list(range(ctx))
            continue
        rest = ctx - n_stab
        order = sorted(range(rest), key=lambda i: (-s_all[i, m], -i))
        assert list(layer.Th[m]) == sorted(order[: b - n_stab] + list(range(rest, ctx)))
        assert np.allclose(layer.Sh[m], s_all[layer.Th[m], m], atol=1e-12)


def test_a_head_whose_budget_covers_the_context_attends_to_everything_while_others_evict():
    sh = shape(n_q_heads=4, n_kv_heads=2, head_dim=8, d_model=16)
    ctx = 29
    layer, (wqkv, _, _) = rand_head_layer(sh, [ctx, 6], 7, 2, seed=54)
    X = np.random.default_rng(55).standard_normal((ctx, sh.d_model))
    got = run_chunks(layer, X, 7)
    want = brute_force_causal_attention(X, wqkv, sh)
    # query heads 0, 1 belong to KV head 0 (nothing evicted): full causal attention at true positions
    assert np.allclose(got[:, :16], want[:, :16], rtol=0, atol=1e-11)
    # query heads 2, 3 see a cache of 6 units: different from full attention, and equal to the hand gather
    assert not np.allclose(got[8:, 16:], want[8:, 16:], atol=1e-3)
    assert layer.lens == [ctx, 6]


def test_head_budget_attention_over_an_evicted_head_uses_that_heads_positions():
    """After eviction head m's kept units sit at positions 0..len_m-1 and the chunk follows at len_m + t:
    checked by an explicit gather for a head with a small budget beside one with a large budget."""
    sh = shape(n_q_heads=2, n_kv_heads=2, head_dim=8, d_model=16)
    layer, (wqkv, w1, w2) = rand_head_layer(sh, [4, 12], 5, 1, seed=56)
    X = np.random.default_rng(57).standard_normal((15, sh.d_model))
    layer.prefill_chunk(X[:5]); layer.prefill_chunk(X[5:10])
    kept = [t.copy() for t in layer.Th]
    assert [len(k) for k in kept] == [4, 10]
    out = layer.prefill_chunk(X[10:15])
    proj = X @ wqkv
    h, hk, d = 2, 2, 8
    for m in range(2):
        toks = list(kept[m]) + list(range(10, 15))
        ln = len(kept[m])
        Kr = O.rope(proj[toks, (h + m) * d:(h + m + 1) * d], np.arange(len(toks)), sh.rope_theta)
        Vv = proj[toks, (h + hk + m) * d:(h + hk + m + 1) * d]
        for t in range(5):
            q = O.rope(proj[10 + t, m * d:(m + 1) * d], ln + t, sh.rope_theta)
            lg = Kr[: ln + t + 1] @ q / math.sqrt(d)
            p = np.exp(lg - lg.max()); p /= p.sum()
            assert np.allclose(out[t, m * d:(m + 1) * d], p @ Vv[: ln + t + 1], atol=1e-12)


def test_mirror_mode_rounds_only_storage_points():
    sh = shape()
    lp, (wqkv, w1, w2) = rand_layer(sh, budget=64, chunk=16, n_stab=0, seed=26)
    lm = O.OracleLayer(sh, wqkv, w1, w2, 64, 16, 0, mirror=True)
    X = O.round_bf16(np.random.default_rng(27).standard_normal((16, sh.d_model)))
    a, b = lp.prefill_chunk(X), lm.prefill_chunk(X)
    assert np.array_equal(lm.K, O.round_bf16(lm.K))            # cached K is on the bf16 grid
    assert np.max(np.abs(a - b)) < 0.05 and not np.array_equal(a, b)


# ------------------------------------------------------------------ the rest of the decoder layer

def test_rmsnorm_matches_library_and_its_invariants():
    g = np.random.default_rng(300)
    x = g.standard_normal((9, 24)) * 3.0
    gain = 1.0 + 0.1 * g.standard_normal(24)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (24,), torch.from_numpy(gain), eps=O.RMS_EPS).numpy()
    assert np.allclose(O.rmsnorm(x, gain), want, rtol=0, atol=1e-13)
    # unit gain: every row has mean square 1 (up to eps); scaling a row by c > 0 changes nothing
    y = O.rmsnorm(x, np.ones(24), eps=0.0)
    assert np.allclose(np.mean(y * y, axis=1), 1.0, atol=1e-12)
    assert np.allclose(O.rmsnorm(7.5 * x, gain, eps=0.0), O.rmsnorm(x, gain, eps=0.0), atol=1e-12)
    # a hand case: x = (3, 4) has mean square 12.5
    assert np.allclose(O.rmsnorm(np.array([[3.0, 4.0]]), np.array([1.0, 2.0]), eps=0.0),
                       [[3.0 / math.sqrt(12.5), 8.0 / math.sqrt(12.5)]])


def test_gated_ffn_matches_library_ops():
    g = np.random.default_rng(301)
    h = g.standard_normal((7, 10))
    wg, wu, wd = g.standard_normal((10, 14)), g.standard_normal((10, 14)), g.standard_normal((14, 10))
    t = torch.from_numpy
    want = ((torch.nn.functional.silu(t(h) @ t(wg)) * (t(h) @ t(wu))) @ t(wd)).numpy()
    assert np.allclose(O.gated_ffn(h, wg, wu, wd), want, rtol=0, atol=1e-12)
    # gate and up are not interchangeable, and a zero gate input gives zero (silu(0) = 0)
    assert not np.allclose(O.gated_ffn(h, wu, wg, wd), want)
    assert np.allclose(O.gated_ffn(h, np.zeros_like(wg), wu, wd), 0.0)


def test_decoder_block_equals_library_composition_when_nothing_is_evicted():
    """Budget >= context: the block is an ordinary pre-norm decoder layer, written here with the
    library's rms_norm / scaled_dot_product_attention / silu, in any chunking."""
    sh = shape(n_q_heads=4, n_kv_heads=2, head_dim=16, d_model=24)
    ctx, F = 41, 40
    h, hk, d, D = 4, 2, 16, 24
    g = np.random.default_rng(302)
    w_o = g.standard_normal((h * d, D)) / math.sqrt(h * d)
    wg, wu = g.standard_normal((D, F)) / math.sqrt(D), g.standard_normal((D, F)) / math.sqrt(D)
    wd = g.standard_normal((F, D)) / math.sqrt(F)
    g1, g2 = 1.0 + 0.1 * g.standard_normal(D), 1.0 + 0.1 * g.standard_normal(D)
    X = g.standard_normal((ctx, D)) * 2.0
    t = torch.from_numpy
    F_ = torch.nn.functional
    outs = []
    for B in (1, 6, 41):
        layer, (wqkv, _, _) = rand_layer(sh, budget=64, chunk=B, n_stab=0, seed=303)
        blk = O.OracleBlock(layer, w_o, wg, wu, wd, g1, g2)
        outs.append(np.concatenate([blk.prefill_chunk(X[s:s + B]) for s in range(0, ctx, B)], axis=0))
    h1 = F_.rms_norm(t(X), (D,), t(g1), eps=O.RMS_EPS)
    proj = h1 @ t(wqkv)
    pos = np.arange(ctx)[:, None]
    Q = t(O.rope(proj[:, : h * d].reshape(ctx, h, d).numpy(), pos, sh.rope_theta))
    K = t(O.rope(proj[:, h * d:(h + hk) * d].reshape(ctx, hk, d).numpy(), pos, sh.rope_theta))
    V = proj[:, (h + hk) * d:].reshape(ctx, hk, d)
    K, V = K.repeat_interleave(h // hk, dim=1), V.repeat_interleave(h // hk, dim=1)
    att = F_.scaled_dot_product_attention(Q.transpose(0, 1), K.transpose(0, 1), V.transpose(0, 1), is_causal=True)
    att = att.transpose(0, 1).reshape(ctx, h * d)
    x1 = t(X) + att @ t(w_o)
    h2 = F_.rms_norm(x1, (D,), t(g2), eps=O.RMS_EPS)
    want = (x1 + (F_.silu(h2 @ t(wg)) * (h2 @ t(wu))) @ t(wd)).numpy()
    for got in outs:
        assert np.allclose(got, want, rtol=0, atol=1e-10)


# ------------------------------------------------------------------ training labels (Section 3.3)

def test_cis_labels_equal_the_definition_by_brute_force():
    g = np.random.default_rng(400)
    for n_a, n_q, h, hk, d in [(1, 5, 2, 2, 4), (3, 7, 4, 2, 6), (5, 4, 6, 1, 3), (4, 9, 3, 3, 8)]:
        q = g.standard_normal((n_a, h, d))
        k = g.standard_normal((n_q, hk, d))
        grp = h // hk
        want = np.full((hk, n_q), -np.inf)
        for kk in range(n_q):
            for j in range(h):
                for p in range(n_a):
                    want[j // grp, kk] = max(want[j // grp, kk], float(np.dot(q[p, j], k[kk, j // grp])))
        assert np.allclose(O.cis_labels(q, k, hk), want, rtol=0, atol=1e-12)
        assert np.allclose(O.cis_labels(q, k, hk, scale=0.25), 0.25 * want, atol=1e-12)


def test_cis_labels_special_cases_and_invariants():
    g = np.random.default_rng(401)
    q = g.standard_normal((6, 4, 8))
    k = g.standard_normal((11, 2, 8))
    full = O.cis_labels(q, k, 2)
    # one answer token, no grouping: a row of the library's Q K^T
    assert np.allclose(O.cis_labels(q[:1, :1], k[:, :1], 1)[0],
                       (torch.from_numpy(q[0, 0]) @ torch.from_numpy(k[:, 0]).T).numpy())
    # more answer tokens can only raise a label; order of answer tokens and of heads in a group is irrelevant
    assert (O.cis_labels(q[:3], k, 2) <= full + 1e-15).all()
    perm = g.permutation(6)
    assert np.allclose(O.cis_labels(q[perm], k, 2), full)
    assert np.allclose(O.cis_labels(q[:, [1, 0, 3, 2]], k, 2), full)
    # an MHA model (h_kv = h) has no maximum over heads
    assert not np.allclose(O.cis_labels(q, np.repeat(k, 2, axis=1), 4)[0], full[0])


# ------------------------------------------------------------------ training objective (Eq. 2, Eq. 3)

def test_rh_loss_and_gradients_match_library_autograd_and_finite_differences():
    g = np.random.default_rng(500)
    n, d_in, d_R, hk = 23, 12, 9, 3
    z = g.standard_normal((n, d_in))
    w1 = g.standard_normal((d_in, d_R)) / math.sqrt(d_in)
    w2 = g.standard_normal((d_R, hk)) / math.sqrt(d_R)
    labels = g.standard_normal((hk, n)) * 2.0              # |error| on both sides of the Smooth-L1 knee
    alpha = 0.3
    loss, dw1, dw2 = O.rh_loss_and_grads(z, labels, w1, w2, alpha)
    t = torch.from_numpy
    W1 = t(w1).clone().requires_grad_(True)
    W2 = t(w2).clone().requires_grad_(True)
    s = torch.nn.functional.silu(t(z) @ W1) @ W2
    ref = torch.nn.functional.smooth_l1_loss(s, t(labels).T, reduction="sum", beta=1.0) \
        + alpha * ((s[:-1] - s[1:]) ** 2).sum()
    ref.backward()
    assert abs(loss - ref.item()) < 1e-10
    assert np.allclose(dw1, W1.grad.numpy(), atol=1e-10) and np.allclose(dw2, W2.grad.numpy(), atol=1e-10)
    # central differences on a few entries
    eps = 1e-6
    for (i, j) in [(0, 0), (5, 3), (11, 8)]:
        wp, wm = w1.copy(), w1.copy()
        wp[i, j] += eps; wm[i, j] -= eps
        fd = (O.rh_loss_and_grads(z, labels, wp, w2, alpha)[0] - O.rh_loss_and_grads(z, labels, wm, w2, alpha)[0]) / (2 * eps)
        assert abs(fd - dw1[i, j]) < 1e-5
    # alpha = 0 and predictions equal to the labels: zero loss, zero gradient
    s0 = O.retaining_scores(z, w1, w2)
    l0, g1, g2 = O.rh_loss_and_grads(z, s0.T, w1, w2, 0.0)
    assert l0 < 1e-25 and np.abs(g1).max() < 1e-12 and np.abs(g2).max() < 1e-12


# ------------------------------------------------------------------ optimiser (Appendix A, training)

def test_adamw_step_matches_the_library_optimiser():
    g = np.random.default_rng(600)
    p0 = g.standard_normal((5, 7))
    p = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.AdamW([p], lr=5e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    mine, m, v = p0.copy(), np.zeros_like(p0), np.zeros_like(p0)
    for step in range(1, 6):
        grad = g.standard_normal((5, 7)) * (10.0 if step == 3 else 1.0)
        p.grad = torch.from_numpy(grad.copy())
        opt.step()
        mine, m, v = O.adamw_step(mine, grad, m, v, step, 5e-4)
        assert np.allclose(mine, p.detach().numpy(), rtol=0, atol=1e-12)


def test_linear_schedule_matches_the_library_scheduler():
    p = torch.nn.Parameter(torch.zeros(1))
    opt = torch.optim.SGD([p], lr=5e-4)
    sched = torch.optim.lr_scheduler.LambdaLR(
        opt, lambda k: k / 2000 if k < 2000 else max(0.0, (3000 - k) / 1000))
    for step in range(1, 3001):
        if step in (1, 2, 1000, 2000, 2001, 2500, 3000):
            assert abs(O.linear_schedule(step) - sched.get_last_lr()[0]) < 1e-15, step
        opt.step(); sched.step()
    assert O.linear_schedule(1) == 0.0 and abs(O.linear_schedule(2001) - 5e-4) < 1e-18


# ------------------------------------------------------------------ heads divided over workers
# Heads attend and evict independently and only the retaining head mixes them, so dividing the
# KV heads over workers and summing the partial first products must reproduce the undivided layer.
@pytest.mark.parametrize("world,rh_input,kv_dtype", [(2, 0, 0), (4, 0, 0), (2, 1, 0), (2, 0, 1)])
def test_heads_divided_over_workers_reproduce_the_undivided_layer(world, rh_input, kv_dtype):
    sh = shape(n_q_heads=8, n_kv_heads=4, head_dim=8, d_retain=12, rh_input=rh_input, kv_dtype=kv_dtype)
    whole, (wqkv, w1, w2) = rand_layer(sh, budget=24, chunk=8, n_stab=3, seed=70 + world)
    sh_l = shape(n_q_heads=8 // world, n_kv_heads=4 // world, head_dim=8, d_retain=12, rh_input=rh_input,
                 kv_dtype=kv_dtype)
    shards = [O.OracleLayer(sh_l, *O.shard_by_kv_head(wqkv, w1, w2, 8, 4, 8, r, world), 24, 8, 3)
              for r in range(world)]
    hk_l = 4 // world
    X = np.random.default_rng(71).standard_normal((50, sh.d_model))
    for s in range(0, 50, 8):
        want = whole.prefill_chunk(X[s:s + 8])
        got = O.tp_prefill_chunk(shards, X[s:s + 8])
        assert np.allclose(got, want, atol=1e-12)
        assert np.allclose(np.concatenate([sh_.last_scores for sh_ in shards], axis=1), whole.last_scores,
                           atol=1e-12)
        for r, sh_ in enumerate(shards):
            assert np.array_equal(sh_.T, whole.T[r * hk_l:(r + 1) * hk_l])
            assert np.allclose(sh_.K, whole.K[r * hk_l:(r + 1) * hk_l], atol=1e-12)
    assert whole.len == 24 and whole.last_keep is not None
    # the slices are what they claim: a worker's own product alone is not the layer's first product
    part = shards[0].partial_preact(X[:8])
    full = (X[:8] @ wqkv) @ w1 if rh_input == 0 else None
    if full is not None:
        assert not np.allclose(part, full, atol=1e-3)
        shards2 = [O.OracleLayer(sh_l, *O.shard_by_kv_head(wqkv, w1, w2, 8, 4, 8, r, world), 24, 8, 3)
                   for r in range(world)]
        assert np.allclose(sum(s2.partial_preact(X[:8]) for s2 in shards2), full, atol=1e-12)


def test_shard_slices_name_the_right_heads():
    h, hk, d = 8, 4, 2
    d_in = (h + 2 * hk) * d
    wqkv = np.arange(3 * d_in, dtype=np.float64).reshape(3, d_in)
    w1 = np.arange(d_in * 5, dtype=np.float64).reshape(d_in, 5)
    w2 = np.arange(5 * hk, dtype=np.float64).reshape(5, hk)
    a, b, c = O.shard_by_kv_head(wqkv, w1, w2, h, hk, d, rank=1, world=2)
    # worker 1 of 2: query heads 4..7 (columns 8..15), key heads 2, 3 (columns 16+4..16+7), value heads 2, 3
    cols = list(range(8, 16)) + list(range(20, 24)) + list(range(28, 32))
    assert np.array_equal(a[0], np.array(cols, dtype=np.float64))
    assert np.array_equal(b[:, 0], np.array(cols, dtype=np.float64) * 5)
    assert np.array_equal(c[0], np.array([2.0, 3.0]))
    with pytest.raises(ValueError):
        O.shard_by_kv_head(wqkv, w1, w2, h, hk, d, rank=0, world=3)
