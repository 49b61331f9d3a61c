"""Parity of the CUDA library (through its C ABI) with the CPU oracle."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


def small_shape(h=4, hk=2, d=64, D=64, dR=40, **kw):
    return W.LayerShape(d_model=D, n_q_heads=h, n_kv_heads=hk, head_dim=d, d_retain=dR, **kw)


def weights_for(shape, seed=0):
    return W.layer_weights(shape, 0, seed=W.BASE_SEED + seed)


def hidden(n, D, seed=0, scale=1.0):
    g = np.random.default_rng(1000 + seed)
    return W.to_bf16_grid((g.standard_normal((n, D)) * scale).astype(np.float32))


def test_c1_lockstep_every_chunk():
    from parity_util import lockstep_chunk, make_pair
    w = W.get_workload("c1_small_gqa")
    wts = W.layer_weights(w.shape, 0)
    ora, gpu = make_pair(w.shape, wts, w.budget, w.chunk, w.n_stab)
    pure = O.OracleLayer(w.shape, *wts, w.budget, w.chunk, w.n_stab, mirror=False)
    start, identical = 0, 0
    for i, n_tok in enumerate(w.chunk_sizes()):
        x = W.hidden_states(w, start, n_tok)
        # no outlier tokens here: the plain stated tolerance (max-abs 2e-2) holds as written
        st = lockstep_chunk(ora, gpu, x, 0, what=f"c1 chunk {i}", pure=pure, plain=True)
        assert st["pure_within_2e-2_share"] == 1.0 and st["score_plain_rel_worst"] < 0.05
        identical += bool(st.get("sets_identical", True))
        start += n_tok
    assert ora.len == w.budget and identical >= len(w.chunk_sizes()) - 1
    gpu.destroy()


def test_c1_free_running_matches_oracle_sets():
    from parity_util import BAND, bf16_dev, check_attention, make_pair
    w = W.get_workload("c1_small_gqa")
    ora, gpu = make_pair(w.shape, W.layer_weights(w.shape, 0), w.budget, w.chunk, w.n_stab)
    out = torch.zeros((w.chunk, w.shape.n_q_heads * w.shape.head_dim), dtype=torch.bfloat16, device="cuda")
    start = 0
    all_scores = []
    diverged = False
    for n_tok in w.chunk_sizes():
        x = W.hidden_states(w, start, n_tok)
        gpu.prefill_chunk(bf16_dev(x), out, 0)
        ref = ora.prefill_chunk(x, 0)
        all_scores.append(ora.last_scores)
        post = gpu.export_state()
        if not diverged and np.array_equal(post["T"], ora.T):
            check_attention(out[:n_tok].float().cpu().numpy().astype(np.float64), ref, "free-running")
        else:
            diverged = True
        start += n_tok
    # the retained sets may differ only by units whose oracle score lies within the band of the cut
    s_all = np.concatenate(all_scores, axis=0)
    post = gpu.export_state()
    for m in range(w.shape.n_kv_heads):
        sym = set(post["T"][m]) ^ set(ora.T[m])
        cut = np.min(s_all[ora.T[m][: w.budget - w.n_stab], m])
        for tok in sym:
            assert abs(s_all[tok, m] - cut) < BAND
        assert len(sym) <= 4
    gpu.destroy()


@pytest.mark.parametrize("d", [64, 96, 128])
@pytest.mark.parametrize("heads", [(4, 2), (3, 3), (8, 1)])
def test_ragged_chunks_lockstep(d, heads):
    from parity_util import lockstep_chunk, make_pair
    # D = 96 / d_R = 72 take the general-shape kernels, D = 128 / d_R = 96 the tcgen05 GEMMs
    D, dR = (96, 72) if heads[1] == 3 else (128, 96)
    sh = small_shape(h=heads[0], hk=heads[1], d=d, D=D, dR=dR, rope_theta=500000.0)
    ora, gpu = make_pair(sh, weights_for(sh, d), budget=300, chunk=200, n_stab=17)
    start = 0
    for i, n_tok in enumerate([1, 127, 129, 200, 64, 200, 3]):
        x = hidden(n_tok, sh.d_model, seed=i)
        lockstep_chunk(ora, gpu, x, 0, what=f"d{d} {heads} chunk {i}")
        start += n_tok
    gpu.destroy()


def test_outlier_tokens_lockstep():
    """0.1 %-style outlier rows at 20x norm: logits reach hundreds."""
    from parity_util import lockstep_chunk, make_pair
    sh = small_shape(h=8, hk=2, d=128, D=256, dR=128, rope_theta=500000.0)
    ora, gpu = make_pair(sh, weights_for(sh, 7), budget=400, chunk=256, n_stab=100)
    for i in range(4):
        x = hidden(256, sh.d_model, seed=50 + i)
        x[[5, 77, 200]] = W.to_bf16_grid(x[[5, 77, 200]] * 20.0)
        lockstep_chunk(ora, gpu, x, 0, what=f"outlier chunk {i}")
    gpu.destroy()


def test_flags_and_decode_lockstep():
    from parity_util import lockstep_chunk, make_pair
    sh = small_shape()
    ora, gpu = make_pair(sh, weights_for(sh, 3), budget=150, chunk=128, n_stab=150, reserve=80)
    lockstep_chunk(ora, gpu, hidden(128, sh.d_model, 1), 0, what="fill")
    lockstep_chunk(ora, gpu, hidden(128, sh.d_model, 2), 0, what="all-stabilizer eviction (k = 0)")
    assert list(ora.T[0]) == list(range(256 - 150, 256))
    lockstep_chunk(ora, gpu, hidden(100, sh.d_model, 3), O.LAST_CHUNK, what="last chunk: no protection")
    lockstep_chunk(ora, gpu, hidden(60, sh.d_model, 4), O.NO_EVICT, what="n_loc tail: append only")
    assert gpu.cache_len == 210
    # decode steps through the dedicated entry point
    from parity_util import bf16_dev, check_attention
    out = torch.zeros((1, sh.n_q_heads * sh.head_dim), dtype=torch.bfloat16, device="cuda")
    st = ora.export_state()
    gpu.import_state(st["K"], st["V"], st["S"], st["T"], st["seen"])
    for t in range(5):
        x = hidden(1, sh.d_model, 10 + t)
        gpu.decode_step(bf16_dev(x), out)
        ref = ora.decode_step(x[0])
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"decode {t}")
        # keep the two caches identical for the next step
        st = ora.export_state()
        gpu.import_state(st["K"], st["V"], st["S"], st["T"], st["seen"])
    assert gpu.cache_len == 215
    gpu.destroy()


@pytest.mark.parametrize("d,heads,n_stab,kv_dtype", [(128, (8, 2), 0, 0), (64, (4, 4), 9, 0), (96, (3, 3), 5, 0),
                                                      (128, (8, 2), 7, 1), (64, (4, 1), 0, 1),
                                                      (64, (40, 1), 3, 0)])  # 40 heads on one KV head: three head groups
def test_single_token_steps_that_evict(d, heads, n_stab, kv_dtype):
    """Decode-time eviction (a multi-turn stream with a small budget): once the cache is full every
    one-token step with flags = 0 scores the new unit, drops one and compacts, through the
    one-token kernels."""
    from parity_util import lockstep_chunk, make_pair
    sh = small_shape(h=heads[0], hk=heads[1], d=d, D=128, dR=64, rope_theta=500000.0, kv_dtype=kv_dtype)
    ora, gpu = make_pair(sh, weights_for(sh, 11), budget=96, chunk=64, n_stab=n_stab)
    lockstep_chunk(ora, gpu, hidden(64, sh.d_model, 70), 0, what="fill 1")
    lockstep_chunk(ora, gpu, hidden(64, sh.d_model, 71), 0, what="fill 2 (evicts)")
    for t in range(6):
        lockstep_chunk(ora, gpu, hidden(1, sh.d_model, 80 + t), 0, what=f"evicting token {t}")
        assert gpu.cache_len == 96 and ora.len == 96
    gpu.destroy()


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_protected_prefix_lockstep_and_crafted_scores(kv_dtype):
    """Query-aware variant (Section 4.4): the first l_q slots survive every eviction."""
    from parity_util import import_oracle_state, lockstep_chunk, make_pair
    sh = small_shape(h=4, hk=2, d=128, D=128, dR=64, rope_theta=500000.0, kv_dtype=kv_dtype)
    ora, gpu = make_pair(sh, weights_for(sh, 21), budget=160, chunk=96, n_stab=20)
    ora.set_protected_prefix(24)
    gpu.set_protected_prefix(24)
    for i, n_tok in enumerate([96, 96, 50, 96, 1, 96]):
        lockstep_chunk(ora, gpu, hidden(n_tok, sh.d_model, 90 + i), 0, what=f"prefix chunk {i}")
        if ora.seen > 160:
            assert list(ora.T[0][:24]) == list(range(24))
    lockstep_chunk(ora, gpu, hidden(40, sh.d_model, 99), O.LAST_CHUNK, what="prefix, last chunk")
    post = gpu.export_state()
    assert list(post["T"][1][:24]) == list(range(24))
    # crafted scores: the prefix holds the worst scores of all and still stays; ties next to the cut
    if kv_dtype == 0:
        st = ora.export_state()
        S = st["S"].copy()
        S[:, :24] = -1e30
        S[:, 24:60] = 0.25
        S[0, 30] = np.nan
        st["S"] = S
        ora.import_state(st)
        x = hidden(96, sh.d_model, 123)
        stats = lockstep_chunk(ora, gpu, x, 0, what="prefix, crafted")
        assert list(ora.T[0][:24]) == list(range(24))
        assert stats["sets_identical"]          # ties resolved alike (most recent first), NaN last
    # argument checks: prefix + stabilizers must fit the budget
    from paper_2410_01805_b200 import LocretError
    with pytest.raises(LocretError):
        gpu.set_protected_prefix(141)
    with pytest.raises(LocretError):
        gpu.set_protected_prefix(-1)
    gpu.set_protected_prefix(140)
    gpu.destroy()


def test_no_stabilizers_and_other_activations():
    from parity_util import lockstep_chunk, make_pair
    for act in (1, 2):
        sh = small_shape(act=act, rh_input=1)
        ora, gpu = make_pair(sh, weights_for(sh, act), budget=100, chunk=64, n_stab=0)
        for i in range(4):
            lockstep_chunk(ora, gpu, hidden(64, sh.d_model, 20 + i), 0, what=f"act {act} chunk {i}")
        gpu.destroy()


@pytest.mark.parametrize("d,heads", [(128, (8, 2)), (96, (3, 3)), (64, (4, 1))])
def test_int4_cache_lockstep(d, heads):
    """4-bit cache: quantise on append, attention over the dequantised units, codes move unchanged."""
    from parity_util import lockstep_chunk, make_pair
    sh = small_shape(h=heads[0], hk=heads[1], d=d, D=128, dR=64, rope_theta=500000.0, kv_dtype=1)
    ora, gpu = make_pair(sh, weights_for(sh, 40 + d), budget=300, chunk=160, n_stab=50, reserve=16)
    for i, n_tok in enumerate([160, 160, 77, 160, 1, 130]):
        x = hidden(n_tok, sh.d_model, seed=300 + i)
        if i == 3:
            x[[7, 90]] = W.to_bf16_grid(x[[7, 90]] * 5.0)
        lockstep_chunk(ora, gpu, x, 0, what=f"int4 d{d} chunk {i}")
    lockstep_chunk(ora, gpu, hidden(10, sh.d_model, 399), O.NO_EVICT, what="int4 tail")
    # the generic exchange refuses a 4-bit layer
    import paper_2410_01805_b200 as P
    buf = np.zeros(8, dtype=np.float32)
    assert P.lib.locret_import_state(gpu._h, buf.ctypes.data, buf.ctypes.data, buf.ctypes.data,
                                     buf.ctypes.data, 1, 1) == -1
    gpu.destroy()


def test_selection_with_ties_nan_and_signed_zero():
    """Crafted imported scores put the cut inside a group of equal scores: ties prefer the
    recent unit, NaN ranks with -inf, -0 equals +0."""
    from parity_util import bf16_dev, make_pair
    sh = small_shape(h=2, hk=2)
    budget, chunk, n_stab = 64, 32, 28          # k = 36 of rest = 64 imported + 4 chunk units
    g = np.random.default_rng(5)
    scenarios = [
        (np.repeat([1000.0, 2000.0, 1000.0, -1000.0], budget // 4),
         g.choice([0.0, -0.0, 5000.0, np.inf, 1e-30], size=budget)),
        (g.choice([np.nan, -np.inf, 7.0], size=budget, p=[0.35, 0.35, 0.3]),
         g.choice([3.0, 3.0000002, -0.0], size=budget)),
    ]
    for s0, s1 in scenarios:
        ora, gpu = make_pair(sh, weights_for(sh, 9), budget=budget, chunk=chunk, n_stab=n_stab)
        K = W.to_bf16_grid(g.standard_normal((2, budget, 64)).astype(np.float32))
        V = W.to_bf16_grid(g.standard_normal((2, budget, 64)).astype(np.float32))
        S = np.stack([s0, s1]).astype(np.float32)
        T = np.broadcast_to(np.arange(budget, dtype=np.int64), (2, budget)).copy()
        ora.import_state(dict(K=K.astype(np.float64), V=V.astype(np.float64), S=S.astype(np.float64),
                              T=T, seen=budget))
        gpu.import_state(K, V, S, T, budget)
        x = hidden(chunk, sh.d_model, 77, scale=0.05)          # chunk scores stay tiny
        out = torch.zeros((chunk, 2 * 64), dtype=torch.bfloat16, device="cuda")
        gpu.prefill_chunk(bf16_dev(x), out, 0)
        ora.prefill_chunk(x, 0)
        post = gpu.export_state()
        assert np.array_equal(post["T"], ora.T)
        gpu.destroy()


def test_budget_covering_context_is_full_causal_attention():
    from parity_util import bf16_dev, check_attention, make_pair
    sh = small_shape(h=4, hk=2, d=64, D=64)
    ctx = 300
    wts = weights_for(sh, 11)
    ora, gpu = make_pair(sh, wts, budget=ctx, chunk=77, n_stab=10)
    x = hidden(ctx, sh.d_model, 99)
    outs = []
    for s in range(0, ctx, 77):
        xc = x[s:s + 77]
        o = torch.zeros((xc.shape[0], 4 * 64), dtype=torch.bfloat16, device="cuda")
        gpu.prefill_chunk(bf16_dev(xc), o, 0)
        outs.append(o.float().cpu().numpy())
    got = np.concatenate(outs).astype(np.float64)
    # one-shot causal attention over the whole context, by the oracle in a single chunk
    full = O.OracleLayer(sh, *wts, budget=ctx, chunk=ctx, n_stab=0, mirror=True)
    check_attention(got, full.prefill_chunk(x), "budget >= context")
    assert gpu.cache_len == ctx
    gpu.destroy()


def test_argument_checks_and_capacity():
    import ctypes as C
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    sh = small_shape()
    wq, w1, w2 = (bf16_dev(a) for a in weights_for(sh))
    with pytest.raises(P.LocretError) as e:
        P.LocretLayer(sh, wq, w1, w2, budget=10, chunk=8, n_stab=11)
    assert e.value.code == -1
    with pytest.raises(P.LocretError):
        P.LocretLayer(small_shape(d=80), wq, w1, w2, budget=10, chunk=8, n_stab=1)
    L = P.LocretLayer(sh, wq, w1, w2, budget=10, chunk=8, n_stab=2, reserve=4)
    x = bf16_dev(hidden(8, sh.d_model))
    out = torch.zeros((8, 4 * 64), dtype=torch.bfloat16, device="cuda")
    assert P.lib.locret_prefill_chunk(L._h, x.data_ptr(), 9, 0, out.data_ptr()) == -1
    assert P.lib.locret_prefill_chunk(L._h, x.data_ptr(), 0, 0, out.data_ptr()) == -1
    assert P.lib.locret_prefill_chunk(L._h, None, 8, 0, out.data_ptr()) == -1
    assert P.lib.locret_prefill_chunk(L._h, x.data_ptr(), 8, 8, out.data_ptr()) == -1
    L.prefill_chunk(x, out)                       # len 8
    L.prefill_chunk(x, out, P.NO_EVICT)           # len 16
    assert L.cache_len == 16
    L.prefill_chunk(x[:6], out, P.NO_EVICT)       # len 22 = cap
    assert P.lib.locret_prefill_chunk(L._h, x.data_ptr(), 1, P.NO_EVICT, out.data_ptr()) == -3
    assert P.lib.locret_prefill_chunk(L._h, x.data_ptr(), 8, 0, out.data_ptr()) == -3
    L.destroy()


def test_reset_and_launch_accounting():
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    sh = small_shape()
    wq, w1, w2 = (bf16_dev(a) for a in weights_for(sh))
    L = P.LocretLayer(sh, wq, w1, w2, budget=40, chunk=32, n_stab=2)
    x = bf16_dev(hidden(32, sh.d_model))
    out = torch.zeros((32, 4 * 64), dtype=torch.bfloat16, device="cuda")
    L.set_timing(True)
    L.prefill_chunk(x, out); L.prefill_chunk(x, out)
    first = out.clone()
    ms, cnt = L.read_timing()
    assert cnt[P.K_NAMES.index("attn")] == 2 and cnt[P.K_NAMES.index("topk")] == 1
    assert L.launch_count == int(cnt.sum()) and np.all(ms[cnt > 0] > 0)
    s1 = L.export_state()
    L.reset()
    assert L.cache_len == 0
    L.prefill_chunk(x, out); L.prefill_chunk(x, out)
    s2 = L.export_state()
    assert torch.equal(first, out)
    for k in ("K", "V", "S", "T"):
        assert np.array_equal(s1[k], s2[k])
    L.destroy()


def test_bounded_wait_reports_a_timeout_and_the_context_survives():
    """A device-side wait that cannot complete gives up, leaves LOCRET_ERR_DEVICE_TIMEOUT in the status
    word and the kernel ends normally; the next step on the same context is still correct."""
    import paper_2410_01805_b200 as P
    from parity_util import lockstep_chunk, make_pair
    assert P.lib.locret_selftest_wait_timeout(torch.cuda.current_stream().cuda_stream) == -5
    assert b"timed out" in P.lib.locret_strerror(-5)
    # the production wait itself: one role runs out of polls, sets the abort flag and the status word;
    # a second role that waits with the full production limit must be stopped by that flag
    rep = np.zeros(4, dtype=np.int64)
    assert P.lib.locret_selftest_wait_abort(torch.cuda.current_stream().cuda_stream, rep.ctypes.data) == 0
    assert rep[0] == -5 and rep[1] == 1
    # the first role gave up after 2^12 polls; the second checks the flag every 2^10 polls, so it
    # stops within about a quarter more, nowhere near its own 2^24 polls
    assert 0 < rep[2] and rep[3] < 4 * rep[2] + 10_000_000, rep
    sh = small_shape(d=128, D=128, dR=64)
    ora, gpu = make_pair(sh, weights_for(sh, 21), budget=200, chunk=128, n_stab=8)
    lockstep_chunk(ora, gpu, hidden(128, sh.d_model, 5), 0, what="after the timed-out wait")
    assert gpu.sync_status() == 0
    gpu.destroy()
