"""The CUDA path running on its own state from step to step.

Lock-step tests import the oracle's state before every chunk, which rebuilds the rotated keys; here
nothing is imported between steps, so attention reads the rotated keys that the compaction kernel
wrote (Section 3.4: positions are re-assigned from the beginning after every eviction), and several
layers' steps are in flight on the two streams at once, as in the benchmark.
"""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


def _shape(h, hk, d, D=128, dR=64, **kw):
    return W.LayerShape(d_model=D, n_q_heads=h, n_kv_heads=hk, head_dim=d, d_retain=dR, rope_theta=500000.0, **kw)


def _hidden(n, D, seed):
    g = np.random.default_rng(9000 + seed)
    return W.to_bf16_grid(g.standard_normal((n, D)).astype(np.float32))


@pytest.mark.parametrize("h,hk,d", [(8, 2, 128), (3, 3, 96), (4, 1, 64)])
def test_attention_reads_the_rotated_keys_compaction_wrote(h, hk, d):
    """Small shapes: GQA at head_dim 128, MHA at head_dim 96, MQA at 64; several key tiles and a ragged tail."""
    from parity_util import forced_state, make_pair, run_pair_without_reimport
    sh = _shape(h, hk, d)
    budget, chunk, n_stab = 700, 256, 100
    ora, gpu = make_pair(sh, W.layer_weights(sh, 0, seed=W.BASE_SEED + d), budget, chunk, n_stab)
    st = forced_state(sh, budget, chunk, seed=d)
    stats = run_pair_without_reimport(ora, gpu, st, _hidden(chunk, sh.d_model, 1), _hidden(200, sh.d_model, 2),
                                      what=f"h{h}/{hk} d{d}")
    assert stats["moved"] > hk * 300 and stats["stayed"] >= hk * 64
    gpu.destroy()


def test_attention_reads_compacted_keys_at_the_headline_shape():
    """The Llama-shaped layer at the benchmark's chunk, budget and stabilizer count: chunk A evicts 3072
    units per head and compacts, chunk B attends to what compaction left.  B is compared on one query
    row of every third 128-row block, on the whole of one block, and on its outlier tokens."""
    from parity_util import forced_state, make_pair, run_pair_without_reimport
    w = W.get_workload("c3_llama_128k")
    ora, gpu = make_pair(w.shape, W.layer_weights(w.shape, 0), w.budget, w.chunk, w.n_stab)
    st = forced_state(w.shape, w.budget, w.chunk, seed=3)
    x_a = W.hidden_states(w, 0, w.chunk)
    x_b = W.hidden_states(w, w.chunk, w.chunk)
    g = np.random.default_rng(11)
    rows_b = {rb * 128 + int(g.integers(0, 128)) for rb in range(0, 24, 3)} | set(range(11 * 128, 12 * 128)) | {0, w.chunk - 1}
    norms = np.linalg.norm(x_b, axis=1)
    rows_b |= set(np.flatnonzero(norms > 5 * np.median(norms)).tolist()[:4])
    stats = run_pair_without_reimport(ora, gpu, st, x_a, x_b, rows_a=[0, 1500, w.chunk - 1], rows_b=sorted(rows_b),
                                      what="c3 pair")
    print("c3 pair without re-import:", stats)
    assert stats["moved"] > 8 * 2500
    gpu.destroy()


def test_attention_reads_compacted_keys_at_the_phi3_shape():
    """MHA, head_dim 96, chunk 1024, budget 16384: the other benchmark shape's steady state."""
    from parity_util import forced_state, make_pair, run_pair_without_reimport
    w = W.get_workload("c4_phi3_128k")
    ora, gpu = make_pair(w.shape, W.layer_weights(w.shape, 1), w.budget, w.chunk, w.n_stab)
    st = forced_state(w.shape, w.budget, w.chunk, seed=4)
    x_a = W.hidden_states(w, 0, w.chunk)
    x_b = W.hidden_states(w, w.chunk, w.chunk)
    rows_b = sorted({rb * 128 + 17 * rb % 128 for rb in range(8)} | {0, w.chunk - 1} | set(range(3 * 128, 3 * 128 + 32)))
    stats = run_pair_without_reimport(ora, gpu, st, x_a, x_b, rows_a=[0, w.chunk - 1], rows_b=rows_b, what="c4 pair")
    print("c4 pair without re-import:", stats)
    gpu.destroy()


def _stack_run(kv_dtype, serial, sizes, n_dec, xs, weights, sh, budget, chunk, n_stab):
    """Three layers on one stream sharing one scratch pool; every step enqueued back to back with no
    host synchronisation in between.  Returns every chunk's attention output per layer and the final
    exported state per layer."""
    from paper_2410_01805_b200 import LocretLayer
    from parity_util import bf16_dev
    stream = torch.cuda.current_stream()
    layers = [LocretLayer(sh, *(bf16_dev(a) for a in wts), budget, chunk, n_stab, reserve=n_dec, stream=stream)
              for wts in weights]
    for L in layers:
        L.set_timing(2 if serial else 0)
    hd = sh.n_q_heads * sh.head_dim
    xd = [bf16_dev(x) for x in xs]
    outs = [[torch.zeros((x.shape[0], hd), dtype=torch.bfloat16, device="cuda") for _ in layers] for x in xs]
    for i, x in enumerate(xd):                        # no host sync anywhere in this loop
        for l, L in enumerate(layers):
            if x.shape[0] == 1 and i >= len(sizes):
                L.decode_step(x, outs[i][l])
            else:
                L.prefill_chunk(x, outs[i][l], 0)
    states = [L.export_state() for L in layers]
    assert all(L.sync_status() == 0 for L in layers)
    res = [[o.clone() for o in row] for row in outs]
    for L in layers:
        L.destroy()
    return res, states


@pytest.mark.parametrize("kv_dtype", [0, 1])
def test_steps_back_to_back_on_two_streams_equal_the_one_stream_schedule(kv_dtype):
    """The schedule the benchmark times: the retaining head, selection and compaction of a layer run
    on the library's second stream while the next layer's projection and attention run on the first,
    against shared double-buffered staging.  The kernels are deterministic, so every attention output
    and the final state must be bit-identical to the same steps issued on one stream."""
    from parity_util import BAND
    sh = _shape(8, 2, 128, D=256, dR=128, kv_dtype=kv_dtype)
    budget, chunk, n_stab, n_dec = 300, 128, 40, 4
    sizes = [128, 128, 128, 100, 128, 128, 77, 128]
    xs = [_hidden(n, sh.d_model, 20 + i) for i, n in enumerate(sizes)] + [_hidden(1, sh.d_model, 60 + t) for t in range(n_dec)]
    weights = [W.layer_weights(sh, l, seed=W.BASE_SEED + 77) for l in range(3)]
    two, st_two = _stack_run(kv_dtype, False, sizes, n_dec, xs, weights, sh, budget, chunk, n_stab)
    one, st_one = _stack_run(kv_dtype, True, sizes, n_dec, xs, weights, sh, budget, chunk, n_stab)
    for i in range(len(xs)):
        for l in range(3):
            assert torch.equal(two[i][l], one[i][l]), f"step {i} layer {l}: attention output differs between schedules"
    keys = ("Kc", "Vc", "Ks", "Vs", "S", "T") if kv_dtype == 1 else ("K", "V", "S", "T")
    for l in range(3):
        assert st_two[l]["seen"] == st_one[l]["seen"] == sum(sizes) + n_dec
        for k in keys:
            assert np.array_equal(st_two[l][k], st_one[l][k]), f"layer {l}: final {k} differs between schedules"
    # the final retained ids against the oracle: scores depend on the token alone, so after the last
    # evicting step the cache is Last_{n_s} ∪ Top_{b - n_s} of the earlier tokens, whatever the chunking
    # (closed form of Algorithm 1); the CUDA path may differ only inside the tolerance band of the cut
    n_pre = sum(sizes)
    X = np.concatenate(xs[:len(sizes)]).astype(np.float64)
    for l in range(3):
        wq, w1, w2 = (np.asarray(a, np.float64) for a in weights[l])
        s_all = O.retaining_scores(O.round_bf16(X @ wq), w1, w2, sh.act)           # [tokens, h_kv]
        T = st_two[l]["T"]
        assert T.shape[1] == budget + n_dec
        for m in range(sh.n_kv_heads):
            got = set(T[m].tolist())
            assert set(range(n_pre - n_stab, n_pre + n_dec)) <= got
            rest = np.arange(n_pre - n_stab)
            order = np.lexsort((-rest, -s_all[rest, m]))
            want = set(rest[order[: budget - n_stab]].tolist()) | set(range(n_pre - n_stab, n_pre + n_dec))
            cut = s_all[rest[order[budget - n_stab - 1]], m]
            for tok in got ^ want:
                assert abs(s_all[tok, m] - cut) < BAND, f"layer {l} head {m}: token {tok} outside the band"
            assert len(got ^ want) <= 6


def _hand_scored_layer(h, hk, d, D, seed):
    """Weights under which the retaining head's score of token t for KV head m is exactly
    relu(x[t, m]): W_qkv routes hidden element m unchanged into the first element of value head m,
    W1 picks that element, the activation is ReLU and W2 passes it on.  With small integers in
    x[:, :h_kv] the scores are exact on both sides and full of ties."""
    sh = W.LayerShape(d_model=D, n_q_heads=h, n_kv_heads=hk, head_dim=d, d_retain=8, rope_theta=500000.0, act=2)
    g = np.random.default_rng(seed)
    d_in = sh.d_in
    wqkv = W.to_bf16_grid((g.standard_normal((D, d_in)) / np.sqrt(D)).astype(np.float32))
    w1 = np.zeros((d_in, 8), dtype=np.float32)
    w2 = np.zeros((8, hk), dtype=np.float32)
    for m in range(hk):
        col = (h + hk + m) * d
        wqkv[:, col] = 0.0
        wqkv[m, col] = 1.0
        w1[col, m] = 1.0
        w2[m, m] = 1.0
    return sh, (wqkv, w1, w2)


@pytest.mark.parametrize("d,heads,n_prefix,last", [(64, (4, 2), 0, False), (128, (8, 2), 5, True), (96, (3, 3), 0, True)])
def test_many_evictions_in_place_stay_identical_to_the_oracle(d, heads, n_prefix, last):
    """Eviction leaves kept units in their slots and refills freed ones, so after a few steps slot order
    and temporal order have nothing in common.  Hand-made scores (exact small integers, many ties) keep
    both sides on the same retained set without any import: after every step the exported state must be
    the oracle's (token ids and scores exactly, K and V up to the rare one-ulp flips of a projection),
    and attention - which reads keys rotated at the units' positions in temporal order - must agree."""
    from parity_util import FLIP_FRACTION, bf16_dev, check_attention, make_pair
    h, hk = heads
    sh, wts = _hand_scored_layer(h, hk, d, 64, seed=d)
    budget, chunk, n_stab = 150, 96, 20
    ora, gpu = make_pair(sh, wts, budget, chunk, n_stab, reserve=8)
    if n_prefix:
        ora.set_protected_prefix(n_prefix)
        gpu.set_protected_prefix(n_prefix)
    g = np.random.default_rng(500 + d)
    sizes = [96, 96, 41, 96, 1, 96, 77, 96, 96, 13]
    for i, n_tok in enumerate(sizes):
        x = W.to_bf16_grid(g.standard_normal((n_tok, 64)).astype(np.float32))
        x[:, :hk] = g.integers(-3, 40, size=(n_tok, hk)).astype(np.float32)
        flags = O.LAST_CHUNK if (last and i == len(sizes) - 1) else 0
        out = torch.zeros((n_tok, h * d), dtype=torch.bfloat16, device="cuda")
        gpu.prefill_chunk(bf16_dev(x), out, flags)
        ref = ora.prefill_chunk(x, flags)
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"step {i}", ora.last_abs_out,
                        ora.last_flip_sens)
        st = gpu.export_state()
        assert np.array_equal(st["T"], ora.T), f"step {i}: retained token ids differ"
        assert np.array_equal(st["S"].astype(np.float64), ora.S), f"step {i}: scores differ"
        for name in ("K", "V"):
            diff = np.abs(st[name] - getattr(ora, name))
            assert np.all(diff <= np.abs(getattr(ora, name)) * 2.0 ** -7 + 1e-6), f"step {i}: {name} differs"
            assert np.mean(diff != 0) < FLIP_FRACTION
        assert gpu.sync_status() == 0
    moved, rotated = gpu.compaction_counters
    assert 0 < moved <= rotated
    # a few one-token steps on top (appended in order behind the shuffled slots)
    for t in range(4):
        x = W.to_bf16_grid(g.standard_normal((1, 64)).astype(np.float32))
        out = torch.zeros((1, h * d), dtype=torch.bfloat16, device="cuda")
        gpu.decode_step(bf16_dev(x), out)
        ref = ora.decode_step(x[0])
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"decode {t}", ora.last_abs_out,
                        ora.last_flip_sens)
    assert np.array_equal(gpu.export_state()["T"], ora.T)
    gpu.destroy()


def test_many_evictions_in_place_with_the_4_bit_cache():
    """The same with codes and scales moving in place: they must arrive unchanged, in temporal order."""
    from parity_util import bf16_dev, check_attention, make_pair
    import dataclasses
    sh, wts = _hand_scored_layer(8, 2, 128, 64, seed=9)
    sh = dataclasses.replace(sh, kv_dtype=1)
    ora, gpu = make_pair(sh, wts, 150, 96, 20, reserve=8)
    g = np.random.default_rng(77)
    for i, n_tok in enumerate([96, 96, 41, 96, 1, 96, 77]):
        x = W.to_bf16_grid(g.standard_normal((n_tok, 64)).astype(np.float32))
        x[:, :2] = g.integers(-3, 40, size=(n_tok, 2)).astype(np.float32)
        out = torch.zeros((n_tok, 8 * 128), dtype=torch.bfloat16, device="cuda")
        gpu.prefill_chunk(bf16_dev(x), out, 0)
        ref = ora.prefill_chunk(x, 0)
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"int4 step {i}", ora.last_abs_out,
                        ora.last_flip_sens)
        st = gpu.export_state()
        assert np.array_equal(st["T"], ora.T), f"step {i}"
        for name in ("Kc", "Vc"):
            assert np.mean(st[name] != getattr(ora, name)) < 0.01, f"step {i}: {name}"
    for t in range(3):
        x = W.to_bf16_grid(g.standard_normal((1, 64)).astype(np.float32))
        out = torch.zeros((1, 8 * 128), dtype=torch.bfloat16, device="cuda")
        gpu.decode_step(bf16_dev(x), out)
        ref = ora.decode_step(x[0])
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"int4 decode {t}", ora.last_abs_out,
                        ora.last_flip_sens)
    gpu.destroy()


def test_one_call_for_a_stack_of_layers_equals_one_call_per_layer():
    from paper_2410_01805_b200 import LayerStack, LocretLayer
    from parity_util import bf16_dev
    sh = _shape(8, 2, 128, D=256, dR=128)
    weights = [W.layer_weights(sh, l, seed=W.BASE_SEED + 5) for l in range(3)]
    runs = []
    for use_stack in (False, True):
        layers = [LocretLayer(sh, *(bf16_dev(a) for a in wts), 300, 128, 40, reserve=8) for wts in weights]
        x0 = bf16_dev(_hidden(128, sh.d_model, 1))
        out = torch.zeros((128, 8 * 128), dtype=torch.bfloat16, device="cuda")
        for L in layers:
            L.prefill_chunk(x0, out, 0)
        outs = torch.zeros((4, 3, 8 * 128), dtype=torch.bfloat16, device="cuda")
        stack = LayerStack(layers)
        for t in range(4):
            x = bf16_dev(_hidden(1, sh.d_model, 50 + t))
            if use_stack:
                stack.decode_step(x, outs[t], out_stride=8 * 128)
            else:
                for l, L in enumerate(layers):
                    L.decode_step(x, outs[t, l])
        states = [L.export_state() for L in layers]
        assert all(L.sync_status() == 0 for L in layers)
        runs.append((outs.clone(), states))
        for L in layers:
            L.destroy()
    assert torch.equal(runs[0][0], runs[1][0])
    for a, b in zip(runs[0][1], runs[1][1]):
        for k in ("K", "V", "S", "T"):
            assert np.array_equal(a[k], b[k])
