"""A budget per KV head (Appendix H: heads evict independently), through the C ABI, against the oracle."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


def make_pair(shape, weights, budgets, chunk, n_stab, reserve=0):
    from paper_2410_01805_b200 import LocretLayer
    from parity_util import bf16_dev
    ora = O.OracleLayerHeadBudgets(shape, *weights, budgets, chunk, n_stab, reserve=reserve, mirror=True)
    ora.want_flip_sens = True
    gpu = LocretLayer(shape, *(bf16_dev(w) for w in weights), max(budgets), chunk, n_stab, reserve=reserve)
    gpu.set_head_budgets(budgets)
    return ora, gpu


def lockstep(ora, gpu, x, flags=0, what=""):
    """The oracle's state goes into the CUDA layer, both run the chunk, everything is compared per head."""
    from parity_util import BAND, FLIP_FRACTION, bf16_dev, check_attention, check_keep_band, check_scores
    sh = ora.s
    h, hk, d = sh.n_q_heads, sh.n_kv_heads, sh.head_dim
    n_tok = x.shape[0]
    st = ora.export_state()
    lens = ora.lens
    xd = bf16_dev(x)
    out_a = torch.zeros((n_tok, h * d), dtype=torch.bfloat16, device="cuda")
    out_b = torch.zeros_like(out_a)
    gpu.import_state_heads(st["K"], st["V"], st["S"], st["T"], st["seen"])
    gpu.prefill_chunk(xd, out_a, O.NO_EVICT)
    pre = gpu.export_state_heads()
    gpu.import_state_heads(st["K"], st["V"], st["S"], st["T"], st["seen"])
    gpu.prefill_chunk(xd, out_b, flags)
    post = gpu.export_state_heads()
    assert gpu.sync_status() == 0 and torch.equal(out_a, out_b)
    ref = ora.prefill_chunk(x, flags)
    check_attention(out_b.float().cpu().numpy().astype(np.float64), ref, what, ora.last_abs_out, ora.last_flip_sens)
    qkv = O.round_bf16(O.project_qkv(x, ora.w_qkv, h, hk, d))
    _, Kc, Vc = O.split_qkv(qkv, h, hk, d)
    got_s = np.stack([pre["S"][m][lens[m]:] for m in range(hk)], axis=1).astype(np.float64)
    check_scores(got_s, ora.last_scores, what)
    identical = True
    for m in range(hk):
        n = lens[m] + n_tok
        assert len(pre["T"][m]) == n
        assert np.array_equal(pre["K"][m][:lens[m]], st["K"][m].astype(np.float32))
        assert np.array_equal(pre["T"][m][lens[m]:], st["seen"] + np.arange(n_tok))
        for name, ref_c in (("K", Kc[:, m]), ("V", Vc[:, m])):
            diff = np.abs(pre[name][m][lens[m]:] - ref_c)
            assert np.all(diff <= np.abs(ref_c) * 2.0 ** -7 + 1e-5 * np.abs(ref_c).max()), f"{what}: head {m} {name}"
            assert np.mean(diff != 0) < 4 * FLIP_FRACTION
        evict = not (flags & O.NO_EVICT) and n > ora.budgets[m]
        if evict:
            n_prot = 0 if (flags & O.LAST_CHUNK) else min(ora.n_stab, n)
            pos = np.searchsorted(pre["T"][m], post["T"][m])
            assert np.array_equal(pre["T"][m][pos], post["T"][m]) and np.all(np.diff(pos) > 0)
            s_ref = np.concatenate([st["S"][m], ora.last_scores[:, m]])
            identical &= check_keep_band(pos, s_ref, ora.budgets[m], n_prot, ora.last_keep[m], f"{what} head {m}",
                                         n_pre=ora.n_prefix)
            for key in ("K", "V"):
                assert np.array_equal(post[key][m], pre[key][m][pos]), f"{what}: head {m} {key} not a bit-exact gather"
            assert np.array_equal(post["S"][m].view(np.uint32), pre["S"][m][pos].view(np.uint32))
        else:
            for key in ("K", "V", "T"):
                assert np.array_equal(post[key][m], pre[key][m])
    assert gpu.cache_lens == ora.lens and gpu.cache_len == max(ora.lens)
    return identical


def hidden(n, D, seed):
    g = np.random.default_rng(4000 + seed)
    return W.to_bf16_grid(g.standard_normal((n, D)).astype(np.float32))


@pytest.mark.parametrize("d,heads,budgets", [(128, (8, 2), [300, 120]), (96, (3, 3), [64, 300, 150]),
                                             (64, (4, 4), [200, 90, 300, 33])])
def test_head_budgets_lockstep(d, heads, budgets):
    sh = W.LayerShape(d_model=128, n_q_heads=heads[0], n_kv_heads=heads[1], head_dim=d, d_retain=96,
                      rope_theta=500000.0)
    ora, gpu = make_pair(sh, W.layer_weights(sh, 0, seed=W.BASE_SEED + 60 + d), budgets, 200, 17, reserve=8)
    for i, (n_tok, flags) in enumerate([(200, 0), (127, 0), (200, 0), (1, 0), (64, 0), (200, O.NO_EVICT), (5, 0),
                                        (150, O.LAST_CHUNK)]):
        lockstep(ora, gpu, hidden(n_tok, sh.d_model, i), flags, what=f"d{d} budgets {budgets} chunk {i}")
    assert ora.lens == budgets
    gpu.destroy()


def test_head_budgets_free_running_with_hand_made_scores():
    """No import between steps: every head evicts in place on its own schedule (a head with a large budget
    starts to evict chunks later than one with a small budget), with exact tie-laden scores."""
    from parity_util import bf16_dev, check_attention
    from test_gpu_free_running import _hand_scored_layer
    h, hk, d = 8, 4, 128
    sh, wts = _hand_scored_layer(h, hk, d, 64, seed=3)
    budgets = [150, 60, 400, 97]
    ora, gpu = make_pair(sh, wts, budgets, 96, 20, reserve=8)
    g = np.random.default_rng(808)
    for i, n_tok in enumerate([96, 96, 41, 96, 1, 96, 77, 96, 96, 13]):
        x = W.to_bf16_grid(g.standard_normal((n_tok, 64)).astype(np.float32))
        x[:, :hk] = g.integers(-3, 40, size=(n_tok, hk)).astype(np.float32)
        out = torch.zeros((n_tok, h * d), dtype=torch.bfloat16, device="cuda")
        gpu.prefill_chunk(bf16_dev(x), out, 0)
        ref = ora.prefill_chunk(x, 0)
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"step {i}", ora.last_abs_out,
                        ora.last_flip_sens)
        st = gpu.export_state_heads()
        for m in range(hk):
            assert np.array_equal(st["T"][m], ora.Th[m]), f"step {i} head {m}: retained token ids differ"
            assert np.array_equal(st["S"][m].astype(np.float64), ora.Sh[m]), f"step {i} head {m}: scores differ"
        assert gpu.sync_status() == 0
    assert gpu.cache_lens == [150, 60, 400, 97]
    gpu.destroy()


def test_head_budgets_argument_checks():
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    sh = W.LayerShape(d_model=128, n_q_heads=4, n_kv_heads=2, head_dim=64, d_retain=96)
    wts = tuple(bf16_dev(w) for w in W.layer_weights(sh, 0))
    L = P.LocretLayer(sh, *wts, 100, 64, 10)
    with pytest.raises(P.LocretError):
        L.set_head_budgets([101, 50])            # beyond the budget that sized the cache
    with pytest.raises(P.LocretError):
        L.set_head_budgets([50, 9])              # below the stabilizers
    L.set_head_budgets([50, 100])
    x = bf16_dev(hidden(64, 128, 1))
    out = torch.zeros((64, 4 * 64), dtype=torch.bfloat16, device="cuda")
    L.prefill_chunk(x, out)
    with pytest.raises(P.LocretError):
        L.set_head_budgets([60, 60])             # only while the layer is empty
    with pytest.raises(P.LocretError):
        L.export_state()                         # the plain exchange is refused: lengths differ
    L.prefill_chunk(x, out)
    assert L.cache_lens == [50, 100] and L.cache_len == 100
    L.reset()
    L.set_head_budgets([60, 60])
    L.destroy()
