"""locret_rh_scores_static: retaining-head scores for hosts that cannot allocate.

A caller that lives inside a device-wide memory pool, or whose allocator is locked while a
request is being served, still has to score new cache units.  This entry point takes only
the caller's buffers and keeps its partial sums in an array inside the library image.  The
tests drive it through the C ABI twice in a row and compare with the scores the regular
layer step stores for the same tokens, and with the CPU oracle's retaining head.
"""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu

SCRATCH_FLOATS = 1 << 20      # LOCRET_STATIC_SCRATCH_FLOATS


def _setup():
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    # d_model == d_in and W_qkv = identity: the staged [Q ‖ K ‖ V] equals hidden_in exactly
    sh = W.LayerShape(d_model=256, n_q_heads=2, n_kv_heads=1, head_dim=64, d_retain=160)
    g = np.random.default_rng(7)
    w1 = W.to_bf16_grid((g.standard_normal((256, 160)) / 16).astype(np.float32))
    w2 = W.to_bf16_grid((g.standard_normal((160, 1)) / 12).astype(np.float32))
    eye = np.eye(256, dtype=np.float32)
    layer = P.LocretLayer(sh, bf16_dev(eye), bf16_dev(w1), bf16_dev(w2), budget=1000, chunk=333, n_stab=0)
    return P, sh, layer, w1, w2, g


def _within_score_tolerance(got, want):
    from parity_util import SCORE_TOL
    rms = np.sqrt(np.mean(want ** 2))
    return np.all(np.abs(got - want) <= SCORE_TOL * np.maximum(np.abs(want), rms))


def test_static_scratch_scores_match_the_layer_step_twice_in_a_row():
    from parity_util import bf16_dev
    P, sh, layer, w1, w2, g = _setup()
    w1_t = bf16_dev(np.ascontiguousarray(w1.T))
    w2_f = torch.from_numpy(w2).float().cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    free_after_first = None
    for call, n_tok in enumerate([333, 200]):
        z_host = W.to_bf16_grid(g.standard_normal((n_tok, 256)).astype(np.float32))
        z = bf16_dev(z_host)
        out = torch.zeros((n_tok, 2 * 64), dtype=torch.bfloat16, device="cuda")
        before = layer.cache_len
        layer.prefill_chunk(z, out, P.NO_EVICT)
        want = layer.export_state()["S"][:, before:]                   # [h_kv, n_tok]
        got = torch.full((1, n_tok), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        if call == 1:
            free_after_first = torch.cuda.mem_get_info()[0]
        rc = P.lib.locret_rh_scores_static(z.data_ptr(), n_tok, 256, w1_t.data_ptr(), 160,
                                           w2_f.data_ptr(), 1, 0, got.data_ptr(), status.data_ptr(), stream)
        assert rc == 0, P.lib.locret_strerror(rc)
        torch.cuda.synchronize()
        if call == 1:
            # the promise in the name: the second call (the first may load the kernels' code)
            # leaves the device's free memory exactly where it was
            assert torch.cuda.mem_get_info()[0] == free_after_first
        got = got.cpu().numpy()
        assert _within_score_tolerance(got, want), f"call {call}: differs from the layer step"
        ref = O.retaining_scores(z_host.astype(np.float64), w1, w2, 0).T        # the oracle itself
        assert _within_score_tolerance(got.astype(np.float64), ref), f"call {call}: differs from the oracle"
    assert int(status.item()) == 0
    layer.destroy()


@pytest.mark.parametrize("n_tok", [1, 31, 128])
@pytest.mark.parametrize("d_retain", [64, 256])
def test_static_scratch_small_token_counts_against_the_oracle(n_tok, d_retain):
    """Token counts below a tile of the GEMM, which the layer step never sends to this kernel."""
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    g = np.random.default_rng(100 + n_tok + d_retain)
    d_in, h_kv = 192, 3
    z = W.to_bf16_grid(g.standard_normal((n_tok, d_in)).astype(np.float32))
    w1 = W.to_bf16_grid((g.standard_normal((d_in, d_retain)) / np.sqrt(d_in)).astype(np.float32))
    w2 = W.to_bf16_grid((g.standard_normal((d_retain, h_kv)) / np.sqrt(d_retain)).astype(np.float32))
    for act in (0, 1, 2):
        got = torch.full((h_kv, n_tok), float("nan"), dtype=torch.float32, device="cuda")
        zd, w1t = bf16_dev(z), bf16_dev(np.ascontiguousarray(w1.T))
        w2f = torch.from_numpy(w2).float().cuda()
        rc = P.lib.locret_rh_scores_static(zd.data_ptr(), n_tok, d_in, w1t.data_ptr(), d_retain, w2f.data_ptr(),
                                           h_kv, act, got.data_ptr(), None, torch.cuda.current_stream().cuda_stream)
        assert rc == 0, P.lib.locret_strerror(rc)
        torch.cuda.synchronize()
        ref = O.retaining_scores(z.astype(np.float64), w1, w2, act).T
        assert _within_score_tolerance(got.cpu().numpy().astype(np.float64), ref), f"act {act}"


def test_static_scratch_rejects_what_does_not_fit():
    import paper_2410_01805_b200 as P
    from parity_util import bf16_dev
    buf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    p = buf.data_ptr()
    # d_retain = 160 is sized as ceil(160 / 64) = 3 tiles -> 3 * n_tok * 1 floats
    too_many = SCRATCH_FLOATS // 3 + 1
    assert P.lib.locret_rh_scores_static(p, too_many, 256, p, 160, p, 1, 0, p, None, None) == -3
    assert P.lib.locret_rh_scores_static(p, 8, 100, p, 160, p, 1, 0, p, None, None) == -1
    assert P.lib.locret_rh_scores_static(None, 8, 256, p, 160, p, 1, 0, p, None, None) == -1
    # exactly at the limit (one tile of d_retain = 64, one head: need = n_tok floats) it runs, one more is refused
    n_tok, d_in = SCRATCH_FLOATS, 64
    g = np.random.default_rng(3)
    z = torch.from_numpy(g.standard_normal((n_tok, d_in)).astype(np.float32)).to(torch.bfloat16).cuda()
    w1 = W.to_bf16_grid((g.standard_normal((d_in, 64)) / 8).astype(np.float32))
    w2 = W.to_bf16_grid((g.standard_normal((64, 1)) / 8).astype(np.float32))
    w1t, w2f = bf16_dev(np.ascontiguousarray(w1.T)), torch.from_numpy(w2).float().cuda()
    got = torch.full((1, n_tok + 1), float("nan"), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert P.lib.locret_rh_scores_static(z.data_ptr(), n_tok + 1, d_in, w1t.data_ptr(), 64, w2f.data_ptr(), 1, 0,
                                         got.data_ptr(), None, st) == -3
    assert P.lib.locret_rh_scores_static(z.data_ptr(), n_tok, d_in, w1t.data_ptr(), 64, w2f.data_ptr(), 1, 0,
                                         got.data_ptr(), None, st) == 0
    torch.cuda.synchronize()
    rows = np.array([0, 1, 127, 128, n_tok // 2, n_tok - 1])
    ref = O.retaining_scores(z[rows].float().cpu().numpy().astype(np.float64), w1, w2, 0)[:, 0]
    sel = got[0, rows].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(sel - ref) <= 1e-2 * np.maximum(np.abs(ref), 0.5))
    assert torch.isnan(got[0, n_tok]).item() and not torch.isnan(got[0, :n_tok]).any().item()
