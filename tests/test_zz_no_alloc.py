"""locret_rh_scores_static: retaining-head scores for hosts that cannot allocate.

A caller that lives inside a device-wide memory pool, or whose allocator is locked while a
request is being served, still has to score new cache units.  This entry point takes only
the caller's buffers and keeps its partial sums in an array inside the library image.  The
test drives it through the C ABI twice in a row and compares with the scores the regular
layer step stores for the same tokens.
"""

import ctypes as C

import numpy as np
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu


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


def test_static_scratch_scores_match_the_layer_step_twice_in_a_row():
    from parity_util import SCORE_TOL, bf16_dev
    P, sh, layer, w1, w2, g = _setup()
    w1_t = bf16_dev(np.ascontiguousarray(w1.T))
    w2_f = torch.from_numpy(w2).float().cuda()
    stream = torch.cuda.current_stream().cuda_stream
    for call, n_tok in enumerate([333, 200]):
        z = bf16_dev(W.to_bf16_grid(g.standard_normal((n_tok, 256)).astype(np.float32)))
        out = torch.zeros((n_tok, 2 * 64), dtype=torch.bfloat16, device="cuda")
        before = layer.cache_len
        layer.prefill_chunk(z, out, P.NO_EVICT)
        want = layer.export_state()["S"][:, before:]                   # [h_kv, n_tok]
        got = torch.full((1, n_tok), float("nan"), dtype=torch.float32, device="cuda")
        rc = P.lib.locret_rh_scores_static(z.data_ptr(), n_tok, 256, w1_t.data_ptr(), 160,
                                           w2_f.data_ptr(), 1, 0, got.data_ptr(), stream)
        assert rc == 0, P.lib.locret_strerror(rc)
        torch.cuda.synchronize()
        got = got.cpu().numpy()
        rms = np.sqrt(np.mean(want ** 2))
        assert np.all(np.abs(got - want) <= SCORE_TOL * np.maximum(np.abs(want), rms)), f"call {call}"
    layer.destroy()


def test_static_scratch_rejects_what_does_not_fit():
    P, sh, layer, w1, w2, g = _setup()
    layer.destroy()
    buf = torch.zeros(1024, dtype=torch.float32, device="cuda")
    p = buf.data_ptr()
    too_many = (1 << 20) // 2 + 1            # 2 tiles of d_retain = 160 -> 2 * n_tok * 1 floats
    assert P.lib.locret_rh_scores_static(p, too_many, 256, p, 160, p, 1, 0, p, None) == -3
    assert P.lib.locret_rh_scores_static(p, 8, 100, p, 160, p, 1, 0, p, None) == -1
    assert P.lib.locret_rh_scores_static(None, 8, 256, p, 160, p, 1, 0, p, None) == -1
