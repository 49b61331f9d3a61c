"""Parity of the whole decoder layer (locret_block_*) with the oracle's OracleBlock."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu

# |Δy| <= BLOCK_TOL * max(1, |y_ref|).  y = x1 + FFN(RMSNorm(x1)) with x1 = x + attn_out W_o: the
# attention output enters with its own 2e-2 bound and is mixed by W_o (entries N(0, 1/fan_in), so the
# error keeps its magnitude); the five bf16 storage points in between (h1, attn_out, x1, h2, the gated
# product) add independent 2^-9 relative roundings whose one-ulp disagreements between fp32 and fp64
# accumulation are amplified by at most the gain of the FFN (about 1 for these weights).
BLOCK_TOL = 3e-2


def block_pair(shape, seed, budget, chunk, n_stab, reserve=0):
    from parity_util import bf16_dev
    from paper_2410_01805_b200 import LocretBlock
    wqkv, w1, w2 = W.layer_weights(shape, 0, seed=W.BASE_SEED + seed)
    bw = W.block_weights(shape, 0, seed=W.BASE_SEED + seed)
    layer = O.OracleLayer(shape, wqkv, w1, w2, budget, chunk, n_stab, reserve=reserve, mirror=True)
    ora = O.OracleBlock(layer, bw["w_o"], bw["w_gate"], bw["w_up"], bw["w_down"], bw["g1"], bw["g2"])
    gpu = LocretBlock(shape, bf16_dev(wqkv), bf16_dev(w1), bf16_dev(w2), bf16_dev(bw["w_o"]),
                      bf16_dev(bw["w_gate"]), bf16_dev(bw["w_up"]), bf16_dev(bw["w_down"]),
                      bf16_dev(bw["g1"]), bf16_dev(bw["g2"]), budget, chunk, n_stab, reserve=reserve)
    return ora, gpu


def hidden(n, D, seed):
    g = np.random.default_rng(5000 + seed)
    return W.to_bf16_grid((g.standard_normal((n, D)) * 1.5).astype(np.float32))


def lockstep_block(ora, gpu, x, flags, what):
    from parity_util import bf16_dev, import_oracle_state
    st = ora.attn.export_state()
    import_oracle_state(gpu.attn, st, bool(ora.attn.int4))
    xd = bf16_dev(x)
    y = torch.zeros_like(xd)
    gpu.prefill_chunk(xd, y, flags)
    assert gpu.attn.sync_status() == 0
    ref = ora.prefill_chunk(x, flags)
    got = y.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref) / np.maximum(1.0, np.abs(ref))
    assert np.isfinite(got).all()
    assert err.max() <= BLOCK_TOL, f"{what}: worst err/bound {err.max() / BLOCK_TOL:.3f}"
    assert gpu.attn.cache_len == ora.attn.len
    return float(err.max())


@pytest.mark.parametrize("dims", [dict(h=4, hk=2, d=64, D=128, dR=64, F=256),      # tcgen05 GEMMs
                                  dict(h=2, hk=1, d=128, D=256, dR=64, F=384),
                                  dict(h=3, hk=3, d=96, D=96, dR=72, F=128)])     # fallback kernels
def test_block_lockstep_with_eviction(dims):
    sh = W.LayerShape(d_model=dims["D"], n_q_heads=dims["h"], n_kv_heads=dims["hk"], head_dim=dims["d"],
                      d_retain=dims["dR"], rope_theta=500000.0, d_ff=dims["F"])
    ora, gpu = block_pair(sh, 31, budget=150, chunk=96, n_stab=16)
    worst = 0.0
    for i, n_tok in enumerate([96, 96, 40, 96, 1, 33]):
        worst = max(worst, lockstep_block(ora, gpu, hidden(n_tok, sh.d_model, i), 0, f"{dims} chunk {i}"))
    assert ora.attn.len == 150
    print("worst relative error", worst)
    gpu.destroy()


def test_block_in_place_and_argument_checks():
    from parity_util import bf16_dev
    from paper_2410_01805_b200 import LocretError
    sh = W.LayerShape(d_model=128, n_q_heads=4, n_kv_heads=2, head_dim=64, d_retain=64, d_ff=256)
    ora, gpu = block_pair(sh, 32, budget=100, chunk=64, n_stab=8)
    x = hidden(64, 128, 9)
    xd = bf16_dev(x)
    ref = ora.prefill_chunk(x, 0)
    gpu.prefill_chunk(xd, xd, 0)                       # y written over x
    got = xd.float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref) / np.maximum(1.0, np.abs(ref))).max() <= BLOCK_TOL
    with pytest.raises(LocretError):
        gpu.prefill_chunk(xd[:0], xd[:0], 0, n_tok=0)
    with pytest.raises(LocretError):
        gpu.prefill_chunk(xd, xd, 0, n_tok=65)
    gpu.destroy()


def test_block_at_the_llama_shape_sampled_rows():
    """Full benchmark shape (d_model 4096, 32/8 heads of 128, d_ff 14336), chunks of 3072 in the
    launch configuration bench.py times; rows sampled (everything after attention is row-wise, the
    oracle computes the sampled rows only)."""
    from parity_util import bf16_dev, import_oracle_state
    w = W.get_workload("c3_llama_128k")
    ora, gpu = block_pair(w.shape, 0, w.budget, w.chunk, w.n_stab)
    start = 0
    for i, n_tok in enumerate(w.chunk_sizes()[:3]):          # the third chunk evicts at full cache
        x = W.hidden_states(w, start, n_tok)
        g = np.random.default_rng(700 + i)
        rows = sorted(set(g.integers(0, n_tok, size=5).tolist()) | {0, 127, 128, n_tok - 1})
        st = ora.attn.export_state()
        import_oracle_state(gpu.attn, st, False)
        xd = bf16_dev(x)
        y = torch.zeros_like(xd)
        gpu.prefill_chunk(xd, y, 0)
        assert gpu.attn.sync_status() == 0
        ref = ora.prefill_chunk(x, 0, rows=rows)
        got = y.float().cpu().numpy().astype(np.float64)
        ok = ~np.isnan(ref)
        err = np.abs(got[ok] - ref[ok]) / np.maximum(1.0, np.abs(ref[ok]))
        assert err.max() <= BLOCK_TOL, f"chunk {i}: worst err/bound {err.max() / BLOCK_TOL:.3f}"
        start += n_tok
    gpu.destroy()
