"""The CTA-pair attention kernel (tcgen05 cta_group::2, head_dim 128; selected with LOCRET_ATTN_PAIR=1 when a
layer is created) against the CPU oracle.  Collected after the other GPU test files."""

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


@pytest.mark.parametrize("d", [64, 128])
def test_attention_rescales_the_accumulator_when_a_later_key_tile_dominates(d, monkeypatch):
    """The tcgen05 attention kernels fix a row's scale at the first key tile they process and rescale the
    accumulator only when a later tile's maximum exceeds it by 2^100.  Ordinary inputs never do that,
    so here the query and key projections are made 12 times larger each (scores 144 times larger):
    rows whose best key tile beats every other tile by more than 100 in log2 units must take the
    rescale path whatever order the kernel walks the tiles in (unless it happens to start at that
    tile).  head_dim 64 runs the one-CTA kernel, 128 the CTA-pair kernel."""
    from parity_util import bf16_dev, check_attention, make_pair
    monkeypatch.setenv("LOCRET_ATTN_PAIR", "1")
    sh = small_shape(h=4, hk=2, d=d, D=128, dR=64)
    h, hk = sh.n_q_heads, sh.n_kv_heads
    wqkv, w1, w2 = weights_for(sh, 33)
    wqkv = wqkv.copy()
    wqkv[:, : (h + hk) * d] *= 12.0
    wqkv = W.to_bf16_grid(wqkv)
    chunk, n_chunks = 512, 3
    ora, gpu = make_pair(sh, (wqkv, w1, w2), budget=chunk * n_chunks, chunk=chunk, n_stab=0)
    out = torch.zeros((chunk, h * d), dtype=torch.bfloat16, device="cuda")
    xs = [hidden(chunk, sh.d_model, 70 + i) for i in range(n_chunks)]
    for i, x in enumerate(xs):
        gpu.prefill_chunk(bf16_dev(x), out, O.NO_EVICT)
        ref = ora.prefill_chunk(x, O.NO_EVICT)
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, f"hot scores, chunk {i}",
                        ora.last_abs_out, ora.last_flip_sens)
    assert gpu.sync_status() == 0
    gpu.destroy()

    # how many rows of the last chunk cannot avoid the rescale: scores from the oracle's own steps
    X = np.concatenate(xs, axis=0)
    qkv = O.round_bf16(O.project_qkv(X, wqkv, h, hk, d))
    Q, K, _ = O.split_qkv(qkv, h, hk, d)
    pos = np.arange(X.shape[0])
    Qr = O.round_bf16(O.rope(Q, pos[:, None], sh.rope_theta))
    Kr = O.round_bf16(O.rope(K, pos[:, None], sh.rope_theta))
    ln = chunk * (n_chunks - 1)          # keys every row of the last chunk sees in full tiles of 128
    forced = 0
    for j in range(h):
        s = (Qr[ln:, j, :] @ Kr[:ln, j // sh.group, :].T) * (np.log2(np.e) / np.sqrt(d))
        tile_max = s.reshape(chunk, ln // 128, 128).max(axis=2)
        top2 = np.sort(tile_max, axis=1)[:, -2:]
        forced += int(np.sum(top2[:, 1] - top2[:, 0] > 101.0))
    assert forced >= 50, forced


def test_both_attention_kernels_for_head_dim_128_in_lock_step_with_the_oracle(monkeypatch):
    """LOCRET_ATTN_PAIR=1 (read when a layer is created) selects the CTA-pair kernel for head_dim 128,
    otherwise the one-CTA kernel runs; both must pass the same lock-step comparison."""
    from parity_util import lockstep_chunk, make_pair
    sh = small_shape(h=8, hk=2, d=128, D=256, dR=64)
    for env in ("0", "1"):
        monkeypatch.setenv("LOCRET_ATTN_PAIR", env)
        ora, gpu = make_pair(sh, weights_for(sh, 44), budget=700, chunk=384, n_stab=16)
        for i, n_tok in enumerate([384, 200, 384, 129]):
            lockstep_chunk(ora, gpu, hidden(n_tok, sh.d_model, 90 + i), 0, what=f"LOCRET_ATTN_PAIR={env} chunk {i}")
        assert gpu.sync_status() == 0
        gpu.destroy()


@pytest.mark.parametrize("h,hk,chunk,budget,n_stab,context", [(8, 2, 256, 512, 32, 2048), (4, 4, 384, 640, 32, 2304),
                                                            (8, 2, 200, 300, 16, 1500)])
def test_pair_kernel_lock_step_gqa_mha_and_ragged_chunks(h, hk, chunk, budget, n_stab, context, monkeypatch):
    # query-head pairs of a GQA group, row-block pairs of an MHA head, and chunks that end inside a tile:
    # every chunk of a short prefill in lock-step with the oracle, eviction included
    from parity_util import lockstep_chunk, make_pair
    monkeypatch.setenv("LOCRET_ATTN_PAIR", "1")
    sh = small_shape(h=h, hk=hk, d=128, D=256, dR=128)
    ora, gpu = make_pair(sh, weights_for(sh, 50 + h), budget=budget, chunk=chunk, n_stab=n_stab)
    start, i = 0, 0
    while start < context:
        n_tok = min(chunk, context - start)
        lockstep_chunk(ora, gpu, hidden(n_tok, sh.d_model, 200 + i), 0, what=f"pair kernel h{h} hk{hk} chunk {i}")
        start += n_tok
        i += 1
    assert gpu.sync_status() == 0 and ora.len == budget
    gpu.destroy()
