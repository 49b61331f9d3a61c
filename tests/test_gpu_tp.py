"""The step with KV heads divided over GPUs, through the C ABI, against the UNDIVIDED oracle layer.

One GPU is available, so the shards of all ranks live on it as separate layer objects and run one
after the other; the exchange step (the all-reduce of the partial first products of the retaining
head) is a plain sum of the ranks' buffers.  No kernel waits on another."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


class ShardsOnOneGpu:
    """Presents `world` per-rank layer objects as one layer to the lock-step comparison."""

    def __init__(self, shape, weights, budget, chunk, n_stab, world, reserve=0, fused=False):
        from dataclasses import replace
        from paper_2410_01805_b200 import LocretLayer, shard_by_kv_head
        from parity_util import bf16_dev
        self.world, self.shape = world, shape
        self.hl, self.hkl, self.d = shape.n_q_heads // world, shape.n_kv_heads // world, shape.head_dim
        wq, w1, w2 = (bf16_dev(w) for w in weights)
        local = replace(shape, n_q_heads=self.hl, n_kv_heads=self.hkl)
        self.cuts = [shard_by_kv_head(wq, w1, w2, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, r, world)
                     for r in range(world)]
        self.layers = [LocretLayer(local, *c, budget, chunk, n_stab, reserve=reserve) for c in self.cuts]
        self.pre = [torch.empty(chunk, shape.d_retain, dtype=torch.float32, device="cuda") for _ in range(world)]
        self.outs = [torch.zeros(chunk, self.hl * self.d, dtype=torch.bfloat16, device="cuda") for _ in range(world)]
        # fused: every rank's GEMM adds its product into every rank's sum buffer (here all on this device)
        self.fused = fused
        if fused:
            for L in self.layers:
                L.tp_set_peers(self.pre)

    def prefill_chunk(self, x, out, flags=0):
        n_tok = x.shape[0]
        if self.fused:
            for p in self.pre:
                p.zero_()                      # first ordering of the exchange: all buffers zero before anyone adds
            for r, L in enumerate(self.layers):
                L.prefill_chunk_tp_begin_peers(x, self.outs[r], flags, n_tok)
            torch.cuda.synchronize()           # second ordering: everybody has added before anybody reads
            for r, L in enumerate(self.layers):
                L.prefill_chunk_tp_finish(self.pre[r])
                out[:n_tok, r * self.hl * self.d:(r + 1) * self.hl * self.d] = self.outs[r][:n_tok]
            torch.cuda.synchronize()           # (the buffers are zeroed again at the next step)
            return
        for r, L in enumerate(self.layers):
            L.prefill_chunk_tp_begin(x, self.outs[r], self.pre[r], flags, n_tok)
        total = torch.stack([p[:n_tok] for p in self.pre]).sum(dim=0).contiguous()   # the exchange step
        for r, L in enumerate(self.layers):
            L.prefill_chunk_tp_finish(total)
            out[:n_tok, r * self.hl * self.d:(r + 1) * self.hl * self.d] = self.outs[r][:n_tok]

    def export_state(self):
        parts = [L.export_state() for L in self.layers]
        st = {k: np.concatenate([p[k] for p in parts], axis=0) for k in parts[0] if k != "seen"}
        assert len({p["seen"] for p in parts}) == 1
        st["seen"] = parts[0]["seen"]
        return st

    def import_state(self, K, V, S, T, seen):
        for r, L in enumerate(self.layers):
            sl = slice(r * self.hkl, (r + 1) * self.hkl)
            L.import_state(K[sl], V[sl], S[sl], T[sl], seen)

    def import_state_int4(self, Kc, Ks, Vc, Vs, S, T, seen):
        for r, L in enumerate(self.layers):
            sl = slice(r * self.hkl, (r + 1) * self.hkl)
            L.import_state_int4(Kc[sl], Ks[sl], Vc[sl], Vs[sl], S[sl], T[sl], seen)

    @property
    def cache_len(self):
        lens = {L.cache_len for L in self.layers}
        assert len(lens) == 1, "ranks disagree on the cache length"
        return lens.pop()

    def sync_status(self):
        return max(abs(L.sync_status()) for L in self.layers)

    def destroy(self):
        for L in self.layers:
            L.destroy()


def oracle_for(shape, weights, budget, chunk, n_stab):
    ora = O.OracleLayer(shape, *weights, budget, chunk, n_stab, mirror=True)
    ora.want_flip_sens = True
    return ora


@pytest.mark.parametrize("world,h,hk,d", [(2, 8, 4, 64), (4, 8, 4, 64), (2, 4, 2, 128), (2, 6, 2, 96), (1, 4, 2, 64)])
def test_divided_heads_lockstep_with_the_undivided_oracle(world, h, hk, d):
    from parity_util import lockstep_chunk
    sh = W.LayerShape(d_model=128, n_q_heads=h, n_kv_heads=hk, head_dim=d, d_retain=96, rope_theta=500000.0)
    weights = W.layer_weights(sh, 0, seed=W.BASE_SEED + 900 + world)
    ora = oracle_for(sh, weights, 300, 200, 17)
    gpu = ShardsOnOneGpu(sh, weights, 300, 200, 17, world)
    g = np.random.default_rng(4242)
    exact = 0
    sizes = [1, 127, 129, 200, 64, 200, 3]
    for i, n_tok in enumerate(sizes):
        x = W.to_bf16_grid(g.standard_normal((n_tok, sh.d_model)).astype(np.float32))
        st = lockstep_chunk(ora, gpu, x, 0, what=f"tp{world} chunk {i}")
        exact += bool(st.get("sets_identical", True))
    assert ora.len == 300 and exact >= len(sizes) - 1
    gpu.destroy()


def test_divided_heads_with_the_4bit_cache():
    from parity_util import lockstep_chunk
    sh = W.LayerShape(d_model=128, n_q_heads=8, n_kv_heads=4, head_dim=128, d_retain=96, kv_dtype=1)
    weights = W.layer_weights(sh, 0, seed=W.BASE_SEED + 930)
    ora = oracle_for(sh, weights, 300, 200, 17)
    gpu = ShardsOnOneGpu(sh, weights, 300, 200, 17, 2)
    g = np.random.default_rng(31)
    for i, n_tok in enumerate([200, 130, 200, 1, 64]):
        x = W.to_bf16_grid(g.standard_normal((n_tok, sh.d_model)).astype(np.float32))
        lockstep_chunk(ora, gpu, x, 0, what=f"tp2 int4 chunk {i}")
    assert ora.len == 300
    gpu.destroy()


def test_divided_heads_general_shape_kernels_and_flags():
    from parity_util import lockstep_chunk
    # D = 96, d_R = 72: neither product fits the tensor-core GEMMs, so the fallback kernels run
    sh = W.LayerShape(d_model=96, n_q_heads=6, n_kv_heads=3, head_dim=64, d_retain=72, act=1)
    weights = W.layer_weights(sh, 0, seed=W.BASE_SEED + 950)
    ora = oracle_for(sh, weights, 150, 100, 9)
    gpu = ShardsOnOneGpu(sh, weights, 150, 100, 9, 3)
    g = np.random.default_rng(77)
    for i, (n_tok, flags) in enumerate([(100, 0), (100, O.NO_EVICT), (40, 0), (100, O.LAST_CHUNK)]):
        x = W.to_bf16_grid(g.standard_normal((n_tok, sh.d_model)).astype(np.float32))
        lockstep_chunk(ora, gpu, x, flags, what=f"tp3 general chunk {i}")
    gpu.destroy()


def test_llama_shape_one_kv_head_per_gpu():
    from parity_util import lockstep_chunk
    w = W.get_workload("c3_llama_128k")
    sh = w.shape
    weights = W.layer_weights(sh, 0)
    ora = oracle_for(sh, weights, 1024, 512, 100)
    gpu = ShardsOnOneGpu(sh, weights, 1024, 512, 100, 8)
    rows = np.array([0, 1, 130, 255, 256, 400, 511])
    start = 0
    for i in range(4):
        x = W.hidden_states(w, start, 512)
        lockstep_chunk(ora, gpu, x, 0, rows=rows, what=f"llama tp8 chunk {i}")
        start += 512
    assert ora.len == 1024
    gpu.destroy()


def test_wrapper_with_one_rank_and_call_order_errors():
    from paper_2410_01805_b200 import LocretError, LocretLayerTP
    from parity_util import bf16_dev, check_attention, check_scores
    sh = W.LayerShape(d_model=128, n_q_heads=4, n_kv_heads=2, head_dim=64, d_retain=96)
    weights = W.layer_weights(sh, 0, seed=W.BASE_SEED + 970)
    ora = oracle_for(sh, weights, 120, 80, 5)
    tp = LocretLayerTP(sh, *(bf16_dev(w) for w in weights), 120, 80, 5, rank=0, world=1, reduce=lambda t: None)
    g = np.random.default_rng(9)
    out = torch.zeros(80, sh.n_q_heads * sh.head_dim, dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        x = W.to_bf16_grid(g.standard_normal((80, sh.d_model)).astype(np.float32))
        before = ora.export_state()
        tp.layer.import_state(before["K"], before["V"], before["S"], before["T"], before["seen"])
        tp.prefill_chunk(bf16_dev(x), out)
        ref = ora.prefill_chunk(x)
        check_attention(out.float().cpu().numpy().astype(np.float64), ref, "tp wrapper", ora.last_abs_out,
                        ora.last_flip_sens)
        assert tp.layer.cache_len == ora.len
    # call order: finish needs a begun step; a begun step blocks every other step; reset abandons it
    L = tp.layer
    pre = torch.zeros(80, sh.d_retain, dtype=torch.float32, device="cuda")
    xd = bf16_dev(W.to_bf16_grid(g.standard_normal((80, sh.d_model)).astype(np.float32)))
    with pytest.raises(LocretError):
        L.prefill_chunk_tp_finish(pre)
    L.reset()
    L.prefill_chunk_tp_begin(xd, out, pre)
    with pytest.raises(LocretError):
        L.prefill_chunk(xd, out)
    with pytest.raises(LocretError):
        L.prefill_chunk_tp_begin(xd, out, pre)
    L.reset()
    L.prefill_chunk(xd, out)
    assert L.cache_len == 80 and L.sync_status() == 0
    tp.destroy()


@pytest.mark.parametrize("world,h,hk,d,D,dR", [(2, 8, 4, 64, 128, 96), (4, 8, 4, 128, 128, 256), (3, 6, 3, 64, 96, 72)])
def test_exchange_inside_the_gemm_epilogue_all_buffers_on_one_device(world, h, hk, d, D, dR):
    """The divided step whose first product is added, tile by tile, into every rank's sum buffer by the
    GEMM's epilogue (reductions to global memory; on several GPUs the buffers are peers' memory, here they
    all live on this device).  D = 96 / d_R = 72 takes the fallback kernels."""
    from parity_util import lockstep_chunk
    sh = W.LayerShape(d_model=D, n_q_heads=h, n_kv_heads=hk, head_dim=d, d_retain=dR, rope_theta=500000.0)
    weights = W.layer_weights(sh, 0, seed=W.BASE_SEED + 990 + world)
    ora = oracle_for(sh, weights, 300, 200, 17)
    gpu = ShardsOnOneGpu(sh, weights, 300, 200, 17, world, fused=True)
    g = np.random.default_rng(777)
    for i, n_tok in enumerate([200, 127, 200, 33, 200]):
        x = W.to_bf16_grid(g.standard_normal((n_tok, sh.d_model)).astype(np.float32))
        lockstep_chunk(ora, gpu, x, 0, what=f"fused tp{world} chunk {i}")
    assert ora.len == 300 and gpu.sync_status() == 0
    gpu.destroy()


def test_exchange_inside_the_gemm_epilogue_at_the_llama_shape():
    from parity_util import lockstep_chunk
    w = W.get_workload("c3_llama_128k")
    weights = W.layer_weights(w.shape, 0)
    ora = oracle_for(w.shape, weights, 1024, 512, 100)
    gpu = ShardsOnOneGpu(w.shape, weights, 1024, 512, 100, 4, fused=True)
    start = 0
    for i in range(3):
        x = W.hidden_states(w, start, 512)
        lockstep_chunk(ora, gpu, x, 0, rows=np.array([0, 130, 511]), what=f"llama fused tp4 chunk {i}")
        start += 512
    gpu.destroy()
