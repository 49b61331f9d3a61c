"""The N > 1 bookkeeping of bench.py (replicas only) on two gloo ranks, CPU only."""

import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    t_ms, t_e2e = bench.max_over_ranks([100.0 + 50.0 * rank, 300.0 - 100.0 * rank])
    out[rank] = (t_ms, t_e2e, bench.job_throughput(world, 131072, t_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_whole_job_tokens():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    t_ms, t_e2e, value = res[0]
    assert t_ms == 150.0 and t_e2e == 300.0
    assert abs(value - 2 * 131072 / 0.150) < 1e-6


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.job_throughput(1, 1000, 500.0) == 2000.0


# ---- the step with KV heads divided over ranks: the one exchange (sum of the partial first
# products of the retaining head) done by a real all-reduce between two processes.  The CUDA
# kernels cannot run here, so each rank steps the oracle's layer for its heads; the weights are
# cut by the product's own host-side helper and checked against the oracle's cut.
def _tp_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import types
    import numpy as np
    from oracle import locret_oracle as O
    from paper_2410_01805_b200 import shard_by_kv_head
    h, hk, d, D, dR = 8, 4, 8, 16, 12
    g = np.random.default_rng(5)  # same seed on every rank: the undivided weights are replicated inputs
    d_in = (h + 2 * hk) * d
    wqkv = g.standard_normal((D, d_in)) / 4.0
    w1 = g.standard_normal((d_in, dR)) / np.sqrt(d_in)
    w2 = g.standard_normal((dR, hk)) / np.sqrt(dR)
    X = g.standard_normal((40, D))
    mk = lambda hq, hkv: types.SimpleNamespace(d_model=D, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, d_retain=dR,
                                               rope_theta=10000.0, act=0, rh_input=0, kv_dtype=0)
    cut = shard_by_kv_head(torch.from_numpy(wqkv), torch.from_numpy(w1), torch.from_numpy(w2), h, hk, d, rank, world)
    cut_ref = O.shard_by_kv_head(wqkv, w1, w2, h, hk, d, rank, world)
    same_cut = all(np.array_equal(a.numpy(), b) for a, b in zip(cut, cut_ref))
    mine = O.OracleLayer(mk(h // world, hk // world), *[c.numpy() for c in cut], 16, 8, 2)
    whole = O.OracleLayer(mk(h, hk), wqkv, w1, w2, 16, 8, 2)
    ok = same_cut
    hl, hkl = h // world, hk // world
    for s in range(0, 40, 8):
        x = X[s:s + 8]
        pre = torch.from_numpy(mine.partial_preact(x))
        dist.all_reduce(pre, op=dist.ReduceOp.SUM)          # the exchange step
        got = mine.prefill_chunk(x, preact=pre.numpy())
        want = whole.prefill_chunk(x)
        ok = ok and np.allclose(got, want[:, rank * hl * d:(rank + 1) * hl * d], atol=1e-12)
        ok = ok and np.array_equal(mine.T, whole.T[rank * hkl:(rank + 1) * hkl])
        ok = ok and np.allclose(mine.S, whole.S[rank * hkl:(rank + 1) * hkl], atol=1e-12)
    out[rank] = (bool(ok), mine.len, int(whole.len))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_with_divided_heads_reproduce_the_undivided_layer():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_tp_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == (True, 16, 16) and res[1] == (True, 16, 16)
