#!/usr/bin/env python
"""Chunked-prefill throughput of the Locret hot path on B200.

One "step" = one whole prefill of the workload's context through the whole layer stack:
every chunk, every layer, all kernels of the per-layer step (projection, position
assignment + RoPE + append, attention, retaining head, top-b selection, compaction).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs the same workload
on an independent request (the path is a sequential recurrence over chunks and shards
only by request: "replicas only", weak scaling, no data-path collective).
"""

from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
# The benchmark runs Eq. 1 for head_dim 128 on the CTA-pair kernel (tcgen05 cta_group::2), which the library
# keeps opt-in; LOCRET_ATTN_PAIR=0 in the environment measures the default one-CTA kernel instead.
os.environ.setdefault("LOCRET_ATTN_PAIR", "1")

import workloads as W  # noqa: E402

METRIC = "chunked-prefill tokens/sec at 128K ctx (1 B200); % tensor/HBM roofline per kernel"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "c3_llama_128k"
# dram__bytes_read.sum + dram__bytes_write.sum of one steady-state attention launch: a literal taken
# from a profiler capture of the same launch shape (not measured during this run)
NCU_ATTN_TRAFFIC_BYTES = {"c3_llama_128k": 70.9e6, "c2_llama_32k": 70.9e6}
# sm__pipe_tensor_cycles_active of the same capture (per cent of cycles; clock-independent)
NCU_ATTN_TENSOR_PIPE_PCT = 60.9
# the other benchmark configurations are sampled in the default run: this many layers, contexts cut to this
OTHER_CONFIGS = ("c2_llama_32k", "c4_phi3_128k", "c5_llama_stream_int4")
OTHER_LAYERS = 4
OTHER_CONTEXT = 65536


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], tf=d["bf16_tflops"], tf_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tf=1590.0, tf_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self.index = index
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True,
                                     timeout=5).stdout.strip().splitlines()[0]
                f = [x.strip() for x in out.split(",")]
                self.samples.append(float(f[0])); self.max_mhz = float(f[1])
                for n, v in zip(names, f[2:]):
                    if v.lower().startswith("active"):
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self.t.start(); return self

    def __exit__(self, *a):
        self._stop.set(); self.t.join(timeout=6)

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- work counts

def chunk_layer_flops(w: W.Workload, ln: int, n_tok: int):
    s = w.shape
    qkv = 2.0 * n_tok * s.d_model * s.d_in
    attn = 4.0 * s.n_q_heads * s.head_dim * (n_tok * ln + n_tok * (n_tok + 1) / 2)
    rh = 2.0 * n_tok * s.d_in * s.d_retain + 2.0 * n_tok * s.d_retain * s.n_kv_heads
    return qkv, attn, rh


def step_flops(w: W.Workload):
    ln, tot = 0, np.zeros(3)
    for n_tok in w.chunk_sizes():
        tot += np.array(chunk_layer_flops(w, ln, n_tok))
        ln = min(w.budget, ln + n_tok)
    return tot * w.n_layers


# ----------------------------------------------------------------------------- reference arm (oracle on CPU)

class OracleSampler:
    """The oracle, as it stands, brought to the workload's steady state once; every sample() then
    times `n_chunks` steady-state chunk-layers of layer 0 on the host cores."""

    def __init__(self, w: W.Workload):
        from oracle import locret_oracle as O
        self.w = w
        self.ora = O.OracleLayer(w.shape, *W.layer_weights(w.shape, 0), w.budget, w.chunk, w.n_stab, mirror=True)
        self.sizes = w.chunk_sizes()
        self.start, self.fill = 0, 0
        # fill the cache without paying for attention (one query row per chunk)
        while self.ora.len < min(w.budget, w.context - w.chunk) and self.fill < len(self.sizes) - 1:
            self.ora.prefill_chunk(W.hidden_states(w, self.start, self.sizes[self.fill]), 0, rows=[0])
            self.start += self.sizes[self.fill]; self.fill += 1

    def sample(self, n_chunks: int = 1):
        from threadpoolctl import threadpool_info
        w, times, toks = self.w, [], 0
        for _ in range(n_chunks):
            idx = min(self.fill, len(self.sizes) - 2)          # a full-size chunk
            if self.start + self.sizes[idx] > w.context:
                self.start = self.fill_start()
            x = W.hidden_states(w, self.start, self.sizes[idx])
            t0 = time.perf_counter()
            self.ora.prefill_chunk(x, 0)
            times.append(time.perf_counter() - t0)
            toks += self.sizes[idx]; self.start += self.sizes[idx]
        cores = max([p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"] + [1])
        sec = float(np.sum(times))
        # one chunk-layer handles n_tok tokens of ONE layer; the whole job does n_layers of them per chunk
        tok_s = toks / sec / w.n_layers
        sample = (f"{n_chunks} steady-state chunk-layer(s) of layer 0 ({toks} tokens, cache {self.ora.len} units/head), "
                  f"{sec:.1f} s; tokens/s = tokens / time / {w.n_layers} layers")
        return tok_s, cores, sample, sec

    def fill_start(self):
        return sum(self.sizes[:self.fill])


def oracle_sample(w: W.Workload, n_chunks: int):
    return OracleSampler(w).sample(n_chunks)


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    t_all = time.perf_counter()
    vals = []
    total = args.steps + args.warmup
    n_per = 1
    sample = ""
    cores = 1
    sampler = OracleSampler(w)
    for i in range(total):
        v, cores, sample, _ = sampler.sample(n_per)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": w.context / value * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "CPU oracle (numpy fp64), bounded sample extrapolated linearly"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": time.perf_counter() - t_all,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- multi-rank bookkeeping

def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world: int, tokens_per_rank: int, ms: float) -> float:
    """Replicas only: every rank prefills its own request; whole-job tokens over the slowest rank's time."""
    return world * tokens_per_rank / (ms * 1e-3)


# ----------------------------------------------------------------------------- per-kernel rates

def compaction_bytes(w, evictions, moved, rotated):
    """Algorithmic bytes of the in-place gather: per evicting launch the index and position arrays of
    every slot; per unit moved to another slot K and V read and written, its score and token id; per
    rotated key rewritten the pre-RoPE key read (a moved unit's is already counted) and the rotated key
    written."""
    s = w.shape
    idx = evictions * s.n_kv_heads * w.budget * 12
    if s.kv_dtype == 1:
        return idx + moved * (2 * (s.head_dim // 2) * 2 + 2 * 2 * 2 + 2 * (4 + 8))
    row = s.head_dim * 2
    return idx + moved * (4 * row + 2 * (4 + 8)) + (rotated - moved) * row + rotated * row


def summarise(w, k_ms, k_cnt, steps, peaks, compact_bytes=None):
    """Per kernel family: launches, time, share, and the rate against the roofline that bounds it
    (tensor kernels: TFLOP/s of the algorithmic flops against the sustained bf16 peak; compaction:
    GB/s of the bytes it had to move, counted by the library, against the measured copy bandwidth)."""
    from paper_2410_01805_b200 import K_NAMES
    s = w.shape
    fl = step_flops(w) * steps
    out_k = {}
    tot = float(k_ms.sum())
    for i, name in enumerate(K_NAMES):
        if k_cnt[i]:
            out_k[name] = {"launches": int(k_cnt[i]), "ms_total": float(k_ms[i]), "share": float(k_ms[i] / tot),
                           "us_per_launch": float(k_ms[i] / k_cnt[i] * 1e3)}
    for name, f in (("qkv", fl[0]), ("attn", fl[1]), ("rh", fl[2])):
        if name in out_k:
            out_k[name]["tflops"] = float(f / (k_ms[K_NAMES.index(name)] * 1e-3) / 1e12)
            out_k[name]["frac_of_sustained_bf16"] = out_k[name]["tflops"] / peaks["tf_sustained"]
    ic = K_NAMES.index("compact")
    if k_cnt[ic] and compact_bytes is not None:
        out_k["compact"]["bytes_per_launch"] = float(compact_bytes / k_cnt[ic])
        out_k["compact"]["gbs"] = float(compact_bytes / (k_ms[ic] * 1e-3) / 1e9)
        out_k["compact"]["frac_of_hbm_copy"] = out_k["compact"]["gbs"] / peaks["hbm_gbs"]
    return out_k


def sample_config(name, dev, peaks, n_layers, context, x_shared=None, weights_shared=None):
    """A short sample of another benchmark configuration, so that the line carries figures for it that
    were measured in the same run: `n_layers` layers of the stack (the layers are identical in shape
    and every layer receives the same chunk, so a pass over the whole stack costs full / n_layers times
    the sample), context cut to `context` tokens; 1 warm-up pass, 2 timed passes, 1 pass with every
    kernel on one stream for the per-kernel rates."""
    import torch
    from paper_2410_01805_b200 import K_NAMES, LocretLayer
    full = W.get_workload(name)
    w = full.with_(n_layers=n_layers, context=min(context, full.context))
    s = w.shape
    stream = torch.cuda.current_stream()
    sizes = w.chunk_sizes()
    if x_shared is not None and x_shared.shape[0] >= w.context and x_shared.shape[1] == s.d_model:
        x_dev = x_shared[:w.context]
    else:
        x_host = torch.empty((w.context, s.d_model), dtype=torch.bfloat16)
        pos = 0
        while pos < w.context:
            n_tok = min(8 * w.chunk, w.context - pos)
            x_host[pos:pos + n_tok] = torch.from_numpy(W.hidden_states(full, pos, n_tok)).to(torch.bfloat16)
            pos += n_tok
        x_dev = x_host.to(dev)
    layers = []
    for l in range(n_layers):
        if weights_shared is not None and l < len(weights_shared):
            wq, w1, w2 = weights_shared[l]
        else:
            wq, w1, w2 = (torch.from_numpy(a).to(torch.bfloat16).to(dev) for a in W.layer_weights(s, l))
        layers.append(LocretLayer(s, wq, w1, w2, w.budget, w.chunk, w.n_stab, stream=stream))
    out = torch.empty((w.chunk, s.n_q_heads * s.head_dim), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def one_pass():
        for L in layers:
            L.reset()
        p = 0
        for n_tok in sizes:
            for L in layers:
                L.prefill_chunk(x_dev[p:p + n_tok], out, 0, n_tok)
            p += n_tok

    one_pass()
    torch.cuda.synchronize()
    times = []
    for _ in range(2):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); one_pass(); b.record(stream)
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    for L in layers:
        L.set_timing(2)
    flush.zero_()
    c0 = np.sum([L.compaction_counters for L in layers], axis=0)
    one_pass()
    c1 = np.sum([L.compaction_counters for L in layers], axis=0)
    k_ms = np.zeros(len(K_NAMES)); k_cnt = np.zeros(len(K_NAMES), dtype=np.int64)
    for L in layers:
        a, c = L.read_timing(); k_ms += a; k_cnt += c
        L.set_timing(0)
    cbytes = compaction_bytes(w, int(k_cnt[K_NAMES.index("compact")]), int(c1[0] - c0[0]), int(c1[1] - c0[1]))
    status = max(abs(L.sync_status()) for L in layers)
    for L in layers:
        L.destroy()
    t_ms = float(np.mean(times))
    scale = full.n_layers / n_layers
    return {"workload": name,
            "sample": f"{n_layers} of {full.n_layers} layers, first {w.context} of {full.context} tokens, "
                      f"1 warm-up + 2 timed passes; tokens_per_s = tokens / (pass time x {scale:g})",
            "tokens_per_s": w.context / (t_ms * 1e-3 * scale), "ms_per_sampled_pass": t_ms,
            "us_per_chunk_layer": t_ms * 1e3 / (len(sizes) * n_layers),
            "tflops_step": float(step_flops(w).sum() / (t_ms * 1e-3) / 1e12),
            "frac_of_sustained_bf16": float(step_flops(w).sum() / (t_ms * 1e-3) / 1e12 / peaks["tf_sustained"]),
            "device_status": status,
            "kernels_isolated": summarise(w, k_ms, k_cnt, 1, peaks, cbytes)}


# ----------------------------------------------------------------------------- our arm

def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2410_01805_b200 import K_NAMES, LocretLayer

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    s = w.shape
    peaks = measured_peaks()

    # ---- inputs: seeded host arrays -> pinned host memory -> HBM
    sizes = w.chunk_sizes()
    t0 = time.perf_counter()
    # a stream longer than 2M tokens re-reads a ring of about 1M resident tokens (whole chunks): its
    # inputs would not fit in memory, and the kernels' time does not depend on the values
    ring = w.context if w.context <= (2 << 20) else max(1, (1 << 20) // w.chunk) * w.chunk
    x_host = torch.empty((ring, s.d_model), dtype=torch.bfloat16).pin_memory()
    pos = 0
    while pos < ring:
        n_tok = min(w.chunk, ring - pos)
        x_host[pos:pos + n_tok] = torch.from_numpy(W.hidden_states(w, pos, n_tok)).to(torch.bfloat16)
        pos += n_tok
    x_dev = x_host.to(dev, non_blocking=True)
    stream = torch.cuda.current_stream()
    layers = []
    kept_weights = []   # the first layers' weights stay on the device for the samples of the other configurations
    for l in range(w.n_layers):
        wq, w1, w2 = (torch.from_numpy(a).to(torch.bfloat16).to(dev) for a in W.layer_weights(s, l))
        layers.append(LocretLayer(s, wq, w1, w2, w.budget, w.chunk, w.n_stab, reserve=args.decode_steps,
                                  stream=stream))
        if l < OTHER_LAYERS and not args.no_other_configs:
            kept_weights.append((wq, w1, w2))
        del wq, w1, w2
    gen_s = time.perf_counter() - t0

    hd = s.n_q_heads * s.head_dim
    out = torch.empty((w.chunk, hd), dtype=torch.bfloat16, device=dev)
    out_host = torch.empty((w.chunk, hd), dtype=torch.bfloat16).pin_memory()
    x_stage = torch.empty((w.chunk, s.d_model), dtype=torch.bfloat16, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)  # > 126 MB L2

    def prefill_resident():
        for L in layers:
            L.reset()
        p = 0
        for n_tok in sizes:
            xc = x_dev[p % ring:p % ring + n_tok]
            for L in layers:
                L.prefill_chunk(xc, out, 0, n_tok)
            p += n_tok

    def prefill_e2e():
        # inputs start in pinned host memory; every chunk is copied in, the last layer's
        # attention output of every chunk is copied back
        for L in layers:
            L.reset()
        p = 0
        for n_tok in sizes:
            x_stage[:n_tok].copy_(x_host[p % ring:p % ring + n_tok], non_blocking=True)
            for L in layers:
                L.prefill_chunk(x_stage, out, 0, n_tok)
            out_host[:n_tok].copy_(out[:n_tok], non_blocking=True)
            p += n_tok

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, timing=False):
        evs = []
        for L in layers:
            L.set_timing(timing)
        for _ in range(steps):
            flush.zero_()                       # flush L2 between timed iterations
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    for _ in range(args.warmup):
        prefill_resident()
    barrier()
    launches0 = sum(L.launch_count for L in layers)
    with ClockSampler(local) as clk:
        ms = timed(prefill_resident, args.steps, timing=0 if args.no_kernel_timing else 3)
    barrier()
    launches = sum(L.launch_count for L in layers) - launches0
    k_ms = np.zeros(len(K_NAMES)); k_cnt = np.zeros(len(K_NAMES), dtype=np.int64)
    for L in layers:
        a, c = L.read_timing(); k_ms += a; k_cnt += c
        L.set_timing(False)
    status = max(abs(L.sync_status()) for L in layers)
    assert status == 0, "device status word set"

    prefill_e2e(); torch.cuda.synchronize()
    ms_e2e = timed(prefill_e2e, max(1, min(args.steps, 3)))
    barrier()

    t_ms = float(np.mean(ms)); t_e2e = float(np.mean(ms_e2e))
    t_ms, t_e2e = max_over_ranks([t_ms, t_e2e], dev)
    value = job_throughput(world, w.context, t_ms)
    e2e = job_throughput(world, w.context, t_e2e)

    # ---- per-kernel rates.  In the timed region the retaining head, selection and compaction run
    # on the library's second stream and overlap attention / the next projection, so their event
    # times (and attention's) include the time they share the SMs; one extra pass with every
    # kernel on one stream gives each kernel's rate when it runs alone.
    # live in the timed region: only the dominant kernel (attention) is bracketed with events, to
    # keep the measurement's own cost out of `value`; the full split comes from the extra pass
    ia = K_NAMES.index("attn")
    live_attn_tf = float(step_flops(w)[1] * args.steps / (k_ms[ia] * 1e-3) / 1e12) if k_cnt[ia] else 0.0
    per_kernel = {"attn": {"launches": int(k_cnt[ia]), "ms_total": float(k_ms[ia]), "tflops": live_attn_tf}}
    for L in layers:
        L.set_timing(2)
    flush.zero_()
    cc0 = np.sum([L.compaction_counters for L in layers], axis=0)
    prefill_resident()
    cc1 = np.sum([L.compaction_counters for L in layers], axis=0)
    iso_ms = np.zeros(len(K_NAMES)); iso_cnt = np.zeros(len(K_NAMES), dtype=np.int64)
    for L in layers:
        a, c = L.read_timing(); iso_ms += a; iso_cnt += c
        L.set_timing(0)
    isolated = summarise(w, iso_ms, iso_cnt, 1, peaks,
                         compaction_bytes(w, int(iso_cnt[K_NAMES.index("compact")]), int(cc1[0] - cc0[0]),
                                          int(cc1[1] - cc0[1])))
    attn_tf = per_kernel["attn"]["tflops"]
    dom = int(np.argmax(iso_ms))
    roofline = {"kernel": "attn", "bound": "tensor", "achieved": float(attn_tf), "peak": peaks["tf_sustained"],
                "unit": "TFLOP/s", "frac": float(attn_tf / peaks["tf_sustained"]),
                "frac_of_measured_sustained": float(attn_tf / peaks["tf_sustained"]),
                "frac_of_datasheet_dense_bf16": float(attn_tf / 2250.0),
                "ncu_tensor_pipe_active_pct": NCU_ATTN_TENSOR_PIPE_PCT,
                "traffic": NCU_ATTN_TRAFFIC_BYTES.get(w.name) if not (args.layers or args.context) else None,
                "traffic_unit": "bytes per steady-state launch (literal from a profiler capture of this launch shape)",
                "peak_source": f"bf16 sustained, {peaks['source']}", "dominant_by_time": K_NAMES[dom],
                "isolated": {"achieved": isolated["attn"]["tflops"],
                             "frac": isolated["attn"]["tflops"] / peaks["tf_sustained"],
                             "note": "same kernel in a pass with every kernel on one stream"}}

    # ---- decoding after the prefill (the B = 1 case): one token through every layer per step
    decode = None
    if args.decode_steps > 0:
        prefill_resident()
        xd = x_dev[:args.decode_steps]
        od = torch.empty((1, hd), dtype=torch.bfloat16, device=dev)

        from paper_2410_01805_b200 import LayerStack
        stack = LayerStack(layers)

        def decode_all():
            # one call per token: the token through every layer's attention block (every layer receives the
            # same hidden state, as in the prefill); the per-layer entry point is the same code
            for t in range(args.decode_steps):
                stack.decode_step(xd[t:t + 1], od)

        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_host = time.perf_counter()
        a.record(stream); decode_all(); b.record(stream)
        t_host = time.perf_counter() - t_host       # how long the host took to enqueue the steps
        torch.cuda.synchronize()
        dms = a.elapsed_time(b) / args.decode_steps
        ln = min(w.budget, w.context)
        kv_bytes = 2 * s.n_kv_heads * ln * s.head_dim * 2          # rotated K + V read by attention
        if s.kv_dtype == 1:   # 4-bit cache: codes of K and V, two fp16 scales and the rank per unit
            kv_bytes = s.n_kv_heads * ln * (s.head_dim + 4 + 4)
        w_bytes = 2 * (s.d_model * s.d_in + s.d_in * s.d_retain)
        step_bytes = w.n_layers * (kv_bytes + w_bytes)
        decode = {"tokens_per_s": 1e3 / dms, "ms_per_token": dms, "steps": args.decode_steps,
                  "algorithmic_gb_per_token": step_bytes / 1e9, "achieved_gbs": step_bytes / (dms * 1e-3) / 1e9,
                  "frac_of_hbm_peak": step_bytes / (dms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                  "cache_units_per_head": ln, "host_enqueue_ms_per_token": t_host * 1e3 / args.decode_steps,
                  "note": "one request, all layers per token, after the prefill; three kernels per layer-step, "
                          "overlapped by programmatic dependent launch"}

    # ---- the other benchmark configurations, sampled (rank 0 of a single-GPU run only)
    other = None
    for L in layers:
        L.destroy()
    layers = []
    if rank == 0 and world == 1 and not args.no_other_configs and not (args.layers or args.context):
        del out, x_stage
        torch.cuda.empty_cache()
        other = []
        for name in OTHER_CONFIGS:
            if name == w.name:
                continue
            share = W.get_workload(name).shape.d_model == s.d_model and W.get_workload(name).hidden == w.hidden
            same_w = W.get_workload(name).shape.d_in == s.d_in and W.get_workload(name).shape.d_retain == s.d_retain
            try:
                other.append(sample_config(name, dev, peaks, OTHER_LAYERS, OTHER_CONTEXT,
                                           x_shared=x_dev if share else None,
                                           weights_shared=kept_weights if (share and same_w) else None))
            except Exception as e:  # a sample must never take the headline down with it
                other.append({"workload": name, "error": repr(e)})
    kept_weights = []

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.n_layers, "context": w.context, "chunk": w.chunk,
                   "budget": w.budget, "n_stab": w.n_stab, "heads": f"{s.n_q_heads}q/{s.n_kv_heads}kv x {s.head_dim}",
                   "d_model": s.d_model, "d_retain": s.d_retain, "l2": "flushed between timed iterations (256 MB write)",
                   "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "attention_kernel": ("cta_pair (LOCRET_ATTN_PAIR=1, set by bench.py)"
                                        if os.environ.get("LOCRET_ATTN_PAIR") == "1" and s.head_dim == 128
                                        else "one_cta (library default)")},
        "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(w.context * s.d_model * 2),
                "d2h_bytes_per_step": int(w.context * hd * 2), "ms_per_step": t_e2e},
        "gpu_launches": int(launches),
        "clocks": clk.summary(),
        "roofline": roofline,
        "kernels": per_kernel,
        "kernels_isolated": isolated,
        "decode": decode,
        "tflops_step": float(step_flops(w).sum() / (t_ms * 1e-3) / 1e12),
        "setup_s": gen_s,
        "other_configs": other,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample, _ = oracle_sample(w, 2)  # two steady-state chunk-layers: about 15 s of host work
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- whole decoder layers

def run_whole_model(args, w):
    """Extra (not the headline metric): the same chunked prefill through whole decoder layers
    (locret_block_*: RMSNorm, attention block with eviction, W_o, gated FFN), hidden states chained
    from layer to layer.  Weights are drawn on the device (seeded torch generator, N(0, 1/fan_in)):
    the host generator would need minutes for 32 layers of FFN weights."""
    import torch
    from paper_2410_01805_b200 import LocretBlock
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    s = w.shape
    if s.d_ff <= 0:
        raise SystemExit("this workload's shape has no d_ff")
    sizes = w.chunk_sizes()
    t0 = time.perf_counter()
    x_dev = torch.empty((w.context, s.d_model), dtype=torch.bfloat16, device=dev)
    pos = 0
    for n_tok in sizes:
        x_dev[pos:pos + n_tok] = torch.from_numpy(W.hidden_states(w, pos, n_tok)).to(torch.bfloat16).to(dev)
        pos += n_tok
    g = torch.Generator(device=dev)
    g.manual_seed(W.BASE_SEED)
    hd = s.n_q_heads * s.head_dim

    def draw(rows, cols):
        return (torch.randn((rows, cols), generator=g, device=dev, dtype=torch.float32) / math.sqrt(rows)).to(torch.bfloat16)

    blocks = []
    stream = torch.cuda.current_stream()
    for l in range(w.n_layers):
        gains = [(1.0 + 0.1 * torch.randn(s.d_model, generator=g, device=dev)).to(torch.bfloat16) for _ in range(2)]
        ws = [draw(s.d_model, s.d_in), draw(s.d_in, s.d_retain), draw(s.d_retain, s.n_kv_heads),
              draw(hd, s.d_model), draw(s.d_model, s.d_ff), draw(s.d_model, s.d_ff), draw(s.d_ff, s.d_model)]
        blocks.append((LocretBlock(s, *ws, gains[0], gains[1], w.budget, w.chunk, w.n_stab, stream=stream), ws[:3]))
        del ws[3:], gains
    setup_s = time.perf_counter() - t0
    bufs = [torch.empty((w.chunk, s.d_model), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    def run():
        for b, _ in blocks:
            b.attn.reset()
        p = 0
        for n_tok in sizes:
            src = x_dev[p:p + n_tok]
            for i, (b, _) in enumerate(blocks):
                dst = bufs[i & 1]
                b.prefill_chunk(src, dst, 0, n_tok)
                src = dst
            p += n_tok

    for _ in range(args.warmup):
        run()
    torch.cuda.synchronize()
    times = []
    with ClockSampler(local) as clk:
        for _ in range(args.steps):
            flush.fill_(1)
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); run(); b_.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b_))
    # decoding through the whole layers: one token at a time, appended without eviction
    n_dec = 32
    tok = [torch.empty((1, s.d_model), dtype=torch.bfloat16, device=dev) for _ in range(2)]

    def decode_all():
        for t in range(n_dec):
            src = x_dev[t:t + 1]
            for i, (b, _) in enumerate(blocks):
                b.prefill_chunk(src, tok[i & 1], 1, 1)   # flags = NO_EVICT
                src = tok[i & 1]

    torch.cuda.synchronize()
    a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream); decode_all(); b_.record(stream)
    torch.cuda.synchronize()
    dec_ms = a.elapsed_time(b_) / n_dec
    w_bytes = 2.0 * (s.d_model * s.d_in + s.d_in * s.d_retain + hd * s.d_model + 3 * s.d_model * s.d_ff)
    kv_bytes = 2.0 * s.n_kv_heads * min(w.budget, w.context) * s.head_dim * 2
    dec_bytes = w.n_layers * (w_bytes + kv_bytes)
    peaks = measured_peaks()
    status = max(b.attn.sync_status() for b, _ in blocks)
    t_ms = float(np.mean(times))
    fl = float(step_flops(w).sum())
    extra = w.n_layers * w.context * (2.0 * hd * s.d_model + 6.0 * s.d_model * s.d_ff)
    finite = bool(torch.isfinite(bufs[(len(blocks) - 1) & 1][: sizes[-1]].float()).all().item())
    line = {
        "metric": "whole-decoder-layer chunked-prefill tokens/sec (extra; the headline metric is the attention block alone)",
        "value": w.context / (t_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic (hidden states from the seeded host generator, weights drawn on the device)",
        "config": {"workload": w.name + " + W_o, RMSNorm, gated FFN (d_ff %d), hidden states chained" % s.d_ff,
                   "layers": w.n_layers, "context": w.context, "chunk": w.chunk, "budget": w.budget,
                   "l2": "flushed between timed iterations (256 MB write)"},
        "tflops_step": (fl + extra) / (t_ms * 1e-3) / 1e12, "flops_attention_block": fl, "flops_rest_of_layer": extra,
        "decode": {"tokens_per_s": 1e3 / dec_ms, "ms_per_token": dec_ms, "steps": n_dec,
                   "algorithmic_gb_per_token": dec_bytes / 1e9, "achieved_gbs": dec_bytes / (dec_ms * 1e-3) / 1e9,
                   "frac_of_hbm_peak": dec_bytes / (dec_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "device_status": status, "outputs_finite": finite, "clocks": clk.summary(), "setup_s": setup_s,
    }
    if rank == 0:
        print(json.dumps(line))
    for b, _ in blocks:
        b.destroy()


def run_cis(args, w):
    """Extra: the training labels of Section 3.3 (locret_cis_labels) at the workload's layer shape,
    131072 prompt tokens and 1024 answer tokens, one layer."""
    import torch
    from paper_2410_01805_b200 import cis_labels
    torch.cuda.set_device(0)
    s = w.shape
    n_q, n_a = w.context, 1024
    g = torch.Generator(device="cuda"); g.manual_seed(W.BASE_SEED)
    q = torch.randn((n_a, s.n_q_heads, s.head_dim), generator=g, device="cuda").to(torch.bfloat16)
    k = torch.randn((n_q, s.n_kv_heads, s.head_dim), generator=g, device="cuda").to(torch.bfloat16)
    for _ in range(args.warmup):
        cis_labels(q, k)
    ts = []
    for _ in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); out = cis_labels(q, k); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = float(np.mean(ts))
    flops = 2.0 * n_q * n_a * s.n_q_heads * s.head_dim
    # loss and gradients of the retaining head (Eq. 2, Eq. 3) for one sequence of the paper's training length
    from paper_2410_01805_b200 import rh_loss_grad
    n_tr = 10240
    z = torch.randn((n_tr, s.d_in), generator=g, device="cuda").to(torch.bfloat16)
    w1 = (torch.randn((s.d_in, s.d_retain), generator=g, device="cuda") / math.sqrt(s.d_in)).to(torch.bfloat16)
    w2 = (torch.randn((s.d_retain, s.n_kv_heads), generator=g, device="cuda") / math.sqrt(s.d_retain)).to(torch.bfloat16)
    lab = torch.randn((s.n_kv_heads, n_tr), generator=g, device="cuda")
    for _ in range(args.warmup):
        rh_loss_grad(z, lab, w1, w2)
    tt = []
    for _ in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); loss, g1, g2 = rh_loss_grad(z, lab, w1, w2); b.record()
        torch.cuda.synchronize()
        tt.append(a.elapsed_time(b))
    ms_tr = float(np.mean(tt))
    fl_tr = 4.0 * n_tr * s.d_in * s.d_retain
    print(json.dumps({"metric": "training labels (Section 3.3), one layer", "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                      "config": {"n_prompt": n_q, "n_answer": n_a, "heads": f"{s.n_q_heads}q/{s.n_kv_heads}kv x {s.head_dim}"},
                      "finite": bool(torch.isfinite(out).all().item()),
                      "loss_and_gradients": {"ms": ms_tr, "tflops": fl_tr / (ms_tr * 1e-3) / 1e12, "n_tokens": n_tr,
                                             "note": "Eq. 2/3 for one sequence and one layer, workspace allocated inside the call",
                                             "finite": bool(torch.isfinite(g1).all().item() and torch.isfinite(loss).item())}}))


def run_tp(args, w):
    """Extra: the step with the KV heads divided over GPUs (locret_prefill_chunk_tp_begin / _finish
    around one all-reduce per chunk-layer).  Under torchrun every rank holds its heads of every layer
    and the exchange is NCCL's all-reduce (total work fixed: strong scaling).  In a single process it
    times ONE rank's share at degree --tp with no exchange, and says so."""
    import torch
    from paper_2410_01805_b200 import LocretLayerTP
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    multi = world > 1
    if multi:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    degree = world if multi else args.tp
    s = w.shape
    if s.n_kv_heads % degree:
        raise SystemExit(f"--tp {degree} does not divide {s.n_kv_heads} KV heads")
    g = torch.Generator(device=dev); g.manual_seed(W.BASE_SEED)

    def mat(rows, cols):
        return (torch.randn((rows, cols), generator=g, device=dev, dtype=torch.float32) / math.sqrt(rows)).to(torch.bfloat16)

    layers = []
    for _ in range(w.n_layers):
        full = (mat(s.d_model, s.d_in), mat(s.d_in, s.d_retain), mat(s.d_retain, s.n_kv_heads))
        layers.append(LocretLayerTP(s, *full, w.budget, w.chunk, w.n_stab, rank if multi else 0, degree,
                                    reduce=None if multi else (lambda t: None)))
        del full
    sizes = w.chunk_sizes()
    x = torch.randn((w.chunk, s.d_model), generator=g, device=dev).to(torch.bfloat16)
    out = torch.zeros((w.chunk, (s.n_q_heads // degree) * s.head_dim), dtype=torch.bfloat16, device=dev)

    def one_pass():
        for L in layers:
            L.layer.reset()
        for n_tok in sizes:
            for L in layers:
                L.prefill_chunk(x[:n_tok], out, 0, n_tok)

    for _ in range(max(1, args.warmup)):
        one_pass()
    torch.cuda.synchronize()
    ts = []
    for _ in range(args.steps):
        if multi:
            dist.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); one_pass(); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b))
    ms = float(np.mean(ts))
    if multi:
        t = torch.tensor([ms], device=dev); dist.all_reduce(t, op=dist.ReduceOp.MAX); ms = float(t.item())
    status = max(abs(L.layer.sync_status()) for L in layers)
    exch = w.chunk * s.d_retain * 4
    if rank == 0:
        print(json.dumps({
            "metric": "prefill tokens/s, KV heads divided over GPUs" if multi else
                      "one rank's share of the divided step (no exchange timed)",
            "value": w.context / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world, "tp_degree": degree,
            "ms_per_step": ms, "steps": args.steps, "warmup": max(1, args.warmup), "scaling": "strong",
            "status": status, "data": "synthetic (device-generated weights and hidden states)",
            "config": {"workload": w.name, "layers": w.n_layers, "heads_per_rank": f"{s.n_q_heads // degree}q/{s.n_kv_heads // degree}kv",
                       "exchange": f"all-reduce of {exch / 1e6:.1f} MB fp32 per chunk-layer" + ("" if multi else " (not run: single process)")}}))
    if multi:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tp", type=int, default=0,
                    help="extra run: KV heads divided over GPUs (degree = world size under torchrun, else this value)")
    ap.add_argument("--cis", action="store_true", help="extra run: the training labels of Section 3.3")
    ap.add_argument("--whole-model", action="store_true",
                    help="extra run: whole decoder layers (attention block + W_o + gated FFN), hidden states chained")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(W.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling only)")
    ap.add_argument("--context", type=int, default=0, help="override the context length (profiling only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short samples of the other benchmark configurations")
    ap.add_argument("--no-kernel-timing", action="store_true",
                    help="do not bracket kernels with events in the timed region (to measure that overhead)")
    ap.add_argument("--decode-steps", type=int, default=256, help="decode steps timed after the prefill (0 = none)")
    args = ap.parse_args()
    w = W.get_workload(args.workload)
    if args.layers:
        w = w.with_(n_layers=args.layers)
    if args.context:
        w = w.with_(context=args.context)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        import __graft_entry__ as G
        G.build()
        if args.tp:
            run_tp(args, w)
        elif args.cis:
            run_cis(args, w)
        elif args.whole_model:
            run_whole_model(args, w)
        else:
            run_ours(args, w)


if __name__ == "__main__":
    main()
