"""ctypes binding with the same names as the C ABI in include/locret.h."""

from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
lib_path = os.path.join(_HERE, "liblocret.so")

NO_EVICT = 1
LAST_CHUNK = 2
K_NAMES = ["qkv", "rope", "attn", "rh", "rh_reduce", "topk", "compact", "dequant", "quant"]


class LocretError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {lib.locret_strerror(code).decode()} ({code})")


class locret_layer_cfg(C.Structure):
    _fields_ = [
        ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("d_retain", C.c_int32), ("act", C.c_int32),
        ("rope_theta", C.c_float), ("rh_input", C.c_int32), ("kv_dtype", C.c_int32),
        ("reserve", C.c_int32),
        ("w_qkv", C.c_void_p), ("w1", C.c_void_p), ("w2", C.c_void_p), ("stream", C.c_void_p),
    ]


class locret_block_cfg(C.Structure):
    _fields_ = [
        ("attn", locret_layer_cfg), ("d_ff", C.c_int32), ("rms_eps", C.c_float),
        ("w_o", C.c_void_p), ("w_gate", C.c_void_p), ("w_up", C.c_void_p), ("w_down", C.c_void_p),
        ("g1", C.c_void_p), ("g2", C.c_void_p),
    ]


def _load():
    if not os.path.exists(lib_path):
        raise ImportError(
            f"{lib_path} is missing: build it with `python paper_2410_01805_b200/build.py` "
            "(there is no CPU fallback)")
    l = C.CDLL(lib_path)
    P = C.c_void_p
    l.locret_strerror.restype = C.c_char_p
    l.locret_strerror.argtypes = [C.c_int]
    l.locret_create.argtypes = [C.POINTER(locret_layer_cfg), C.c_int32, C.c_int32, C.c_int32, C.POINTER(P)]
    l.locret_prefill_chunk.argtypes = [P, P, C.c_int32, C.c_uint32, P]
    l.locret_decode_step.argtypes = [P, P, P]
    l.locret_decode_step_stack.argtypes = [P, C.c_int32, P, P, C.c_int64]
    l.locret_prefill_chunk_tp_begin.argtypes = [P, P, C.c_int32, C.c_uint32, P, P]
    l.locret_prefill_chunk_tp_finish.argtypes = [P, P]
    l.locret_tp_set_peers.argtypes = [P, P, C.c_int32]
    l.locret_prefill_chunk_tp_begin_peers.argtypes = [P, P, C.c_int32, C.c_uint32, P]
    l.locret_cache_len.argtypes = [P, C.POINTER(C.c_int32)]
    l.locret_export_state.argtypes = [P, P, P, P, P, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    l.locret_import_state.argtypes = [P, P, P, P, P, C.c_int32, C.c_int64]
    l.locret_export_state_int4.argtypes = [P, P, P, P, P, P, P, C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    l.locret_import_state_int4.argtypes = [P, P, P, P, P, P, P, C.c_int32, C.c_int64]
    l.locret_selftest_wait_timeout.argtypes = [P]
    l.locret_sync_status.argtypes = [P]
    l.locret_reset.argtypes = [P]
    l.locret_set_protected_prefix.argtypes = [P, C.c_int32]
    l.locret_set_timing.argtypes = [P, C.c_int32]
    l.locret_read_timing.argtypes = [P, P, P]
    l.locret_launch_count.argtypes = [P, C.POINTER(C.c_int64)]
    l.locret_compaction_counters.argtypes = [P, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    l.locret_set_head_budgets.argtypes = [P, P]
    l.locret_cache_lens.argtypes = [P, P]
    l.locret_export_state_heads.argtypes = [P, P, P, P, P, C.c_int32, P, C.POINTER(C.c_int64)]
    l.locret_import_state_heads.argtypes = [P, P, P, P, P, C.c_int32, P, C.c_int64]
    l.locret_rh_scores_static.argtypes = [P, C.c_int32, C.c_int32, P, C.c_int32, P, C.c_int32, C.c_int32, P, P, P]
    l.locret_selftest_wait_abort.argtypes = [P, P]
    l.locret_destroy.argtypes = [P]
    l.locret_destroy.restype = None
    l.locret_block_create.argtypes = [C.POINTER(locret_block_cfg), C.c_int32, C.c_int32, C.c_int32, C.POINTER(P)]
    l.locret_block_prefill_chunk.argtypes = [P, P, C.c_int32, C.c_uint32, P]
    l.locret_block_attention.argtypes = [P]
    l.locret_block_attention.restype = P
    l.locret_block_destroy.argtypes = [P]
    l.locret_block_destroy.restype = None
    l.locret_rh_loss_grad.argtypes = [P, P, P, P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, P, P, P, P]
    l.locret_adamw_step.argtypes = [P, P, P, P, P, C.c_int64, C.c_int32, C.c_float, C.c_float, C.c_float, C.c_float, C.c_float, P]
    l.locret_cis_labels.argtypes = [P, P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, P, P]
    return l


lib = _load()


def _check(code: int, what: str):
    if code != 0:
        raise LocretError(code, what)


def _bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy()


class LocretLayer:
    """One decoder layer's state; methods mirror the C entry points one to one."""

    def __init__(self, shape, w_qkv: torch.Tensor, w1: torch.Tensor, w2: torch.Tensor,
                 budget: int, chunk: int, n_stab: int, reserve: int = 0, stream=None):
        for w in (w_qkv, w1, w2):
            if not (w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()):
                raise ValueError("weights must be contiguous CUDA bfloat16 tensors")
        self.shape = shape
        self.h, self.h_kv, self.d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
        self.chunk, self.budget, self.n_stab = chunk, budget, n_stab
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        cfg = locret_layer_cfg(
            shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_retain,
            shape.act, float(shape.rope_theta), shape.rh_input, shape.kv_dtype, reserve,
            w_qkv.data_ptr(), w1.data_ptr(), w2.data_ptr(), self.stream.cuda_stream)
        self._h = C.c_void_p()
        _check(lib.locret_create(C.byref(cfg), budget, chunk, n_stab, C.byref(self._h)), "locret_create")

    # -- the hot path
    def prefill_chunk(self, hidden_in: torch.Tensor, attn_out: torch.Tensor, flags: int = 0,
                      n_tok: int | None = None):
        n_tok = hidden_in.shape[0] if n_tok is None else n_tok
        _check(lib.locret_prefill_chunk(self._h, hidden_in.data_ptr(), n_tok, flags,
                                        attn_out.data_ptr()), "locret_prefill_chunk")

    def decode_step(self, hidden_in: torch.Tensor, attn_out: torch.Tensor):
        _check(lib.locret_decode_step(self._h, hidden_in.data_ptr(), attn_out.data_ptr()),
               "locret_decode_step")

    # -- the same step with the heads divided over GPUs (this object holds one GPU's heads)
    def prefill_chunk_tp_begin(self, hidden_in: torch.Tensor, attn_out: torch.Tensor,
                               preact_partial: torch.Tensor, flags: int = 0, n_tok: int | None = None):
        n_tok = hidden_in.shape[0] if n_tok is None else n_tok
        if not (preact_partial.is_cuda and preact_partial.dtype == torch.float32 and preact_partial.is_contiguous()
                and preact_partial.numel() >= n_tok * self.shape.d_retain):
            raise ValueError("preact_partial must be a contiguous CUDA float32 tensor of n_tok x d_retain")
        _check(lib.locret_prefill_chunk_tp_begin(self._h, hidden_in.data_ptr(), n_tok, flags, attn_out.data_ptr(),
                                                 preact_partial.data_ptr()), "locret_prefill_chunk_tp_begin")

    def tp_set_peers(self, peer_sums):
        """peer_sums: float32 CUDA tensors [chunk, d_retain], one per GPU (this GPU's among them)."""
        arr = (C.c_void_p * len(peer_sums))(*[t.data_ptr() for t in peer_sums])
        _check(lib.locret_tp_set_peers(self._h, arr, len(peer_sums)), "locret_tp_set_peers")

    def prefill_chunk_tp_begin_peers(self, hidden_in: torch.Tensor, attn_out: torch.Tensor, flags: int = 0,
                                     n_tok: int | None = None):
        n_tok = hidden_in.shape[0] if n_tok is None else n_tok
        _check(lib.locret_prefill_chunk_tp_begin_peers(self._h, hidden_in.data_ptr(), n_tok, flags,
                                                       attn_out.data_ptr()), "locret_prefill_chunk_tp_begin_peers")

    def prefill_chunk_tp_finish(self, preact_sum: torch.Tensor):
        if not (preact_sum.is_cuda and preact_sum.dtype == torch.float32 and preact_sum.is_contiguous()):
            raise ValueError("preact_sum must be a contiguous CUDA float32 tensor")
        _check(lib.locret_prefill_chunk_tp_finish(self._h, preact_sum.data_ptr()), "locret_prefill_chunk_tp_finish")

    # -- state
    @property
    def cache_len(self) -> int:
        n = C.c_int32()
        _check(lib.locret_cache_len(self._h, C.byref(n)), "locret_cache_len")
        return n.value

    def export_state(self):
        """dict(K, V [h_kv, len, d] float32 holding bf16 values; S [h_kv, len]; T int64; seen).

        For a 4-bit cache: Kc, Vc int8 codes [h_kv, len, d], Ks, Vs float32 scales [h_kv, len],
        and K, V = codes * scales."""
        n = self.cache_len
        if self.shape.kv_dtype == 1:
            return self._export_int4(n)
        K = torch.empty((self.h_kv, n, self.d), dtype=torch.bfloat16)
        V = torch.empty_like(K)
        S = np.empty((self.h_kv, n), dtype=np.float32)
        T = np.empty((self.h_kv, n), dtype=np.int64)
        ln, seen = C.c_int32(), C.c_int64()
        _check(lib.locret_export_state(self._h, K.data_ptr(), V.data_ptr(), S.ctypes.data,
                                       T.ctypes.data, C.byref(ln), C.byref(seen)), "locret_export_state")
        return dict(K=K.float().numpy(), V=V.float().numpy(), S=S, T=T, seen=seen.value)

    def _export_int4(self, n):
        half = self.d // 2
        kc = np.empty((self.h_kv, n, half), dtype=np.uint8); vc = np.empty_like(kc)
        ks = np.empty((self.h_kv, n), dtype=np.float16); vs = np.empty_like(ks)
        S = np.empty((self.h_kv, n), dtype=np.float32)
        T = np.empty((self.h_kv, n), dtype=np.int64)
        ln, seen = C.c_int32(), C.c_int64()
        _check(lib.locret_export_state_int4(self._h, kc.ctypes.data, ks.ctypes.data, vc.ctypes.data,
                                            vs.ctypes.data, S.ctypes.data, T.ctypes.data,
                                            C.byref(ln), C.byref(seen)), "locret_export_state_int4")

        def unpack(b):
            lo = (b & 0xF).astype(np.int8); hi = (b >> 4).astype(np.int8)
            lo = np.where(lo > 7, lo - 16, lo); hi = np.where(hi > 7, hi - 16, hi)
            return np.stack([lo, hi], axis=-1).reshape(b.shape[0], b.shape[1], -1).astype(np.int8)

        Kc, Vc = unpack(kc), unpack(vc)
        Ks, Vs = ks.astype(np.float32), vs.astype(np.float32)
        return dict(Kc=Kc, Vc=Vc, Ks=Ks, Vs=Vs, K=Kc * Ks[..., None], V=Vc * Vs[..., None],
                    S=S, T=T, seen=seen.value)

    def import_state_int4(self, Kc, Ks, Vc, Vs, S, T, seen: int):
        """Codes int8 [h_kv, len, d] in [-8, 7]; scales [h_kv, len] (values exact in fp16)."""
        def pack(c):
            c = np.ascontiguousarray(c).astype(np.int16) & 0xF
            return np.ascontiguousarray((c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8))

        kc, vc = pack(Kc), pack(Vc)
        ks = np.ascontiguousarray(Ks, dtype=np.float16); vs = np.ascontiguousarray(Vs, dtype=np.float16)
        Sb = np.ascontiguousarray(S, dtype=np.float32); Tb = np.ascontiguousarray(T, dtype=np.int64)
        _check(lib.locret_import_state_int4(self._h, kc.ctypes.data, ks.ctypes.data, vc.ctypes.data,
                                            vs.ctypes.data, Sb.ctypes.data, Tb.ctypes.data,
                                            kc.shape[1], int(seen)), "locret_import_state_int4")

    def import_state(self, K, V, S, T, seen: int):
        Kb = torch.from_numpy(np.ascontiguousarray(K, dtype=np.float32)).to(torch.bfloat16).contiguous()
        Vb = torch.from_numpy(np.ascontiguousarray(V, dtype=np.float32)).to(torch.bfloat16).contiguous()
        Sb = np.ascontiguousarray(S, dtype=np.float32)
        Tb = np.ascontiguousarray(T, dtype=np.int64)
        n = Kb.shape[1]
        _check(lib.locret_import_state(self._h, Kb.data_ptr(), Vb.data_ptr(), Sb.ctypes.data,
                                       Tb.ctypes.data, n, int(seen)), "locret_import_state")

    # -- a budget per KV head
    def set_head_budgets(self, budgets):
        b = np.ascontiguousarray(budgets, dtype=np.int32)
        if b.shape != (self.h_kv,):
            raise ValueError("one budget per KV head")
        _check(lib.locret_set_head_budgets(self._h, b.ctypes.data), "locret_set_head_budgets")

    @property
    def cache_lens(self):
        lens = np.zeros(self.h_kv, dtype=np.int32)
        _check(lib.locret_cache_lens(self._h, lens.ctypes.data), "locret_cache_lens")
        return lens.tolist()

    def export_state_heads(self):
        """dict(K, V: lists of [len_m, d] float32 arrays; S, T: lists of [len_m]; seen)."""
        lens = self.cache_lens
        pitch = max(max(lens), 1)
        K = torch.zeros((self.h_kv, pitch, self.d), dtype=torch.bfloat16)
        V = torch.zeros_like(K)
        S = np.zeros((self.h_kv, pitch), dtype=np.float32)
        T = np.zeros((self.h_kv, pitch), dtype=np.int64)
        out_lens = np.zeros(self.h_kv, dtype=np.int32)
        seen = C.c_int64()
        _check(lib.locret_export_state_heads(self._h, K.data_ptr(), V.data_ptr(), S.ctypes.data, T.ctypes.data, pitch,
                                             out_lens.ctypes.data, C.byref(seen)), "locret_export_state_heads")
        Kf, Vf = K.float().numpy(), V.float().numpy()
        return dict(K=[Kf[m, :n] for m, n in enumerate(out_lens)], V=[Vf[m, :n] for m, n in enumerate(out_lens)],
                    S=[S[m, :n] for m, n in enumerate(out_lens)], T=[T[m, :n] for m, n in enumerate(out_lens)],
                    seen=seen.value)

    def import_state_heads(self, K, V, S, T, seen: int):
        lens = np.array([len(t) for t in T], dtype=np.int32)
        pitch = max(int(lens.max()), 1)
        Kb = torch.zeros((self.h_kv, pitch, self.d), dtype=torch.bfloat16)
        Vb = torch.zeros_like(Kb)
        Sb = np.zeros((self.h_kv, pitch), dtype=np.float32)
        Tb = np.zeros((self.h_kv, pitch), dtype=np.int64)
        for m, n in enumerate(lens):
            if n:
                Kb[m, :n] = torch.from_numpy(np.ascontiguousarray(K[m], dtype=np.float32)).to(torch.bfloat16)
                Vb[m, :n] = torch.from_numpy(np.ascontiguousarray(V[m], dtype=np.float32)).to(torch.bfloat16)
                Sb[m, :n] = S[m]
                Tb[m, :n] = T[m]
        _check(lib.locret_import_state_heads(self._h, Kb.data_ptr(), Vb.data_ptr(), Sb.ctypes.data, Tb.ctypes.data, pitch,
                                             lens.ctypes.data, int(seen)), "locret_import_state_heads")

    def sync_status(self) -> int:
        return lib.locret_sync_status(self._h)

    def reset(self):
        _check(lib.locret_reset(self._h), "locret_reset")

    # -- measurement
    def set_protected_prefix(self, n_prefix: int):
        _check(lib.locret_set_protected_prefix(self._h, int(n_prefix)), "locret_set_protected_prefix")

    def set_timing(self, mode):
        """0 off, 1 time every kernel, 2 time every kernel and run them on one stream, 3 time attention only."""
        _check(lib.locret_set_timing(self._h, int(mode)), "locret_set_timing")

    def read_timing(self):
        ms = np.zeros(len(K_NAMES), dtype=np.float32)
        cnt = np.zeros(len(K_NAMES), dtype=np.int64)
        _check(lib.locret_read_timing(self._h, ms.ctypes.data, cnt.ctypes.data), "locret_read_timing")
        return ms, cnt

    @property
    def launch_count(self) -> int:
        n = C.c_int64()
        _check(lib.locret_launch_count(self._h, C.byref(n)), "locret_launch_count")
        return n.value

    @property
    def compaction_counters(self):
        """(units moved to another slot, rotated keys rewritten) by this layer's evictions since create."""
        a, b = C.c_int64(), C.c_int64()
        _check(lib.locret_compaction_counters(self._h, C.byref(a), C.byref(b)), "locret_compaction_counters")
        return a.value, b.value

    def destroy(self):
        if self._h:
            lib.locret_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class LayerStack:
    """Handles of several layers as one C array, for locret_decode_step_stack."""

    def __init__(self, layers):
        self.layers = list(layers)
        self._arr = (C.c_void_p * len(self.layers))(*[L._h.value for L in self.layers])

    def decode_step(self, hidden_in: torch.Tensor, attn_out: torch.Tensor, out_stride: int = 0):
        _check(lib.locret_decode_step_stack(self._arr, len(self.layers), hidden_in.data_ptr(), attn_out.data_ptr(),
                                            int(out_stride)), "locret_decode_step_stack")


def shard_by_kv_head(w_qkv: torch.Tensor, w1: torch.Tensor, w2: torch.Tensor, n_q_heads: int,
                     n_kv_heads: int, head_dim: int, rank: int, world: int):
    """One GPU's slices of a layer's weights when KV heads [rank * n_kv_heads / world, ...) and the
    query heads of their groups live on it: columns of w_qkv, the matching rows of w1 (local query
    heads, local key heads, local value heads, in that order), the matching columns of w2."""
    if n_kv_heads % world or not 0 <= rank < world:
        raise ValueError("n_kv_heads must divide evenly over the GPUs")
    g, hk = n_q_heads // n_kv_heads, n_kv_heads // world
    d = head_dim
    q0, k0, v0 = rank * hk * g * d, (n_q_heads + rank * hk) * d, (n_q_heads + n_kv_heads + rank * hk) * d
    idx = torch.cat([torch.arange(q0, q0 + hk * g * d), torch.arange(k0, k0 + hk * d),
                     torch.arange(v0, v0 + hk * d)]).to(w_qkv.device)
    return (w_qkv.index_select(1, idx).contiguous(), w1.index_select(0, idx).contiguous(),
            w2[:, rank * hk:(rank + 1) * hk].contiguous())


class LocretLayerTP:
    """A layer whose heads are divided over the ranks of a process group, one rank per GPU.

    Each rank holds the cache of its own KV heads; a step is the library's begin call, one
    all-reduce (sum) of the [n_tok x d_retain] float32 partial products on the current stream,
    and the library's finish call.  The layer's stream must be torch's current stream when a step
    is issued, so that the collective is ordered between the two calls.  ``reduce`` replaces the
    all-reduce (a callable that sums the tensor in place across the ranks)."""

    def __init__(self, shape, w_qkv, w1, w2, budget: int, chunk: int, n_stab: int, rank: int, world: int,
                 reserve: int = 0, group=None, reduce=None, stream=None):
        from dataclasses import replace
        wq, wa, wb = shard_by_kv_head(w_qkv, w1, w2, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                      rank, world)
        self.rank, self.world = rank, world
        self.local_shape = replace(shape, n_q_heads=shape.n_q_heads // world,
                                   n_kv_heads=shape.n_kv_heads // world)
        self._weights = (wq, wa, wb)  # the library borrows them
        self.layer = LocretLayer(self.local_shape, wq, wa, wb, budget, chunk, n_stab, reserve, stream)
        self.preact = torch.empty(chunk, shape.d_retain, dtype=torch.float32, device=wq.device)
        if reduce is None:
            import torch.distributed as dist

            def reduce(t, _g=group):
                dist.all_reduce(t, op=dist.ReduceOp.SUM, group=_g)
        self._reduce = reduce

    def prefill_chunk(self, hidden_in: torch.Tensor, attn_out_local: torch.Tensor, flags: int = 0,
                      n_tok: int | None = None):
        """attn_out_local: bf16 [n_tok x (n_q_heads / world) * head_dim], this rank's heads."""
        n_tok = hidden_in.shape[0] if n_tok is None else n_tok
        pre = self.preact[:n_tok]
        self.layer.prefill_chunk_tp_begin(hidden_in, attn_out_local, pre, flags, n_tok)
        self._reduce(pre)
        self.layer.prefill_chunk_tp_finish(pre)

    def destroy(self):
        self.layer.destroy()


class LocretBlock:
    """A whole decoder layer (RMSNorm, attention block with eviction, W_o, gated FFN); methods
    mirror the locret_block_* entry points.  `attn` is the block's attention layer (owned by the
    block), with the state / status / timing methods of LocretLayer."""

    def __init__(self, shape, w_qkv, w1, w2, w_o, w_gate, w_up, w_down, g1, g2,
                 budget: int, chunk: int, n_stab: int, reserve: int = 0, rms_eps: float = 1e-5, stream=None):
        for w in (w_qkv, w1, w2, w_o, w_gate, w_up, w_down, g1, g2):
            if not (w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()):
                raise ValueError("weights must be contiguous CUDA bfloat16 tensors")
        self.shape, self.chunk = shape, chunk
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        cfg = locret_block_cfg(
            locret_layer_cfg(
                shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_retain,
                shape.act, float(shape.rope_theta), shape.rh_input, shape.kv_dtype, reserve,
                w_qkv.data_ptr(), w1.data_ptr(), w2.data_ptr(), self.stream.cuda_stream),
            shape.d_ff, float(rms_eps), w_o.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr(),
            g1.data_ptr(), g2.data_ptr())
        self._b = C.c_void_p()
        _check(lib.locret_block_create(C.byref(cfg), budget, chunk, n_stab, C.byref(self._b)), "locret_block_create")
        # a non-owning view of the attention layer
        self.attn = LocretLayer.__new__(LocretLayer)
        self.attn.shape = shape
        self.attn.h, self.attn.h_kv, self.attn.d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
        self.attn.chunk, self.attn.budget, self.attn.n_stab = chunk, budget, n_stab
        self.attn.stream = self.stream
        self.attn._h = C.c_void_p(lib.locret_block_attention(self._b))
        self.attn.destroy = lambda: None

    def prefill_chunk(self, x_in: torch.Tensor, y_out: torch.Tensor, flags: int = 0, n_tok: int | None = None):
        n_tok = x_in.shape[0] if n_tok is None else n_tok
        _check(lib.locret_block_prefill_chunk(self._b, x_in.data_ptr(), n_tok, flags, y_out.data_ptr()),
               "locret_block_prefill_chunk")

    def destroy(self):
        if self._b:
            self.attn._h = C.c_void_p()
            lib.locret_block_destroy(self._b)
            self._b = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def cis_labels(q_ans: torch.Tensor, k_prompt: torch.Tensor, scale: float = 1.0) -> torch.Tensor:
    """Training labels (Section 3.3): q_ans [n_a, h, d], k_prompt [n_q, h_kv, d] (CUDA bf16,
    contiguous) -> fp32 [h_kv, n_q]."""
    n_a, h, d = q_ans.shape
    n_q, h_kv, _ = k_prompt.shape
    out = torch.empty((h_kv, n_q), dtype=torch.float32, device=q_ans.device)
    _check(lib.locret_cis_labels(q_ans.data_ptr(), k_prompt.data_ptr(), n_a, n_q, h, h_kv, d, float(scale),
                                 out.data_ptr(), torch.cuda.current_stream().cuda_stream), "locret_cis_labels")
    return out


def rh_loss_grad(z: torch.Tensor, labels: torch.Tensor, w1: torch.Tensor, w2: torch.Tensor, alpha: float = 2.5e-3):
    """Eq. 2 / Eq. 3 for one sequence: z [n, d_in] bf16, labels [h_kv, n] fp32, w1 [d_in, d_R], w2 [d_R, h_kv]
    bf16 (CUDA, contiguous) -> (loss fp32 scalar tensor, d_w1 fp32 [d_in, d_R], d_w2 fp32 [d_R, h_kv])."""
    n, d_in = z.shape
    d_R, h_kv = w2.shape
    loss = torch.empty((), dtype=torch.float32, device=z.device)
    d_w1 = torch.empty((d_in, d_R), dtype=torch.float32, device=z.device)
    d_w2 = torch.empty((d_R, h_kv), dtype=torch.float32, device=z.device)
    _check(lib.locret_rh_loss_grad(z.data_ptr(), labels.data_ptr(), w1.data_ptr(), w2.data_ptr(), n, d_in, d_R, h_kv,
                                   float(alpha), loss.data_ptr(), d_w1.data_ptr(), d_w2.data_ptr(),
                                   torch.cuda.current_stream().cuda_stream), "locret_rh_loss_grad")
    return loss, d_w1, d_w2


def adamw_step(param: torch.Tensor, grad: torch.Tensor, m: torch.Tensor, v: torch.Tensor, step: int, lr: float,
               param_bf16: torch.Tensor | None = None, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
               weight_decay: float = 0.01):
    """In-place AdamW update of a contiguous fp32 CUDA tensor (and its bf16 copy, if given)."""
    _check(lib.locret_adamw_step(param.data_ptr(), param_bf16.data_ptr() if param_bf16 is not None else None,
                                 grad.data_ptr(), m.data_ptr(), v.data_ptr(), param.numel(), int(step), float(lr),
                                 float(beta1), float(beta2), float(eps), float(weight_decay),
                                 torch.cuda.current_stream().cuda_stream), "locret_adamw_step")
