"""Shape table of the synthetic workloads.

Each workload is a stack of identical decoder-layer attention blocks (random
weights) fed a seeded synthetic hidden-state stream in chunks, with the
eviction hyper-parameters of the paper's Table 4 notation: budget ``b``, chunk
size ``B``, stabilizer length ``n_s``.
"""

from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class LayerShape:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_retain: int
    rope_theta: float = 10000.0
    act: int = 0          # 0 SiLU, 1 GELU(tanh), 2 ReLU
    rh_input: int = 0     # 0: retaining head sees pre-RoPE [Q;K;V], 1: post-RoPE Q,K
    kv_dtype: int = 0     # 0 bf16 cache, 1 int4 (group = head vector) + fp16 scale
    d_ff: int = 0         # hidden size of the gated FFN that closes the decoder layer (0: none given)

    @property
    def d_in(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass(frozen=True)
class Workload:
    name: str
    shape: LayerShape
    n_layers: int
    context: int
    chunk: int
    budget: int
    n_stab: int
    hidden: str            # "normal" | "outlier" | "topics"
    decode_steps: int = 0
    note: str = ""

    def chunk_sizes(self):
        full, rem = divmod(self.context, self.chunk)
        return [self.chunk] * full + ([rem] if rem else [])

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_LLAMA = LayerShape(d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                    d_retain=1024, rope_theta=500000.0, d_ff=14336)
_PHI3 = LayerShape(d_model=3072, n_q_heads=32, n_kv_heads=32, head_dim=96,
                   d_retain=1024, rope_theta=10000.0, d_ff=8192)

CONFIGS = {
    # configs[0]: the small case the oracle runs in full within seconds.
    "c1_small_gqa": Workload(
        "c1_small_gqa",
        LayerShape(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, d_retain=256, d_ff=1536),
        n_layers=1, context=4096, chunk=512, budget=1024, n_stab=64, hidden="normal"),
    # configs[1]
    "c2_llama_32k": Workload(
        "c2_llama_32k", _LLAMA, n_layers=32, context=32768, chunk=3072,
        budget=6000, n_stab=128, hidden="outlier"),
    # configs[2]: the headline run.
    "c3_llama_128k": Workload(
        "c3_llama_128k", _LLAMA, n_layers=32, context=131072, chunk=3072,
        budget=6000, n_stab=2500, hidden="outlier"),
    # configs[3]
    "c4_phi3_128k": Workload(
        "c4_phi3_128k", _PHI3, n_layers=32, context=131072, chunk=1024,
        budget=16384, n_stab=1024, hidden="topics"),
    # configs[4]: streaming, int4 cache, then decode.
    "c5_llama_stream_int4": Workload(
        "c5_llama_stream_int4", replace(_LLAMA, kv_dtype=1), n_layers=32,
        context=1_000_000, chunk=3072, budget=6000, n_stab=2500,
        hidden="outlier", decode_steps=256),
    # extra (not one of the five benchmark configurations): a soak run, 10M tokens in chunks of 10240
    "x_llama_10m_stream": Workload(
        "x_llama_10m_stream", _LLAMA, n_layers=32, context=10_000_000 // 10240 * 10240, chunk=10240,
        budget=6000, n_stab=2500, hidden="outlier"),
}


def get_workload(name: str) -> Workload:
    return CONFIGS[name]
