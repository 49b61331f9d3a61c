"""Seeded input generators shared by the oracle's tests and the CUDA path.

Every array is a pure function of (seed, stream id, block index): the draws
come from numpy's counter-based Philox generator keyed by those integers, so a
token's hidden state does not depend on how the context is cut into chunks.
Values are returned as float32 that are exactly representable in bfloat16
(round-to-nearest-even), which is the storage type of every input tensor.
"""

from __future__ import annotations

import numpy as np

from .configs import LayerShape, Workload

BASE_SEED = 241001805

# stream ids
_S_HIDDEN = 1
_S_OUTLIER = 2
_S_TOPIC_SEQ = 3
_S_TOPIC_MEAN = 4
_S_WQKV = 1000
_S_W1 = 2000
_S_W2 = 3000
_S_WO = 4000
_S_WGATE = 5000
_S_WUP = 6000
_S_WDOWN = 7000
_S_NORM = 8000

hidden_block_tokens = 1024


def _rng(seed: int, stream: int, block: int = 0) -> np.random.Generator:
    key = np.array([(seed & 0xFFFFFFFFFFFFFFFF),
                    ((stream & 0xFFFFFFFF) << 32) | (block & 0xFFFFFFFF)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def layer_weights(shape: LayerShape, layer: int, seed: int = BASE_SEED):
    """(W_qkv [D x d_in], W1 [d_in x d_R], W2 [d_R x h_kv]), each ~ N(0, 1/fan_in)."""
    D, d_in, d_R, hk = shape.d_model, shape.d_in, shape.d_retain, shape.n_kv_heads
    wqkv = _rng(seed, _S_WQKV + layer).standard_normal((D, d_in), dtype=np.float32)
    wqkv *= np.float32(1.0 / np.sqrt(D))
    w1 = _rng(seed, _S_W1 + layer).standard_normal((d_in, d_R), dtype=np.float32)
    w1 *= np.float32(1.0 / np.sqrt(d_in))
    w2 = _rng(seed, _S_W2 + layer).standard_normal((d_R, hk), dtype=np.float32)
    w2 *= np.float32(1.0 / np.sqrt(d_R))
    return to_bf16_grid(wqkv), to_bf16_grid(w1), to_bf16_grid(w2)


def block_weights(shape: LayerShape, layer: int, seed: int = BASE_SEED):
    """Weights that close the decoder layer around the attention block: W_o [h*d x D],
    W_gate, W_up [D x d_ff], W_down [d_ff x D], each ~ N(0, 1/fan_in), and the two RMSNorm gains
    (1 + N(0, 0.1^2)), all on the bfloat16 grid."""
    D, hd, F = shape.d_model, shape.n_q_heads * shape.head_dim, shape.d_ff
    if F <= 0:
        raise ValueError("the shape has no d_ff")
    def w(stream, rows, cols):
        a = _rng(seed, stream + layer).standard_normal((rows, cols), dtype=np.float32)
        a *= np.float32(1.0 / np.sqrt(rows))
        return to_bf16_grid(a)
    g = _rng(seed, _S_NORM + layer)
    g1 = to_bf16_grid(1.0 + 0.1 * g.standard_normal(D, dtype=np.float32))
    g2 = to_bf16_grid(1.0 + 0.1 * g.standard_normal(D, dtype=np.float32))
    return {"w_o": w(_S_WO, hd, D), "w_gate": w(_S_WGATE, D, F), "w_up": w(_S_WUP, D, F),
            "w_down": w(_S_WDOWN, F, D), "g1": g1, "g2": g2}


def _topic_sequence(context: int, seed: int, n_topics: int = 64, mean_len: int = 512):
    """Topic id per token: segments of geometric length, topic uniform per segment."""
    g = _rng(seed, _S_TOPIC_SEQ)
    ids = np.empty(context, dtype=np.int32)
    pos = 0
    while pos < context:
        seg = int(g.geometric(1.0 / mean_len))
        ids[pos:pos + seg] = int(g.integers(0, n_topics))
        pos += seg
    return ids


_topic_cache: dict = {}


def _topics(w: Workload, seed: int):
    key = (w.context, w.shape.d_model, seed)
    if key not in _topic_cache:
        means = _rng(seed, _S_TOPIC_MEAN).standard_normal(
            (64, w.shape.d_model), dtype=np.float32)
        _topic_cache[key] = (_topic_sequence(w.context, seed), means)
    return _topic_cache[key]


def _hidden_block(w: Workload, block: int, seed: int) -> np.ndarray:
    D = w.shape.d_model
    n = hidden_block_tokens
    x = _rng(seed, _S_HIDDEN, block).standard_normal((n, D), dtype=np.float32)
    if w.hidden == "outlier":
        # each token independently, with probability 0.001, has its row scaled by 20
        u = _rng(seed, _S_OUTLIER, block).random(n)
        x[u < 0.001] *= np.float32(20.0)
    elif w.hidden == "topics":
        ids, means = _topics(w, seed)
        t0 = block * n
        seg = ids[t0:t0 + n]
        mu = np.zeros((n, D), dtype=np.float32)
        mu[:len(seg)] = means[seg]
        x = np.float32(np.sqrt(0.5)) * mu + np.float32(np.sqrt(0.5)) * x
    elif w.hidden != "normal":
        raise ValueError(w.hidden)
    return x


def hidden_states(w: Workload, start: int, n_tok: int, seed: int = BASE_SEED) -> np.ndarray:
    """Hidden-state rows [start, start + n_tok) of the workload's token stream."""
    n = hidden_block_tokens
    b0, b1 = start // n, (start + n_tok - 1) // n
    parts = [_hidden_block(w, b, seed) for b in range(b0, b1 + 1)]
    x = np.concatenate(parts, axis=0) if len(parts) > 1 else parts[0]
    off = start - b0 * n
    return to_bf16_grid(x[off:off + n_tok])
