"""Seeded synthetic workloads: shape table and input generators.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds no arithmetic of the method itself: only shapes, the
pseudo-random draws, and the encoding of the draws as bf16-representable
float32 values.
"""

from .configs import CONFIGS, LayerShape, Workload, get_workload  # noqa: F401
from .generate import (  # noqa: F401
    BASE_SEED,
    block_weights,
    hidden_block_tokens,
    hidden_states,
    layer_weights,
    to_bf16_grid,
)
