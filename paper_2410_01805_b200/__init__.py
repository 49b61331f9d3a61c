"""B200-native chunked-prefill step with retaining-head eviction (Locret).

The package is a thin ctypes binding over ``liblocret.so`` (hand-written CUDA for
sm_100a).  Every step of the path runs in the library's kernels; Python only
marshals pointers.  There is no CPU fallback: importing the binding without the
built library raises.
"""

from .binding import (  # noqa: F401
    K_NAMES,
    LAST_CHUNK,
    LayerStack,
    NO_EVICT,
    LocretBlock,
    LocretError,
    LocretLayer,
    LocretLayerTP,
    adamw_step,
    cis_labels,
    lib,
    lib_path,
    rh_loss_grad,
    shard_by_kv_head,
)
