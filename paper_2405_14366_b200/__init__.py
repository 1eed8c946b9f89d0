"""MiniCache hot path on B200: cross-layer KV merge, restore and compressed decode attention.

The arithmetic lives in hand-written CUDA kernels behind the C ABI declared in
``include/minicache.h``; this package is only the ctypes binding."""
from .binding import (  # noqa: F401
    MiniCacheLib,
    McConfig,
    PairCache,
    Batch,
    lib,
    MC_LAYER_LM1,
    MC_LAYER_L,
    MC_LAYER_BOTH,
    MC_RETAIN_DISTINCT,
    MC_RETAIN_LITERAL,
    MC_RETAIN_TOPK,
    McError,
)
