"""Batch-Max (arXiv 2412.05693) evicting-attention hot path for NVIDIA B200.

The product is the C-ABI library ``libbatchmax.so`` (declared in ``include/batchmax.h``);
:mod:`paper_2412_05693_b200.binding` is a thin ctypes layer with the same names that only marshals
arguments.  There is no CPU fallback: without the built CUDA library every call fails loudly.
"""
from .binding import (  # noqa: F401
    BMError,
    BatchMaxCache,
    Config,
    arena_bytes,
    cache_bytes_per_sample,
    debug_build,
    kernel_launch_count,
    last_prefill_path,
    lib,
    max_batch,
    workspace_bytes,
)
