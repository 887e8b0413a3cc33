"""CPU oracle for the Batch-Max evicting-attention path.

TEST INFRASTRUCTURE ONLY.  Nothing under this package is part of the product:
only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it.  It shares no code with the CUDA path and never imports it.
"""
from .batchmax_oracle import (  # noqa: F401
    UnitCache,
    dense_causal_attention,
    run_north_star,
    run_algorithm1,
    run_decode_only,
    run_extreme_decoding,
)
