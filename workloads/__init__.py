"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This package only draws random numbers and names shapes.  It holds none of the method's
arithmetic (no softmax, no attention, no selection rule) so that the CPU oracle and the
CUDA library stay independent of each other: both consume the same bits from here.
"""
from .configs import CONFIGS, WorkloadConfig, get_config  # noqa: F401
from .generators import (  # noqa: F401
    seed_for, make_attn_inputs, make_kv_rows, make_cache, make_logits, make_mask,
    make_tok_ar, bf16_bits, widen,
)
