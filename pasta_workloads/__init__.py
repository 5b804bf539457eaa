"""Seeded synthetic workloads for asynchronous-thread decode attention.

This package only *describes* inputs: which requests exist, which threads are
spawned, finished and merged when, how many tokens each stream receives, and the
random bf16 tensors that are appended or used as queries.  It contains none of
the method's arithmetic (no page tables, no visibility rule, no attention), so
the CPU oracle and the CUDA library can both replay the same script while
sharing no code with each other.
"""
from .scripts import (  # noqa: F401
    SEED,
    Geometry,
    Script,
    cfg1_tiny,
    cfg2_single_request,
    cfg3_batched,
    cfg4_long_prefix,
    cfg5_trace,
    random_script,
    step_tensors,
    run_tensors,
    token_tensors,
)
