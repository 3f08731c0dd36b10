"""Seeded synthetic inputs for speculative-prefill scoring and selection.

This package only *produces inputs* (lookahead queries, prompt key caches, token ids,
character offsets).  It contains none of the method's arithmetic: no softmax, no
aggregation, no pooling, no selection.  Both the CUDA path's tests/bench and the CPU
oracle's tests draw their inputs from here so that they see the same bytes.
"""
from .synthetic import (  # noqa: F401
    CONFIGS,
    Prompt,
    WorkloadConfig,
    bf16_bits,
    make_prompt,
    make_workload,
    quantize_keys_e4m3,
    small_config,
)
