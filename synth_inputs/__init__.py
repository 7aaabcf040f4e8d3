"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package holds data recipes only: model shapes, random weights, ragged KV
lengths, page tables, random logits.  It contains none of the method's
arithmetic (no softmax, no norm, no attention, no sampling, no Philox): both
the oracle and the CUDA library receive the arrays produced here as inputs.
"""
from .configs import ModelConfig, CONFIGS, get_config  # noqa: F401
from .weights import make_weights, bf16_round  # noqa: F401
from .workload import (  # noqa: F401
    kv_lengths_uniform,
    kv_lengths_lognormal,
    make_page_tables,
    sampler_only_logits,
    random_prompts,
)
