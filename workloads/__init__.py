"""Seeded synthetic inputs for the tree-verification hot path.

This package only *draws inputs* (trees, tokens, logits, bf16 K/V/Q bit patterns) and
names the five workload shapes. It holds none of the verification arithmetic: no
attention, no softmax, no argmax, no path walk, no compaction. Both the CUDA parity
tests and the CPU oracle tests take their inputs from here so that the two sides read
identical bytes.
"""

from .configs import CONFIGS, WorkloadConfig, get_config  # noqa: F401
from .gen import (  # noqa: F401
    bf16_bits_from_f32,
    chain_tree,
    config1_tree,
    draw_prefix_lens,
    eagle2_like_tree,
    normal_bf16_bits,
    planted_logits,
    sibling_distinct_tokens,
    single_node_tree,
    star_tree,
)
