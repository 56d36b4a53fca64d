"""The five synthetic workload shapes (LLaVA-class verify steps).

Shapes follow the models the paper evaluates (Section 4.1: LLaVA-1.5/1.6 7B and 13B,
i.e. 32 layers x 32 heads and 40 layers x 40 heads, head_dim 128, vocabulary 32000) and
its draft-tree setting (Section 4.1: EAGLE-2 tree attention, top-k 10, 60 tokens).
Datasets and weights are not used; only the shapes are.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    L: int            # decoder layers
    H: int            # attention heads (MHA: H_kv == H)
    D: int            # head dim
    B: int            # batch (sequences)
    T: int            # tree nodes including the root (node 0)
    max_depth: int    # deepest tree level (edges from the root)
    V: int            # vocabulary size
    seed: int
    prefix_nominal: int                   # nominal prefix length P
    prefix_rule: str = "fixed"            # fixed | pm25 | cfg4 | cfg5
    tree_kind: str = "eagle2"             # eagle2 | config1
    note: str = ""
    visual_text: Tuple[int, int] = field(default=(0, 0))

    @property
    def s_cap(self) -> int:
        """Cache capacity in token slots: longest possible prefix + 64 tree slots."""
        if self.prefix_rule == "pm25":
            return int(round(self.prefix_nominal * 1.25)) + 64
        return self.prefix_nominal + 64


CONFIGS = {
    # Tiny reference case the oracle finishes in well under a second.
    "cfg1": WorkloadConfig("cfg1", L=1, H=32, D=128, B=1, T=26, max_depth=5, V=32000,
                           seed=1001, prefix_nominal=640, tree_kind="config1",
                           visual_text=(576, 64), note="tiny reference"),
    # Headline: LLaVA-1.6-7B-shaped verify step.
    "cfg2": WorkloadConfig("cfg2", L=32, H=32, D=128, B=1, T=60, max_depth=6, V=32000,
                           seed=2002, prefix_nominal=3008, visual_text=(2880, 128),
                           note="LLaVA-1.6-7B shape, AnyRes 5x576 visual + 128 text"),
    # Compressed-visual regime, batch 1 (two pooled sizes) and batch 16 ragged.
    "cfg3_b1_144": WorkloadConfig("cfg3_b1_144", L=32, H=32, D=128, B=1, T=60, max_depth=6,
                                  V=32000, seed=3003, prefix_nominal=272,
                                  visual_text=(144, 128), note="compressed visual 144"),
    "cfg3_b1_288": WorkloadConfig("cfg3_b1_288", L=32, H=32, D=128, B=1, T=60, max_depth=6,
                                  V=32000, seed=3004, prefix_nominal=416,
                                  visual_text=(288, 128), note="compressed visual 288"),
    "cfg3_b16_144": WorkloadConfig("cfg3_b16_144", L=32, H=32, D=128, B=16, T=60, max_depth=6,
                                   V=32000, seed=3005, prefix_nominal=272, prefix_rule="pm25",
                                   visual_text=(144, 128), note="compressed, ragged +-25%"),
    "cfg3_b16_288": WorkloadConfig("cfg3_b16_288", L=32, H=32, D=128, B=16, T=60, max_depth=6,
                                   V=32000, seed=3006, prefix_nominal=416, prefix_rule="pm25",
                                   visual_text=(288, 128), note="compressed, ragged +-25%"),
    # LLaVA-1.6-13B-shaped, batch 4 ragged.
    "cfg4": WorkloadConfig("cfg4", L=40, H=40, D=128, B=4, T=60, max_depth=6, V=32000,
                           seed=4004, prefix_nominal=3336, prefix_rule="cfg4",
                           visual_text=(2880, 256), note="13B shape, +200 generated"),
    # Video-like long prefix, batch 8 ragged.
    "cfg5": WorkloadConfig("cfg5", L=32, H=32, D=128, B=8, T=60, max_depth=6, V=32000,
                           seed=5005, prefix_nominal=9728, prefix_rule="cfg5",
                           visual_text=(9216, 512), note="16 frames x 576 + 512 text"),
}


def get_config(name: str) -> WorkloadConfig:
    return CONFIGS[name]
