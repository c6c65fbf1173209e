"""The five workload configurations, as plain data.

Shapes follow the drafter the paper uses (a 130M-parameter Mamba: 24 layers,
d_model 768, d_inner 1536, d_state 16, d_conv 4; paper Section 3.1 and
Appendix A.2), contexts of 1k-8k tokens (Section 5.2) and draft trees of a few
levels (Section 4.1, Tables 4-5).  They stand in for the paper's datasets and
trained weights, which are not available here.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class Config:
    cid: int
    name: str
    n_layers: int
    d_inner: int
    d_state: int
    d_conv: int
    act: str                 # "f32" or "bf16" (activation dtype; state is always fp32)
    n_seq: int
    context: Tuple[int, int]  # (lo, hi) inclusive token range per sequence; lo==hi => fixed
    tree: str                # "full:2x4" | "capped150" | "chain16" | "rand32" | "none"
    rounds: int
    seed: int = 0
    notes: str = ""


CONFIGS = {
    0: Config(0, "tiny-f32", 1, 64, 16, 4, "f32", 1, (256, 256), "full:2x4", 1,
              notes="15-node tree, 4 levels of width 2, BFS parents"),
    1: Config(1, "130m-prefill-2k", 24, 1536, 16, 4, "bf16", 1, (2048, 2048), "none", 0),
    2: Config(2, "130m-tree-150", 24, 1536, 16, 4, "bf16", 1, (2048, 2048), "capped150", 8,
              notes="6 levels: branching 4,4 then 2,2,2 below a root; capped at 150 nodes"),
    3: Config(3, "130m-long-32k", 24, 1536, 16, 4, "bf16", 1, (32768, 32768), "chain16", 1,
              notes="16 single-chain decode steps after the prefill"),
    4: Config(4, "130m-batch32", 24, 1536, 16, 4, "bf16", 32, (1024, 8192), "rand32", 4,
              notes="packed varlen prefill; 32-node random trees per sequence"),
}


def get_config(cid: int) -> Config:
    return CONFIGS[int(cid)]
