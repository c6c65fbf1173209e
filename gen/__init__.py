"""Seeded synthetic inputs for the Mamba-drafter hot path.

This package only *draws inputs*: layer constants, activations, draft-tree
topologies, sequence-length mixes and accepted-path choices.  It contains none
of the method's arithmetic (no convolution, no recurrence, no activation
functions applied to data), so both the CPU oracle's tests and the CUDA
harness may import it without sharing any computation.

Every array is a pure function of ``(seed, config, layer, round, tensor)``
through a counter-based generator (Philox), so the two sides can regenerate
identical inputs independently and in any order.
"""

from .configs import CONFIGS, Config, get_config
from .draw import (
    LayerParams,
    layer_params,
    select_proj,
    prefill_inputs,
    node_inputs,
    seq_lengths,
    round_to_act,
    bf16_bits,
    from_bf16_bits,
    DT_BIAS,
    DT_PRE_LO,
    DT_PRE_HI,
    SsdParams,
    ssd_params,
    ssd_inputs,
)
from .trees import (
    Tree,
    full_tree,
    paper_tree,
    capped_tree,
    random_branching_tree,
    chain_tree,
    random_accepted_node,
    config_tree,
)

__all__ = [
    "CONFIGS", "Config", "get_config", "LayerParams", "layer_params",
    "prefill_inputs", "node_inputs", "seq_lengths", "round_to_act",
    "bf16_bits", "from_bf16_bits", "DT_BIAS", "DT_PRE_LO", "DT_PRE_HI", "SsdParams", "ssd_params", "ssd_inputs",
    "Tree", "full_tree", "paper_tree", "capped_tree",
    "random_branching_tree", "chain_tree", "random_accepted_node",
    "config_tree",
]
