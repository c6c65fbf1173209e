"""Small, self-contained runs of each kernel for a profiler.

    python -m paper_2506_01206_b200.profile_case prefill [tokens] [layers]
    python -m paper_2506_01206_b200.profile_case tree    [layers]
    python -m paper_2506_01206_b200.profile_case proj    [nodes] [layers]

`prefill` encodes a 130M-shaped context (default 2048 tokens x 1536 channels, bf16, 4 layers) three times;
`tree` runs one batched-serving draft round (32 sequences x 32-node trees, default 4 layers) twice; `proj` runs one
tree level (default 18 nodes, the paper's widest, 24 layers) through the step that forms dt, B, C itself.  All hold well
under 1 GB on the device and launch a few dozen kernels, which keeps a multi-pass profiler capture short; inputs are
larger than L2 across the layers, so DRAM counters still mean something.
"""

from __future__ import annotations

import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402
import paper_2506_01206_b200 as md  # noqa: E402
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer  # noqa: E402

FLAGS = md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_A_POWERS


def prefill(tokens: int = 2048, n_layers: int = 4, reps: int = 3) -> None:
    cfg = gen.get_config(1)
    tdt, D = torch_act(cfg.act), cfg.d_inner
    lays = [upload_layer(gen.layer_params(cfg, l), cfg.act, FLAGS) for l in range(n_layers)]
    ins = [[to_device(a, tdt) for a in gen.prefill_inputs(cfg, l, tokens)] for l in range(n_layers)]
    outs = [torch.empty((tokens, D), dtype=tdt, device="cuda") for _ in range(n_layers)]
    cache = md.StateCache(n_layers, 1, D, act=tdt)
    ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lays[0], tokens, 1, tokens)), dtype=torch.uint8, device="cuda")
    cu, slot, status = i32([0, tokens]), i32([0]), torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(reps):
        for l in range(n_layers):
            md.mdraft_conv_scan_prefill(lays[l], cache, l, *ins[l], outs[l], cu, tokens, None, slot, ws, 0, status)
    torch.cuda.synchronize()
    print("prefill: %d tokens x %d channels, %d layers x %d, status %d" % (tokens, D, n_layers, reps, int(status.item())))


def tree(n_layers: int = 4, reps: int = 2) -> None:
    cfg = gen.get_config(4)
    tdt, D, S = torch_act(cfg.act), cfg.d_inner, cfg.n_seq
    trees = [gen.config_tree(cfg, 0, s) for s in range(S)]
    off = np.cumsum([0] + [t.n_nodes for t in trees])
    parent, nodes, lvl = [], [], [0]
    for l in range(max(t.n_levels for t in trees)):
        for s, t in enumerate(trees):
            if l >= t.n_levels:
                continue
            for i in range(int(t.level_offsets[l]), int(t.level_offsets[l + 1])):
                par = int(t.parents[i])
                parent.append(s if par < 0 else S + int(off[s]) + par)
                nodes.append(S + int(off[s]) + i)
        lvl.append(len(nodes))
    M = len(nodes)
    lays = [upload_layer(gen.layer_params(cfg, l), cfg.act, FLAGS) for l in range(n_layers)]
    ins = [[to_device(a, tdt) for a in gen.node_inputs(cfg, l, 0, M)] for l in range(n_layers)]
    outs = [torch.empty((M, D), dtype=tdt, device="cuda") for _ in range(n_layers)]
    cache = md.StateCache(n_layers, S + M, D, act=tdt)
    cache.ssm.normal_()
    par, nod, status = i32(parent), i32(nodes), torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(reps):
        for l in range(n_layers):
            md.mdraft_tree_step(lays[l], cache, l, *ins[l], outs[l], par, nod, lvl, status)
    torch.cuda.synchronize()
    print("tree: %d nodes, levels %s, %d layers x %d, status %d" % (M, np.diff(lvl).tolist(), n_layers, reps, int(status.item())))


def proj(n_nodes: int = 18, n_layers: int = 24, reps: int = 3, dt_rank: int = 48) -> None:
    cfg = gen.get_config(1)
    tdt, D = torch_act(cfg.act), cfg.d_inner
    lays = [upload_layer(gen.layer_params(cfg, l), cfg.act, FLAGS) for l in range(n_layers)]
    Ws = [[to_device(w, tdt) for w in gen.select_proj(cfg, l, dt_rank)] for l in range(n_layers)]
    ins = [[to_device(a, tdt) for a in gen.node_inputs(cfg, l, 0, n_nodes)[:2]] for l in range(n_layers)]
    out = torch.empty((n_nodes, D), dtype=tdt, device="cuda")
    cache = md.StateCache(n_layers, 1 + n_nodes, D, act=tdt)
    cache.ssm.normal_()
    cache.conv.normal_()
    par, nod, status = i32([0] * n_nodes), i32(list(range(1, n_nodes + 1))), torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(reps):
        for l in range(n_layers):
            md.mdraft_tree_step_proj(lays[l], cache, l, Ws[l][0], Ws[l][1], ins[l][0], ins[l][1], out, par, nod, status)
    torch.cuda.synchronize()
    print("proj: %d nodes x %d channels, dt_rank %d, %d layers x %d, status %d" % (n_nodes, D, dt_rank, n_layers, reps, int(status.item())))


if __name__ == "__main__":
    what = sys.argv[1] if len(sys.argv) > 1 else "prefill"
    nums = [int(v) for v in sys.argv[2:]]
    if what == "prefill":
        prefill(*nums)
    elif what == "tree":
        tree(*nums)
    elif what == "proj":
        proj(*nums)
    else:
        raise SystemExit(__doc__)
