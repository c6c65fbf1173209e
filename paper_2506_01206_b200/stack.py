"""A stack of drafter layers driven through the C ABI: launch sequencing only.

The real drafter interleaves these calls with its projections (which are outside this library); here the
per-layer inputs are independent tensors, so one "pass" is simply every layer's call issued on one stream.
"""

from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as mb


class DrafterStack:
    def __init__(self, layers: Sequence[mb.Layer], n_slots: int, max_tokens: int, n_seq: int, max_seqlen: int,
                 chunk_len: int = 0, device="cuda"):
        self.layers = list(layers)
        l0 = self.layers[0]
        self.d_inner, self.act = l0.d_inner, l0.act
        self.cache = mb.StateCache(len(self.layers), n_slots, l0.d_inner, l0.d_state, l0.d_conv, l0.act, device)
        self.chunk_len = chunk_len
        self.ws_bytes = max(mb.mdraft_prefill_workspace_bytes(l, max_tokens, n_seq, max_seqlen, chunk_len) for l in self.layers)
        self.workspace = torch.empty(max(self.ws_bytes, 256), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    # number of kernels one prefill call launches (chunk summary + carry scan + main scan, or the main scan alone)
    def prefill_launches_per_layer(self, total_tokens: int, n_seq: int, max_seqlen: int) -> int:
        chunked = mb.mdraft_prefill_workspace_bytes(self.layers[0], total_tokens, n_seq, max_seqlen, self.chunk_len) > 0
        return 3 if chunked else 1

    def prefill(self, inputs: Sequence[Sequence[torch.Tensor]], outs: Sequence[torch.Tensor], cu_seqlens: torch.Tensor,
                max_seqlen: int, init_slot: Optional[torch.Tensor], final_slot: Optional[torch.Tensor], stream=None,
                phase_events: Optional[List] = None, layer_range=None) -> None:
        """inputs[l] = (x, z, dt, B, C) of layer l.  phase_events[l] = (start, after_state, after_carry, end)."""
        rng = range(len(self.layers)) if layer_range is None else layer_range
        for l in rng:
            x, z, dt, B, C = inputs[l]
            pe = None
            if phase_events is not None:
                phase_events[l][0].record(stream)
                pe = (phase_events[l][1], phase_events[l][2])
            mb.mdraft_conv_scan_prefill(self.layers[l], self.cache, l, x, z, dt, B, C, outs[l], cu_seqlens, max_seqlen,
                                        init_slot, final_slot, self.workspace, self.chunk_len, self.status, stream,
                                        phase_events=pe)
            if phase_events is not None:
                phase_events[l][3].record(stream)

    def tree_round(self, inputs: Sequence[Sequence[torch.Tensor]], outs: Sequence[torch.Tensor], parent_slot: torch.Tensor,
                   node_slot: torch.Tensor, level_offsets: Optional[Sequence[int]], stream=None, layer_range=None) -> None:
        rng = range(len(self.layers)) if layer_range is None else layer_range
        for l in rng:
            x, z, dt, B, C = inputs[l]
            mb.mdraft_tree_step(self.layers[l], self.cache, l, x, z, dt, B, C, outs[l], parent_slot, node_slot,
                                level_offsets, self.status, stream)

    def commit(self, src_slot: torch.Tensor, dst_slot: torch.Tensor, stream=None) -> None:
        mb.mdraft_state_commit(self.cache, src_slot, dst_slot, self.status, stream)

    def check_status(self) -> None:
        s = int(self.status.item())
        if s:
            raise RuntimeError(f"device status bits set: {s:#x}")


class RoundGraphCache:
    """CUDA graphs of draft rounds, one per tree shape, replayed instead of re-launched.

    The paper caches one CUDA graph per batch size of its drafter (Section 4.1, "Efficient cache utilization"); here
    a graph covers a whole round — every level of every layer plus the commit — and is keyed by the tree's level
    sizes, which is all the launch geometry depends on.  Everything a round reads lives in static device buffers owned
    by this object (node inputs per layer, parent / node slots, the accepted node's slot), so a replay sees whatever
    the caller last copied into them; the library's calls take their indices from device memory, which is what makes
    one capture valid for every tree of that shape.
    """

    def __init__(self, stack: DrafterStack, max_nodes: int, seq_slot: int = 0):
        self.stack = stack
        dev, D, act = stack.status.device, stack.d_inner, stack.act
        n = len(stack.layers)
        self.x = [torch.zeros((max_nodes, D), dtype=act, device=dev) for _ in range(n)]
        self.z = [torch.zeros((max_nodes, D), dtype=act, device=dev) for _ in range(n)]
        self.dt = [torch.zeros((max_nodes, D), dtype=act, device=dev) for _ in range(n)]
        self.B = [torch.zeros((max_nodes, 16), dtype=act, device=dev) for _ in range(n)]
        self.C = [torch.zeros((max_nodes, 16), dtype=act, device=dev) for _ in range(n)]
        self.out = [torch.zeros((max_nodes, D), dtype=act, device=dev) for _ in range(n)]
        self.parent_slot = torch.zeros(max_nodes, dtype=torch.int32, device=dev)
        self.node_slot = torch.zeros(max_nodes, dtype=torch.int32, device=dev)
        self.accepted_slot = torch.zeros(1, dtype=torch.int32, device=dev)
        self.seq_slot = torch.full((1,), seq_slot, dtype=torch.int32, device=dev)
        self.max_nodes = max_nodes
        self._graphs = {}

    def _launch(self, level_offsets) -> None:
        m = level_offsets[-1]
        ins = [(self.x[l][:m], self.z[l][:m], self.dt[l][:m], self.B[l][:m], self.C[l][:m]) for l in range(len(self.stack.layers))]
        outs = [o[:m] for o in self.out]
        self.stack.tree_round(ins, outs, self.parent_slot[:m], self.node_slot[:m], level_offsets)
        self.stack.commit(self.accepted_slot, self.seq_slot)

    def run(self, level_offsets: Sequence[int]) -> bool:
        """Run one round (all levels, all layers, then the commit of `accepted_slot`) for a tree with these level
        offsets.  Returns True when an existing graph was replayed, False when the shape was new and got captured."""
        key = tuple(int(v) for v in level_offsets)
        if key[-1] > self.max_nodes:
            raise ValueError("tree larger than the buffers of this cache")
        g = self._graphs.get(key)
        if g is not None:
            g.replay()
            return True
        self._launch(list(key))           # first use of a shape runs eagerly once (nothing new happens inside a capture)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self._launch(list(key))
        self._graphs[key] = g
        return False

    def __len__(self) -> int:
        return len(self._graphs)
