"""A Mamba drafter block stack around the library, with the data dependence a real drafter has.

In a Mamba block the step size, B and C are projections of the conv output, so the fused conv+scan call cannot be
fed by a real model.  The library offers two ways: the split mode, `MDRAFT_CONV_ONLY` (conv window + SiLU), the
caller's projections, then `MDRAFT_PRECONV` (recurrence + gate); or `mdraft_tree_step_proj`, which takes the two
projection matrices and does conv step, projections, recurrence and gate in one launch (`fused=True` here).  This
module is the caller, for drafting only: embedding,
24 x [RMSNorm, in_proj, conv step, x_proj, dt_proj, S6 step, out_proj, residual], final norm, LM head, and
tree-structured drafting by batch generation (paper Section 4.1): generation i is one batch of all nodes of level
i, each node forks its parent's conv / SSM state by slot index, and the children of a node are its N_i most
probable next tokens.  The projections are plain torch matmuls on random weights (they are outside the library,
and there are no trained weights here): what this measures is the drafting LATENCY of the whole stack per round,
the quantity of the paper's Table 4, not acceptance.

Slots: 0 = the sequence's committed state; node i of the current round = slot 1 + i.
"""

from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as mb


# Above this many nodes in a level the one-launch projection step loses to the split mode (its per-node re-reads of
# the two projection matrices cost more than the split mode's matrix products); the stack switches path there.
PROJ_STEP_MAX_NODES = 256


class ToyDrafter:
    def __init__(self, n_layers: int = 24, d_model: int = 768, d_inner: int = 1536, dt_rank: int = 48, vocab: int = 50280,
                 max_nodes: int = 64, act: torch.dtype = torch.bfloat16, seed: int = 0, device="cuda", fused: bool = False):
        g = torch.Generator(device=device).manual_seed(seed)
        self.n_layers, self.d_model, self.d_inner, self.dt_rank, self.vocab, self.act, self.dev = n_layers, d_model, d_inner, dt_rank, vocab, act, device
        N = 16

        def rnd(*shape, scale):
            return (torch.randn(shape, generator=g, device=device) * scale).to(act)

        self.embed = rnd(vocab, d_model, scale=1.0)
        self.W_in = [rnd(d_model, 2 * d_inner, scale=d_model ** -0.5) for _ in range(n_layers)]
        self.W_x = [rnd(d_inner, dt_rank + 2 * N, scale=d_inner ** -0.5) for _ in range(n_layers)]
        self.W_dt = [rnd(dt_rank, d_inner, scale=dt_rank ** -0.5) for _ in range(n_layers)]
        self.W_out = [rnd(d_inner, d_model, scale=d_inner ** -0.5 / (2 * n_layers) ** 0.5) for _ in range(n_layers)]
        self.W_lm = rnd(d_model, vocab, scale=d_model ** -0.5)
        self.fused = fused
        if fused:   # the library takes both matrices as (out features, in features), rows contiguous
            self.W_x_rows = [w.T.contiguous() for w in self.W_x]
            self.W_dt_rows = [w.T.contiguous() for w in self.W_dt]
        A = -torch.arange(1, N + 1, dtype=torch.float32, device=device).repeat(d_inner, 1).contiguous()
        self.layers: List[mb.Layer] = []
        for _ in range(n_layers):
            conv_w = (torch.randn((d_inner, 4), generator=g, device=device) * 0.5).contiguous()
            dt_bias = torch.full((d_inner,), -4.579712, device=device)
            self.layers.append(mb.Layer(A, torch.ones(d_inner, device=device), conv_w, None, dt_bias, act, mb.MDRAFT_DT_SOFTPLUS))
        self.cache = mb.StateCache(n_layers, 1 + max_nodes, d_inner, act=act, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.max_nodes = max_nodes
        # static buffers, so that a generation step can be captured once per batch size and replayed
        self.tokens = torch.zeros(max_nodes, dtype=torch.int64, device=device)
        self.parent_slot = torch.zeros(max_nodes, dtype=torch.int32, device=device)
        self.node_slot = torch.zeros(max_nodes, dtype=torch.int32, device=device)
        self.u = torch.zeros((max_nodes, d_inner), dtype=act, device=device)
        self.y = torch.zeros((max_nodes, d_inner), dtype=act, device=device)
        self.logits = torch.zeros((max_nodes, vocab), dtype=act, device=device)
        self._graphs = {}
        self._round_graphs = {}
        self.root_token = torch.zeros(1, dtype=torch.int64, device=device)   # read by the round, so that a captured round can be replayed with another root

    @staticmethod
    def _norm(h: torch.Tensor) -> torch.Tensor:
        return torch.nn.functional.rms_norm(h, (h.shape[-1],), eps=1e-5)

    def _generation(self, lo: int, hi: int) -> None:
        """One batch-generation step for nodes [lo, hi): tokens / parent_slot / node_slot rows lo..hi-1 are read,
        logits rows lo..hi-1 are written; conv and SSM states of the nodes' slots are written."""
        N, R = 16, self.dt_rank
        h = self.embed[self.tokens[lo:hi]]
        ps, ns = self.parent_slot[lo:hi], self.node_slot[lo:hi]
        u, y = self.u[lo:hi], self.y[lo:hi]
        for l in range(self.n_layers):
            xz = self._norm(h) @ self.W_in[l]
            x, z = xz[:, :self.d_inner], xz[:, self.d_inner:]
            if self.fused and hi - lo <= PROJ_STEP_MAX_NODES:
                mb.mdraft_tree_step_proj(self.layers[l], self.cache, l, self.W_x_rows[l], self.W_dt_rows[l], x, z, y, ps, ns, self.status,
                                         flags=mb.MDRAFT_DT_SOFTPLUS | mb.MDRAFT_A_POWERS)
                h = h + y @ self.W_out[l]
                continue
            mb.mdraft_tree_step(self.layers[l], self.cache, l, x, None, None, None, None, u, ps, ns, None, self.status,
                                flags=mb.MDRAFT_CONV_ONLY)
            dbc = u @ self.W_x[l]
            dt = (dbc[:, :R] @ self.W_dt[l]).contiguous()
            Bm, Cm = dbc[:, R:R + N].contiguous(), dbc[:, R + N:].contiguous()
            mb.mdraft_tree_step(self.layers[l], self.cache, l, u, z, dt, Bm, Cm, y, ps, ns, None, self.status,
                                flags=mb.MDRAFT_DT_SOFTPLUS | mb.MDRAFT_PRECONV | mb.MDRAFT_A_POWERS)
            h = h + y @ self.W_out[l]
        self.logits[lo:hi] = self._norm(h) @ self.W_lm

    def generation(self, lo: int, hi: int, use_graph: bool = True) -> None:
        if not use_graph:
            self._generation(lo, hi)
            return
        key = (lo, hi)
        g = self._graphs.get(key)
        if g is None:
            self._generation(lo, hi)   # the first call of a shape happens outside the capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._generation(lo, hi)
            self._graphs[key] = g
        g.replay()

    def _round(self, config: Sequence[int], use_graph: bool):
        """All generations of one draft tree below the committed state, root token taken from `self.root_token`."""
        parents = [-1]
        level = [0]
        self.tokens[0:1] = self.root_token
        self.parent_slot[0:1] = 0
        self.node_slot[0:1] = 1
        self.generation(0, 1, use_graph)
        lo = 1
        for n_i in config:
            width = len(level) * n_i
            top = torch.topk(self.logits[level[0]:level[-1] + 1].float(), n_i, dim=-1).indices   # (len(level), n_i)
            self.tokens[lo:lo + width] = top.reshape(-1)
            par = torch.arange(level[0], level[-1] + 1, device=self.dev).repeat_interleave(n_i)   # built on the device: no host sync
            self.parent_slot[lo:lo + width] = (par + 1).to(torch.int32)
            self.node_slot[lo:lo + width] = torch.arange(lo + 1, lo + width + 1, device=self.dev, dtype=torch.int32)
            parents += [v for v in level for _ in range(n_i)]
            self.generation(lo, lo + width, use_graph)
            level = list(range(lo, lo + width))
            lo += width
        return self.tokens[:lo].clone(), parents

    def draft_round(self, root_token: int, config: Sequence[int], use_graph: bool = True):
        """Draft one tree below the committed state.  config = (N_1, ..., N_gamma) as the paper writes it; the root
        (the last verified token) is node 0.  Returns (tokens (M,), parents list); node states are in slots 1..M.
        With `use_graph` every generation step is one replayed CUDA graph; the host launches them and the top-k
        between them."""
        self.root_token.fill_(int(root_token))
        return self._round(config, use_graph)

    def draft_round_one_graph(self, root_token: int, config: Sequence[int]):
        """The same round as ONE replayed CUDA graph per tree configuration (the paper's graph cache, Section 4.1, taken
        to the whole round: generation steps, top-k and index bookkeeping all sit inside the graph, so the host does one
        launch per round).  Returns (tokens (M,), parents list); the token tensor is overwritten by the next replay."""
        key = tuple(int(v) for v in config)
        self.root_token.fill_(int(root_token))
        entry = self._round_graphs.get(key)
        if entry is None:
            self._round(key, use_graph=False)   # first use of every shape happens outside the capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                out = self._round(key, use_graph=False)
            entry = self._round_graphs[key] = (g, out)
        entry[0].replay()
        return entry[1]

    def commit(self, node: int) -> None:
        mb.mdraft_state_commit(self.cache, torch.tensor([1 + node], dtype=torch.int32, device=self.dev),
                               torch.zeros(1, dtype=torch.int32, device=self.dev), self.status)
