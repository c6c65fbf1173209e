"""The split mode and the one-launch projection step inside a real block stack (conv step -> projections -> S6 step,
states forked by slot) against an
fp64 replica assembled from the oracle: every node's logits must equal those of its root-to-node token path pushed
through the same weights layer by layer."""

import numpy as np
import pytest
import torch

import oracle
from parity import assert_close

pytestmark = pytest.mark.gpu

from paper_2506_01206_b200.drafter import ToyDrafter


def _replica_logits(d: ToyDrafter, path_tokens, conv0, h0):
    """fp64: the tokens of one root-to-node path as a short sequence; returns the logits after the last token."""
    f = lambda t: t.detach().double().cpu().numpy()
    N, R = 16, d.dt_rank

    def norm(h):
        return h / np.sqrt((h * h).mean(-1, keepdims=True) + 1e-5)

    h = f(d.embed)[path_tokens]
    L = len(path_tokens)
    zeros = np.zeros((L, d.d_inner)); zn = np.zeros((L, N))
    for l in range(d.n_layers):
        lay = d.layers[l]
        ol = oracle.Layer(f(lay.A), f(lay.D), f(lay.conv_w), None, f(lay.dt_bias))
        xz = norm(h) @ f(d.W_in[l])
        x, z = xz[:, :d.d_inner], xz[:, d.d_inner:]
        u, _, _ = oracle.prefill(ol, x, zeros, zeros, zn, zn, conv_init=conv0[l][None], flags=oracle.CONV_ONLY)
        dbc = u @ f(d.W_x[l])
        dt = dbc[:, :R] @ f(d.W_dt[l])
        y, _, _ = oracle.prefill(ol, u, z, dt, dbc[:, R:R + N], dbc[:, R + N:], h_init=h0[l][None], flags=oracle.DT_SOFTPLUS | oracle.PRECONV)
        h = h + y @ f(d.W_out[l])
    return (norm(h) @ f(d.W_lm))[-1]


@pytest.mark.parametrize("fused", [False, True])
def test_toy_drafter_tree_matches_path_replica(fused):
    d = ToyDrafter(n_layers=2, d_model=32, d_inner=64, dt_rank=8 if fused else 4, vocab=97, max_nodes=32, act=torch.float32, seed=1,
                   fused=fused)
    g = torch.Generator(device="cuda").manual_seed(2)
    d.cache.ssm[:, 0] = torch.randn(d.cache.ssm[:, 0].shape, generator=g, device="cuda")
    d.cache.conv[:, 0] = torch.randn(d.cache.conv[:, 0].shape, generator=g, device="cuda")
    conv0 = d.cache.conv[:, 0].double().cpu().numpy()
    h0 = d.cache.ssm[:, 0].double().cpu().numpy()
    for use_graph in (False, True):
        tokens, parents = d.draft_round(5, (3, 2, 1), use_graph=use_graph)
        torch.cuda.synchronize()
        assert int(d.status.item()) == 0
        M = len(parents)
        assert M == 1 + 3 + 6 + 6 and tokens.numel() == M
        toks = tokens.cpu().numpy()
        logits = d.logits[:M].double().cpu().numpy()
        for v in range(M):
            path = []
            a = v
            while a >= 0:
                path.append(int(toks[a])); a = parents[a]
            want = _replica_logits(d, path[::-1], conv0, h0)
            assert_close(logits[v], want, 1e-3, f"node {v} (graph={use_graph})")
    # the children of a node are its most probable tokens: siblings carry distinct tokens
    for p_ in set(parents[1:]):
        sib = [int(toks[i]) for i in range(M) if parents[i] == p_]
        assert len(set(sib)) == len(sib)
    # committing a node makes it the starting point of the next round
    d.commit(4)
    torch.cuda.synchronize()
    assert torch.equal(d.cache.ssm[:, 0], d.cache.ssm[:, 5]) and torch.equal(d.cache.conv[:, 0], d.cache.conv[:, 5])


def test_whole_round_in_one_graph_equals_generation_by_generation():
    d = ToyDrafter(n_layers=2, d_model=32, d_inner=64, dt_rank=8, vocab=97, max_nodes=32, act=torch.float32, seed=3, fused=True)
    g = torch.Generator(device="cuda").manual_seed(4)
    d.cache.ssm[:, 0] = torch.randn(d.cache.ssm[:, 0].shape, generator=g, device="cuda")
    d.cache.conv[:, 0] = torch.randn(d.cache.conv[:, 0].shape, generator=g, device="cuda")
    for root in (5, 41, 5):   # the second and third calls replay the captured round with another root token
        tok_a, par_a = d.draft_round(root, (3, 2, 1), use_graph=False)
        logits_a = d.logits[:len(par_a)].clone()
        states_a = d.cache.ssm[:, 1:1 + len(par_a)].clone()
        tok_b, par_b = d.draft_round_one_graph(root, (3, 2, 1))
        torch.cuda.synchronize()
        assert int(d.status.item()) == 0
        assert par_a == par_b and torch.equal(tok_a, tok_b)
        assert torch.equal(logits_a, d.logits[:len(par_a)]) and torch.equal(states_a, d.cache.ssm[:, 1:1 + len(par_a)])
