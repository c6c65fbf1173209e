"""The five workload configurations at their full sizes, in the launch configuration the benchmark times (default
chunk plan, structured-A dispatch decided by mdraft_classify_A), against the fp64 oracle.

Where the oracle finishes a whole tensor in seconds the comparison is element by element; for the two large
configurations it covers whole layers / whole sequences chosen by a fixed sample (a packed sequence equals the same
sequence run alone, which is what makes a per-sequence sample exact).  Index work (conv windows, commits) is compared
bit for bit everywhere.
"""

import numpy as np
import pytest
import torch

import gen
import oracle
from parity import TOL, TOL_STATE, assert_close

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer


def _layer(cfg, l):
    p = gen.layer_params(cfg, l)
    lay = upload_layer(p, cfg.act, md.MDRAFT_DT_SOFTPLUS)
    is_pow, nonpos = md.mdraft_classify_A(lay.A)
    assert nonpos
    if is_pow:
        lay.flags |= md.MDRAFT_A_POWERS
    return p, lay, oracle.layer_from_params(p)


def _prefill(cfg, lay, cache, layer_index, ins, cu, final_slots, status):
    tdt = torch_act(cfg.act)
    T = int(cu[-1]); S = len(cu) - 1
    max_len = int(np.max(np.diff(cu)))
    dev = [to_device(a, tdt) for a in ins]
    out = torch.full((T, cfg.d_inner), float("nan"), dtype=tdt, device="cuda")
    ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lay, T, S, max_len)), dtype=torch.uint8, device="cuda")
    md.mdraft_conv_scan_prefill(lay, cache, layer_index, *dev, out, i32(cu), max_len, None, i32(final_slots), ws, 0, status)
    return out


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


class Drafting:
    """Several draft rounds with commits for a set of sequences, GPU and oracle side by side.
    Slots: sequence s -> slot s; node i of sequence s -> slot S + off[s] + i."""

    def __init__(self, cfg, lay, olay, cache, layer_index, S, watch, status):
        self.cfg, self.lay, self.olay, self.cache, self.li, self.S, self.watch, self.status = cfg, lay, olay, cache, layer_index, S, watch, status
        self.tdt = torch_act(cfg.act)

    def round(self, rnd, committed, trees=None, accepted=None):
        """committed: {s: (conv (3,D), h (D,N))} oracle-side states of the watched sequences; updated in place.
        trees / accepted default to the configuration's own trees and seeded accepted nodes."""
        cfg, S = self.cfg, self.S
        if trees is None:
            trees = [gen.config_tree(cfg, rnd, s) for s in range(S)]
        off = np.cumsum([0] + [t.n_nodes for t in trees])
        M = int(off[-1])
        x, z, dt, B, C = gen.node_inputs(cfg, self.li, rnd, M)          # rows in sequence-major order
        order, parent, nodes, lvl = [], [], [], [0]
        for l in range(max(t.n_levels for t in trees)):                 # the GPU wants level-major order
            for s, t in enumerate(trees):
                if l >= t.n_levels:
                    continue
                for i in range(int(t.level_offsets[l]), int(t.level_offsets[l + 1])):
                    par = int(t.parents[i])
                    order.append(int(off[s]) + i)
                    parent.append(s if par < 0 else S + int(off[s]) + par)
                    nodes.append(S + int(off[s]) + i)
            lvl.append(len(order))
        order = np.asarray(order)
        dev = [to_device(a[order], self.tdt) for a in (x, z, dt, B, C)]
        out = torch.full((M, cfg.d_inner), float("nan"), dtype=self.tdt, device="cuda")
        md.mdraft_tree_step(self.lay, self.cache, self.li, *dev, out, i32(parent), i32(nodes), lvl, self.status)
        if accepted is None:
            accepted = [gen.random_accepted_node(trees[s], cfg.seed, cfg.cid, rnd, s) for s in range(S)]
        g_out = np.empty((M, cfg.d_inner))
        g_out[order] = _f64(out)
        worst = 0.0
        for s in self.watch:
            a, b = int(off[s]), int(off[s + 1])
            conv0, h0 = committed[s]
            o_out, o_conv, o_h = oracle.tree(self.olay, trees[s].parents, x[a:b], z[a:b], dt[a:b], B[a:b], C[a:b], conv0, h0)
            worst = max(worst, assert_close(g_out[a:b], o_out, TOL[cfg.act], f"round {rnd} seq {s}: node outputs"))
            slots = torch.arange(S + a, S + b, device="cuda")
            assert_close(self.cache.ssm[self.li, slots].cpu().numpy(), o_h, TOL_STATE, f"round {rnd} seq {s}: node states")
            assert np.array_equal(_f64(self.cache.conv[self.li, slots]), o_conv), "node conv windows are copies of raw inputs"
            committed[s] = (o_conv[accepted[s]], o_h[accepted[s]])
        src = i32([S + int(off[s]) + accepted[s] for s in range(S)])
        before = self.cache.ssm[self.li, src.long()].clone(), self.cache.conv[self.li, src.long()].clone()
        md.mdraft_state_commit(self.cache, src, i32(np.arange(S)), self.status)
        torch.cuda.synchronize()
        assert torch.equal(self.cache.ssm[self.li, :S].view(torch.int32), before[0].view(torch.int32)), "commit must be bit-exact"
        assert torch.equal(self.cache.conv[self.li, :S].view(torch.uint8), before[1].view(torch.uint8)), "commit must be bit-exact"
        return worst


def test_config0_tiny_fp32_everything():
    cfg = gen.get_config(0)
    p, lay, olay = _layer(cfg, 0)
    tree = gen.config_tree(cfg)
    L, M = cfg.context[0], tree.n_nodes
    cache = md.StateCache(1, 1 + M, cfg.d_inner, act=torch.float32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = gen.prefill_inputs(cfg, 0, L)
    out = _prefill(cfg, lay, cache, 0, ins, np.array([0, L]), [0], status)
    o_out, o_conv, o_h = oracle.prefill(olay, *ins)
    assert_close(_f64(out), o_out, TOL["f32"], "prefill out")
    assert_close(cache.ssm[0, 0].cpu().numpy(), o_h[0], TOL_STATE, "prefill state")
    assert np.array_equal(_f64(cache.conv[0, 0]), o_conv[0])
    committed = {0: (o_conv[0], o_h[0])}
    Drafting(cfg, lay, olay, cache, 0, 1, [0], status).round(0, committed)
    assert int(status.item()) == 0


@pytest.mark.parametrize("layer", [0, 11, 23])
def test_config1_prefill_2k_whole_layers(layer):
    cfg = gen.get_config(1)
    p, lay, olay = _layer(cfg, layer)
    assert lay.flags & md.MDRAFT_A_POWERS, "the S4D-real initialisation must be recognised on the device"
    L = cfg.context[0]
    cache = md.StateCache(1, 1, cfg.d_inner, act=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = gen.prefill_inputs(cfg, layer, L)
    out = _prefill(cfg, lay, cache, 0, ins, np.array([0, L]), [0], status)
    o_out, o_conv, o_h = oracle.prefill(olay, *ins)
    assert int(status.item()) == 0
    assert_close(_f64(out), o_out, TOL["bf16"], "out")
    assert_close(cache.ssm[0, 0].cpu().numpy(), o_h[0], TOL_STATE, "final state")
    assert np.array_equal(_f64(cache.conv[0, 0]), o_conv[0])


def test_config2_eight_draft_rounds_with_commits():
    cfg = gen.get_config(2)
    p, lay, olay = _layer(cfg, 3)
    L = cfg.context[0]
    cache = md.StateCache(1, 1 + 150, cfg.d_inner, act=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = gen.prefill_inputs(cfg, 3, L)
    _prefill(cfg, lay, cache, 0, ins, np.array([0, L]), [0], status)
    _, o_conv, o_h = oracle.prefill(olay, *ins)
    committed = {0: (o_conv[0], o_h[0])}
    d = Drafting(cfg, lay, olay, cache, 0, 1, [0], status)
    for rnd in range(cfg.rounds):
        d.round(rnd, committed)
    assert int(status.item()) == 0
    assert gen.config_tree(cfg, 0).n_nodes == 150


def test_config3_long_context_and_constant_decode_cost():
    cfg = gen.get_config(3)
    p, lay, olay = _layer(cfg, 5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    caches = {}
    for L in (2048, cfg.context[0]):
        cache = md.StateCache(1, 1, cfg.d_inner, act=torch.bfloat16)
        ins = gen.prefill_inputs(cfg, 5, L)
        out = _prefill(cfg, lay, cache, 0, ins, np.array([0, L]), [0], status)
        o_out, o_conv, o_h = oracle.prefill(olay, *ins)
        assert_close(_f64(out), o_out, TOL["bf16"], f"L={L}: out")
        assert_close(cache.ssm[0, 0].cpu().numpy(), o_h[0], TOL_STATE, f"L={L}: state")
        assert np.array_equal(_f64(cache.conv[0, 0]), o_conv[0])
        # 16 single-chain decode steps in place: the tree step with branching 1
        x, z, dt, B, C = gen.node_inputs(cfg, 5, 0, 16)
        t_out, _, t_h = oracle.tree(olay, np.arange(-1, 15), x, z, dt, B, C, o_conv[0], o_h[0])
        tdt = torch.bfloat16
        dev = [to_device(a, tdt) for a in (x, z, dt, B, C)]
        o = torch.empty((16, cfg.d_inner), dtype=tdt, device="cuda")
        zero = i32([0])
        for k in range(16):
            md.mdraft_tree_step(lay, cache, 0, *[a[k:k + 1] for a in dev], o[k:k + 1], zero, zero, None, status)
        torch.cuda.synchronize()
        assert_close(_f64(o), t_out, TOL["bf16"], f"L={L}: decode outputs")
        assert_close(cache.ssm[0, 0].cpu().numpy(), t_h[-1], TOL_STATE, f"L={L}: state after decode")
        caches[L] = cache
    # the state a decode step works on does not grow with the context (paper Section 3.1)
    assert caches[2048].nbytes() == caches[cfg.context[0]].nbytes() == cfg.d_inner * 16 * 4 + 3 * cfg.d_inner * 2
    assert int(status.item()) == 0


def test_config4_packed_batch_and_four_rounds():
    cfg = gen.get_config(4)
    p, lay, olay = _layer(cfg, 2)
    cu = gen.seq_lengths(cfg)
    S, T = cfg.n_seq, int(cu[-1])
    lens = np.diff(cu)
    assert S == 32 and lens.min() >= 1024 and lens.max() <= 8192
    watch = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 7, 20})   # shortest, longest and two more sequences
    cache = md.StateCache(1, S + 32 * S, cfg.d_inner, act=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = gen.prefill_inputs(cfg, 2, T)
    out = _prefill(cfg, lay, cache, 0, ins, cu, np.arange(S), status)
    g_out = _f64(out)
    committed = {}
    for s in watch:
        a, b = int(cu[s]), int(cu[s + 1])
        o_out, o_conv, o_h = oracle.prefill(olay, *[t[a:b] for t in ins])
        assert_close(g_out[a:b], o_out, TOL["bf16"], f"seq {s}: out")
        assert_close(cache.ssm[0, s].cpu().numpy(), o_h[0], TOL_STATE, f"seq {s}: state")
        assert np.array_equal(_f64(cache.conv[0, s]), o_conv[0])
        committed[s] = (o_conv[0], o_h[0])
    assert np.all(np.isfinite(g_out)), "every packed sequence must have been written"
    d = Drafting(cfg, lay, olay, cache, 0, S, watch, status)
    for rnd in range(cfg.rounds):
        d.round(rnd, committed)
    assert int(status.item()) == 0


def test_tree_search_drives_changing_tree_shapes():
    """Section 4.2 end to end on the device path: a UCB bandit picks one of the paper's three tree configurations per
    round, a synthetic verifier accepts a prefix of a random root-to-leaf path, the accepted node is committed, and
    every round's node outputs and states are checked against the oracle.  The library's bandit and the oracle's
    must take the same decisions."""
    from oracle import tree_search as ots
    configs = [(3, 3, 2, 1), (3, 2, 2, 1, 1), (2, 2, 2, 1, 1, 1)]
    cfg = gen.Config(2, "search", 1, 1536, 16, 4, "bf16", 1, (512, 512), "none", 12, 5)
    p, lay, olay = _layer(cfg, 1)
    L = cfg.context[0]
    max_nodes = max(gen.paper_tree(c).n_nodes for c in configs)
    cache = md.StateCache(1, 1 + max_nodes, cfg.d_inner, act=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ins = gen.prefill_inputs(cfg, 1, L)
    _prefill(cfg, lay, cache, 0, ins, np.array([0, L]), [0], status)
    _, o_conv, o_h = oracle.prefill(olay, *ins)
    committed = {0: (o_conv[0], o_h[0])}
    d = Drafting(cfg, lay, olay, cache, 0, 1, [0], status)
    lib_b, ora_b = md.UcbBandit(3, 1.0, 0.05), ots.Bandit(3, 1.0, 0.05)
    g = np.random.default_rng(3)
    played = []
    for rnd in range(cfg.rounds):
        k = lib_b.mdraft_ucb_select()
        assert k == ora_b.select()
        tree = gen.paper_tree(configs[k])
        ch, v, n_acc = tree.children(), 0, 1          # the root is the last verified token; walk down while accepted
        while ch[v] and g.random() < 0.6:
            v = ch[v][int(g.integers(0, len(ch[v])))]
            n_acc += 1
        d.round(rnd, committed, trees=[tree], accepted=[v])
        lib_b.mdraft_ucb_update(k, len(configs[k]), n_acc)
        ora_b.update(k, len(configs[k]), n_acc)
        played.append(k)
    assert int(status.item()) == 0
    assert set(played[:3]) == {0, 1, 2} and lib_b.count == ora_b.n and lib_b.reward_sum == ora_b.r_sum
