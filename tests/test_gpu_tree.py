"""Tree step and commit against the oracle (every node = its root-to-node path) and against the bit-exactness
properties that index work must have."""

import numpy as np
import pytest
import torch

import gen
import oracle
import parity
from parity import TOL, TOL_STATE, assert_close

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer


class TreeRig:
    """One layer, one sequence: committed state in slot 0, node i in slot 1+i."""

    def __init__(self, cfg, tree, conv_bias=True, general_A=True, seed_state=3, flags=md.MDRAFT_DT_SOFTPLUS, extra_slots=4):
        self.cfg, self.tree, self.flags = cfg, tree, flags
        self.tdt = torch_act(cfg.act)
        self.params = gen.layer_params(cfg, 0, conv_bias=conv_bias, general_A=general_A)
        self.lay = upload_layer(self.params, cfg.act, flags)
        M, Dn = tree.n_nodes, cfg.d_inner
        self.x, self.z, self.dt, self.B, self.C = gen.node_inputs(cfg, 0, 0, M)
        g = np.random.default_rng(seed_state)
        self.h0 = g.normal(size=(Dn, 16)).astype(np.float32)
        self.c0 = gen.round_to_act(g.normal(size=(3, Dn)).astype(np.float32), cfg.act)
        self.cache = md.StateCache(1, 1 + M + extra_slots, Dn, act=self.tdt)
        self.reset()
        self.dev = [to_device(a, self.tdt) for a in (self.x, self.z, self.dt, self.B, self.C)]
        self.parent_slot = np.where(tree.parents < 0, 0, tree.parents + 1).astype(np.int32)
        self.node_slot = (np.arange(M) + 1).astype(np.int32)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def reset(self):
        self.cache.ssm.fill_(float("nan"))
        self.cache.conv.fill_(float("nan"))
        self.cache.ssm[0, 0] = torch.from_numpy(self.h0).cuda()
        self.cache.conv[0, 0] = to_device(self.c0, self.tdt)

    def step(self, lo, hi, level_offsets=None, order=None):
        """Run nodes [lo, hi) (optionally permuted by ``order``) in one call."""
        idx = np.arange(lo, hi) if order is None else np.asarray(order)
        t = torch.from_numpy(idx).cuda()
        args = [a[t].contiguous() for a in self.dev]
        out = torch.full((len(idx), self.cfg.d_inner), float("nan"), dtype=self.tdt, device="cuda")
        md.mdraft_tree_step(self.lay, self.cache, 0, *args, out, i32(self.parent_slot[idx]), i32(self.node_slot[idx]),
                            level_offsets, self.status)
        torch.cuda.synchronize()
        return out

    def run_levels(self):
        outs = [self.step(int(a), int(b)) for a, b in zip(self.tree.level_offsets[:-1], self.tree.level_offsets[1:])]
        return torch.cat(outs)

    def oracle(self):
        lay = oracle.layer_from_params(self.params, parity.oracle_flags(self.flags))
        return oracle.tree(lay, self.tree.parents, self.x, self.z, self.dt, self.B, self.C, self.c0, self.h0)

    def states(self):
        s = torch.from_numpy(self.node_slot.astype(np.int64)).cuda()
        return self.cache.ssm[0, s].cpu().numpy(), self.cache.conv[0, s].float().cpu().numpy()


@pytest.mark.parametrize("act,Dn,shape", [
    ("f32", 64, "cfg0"), ("bf16", 64, "cfg0"), ("f32", 200, "paper32211"), ("bf16", 1536, "paper3321"),
    ("bf16", 136, "rand32"), ("f32", 72, "chain"),
])
def test_tree_matches_oracle(act, Dn, shape):
    cfg = parity.small_config(Dn, act)
    tree = {"cfg0": gen.full_tree([2, 2, 2]), "paper32211": gen.paper_tree((3, 2, 2, 1, 1)),
            "paper3321": gen.paper_tree((3, 3, 2, 1)), "rand32": gen.random_branching_tree(32, 5, 1),
            "chain": gen.chain_tree(9)}[shape]
    rig = TreeRig(cfg, tree)
    out = rig.run_levels()
    assert int(rig.status.item()) == 0
    o_out, o_conv, o_h = rig.oracle()
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs")
    h, conv = rig.states()
    assert_close(h, o_h, TOL_STATE, "node SSM states")
    assert np.array_equal(conv.astype(np.float64), o_conv), "node conv windows are copies of raw inputs"


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_levels_in_one_call_equal_level_by_level_bitwise(act):
    cfg = parity.small_config(200, act)
    tree = gen.paper_tree((3, 2, 2, 1, 1))
    rig = TreeRig(cfg, tree)
    a = rig.run_levels()
    ha, ca = rig.states()
    rig.reset()
    b = rig.step(0, tree.n_nodes, level_offsets=[int(v) for v in tree.level_offsets])
    hb, cb = rig.states()
    assert torch.equal(a, b) and np.array_equal(ha, hb) and np.array_equal(ca, cb)


def test_node_order_within_a_level_changes_no_bit():
    cfg = parity.small_config(136, "bf16")
    tree = gen.random_branching_tree(32, 5, 2)
    rig = TreeRig(cfg, tree)
    a = rig.run_levels()
    ha, ca = rig.states()
    rig.reset()
    g = np.random.default_rng(0)
    outs = torch.empty_like(a)
    for lo, hi in zip(tree.level_offsets[:-1], tree.level_offsets[1:]):
        order = g.permutation(np.arange(lo, hi))  # breaks up sibling runs as well
        o = rig.step(lo, hi, order=order)
        outs[torch.from_numpy(order).cuda()] = o
    hb, cb = rig.states()
    assert torch.equal(a, outs) and np.array_equal(ha, hb) and np.array_equal(ca, cb)


def test_twin_siblings_and_copied_parent_give_identical_bits():
    cfg = parity.small_config(128, "f32")
    tree = gen.full_tree([3])
    rig = TreeRig(cfg, tree)
    for arr in (rig.x, rig.z, rig.dt, rig.B, rig.C):
        arr[2] = arr[1]
    rig.dev = [to_device(a, rig.tdt) for a in (rig.x, rig.z, rig.dt, rig.B, rig.C)]
    out = rig.run_levels()
    h, conv = rig.states()
    assert torch.equal(out[1], out[2]) and np.array_equal(h[1], h[2]) and np.array_equal(conv[1], conv[2])
    # a child computed from a byte copy of the parent slot equals the child computed from the parent slot
    spare = rig.cache.n_slots - 1
    md.mdraft_state_commit(rig.cache, i32([1]), i32([spare]))   # slot 1 = the root node's state
    o2 = torch.empty((1, 128), device="cuda")
    args = [a[3:4].contiguous() for a in rig.dev]
    md.mdraft_tree_step(rig.lay, rig.cache, 0, *args, o2, i32([spare]), i32([spare - 1]), None, rig.status)
    torch.cuda.synchronize()
    assert torch.equal(o2[0], out[3])
    assert torch.equal(rig.cache.ssm[0, spare - 1], rig.cache.ssm[0, 4])


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_in_place_chain_decode_equals_longer_prefill(act):
    """prefill(L+k) == prefill(L) then k single-node steps that overwrite the sequence's own slot."""
    cfg = parity.small_config(136, act)
    L, k = 90, 6
    prob = parity.make_problem(cfg, [L + k], conv_bias=True, general_A=True)
    lay_o = oracle.layer_from_params(prob.params)
    o_out, o_conv, o_h = oracle.prefill(lay_o, prob.x, prob.z, prob.dt, prob.B, prob.C)
    tdt = torch_act(act)
    lay = upload_layer(prob.params, act)
    cache = md.StateCache(1, 1, 136, act=tdt)
    dev = [to_device(a, tdt) for a in (prob.x, prob.z, prob.dt, prob.B, prob.C)]
    out = torch.empty((L + k, 136), dtype=tdt, device="cuda")
    zero = i32([0])
    ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lay, L, 1, L, 32)), dtype=torch.uint8, device="cuda")
    md.mdraft_conv_scan_prefill(lay, cache, 0, *[a[:L] for a in dev], out[:L], i32([0, L]), L, None, zero, ws, 32)
    for t in range(L, L + k):
        md.mdraft_tree_step(lay, cache, 0, *[a[t:t + 1] for a in dev], out[t:t + 1], zero, zero)
    torch.cuda.synchronize()
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "prefill + chain")
    assert_close(cache.ssm[0, 0].cpu().numpy(), o_h[0], TOL_STATE, "state after the chain")
    assert np.array_equal(cache.conv[0, 0].float().cpu().numpy().astype(np.float64), o_conv[0])


def test_commit_is_a_bit_exact_indexed_copy():
    g = torch.Generator(device="cuda").manual_seed(1)
    cache = md.StateCache(3, 10, 136, act=torch.bfloat16)
    cache.ssm.copy_(torch.randn(cache.ssm.shape, generator=g, device="cuda"))
    cache.conv.copy_(torch.randn(cache.conv.shape, generator=g, device="cuda"))
    # include NaN / inf / -0 bit patterns: a copy must not canonicalise anything
    cache.ssm[1, 7, 0, :4] = torch.tensor([float("nan"), float("inf"), -0.0, 1e-42], device="cuda")
    ssm0, conv0 = cache.ssm.clone(), cache.conv.clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_state_commit(cache, i32([7, 4, 9, 3]), i32([0, 1, 9, 2]), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    exp_ssm, exp_conv = ssm0.clone(), conv0.clone()
    for s, d in ((7, 0), (4, 1), (3, 2)):
        exp_ssm[:, d] = ssm0[:, s]; exp_conv[:, d] = conv0[:, s]
    assert torch.equal(cache.ssm.view(torch.int32), exp_ssm.view(torch.int32))
    assert torch.equal(cache.conv.view(torch.int16), exp_conv.view(torch.int16))
    md.mdraft_state_commit(cache, i32([5, 77]), i32([-1, 3]), status)
    torch.cuda.synchronize()
    assert int(status.item()) & md.MDRAFT_DEV_BAD_SLOT
    assert torch.equal(cache.ssm.view(torch.int32), exp_ssm.view(torch.int32)), "bad indices must copy nothing"


def test_tree_step_bad_slots_are_skipped_and_flagged():
    cfg = parity.small_config(64, "f32")
    rig = TreeRig(cfg, gen.full_tree([4]))
    rig.parent_slot[2] = 10_000
    rig.node_slot[4] = -3
    out = rig.run_levels()
    assert int(rig.status.item()) & md.MDRAFT_DEV_BAD_SLOT
    o = out.float().cpu().numpy()
    assert np.all(np.isnan(o[2])) and np.all(np.isnan(o[4])), "skipped nodes write nothing"
    assert np.all(np.isfinite(o[[0, 1, 3]]))


def test_round_graph_cache_replays_what_eager_launches_compute():
    """One captured graph per tree shape (the paper caches one per batch size, Section 4.1): a replay with new inputs,
    new slot indices and another accepted node must give, bit for bit, what the same round gives launched eagerly."""
    from paper_2506_01206_b200.stack import DrafterStack, RoundGraphCache
    cfg = parity.small_config(264, "bf16")
    n_layers = 3
    params = [gen.layer_params(cfg, l, conv_bias=True, general_A=True) for l in range(n_layers)]
    tdt = torch.bfloat16

    def fresh_stack():
        st = DrafterStack([upload_layer(p, "bf16") for p in params], 1 + 48, 16, 1, 16)
        g = torch.Generator(device="cuda").manual_seed(7)
        st.cache.ssm[:, 0] = torch.randn(st.cache.ssm[:, 0].shape, generator=g, device="cuda")
        st.cache.conv[:, 0] = torch.randn(st.cache.conv[:, 0].shape, generator=g, device="cuda").to(tdt)
        return st

    shapes = [gen.paper_tree((3, 2, 2, 1, 1)), gen.paper_tree((2, 2, 2, 1, 1, 1)), gen.paper_tree((3, 2, 2, 1, 1))]
    graph_stack, eager_stack = fresh_stack(), fresh_stack()
    cache = RoundGraphCache(graph_stack, max_nodes=48)
    replayed = []
    for rnd, tree in enumerate(shapes):
        M = tree.n_nodes
        levels = [int(v) for v in tree.level_offsets]
        parent = i32(np.where(tree.parents < 0, 0, tree.parents + 1))
        nodes = i32(np.arange(M) + 1)
        accepted = i32([1 + gen.random_accepted_node(tree, 0, 93, rnd)])
        ins = [[to_device(a, tdt) for a in gen.node_inputs(cfg, l, rnd, M)] for l in range(n_layers)]
        for l in range(n_layers):
            for buf, a in zip((cache.x[l], cache.z[l], cache.dt[l], cache.B[l], cache.C[l]), ins[l]):
                buf[:M].copy_(a)
        cache.parent_slot[:M].copy_(parent); cache.node_slot[:M].copy_(nodes); cache.accepted_slot.copy_(accepted)
        replayed.append(cache.run(levels))
        outs = [torch.empty((M, 264), dtype=tdt, device="cuda") for _ in range(n_layers)]
        eager_stack.tree_round(ins, outs, parent, nodes, levels)
        eager_stack.commit(accepted, i32([0]))
        torch.cuda.synchronize()
        for l in range(n_layers):
            assert torch.equal(cache.out[l][:M], outs[l])
        assert torch.equal(graph_stack.cache.ssm.view(torch.int32), eager_stack.cache.ssm.view(torch.int32))
        assert torch.equal(graph_stack.cache.conv.view(torch.int16), eager_stack.cache.conv.view(torch.int16))
    assert replayed == [False, False, True] and len(cache) == 2
    graph_stack.check_status(); eager_stack.check_status()


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_chained_launches_keep_their_order_when_buffers_are_shared(act):
    """Levels of one call start while the level ahead still runs.  Two arrangements in which a late read would show:
    (a) `out` is the same buffer as `x` (every node overwrites its own input row), all levels in one call;
    (b) a conv-only call whose output is the very next call's pre-convolved input, nothing in between.
    Both, replayed many times from one CUDA graph, must give the bits of the level-by-level run."""
    cfg = parity.small_config(392, act)
    tree = gen.paper_tree((3, 2, 2, 1, 1))
    rig = TreeRig(cfg, tree)
    ref = rig.run_levels()
    h_ref, c_ref = rig.states()
    lv = [int(v) for v in tree.level_offsets]
    par, nod = i32(rig.parent_slot), i32(rig.node_slot)
    x0 = rig.dev[0].clone()
    xio = rig.dev[0].clone()
    u = torch.empty_like(x0); y = torch.empty_like(x0)

    def in_place():
        xio.copy_(x0)
        md.mdraft_tree_step(rig.lay, rig.cache, 0, xio, rig.dev[1], rig.dev[2], rig.dev[3], rig.dev[4], xio, par, nod, lv, rig.status)

    def split():
        md.mdraft_tree_step(rig.lay, rig.cache, 0, x0, None, None, None, None, u, par, nod, lv, rig.status, flags=md.MDRAFT_CONV_ONLY)
        md.mdraft_tree_step(rig.lay, rig.cache, 0, u, rig.dev[1], rig.dev[2], rig.dev[3], rig.dev[4], y, par, nod, lv, rig.status,
                            flags=md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_PRECONV)

    for fn, result in ((in_place, xio), (split, y)):
        rig.reset()
        fn(); torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        for _ in range(20):
            rig.reset()
            g.replay()
        torch.cuda.synchronize()
        assert int(rig.status.item()) == 0
        h, c = rig.states()
        if fn is in_place:
            assert torch.equal(result, ref) and np.array_equal(h, h_ref) and np.array_equal(c, c_ref)
        else:   # split mode rounds u to the activation dtype on the way: equal within tolerance, states likewise
            assert_close(result.float().cpu().numpy(), ref.float().cpu().numpy(), 3 * TOL[act], "split-mode chain")
            assert_close(h, h_ref, 3 * TOL[act], "split-mode chain states")
