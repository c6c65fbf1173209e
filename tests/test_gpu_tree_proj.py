"""Tree step with the block's own selection projections against the oracle's projection tree (every node rebuilt
along its root-to-node path in fp64), plus the bit-exactness properties of its index work."""

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


class ProjRig:
    """One layer, one sequence: committed state in slot 0, node i in slot 1+i."""

    def __init__(self, cfg, tree, dt_rank, conv_bias=True, general_A=True, flags=md.MDRAFT_DT_SOFTPLUS, seed_state=5, nodes_per_cluster=0):
        self.cfg, self.tree, self.flags, self.nodes_per_cluster = cfg, tree, flags, nodes_per_cluster
        self.tdt = torch_act(cfg.act)
        self.params = gen.layer_params(cfg, 0, conv_bias=conv_bias, general_A=general_A)
        self.lay = upload_layer(self.params, cfg.act, flags)
        self.W_x, self.W_dt = gen.select_proj(cfg, 0, dt_rank)
        self.dW_x, self.dW_dt = to_device(self.W_x, self.tdt), to_device(self.W_dt, self.tdt)
        M, Dn = tree.n_nodes, cfg.d_inner
        self.x, self.z, _, _, _ = gen.node_inputs(cfg, 0, 0, M)
        g = np.random.default_rng(seed_state)
        self.h0 = g.normal(size=(Dn, 16)).astype(np.float32)
        self.c0 = gen.round_to_act(g.normal(size=(3, Dn)).astype(np.float32), cfg.act)
        self.cache = md.StateCache(1, 1 + M, Dn, act=self.tdt)
        self.reset()
        self.dx, self.dz = to_device(self.x, self.tdt), to_device(self.z, self.tdt)
        self.parent_slot = np.where(tree.parents < 0, 0, tree.parents + 1).astype(np.int32)
        self.node_slot = (np.arange(M) + 1).astype(np.int32)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def reset(self):
        self.cache.ssm.fill_(float("nan"))
        self.cache.conv.fill_(float("nan"))
        self.cache.ssm[0, 0] = torch.from_numpy(self.h0).cuda()
        self.cache.conv[0, 0] = to_device(self.c0, self.tdt)

    def step(self, idx):
        t = torch.from_numpy(np.asarray(idx)).cuda()
        out = torch.full((len(idx), self.cfg.d_inner), float("nan"), dtype=self.tdt, device="cuda")
        md.mdraft_tree_step_proj(self.lay, self.cache, 0, self.dW_x, self.dW_dt, self.dx[t].contiguous(), self.dz[t].contiguous(),
                                 out, i32(self.parent_slot[idx]), i32(self.node_slot[idx]), self.status,
                                 nodes_per_cluster=self.nodes_per_cluster)
        torch.cuda.synchronize()
        return out

    def run_levels(self, rng=None):
        outs = torch.empty((self.tree.n_nodes, self.cfg.d_inner), dtype=self.tdt, device="cuda")
        for lo, hi in zip(self.tree.level_offsets[:-1], self.tree.level_offsets[1:]):
            idx = np.arange(lo, hi) if rng is None else rng.permutation(np.arange(lo, hi))
            outs[torch.from_numpy(idx).cuda()] = self.step(idx)
        return outs

    def oracle(self):
        lay = oracle.layer_from_params(self.params, parity.oracle_flags(self.flags))
        return oracle.tree_proj(lay, self.W_x, self.W_dt, self.tree.parents, self.x, self.z, self.c0, self.h0)

    def states(self):
        s = torch.from_numpy(self.node_slot.astype(np.int64)).cuda()
        return self.cache.ssm[0, s].cpu().numpy(), self.cache.conv[0, s].float().cpu().numpy()


TREES = {"cfg0": lambda: gen.full_tree([2, 2, 2]), "paper32211": lambda: gen.paper_tree((3, 2, 2, 1, 1)),
         "paper3321": lambda: gen.paper_tree((3, 3, 2, 1)), "rand32": lambda: gen.random_branching_tree(32, 5, 1),
         "chain": lambda: gen.chain_tree(7)}


# Widths chosen to meet every block width (128 / 256 / 512 channels), cluster sizes 1..8 and ragged last blocks.
@pytest.mark.parametrize("act,Dn,R,shape", [
    ("f32", 64, 8, "cfg0"), ("bf16", 64, 8, "cfg0"), ("f32", 200, 16, "paper32211"), ("bf16", 136, 8, "rand32"),
    ("bf16", 1024, 32, "chain"), ("bf16", 1536, 48, "paper3321"), ("f32", 1536, 48, "chain"), ("bf16", 2048, 64, "cfg0"),
    ("bf16", 2560, 160, "chain"), ("f32", 4096, 256, "chain"), ("bf16", 3976, 24, "cfg0"),
])
def test_projection_tree_matches_oracle(act, Dn, R, shape):
    cfg = parity.small_config(Dn, act)
    rig = ProjRig(cfg, TREES[shape](), R)
    out = rig.run_levels()
    assert int(rig.status.item()) == 0
    o_out, o_conv, o_h, _, _, _ = rig.oracle()
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs")
    h, conv = rig.states()
    assert_close(h, o_h, TOL_STATE, "node SSM states")
    assert np.array_equal(conv.astype(np.float64), o_conv), "node conv windows are copies of raw inputs"


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_structured_A_fast_path_and_plain_step_size(act):
    cfg = parity.small_config(1536, act)
    for flags in (md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_A_POWERS, md.MDRAFT_A_POWERS, 0):
        rig = ProjRig(cfg, gen.paper_tree((3, 2, 2, 1, 1)), 48, conv_bias=False, general_A=False, flags=flags)
        if not (flags & md.MDRAFT_DT_SOFTPLUS):
            rig.params.dt_bias[:] = 0.05   # a raw step size must stay positive: bias well above the projected spread
            rig.W_dt *= 0.02
            rig.W_dt = gen.round_to_act(rig.W_dt, act)
            rig.dW_dt = to_device(rig.W_dt, rig.tdt)
            rig.lay = upload_layer(rig.params, cfg.act, flags)
        out = rig.run_levels()
        assert int(rig.status.item()) == 0
        o_out, _, o_h, _, _, _ = rig.oracle()
        assert_close(out.float().cpu().numpy(), o_out, TOL[act], f"node outputs (flags {flags})")
        assert_close(rig.states()[0], o_h, TOL_STATE, f"node SSM states (flags {flags})")


@pytest.mark.parametrize("act,Dn,R", [("bf16", 1536, 48), ("f32", 200, 16), ("bf16", 1024, 96), ("f32", 2048, 64)])
def test_nodes_per_cluster_changes_no_bit_and_matches_oracle(act, Dn, R):
    """Levels of 1, 3, 9, 18 nodes (ragged against groups of 2 and 4) with 1, 2 and 4 nodes per cluster."""
    cfg = parity.small_config(Dn, act)
    tree = gen.paper_tree((3, 3, 2))
    ref = None
    for npc in (1, 2, 4):
        rig = ProjRig(cfg, tree, R, nodes_per_cluster=npc)
        out = rig.run_levels()
        assert int(rig.status.item()) == 0
        h, conv = rig.states()
        if ref is None:
            ref = (out, h, conv)
            o_out, o_conv, o_h, _, _, _ = rig.oracle()
            assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs")
            assert_close(h, o_h, TOL_STATE, "node SSM states")
        else:
            assert torch.equal(out, ref[0]) and np.array_equal(h, ref[1]) and np.array_equal(conv, ref[2]), f"{npc} nodes per cluster"


def test_wide_level_takes_the_grouped_path_by_itself():
    """300 children of the committed state: the library's own choice groups nodes; every node still equals the oracle's."""
    cfg = parity.small_config(1536, "bf16")
    tree = gen.full_tree([300])
    rig = ProjRig(cfg, tree, 48, general_A=False, flags=md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_A_POWERS)
    out = rig.run_levels()
    assert int(rig.status.item()) == 0
    o_out, _, o_h, _, _, _ = rig.oracle()
    assert_close(out.float().cpu().numpy(), o_out, TOL["bf16"], "node outputs")
    assert_close(rig.states()[0], o_h, TOL_STATE, "node SSM states")


def test_node_order_within_a_level_changes_no_bit():
    cfg = parity.small_config(1536, "bf16")
    rig = ProjRig(cfg, gen.random_branching_tree(32, 5, 2), 48)
    a = rig.run_levels()
    ha, ca = rig.states()
    rig.reset()
    b = rig.run_levels(np.random.default_rng(0))
    hb, cb = rig.states()
    assert torch.equal(a, b) and np.array_equal(ha, hb) and np.array_equal(ca, cb)


def test_matches_the_split_mode_calls():
    """conv-only step, projections in torch fp32, pre-convolved step: the fused call agrees within the bf16 rounding the
    split path applies to u, dt, B and C on the way."""
    cfg = parity.small_config(1536, "bf16")
    rig = ProjRig(cfg, gen.full_tree([3, 2]), 48, general_A=False, flags=md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_A_POWERS)
    fused = rig.run_levels()
    hf, _ = rig.states()
    rig.reset()
    M, Dn, R = rig.tree.n_nodes, cfg.d_inner, 48
    outs = torch.empty_like(fused)
    for lo, hi in zip(rig.tree.level_offsets[:-1], rig.tree.level_offsets[1:]):
        ps, ns = i32(rig.parent_slot[lo:hi]), i32(rig.node_slot[lo:hi])
        u = torch.empty((hi - lo, Dn), dtype=rig.tdt, device="cuda")
        md.mdraft_tree_step(rig.lay, rig.cache, 0, rig.dx[lo:hi], None, None, None, None, u, ps, ns, None, rig.status, flags=md.MDRAFT_CONV_ONLY)
        s = u.float() @ rig.dW_x.float().T
        dt = (s[:, :R] @ rig.dW_dt.float().T).to(rig.tdt)
        Bm, Cm = s[:, R:R + 16].to(rig.tdt).contiguous(), s[:, R + 16:].to(rig.tdt).contiguous()
        md.mdraft_tree_step(rig.lay, rig.cache, 0, u, rig.dz[lo:hi], dt, Bm, Cm, outs[lo:hi], ps, ns, None, rig.status,
                            flags=md.MDRAFT_DT_SOFTPLUS | md.MDRAFT_PRECONV | md.MDRAFT_A_POWERS)
    torch.cuda.synchronize()
    assert int(rig.status.item()) == 0
    assert_close(fused.float().cpu().numpy(), outs.float().cpu().numpy(), 3 * TOL["bf16"], "fused vs split outputs")
    assert_close(hf, rig.states()[0], 3 * TOL["bf16"], "fused vs split states")


def test_bad_slot_is_reported_and_skipped():
    cfg = parity.small_config(256, "f32")
    rig = ProjRig(cfg, gen.full_tree([2]), 8, nodes_per_cluster=2)
    rig.node_slot[2] = rig.cache.n_slots + 3
    rig.step(np.arange(1))
    assert int(rig.status.item()) == 0
    out = rig.step(np.arange(1, 3))
    assert int(rig.status.item()) & md.MDRAFT_DEV_BAD_SLOT
    assert torch.isnan(out[1]).all() and not torch.isnan(out[0]).any()


def test_argument_checks():
    cfg = parity.small_config(256, "bf16")
    rig = ProjRig(cfg, gen.full_tree([2]), 8)
    out = torch.empty((1, 256), dtype=rig.tdt, device="cuda")
    one = (rig.dx[:1], rig.dz[:1], out, i32([0]), i32([1]), rig.status)
    with pytest.raises(md.MdraftError) as e:
        md.mdraft_tree_step_proj(rig.lay, rig.cache, 0, rig.dW_x, rig.dW_dt, *one, flags=md.MDRAFT_PRECONV)
    assert e.value.status == -1
    W_x12 = torch.zeros((12 + 32, 256), dtype=rig.tdt, device="cuda"); W_dt12 = torch.zeros((256, 12), dtype=rig.tdt, device="cuda")
    with pytest.raises(md.MdraftError) as e:
        md.mdraft_tree_step_proj(rig.lay, rig.cache, 0, W_x12, W_dt12, *one)
    assert e.value.status == -2
    with pytest.raises(ValueError):
        md.mdraft_tree_step_proj(rig.lay, rig.cache, 0, rig.dW_dt, rig.dW_x, *one)
    with pytest.raises(md.MdraftError) as e:
        md.mdraft_tree_step_proj(rig.lay, rig.cache, 0, rig.dW_x, rig.dW_dt, *one, nodes_per_cluster=3)
    assert e.value.status == -1
    with pytest.raises(md.MdraftError) as e:   # weights must start on a 16-byte boundary
        md.mdraft_tree_step_proj(rig.lay, rig.cache, 0, torch.zeros(40 * 256 + 1, dtype=rig.tdt, device="cuda")[1:].view(40, 256), rig.dW_dt, *one)
    assert e.value.status == -3
    wide = parity.small_config(4104, "bf16")
    lay = upload_layer(gen.layer_params(wide, 0), "bf16", md.MDRAFT_DT_SOFTPLUS)
    cache = md.StateCache(1, 2, 4104, act=rig.tdt)
    xw = torch.zeros((1, 4104), dtype=rig.tdt, device="cuda")
    with pytest.raises(md.MdraftError) as e:
        md.mdraft_tree_step_proj(lay, cache, 0, torch.zeros((40, 4104), dtype=rig.tdt, device="cuda"),
                                 torch.zeros((4104, 8), dtype=rig.tdt, device="cuda"), xw, xw, torch.empty_like(xw), i32([0]), i32([1]))
    assert e.value.status == -2
