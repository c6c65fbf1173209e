"""Seeded random sweep of the prefill over shapes, modes, chunk plans, block widths and slot arrangements, and of the
tree step (plain and with the projections inside) over random trees, each case against the fp64 oracle.  The cases are small (the oracle takes milliseconds)
but cross every tile, chunk and block boundary in many different ways."""

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


def _case(seed):
    g = np.random.default_rng(seed)
    act = "bf16" if g.random() < 0.6 else "f32"
    Dn = int(g.choice([8, 64, 72, 128, 136, 256, 392, 512, 520, 648, 1032]))
    S = int(g.integers(1, 6))
    lens = [int(v) for v in g.choice([0, 1, 2, 3, 4, 5, 15, 16, 17, 31, 33, 47, 64, 100, 130, 257], size=S)]
    if sum(lens) == 0:
        lens[0] = 9
    mode = g.choice(["fused", "fused", "conv_only", "preconv"])
    chunk = int(g.choice([0, 4, 7, 16, 33, 64, 500]))
    block = int(g.choice([0, 128, 512]))
    return dict(act=act, Dn=Dn, lens=lens, mode=str(mode), chunk=chunk, block=block, general_A=bool(g.random() < 0.5),
                conv_bias=bool(g.random() < 0.5), softplus=bool(g.random() < 0.8), init=str(g.choice(["none", "slots", "in_place", "mixed"])),
                powers_hint=bool(g.random() < 0.5), no_offsets=bool(S == 1 and g.random() < 0.5), seed=seed)


@pytest.mark.parametrize("seed", range(60))
def test_random_prefill_case(seed):
    c = _case(seed)
    cfg = parity.small_config(c["Dn"], c["act"], len(c["lens"]), cid=91, seed=seed)
    prob = parity.make_problem(cfg, c["lens"], conv_bias=c["conv_bias"], general_A=c["general_A"])
    S, T, Dn = len(c["lens"]), sum(c["lens"]), c["Dn"]
    tdt = torch_act(c["act"])
    flags = (md.MDRAFT_DT_SOFTPLUS if c["softplus"] else 0) | {"fused": 0, "conv_only": md.MDRAFT_CONV_ONLY, "preconv": md.MDRAFT_PRECONV}[c["mode"]]
    if not c["softplus"]:
        prob.dt = np.abs(prob.dt) * np.float32(0.05)   # a step size given as such must be non-negative
        prob.dt = gen.round_to_act(prob.dt, c["act"])
        prob.params.dt_bias[:] = 0
    gflags = flags | (md.MDRAFT_A_POWERS if (c["powers_hint"] and not c["general_A"]) else 0)
    g = np.random.default_rng(1000 + seed)
    h0 = g.normal(size=(S, Dn, 16)).astype(np.float32)
    c0 = gen.round_to_act(g.normal(size=(S, 3, Dn)).astype(np.float32), c["act"])
    if c["init"] == "none":
        init = None
    elif c["init"] == "mixed":
        init = np.where(g.random(S) < 0.5, np.arange(S), -1)
    else:
        init = np.arange(S)
    final = np.arange(S) if c["init"] == "in_place" else np.arange(S, 2 * S)
    if g.random() < 0.3:
        final = np.where(g.random(S) < 0.5, final, -1)
    cache = md.StateCache(1, 2 * S, Dn, act=tdt)
    cache.ssm[0, :S] = torch.from_numpy(h0).cuda()
    cache.conv[0, :S] = to_device(c0, tdt)
    before = cache.ssm.clone(), cache.conv.clone()
    lay = upload_layer(prob.params, c["act"], gflags)
    dev = [to_device(a, tdt) for a in (prob.x, prob.z, prob.dt, prob.B, prob.C)]
    out = torch.full((T, Dn), float("nan"), dtype=tdt, device="cuda")
    opts = (c["chunk"], c["block"])
    max_len = max(c["lens"])
    ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lay, T, S, max_len, opts)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cu = None if c["no_offsets"] else i32(prob.cu)
    md.mdraft_conv_scan_prefill(lay, cache, 0, *dev, out, cu, max_len, None if init is None else i32(init), i32(final), ws, opts, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, c

    has = np.zeros(S, bool) if init is None else (np.asarray(init) >= 0)
    ci = np.where(has[:, None, None], c0.astype(np.float64), 0.0)
    hi = np.where(has[:, None, None], h0.astype(np.float64), 0.0)
    olay = oracle.layer_from_params(prob.params, parity.oracle_flags(flags))
    o_out, o_conv, o_h = oracle.prefill(olay, prob.x, prob.z, prob.dt, prob.B, prob.C, prob.cu, ci, hi)
    if T:
        assert_close(out.float().cpu().numpy(), o_out, TOL[c["act"]], f"out {c}")
    for s in range(S):
        f = int(final[s])
        if f < 0:
            continue
        if c["mode"] != "conv_only":
            assert_close(cache.ssm[0, f].cpu().numpy(), o_h[s], TOL_STATE, f"state of sequence {s} {c}")
        if c["mode"] != "preconv":
            assert np.array_equal(cache.conv[0, f].float().cpu().numpy().astype(np.float64), o_conv[s]), f"window of sequence {s} {c}"
    untouched = [k for k in range(2 * S) if k not in set(int(v) for v in final if v >= 0)]
    for k in untouched:
        same = torch.equal(cache.ssm[0, k], before[0][0, k]) and torch.equal(cache.conv[0, k].view(torch.uint8), before[1][0, k].view(torch.uint8))
        assert same, f"slot {k} is nobody's final slot and must not change {c}"


@pytest.mark.parametrize("seed", range(20))
def test_random_tree_case(seed):
    g = np.random.default_rng(500 + seed)
    act = "bf16" if g.random() < 0.6 else "f32"
    Dn = int(g.choice([8, 72, 128, 136, 392, 520]))
    n_levels = int(g.integers(1, 6))
    n_nodes = min(int(g.integers(n_levels, 4 * n_levels + 1)), 1 + 4 * (n_levels - 1))   # what a tree of that depth can hold for sure
    tree = gen.random_branching_tree(n_nodes, n_levels, seed, max_children=4) if n_levels > 1 else gen.chain_tree(1)
    mode = str(g.choice(["fused", "fused", "conv_only", "preconv"]))
    cfg = parity.small_config(Dn, act, cid=92, seed=seed)
    params = gen.layer_params(cfg, 0, conv_bias=bool(g.random() < 0.5), general_A=bool(g.random() < 0.5))
    flags = md.MDRAFT_DT_SOFTPLUS | {"fused": 0, "conv_only": md.MDRAFT_CONV_ONLY, "preconv": md.MDRAFT_PRECONV}[mode]
    tdt = torch_act(act)
    M = tree.n_nodes
    x, z, dt, B, C = gen.node_inputs(cfg, 0, 0, M)
    have_root_state = bool(g.random() < 0.7)
    h0 = g.normal(size=(Dn, 16)).astype(np.float32)
    c0 = gen.round_to_act(g.normal(size=(3, Dn)).astype(np.float32), act)
    cache = md.StateCache(1, 1 + M, Dn, act=tdt)
    cache.ssm[0, 0] = torch.from_numpy(h0).cuda()
    cache.conv[0, 0] = to_device(c0, tdt)
    root_parent = 0 if have_root_state else -1
    parent_slot = np.where(tree.parents < 0, root_parent, tree.parents + 1)
    lay = upload_layer(params, act, flags)
    dev = [to_device(a, tdt) for a in (x, z, dt, B, C)]
    out = torch.full((M, Dn), float("nan"), dtype=tdt, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_tree_step(lay, cache, 0, *dev, out, i32(parent_slot), i32(np.arange(M) + 1), [int(v) for v in tree.level_offsets], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    olay = oracle.layer_from_params(params, parity.oracle_flags(flags))
    o_out, o_conv, o_h = oracle.tree(olay, tree.parents, x, z, dt, B, C, c0 if have_root_state else None, h0 if have_root_state else None)
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs")
    if mode != "conv_only":
        assert_close(cache.ssm[0, 1:].cpu().numpy(), o_h, TOL_STATE, "node states")
    if mode != "preconv":
        assert np.array_equal(cache.conv[0, 1:].float().cpu().numpy().astype(np.float64), o_conv)


@pytest.mark.parametrize("seed", range(24))
def test_random_projection_tree_case(seed):
    """Random width (every block width and cluster size, ragged last blocks), rank, tree, grouping, dtype, A and step-size mode."""
    g = np.random.default_rng(900 + seed)
    act = "bf16" if g.random() < 0.6 else "f32"
    Dn = int(g.choice([8, 72, 128, 136, 392, 520, 1024, 1032, 1536, 2048, 2056, 3072, 4096]))
    R = int(g.choice([8, 16, 24, 48, 64, 96, 160, 256]))
    n_levels = int(g.integers(1, 5))
    n_nodes = min(int(g.integers(n_levels, 4 * n_levels + 1)), 1 + 4 * (n_levels - 1))
    tree = gen.random_branching_tree(n_nodes, n_levels, seed, max_children=4) if n_levels > 1 else gen.chain_tree(1)
    cfg = parity.small_config(Dn, act, cid=93, seed=seed)
    general_A = bool(g.random() < 0.5)
    params = gen.layer_params(cfg, 0, conv_bias=bool(g.random() < 0.5), general_A=general_A)
    flags = md.MDRAFT_DT_SOFTPLUS | (md.MDRAFT_A_POWERS if (not general_A and g.random() < 0.7) else 0)
    W_x, W_dt = gen.select_proj(cfg, 0, R)
    tdt = torch_act(act)
    M = tree.n_nodes
    x, z, _, _, _ = gen.node_inputs(cfg, 0, 0, M)
    have_root_state = bool(g.random() < 0.7)
    h0 = g.normal(size=(Dn, 16)).astype(np.float32)
    c0 = gen.round_to_act(g.normal(size=(3, Dn)).astype(np.float32), act)
    cache = md.StateCache(1, 1 + M, Dn, act=tdt)
    cache.ssm[0, 0] = torch.from_numpy(h0).cuda()
    cache.conv[0, 0] = to_device(c0, tdt)
    parent_slot = np.where(tree.parents < 0, 0 if have_root_state else -1, tree.parents + 1).astype(np.int32)
    node_slot = (np.arange(M) + 1).astype(np.int32)
    lay = upload_layer(params, act, flags)
    dx, dz, dWx, dWdt = (to_device(a, tdt) for a in (x, z, W_x, W_dt))
    out = torch.full((M, Dn), float("nan"), dtype=tdt, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    npc = int(g.choice([0, 1, 2, 4]))
    for lo, hi in zip(tree.level_offsets[:-1], tree.level_offsets[1:]):
        md.mdraft_tree_step_proj(lay, cache, 0, dWx, dWdt, dx[lo:hi], dz[lo:hi], out[lo:hi], i32(parent_slot[lo:hi]), i32(node_slot[lo:hi]),
                                 status, nodes_per_cluster=npc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    olay = oracle.layer_from_params(params, parity.oracle_flags(flags))
    o_out, o_conv, o_h, _, _, _ = oracle.tree_proj(olay, W_x, W_dt, tree.parents, x, z, c0 if have_root_state else None, h0 if have_root_state else None)
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs")
    assert_close(cache.ssm[0, 1:].cpu().numpy(), o_h, TOL_STATE, "node states")
    assert np.array_equal(cache.conv[0, 1:].float().cpu().numpy().astype(np.float64), o_conv)
