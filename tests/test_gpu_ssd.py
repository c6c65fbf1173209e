"""The Mamba-2 (SSD) path against the fp64 oracle: context encode (tensor-core chunk kernels) and draft-tree step.

Tolerances.  `out` is bf16 and the chunk-local products take bf16 operands (u * Delta, the masked C.B products, the
incoming state), so the encode's outputs are held to the bf16 tolerance of this library (2e-2, RMS-floored); the
states are fp32 and the state product runs on operands split into a bf16 value plus a bf16 remainder, so they are held
to the state tolerance (1e-3).  The tree step is plain fp32 arithmetic: same two tolerances, far inside them.
"""

import numpy as np
import pytest
import torch

import gen
import oracle
import parity
from parity import TOL, TOL_STATE, assert_close

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200.device_inputs import i32, to_device, upload_ssd_layer

P, N = 64, 128
BF = torch.bfloat16


def ssd_cache(n_slots, Dn, n_layers=1):
    return md.StateCache(n_layers, n_slots, Dn, d_state=N, act=BF)


def make(Dn, lens, seed=0, conv_bias=True):
    cfg = gen.Config(95, "ssd-test", 1, Dn, N, 4, "bf16", len(lens), (1, 1), "none", 0, seed)
    prm = gen.ssd_params(cfg, 0, P, N, conv_bias=conv_bias)
    T = int(sum(lens))
    x, z, dt, B, C = gen.ssd_inputs(cfg, 0, 0, 0, T, P, N)
    cu = np.zeros(len(lens) + 1, dtype=np.int32); cu[1:] = np.cumsum(lens)
    return cfg, prm, (x, z, dt, B, C), cu


def run_gpu(prm, arrs, cu, conv_init=None, h_init=None, no_offsets=False, flags=md.MDRAFT_DT_SOFTPLUS):
    S, T, Dn = len(cu) - 1, int(cu[-1]), prm.conv_w.shape[0]
    lay = upload_ssd_layer(prm, flags)
    cache = ssd_cache(2 * S, Dn)
    cache.ssm.fill_(float("nan")); cache.conv.fill_(float("nan"))
    have_init = h_init is not None
    if have_init:
        cache.ssm[0, :S] = torch.from_numpy(h_init.astype(np.float32)).cuda()
        cache.conv[0, :S] = to_device(conv_init.astype(np.float32), BF)
    dev = [to_device(a, BF) for a in arrs]
    out = torch.full((T, Dn), float("nan"), dtype=BF, device="cuda")
    ws = torch.empty(max(256, md.mdraft_ssd_prefill_workspace_bytes(lay, T, S)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    final = i32(np.arange(S, 2 * S))
    md.mdraft_ssd_prefill(lay, cache, 0, *dev, out, None if no_offsets else i32(cu), i32(np.arange(S)) if have_init else None, final, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return (out.float().cpu().numpy().astype(np.float64), cache.conv[0, S:].float().cpu().numpy().astype(np.float64),
            cache.ssm[0, S:].cpu().numpy().astype(np.float64))


@pytest.mark.parametrize("Dn,lens,init", [
    (64, [128], False),                       # one head, one full chunk
    (128, [40], True),                        # a partial chunk from a given state
    (192, [300], True),                       # three heads, three chunks (the last one partial): state passing
    (64, [1, 2, 3, 130, 0, 127, 129], True),  # packed: lengths around d_conv and around the chunk size, an empty one
    (1536, [700], False),                     # the 130M shape: 24 heads
])
def test_ssd_prefill_matches_oracle(Dn, lens, init):
    cfg, prm, arrs, cu = make(Dn, lens)
    S = len(lens)
    g = np.random.default_rng(7)
    ci = gen.round_to_act(g.normal(size=(S, 3, Dn)).astype(np.float32), "bf16") if init else None
    hi = g.normal(size=(S, Dn, N)).astype(np.float32) if init else None
    g_out, g_conv, g_h = run_gpu(prm, arrs, cu, ci, hi)
    o_out, o_conv, o_h = oracle.ssd_prefill(oracle.ssd_layer_from_params(prm), *arrs, cu_seqlens=cu, conv_init=ci, h_init=hi)
    assert_close(g_out, o_out, TOL["bf16"], "out")
    assert_close(g_h, o_h, TOL_STATE, "final SSM state")
    assert np.array_equal(g_conv, o_conv), "conv window must be an exact copy of the last raw inputs"


def test_ssd_prefill_at_the_timed_shape():
    """2048 tokens x 1536 channels (24 heads), one sequence given without offsets, no starting slot: the call bench.py times."""
    cfg, prm, arrs, cu = make(1536, [2048], seed=2)
    g_out, g_conv, g_h = run_gpu(prm, arrs, cu, no_offsets=True)
    o_out, o_conv, o_h = oracle.ssd_prefill(oracle.ssd_layer_from_params(prm), *arrs, cu_seqlens=cu)
    assert_close(g_out, o_out, TOL["bf16"], "out")
    assert_close(g_h, o_h, TOL_STATE, "final SSM state")
    assert np.array_equal(g_conv, o_conv)


def test_ssd_prefill_in_pieces_equals_whole():
    """Encode 300 tokens at once, and as 128 + 172 through the slot: the same outputs and state within rounding of
    the different chunk boundaries (chunks 128/128/44 against 128 | 128/44: here identical cuts, so bit for bit)."""
    cfg, prm, arrs, cu = make(128, [300])
    whole = run_gpu(prm, arrs, cu, no_offsets=True)
    a = run_gpu(prm, [v[:128] for v in arrs], np.array([0, 128], dtype=np.int32))
    b = run_gpu(prm, [v[128:] for v in arrs], np.array([0, 172], dtype=np.int32), conv_init=a[1], h_init=a[2])
    assert np.array_equal(np.concatenate([a[0], b[0]]), whole[0])
    assert np.array_equal(b[2], whole[2]) and np.array_equal(b[1], whole[1])


def test_ssd_prefill_raw_step_size_and_zero_step_size():
    cfg, prm, arrs, cu = make(128, [200])
    x, z, dt, B, C = arrs
    g = np.random.default_rng(3)
    prm.dt_bias[:] = 0
    dt = gen.round_to_act(np.where(g.random(dt.shape) < 0.4, 0.0, g.uniform(0.001, 0.2, size=dt.shape)).astype(np.float32), "bf16")
    hi = g.normal(size=(1, 128, N)).astype(np.float32); ci = gen.round_to_act(g.normal(size=(1, 3, 128)).astype(np.float32), "bf16")
    got = run_gpu(prm, (x, z, dt, B, C), cu, ci, hi, flags=0)
    want = oracle.ssd_prefill(oracle.ssd_layer_from_params(prm, flags=0), x, z, dt, B, C, cu_seqlens=cu, conv_init=ci, h_init=hi)
    assert_close(got[0], want[0], TOL["bf16"], "out")
    assert_close(got[2], want[2], TOL_STATE, "state")
    # all step sizes zero: the state is the starting state, exactly
    got0 = run_gpu(prm, (x, z, np.zeros_like(dt), B, C), cu, ci, hi, flags=0)
    assert np.array_equal(got0[2].astype(np.float32).view(np.uint32), hi.view(np.uint32))


class SsdTreeRig:
    def __init__(self, Dn, tree, seed=0):
        self.cfg = gen.Config(96, "ssd-tree", 1, Dn, N, 4, "bf16", 1, (1, 1), "none", 0, seed)
        self.prm = gen.ssd_params(self.cfg, 0, P, N, conv_bias=True)
        self.lay = upload_ssd_layer(self.prm)
        self.tree, M = tree, tree.n_nodes
        self.arrs = gen.ssd_inputs(self.cfg, 0, 0, 1, M, P, N)
        g = np.random.default_rng(5)
        self.h0 = g.normal(size=(Dn, N)).astype(np.float32)
        self.c0 = gen.round_to_act(g.normal(size=(3, Dn)).astype(np.float32), "bf16")
        self.cache = ssd_cache(1 + M, Dn)
        self.cache.ssm.fill_(float("nan")); self.cache.conv.fill_(float("nan"))
        self.cache.ssm[0, 0] = torch.from_numpy(self.h0).cuda(); self.cache.conv[0, 0] = to_device(self.c0, BF)
        self.dev = [to_device(a, BF) for a in self.arrs]
        self.parent_slot = np.where(tree.parents < 0, 0, tree.parents + 1).astype(np.int32)
        self.node_slot = (np.arange(M) + 1).astype(np.int32)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run(self, one_call):
        M, Dn = self.tree.n_nodes, self.cfg.d_inner
        out = torch.full((M, Dn), float("nan"), dtype=BF, device="cuda")
        lv = [int(v) for v in self.tree.level_offsets]
        if one_call:
            md.mdraft_ssd_tree_step(self.lay, self.cache, 0, *self.dev, out, i32(self.parent_slot), i32(self.node_slot), lv, self.status)
        else:
            for a, b in zip(lv[:-1], lv[1:]):
                md.mdraft_ssd_tree_step(self.lay, self.cache, 0, *[t[a:b] for t in self.dev], out[a:b], i32(self.parent_slot[a:b]),
                                        i32(self.node_slot[a:b]), None, self.status)
        torch.cuda.synchronize()
        assert int(self.status.item()) == 0
        return out


@pytest.mark.parametrize("Dn,shape", [(64, "cfg0"), (192, "paper32211"), (1536, "paper3321"), (128, "chain")])
def test_ssd_tree_matches_oracle(Dn, shape):
    tree = {"cfg0": gen.full_tree([2, 2, 2]), "paper32211": gen.paper_tree((3, 2, 2, 1, 1)), "paper3321": gen.paper_tree((3, 3, 2, 1)),
            "chain": gen.chain_tree(6)}[shape]
    rig = SsdTreeRig(Dn, tree)
    out = rig.run(one_call=True)
    o_out, o_conv, o_h = oracle.ssd_tree(oracle.ssd_layer_from_params(rig.prm), tree.parents, *rig.arrs, conv0=rig.c0, h0=rig.h0)
    assert_close(out.float().cpu().numpy(), o_out, TOL["bf16"], "node outputs")
    s = torch.from_numpy(rig.node_slot.astype(np.int64)).cuda()
    assert_close(rig.cache.ssm[0, s].cpu().numpy(), o_h, TOL_STATE, "node states")
    assert np.array_equal(rig.cache.conv[0, s].float().cpu().numpy().astype(np.float64), o_conv)
    # level by level gives the same bits
    rig2 = SsdTreeRig(Dn, tree)
    out2 = rig2.run(one_call=False)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(rig.cache.ssm[0, 1:], rig2.cache.ssm[0, 1:])


def test_ssd_prefill_then_chain_equals_longer_prefill_and_commit_moves_ssd_slots():
    """prefill(L) followed by k chained steps lands (within tolerance) where prefill(L + k) lands; the commit call
    copies (D, 128) slots bit for bit."""
    Dn, L, k = 128, 150, 4
    cfg, prm, arrs, cu = make(Dn, [L + k])
    whole = run_gpu(prm, arrs, cu)
    lay = upload_ssd_layer(prm)
    cache = ssd_cache(3, Dn)
    dev = [to_device(a, BF) for a in arrs]
    out = torch.empty((L, Dn), dtype=BF, device="cuda")
    ws = torch.empty(md.mdraft_ssd_prefill_workspace_bytes(lay, L, 1), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_ssd_prefill(lay, cache, 0, *[t[:L] for t in dev], out, None, None, i32([0]), ws, status)
    step_out = torch.empty((k, Dn), dtype=BF, device="cuda")
    for i in range(k):   # in-place chain decode on slot 0
        md.mdraft_ssd_tree_step(lay, cache, 0, *[t[L + i:L + i + 1] for t in dev], step_out[i:i + 1], i32([0]), i32([0]), None, status)
    md.mdraft_state_commit(cache, i32([0]), i32([2]), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_close(step_out.float().cpu().numpy(), whole[0][L:], TOL["bf16"], "chained steps == prefill tail")
    assert_close(cache.ssm[0, 0].cpu().numpy(), whole[2][0], TOL_STATE, "state after the chain")
    assert torch.equal(cache.ssm[0, 2], cache.ssm[0, 0]) and torch.equal(cache.conv[0, 2].view(torch.int16), cache.conv[0, 0].view(torch.int16))


def test_ssd_bad_slots_are_flagged_not_followed():
    cfg, prm, arrs, cu = make(64, [30, 20])
    lay = upload_ssd_layer(prm)
    cache = ssd_cache(2, 64)
    dev = [to_device(a, BF) for a in arrs]
    out = torch.zeros((50, 64), dtype=BF, device="cuda")
    ws = torch.empty(md.mdraft_ssd_prefill_workspace_bytes(lay, 50, 2), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_ssd_prefill(lay, cache, 0, *dev, out, i32(cu), None, i32([0, 77]), ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) & md.MDRAFT_DEV_BAD_SLOT
    assert float(out[:30].float().abs().max()) > 0 and float(out[30:].float().abs().max()) == 0.0
    status.zero_()
    md.mdraft_ssd_tree_step(lay, cache, 0, *[t[:1] for t in dev], out[:1], i32([5]), i32([0]), None, status)
    torch.cuda.synchronize()
    assert int(status.item()) & md.MDRAFT_DEV_BAD_SLOT


def _ssd_case(seed):
    g = np.random.default_rng(5000 + seed)
    Dn = int(g.choice([64, 128, 192, 320]))
    S = int(g.integers(1, 5))
    lens = [int(v) for v in g.choice([0, 1, 2, 3, 5, 31, 64, 127, 128, 129, 200, 257, 300], size=S)]
    if sum(lens) == 0:
        lens[0] = 17
    return dict(Dn=Dn, lens=lens, conv_bias=bool(g.random() < 0.5), softplus=bool(g.random() < 0.75),
                init=str(g.choice(["none", "slots", "mixed"])), regime=str(g.choice(["recipe", "recipe", "big_dt", "A_zero", "A_steep"])), seed=seed)


@pytest.mark.parametrize("seed", range(24))
def test_random_ssd_prefill_case(seed):
    """Seeded sweep over widths, packed length mixes around the chunk size, starting-slot arrangements and value regimes
    outside the recipe (pre-activations from -60 to +30 under softplus; heads with A = 0; A down to -200)."""
    c = _ssd_case(seed)
    cfg, prm, arrs, cu = make(c["Dn"], c["lens"], seed=seed, conv_bias=c["conv_bias"])
    x, z, dt, B, C = arrs
    S, Dn = len(c["lens"]), c["Dn"]
    g = np.random.default_rng(6000 + seed)
    H = Dn // P
    flags = md.MDRAFT_DT_SOFTPLUS if c["softplus"] else 0
    if c["regime"] == "A_zero":
        prm.A[::2] = 0.0
    elif c["regime"] == "A_steep":
        prm.A[:] = -g.uniform(40.0, 200.0, size=H).astype(np.float32)
    if not c["softplus"]:
        dt = gen.round_to_act(np.where(g.random(dt.shape) < 0.3, 0.0, np.abs(dt) * 0.05).astype(np.float32), "bf16")
        prm.dt_bias[:] = 0
    elif c["regime"] == "big_dt":
        kind = g.integers(0, 3, size=dt.shape)
        dt = gen.round_to_act(np.where(kind == 0, dt, np.where(kind == 1, g.uniform(10.0, 30.0, size=dt.shape), g.uniform(-60.0, -10.0, size=dt.shape))).astype(np.float32), "bf16")
        prm.dt_bias[:] = 0
    arrs = (x, z, dt, B, C)
    h0 = g.normal(size=(S, Dn, N)).astype(np.float32)
    c0 = gen.round_to_act(g.normal(size=(S, 3, Dn)).astype(np.float32), "bf16")
    init = None if c["init"] == "none" else (np.arange(S) if c["init"] == "slots" else np.where(g.random(S) < 0.5, np.arange(S), -1))
    lay = upload_ssd_layer(prm, flags)
    cache = ssd_cache(2 * S, Dn)
    cache.ssm.fill_(float("nan")); cache.conv.fill_(float("nan"))
    cache.ssm[0, :S] = torch.from_numpy(h0).cuda(); cache.conv[0, :S] = to_device(c0, BF)
    T = int(cu[-1])
    out = torch.full((T, Dn), float("nan"), dtype=BF, device="cuda")
    ws = torch.empty(max(256, md.mdraft_ssd_prefill_workspace_bytes(lay, T, S)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_ssd_prefill(lay, cache, 0, *[to_device(a, BF) for a in arrs], out, i32(cu), None if init is None else i32(init), i32(np.arange(S, 2 * S)), ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_ci = np.zeros((S, 3, Dn)); o_hi = np.zeros((S, Dn, N))
    if init is not None:
        for s_ in range(S):
            if init[s_] >= 0:
                o_ci[s_] = c0[s_]; o_hi[s_] = h0[s_]
    o_out, o_conv, o_h = oracle.ssd_prefill(oracle.ssd_layer_from_params(prm, flags=flags & 1), *arrs, cu_seqlens=cu, conv_init=o_ci, h_init=o_hi)
    assert_close(out.float().cpu().numpy(), o_out, TOL["bf16"], f"out ({c})")
    assert_close(cache.ssm[0, S:].cpu().numpy(), o_h, TOL_STATE, f"state ({c})")
    assert np.array_equal(cache.conv[0, S:].float().cpu().numpy().astype(np.float64), o_conv), f"window ({c})"
