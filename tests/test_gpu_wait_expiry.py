"""The give-up paths of the bounded on-chip waits, run on a healthy GPU.

Every wait on an mbarrier in the kernels has a poll limit; when it runs out the block raises
MDRAFT_DEV_WAIT_EXPIRED, stores nothing, and the call returns.  In the ordinary library those paths run only if a
copy really stalls.  A second build of the same sources (``libmdraft_waittest.so``: a limit of 4096 polls, and every
copy barrier told to expect 16 bytes more than will arrive) makes every such wait run out while the copies themselves
complete normally, so the paths execute without any fault, trap or endless loop.  Each test checks the status bit,
that no output or state slot was touched, and that the ordinary library then gives a correct result in the same
process.
"""

import contextlib

import numpy as np
import pytest
import torch

import gen
import parity
from parity import TOL, TOL_STATE, assert_close
from test_gpu_parity_small import run_oracle_prefill
from test_gpu_tree import TreeRig
from test_gpu_tree_proj import ProjRig

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200 import binding
from paper_2506_01206_b200.build import build_library
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer


@pytest.fixture(scope="module")
def waitlib():
    return binding.load_library(build_library(variant="waittest"))


@contextlib.contextmanager
def using(lib):
    """Route the binding's calls to ``lib`` for the duration of the block."""
    md.load_library()
    keep = binding._lib
    binding._lib = lib
    try:
        yield
    finally:
        binding._lib = keep


def _prefill(prob, cache, out, ws, chunk_len, status):
    cfg = prob.cfg
    tdt = torch_act(cfg.act)
    lay = upload_layer(prob.params, cfg.act, md.MDRAFT_DT_SOFTPLUS)
    dev = [to_device(a, tdt) for a in (prob.x, prob.z, prob.dt, prob.B, prob.C)]
    S = len(prob.cu) - 1
    md.mdraft_conv_scan_prefill(lay, cache, 0, *dev, out, i32(prob.cu), int(np.max(np.diff(prob.cu))), None, i32(np.arange(S)),
                                ws, chunk_len, status)
    torch.cuda.synchronize()


@pytest.mark.parametrize("act", ["f32", "bf16"])
@pytest.mark.parametrize("chunk_len", [32, 4096])
def test_prefill_wait_runs_out_and_the_call_returns(waitlib, act, chunk_len):
    lens = [100, 37]
    cfg = parity.small_config(200, act, len(lens), cid=94)
    prob = parity.make_problem(cfg, lens, conv_bias=True, general_A=True)
    tdt = torch_act(act)
    T = sum(lens)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    cache = md.StateCache(1, len(lens), 200, act=tdt)
    cache.ssm.fill_(3.0); cache.conv.fill_(3.0)
    out = torch.full((T, 200), 7.0, dtype=tdt, device="cuda")
    with using(waitlib):
        _prefill(prob, cache, out, ws, chunk_len, status)
    assert int(status.item()) == md.MDRAFT_DEV_WAIT_EXPIRED
    assert bool((out == 7.0).all()), "a block that gave up must not have written outputs"
    assert bool((cache.ssm == 3.0).all()) and bool((cache.conv == 3.0).all()), "... nor state slots"
    # the context is intact: the ordinary library, same process, same buffers
    status.zero_()
    _prefill(prob, cache, out, ws, chunk_len, status)
    assert int(status.item()) == 0
    o_out, o_conv, o_h = run_oracle_prefill(prob, md.MDRAFT_DT_SOFTPLUS)
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "out after recovery")
    assert_close(cache.ssm[0].cpu().numpy(), o_h, TOL_STATE, "state after recovery")


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_tree_step_wait_runs_out_and_the_call_returns(waitlib, act):
    cfg = parity.small_config(200, act, cid=94)
    tree = gen.paper_tree((3, 2, 2, 1, 1))
    rig = TreeRig(cfg, tree)
    with using(waitlib):
        out = rig.run_levels()   # one call per level: the kernel that stages a node's data with bulk copies
    assert int(rig.status.item()) == md.MDRAFT_DEV_WAIT_EXPIRED
    assert bool(torch.isnan(out).all()), "no node output may have been written"
    assert bool(torch.isnan(rig.cache.ssm[0, 1:]).all()) and bool(torch.isnan(rig.cache.conv[0, 1:].float()).all()), "no node slot either"
    rig.status.zero_()
    out = rig.step(0, tree.n_nodes, level_offsets=[int(v) for v in tree.level_offsets])
    assert int(rig.status.item()) == 0
    o_out, _, o_h = rig.oracle()
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs after recovery")
    assert_close(rig.states()[0], o_h, TOL_STATE, "node states after recovery")


@pytest.mark.parametrize("act,Dn,R,npc", [("f32", 200, 16, 0), ("bf16", 1536, 48, 0), ("bf16", 392, 16, 2)])
def test_projection_step_wait_runs_out_and_the_cluster_still_meets(waitlib, act, Dn, R, npc):
    """The blocks of a node meet at the cluster barrier whether or not their copies arrived: a block that gave up
    takes part in both barriers, stores nothing, and the launch ends."""
    cfg = parity.small_config(Dn, act, cid=94)
    tree = gen.full_tree([3])
    rig = ProjRig(cfg, tree, R, nodes_per_cluster=npc)
    with using(waitlib):
        out = rig.step(np.arange(0, 1))
        kids = rig.step(np.arange(1, tree.n_nodes))   # a level of three nodes (two node groups when a cluster takes two)
    assert int(rig.status.item()) == md.MDRAFT_DEV_WAIT_EXPIRED
    assert bool(torch.isnan(out).all()) and bool(torch.isnan(kids).all())
    assert bool(torch.isnan(rig.cache.ssm[0, 1:]).all())
    rig.status.zero_()
    out = rig.run_levels()
    assert int(rig.status.item()) == 0
    o_out, _, o_h, _, _, _ = rig.oracle()
    assert_close(out.float().cpu().numpy(), o_out, TOL[act], "node outputs after recovery")
    assert_close(rig.states()[0], o_h, TOL_STATE, "node states after recovery")


def test_ssd_prefill_wait_runs_out_tensor_memory_is_freed_and_the_next_call_is_correct(waitlib):
    """The tensor-core kernels of the SSD encode allocate tensor memory before they wait for their copies: when the
    wait runs out they must still free it (a leak would stall later blocks on the same SM for good) and store no
    output.  Several rounds of failing calls, then an ordinary call checked against the oracle."""
    import oracle
    from paper_2506_01206_b200.device_inputs import upload_ssd_layer
    Dn, T, Pn, Nn = 192, 300, 64, 128
    cfg = gen.Config(95, "ssd-wait", 1, Dn, Nn, 4, "bf16", 1, (1, 1), "none", 0, 0)
    prm = gen.ssd_params(cfg, 0, Pn, Nn, conv_bias=True)
    arrs = gen.ssd_inputs(cfg, 0, 0, 0, T, Pn, Nn)
    lay = upload_ssd_layer(prm)
    dev = [to_device(a, torch.bfloat16) for a in arrs]
    cache = md.StateCache(1, 1, Dn, d_state=Nn, act=torch.bfloat16)
    ws = torch.empty(md.mdraft_ssd_prefill_workspace_bytes(lay, T, 1), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((T, Dn), 7.0, dtype=torch.bfloat16, device="cuda")
    with using(waitlib):
        for _ in range(6):   # more failing blocks than an SM has tensor-memory columns for, if any were leaked
            md.mdraft_ssd_prefill(lay, cache, 0, *dev, out, None, None, i32([0]), ws, status)
        torch.cuda.synchronize()
    assert int(status.item()) == md.MDRAFT_DEV_WAIT_EXPIRED
    assert bool((out == 7.0).all()), "a block that gave up must not have written outputs"
    status.zero_()
    md.mdraft_ssd_prefill(lay, cache, 0, *dev, out, None, None, i32([0]), ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_out, _, o_h = oracle.ssd_prefill(oracle.ssd_layer_from_params(prm), *arrs)
    assert_close(out.float().cpu().numpy(), o_out, TOL["bf16"], "out after recovery")
    assert_close(cache.ssm[0].cpu().numpy(), o_h, TOL_STATE, "state after recovery")
