"""Calls that follow one another on a stream with no host synchronisation between them, sharing one workspace.

The kernels of a context-encode call, and the first kernel of the call behind it, are launched programmatically: a kernel
may start while the one ahead of it is still running.  What keeps that correct is the order of waits inside the kernels
(a call must not overwrite workspace the call before it is still reading, nor read inputs before they are complete).
These tests make several different layers' calls in a row on ONE workspace, eagerly and as a replayed CUDA graph, and
require every output and every final state to equal, bit for bit, what the same call gives when it runs alone.
"""

import numpy as np
import pytest
import torch

import gen
import parity

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer, upload_ssd_layer

BF = torch.bfloat16


def _bits(t):
    return t.contiguous().view(torch.int16 if t.dtype == BF else torch.int32)


def _check(run_layer, n_layers, read_results):
    """run_layer(l) queues layer l's call.  Alone (synchronised) first, then all in a row, then as a graph replayed twice."""
    alone = []
    for l in range(n_layers):
        run_layer(l)
        torch.cuda.synchronize()
        alone.append([r.clone() for r in read_results(l)])

    def wipe():
        for l in range(n_layers):
            for r in read_results(l):
                r.fill_(float("nan"))

    def same(tag):
        torch.cuda.synchronize()
        for l in range(n_layers):
            for k, (a, b) in enumerate(zip(alone[l], read_results(l))):
                assert torch.equal(_bits(a), _bits(b)), f"{tag}: layer {l}, result {k} differs from the call made alone"

    wipe()
    for l in range(n_layers):
        run_layer(l)
    same("in a row")

    wipe()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for l in range(n_layers):
            run_layer(l)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for l in range(n_layers):
            run_layer(l)
    for rep in range(2):
        wipe()
        g.replay()
        same(f"graph replay {rep}")


@pytest.mark.parametrize("lens", [[700], [130, 0, 517, 64]])
def test_ssd_encodes_in_a_row_on_one_workspace(lens):
    NL, Dn, P, N = 4, 192, 64, 128
    cfg = gen.Config(96, "ssd-row", NL, Dn, N, 4, "bf16", len(lens), (1, 1), "none", 0, 3)
    S, T = len(lens), int(sum(lens))
    cu = np.zeros(S + 1, dtype=np.int32); cu[1:] = np.cumsum(lens)
    lays = [upload_ssd_layer(gen.ssd_params(cfg, l, P, N), md.MDRAFT_DT_SOFTPLUS) for l in range(NL)]
    ins = [[to_device(a, BF) for a in gen.ssd_inputs(cfg, l, 0, 0, T, P, N)] for l in range(NL)]
    outs = [torch.empty((T, Dn), dtype=BF, device="cuda") for _ in range(NL)]
    cache = md.StateCache(NL, 2 * S, Dn, d_state=N, act=BF)
    g = np.random.default_rng(11)
    cache.ssm[:, :S] = torch.from_numpy(g.normal(size=(NL, S, Dn, N)).astype(np.float32)).cuda()
    cache.conv[:, :S] = to_device(g.normal(size=(NL, S, 3, Dn)).astype(np.float32), BF)
    ws = torch.empty(md.mdraft_ssd_prefill_workspace_bytes(lays[0], T, S), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cu_d, init, final = i32(cu), i32(np.arange(S)), i32(np.arange(S, 2 * S))

    def run_layer(l):
        md.mdraft_ssd_prefill(lays[l], cache, l, *ins[l], outs[l], cu_d, init, final, ws, status)

    _check(run_layer, NL, lambda l: [outs[l], cache.ssm[l, S:], cache.conv[l, S:]])
    assert int(status.item()) == 0


@pytest.mark.parametrize("act", ["bf16", "f32"])
@pytest.mark.parametrize("powers", [False, True])
def test_prefills_in_a_row_on_one_workspace(act, powers):
    NL, Dn, lens, chunk_len = 4, 264, [611, 0, 90, 333], 48
    tdt = torch_act(act)
    S, T = len(lens), int(sum(lens))
    flags = md.MDRAFT_DT_SOFTPLUS | (md.MDRAFT_A_POWERS if powers else 0)
    cfg = gen.Config(96, "row", NL, Dn, 16, 4, act, S, (1, 1), "none", 0, 5)
    probs = [parity.make_problem(cfg, lens, layer=l, conv_bias=True, general_A=not powers) for l in range(NL)]
    lays = [upload_layer(pr.params, act, flags) for pr in probs]
    ins = [[to_device(a, tdt) for a in (pr.x, pr.z, pr.dt, pr.B, pr.C)] for pr in probs]
    outs = [torch.empty((T, Dn), dtype=tdt, device="cuda") for _ in range(NL)]
    cache = md.StateCache(NL, 2 * S, Dn, act=tdt)
    g = np.random.default_rng(12)
    cache.ssm[:, :S] = torch.from_numpy(g.normal(size=(NL, S, Dn, 16)).astype(np.float32)).cuda()
    cache.conv[:, :S] = to_device(g.normal(size=(NL, S, 3, Dn)).astype(np.float32), tdt)
    max_len = max(lens)
    ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lays[0], T, S, max_len, chunk_len)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cu_d, init, final = i32(probs[0].cu), i32(np.arange(S)), i32(np.arange(S, 2 * S))

    def run_layer(l):
        md.mdraft_conv_scan_prefill(lays[l], cache, l, *ins[l], outs[l], cu_d, max_len, init, final, ws, chunk_len, status)

    _check(run_layer, NL, lambda l: [outs[l], cache.ssm[l, S:], cache.conv[l, S:]])
    assert int(status.item()) == 0
