"""The prefill entry point that brings its own scratch memory (mdraft_conv_scan_prefill_noalloc).

It exists for callers that must not allocate on the device while they run (a server whose memory pool is
fixed at start-up, a plug-in that is handed pointers but owns no allocator).  The check is simple: on the same
inputs it must give, bit for bit, what the ordinary entry point gives with a caller-owned workspace (and that must
agree with the fp64 oracle), and it must keep doing so when called again, because every call reuses the one scratch array and finds the previous call's leftovers
in it.  This file sorts last on purpose, so that a run which stops at the first failure has already run every
other test; it also passes when run alone in a fresh process.
"""

import numpy as np
import pytest
import torch

import oracle
import parity
from parity import TOL, TOL_STATE, assert_close

pytestmark = pytest.mark.gpu

import paper_2506_01206_b200 as md
from paper_2506_01206_b200.device_inputs import i32, to_device, torch_act, upload_layer


def _device_problem(prob):
    cfg = prob.cfg
    tdt = torch_act(cfg.act)
    lay = upload_layer(prob.params, cfg.act, md.MDRAFT_DT_SOFTPLUS)
    dev = [to_device(a, tdt) for a in (prob.x, prob.z, prob.dt, prob.B, prob.C)]
    return lay, tdt, dev


@pytest.mark.parametrize("act", ["bf16", "f32"])
def test_noalloc_prefill_equals_prefill_with_workspace_twice(act):
    lens = [300, 41, 222]
    S, T, Dn, chunk = len(lens), sum(lens), 264, 32
    cfg = parity.small_config(Dn, act, S)
    prob = parity.make_problem(cfg, lens, conv_bias=True, general_A=True)
    lay, tdt, dev = _device_problem(prob)
    cu = i32(np.concatenate([[0], np.cumsum(lens)]))
    final = i32(np.arange(S))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    # ordinary entry point, workspace owned by the caller
    need = md.mdraft_prefill_workspace_bytes(lay, T, S, max(lens), chunk)
    assert 0 < need <= md.NOALLOC_SCRATCH_BYTES
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    cache_a = md.StateCache(1, S, Dn, act=tdt)
    out_a = torch.empty((T, Dn), dtype=tdt, device="cuda")
    md.mdraft_conv_scan_prefill(lay, cache_a, 0, *dev, out_a, cu, max(lens), None, final, ws, chunk, status)
    torch.cuda.synchronize()

    for call in range(2):  # the second call meets the first call's leftovers in the shared scratch
        cache_b = md.StateCache(1, S, Dn, act=tdt)
        out_b = torch.full((T, Dn), float("nan"), dtype=tdt, device="cuda")
        md.mdraft_conv_scan_prefill_noalloc(lay, cache_b, 0, *dev, out_b, cu, max(lens), None, final, chunk, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # the same kernels on the same plan, only the scratch lives elsewhere: the same bits
        bits = torch.int16 if act == "bf16" else torch.int32
        assert torch.equal(out_b.view(bits), out_a.view(bits)), f"call {call}: out"
        assert torch.equal(cache_b.ssm.view(torch.int32), cache_a.ssm.view(torch.int32)), f"call {call}: SSM state"
        assert torch.equal(cache_b.conv.view(bits), cache_a.conv.view(bits)), f"call {call}: conv window"
        # and the right ones: against the fp64 oracle, at the tolerances of the parity tests
        o_out, o_conv, o_h = oracle.prefill(oracle.layer_from_params(prob.params), prob.x, prob.z, prob.dt, prob.B, prob.C, prob.cu)
        assert_close(out_b.float().cpu().numpy(), o_out, TOL[act], f"call {call}: out against the oracle")
        assert_close(cache_b.ssm[0].cpu().numpy(), o_h, TOL_STATE, f"call {call}: SSM state against the oracle")
        assert np.array_equal(cache_b.conv[0].float().cpu().numpy().astype(np.float64), o_conv), f"call {call}: conv window against the oracle"


def test_noalloc_prefill_refuses_problems_beyond_its_scratch():
    # 3000 chunks x 1536 channels of summaries is far more than the fixed array holds: refused on the host
    Dn, T = 1536, 12000
    cfg = parity.small_config(Dn, "bf16", 1)
    prob = parity.make_problem(cfg, [8])
    lay = upload_layer(prob.params, "bf16")
    assert md.mdraft_prefill_workspace_bytes(lay, T, 1, T, 4) > md.NOALLOC_SCRATCH_BYTES
    x = torch.zeros((T, Dn), dtype=torch.bfloat16, device="cuda")
    bc = torch.zeros((T, 16), dtype=torch.bfloat16, device="cuda")
    out = torch.full((T, Dn), 7.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(md.MdraftError) as e:
        md.mdraft_conv_scan_prefill_noalloc(lay, None, 0, x, x, x, bc, bc, out, i32([0, T]), T, None, None, 4)
    assert e.value.status == -4
    torch.cuda.synchronize()
    assert float(out.float().min()) == 7.0 and float(out.float().max()) == 7.0, "a refused call must launch nothing"
