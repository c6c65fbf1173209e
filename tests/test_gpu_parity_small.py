"""CUDA library vs the fp64 oracle, element by element, on small seeded problems that still span several
channel blocks, several token chunks, several B/C tiles and ragged tails.  All calls go through the C ABI."""

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


def run_gpu_prefill(prob, flags, chunk_len=0, conv_init=None, h_init=None, in_place=False, strided=False):
    """Returns out (T,D) float64, conv_final (S,3,D), h_final (S,D,N) from the CUDA library."""
    cfg = prob.cfg
    S = len(prob.cu) - 1
    T = int(prob.cu[-1])
    Dn = cfg.d_inner
    tdt = torch_act(cfg.act)
    lay = upload_layer(prob.params, cfg.act, flags)
    cache = md.StateCache(1, 2 * S, Dn, act=tdt)
    have_init = conv_init is not None or h_init is not None
    if h_init is not None:
        cache.ssm[0, :S] = torch.from_numpy(h_init.astype(np.float32)).cuda()
    if conv_init is not None:
        cache.conv[0, :S] = to_device(conv_init.astype(np.float32), tdt)
    init_slot = i32(np.arange(S)) if have_init else None
    final_slot = i32(np.arange(S) if in_place else np.arange(S, 2 * S))
    if strided:  # x and z as the two halves of one wider matrix, B and C as slices of another
        xz = torch.empty((T, 2 * Dn + 8), dtype=tdt, device="cuda")
        xz[:, :Dn] = to_device(prob.x, tdt); xz[:, Dn:2 * Dn] = to_device(prob.z, tdt)
        x, z = xz[:, :Dn], xz[:, Dn:2 * Dn]
        bc = torch.empty((T, 48), dtype=tdt, device="cuda")
        bc[:, 8:24] = to_device(prob.B, tdt); bc[:, 24:40] = to_device(prob.C, tdt)
        B, C = bc[:, 8:24], bc[:, 24:40]
    else:
        x, z = to_device(prob.x, tdt), to_device(prob.z, tdt)
        B, C = to_device(prob.B, tdt), to_device(prob.C, tdt)
    dt = to_device(prob.dt, tdt)
    out = torch.full((T, Dn), float("nan"), dtype=tdt, device="cuda")
    cu = i32(prob.cu)
    max_len = int(np.max(np.diff(prob.cu))) if S else 0
    ws_bytes = md.mdraft_prefill_workspace_bytes(lay, T, S, max_len, chunk_len)
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    md.mdraft_conv_scan_prefill(lay, cache, 0, x, z, dt, B, C, out, cu, max_len, init_slot, final_slot, ws, chunk_len, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    fs = final_slot.cpu().numpy()
    return (out.float().cpu().numpy().astype(np.float64),
            cache.conv[0, fs].float().cpu().numpy().astype(np.float64),
            cache.ssm[0, fs].cpu().numpy().astype(np.float64))


def run_oracle_prefill(prob, flags, conv_init=None, h_init=None):
    lay = oracle.layer_from_params(prob.params, parity.oracle_flags(flags))
    return oracle.prefill(lay, prob.x, prob.z, prob.dt, prob.B, prob.C, prob.cu, conv_init, h_init)


def random_state(cfg, S, seed):
    g = np.random.default_rng(seed)
    h = g.normal(size=(S, cfg.d_inner, 16)).astype(np.float32)
    c = gen.round_to_act(g.normal(size=(S, 3, cfg.d_inner)).astype(np.float32), cfg.act)
    return c, h


CASES = [
    # act,   D,   lens,                       chunk_len, general_A, conv_bias, init
    ("f32", 64, [256], 0, False, False, False),                 # tiny configuration's prefill, default plan
    ("f32", 64, [256], 64, False, False, False),                # same, 4 chunks
    ("f32", 200, [333], 50, True, True, True),                  # ragged: D not a multiple of the block, 7 chunks
    ("bf16", 200, [333], 50, True, True, True),
    ("bf16", 136, [97], 32, False, True, True),
    ("f32", 128, [1, 2, 3, 4, 0, 70, 33, 5], 8, True, True, True),     # packed, lengths around d_conv, an empty one
    ("bf16", 256, [40, 300, 7, 129], 37, True, False, True),    # chunk length that is not a multiple of anything
    ("bf16", 1536, [700], 0, False, False, False),              # drafter width, default plan
    ("f32", 64, [1200], 4, True, True, True),                   # 300 chunks: several rounds of the 32-wide carry scan
]


@pytest.mark.parametrize("act,Dn,lens,chunk_len,general_A,conv_bias,init", CASES)
@pytest.mark.parametrize("powers", [False, True])
def test_prefill_matches_oracle(act, Dn, lens, chunk_len, general_A, conv_bias, init, powers):
    if powers and general_A:
        pytest.skip("A_POWERS promises a structured A")
    cfg = parity.small_config(Dn, act, len(lens))
    prob = parity.make_problem(cfg, lens, conv_bias=conv_bias, general_A=general_A)
    ci, hi = random_state(cfg, len(lens), 5) if init else (None, None)
    flags = md.MDRAFT_DT_SOFTPLUS | (md.MDRAFT_A_POWERS if powers else 0)
    g_out, g_conv, g_h = run_gpu_prefill(prob, flags, chunk_len, ci, hi)
    o_out, o_conv, o_h = run_oracle_prefill(prob, flags, ci, hi)
    assert_close(g_out, o_out, TOL[act], "out")
    assert_close(g_h, o_h, TOL_STATE, "final SSM state")
    assert np.array_equal(g_conv, o_conv), "conv window must be an exact copy of the last raw inputs"


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_prefill_in_place_slots_and_strided_views(act):
    cfg = parity.small_config(264, act, 3)
    prob = parity.make_problem(cfg, [90, 17, 150], conv_bias=True, general_A=True)
    ci, hi = random_state(cfg, 3, 9)
    flags = md.MDRAFT_DT_SOFTPLUS
    ref = run_gpu_prefill(prob, flags, 32, ci, hi)
    for kw in ({"in_place": True}, {"strided": True}):
        got = run_gpu_prefill(prob, flags, 32, ci, hi, **kw)
        for a, b in zip(got, ref):
            assert np.array_equal(a, b), f"{kw}: results must not depend on where the data lives"
    o = run_oracle_prefill(prob, flags, ci, hi)
    assert_close(ref[0], o[0], TOL[act], "out")


@pytest.mark.parametrize("act,Dn,lens,chunk_len", [
    ("bf16", 200, [333], 50),                    # two boxes of channels, the second one partly outside the matrix
    ("f32", 264, [90, 17, 150], 32),             # three boxes, packed sequences
    ("bf16", 1024, [40, 300, 7, 129], 37),       # two full wide blocks
    ("bf16", 520, [260], 0),                     # a second wide block that holds 8 channels only; default chunk plan
])
def test_prefill_wide_and_narrow_blocks_agree_with_the_oracle(act, Dn, lens, chunk_len):
    """Both block widths (128 channels with 4 channel warps, 512 channels with 16) against the oracle, forced through
    the block_channels option, on channel counts that leave boxes partly or wholly empty."""
    cfg = parity.small_config(Dn, act, len(lens))
    prob = parity.make_problem(cfg, lens, conv_bias=True, general_A=True)
    ci, hi = random_state(cfg, len(lens), 5)
    flags = md.MDRAFT_DT_SOFTPLUS
    o_out, o_conv, o_h = run_oracle_prefill(prob, flags, ci, hi)
    for block_channels in (128, 512):
        g_out, g_conv, g_h = run_gpu_prefill(prob, flags, (chunk_len, block_channels), ci, hi)
        assert_close(g_out, o_out, TOL[act], f"out, {block_channels}-channel blocks")
        assert_close(g_h, o_h, TOL_STATE, f"final SSM state, {block_channels}-channel blocks")
        assert np.array_equal(g_conv, o_conv)


@pytest.mark.parametrize("chunk_len", [0, 48])
def test_single_sequence_without_offsets_is_the_same_call(chunk_len):
    """cu_seqlens = NULL with one sequence means rows 0..T-1: bit for bit what cu_seqlens = [0, T] gives."""
    cfg = parity.small_config(264, "bf16", 1)
    prob = parity.make_problem(cfg, [301], conv_bias=True, general_A=True)
    tdt = torch.bfloat16
    lay = upload_layer(prob.params, "bf16", md.MDRAFT_DT_SOFTPLUS)
    dev = [to_device(a, tdt) for a in (prob.x, prob.z, prob.dt, prob.B, prob.C)]
    res = []
    for cu in (i32([0, 301]), None):
        cache = md.StateCache(1, 1, 264, act=tdt)
        out = torch.full((301, 264), float("nan"), dtype=tdt, device="cuda")
        ws = torch.empty(max(256, md.mdraft_prefill_workspace_bytes(lay, 301, 1, 301, chunk_len)), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        md.mdraft_conv_scan_prefill(lay, cache, 0, *dev, out, cu, 301, None, i32([0]), ws, chunk_len, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        res.append((out.clone(), cache.ssm.clone(), cache.conv.clone()))
    for a, b in zip(*res):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_prefill_chunking_is_only_a_schedule(act):
    """Different chunk lengths (including no chunking) agree with each other far inside the tolerance."""
    cfg = parity.small_config(128, act, 1)
    prob = parity.make_problem(cfg, [500], general_A=True)
    flags = md.MDRAFT_DT_SOFTPLUS
    base = run_gpu_prefill(prob, flags, 4096)  # one chunk
    for cl in (16, 100, 250):
        got = run_gpu_prefill(prob, flags, cl)
        assert_close(got[2], base[2], 2e-5, f"state, chunk_len={cl}")
        assert_close(got[0], base[0], 1e-5 if act == "f32" else 8e-3, f"out, chunk_len={cl}")


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_split_mode_matches_fused(act):
    """conv-only pass, then the recurrence on its output (x marked as already convolved)."""
    cfg = parity.small_config(136, act, 2)
    prob = parity.make_problem(cfg, [75, 40], conv_bias=True, general_A=True)
    ci, hi = random_state(cfg, 2, 11)
    f = md.MDRAFT_DT_SOFTPLUS
    u, conv_after, _ = run_gpu_prefill(prob, f | md.MDRAFT_CONV_ONLY, 32, ci, hi)
    o_u, o_conv, _ = oracle.prefill(oracle.layer_from_params(prob.params, f | oracle.CONV_ONLY), prob.x, prob.z, prob.dt,
                                    prob.B, prob.C, prob.cu, ci, hi)
    assert_close(u, o_u, TOL[act], "conv-only output")
    assert np.array_equal(conv_after, o_conv)
    prob2 = parity.Problem(cfg, prob.params, gen.round_to_act(u.astype(np.float32), act), prob.z, prob.dt, prob.B, prob.C, prob.cu)
    out2, _, h2 = run_gpu_prefill(prob2, f | md.MDRAFT_PRECONV, 32, ci, hi)
    o_out2, _, o_h2 = oracle.prefill(oracle.layer_from_params(prob.params, f | oracle.PRECONV), prob2.x, prob.z, prob.dt,
                                     prob.B, prob.C, prob.cu, ci, hi)
    assert_close(out2, o_out2, TOL[act], "pre-convolved output")
    assert_close(h2, o_h2, TOL_STATE, "pre-convolved state")


def test_prefill_flags_bad_sequence_lengths_and_slots():
    cfg = parity.small_config(64, "f32", 2)
    prob = parity.make_problem(cfg, [10, 12])
    lay = upload_layer(prob.params, "f32")
    cache = md.StateCache(1, 4, 64, act=torch.float32)
    x, z, dt = (to_device(a, torch.float32) for a in (prob.x, prob.z, prob.dt))
    B, C = to_device(prob.B, torch.float32), to_device(prob.C, torch.float32)
    out = torch.zeros((22, 64), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad_cu = i32([0, 30, 22])  # out of range, decreasing
    md.mdraft_conv_scan_prefill(lay, cache, 0, x, z, dt, B, C, out, bad_cu, 12, None, i32([0, 1]), None, 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) & md.MDRAFT_DEV_BAD_SEQLENS
    assert float(out.abs().max()) == 0.0, "a malformed sequence must be skipped, not guessed at"
    status.zero_()
    md.mdraft_conv_scan_prefill(lay, cache, 0, x, z, dt, B, C, out, i32(prob.cu), 12, None, i32([0, 99]), None, 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) & md.MDRAFT_DEV_BAD_SLOT
    assert float(out[:10].abs().max()) > 0 and float(out[10:].abs().max()) == 0.0


@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_batch_of_empty_sequences_moves_the_state_and_needs_no_workspace(act):
    """No tokens at all: every sequence's final state is its starting state, copied from slot to slot (zeros where
    there is no starting slot), with no workspace even when the caller's static length bound is large."""
    Dn, S = 136, 3
    tdt = torch.float32 if act == "f32" else torch.bfloat16
    cfg = parity.small_config(Dn, act, S)
    prob = parity.make_problem(cfg, [4])   # only for the layer constants
    lay = upload_layer(prob.params, act, md.MDRAFT_DT_SOFTPLUS)
    assert md.mdraft_prefill_workspace_bytes(lay, 0, S, 5000) == 0
    cache = md.StateCache(1, 2 * S, Dn, act=tdt)
    cache.ssm.normal_(); cache.conv.normal_()
    before_h, before_c = cache.ssm.clone(), cache.conv.clone()
    empty = torch.empty((0, Dn), dtype=tdt, device="cuda")
    empty_bc = torch.empty((0, 16), dtype=tdt, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    init = i32([0, -1, 2]); final = i32([3, 4, 2])
    md.mdraft_conv_scan_prefill(lay, cache, 0, empty, empty, empty, empty_bc, empty_bc, empty, i32([0, 0, 0, 0]), 5000, init, final, None, 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(cache.ssm[0, 3], before_h[0, 0]) and torch.equal(cache.conv[0, 3], before_c[0, 0])
    assert float(cache.ssm[0, 4].abs().max()) == 0.0 and float(cache.conv[0, 4].float().abs().max()) == 0.0
    for s in (0, 1, 2, 5):
        assert torch.equal(cache.ssm[0, s], before_h[0, s]) and torch.equal(cache.conv[0, s], before_c[0, s])
