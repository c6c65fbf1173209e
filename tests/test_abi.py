"""The C-ABI library builds for sm_100a, loads without a GPU, exports every function the header declares,
and rejects bad arguments on the host before anything is launched (no GPU needed: no launch happens)."""

import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_01206_b200.build import build_library
    from paper_2506_01206_b200 import binding
    build_library()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mdraft.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mdraft_[a-zA-Z0-9_]+)\s*\(", text)))


def test_header_and_library_agree(lib):
    from paper_2506_01206_b200 import binding
    names = declared_functions()
    assert "mdraft_conv_scan_prefill" in names and "mdraft_tree_step" in names and "mdraft_state_commit" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/mdraft.h but not exported"
    assert sorted(binding.EXPORTS) == names, "the Python binding must expose exactly the declared entry points"
    assert lib.mdraft_version() >= 100
    assert lib.mdraft_status_string(0) == b"ok"
    assert b"16 bytes" in lib.mdraft_status_string(-3)


def _layer(binding, **kw):
    base = dict(d_inner=64, d_state=16, d_conv=4, act=0, flags=1, reserved=0, A=0x1000, D=0, conv_w=0x2000, conv_b=0, dt_bias=0)
    base.update(kw)
    return binding._Layer(*[base[k] for k in ("d_inner", "d_state", "d_conv", "act", "flags", "reserved", "A", "D", "conv_w", "conv_b", "dt_bias")])


def _cache(binding, **kw):
    base = dict(ssm=0x10000, ssm_layer_stride=4 * 1024, ssm_slot_stride=1024, conv=0x20000, conv_layer_stride=4 * 192,
                conv_slot_stride=192, n_layers=1, n_slots=4)
    base.update(kw)
    return binding._Cache(*[base[k] for k in ("ssm", "ssm_layer_stride", "ssm_slot_stride", "conv", "conv_layer_stride", "conv_slot_stride", "n_layers", "n_slots")])


def _prefill(lib, binding, layer, cache, **kw):
    a = dict(x=0x100000, ldx=64, z=0x200000, ldz=64, dt=0x300000, lddt=64, B=0x400000, ldb=16, C=0x500000, ldc=16,
             out=0x600000, ldo=64, T=8, n_seq=1, max_seqlen=8, cu=0x700000, init=None, final=None, ws=None, ws_bytes=0, opts=None)
    a.update(kw)
    return lib.mdraft_conv_scan_prefill(C.byref(layer), C.byref(cache) if cache is not None else None, 0,
                                        a["x"], a["ldx"], a["z"], a["ldz"], a["dt"], a["lddt"], a["B"], a["ldb"], a["C"], a["ldc"],
                                        a["out"], a["ldo"], a["T"], a["n_seq"], a["max_seqlen"], a["cu"], a["init"], a["final"],
                                        a["ws"], a["ws_bytes"], a["opts"], None, None)


def test_host_side_argument_checks(lib):
    from paper_2506_01206_b200 import binding
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = -1, -2, -3, -4
    ok_layer, ok_cache = _layer(binding), _cache(binding)
    assert _prefill(lib, binding, _layer(binding, d_state=8), ok_cache) == UNSUPPORTED
    assert _prefill(lib, binding, _layer(binding, d_conv=3), ok_cache) == UNSUPPORTED
    assert _prefill(lib, binding, _layer(binding, d_inner=60), ok_cache) == UNSUPPORTED
    assert _prefill(lib, binding, _layer(binding, act=7), ok_cache) == UNSUPPORTED
    assert _prefill(lib, binding, _layer(binding, A=0), ok_cache) == INVALID
    assert _prefill(lib, binding, _layer(binding, flags=2 | 4), ok_cache) == INVALID
    assert _prefill(lib, binding, ok_layer, ok_cache, x=None) == INVALID
    assert _prefill(lib, binding, ok_layer, ok_cache, cu=None, n_seq=2) == INVALID   # offsets may be left out for one sequence only
    assert _prefill(lib, binding, ok_layer, ok_cache, ldx=32) == INVALID          # stride shorter than a row
    assert _prefill(lib, binding, ok_layer, ok_cache, x=0x100004) == MISALIGNED
    assert _prefill(lib, binding, ok_layer, ok_cache, ldb=18) == MISALIGNED       # 72-byte rows
    assert _prefill(lib, binding, ok_layer, ok_cache, T=-1) == INVALID
    assert _prefill(lib, binding, ok_layer, None, final=0x800000) == INVALID      # slots named but no pool
    assert _prefill(lib, binding, ok_layer, _cache(binding, ssm_slot_stride=1000)) == INVALID
    assert _prefill(lib, binding, ok_layer, _cache(binding, conv_slot_stride=194)) == MISALIGNED
    # chunked plan without a workspace
    opts = binding._PrefillOpts(); opts.chunk_len = 4
    assert _prefill(lib, binding, ok_layer, ok_cache, opts=C.byref(opts)) == WORKSPACE
    need = lib.mdraft_prefill_workspace_bytes(C.byref(ok_layer), 8, 1, 8, C.byref(opts))
    assert need > 0 and need % 256 == 0
    assert _prefill(lib, binding, ok_layer, ok_cache, opts=C.byref(opts), ws=0x900000, ws_bytes=need - 1) == WORKSPACE
    assert _prefill(lib, binding, ok_layer, ok_cache, opts=C.byref(opts), ws=0x900010, ws_bytes=need) == MISALIGNED
    bad = binding._PrefillOpts(); bad.chunk_len = 8; bad.reserved[1] = 1
    assert _prefill(lib, binding, ok_layer, ok_cache, opts=C.byref(bad)) == INVALID
    # nothing to do is fine and launches nothing
    assert _prefill(lib, binding, ok_layer, ok_cache, n_seq=0, T=0, cu=None) == 0
    # A batch of empty sequences needs no workspace whatever static length bound comes with it: the query says 0 and
    # the call must agree (it may only fail later, at the launch, where there is no GPU).
    assert lib.mdraft_prefill_workspace_bytes(C.byref(ok_layer), 0, 2, 5000, None) == 0
    assert _prefill(lib, binding, ok_layer, ok_cache, T=0, n_seq=2, max_seqlen=5000, x=None, z=None, dt=None, B=None, C=None, out=None,
                    final=0x800000) != WORKSPACE
    # and a static bound looser than the batch itself does not change the plan
    assert lib.mdraft_prefill_workspace_bytes(C.byref(ok_layer), 8, 1, 100000, C.byref(opts)) == need

    def tree(layer=ok_layer, cache=ok_cache, n=4, parent=0xA00000, node=0xB00000, n_levels=1, levels=None, x=0x100000):
        return lib.mdraft_tree_step(C.byref(layer), C.byref(cache) if cache is not None else None, 0, x, 64, 0x200000, 64,
                                    0x300000, 64, 0x400000, 16, 0x500000, 16, 0x600000, 64, n, parent, node, n_levels, levels, None, None)

    assert tree(cache=None) == INVALID
    assert tree(parent=None) == INVALID
    assert tree(n=0) == 0
    assert tree(n_levels=2) == INVALID                                  # several levels need their offsets
    assert tree(n_levels=2, levels=(C.c_int32 * 3)(0, 3, 5)) == INVALID     # must end at n_nodes
    assert tree(n_levels=2, levels=(C.c_int32 * 3)(0, 5, 4)) == INVALID     # must not decrease
    assert tree(layer=_layer(binding, d_state=32)) == UNSUPPORTED
    assert tree(x=0x100002) == MISALIGNED

    def commit(cache=ok_cache, d_inner=64, n=2, src=0xA00000, dst=0xB00000, act=0, d_state=16):
        return lib.mdraft_state_commit(C.byref(cache) if cache is not None else None, d_inner, d_state, 4, act, n, src, dst, None, None)

    assert commit(cache=None) == INVALID
    assert commit(src=None) == INVALID
    assert commit(n=0) == 0
    assert commit(d_state=4) == UNSUPPORTED
    assert commit(cache=_cache(binding, ssm_slot_stride=1026)) == MISALIGNED


def test_missing_library_is_a_loud_error(tmp_path):
    from paper_2506_01206_b200 import binding
    with pytest.raises(ImportError):
        binding.load_library(str(tmp_path / "nope.so"))


def test_projection_step_host_side_checks(lib):
    """mdraft_tree_step_proj turns bad arguments away before any launch (so this runs without a GPU)."""
    from paper_2506_01206_b200 import binding
    INVALID, UNSUPPORTED, MISALIGNED = -1, -2, -3
    layer, cache = _layer(binding), _cache(binding)

    def call(layer=layer, cache=cache, W_x=0x900000, W_dt=0xA00000, rank=8, npc=0, x=0x100000, z=0x200000, out=0x600000, n=1,
             par=0x700000, nod=0x800000, ldx=64):
        pr = binding._SelectProj(W_x, W_dt, rank, npc)
        return lib.mdraft_tree_step_proj(C.byref(layer), C.byref(cache), 0, C.byref(pr) if W_x is not None else None, x, ldx, z, 64, out, 64,
                                         n, par, nod, None, None)

    assert call(rank=12) == UNSUPPORTED            # not a multiple of 8
    assert call(rank=264) == UNSUPPORTED           # beyond the shared-memory vectors
    assert call(rank=0) == UNSUPPORTED
    big = _cache(binding, ssm_slot_stride=4104 * 16, ssm_layer_stride=4 * 4104 * 16, conv_slot_stride=3 * 4104, conv_layer_stride=12 * 4104)
    assert call(layer=_layer(binding, d_inner=4104), cache=big, ldx=4104) == UNSUPPORTED   # more than one cluster of the widest blocks
    assert call(layer=_layer(binding, flags=1 | 2)) == INVALID           # pre-convolved input makes no sense here
    assert call(layer=_layer(binding, flags=1 | 4)) == INVALID
    assert call(W_x=None) == INVALID
    assert call(W_dt=0) == INVALID
    assert call(W_x=0x900008) == MISALIGNED
    assert call(npc=3) == INVALID
    assert call(n=-1) == INVALID
    assert call(x=None) == INVALID
    assert call(ldx=32) == INVALID
    assert call(par=None) == INVALID
    assert call(n=0, par=None, nod=None) == 0      # nothing to do is not an error


def test_prefill_plan_seen_through_the_workspace_query(lib):
    """The chunk plan is host logic; its workspace query shows it: one wave of equal chunks for a single sequence at
    any length (so the scratch stops growing with the context), several waves of short chunks for a packed batch."""
    from paper_2506_01206_b200 import binding
    layer = _layer(binding, d_inner=1536, act=1)
    q = lambda T, S, mx, opts=None: lib.mdraft_prefill_workspace_bytes(C.byref(layer), T, S, mx, opts)
    per_chunk = 1536 * 16 * 4 + 1536 * 4          # one summary: state + summed step size
    assert q(8, 1, 8) == 0                         # shorter than one chunk: nothing to carry
    one = [q(T, 1, T) for T in (2048, 8192, 32768, 131072)]
    assert all(b > 0 for b in one)
    assert max(one) <= 52 * per_chunk + 4 * per_chunk, "a single sequence stays at about 49 chunks whatever its length"
    packed = q(141650, 32, 8192)
    assert packed > 10 * max(one), "a packed batch is cut into many short chunks"
    o = binding._PrefillOpts(chunk_len=64, block_channels=0)
    assert q(2048, 1, 2048, C.byref(o)) >= 32 * per_chunk      # a forced chunk length is honoured
    assert q(0, 1, 8) == 0 and q(8, 0, 8) == 0     # nonsense sizes give 0, not garbage


def test_ssd_host_side_checks(lib):
    """The SSD entry points turn unsupported shapes and bad arguments away before any launch."""
    from paper_2506_01206_b200 import binding
    INVALID, UNSUPPORTED, MISALIGNED, WORKSPACE = -1, -2, -3, -4

    def layer(**kw):
        base = dict(d_inner=128, headdim=64, d_state=128, d_conv=4, act=1, flags=1, A=0x1000, D=0, conv_w=0x2000, conv_b=0, dt_bias=0)
        base.update(kw)
        return binding._SsdLayer(*[base[k] for k in ("d_inner", "headdim", "d_state", "d_conv", "act", "flags", "A", "D", "conv_w", "conv_b", "dt_bias")])

    cache = _cache(binding, ssm_slot_stride=128 * 128, ssm_layer_stride=4 * 128 * 128, conv_slot_stride=3 * 128, conv_layer_stride=12 * 128)

    def prefill(lay=None, cache=cache, T=300, n_seq=1, x=0x100000, ldx=128, dt=0x300000, lddt=2, B=0x400000, ldb=128, ws=0x900000, ws_bytes=1 << 30, cu=None):
        lay = lay or layer()
        return lib.mdraft_ssd_prefill(C.byref(lay), C.byref(cache) if cache is not None else None, 0, x, ldx, 0x200000, 128, dt, lddt, B, ldb,
                                      0x500000, 128, 0x600000, 128, T, n_seq, cu, None, 0x800000, ws, ws_bytes, None, None)

    ok = layer()
    need = lib.mdraft_ssd_prefill_workspace_bytes(C.byref(ok), 300, 1)
    assert need > 0 and need % 256 == 0
    assert lib.mdraft_ssd_prefill_workspace_bytes(C.byref(layer(headdim=32)), 300, 1) == 0
    assert prefill(lay=layer(headdim=32)) == UNSUPPORTED
    assert prefill(lay=layer(d_state=16)) == UNSUPPORTED
    assert prefill(lay=layer(act=0)) == UNSUPPORTED            # bf16 activations only
    assert prefill(lay=layer(d_inner=96)) == UNSUPPORTED       # whole heads only
    assert prefill(lay=layer(flags=2)) == INVALID              # only the softplus flag has a meaning here
    assert prefill(lay=layer(A=0)) == INVALID
    assert prefill(x=None) == INVALID
    assert prefill(lddt=1) == INVALID                          # dt rows shorter than the head count
    assert prefill(ldb=64) == INVALID
    assert prefill(B=0x400008) == MISALIGNED
    assert prefill(ws=None) == WORKSPACE
    assert prefill(ws_bytes=need - 1) == WORKSPACE
    assert prefill(ws=0x900010) == MISALIGNED
    assert prefill(n_seq=2) == INVALID                         # offsets may be left out for one sequence only
    small = _cache(binding)                                    # slots sized for 16 states
    assert prefill(cache=small) == INVALID
    assert prefill(n_seq=0, T=0) == 0

    def step(lay=None, cache=cache, n=2, par=0x700000, nod=0x800000, n_levels=1, levels=None, lddt=2):
        lay = lay or layer()
        return lib.mdraft_ssd_tree_step(C.byref(lay), C.byref(cache) if cache is not None else None, 0, 0x100000, 128, 0x200000, 128, 0x300000, lddt,
                                        0x400000, 128, 0x500000, 128, 0x600000, 128, n, par, nod, n_levels, levels, None, None)

    assert step(cache=None) == INVALID
    assert step(par=None) == INVALID
    assert step(n=0) == 0
    assert step(n_levels=2) == INVALID
    assert step(lay=layer(d_conv=3)) == UNSUPPORTED
    assert step(lddt=1) == INVALID
    # the commit call moves 128-state slots too, and nothing between the two sizes
    commit = lambda ds: lib.mdraft_state_commit(C.byref(cache), 128, ds, 4, 1, 0, None, None, None, None)
    assert commit(128) == 0 and commit(64) == UNSUPPORTED
