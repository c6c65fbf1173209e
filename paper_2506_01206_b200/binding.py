"""ctypes binding of ``libmdraft.so`` — argument marshalling only.

Every function here has the name of the C entry point it calls (see
``include/mdraft.h``) and does nothing but turn torch tensors into pointers,
strides and sizes.  All computation happens in the CUDA library; there is no
fallback of any kind: if the library is missing or a call fails, an exception
is raised.  PyTorch is used for device memory and streams only.
"""

from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmdraft.so")

MDRAFT_F32, MDRAFT_BF16 = 0, 1
MDRAFT_DT_SOFTPLUS, MDRAFT_PRECONV, MDRAFT_CONV_ONLY, MDRAFT_A_POWERS = 1, 2, 4, 8
MDRAFT_DEV_BAD_SLOT, MDRAFT_DEV_BAD_SEQLENS, MDRAFT_DEV_WAIT_EXPIRED = 1, 2, 4

EXPORTS = (
    "mdraft_prefill_workspace_bytes", "mdraft_conv_scan_prefill", "mdraft_conv_scan_prefill_noalloc", "mdraft_tree_step",
    "mdraft_tree_step_proj", "mdraft_state_commit", "mdraft_classify_A", "mdraft_status_string", "mdraft_version",
    "mdraft_ucb_reward", "mdraft_ucb_select", "mdraft_ucb_update",
    "mdraft_ssd_prefill_workspace_bytes", "mdraft_ssd_prefill", "mdraft_ssd_tree_step",
)


class MdraftError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Layer(C.Structure):
    _fields_ = [("d_inner", C.c_int32), ("d_state", C.c_int32), ("d_conv", C.c_int32), ("act", C.c_int32),
                ("flags", C.c_uint32), ("reserved", C.c_uint32),
                ("A", C.c_void_p), ("D", C.c_void_p), ("conv_w", C.c_void_p), ("conv_b", C.c_void_p),
                ("dt_bias", C.c_void_p)]


class _Cache(C.Structure):
    _fields_ = [("ssm", C.c_void_p), ("ssm_layer_stride", C.c_int64), ("ssm_slot_stride", C.c_int64),
                ("conv", C.c_void_p), ("conv_layer_stride", C.c_int64), ("conv_slot_stride", C.c_int64),
                ("n_layers", C.c_int32), ("n_slots", C.c_int32)]


class _PrefillOpts(C.Structure):
    _fields_ = [("chunk_len", C.c_int32), ("block_channels", C.c_int32), ("reserved", C.c_int32 * 2),
                ("event_after_chunk_state", C.c_void_p), ("event_after_carry_scan", C.c_void_p)]


class _SelectProj(C.Structure):
    _fields_ = [("W_x", C.c_void_p), ("W_dt", C.c_void_p), ("dt_rank", C.c_int32), ("nodes_per_cluster", C.c_int32)]


class _SsdLayer(C.Structure):
    _fields_ = [("d_inner", C.c_int32), ("headdim", C.c_int32), ("d_state", C.c_int32), ("d_conv", C.c_int32),
                ("act", C.c_int32), ("flags", C.c_uint32),
                ("A", C.c_void_p), ("D", C.c_void_p), ("conv_w", C.c_void_p), ("conv_b", C.c_void_p), ("dt_bias", C.c_void_p)]


class _Ucb(C.Structure):
    _fields_ = [("n_arms", C.c_int32), ("reserved", C.c_int32), ("round", C.c_int64), ("lambda_ucb", C.c_double),
                ("lambda_gamma", C.c_double), ("reward_sum", C.POINTER(C.c_double)), ("count", C.POINTER(C.c_int64))]


_lib = None


def load_library(path: Optional[str] = None):
    """Load the CUDA library; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ImportError(f"{p} not found: build it with `python -m paper_2506_01206_b200.build` "
                          "(nvcc, sm_100a); this package has no fallback path")
    lib = C.CDLL(p)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.mdraft_status_string.restype = C.c_char_p
    lib.mdraft_status_string.argtypes = [C.c_int]
    lib.mdraft_version.restype = C.c_int
    lib.mdraft_version.argtypes = []
    lib.mdraft_prefill_workspace_bytes.restype = C.c_size_t
    lib.mdraft_prefill_workspace_bytes.argtypes = [C.POINTER(_Layer), i32, i32, i32, C.POINTER(_PrefillOpts)]
    lib.mdraft_conv_scan_prefill.restype = C.c_int
    lib.mdraft_conv_scan_prefill.argtypes = [C.POINTER(_Layer), C.POINTER(_Cache), i32,
                                             vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                             i32, i32, i32, vp, vp, vp, vp, C.c_size_t, C.POINTER(_PrefillOpts), vp, vp]
    lib.mdraft_conv_scan_prefill_noalloc.restype = C.c_int
    lib.mdraft_conv_scan_prefill_noalloc.argtypes = [C.POINTER(_Layer), C.POINTER(_Cache), i32,
                                                     vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                                     i32, i32, i32, vp, vp, vp, C.POINTER(_PrefillOpts), vp, vp]
    lib.mdraft_tree_step.restype = C.c_int
    lib.mdraft_tree_step.argtypes = [C.POINTER(_Layer), C.POINTER(_Cache), i32,
                                     vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                     i32, vp, vp, i32, C.POINTER(i32), vp, vp]
    lib.mdraft_tree_step_proj.restype = C.c_int
    lib.mdraft_tree_step_proj.argtypes = [C.POINTER(_Layer), C.POINTER(_Cache), i32, C.POINTER(_SelectProj),
                                          vp, i64, vp, i64, vp, i64, i32, vp, vp, vp, vp]
    lib.mdraft_state_commit.restype = C.c_int
    lib.mdraft_state_commit.argtypes = [C.POINTER(_Cache), i32, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.mdraft_classify_A.restype = C.c_int
    lib.mdraft_classify_A.argtypes = [vp, i32, i32, vp, C.POINTER(i32), C.POINTER(i32), vp]
    lib.mdraft_ucb_reward.restype = C.c_double
    lib.mdraft_ucb_reward.argtypes = [C.c_double, i32, i32]
    lib.mdraft_ucb_select.restype = C.c_int
    lib.mdraft_ucb_select.argtypes = [C.POINTER(_Ucb), C.POINTER(i32)]
    lib.mdraft_ucb_update.restype = C.c_int
    lib.mdraft_ucb_update.argtypes = [C.POINTER(_Ucb), i32, i32, i32]
    lib.mdraft_ssd_prefill_workspace_bytes.restype = C.c_size_t
    lib.mdraft_ssd_prefill_workspace_bytes.argtypes = [C.POINTER(_SsdLayer), i32, i32]
    lib.mdraft_ssd_prefill.restype = C.c_int
    lib.mdraft_ssd_prefill.argtypes = [C.POINTER(_SsdLayer), C.POINTER(_Cache), i32,
                                       vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                       i32, i32, vp, vp, vp, vp, C.c_size_t, vp, vp]
    lib.mdraft_ssd_tree_step.restype = C.c_int
    lib.mdraft_ssd_tree_step.argtypes = [C.POINTER(_SsdLayer), C.POINTER(_Cache), i32,
                                         vp, i64, vp, i64, vp, i64, vp, i64, vp, i64, vp, i64,
                                         i32, vp, vp, i32, C.POINTER(i32), vp, vp]
    if path is None:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().mdraft_status_string(int(status)).decode()


def mdraft_version() -> int:
    return int(load_library().mdraft_version())


def _act_of(dtype: torch.dtype) -> int:
    if dtype == torch.float32:
        return MDRAFT_F32
    if dtype == torch.bfloat16:
        return MDRAFT_BF16
    raise TypeError(f"activation dtype must be float32 or bfloat16, got {dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _mat(t: Optional[torch.Tensor], name: str):
    """(pointer, row stride in elements) of a 2-D tensor whose last dim is contiguous."""
    if t is None:
        return None, 0
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: need a 2-D tensor with unit stride along the last dim")
    if not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    return C.c_void_p(t.data_ptr()), int(t.stride(0))


def _stream_ptr(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream))


def _f32(t: Optional[torch.Tensor], n: int, name: str) -> Optional[torch.Tensor]:
    if t is None:
        return None
    if t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != n or not t.is_cuda:
        raise ValueError(f"{name}: need a contiguous float32 CUDA tensor of {n} elements")
    return t


@dataclass
class Layer:
    """Per-layer constants on the device (fp32) plus the descriptor handed to the library."""
    A: torch.Tensor
    D: Optional[torch.Tensor]
    conv_w: torch.Tensor
    conv_b: Optional[torch.Tensor]
    dt_bias: Optional[torch.Tensor]
    act: torch.dtype
    flags: int = MDRAFT_DT_SOFTPLUS

    def __post_init__(self):
        Dn, N = self.A.shape
        W = self.conv_w.shape[1]
        _f32(self.A, Dn * N, "A"); _f32(self.conv_w, Dn * W, "conv_w")
        _f32(self.D, Dn, "D"); _f32(self.conv_b, Dn, "conv_b"); _f32(self.dt_bias, Dn, "dt_bias")
        self.d_inner, self.d_state, self.d_conv = int(Dn), int(N), int(W)

    def c(self, flags: Optional[int] = None) -> _Layer:
        return _Layer(self.d_inner, self.d_state, self.d_conv, _act_of(self.act),
                      self.flags if flags is None else int(flags), 0,
                      self.A.data_ptr(), 0 if self.D is None else self.D.data_ptr(), self.conv_w.data_ptr(),
                      0 if self.conv_b is None else self.conv_b.data_ptr(),
                      0 if self.dt_bias is None else self.dt_bias.data_ptr())


class StateCache:
    """Slot pool: ssm (n_layers, n_slots, D, N) fp32 and conv (n_layers, n_slots, W-1, D) activations."""

    def __init__(self, n_layers: int, n_slots: int, d_inner: int, d_state: int = 16, d_conv: int = 4,
                 act: torch.dtype = torch.bfloat16, device="cuda", zero: bool = True):
        alloc = torch.zeros if zero else torch.empty
        self.ssm = alloc((n_layers, n_slots, d_inner, d_state), dtype=torch.float32, device=device)
        self.conv = alloc((n_layers, n_slots, d_conv - 1, d_inner), dtype=act, device=device)
        self.n_layers, self.n_slots, self.d_inner, self.d_state, self.d_conv, self.act = n_layers, n_slots, d_inner, d_state, d_conv, act

    def c(self) -> _Cache:
        return _Cache(self.ssm.data_ptr(), self.ssm.stride(0), self.ssm.stride(1),
                      self.conv.data_ptr(), self.conv.stride(0), self.conv.stride(1), self.n_layers, self.n_slots)

    def nbytes(self) -> int:
        return self.ssm.numel() * 4 + self.conv.numel() * self.conv.element_size()


def _opts(chunk_len, phase_events=None):
    """chunk_len: tokens per chunk (0 = library's plan), or a pair (chunk_len, block_channels)."""
    block_channels = 0
    if isinstance(chunk_len, (tuple, list)):
        chunk_len, block_channels = chunk_len
    if not chunk_len and not block_channels and phase_events is None:
        return None
    o = _PrefillOpts()
    o.chunk_len = int(chunk_len)
    o.block_channels = int(block_channels)
    if phase_events is not None:  # two torch.cuda.Event objects (already created with enable_timing=True)
        o.event_after_chunk_state = phase_events[0].cuda_event
        o.event_after_carry_scan = phase_events[1].cuda_event
    return C.byref(o)


def mdraft_prefill_workspace_bytes(layer: Layer, total_tokens: int, n_seq: int, max_seqlen: int, chunk_len: int = 0,
                                   flags: Optional[int] = None) -> int:
    cl = layer.c(flags)
    return int(load_library().mdraft_prefill_workspace_bytes(C.byref(cl), int(total_tokens), int(n_seq), int(max_seqlen), _opts(chunk_len)))


def mdraft_conv_scan_prefill(layer: Layer, cache: Optional[StateCache], layer_index: int,
                             x, z, dt, B, Cm, out, cu_seqlens: Optional[torch.Tensor], max_seqlen: int,
                             init_slot: Optional[torch.Tensor] = None, final_slot: Optional[torch.Tensor] = None,
                             workspace: Optional[torch.Tensor] = None, chunk_len: int = 0,
                             dev_status: Optional[torch.Tensor] = None, stream=None, flags: Optional[int] = None,
                             phase_events=None) -> None:
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c() if cache is not None else None
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); pdt, lddt = _mat(dt, "dt")
    pB, ldb = _mat(B, "B"); pC, ldc = _mat(Cm, "C"); po, ldo = _mat(out, "out")
    T = int(x.shape[0])
    n_seq = 1 if cu_seqlens is None else int(cu_seqlens.numel()) - 1   # None: a single sequence of all T rows
    if cu_seqlens is not None and cu_seqlens.dtype != torch.int32:
        raise TypeError("cu_seqlens must be int32")
    for t, nm in ((init_slot, "init_slot"), (final_slot, "final_slot")):
        if t is not None and (t.dtype != torch.int32 or t.numel() != n_seq):
            raise TypeError(f"{nm} must be int32 with one entry per sequence")
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (C.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    rc = lib.mdraft_conv_scan_prefill(C.byref(cl), C.byref(cc) if cc is not None else None, int(layer_index),
                                      px, ldx, pz, ldz, pdt, lddt, pB, ldb, pC, ldc, po, ldo,
                                      T, n_seq, int(max_seqlen), _ptr(cu_seqlens), _ptr(init_slot), _ptr(final_slot),
                                      ws_ptr, ws_bytes, _opts(chunk_len, phase_events), _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_conv_scan_prefill")


NOALLOC_SCRATCH_BYTES = 8 << 20


def mdraft_conv_scan_prefill_noalloc(layer: Layer, cache: Optional[StateCache], layer_index: int,
                                     x, z, dt, B, Cm, out, cu_seqlens: Optional[torch.Tensor], max_seqlen: int,
                                     init_slot: Optional[torch.Tensor] = None, final_slot: Optional[torch.Tensor] = None,
                                     chunk_len: int = 0, dev_status: Optional[torch.Tensor] = None, stream=None,
                                     flags: Optional[int] = None) -> None:
    """Prefill without a caller workspace: the library's own fixed scratch array is used (see the header for
    who needs this and for the sharing rules).  Raises MdraftError(MDRAFT_ERR_WORKSPACE) when the problem needs
    more than NOALLOC_SCRATCH_BYTES of scratch."""
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c() if cache is not None else None
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); pdt, lddt = _mat(dt, "dt")
    pB, ldb = _mat(B, "B"); pC, ldc = _mat(Cm, "C"); po, ldo = _mat(out, "out")
    T = int(x.shape[0])
    n_seq = 1 if cu_seqlens is None else int(cu_seqlens.numel()) - 1   # None: a single sequence of all T rows
    if cu_seqlens is not None and cu_seqlens.dtype != torch.int32:
        raise TypeError("cu_seqlens must be int32")
    for t, nm in ((init_slot, "init_slot"), (final_slot, "final_slot")):
        if t is not None and (t.dtype != torch.int32 or t.numel() != n_seq):
            raise TypeError(f"{nm} must be int32 with one entry per sequence")
    rc = lib.mdraft_conv_scan_prefill_noalloc(C.byref(cl), C.byref(cc) if cc is not None else None, int(layer_index),
                                              px, ldx, pz, ldz, pdt, lddt, pB, ldb, pC, ldc, po, ldo,
                                              T, n_seq, int(max_seqlen), _ptr(cu_seqlens), _ptr(init_slot), _ptr(final_slot),
                                              _opts(chunk_len), _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_conv_scan_prefill_noalloc")


def mdraft_tree_step(layer: Layer, cache: StateCache, layer_index: int, x, z, dt, B, Cm, out,
                     parent_slot: torch.Tensor, node_slot: torch.Tensor,
                     level_offsets: Optional[Sequence[int]] = None,
                     dev_status: Optional[torch.Tensor] = None, stream=None, flags: Optional[int] = None) -> None:
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c()
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); pdt, lddt = _mat(dt, "dt")
    pB, ldb = _mat(B, "B"); pC, ldc = _mat(Cm, "C"); po, ldo = _mat(out, "out")
    M = int(x.shape[0])
    if parent_slot.dtype != torch.int32 or node_slot.dtype != torch.int32:
        raise TypeError("slot index arrays must be int32")
    if parent_slot.numel() != M or node_slot.numel() != M:
        raise ValueError("one parent slot and one node slot per node")
    if level_offsets is None:
        n_levels, lo = 1, None
    else:
        n_levels = len(level_offsets) - 1
        lo = (C.c_int32 * (n_levels + 1))(*[int(v) for v in level_offsets])
    rc = lib.mdraft_tree_step(C.byref(cl), C.byref(cc), int(layer_index),
                              px, ldx, pz, ldz, pdt, lddt, pB, ldb, pC, ldc, po, ldo,
                              M, _ptr(parent_slot), _ptr(node_slot), n_levels, lo, _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_tree_step")


def mdraft_tree_step_proj(layer: Layer, cache: StateCache, layer_index: int, W_x: torch.Tensor, W_dt: torch.Tensor,
                          x, z, out, parent_slot: torch.Tensor, node_slot: torch.Tensor,
                          dev_status: Optional[torch.Tensor] = None, stream=None, flags: Optional[int] = None,
                          nodes_per_cluster: int = 0) -> None:
    """One tree level where dt, B and C come from the block's projections of the conv output.
    W_x: (dt_rank + 2 N, D) and W_dt: (D, dt_rank), contiguous, in the layer's activation dtype."""
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c()
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); po, ldo = _mat(out, "out")
    M = int(x.shape[0])
    if parent_slot.dtype != torch.int32 or node_slot.dtype != torch.int32:
        raise TypeError("slot index arrays must be int32")
    if parent_slot.numel() != M or node_slot.numel() != M:
        raise ValueError("one parent slot and one node slot per node")
    if W_x.dtype != x.dtype or W_dt.dtype != x.dtype or not W_x.is_contiguous() or not W_dt.is_contiguous():
        raise TypeError("W_x and W_dt must be contiguous and of the activation dtype")
    R = int(W_dt.shape[1])
    if tuple(W_dt.shape) != (layer.d_inner, R) or tuple(W_x.shape) != (R + 2 * layer.d_state, layer.d_inner):
        raise ValueError("W_x must be (dt_rank + 2 d_state, d_inner) and W_dt (d_inner, dt_rank)")
    pr = _SelectProj(W_x.data_ptr(), W_dt.data_ptr(), R, int(nodes_per_cluster))
    rc = lib.mdraft_tree_step_proj(C.byref(cl), C.byref(cc), int(layer_index), C.byref(pr), px, ldx, pz, ldz, po, ldo,
                                   M, _ptr(parent_slot), _ptr(node_slot), _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_tree_step_proj")


def mdraft_state_commit(cache: StateCache, src_slot: torch.Tensor, dst_slot: torch.Tensor,
                        dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    lib = load_library()
    cc = cache.c()
    if src_slot.dtype != torch.int32 or dst_slot.dtype != torch.int32 or src_slot.numel() != dst_slot.numel():
        raise TypeError("src_slot / dst_slot must be int32 arrays of equal length")
    rc = lib.mdraft_state_commit(C.byref(cc), cache.d_inner, cache.d_state, cache.d_conv, _act_of(cache.act),
                                 int(src_slot.numel()), _ptr(src_slot), _ptr(dst_slot), _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_state_commit")


def mdraft_classify_A(A: torch.Tensor, stream=None):
    """(is_powers, is_nonpositive) for a (D, N) fp32 device tensor; synchronises the stream."""
    lib = load_library()
    _f32(A, A.numel(), "A")
    scratch = torch.zeros(2, dtype=torch.int32, device=A.device)
    a, b = C.c_int32(0), C.c_int32(0)
    rc = lib.mdraft_classify_A(_ptr(A), int(A.shape[0]), int(A.shape[1]), _ptr(scratch), C.byref(a), C.byref(b), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_classify_A")
    return bool(a.value), bool(b.value)


class UcbBandit:
    """Arm statistics of the tree-configuration bandit, owned here, updated by the library (host code, no GPU)."""

    def __init__(self, n_arms: int, lambda_ucb: float, lambda_gamma: float):
        self._sum = (C.c_double * n_arms)()
        self._cnt = (C.c_int64 * n_arms)()
        self._c = _Ucb(int(n_arms), 0, 0, float(lambda_ucb), float(lambda_gamma), self._sum, self._cnt)

    def mdraft_ucb_select(self) -> int:
        arm = C.c_int32(-1)
        rc = load_library().mdraft_ucb_select(C.byref(self._c), C.byref(arm))
        if rc != 0:
            raise MdraftError(rc, "mdraft_ucb_select")
        return int(arm.value)

    def mdraft_ucb_update(self, arm: int, draft_len: int, n_accept: int) -> None:
        rc = load_library().mdraft_ucb_update(C.byref(self._c), int(arm), int(draft_len), int(n_accept))
        if rc != 0:
            raise MdraftError(rc, "mdraft_ucb_update")

    @property
    def reward_sum(self):
        return list(self._sum)

    @property
    def count(self):
        return list(self._cnt)

    @property
    def round(self) -> int:
        return int(self._c.round)


def mdraft_ucb_reward(lambda_gamma: float, draft_len: int, n_accept: int) -> float:
    return float(load_library().mdraft_ucb_reward(float(lambda_gamma), int(draft_len), int(n_accept)))


# ---------------------------------------------------------------- Mamba-2 (SSD) layer
@dataclass
class SsdLayer:
    """Constants of an SSD layer on the device (fp32): A (H,), dt_bias (H,), D (D,), conv taps (D, W)."""
    A: torch.Tensor
    D: Optional[torch.Tensor]
    conv_w: torch.Tensor
    conv_b: Optional[torch.Tensor]
    dt_bias: Optional[torch.Tensor]
    headdim: int = 64
    d_state: int = 128
    flags: int = MDRAFT_DT_SOFTPLUS

    def __post_init__(self):
        Dn, W = self.conv_w.shape
        H = int(self.A.numel())
        if H * self.headdim != Dn:
            raise ValueError("A must hold one value per head of `headdim` channels")
        _f32(self.A, H, "A"); _f32(self.conv_w, Dn * W, "conv_w")
        _f32(self.D, Dn, "D"); _f32(self.conv_b, Dn, "conv_b"); _f32(self.dt_bias, H, "dt_bias")
        self.d_inner, self.n_heads, self.d_conv = int(Dn), H, int(W)

    def c(self, flags: Optional[int] = None) -> _SsdLayer:
        return _SsdLayer(self.d_inner, self.headdim, self.d_state, self.d_conv, MDRAFT_BF16,
                         self.flags if flags is None else int(flags),
                         self.A.data_ptr(), 0 if self.D is None else self.D.data_ptr(), self.conv_w.data_ptr(),
                         0 if self.conv_b is None else self.conv_b.data_ptr(),
                         0 if self.dt_bias is None else self.dt_bias.data_ptr())


def mdraft_ssd_prefill_workspace_bytes(layer: SsdLayer, total_tokens: int, n_seq: int) -> int:
    cl = layer.c()
    return int(load_library().mdraft_ssd_prefill_workspace_bytes(C.byref(cl), int(total_tokens), int(n_seq)))


def mdraft_ssd_prefill(layer: SsdLayer, cache: Optional[StateCache], layer_index: int, x, z, dt, B, Cm, out,
                       cu_seqlens: Optional[torch.Tensor], init_slot: Optional[torch.Tensor] = None,
                       final_slot: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                       dev_status: Optional[torch.Tensor] = None, stream=None, flags: Optional[int] = None) -> None:
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c() if cache is not None else None
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); pdt, lddt = _mat(dt, "dt")
    pB, ldb = _mat(B, "B"); pC, ldc = _mat(Cm, "C"); po, ldo = _mat(out, "out")
    T = int(x.shape[0])
    n_seq = 1 if cu_seqlens is None else int(cu_seqlens.numel()) - 1
    if cu_seqlens is not None and cu_seqlens.dtype != torch.int32:
        raise TypeError("cu_seqlens must be int32")
    for t, nm in ((init_slot, "init_slot"), (final_slot, "final_slot")):
        if t is not None and (t.dtype != torch.int32 or t.numel() != n_seq):
            raise TypeError(f"{nm} must be int32 with one entry per sequence")
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (C.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size())
    rc = lib.mdraft_ssd_prefill(C.byref(cl), C.byref(cc) if cc is not None else None, int(layer_index),
                                px, ldx, pz, ldz, pdt, lddt, pB, ldb, pC, ldc, po, ldo, T, n_seq,
                                _ptr(cu_seqlens), _ptr(init_slot), _ptr(final_slot), ws_ptr, ws_bytes, _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_ssd_prefill")


def mdraft_ssd_tree_step(layer: SsdLayer, cache: StateCache, layer_index: int, x, z, dt, B, Cm, out,
                         parent_slot: torch.Tensor, node_slot: torch.Tensor, level_offsets: Optional[Sequence[int]] = None,
                         dev_status: Optional[torch.Tensor] = None, stream=None, flags: Optional[int] = None) -> None:
    lib = load_library()
    cl = layer.c(flags)
    cc = cache.c()
    px, ldx = _mat(x, "x"); pz, ldz = _mat(z, "z"); pdt, lddt = _mat(dt, "dt")
    pB, ldb = _mat(B, "B"); pC, ldc = _mat(Cm, "C"); po, ldo = _mat(out, "out")
    M = int(x.shape[0])
    if parent_slot.dtype != torch.int32 or node_slot.dtype != torch.int32:
        raise TypeError("slot index arrays must be int32")
    if parent_slot.numel() != M or node_slot.numel() != M:
        raise ValueError("one parent slot and one node slot per node")
    if level_offsets is None:
        n_levels, lo = 1, None
    else:
        n_levels = len(level_offsets) - 1
        lo = (C.c_int32 * (n_levels + 1))(*[int(v) for v in level_offsets])
    rc = lib.mdraft_ssd_tree_step(C.byref(cl), C.byref(cc), int(layer_index),
                                  px, ldx, pz, ldz, pdt, lddt, pB, ldb, pC, ldc, po, ldo,
                                  M, _ptr(parent_slot), _ptr(node_slot), n_levels, lo, _ptr(dev_status), _stream_ptr(stream))
    if rc != 0:
        raise MdraftError(rc, "mdraft_ssd_tree_step")
