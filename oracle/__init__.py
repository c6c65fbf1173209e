"""fp64 CPU oracle for the conv1d + S6 + gate path (numpy front end).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
it exists so that the tests, the smoke check and the benchmark's CPU-baseline
leg can compare the CUDA library against a slow, sequential statement of the
same computation (see ``mdraft_oracle.c`` for the definition and its pins).

All arrays cross this boundary as float64.  Inputs that the GPU sees in bf16
are rounded by the caller first and then widened exactly.
"""

from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

import numpy as np

from .build import compile_oracle

DT_SOFTPLUS = 1
PRECONV = 2
CONV_ONLY = 4

_c_double_p = C.POINTER(C.c_double)
_c_int32_p = C.POINTER(C.c_int32)


class _Layer(C.Structure):
    _fields_ = [("d_inner", C.c_int32), ("d_state", C.c_int32), ("d_conv", C.c_int32),
                ("flags", C.c_uint32),
                ("A", _c_double_p), ("Dskip", _c_double_p), ("conv_w", _c_double_p),
                ("conv_b", _c_double_p), ("dt_bias", _c_double_p)]


class _SsdLayer(C.Structure):
    _fields_ = [("d_inner", C.c_int32), ("headdim", C.c_int32), ("d_state", C.c_int32), ("d_conv", C.c_int32),
                ("flags", C.c_uint32),
                ("A", _c_double_p), ("Dskip", _c_double_p), ("conv_w", _c_double_p),
                ("conv_b", _c_double_p), ("dt_bias", _c_double_p)]


_lib = None


def lib(path: Optional[str] = None):
    """Load (building if needed) the oracle shared library."""
    global _lib
    if path is not None:
        return _bind(C.CDLL(path))
    if _lib is None:
        _lib = _bind(C.CDLL(compile_oracle()))
    return _lib


def _bind(l):
    l.mdo_silu.restype = C.c_double
    l.mdo_silu.argtypes = [C.c_double]
    l.mdo_softplus.restype = C.c_double
    l.mdo_softplus.argtypes = [C.c_double]
    l.mdo_set_threads.restype = C.c_int
    l.mdo_set_threads.argtypes = [C.c_int]
    l.mdo_prefill.restype = None
    l.mdo_prefill.argtypes = [C.POINTER(_Layer), C.c_int, _c_int32_p] + [_c_double_p] * 10
    l.mdo_tree.restype = C.c_int
    l.mdo_tree.argtypes = [C.POINTER(_Layer), C.c_int, _c_int32_p] + [_c_double_p] * 10
    l.mdo_tree_proj.restype = C.c_int
    l.mdo_tree_proj.argtypes = [C.POINTER(_Layer), C.c_int, _c_double_p, _c_double_p, C.c_int, _c_int32_p] + [_c_double_p] * 10
    l.mdo_ssd_prefill.restype = None
    l.mdo_ssd_prefill.argtypes = [C.POINTER(_SsdLayer), C.c_int, _c_int32_p] + [_c_double_p] * 10
    l.mdo_ssd_tree.restype = C.c_int
    l.mdo_ssd_tree.argtypes = [C.POINTER(_SsdLayer), C.c_int, _c_int32_p] + [_c_double_p] * 10
    return l


def _f64(a, shape=None) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_c_double_p)


@dataclass
class Layer:
    """Per-layer constants in fp64."""
    A: np.ndarray
    D: Optional[np.ndarray]
    conv_w: np.ndarray
    conv_b: Optional[np.ndarray] = None
    dt_bias: Optional[np.ndarray] = None
    flags: int = DT_SOFTPLUS

    def __post_init__(self):
        self.A = _f64(self.A)
        Dn, N = self.A.shape
        self.conv_w = _f64(self.conv_w)
        if self.conv_w.shape[0] != Dn:
            raise ValueError("conv_w must be (D, W)")
        W = self.conv_w.shape[1]
        if not (1 <= W <= 17 and 1 <= N <= 256):
            raise ValueError("oracle limits: d_conv <= 17, d_state <= 256")
        self.D = _f64(self.D, (Dn,))
        self.conv_b = _f64(self.conv_b, (Dn,))
        self.dt_bias = _f64(self.dt_bias, (Dn,))

    @property
    def dims(self) -> Tuple[int, int, int]:
        return self.A.shape[0], self.A.shape[1], self.conv_w.shape[1]

    def _c(self, flags=None) -> _Layer:
        Dn, N, W = self.dims
        return _Layer(Dn, N, W, self.flags if flags is None else flags,
                      _p(self.A), _p(self.D), _p(self.conv_w), _p(self.conv_b), _p(self.dt_bias))


def set_threads(n: int) -> int:
    """Set the OpenMP thread count (channels are split across threads); returns the count in use."""
    return int(lib().mdo_set_threads(int(n)))


def silu(v: float) -> float:
    return float(lib().mdo_silu(float(v)))


def softplus(v: float) -> float:
    return float(lib().mdo_softplus(float(v)))


def prefill(layer: Layer, x, z, dt, B, Cm, cu_seqlens=None, conv_init=None, h_init=None, flags=None, _lib_override=None):
    """Encode packed sequences.  Returns (out (T,D), conv_final (S,W-1,D), h_final (S,D,N))."""
    L = _lib_override or lib()
    Dn, N, W = layer.dims
    x = _f64(x)
    T = x.shape[0]
    x = _f64(x, (T, Dn)); z = _f64(z, (T, Dn)); dt = _f64(dt, (T, Dn))
    B = _f64(B, (T, N)); Cm = _f64(Cm, (T, N))
    if cu_seqlens is None:
        cu_seqlens = [0, T]
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    S = cu.shape[0] - 1
    if cu[0] != 0 or cu[-1] != T or np.any(np.diff(cu) < 0):
        raise ValueError("cu_seqlens must rise from 0 to the token count")
    conv_init = _f64(conv_init, (S, W - 1, Dn))
    h_init = _f64(h_init, (S, Dn, N))
    out = np.empty((T, Dn)); conv_final = np.empty((S, W - 1, Dn)); h_final = np.empty((S, Dn, N))
    cl = layer._c(flags)
    L.mdo_prefill(C.byref(cl), S, cu.ctypes.data_as(_c_int32_p), _p(x), _p(z), _p(dt), _p(B), _p(Cm),
                  _p(conv_init), _p(h_init), _p(out), _p(conv_final), _p(h_final))
    return out, conv_final, h_final


def tree(layer: Layer, parents, x, z, dt, B, Cm, conv0=None, h0=None, flags=None, _lib_override=None):
    """Draft tree of one sequence, every node recomputed along its root-to-node path.
    Returns (out (M,D), conv_nodes (M,W-1,D), h_nodes (M,D,N))."""
    L = _lib_override or lib()
    Dn, N, W = layer.dims
    par = np.ascontiguousarray(parents, dtype=np.int32)
    M = par.shape[0]
    x = _f64(x, (M, Dn)); z = _f64(z, (M, Dn)); dt = _f64(dt, (M, Dn))
    B = _f64(B, (M, N)); Cm = _f64(Cm, (M, N))
    conv0 = _f64(conv0, (W - 1, Dn)); h0 = _f64(h0, (Dn, N))
    out = np.empty((M, Dn)); conv_nodes = np.empty((M, W - 1, Dn)); h_nodes = np.empty((M, Dn, N))
    cl = layer._c(flags)
    rc = L.mdo_tree(C.byref(cl), M, par.ctypes.data_as(_c_int32_p), _p(x), _p(z), _p(dt), _p(B), _p(Cm),
                    _p(conv0), _p(h0), _p(out), _p(conv_nodes), _p(h_nodes))
    if rc != 0:
        raise ValueError("parent indices must point to earlier nodes (or be -1)")
    return out, conv_nodes, h_nodes


def tree_proj(layer: Layer, W_x, W_dt, parents, x, z, conv0=None, h0=None, flags=None, _lib_override=None):
    """Draft tree of one sequence where the step size, B and C of a node are the block's projections of its conv
    output: s = W_x u, dt = W_dt s[:R], B = s[R:R+N], C = s[R+N:].  W_x: (R+2N, D); W_dt: (D, R).
    Returns (out (M,D), conv_nodes (M,W-1,D), h_nodes (M,D,N), dt (M,D), B (M,N), C (M,N))."""
    L = _lib_override or lib()
    Dn, N, W = layer.dims
    W_dt = _f64(W_dt)
    R = W_dt.shape[1]
    W_dt = _f64(W_dt, (Dn, R)); W_x = _f64(W_x, (R + 2 * N, Dn))
    par = np.ascontiguousarray(parents, dtype=np.int32)
    M = par.shape[0]
    x = _f64(x, (M, Dn)); z = _f64(z, (M, Dn))
    conv0 = _f64(conv0, (W - 1, Dn)); h0 = _f64(h0, (Dn, N))
    out = np.empty((M, Dn)); conv_nodes = np.empty((M, W - 1, Dn)); h_nodes = np.empty((M, Dn, N))
    dt = np.empty((M, Dn)); B = np.empty((M, N)); Cm = np.empty((M, N))
    cl = layer._c(flags)
    rc = L.mdo_tree_proj(C.byref(cl), R, _p(W_x), _p(W_dt), M, par.ctypes.data_as(_c_int32_p), _p(x), _p(z), _p(conv0), _p(h0),
                         _p(out), _p(conv_nodes), _p(h_nodes), _p(dt), _p(B), _p(Cm))
    if rc != 0:
        raise ValueError("parent indices must point to earlier nodes (or be -1)")
    return out, conv_nodes, h_nodes, dt, B, Cm


def layer_from_params(p, flags: int = DT_SOFTPLUS) -> Layer:
    """Widen a generator's float32 layer constants to an oracle layer."""
    return Layer(p.A, p.D, p.conv_w, p.conv_b, p.dt_bias, flags)


# ---------------------------------------------------------------- Mamba-2 (SSD): one scalar A per head
@dataclass
class SsdLayer:
    """Constants of an SSD layer in fp64: A (H,) one scalar per head, dt_bias (H,), D (D,), conv taps (D, W)."""
    A: np.ndarray
    D: Optional[np.ndarray]
    conv_w: np.ndarray
    conv_b: Optional[np.ndarray]
    dt_bias: Optional[np.ndarray]
    headdim: int
    d_state: int
    flags: int = DT_SOFTPLUS

    def __post_init__(self):
        self.A = _f64(self.A)
        H = self.A.shape[0]
        self.conv_w = _f64(self.conv_w)
        Dn, W = self.conv_w.shape
        if self.A.ndim != 1 or H * self.headdim != Dn:
            raise ValueError("A must be (H,) with H * headdim == D")
        if not (1 <= W <= 17 and 1 <= self.d_state <= 256):
            raise ValueError("oracle limits: d_conv <= 17, d_state <= 256")
        self.D = _f64(self.D, (Dn,))
        self.conv_b = _f64(self.conv_b, (Dn,))
        self.dt_bias = _f64(self.dt_bias, (H,))

    @property
    def dims(self):
        return self.conv_w.shape[0], self.A.shape[0], self.d_state, self.conv_w.shape[1]   # D, H, N, W

    def _c(self, flags=None) -> _SsdLayer:
        Dn, H, N, W = self.dims
        return _SsdLayer(Dn, self.headdim, N, W, self.flags if flags is None else flags,
                         _p(self.A), _p(self.D), _p(self.conv_w), _p(self.conv_b), _p(self.dt_bias))


def ssd_layer_from_params(p, flags: int = DT_SOFTPLUS) -> SsdLayer:
    return SsdLayer(p.A, p.D, p.conv_w, p.conv_b, p.dt_bias, p.headdim, p.d_state, flags)


def ssd_prefill(layer: SsdLayer, x, z, dt, B, Cm, cu_seqlens=None, conv_init=None, h_init=None, flags=None, _lib_override=None):
    """Encode packed sequences with the SSD recurrence.  x, z: (T, D); dt: (T, H); B, C: (T, N).
    Returns (out (T,D), conv_final (S,W-1,D), h_final (S,D,N))."""
    L = _lib_override or lib()
    Dn, H, N, W = layer.dims
    x = _f64(x)
    T = x.shape[0]
    x = _f64(x, (T, Dn)); z = _f64(z, (T, Dn)); dt = _f64(dt, (T, H))
    B = _f64(B, (T, N)); Cm = _f64(Cm, (T, N))
    if cu_seqlens is None:
        cu_seqlens = [0, T]
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    S = cu.shape[0] - 1
    if cu[0] != 0 or cu[-1] != T or np.any(np.diff(cu) < 0):
        raise ValueError("cu_seqlens must rise from 0 to the token count")
    conv_init = _f64(conv_init, (S, W - 1, Dn))
    h_init = _f64(h_init, (S, Dn, N))
    out = np.empty((T, Dn)); conv_final = np.empty((S, W - 1, Dn)); h_final = np.empty((S, Dn, N))
    cl = layer._c(flags)
    L.mdo_ssd_prefill(C.byref(cl), S, cu.ctypes.data_as(_c_int32_p), _p(x), _p(z), _p(dt), _p(B), _p(Cm),
                      _p(conv_init), _p(h_init), _p(out), _p(conv_final), _p(h_final))
    return out, conv_final, h_final


def ssd_tree(layer: SsdLayer, parents, x, z, dt, B, Cm, conv0=None, h0=None, flags=None, _lib_override=None):
    """Draft tree of one sequence under the SSD recurrence, every node recomputed along its root-to-node path.
    Returns (out (M,D), conv_nodes (M,W-1,D), h_nodes (M,D,N))."""
    L = _lib_override or lib()
    Dn, H, N, W = layer.dims
    par = np.ascontiguousarray(parents, dtype=np.int32)
    M = par.shape[0]
    x = _f64(x, (M, Dn)); z = _f64(z, (M, Dn)); dt = _f64(dt, (M, H))
    B = _f64(B, (M, N)); Cm = _f64(Cm, (M, N))
    conv0 = _f64(conv0, (W - 1, Dn)); h0 = _f64(h0, (Dn, N))
    out = np.empty((M, Dn)); conv_nodes = np.empty((M, W - 1, Dn)); h_nodes = np.empty((M, Dn, N))
    cl = layer._c(flags)
    rc = L.mdo_ssd_tree(C.byref(cl), M, par.ctypes.data_as(_c_int32_p), _p(x), _p(z), _p(dt), _p(B), _p(Cm),
                        _p(conv0), _p(h0), _p(out), _p(conv_nodes), _p(h_nodes))
    if rc != 0:
        raise ValueError("parent indices must point to earlier nodes (or be -1)")
    return out, conv_nodes, h_nodes
