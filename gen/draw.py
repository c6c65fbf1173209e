"""Counter-based draws of layer constants and activations.

Recipe (the benchmark's tiny fp32 configuration states it; every other
configuration reuses it):  x, z, B, C ~ N(0,1);  the step-size pre-activation
is 0.5*N(0,1), to which the layer adds a per-channel bias chosen so that the
activated step size stays inside [1e-3, 1e-1];  A[d][n] = -(n+1) for every
channel (S4D-real);  D = 1;  conv taps ~ N(0, 0.5^2);  no conv bias unless asked.

Arrays come back as float32 whose values are exactly representable in the
activation dtype ("f32" or "bf16"), so a conversion to bf16 bits on one side
and to float64 on the other loses nothing.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np

from .configs import Config

# Bias b with  log(1+exp(v+b)) in [1e-3, 1e-1]  for |v| <= DT_PRE_HI:
# the interval ends are log(expm1(1e-3)) = -6.90725524 and log(expm1(1e-1)) =
# -2.25216846; b is their midpoint; the half-width 2.3275 is rounded inward to
# a value bf16 can hold, so the clip commutes with the rounding.
DT_BIAS = np.float32(-4.579712)
DT_PRE_LO = np.float32(-2.3125)
DT_PRE_HI = np.float32(2.3125)

_TENSOR_ID = {"x": 0, "z": 1, "dt": 2, "B": 3, "C": 4, "conv_w": 5, "conv_b": 6,
              "lens": 7, "tree": 8, "accept": 9, "h0": 10, "conv0": 11, "W_x": 12, "W_dt": 13}


def rng_for(seed: int, cid: int, layer: int, rnd: int, tensor: str, phase: int = 0) -> np.random.Generator:
    """Generator keyed by (seed, config, layer, round, tensor, phase)."""
    k0 = (int(seed) & 0xFFFFFFFF) << 32 | (int(cid) & 0xFFFF) << 16 | (int(phase) & 0xFFFF)
    k1 = (int(layer) & 0xFFFF) << 40 | (int(rnd) & 0xFFFFF) << 20 | _TENSOR_ID[tensor]
    return np.random.Generator(np.random.Philox(key=np.array([k0, k1], dtype=np.uint64)))


# ---------------------------------------------------------------- dtype helpers
def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32, exact."""
    return (b.astype(np.uint32) << 16).view(np.float32)


def round_to_act(a: np.ndarray, act: str) -> np.ndarray:
    """Round float32 values to the activation dtype; result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if act == "f32":
        return a
    if act == "bf16":
        return from_bf16_bits(bf16_bits(a))
    raise ValueError(f"unknown activation dtype {act!r}")


# ---------------------------------------------------------------- layer constants
@dataclass
class LayerParams:
    A: np.ndarray                 # (D, N) float32, <= 0
    D: np.ndarray                 # (D,)   float32 skip weight
    conv_w: np.ndarray            # (D, W) float32, tap W-1 multiplies the current token
    conv_b: Optional[np.ndarray]  # (D,)   float32 or None
    dt_bias: np.ndarray           # (D,)   float32


def layer_params(cfg: Config, layer: int, seed: Optional[int] = None, *,
                 conv_bias: bool = False, general_A: bool = False) -> LayerParams:
    """Per-layer constants.  ``general_A`` perturbs A away from the S4D-real
    pattern (as training would), keeping it strictly negative."""
    seed = cfg.seed if seed is None else seed
    Dn, N, W = cfg.d_inner, cfg.d_state, cfg.d_conv
    A = -np.tile(np.arange(1, N + 1, dtype=np.float32), (Dn, 1))
    if general_A:
        g = rng_for(seed, cfg.cid, layer, 0, "h0", phase=7)
        A = (A * np.exp(0.25 * g.standard_normal((Dn, N), dtype=np.float32))).astype(np.float32)
    Dskip = np.ones(Dn, dtype=np.float32)
    conv_w = (0.5 * rng_for(seed, cfg.cid, layer, 0, "conv_w").standard_normal((Dn, W), dtype=np.float32)).astype(np.float32)
    conv_b = None
    if conv_bias:
        conv_b = (0.25 * rng_for(seed, cfg.cid, layer, 0, "conv_b").standard_normal(Dn, dtype=np.float32)).astype(np.float32)
    dt_bias = np.full(Dn, DT_BIAS, dtype=np.float32)
    return LayerParams(np.ascontiguousarray(A), Dskip, np.ascontiguousarray(conv_w), conv_b, dt_bias)


def select_proj(cfg: Config, layer: int, dt_rank: int, seed: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Random weights of a block's two selection projections, in the activation dtype's values:
    W_x (dt_rank + 2 N, D) ~ N(0, 1.6^2 / D) and W_dt (D, dt_rank) ~ N(0, 0.5^2 / dt_rank), scaled so that the
    projected B, C and step-size pre-activation land near the spreads the direct recipe draws (1, 1 and 0.5)."""
    seed = cfg.seed if seed is None else seed
    Dn, N = cfg.d_inner, cfg.d_state
    W_x = rng_for(seed, cfg.cid, layer, 0, "W_x").standard_normal((dt_rank + 2 * N, Dn), dtype=np.float32) * np.float32(1.6 / np.sqrt(Dn))
    W_dt = rng_for(seed, cfg.cid, layer, 0, "W_dt").standard_normal((Dn, dt_rank), dtype=np.float32) * np.float32(0.5 / np.sqrt(dt_rank))
    return round_to_act(W_x, cfg.act), round_to_act(W_dt, cfg.act)


# ---------------------------------------------------------------- activations
def _activations(cfg: Config, layer: int, rnd: int, phase: int, rows: int, seed: int):
    Dn, N = cfg.d_inner, cfg.d_state

    def normal(name, shape):
        return rng_for(seed, cfg.cid, layer, rnd, name, phase).standard_normal(shape, dtype=np.float32)

    x = round_to_act(normal("x", (rows, Dn)), cfg.act)
    z = round_to_act(normal("z", (rows, Dn)), cfg.act)
    dt = round_to_act(0.5 * normal("dt", (rows, Dn)), cfg.act)
    np.clip(dt, DT_PRE_LO, DT_PRE_HI, out=dt)
    B = round_to_act(normal("B", (rows, N)), cfg.act)
    C = round_to_act(normal("C", (rows, N)), cfg.act)
    return x, z, dt, B, C


def prefill_inputs(cfg: Config, layer: int, total_tokens: int, seed: Optional[int] = None):
    """(x, z, dt, B, C) for a packed context of ``total_tokens`` rows."""
    seed = cfg.seed if seed is None else seed
    return _activations(cfg, layer, 0, 0, int(total_tokens), seed)


def node_inputs(cfg: Config, layer: int, rnd: int, n_nodes: int, seed: Optional[int] = None):
    """(x, z, dt, B, C) for ``n_nodes`` tree nodes of draft round ``rnd``."""
    seed = cfg.seed if seed is None else seed
    return _activations(cfg, layer, rnd, 1, int(n_nodes), seed)


def seq_lengths(cfg: Config, seed: Optional[int] = None) -> np.ndarray:
    """cu_seqlens (int32, n_seq+1) for the configuration's context mix."""
    seed = cfg.seed if seed is None else seed
    lo, hi = cfg.context
    if lo == hi:
        lens = np.full(cfg.n_seq, lo, dtype=np.int64)
    else:
        lens = rng_for(seed, cfg.cid, 0, 0, "lens").integers(lo, hi + 1, size=cfg.n_seq)
    cu = np.zeros(cfg.n_seq + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return cu


# ---------------------------------------------------------------- Mamba-2 (SSD) shapes
@dataclass
class SsdParams:
    A: np.ndarray                 # (H,)   float32, <= 0: one scalar per head
    D: np.ndarray                 # (D,)   float32 skip weight
    conv_w: np.ndarray            # (D, W) float32
    conv_b: Optional[np.ndarray]  # (D,)   float32 or None
    dt_bias: np.ndarray           # (H,)   float32
    headdim: int
    d_state: int


def ssd_params(cfg: Config, layer: int, headdim: int, d_state: int, seed: Optional[int] = None, *, conv_bias: bool = False) -> SsdParams:
    """Constants of one SSD layer: A[j] = -(1 + 15 j / (H - 1)) spreads the heads over the same range -(1..16) as the
    S4D-real rows of the S6 recipe; D = 1; conv taps ~ N(0, 0.5^2); the recipe's step-size bias."""
    seed = cfg.seed if seed is None else seed
    Dn, W = cfg.d_inner, cfg.d_conv
    H = Dn // headdim
    A = -(1.0 + 15.0 * np.arange(H, dtype=np.float32) / np.float32(max(H - 1, 1))).astype(np.float32)
    conv_w = (0.5 * rng_for(seed, cfg.cid, layer, 0, "conv_w").standard_normal((Dn, W), dtype=np.float32)).astype(np.float32)
    conv_b = None
    if conv_bias:
        conv_b = (0.25 * rng_for(seed, cfg.cid, layer, 0, "conv_b").standard_normal(Dn, dtype=np.float32)).astype(np.float32)
    return SsdParams(A, np.ones(Dn, dtype=np.float32), np.ascontiguousarray(conv_w), conv_b, np.full(H, DT_BIAS, dtype=np.float32), headdim, d_state)


def ssd_inputs(cfg: Config, layer: int, rnd: int, phase: int, rows: int, headdim: int, d_state: int, seed: Optional[int] = None):
    """(x, z, dt, B, C) for ``rows`` tokens or nodes of an SSD layer: x, z (rows, D); dt (rows, H); B, C (rows, N), drawn
    as in the S6 recipe, with B and C scaled by 1 / sqrt(N / 16) so that C.h keeps the recipe's spread at N = 128."""
    seed = cfg.seed if seed is None else seed
    Dn = cfg.d_inner
    H = Dn // headdim

    def normal(name, shape):
        return rng_for(seed, cfg.cid, layer, rnd, name, phase).standard_normal(shape, dtype=np.float32)

    x = round_to_act(normal("x", (rows, Dn)), cfg.act)
    z = round_to_act(normal("z", (rows, Dn)), cfg.act)
    dt = round_to_act(0.5 * normal("dt", (rows, H)), cfg.act)
    np.clip(dt, DT_PRE_LO, DT_PRE_HI, out=dt)
    sc = np.float32(1.0 / np.sqrt(d_state / 16.0))
    B = round_to_act(sc * normal("B", (rows, d_state)), cfg.act)
    C = round_to_act(sc * normal("C", (rows, d_state)), cfg.act)
    return x, z, dt, B, C
