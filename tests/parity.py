"""Helpers for the GPU-vs-oracle parity tests: error metric, oracle runs, GPU runs on the same inputs."""

from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

import gen
import oracle

# Tolerances stated for this path: max relative error 1e-3 with fp32 activations, 2e-2 with bf16 activations
# (fp32 state in both).  "Relative" is taken per tensor with a floor at the tensor's RMS, so that an output
# that happens to be near zero does not turn a rounding error into a large ratio.
TOL = {"f32": 1e-3, "bf16": 2e-2}
TOL_STATE = 1e-3  # SSM state is fp32 in both modes


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if want.size == 0:
        return 0.0
    floor = float(np.sqrt(np.mean(want * want)))
    if floor == 0.0:
        return float(np.max(np.abs(got - want)))
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), floor)))


def assert_close(got, want, tol, what):
    e = rel_err(got, want)
    assert np.all(np.isfinite(np.asarray(got, dtype=np.float64))), f"{what}: non-finite values"
    assert e <= tol, f"{what}: max relative error {e:.3e} > {tol:.1e}"
    return e


def oracle_flags(flags: int) -> int:
    """Library flags -> oracle flags (the A_POWERS hint has no meaning for the oracle)."""
    return flags & 7


@dataclass
class Problem:
    cfg: gen.Config
    params: gen.LayerParams
    x: np.ndarray
    z: np.ndarray
    dt: np.ndarray
    B: np.ndarray
    C: np.ndarray
    cu: np.ndarray


def small_config(d_inner: int, act: str, n_seq: int = 1, cid: int = 90, seed: int = 0) -> gen.Config:
    return gen.Config(cid, "test", 1, d_inner, 16, 4, act, n_seq, (1, 1), "none", 0, seed)


def make_problem(cfg: gen.Config, lens: Sequence[int], layer: int = 0, conv_bias: bool = False, general_A: bool = False) -> Problem:
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    T = int(cu[-1])
    p = gen.layer_params(cfg, layer, conv_bias=conv_bias, general_A=general_A)
    x, z, dt, B, C = gen.prefill_inputs(cfg, layer, T)
    return Problem(cfg, p, x, z, dt, B, C, cu)
