"""Move generated inputs (numpy, see the ``gen`` package) into device tensors.

Plumbing shared by the tests, the smoke check and the benchmark: dtype
conversion and uploads only.
"""

from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as mb


def torch_act(act: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[act]


def to_device(a: Optional[np.ndarray], dtype: torch.dtype, device="cuda", pinned: bool = False):
    """float32 numpy array (values already representable in ``dtype``) -> device tensor."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype != t.dtype:
        t = t.to(dtype)
    if pinned:
        return t.pin_memory()
    return t.to(device)


def upload_layer(p, act: str, flags: int = mb.MDRAFT_DT_SOFTPLUS, device="cuda") -> mb.Layer:
    f = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return mb.Layer(f(p.A), f(p.D), f(p.conv_w), f(p.conv_b), f(p.dt_bias), torch_act(act), flags)


def i32(values, device="cuda") -> torch.Tensor:
    return torch.tensor(np.asarray(values, dtype=np.int32), dtype=torch.int32, device=device)


def upload_ssd_layer(p, flags: int = mb.MDRAFT_DT_SOFTPLUS, device="cuda") -> mb.SsdLayer:
    f = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return mb.SsdLayer(f(p.A), f(p.D), f(p.conv_w), f(p.conv_b), f(p.dt_bias), p.headdim, p.d_state, flags)
