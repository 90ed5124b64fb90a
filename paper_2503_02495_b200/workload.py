"""Glue between a workload description and the binding: workload -> Problem, stored host array -> device tensor.

A workload is any object with the fields B, L, L_valid, d, n, k, m, c, d_e, H, d_h, dtype, act, causal (the
seeded generator's Workload has them); a stored array is any object with `raw` (float32 values, or uint16
bfloat16 bit patterns) and `dtype` ("f32" | "bf16").  Nothing of the method is computed here.
"""
from __future__ import annotations

import numpy as np
import torch

from .binding import Problem


def to_dev(st, device="cuda") -> torch.Tensor:
    """Device tensor holding exactly the stored bits (float32, or bfloat16 from its bit patterns)."""
    if st.dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(st.raw)).to(device)
    return torch.from_numpy(np.ascontiguousarray(st.raw).view(np.int16)).to(device).view(torch.bfloat16)


def problem_of(w, block: str = "mlp", **kw) -> Problem:
    """The uoe_problem of one half of a block: block = "mlp" (UoME, Eq. 37-40) or "att" (SMHA, Eq. 27-36)."""
    base = dict(B=w.B, L=w.L, L_valid=w.L_valid, d=w.d, n=w.n, k=w.k, m=w.m, c=w.c,
                d_e=w.d_e if block == "mlp" else 0, H=w.H if block == "att" else 0,
                d_h=w.d_h if block == "att" else 0, dtype=w.dtype, act=w.act, residual=True, gate=True,
                causal=w.causal if block == "att" else False)
    base.update(kw)
    return Problem(**base)
