"""Glue for the GPU parity tests: seeded inputs -> torch tensors, workload -> Problem, comparisons."""
from __future__ import annotations

import numpy as np
import torch

import uoe_inputs as gen


def to_dev(st: gen.Stored, device="cuda") -> torch.Tensor:
    if st.dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(st.raw)).to(device)
    return torch.from_numpy(np.ascontiguousarray(st.raw).view(np.int16)).to(device).view(torch.bfloat16)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def problem_of(w: gen.Workload, block: str = "mlp", **kw):
    import paper_2503_02495_b200 as uoe
    base = dict(B=w.B, L=w.L, L_valid=w.L_valid, d=w.d, n=w.n, k=w.k, m=w.m, c=w.c,
                d_e=w.d_e if block == "mlp" else 0, H=w.H if block == "att" else 0,
                d_h=w.d_h if block == "att" else 0, dtype=w.dtype, act=w.act, residual=True, gate=True,
                causal=w.causal if block == "att" else False)
    base.update(kw)
    return uoe.Problem(**base)


def check_routing(r_gpu, r_or, margin_tol=1e-5):
    """Indices must equal the oracle's wherever its selection margin exceeds margin_tol (relative);
    returns (near-tie sample mismatches, near-tie patch-set mismatches)."""
    e_gpu = r_gpu.expert_idx.cpu().numpy()
    p_gpu = r_gpu.patch_idx.cpu().numpy()
    near_e = near_p = 0
    for b in range(e_gpu.shape[0]):
        if not np.array_equal(e_gpu[b], r_or.expert_idx[b]):
            assert r_or.expert_margin[b] <= margin_tol, f"sample {b}: expert set differs at margin {r_or.expert_margin[b]}"
            near_e += 1
            continue
        for s in range(e_gpu.shape[1]):
            if not np.array_equal(p_gpu[b, s], r_or.patch_idx[b, s]):
                assert r_or.patch_margin[b, s] <= margin_tol, \
                    f"sample {b} slot {s}: patch set differs at margin {r_or.patch_margin[b, s]}"
                near_p += 1
    return near_e, near_p


def rel_inf(got: np.ndarray, ref: np.ndarray) -> float:
    den = np.abs(ref).max()
    return float(np.abs(got - ref).max() / den) if den > 0 else float(np.abs(got - ref).max())
