"""Glue for the GPU parity tests: seeded inputs -> torch tensors, workload -> Problem, comparisons."""
from __future__ import annotations

import numpy as np
import torch

import uoe_inputs as gen


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def to_dev(st, device="cuda"):
    from paper_2503_02495_b200.workload import to_dev as f
    return f(st, device)


def problem_of(w, block: str = "mlp", **kw):
    from paper_2503_02495_b200.workload import problem_of as f
    return f(w, block, **kw)


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
