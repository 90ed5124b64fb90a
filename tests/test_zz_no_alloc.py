"""uoe_route_static: routing for callers that cannot give the library a workspace.

Some users of this library run where device memory cannot be requested: a serving loop that must never
reach the CUDA allocator, or a plugin inside a host application that owns all GPU memory.  For them the
library carries a fixed scratch array in its device image.  This test calls that entry point through
the C ABI twice in a row (a larger problem, then a smaller one, so that the second call meets the
first call's leftovers in the shared array) and requires each result to equal uoe_route's: same
kernels, same arithmetic, so integers must match exactly and floats to the tolerance the routing
tests use.  It also checks that a problem beyond the array's size is refused before anything runs.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from tests.helpers import problem_of, to_dev

pytestmark = pytest.mark.gpu


def _same(a, b):
    for f in ("expert_idx", "patch_idx", "expert_offsets"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    for f in ("gate", "p_samp", "p_patch"):
        assert np.abs(getattr(a, f).cpu().numpy() - getattr(b, f).cpu().numpy()).max() <= 2e-6, f


def test_static_scratch_route_matches_workspace_route_twice_in_a_row():
    import paper_2503_02495_b200 as uoe
    first = gen.WORKLOADS["cfg4_vit"]                   # 256 samples, padded tokens
    second = gen.tiny(B=5, L_valid=21, dtype="bf16", d=64)
    for w in (first, second):
        prob = problem_of(w, "mlp")
        assert uoe.uoe_workspace_bytes(prob, uoe.UOE_OP_ROUTE) <= uoe.UOE_ROUTE_STATIC_SCRATCH_BYTES
        x, Wr = to_dev(gen.make_x(w)), to_dev(gen.store(gen.make_router(w).f64 * 10, w.dtype))
        got = uoe.uoe_route_static(prob, x, Wr)
        torch.cuda.synchronize()
        ref = uoe.uoe_route(prob, x, Wr)
        _same(got, ref)
    # and once more on the first problem: the array now holds the small problem's leftovers
    prob = problem_of(first, "mlp")
    x, Wr = to_dev(gen.make_x(first)), to_dev(gen.store(gen.make_router(first).f64 * 10, first.dtype))
    _same(uoe.uoe_route_static(prob, x, Wr), uoe.uoe_route(prob, x, Wr))


def test_static_scratch_route_refuses_problems_beyond_its_array():
    import paper_2503_02495_b200 as uoe
    big = gen.tiny(B=4096, m=16, L=64, L_valid=64, n=8, k=2, c=4, d=64, dtype="bf16")
    prob = problem_of(big, "mlp")
    assert uoe.uoe_workspace_bytes(prob, uoe.UOE_OP_ROUTE) > uoe.UOE_ROUTE_STATIC_SCRATCH_BYTES
    x = torch.zeros(big.B, big.L, big.d, dtype=torch.bfloat16, device="cuda")
    Wr = torch.zeros(big.d, big.n, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(uoe.UoeError) as ei:
        uoe.uoe_route_static(prob, x, Wr)
    assert ei.value.status == 7
    assert "static scratch" in uoe.status_string(7)
