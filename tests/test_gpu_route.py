"""GPU parity: uoe_route against the float64 oracle (Eq. 12-17, 21-23) on the same seeded inputs."""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import check_routing, problem_of, to_dev

pytestmark = pytest.mark.gpu

CASES = {
    "tiny": gen.tiny(),
    "tiny_pad": gen.tiny(L_valid=21, B=5),
    "tiny_k1": gen.tiny(k=1, c=1),
    "tiny_full": gen.tiny(k=4, c=6),
    "tiny_bf16": gen.tiny(dtype="bf16", d=64, B=7),
    "wide_m": gen.tiny(B=3, m=48, c=20, L=96, L_valid=91, d=40, n=5, k=3, d_ff=40),
    # more than a thousand tiny patches: the 64-thread-CTA variant of the router (float32 and bfloat16)
    "many_small_f32": gen.tiny(B=200, L=24, L_valid=22, m=6, c=3, d=48, n=4, k=2, d_ff=48),
    "many_small_bf16": gen.tiny(B=180, L=96, L_valid=96, m=6, c=2, d=128, n=5, k=3, d_ff=40, dtype="bf16"),
    "cfg1": gen.WORKLOADS["cfg1_small_f32"],
    "cfg2": gen.WORKLOADS["cfg2_lm"],
    "cfg3": gen.WORKLOADS["cfg3_long"],
    "cfg4": gen.WORKLOADS["cfg4_vit"],
}


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("use_gate", [True, False])
def test_route_matches_oracle(name, use_gate):
    import paper_2503_02495_b200 as uoe
    w = CASES[name]
    if name.startswith("cfg") and not use_gate:
        pytest.skip("gate-off variant covered by the small cases")
    x, Wr = gen.make_x(w), gen.make_router(w)
    scale = 40.0 if name.startswith("tiny") or name.startswith("many") or name == "wide_m" else 1.0
    Wr = gen.store(Wr.f64 * scale, w.dtype)
    prob = problem_of(w, "mlp", gate=use_gate)
    r = uoe.uoe_route(prob, to_dev(x), to_dev(Wr))
    ro = orc.route(x.f64, Wr.f64, w.k, w.m, w.c, L_valid=w.L_valid, use_gate=use_gate)
    assert np.abs(r.p_samp.cpu().numpy() - ro.p_samp).max() < 2e-6
    assert np.abs(r.p_patch.cpu().numpy() - ro.p_patch).max() < 2e-6
    near_e, near_p = check_routing(r, ro)
    print(f"{name}: near-tie mismatches experts={near_e} patches={near_p}")
    if near_e == 0 and near_p == 0:
        assert np.array_equal(r.expert_offsets.cpu().numpy(), ro.offsets)
        g = r.gate.cpu().numpy()
        assert np.abs(g - ro.gate).max() <= 1e-5 * max(1.0, np.abs(ro.gate).max())
        assert np.all(g[r.patch_idx.cpu().numpy() < 0] == 0)
    # structural invariants hold for any tie-break
    e = r.expert_idx.cpu().numpy()
    p = r.patch_idx.cpu().numpy()
    assert np.all(np.diff(e, axis=1) > 0) and e.min() >= 0 and e.max() < w.n
    n_elig = -(-w.L_valid // w.l_p)
    for b in range(w.B):
        for s in range(w.k):
            sel = p[b, s][p[b, s] >= 0]
            assert len(sel) == min(w.c, n_elig) and np.all(np.diff(sel) > 0) and sel.max() < n_elig
            assert np.all(p[b, s][len(sel):] == -1)
    off = r.expert_offsets.cpu().numpy()
    load = np.bincount(e.ravel(), minlength=w.n)
    exp = np.concatenate([[0], np.cumsum((load * w.l_a + 127) // 128 * 128)])
    assert np.array_equal(off, exp)


def test_route_planted_ties_take_lower_index():
    import paper_2503_02495_b200 as uoe
    # identical patches and a zero router: every probability ties exactly -> lowest indices win
    w = gen.tiny(B=2)
    x = np.tile(gen.normal(3, 0, (1, w.l_p, w.d)), (w.B, w.m, 1))
    prob = problem_of(w, "mlp")
    r = uoe.uoe_route(prob, torch.from_numpy(x.astype(np.float32)).cuda(),
                      torch.zeros(w.d, w.n, device="cuda"))
    assert r.expert_idx.cpu().tolist() == [[0, 1]] * w.B
    assert r.patch_idx.cpu().tolist() == [[[0, 1, 2]] * w.k] * w.B
    assert torch.allclose(r.gate.cpu(), torch.full((w.B, w.k, w.c), 1.0 / (w.n * w.n)))


def test_route_is_deterministic():
    import paper_2503_02495_b200 as uoe
    w = gen.WORKLOADS["cfg2_lm"]
    x, Wr = to_dev(gen.make_x(w)), to_dev(gen.make_router(w))
    prob = problem_of(w, "mlp")
    a = uoe.uoe_route(prob, x, Wr)
    b = uoe.uoe_route(prob, x, Wr)
    for f in ("expert_idx", "patch_idx", "gate", "p_samp", "p_patch", "expert_offsets"):
        assert torch.equal(getattr(a, f), getattr(b, f)), f


# ------------------------------------------------------------------------------------------------
# two-stage dynamic capacity (Eq. 15-16) and the load-balancing loss (Eq. 42-44)
# ------------------------------------------------------------------------------------------------

BAL_CASES = {
    "tiny": (gen.tiny(B=5, n=4, k=2, m=6, c=6), 30.0),
    "tiny_pad": (gen.tiny(B=4, n=5, k=2, m=6, c=4, L_valid=19), 30.0),
    "wide_m": (gen.tiny(B=3, m=48, c=40, L=96, L_valid=91, d=40, n=5, k=3, d_ff=40), 40.0),
    "cfg2": (gen.WORKLOADS["cfg2_lm"], 20.0),
    "cfg4": (gen.WORKLOADS["cfg4_vit"], 20.0),
}


def _patch_counts(w):
    return orc.patch_valid_counts(w.L, w.m, w.L_valid)


@pytest.mark.parametrize("name", list(BAL_CASES))
def test_route_balance_matches_oracle(name):
    """Integers exact, the loss to float32 rounding: the oracle is given the gate values the GPU wrote, so both
    sides rank the same numbers (ties: lower index on both)."""
    import paper_2503_02495_b200 as uoe
    w, scale = BAL_CASES[name]
    x = gen.make_x(w)
    Wr = gen.store(gen.make_router(w).f64 * scale, w.dtype)
    prob = problem_of(w, "mlp")
    r = uoe.uoe_route(prob, to_dev(x), to_dev(Wr))
    lb, cnt, cd = uoe.uoe_route_balance(prob, r.p_patch, alpha=0.01)
    pp = r.p_patch.cpu().numpy().astype(np.float64)
    pc = _patch_counts(w)
    ref_cnt = np.stack([orc.patch_expert_counts(pp[b], pc, w.k) for b in range(w.B)])
    assert np.array_equal(cnt.cpu().numpy(), ref_cnt)
    assert np.array_equal(cd.cpu().numpy(), orc.dynamic_capacity(pp, pc, w.k))
    ref_lb = orc.balance_loss(pp, pc, w.k, alpha=0.01)
    assert np.abs(lb.cpu().numpy() - ref_lb).max() <= 1e-5 * np.abs(ref_lb).max()


@pytest.mark.parametrize("name", list(BAL_CASES))
def test_route_with_dynamic_capacity_matches_oracle(name):
    import paper_2503_02495_b200 as uoe
    w, scale = BAL_CASES[name]
    x = gen.make_x(w)
    Wr = gen.store(gen.make_router(w).f64 * scale, w.dtype)
    prob = problem_of(w, "mlp", dynamic_c=True)
    r = uoe.uoe_route(prob, to_dev(x), to_dev(Wr))
    # selection by the oracle on the probabilities the GPU wrote: every integer decision must agree exactly
    ps = r.p_samp.cpu().numpy().astype(np.float64)
    pp = r.p_patch.cpu().numpy().astype(np.float64)
    pc = _patch_counts(w)
    e_ref, p_ref, _, _ = orc.select(ps, pp, pc, w.k, w.c, dynamic_c=True)
    assert np.array_equal(r.expert_idx.cpu().numpy(), e_ref)
    assert np.array_equal(r.patch_idx.cpu().numpy(), p_ref)
    c_dyn = orc.dynamic_capacity(pp, pc, w.k)
    used = (r.patch_idx.cpu().numpy() >= 0).sum(axis=2)
    n_elig = int((pc > 0).sum())
    assert np.array_equal(used, np.minimum(np.minimum(c_dyn, w.c), n_elig)[:, None].repeat(w.k, 1))
    g = r.gate.cpu().numpy()
    assert np.all(g[r.patch_idx.cpu().numpy() < 0] == 0)
    # and the layer runs on it: unused slots contribute nothing (compare with the oracle on the same routing)
    if w.d_ff and w.dtype == "bf16":
        W1, W2 = gen.make_mlp_weights(w)
        pm = problem_of(w, "mlp", residual=False, dynamic_c=True)
        y = uoe.uoe_mlp_forward(pm, to_dev(x), to_dev(W1), to_dev(W2), r)
        ro = orc.with_selection(x.f64, Wr.f64, e_ref, p_ref, w.m, w.L_valid)
        ref = orc.mlp_forward(x.f64, W1.f64, W2.f64, ro, w.act, residual=False)
        got = y.detach().to(torch.float64).cpu().numpy()
        assert np.abs(got - ref).max() <= 2e-2 * np.abs(ref).max()


@pytest.mark.parametrize("name", ["tiny_pad", "cfg2", "cfg4"])
def test_route_balance_backward_matches_oracle(name):
    """Gradient of sum(dloss * lb_loss) w.r.t. x and W_r: bf16 inputs, fp32 arithmetic; the oracle recomputes the
    gate in float64 from the same stored inputs.  Tolerance 2e-2 * max|ref| as for the other bf16 gradients (dx is
    stored in bf16)."""
    import paper_2503_02495_b200 as uoe
    w, scale = BAL_CASES[name]
    if w.dtype != "bf16":
        w = w.replace(dtype="bf16", d=64)
    x = gen.make_x(w)
    Wr = gen.store(gen.make_router(w).f64 * scale, w.dtype)
    prob = problem_of(w, "mlp")
    xd, Wrd = to_dev(x), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    dloss = gen.normal(77, 0, (w.B,))
    dl = torch.from_numpy(dloss.astype(np.float32)).cuda()
    dx, dWr = uoe.uoe_route_balance_backward(prob, xd, Wrd, r.p_patch, 0.05, dl)
    ref_dx, ref_dWr = orc.balance_loss_backward(x.f64, Wr.f64, w.m, w.L_valid, w.k, 0.05, dloss.astype(np.float32).astype(np.float64))
    got_dx = dx.detach().to(torch.float64).cpu().numpy()
    assert np.abs(got_dx - ref_dx).max() <= 2e-2 * np.abs(ref_dx).max()
    assert np.abs(dWr.cpu().numpy() - ref_dWr).max() <= 2e-2 * np.abs(ref_dWr).max()
    assert np.all(got_dx[:, w.L_valid:] == 0)
