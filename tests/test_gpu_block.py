"""uoe_block_forward (router -> SMHA -> router -> UoME in one call, Section III-C) against the float64 oracle's
smha_forward -> mlp_forward chain, and against the sequence of per-half entry points it replaces.

The second router sees the bfloat16 output of the first half, so the oracle's second half is fed exactly those
bits (u as the GPU stored it) and both halves use the GPU's selection; the selection itself is checked against the
oracle's with the near-tie rule.
"""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import check_routing, problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _weights(w):
    d = {}
    if w.H:
        d["Wr_att"] = gen.make_router(w, "att")
        d["Wq"], d["Wk"], d["Wv"], d["Wo"] = gen.make_attn_weights(w)
    if w.d_ff:
        d["Wr_mlp"] = gen.make_router(w, "mlp")
        d["W1"], d["W2"] = gen.make_mlp_weights(w)
    return d


def _run_block(w, residual=True, boost=1.0):
    import paper_2503_02495_b200 as uoe
    h = _weights(w)
    if boost != 1.0:
        for kname in ("Wr_att", "Wr_mlp"):
            if kname in h:
                h[kname] = gen.store(h[kname].f64 * boost, w.dtype)
    x = gen.make_x(w)
    wd = {k: to_dev(v) for k, v in h.items()}
    pa = problem_of(w, "att", residual=residual) if w.H else None
    pm = problem_of(w, "mlp", residual=residual) if w.d_ff else None
    ra = uoe.alloc_routing(pa) if pa else None
    rm = uoe.alloc_routing(pm) if pm else None
    xd = to_dev(x)
    u = torch.empty_like(xd) if (pa and pm) else None
    y = uoe.uoe_block_forward(pa, pm, xd, wd, r_att=ra, r_mlp=rm, u=u)
    return uoe, h, x, wd, pa, pm, ra, rm, xd, u, y


@pytest.mark.parametrize("name,B", [("cfg2_lm", 16), ("cfg3_long", 4), ("cfg4_vit", 48), ("cfg2_lm", 3)])
def test_block_forward_matches_oracle_chain(name, B):
    w = gen.WORKLOADS[name].replace(B=B)
    uoe, h, x, wd, pa, pm, ra, rm, xd, u, y = _run_block(w)
    # ---- attention half: routing and u ----
    ro = orc.route(x.f64, h["Wr_att"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
    check_routing(ra, ro)
    ro_g = orc.with_selection(x.f64, h["Wr_att"].f64, ra.expert_idx.cpu().numpy(), ra.patch_idx.cpu().numpy(), w.m, w.L_valid)
    assert np.array_equal(ra.expert_offsets.cpu().numpy(), ro_g.offsets)
    u_ref = orc.smha_forward(x.f64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro_g, w.d_h, w.causal)
    assert rel_inf(to_f64(u), u_ref) <= TOL
    # ---- MLP half on the bits of u the GPU produced ----
    u64 = to_f64(u)
    ro2 = orc.route(u64, h["Wr_mlp"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
    check_routing(rm, ro2)
    ro2_g = orc.with_selection(u64, h["Wr_mlp"].f64, rm.expert_idx.cpu().numpy(), rm.patch_idx.cpu().numpy(), w.m, w.L_valid)
    assert np.array_equal(rm.expert_offsets.cpu().numpy(), ro2_g.offsets)
    assert np.abs(rm.p_patch.cpu().numpy() - ro2.p_patch).max() <= 2e-6
    assert np.abs(rm.gate.cpu().numpy() - ro2_g.gate).max() <= 2e-6
    y_ref = orc.mlp_forward(u64, h["W1"].f64, h["W2"].f64, ro2_g, w.act)
    assert rel_inf(to_f64(y), y_ref) <= TOL
    # the expert term of the second half alone (y - u is dominated by neither rounding of u nor of y here)
    z_ref = y_ref - u64
    z_gpu = to_f64(y) - u64
    assert np.abs(z_gpu - z_ref).max() <= TOL * np.abs(z_ref).max() + 2.0 ** -8 * np.abs(y_ref).max()


@pytest.mark.parametrize("name,B", [("cfg2_lm", 5), ("cfg4_vit", 20), ("cfg3_long", 2)])
def test_block_forward_equals_the_separate_calls_bitwise(name, B):
    w = gen.WORKLOADS[name].replace(B=B)
    uoe, h, x, wd, pa, pm, ra, rm, xd, u, y = _run_block(w, boost=10.0)
    r1 = uoe.uoe_route(pa, xd, wd["Wr_att"])
    for f in ("expert_idx", "patch_idx", "expert_offsets", "gate", "p_samp", "p_patch"):
        assert torch.equal(getattr(r1, f), getattr(ra, f)), f
    u1 = uoe.uoe_smha_forward(pa, xd, wd["Wq"], wd["Wk"], wd["Wv"], wd["Wo"], r1)
    assert torch.equal(u1, u)
    r2 = uoe.uoe_route(pm, u1, wd["Wr_mlp"])
    for f in ("expert_idx", "patch_idx", "expert_offsets", "gate", "p_samp", "p_patch"):
        assert torch.equal(getattr(r2, f), getattr(rm, f)), f
    y1 = uoe.uoe_mlp_forward(pm, u1, wd["W1"], wd["W2"], r2)
    assert torch.equal(y1, y)


def test_block_forward_single_halves_and_float32():
    import paper_2503_02495_b200 as uoe
    # MLP half alone in float32 (the small workload): gather kernel + FFMA GEMMs behind the router-written plan
    w = gen.WORKLOADS["cfg1_small_f32"]
    uoe_, h, x, wd, pa, pm, ra, rm, xd, u, y = _run_block(w, residual=False)
    assert pa is None and u is None
    ro_g = orc.with_selection(x.f64, h["Wr_mlp"].f64, rm.expert_idx.cpu().numpy(), rm.patch_idx.cpu().numpy(), w.m, w.L_valid)
    ref = orc.mlp_forward(x.f64, h["W1"].f64, h["W2"].f64, ro_g, w.act, residual=False)
    assert rel_inf(to_f64(y), ref) <= 1e-4
    # attention half alone, routing kept inside the workspace
    w = gen.WORKLOADS["cfg2_lm"].replace(B=2, d_ff=0)
    h = _weights(w)
    x = gen.make_x(w)
    wd = {k: to_dev(v) for k, v in h.items()}
    pa = problem_of(w, "att", residual=False)
    y = uoe.uoe_block_forward(pa, None, to_dev(x), wd)
    r = uoe.uoe_route(pa, to_dev(x), wd["Wr_att"])
    ro_g = orc.with_selection(x.f64, h["Wr_att"].f64, r.expert_idx.cpu().numpy(), r.patch_idx.cpu().numpy(), w.m, w.L_valid)
    ref = orc.smha_forward(x.f64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro_g, w.d_h, w.causal, residual=False)
    assert rel_inf(to_f64(y), ref) <= TOL


def test_block_forward_reuses_one_workspace_across_shapes_and_skewed_loads():
    import paper_2503_02495_b200 as uoe
    big = gen.WORKLOADS["cfg4_vit"].replace(B=40)
    small = gen.WORKLOADS["cfg4_vit"].replace(B=7)
    pa_b, pm_b = problem_of(big, "att"), problem_of(big, "mlp")
    ws = uoe.alloc_block_workspace(pa_b, pm_b)
    for w in (big, small, big):
        h = _weights(w)
        Wr = h["Wr_att"]
        x = gen.make_x(w, skew_beta=4.0, W_r=Wr.f64)           # imbalanced expert loads, some experts empty
        wd = {k: to_dev(v) for k, v in h.items()}
        pa, pm = problem_of(w, "att"), problem_of(w, "mlp")
        xd = to_dev(x)
        u = torch.empty_like(xd)
        ra, rm = uoe.alloc_routing(pa), uoe.alloc_routing(pm)
        y = uoe.uoe_block_forward(pa, pm, xd, wd, r_att=ra, r_mlp=rm, u=u, ws=ws)
        ro_g = orc.with_selection(x.f64, Wr.f64, ra.expert_idx.cpu().numpy(), ra.patch_idx.cpu().numpy(), w.m, w.L_valid)
        u_ref = orc.smha_forward(x.f64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro_g, w.d_h, w.causal)
        assert rel_inf(to_f64(u), u_ref) <= TOL
        u64 = to_f64(u)
        ro2_g = orc.with_selection(u64, h["Wr_mlp"].f64, rm.expert_idx.cpu().numpy(), rm.patch_idx.cpu().numpy(), w.m, w.L_valid)
        y_ref = orc.mlp_forward(u64, h["W1"].f64, h["W2"].f64, ro2_g, w.act)
        assert rel_inf(to_f64(y), y_ref) <= TOL


def test_block_forward_rejects_bad_arguments_before_launching():
    import paper_2503_02495_b200 as uoe
    w = gen.WORKLOADS["cfg2_lm"].replace(B=2)
    pa, pm = problem_of(w, "att"), problem_of(w, "mlp")
    x = torch.zeros(w.B, w.L, w.d, dtype=torch.bfloat16, device="cuda")
    wd = {k: to_dev(v) for k, v in _weights(w).items()}
    ws = uoe.alloc_block_workspace(pa, pm)
    n0 = uoe.uoe_launch_count()
    with pytest.raises(uoe.UoeError) as ei:                   # u aliases x
        uoe.uoe_block_forward(pa, pm, x, wd, u=x, ws=ws)
    assert ei.value.status == 1
    with pytest.raises(uoe.UoeError) as ei:                   # workspace too small
        uoe.uoe_block_forward(pa, pm, x, wd, ws=ws[:4096])
    assert ei.value.status == 3
    bad = dict(wd)
    del bad["W1"]
    with pytest.raises(uoe.UoeError) as ei:                   # a missing weight
        uoe.uoe_block_forward(pa, pm, x, bad, ws=ws)
    assert ei.value.status == 1
    pm2 = problem_of(w.replace(B=3), "mlp")
    assert uoe.uoe_block_workspace_bytes(pa, pm2) > 0
    with pytest.raises(uoe.UoeError):                         # halves disagree on B
        uoe.uoe_block_forward(pa, pm2, x, wd, ws=uoe.alloc_block_workspace(pa, pm2))
    assert uoe.uoe_launch_count() == n0
    assert uoe.uoe_block_workspace_bytes(None, None) == 0


def test_repeated_calls_on_the_same_buffers_encode_no_new_tensor_maps():
    import paper_2503_02495_b200 as uoe
    w = gen.WORKLOADS["cfg2_lm"].replace(B=2)
    pa, pm = problem_of(w, "att"), problem_of(w, "mlp")
    x = to_dev(gen.make_x(w))
    wd = {k: to_dev(v) for k, v in _weights(w).items()}
    ws = uoe.alloc_block_workspace(pa, pm)
    u, y = torch.empty_like(x), torch.empty_like(x)
    uoe.uoe_block_forward(pa, pm, x, wd, u=u, y=y, ws=ws)
    n1 = uoe.uoe_tensor_map_encodings()
    assert n1 > 0
    y1 = y.clone()
    for _ in range(3):
        uoe.uoe_block_forward(pa, pm, x, wd, u=u, y=y, ws=ws)
    assert uoe.uoe_tensor_map_encodings() == n1
    assert torch.equal(y, y1)
