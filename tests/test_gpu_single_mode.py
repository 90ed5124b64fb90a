"""The two selection modes the paper uses on their own (end of Section III-B) through their shorter paths:
pure data selection (k = n, Eq. 12-20: every sample uses all experts, each expert picks its c patches) and pure
expert selection (c = m, Eq. 21-26: a chosen expert takes the whole sample).

Each case is checked three ways: the routing against the oracle's (near-tie rule), the block's outputs against the
float64 oracle chain smha_forward -> mlp_forward, and the shortcut against the general routed path
(UOE_FLAG_GENERAL_PATH) bit for bit -- the shortcuts skip bookkeeping, never arithmetic.
"""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import check_routing, problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2
ROUTING_FIELDS = ("expert_idx", "patch_idx", "expert_offsets", "gate", "p_samp", "p_patch")


def _weights(w):
    d = {}
    if w.H:
        d["Wr_att"] = gen.make_router(w, "att")
        d["Wq"], d["Wk"], d["Wv"], d["Wo"] = gen.make_attn_weights(w)
    if w.d_ff:
        d["Wr_mlp"] = gen.make_router(w, "mlp")
        d["W1"], d["W2"] = gen.make_mlp_weights(w)
    return d


def _block(uoe, w, wd, xd, general):
    pa = problem_of(w, "att", general_path=general)
    pm = problem_of(w, "mlp", general_path=general)
    ra, rm = uoe.alloc_routing(pa), uoe.alloc_routing(pm)
    u = torch.empty_like(xd)
    y = uoe.uoe_block_forward(pa, pm, xd, wd, r_att=ra, r_mlp=rm, u=u)
    return ra, rm, u, y


CASES = [
    # name, B, overrides: data selection keeps the workload's c < m and takes k = n; expert selection keeps k < n, c = m
    ("cfg2_lm", 6, "data"), ("cfg2_lm", 6, "expert"), ("cfg4_vit", 24, "data"), ("cfg4_vit", 24, "expert"),
    ("cfg2_lm", 3, "both"),
]


@pytest.mark.parametrize("name,B,mode", CASES)
def test_single_mode_block_matches_oracle_and_general_path(name, B, mode):
    import paper_2503_02495_b200 as uoe
    w0 = gen.WORKLOADS[name]
    kw = dict(B=B)
    if mode in ("data", "both"):
        kw["k"] = w0.n
    if mode in ("expert", "both"):
        kw["c"] = w0.m
    w = w0.replace(**kw)
    h = _weights(w)
    for kname in ("Wr_att", "Wr_mlp"):            # sharper gates: selections with clear margins
        h[kname] = gen.store(h[kname].f64 * 10, w.dtype)
    x = gen.make_x(w)
    wd = {k: to_dev(v) for k, v in h.items()}
    xd = to_dev(x)
    ra, rm, u, y = _block(uoe, w, wd, xd, general=False)

    # ---- routing of the attention half against the oracle ----
    ro = orc.route(x.f64, h["Wr_att"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
    check_routing(ra, ro)
    n_elig = -(-w.L_valid // (w.L // w.m))
    e = ra.expert_idx.cpu().numpy()
    pidx = ra.patch_idx.cpu().numpy()
    if mode in ("data", "both"):                  # Eq. 12-20: all experts, regions of exactly B pairs
        assert np.array_equal(e, np.tile(np.arange(w.n), (w.B, 1)))
        region = -(-(w.B * w.c * (w.L // w.m)) // 128) * 128
        assert np.array_equal(ra.expert_offsets.cpu().numpy(), np.arange(w.n + 1) * region)
    if mode in ("expert", "both"):                # Eq. 21-26: whole samples
        want = np.where(np.arange(w.c) < n_elig, np.arange(w.c), -1)
        assert np.array_equal(pidx, np.broadcast_to(want, pidx.shape))
    ro_g = orc.with_selection(x.f64, h["Wr_att"].f64, e, pidx, w.m, w.L_valid)
    assert np.array_equal(ra.expert_offsets.cpu().numpy(), ro_g.offsets)
    assert np.abs(ra.gate.cpu().numpy() - ro_g.gate).max() <= 2e-6

    # ---- outputs against the oracle chain ----
    u_ref = orc.smha_forward(x.f64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro_g, w.d_h, w.causal)
    assert rel_inf(to_f64(u), u_ref) <= TOL
    u64 = to_f64(u)
    ro2 = orc.route(u64, h["Wr_mlp"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
    check_routing(rm, ro2)
    ro2_g = orc.with_selection(u64, h["Wr_mlp"].f64, rm.expert_idx.cpu().numpy(), rm.patch_idx.cpu().numpy(), w.m, w.L_valid)
    y_ref = orc.mlp_forward(u64, h["W1"].f64, h["W2"].f64, ro2_g, w.act)
    assert rel_inf(to_f64(y), y_ref) <= TOL
    z_ref, z_gpu = y_ref - u64, to_f64(y) - u64      # the expert term of the second half alone
    assert np.abs(z_gpu - z_ref).max() <= TOL * np.abs(z_ref).max() + 2.0 ** -8 * np.abs(y_ref).max()

    # ---- the shortcut against the general path: same bits ----
    ra2, rm2, u2, y2 = _block(uoe, w, wd, xd, general=True)
    for f in ROUTING_FIELDS:
        assert torch.equal(getattr(ra, f), getattr(ra2, f)), ("att", f)
        assert torch.equal(getattr(rm, f), getattr(rm2, f)), ("mlp", f)
    assert torch.equal(u, u2)
    assert torch.equal(y, y2)


@pytest.mark.parametrize("mode", ["data", "expert"])
def test_single_mode_route_alone_and_per_half_calls(mode):
    """uoe_route takes the same shortcuts; its arrays feed the per-half entry points (general plan kernel) and the
    result equals the block entry's."""
    import paper_2503_02495_b200 as uoe
    w0 = gen.WORKLOADS["cfg4_vit"]
    w = w0.replace(B=9, k=w0.n) if mode == "data" else w0.replace(B=9, c=w0.m)
    h = _weights(w)
    x = gen.make_x(w)
    wd = {k: to_dev(v) for k, v in h.items()}
    xd = to_dev(x)
    ra, rm, u, y = _block(uoe, w, wd, xd, general=False)
    pa, pm = problem_of(w, "att"), problem_of(w, "mlp")
    r1 = uoe.uoe_route(pa, xd, wd["Wr_att"])
    for f in ROUTING_FIELDS:
        assert torch.equal(getattr(r1, f), getattr(ra, f)), f
    u1 = uoe.uoe_smha_forward(pa, xd, wd["Wq"], wd["Wk"], wd["Wv"], wd["Wo"], r1)
    assert torch.equal(u1, u)
    r2 = uoe.uoe_route(pm, u1, wd["Wr_mlp"])
    y1 = uoe.uoe_mlp_forward(pm, u1, wd["W1"], wd["W2"], r2)
    assert torch.equal(y1, y)


def test_dynamic_capacity_keeps_the_general_path_at_c_equal_m():
    """With Eq. 15-16 a chosen expert may take fewer than all patches even when c = m: no whole-sample shortcut."""
    import paper_2503_02495_b200 as uoe
    w0 = gen.WORKLOADS["cfg2_lm"]
    w = w0.replace(B=4, c=w0.m)
    h = _weights(w)
    x = gen.make_x(w)
    wd = {k: to_dev(v) for k, v in h.items()}
    xd = to_dev(x)
    pa = problem_of(w, "att", dynamic_c=True)
    pm = problem_of(w, "mlp", dynamic_c=True)
    ra, rm = uoe.alloc_routing(pa), uoe.alloc_routing(pm)
    u = torch.empty_like(xd)
    y = uoe.uoe_block_forward(pa, pm, xd, wd, r_att=ra, r_mlp=rm, u=u)
    pidx = ra.patch_idx.cpu().numpy()
    assert (pidx == -1).any()                      # the dynamic capacity is below m on this input
    ro_g = orc.with_selection(x.f64, h["Wr_att"].f64, ra.expert_idx.cpu().numpy(), pidx, w.m, w.L_valid)
    u_ref = orc.smha_forward(x.f64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro_g, w.d_h, w.causal)
    assert rel_inf(to_f64(u), u_ref) <= TOL
    u64 = to_f64(u)
    ro2_g = orc.with_selection(u64, h["Wr_mlp"].f64, rm.expert_idx.cpu().numpy(), rm.patch_idx.cpu().numpy(), w.m, w.L_valid)
    y_ref = orc.mlp_forward(u64, h["W1"].f64, h["W2"].f64, ro2_g, w.act)
    assert rel_inf(to_f64(y), y_ref) <= TOL
