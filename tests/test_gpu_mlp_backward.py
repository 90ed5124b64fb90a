"""GPU parity: uoe_mlp_backward against the float64 oracle (derivative of Eq. 38-40 and of the gates,
Eq. 14 / 21, with the selection held constant; the oracle's backward is itself pinned by finite
differences).  bfloat16 tolerance: max|err| <= 2e-2 * max|ref| for each of dx, dW1, dW2, dW_r
(dx also with the residual off, where dy does not dominate it)."""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _w(**kw):
    base = dict(B=4, L=96, L_valid=96, m=6, c=3, d=128, n=4, k=2, d_ff=512, H=0, d_h=0, dtype="bf16", w_std=0.05,
                act="silu")
    base.update(kw)
    return gen.tiny(**base)


CASES = {
    "base": _w(),
    "pad_gelu": _w(L_valid=83, act="gelu_erf", B=5),
    "k1_tanh": _w(k=1, c=2, act="gelu_tanh"),
    "full": _w(k=4, c=6),
    "wide": _w(B=3, d=256, d_ff=1024, n=4, k=3, L=256, L_valid=250, m=8, c=5),
    "skewed": _w(B=9, n=5, k=2, d_ff=640),
    # narrow experts (d_e = 256): the forward is the one-kernel MLP, which also writes the saved pre-activation;
    # 384 and 512 output columns take two output halves, with pad tokens and a ragged second half
    "fused_fwd_d384_pad": _w(B=6, L=224, L_valid=197, m=14, c=7, d=384, n=3, k=2, d_ff=768),
    "fused_fwd_d512": _w(B=4, L=256, L_valid=256, m=8, c=4, d=512, n=4, k=2, d_ff=1024, act="gelu_tanh"),
    # long K and many row tiles: 256-row GEMM tiles with half tiles at the region ends
    "tall_tiles": _w(B=40, L=1152, L_valid=1152, m=9, c=3, d=1024, n=4, k=2, d_ff=4096, w_std=0.02),
    # imbalanced loads on shapes large enough for the 256-row GEMM tiles and for the weight-gradient kernel's
    # 256 x 256 tiles handed out longest-first (320 of them, the experts' row counts far apart)
    "tall_tiles_skewed": _w(B=40, L=1152, L_valid=1152, m=9, c=3, d=1024, n=4, k=2, d_ff=4096, w_std=0.02),
    "wgrad_256_skewed": _w(B=12, L=1152, L_valid=1152, m=9, c=3, d=1024, n=5, k=2, d_ff=5 * 4096, w_std=0.02),
    # the same tiles with patches shorter than a 64-row contraction block (two gathered boxes per block), pad tokens,
    # and an expert that may get no rows at all
    # CTA-pair GEMMs with 16-token patches: dy gathered in eight boxes per block in the dA/dh step, x in GEMM1
    "pair_tiles_short_patches": _w(B=80, L=256, L_valid=250, m=16, c=8, d=512, n=4, k=2, d_ff=4096, w_std=0.03),
    "wgrad_256_short_patches_skewed": _w(B=10, L=288, L_valid=270, m=9, c=4, d=1024, n=5, k=2, d_ff=5 * 4096, w_std=0.02),
}


def _run(w, residual, use_gate, skew=0.0):
    import paper_2503_02495_b200 as uoe
    Wr = gen.store(gen.make_router(w).f64 * 10, w.dtype)
    x = gen.make_x(w, skew_beta=skew, W_r=Wr.f64)
    W1, W2 = gen.make_mlp_weights(w)
    dy = gen.make_dy(w)
    prob = problem_of(w, "mlp", residual=residual, gate=use_gate)
    xd, W1d, W2d, Wrd = to_dev(x), to_dev(W1), to_dev(W2), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    saved_h = uoe.alloc_saved_h(prob)
    uoe.uoe_mlp_forward(prob, xd, W1d, W2d, r, saved_h=saved_h)
    got = uoe.uoe_mlp_backward(prob, xd, W1d, W2d, Wrd, r, saved_h, to_dev(dy))
    ro = orc.with_selection(x.f64, Wr.f64, r.expert_idx.cpu().numpy(), r.patch_idx.cpu().numpy(), w.m, w.L_valid,
                            use_gate)
    ref = orc.mlp_backward(x.f64, W1.f64, W2.f64, Wr.f64, ro, dy.f64, w.act, residual, use_gate)
    return [to_f64(t) for t in got], ref, ro


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("residual", [False, True])
def test_backward_matches_oracle(name, residual):
    w = CASES[name]
    if w.B * w.L > 10000 and residual:
        pytest.skip("large case: run once")
    got, ref, ro = _run(w, residual, True, skew=(3.0 if name == "skewed" else 12.0) if "skewed" in name else 0.0)
    for nm, g, r in zip(("dx", "dW1", "dW2", "dW_r"), got, ref[:4]):
        err = rel_inf(g, r)
        print(f"{name} residual={residual} {nm}: {err:.3e}  (|ref|max {np.abs(r).max():.3e})")
        assert err <= TOL, nm
    if "skewed" in name:
        assert ro.load.min() == 0 or ro.load.max() >= 1.5 * ro.load.mean()      # the load really is uneven


def test_backward_without_gates_has_zero_router_gradient():
    got, ref, _ = _run(CASES["base"], False, False)
    for g, r in zip(got[:3], ref[:3]):
        assert rel_inf(g, r) <= TOL
    assert np.all(got[3] == 0)


def test_backward_is_deterministic():
    a, _, _ = _run(CASES["wide"], True, True)
    b, _, _ = _run(CASES["wide"], True, True)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


def test_backward_unsupported_shapes():
    import paper_2503_02495_b200 as uoe
    w = gen.tiny(dtype="bf16", d=64, d_ff=256)
    prob = problem_of(w, "mlp")
    assert uoe.uoe_workspace_bytes(prob, uoe.UOE_OP_MLP_BWD) > 0
    x, Wr = to_dev(gen.make_x(w)), to_dev(gen.make_router(w))
    W1, W2 = (to_dev(t) for t in gen.make_mlp_weights(w))
    r = uoe.uoe_route(prob, x, Wr)
    sh = uoe.alloc_saved_h(prob)
    with pytest.raises(uoe.UoeError) as ei:
        uoe.uoe_mlp_backward(prob, x, W1, W2, Wr, r, sh, x)
    assert ei.value.status == 2
