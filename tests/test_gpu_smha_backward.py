"""GPU parity: uoe_smha_backward against the float64 oracle (derivative of Eq. 27-36 and of the gates, Eq. 14 / 21,
with the selection held constant; the oracle's backward is itself pinned by finite differences and by the dense
multi-head attention gradient).  bfloat16 tolerance: max|err| <= 2e-2 * max|ref| for each of dx (residual off,
where dy does not dominate it, and on), dWq, dWk, dWv, dWo, dW_r."""
import numpy as np
import pytest

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2
NAMES = ("dx", "dWq", "dWk", "dWv", "dWo", "dW_r")


def _w(**kw):
    base = dict(B=3, L=96, L_valid=96, m=6, c=3, d=128, n=2, k=1, d_ff=128, H=2, d_h=64, dtype="bf16",
                w_std=0.08, causal=False)
    base.update(kw)
    return gen.tiny(**base)


CASES = {
    "one_tile": _w(),
    "one_tile_causal": _w(causal=True, k=2),
    "pad": _w(L_valid=83, B=4, k=2),
    "pad_causal": _w(L_valid=70, causal=True),
    "two_heads_per_expert": _w(H=4, k=2),
    "three_tiles_ragged": _w(B=2, L=512, L_valid=512, m=8, c=5, n=4, k=2, H=4),
    "three_tiles_causal_pad": _w(B=2, L=512, L_valid=470, m=8, c=5, n=4, k=3, H=8, causal=True),
    "full_selection": _w(k=2, c=6, causal=True),
    # the three block shapes of the benchmark workloads, fewer samples
    "lm_shape": gen.WORKLOADS["cfg2_lm"].replace(B=4),
    "long_shape": gen.WORKLOADS["cfg3_long"].replace(B=2),
    "vit_shape": gen.WORKLOADS["cfg4_vit"].replace(B=12),
    # imbalanced expert loads (every sample pushed toward one expert drawn with Zipf weights) on the language-model shape
    "lm_shape_skewed": gen.WORKLOADS["cfg2_lm"].replace(B=6),
}


def _run(w, residual, use_gate=True, d_rope=0, skew=0.0):
    import paper_2503_02495_b200 as uoe
    Wr = gen.make_router(w, "att")
    x = gen.make_x(w, skew_beta=skew, W_r=Wr.f64) if skew else gen.make_x(w)
    if not w.name.startswith("cfg"):
        Wr = gen.store(Wr.f64 * 20, w.dtype)
    Wq, Wk, Wv, Wo = gen.make_attn_weights(w)
    dy = gen.make_dy(w)
    prob = problem_of(w, "att", residual=residual, gate=use_gate, d_rope=d_rope)
    xd, Wrd = to_dev(x), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    got = uoe.uoe_smha_backward(prob, xd, to_dev(Wq), to_dev(Wk), to_dev(Wv), to_dev(Wo), Wrd, r, to_dev(dy))
    ro = orc.with_selection(x.f64, Wr.f64, r.expert_idx.cpu().numpy(), r.patch_idx.cpu().numpy(), w.m, w.L_valid,
                            use_gate)
    ref = orc.smha_backward(x.f64, Wq.f64, Wk.f64, Wv.f64, Wo.f64, Wr.f64, ro, dy.f64, w.d_h, w.causal, residual,
                            use_gate, d_rope=d_rope)
    return [to_f64(t) for t in got], ref


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("residual", [False, True])
def test_smha_backward_matches_oracle(name, residual):
    w = CASES[name]
    if residual and "_shape" in name:
        pytest.skip("larger case: run once")
    got, ref = _run(w, residual, skew=4.0 if "skewed" in name else 0.0)
    for nm, g, r in zip(NAMES, got, ref[:6]):
        assert np.isfinite(g).all(), nm
        err = rel_inf(g, r)
        print(f"{name} residual={residual} {nm}: {err:.3e}  (|ref|max {np.abs(r).max():.3e})")
        assert err <= TOL, nm


@pytest.mark.parametrize("name,d_rope", [("one_tile_causal", 64), ("pad", 32), ("three_tiles_causal_pad", 16),
                                         ("lm_shape", 32)])
def test_smha_backward_with_rotary_embedding_matches_oracle(name, d_rope):
    got, ref = _run(CASES[name], False, d_rope=d_rope)
    for nm, g, r in zip(NAMES, got, ref[:6]):
        err = rel_inf(g, r)
        print(f"{name} d_rope={d_rope} {nm}: {err:.3e}")
        assert err <= TOL, nm


def test_smha_backward_without_gates_has_zero_router_gradient():
    got, ref = _run(CASES["pad"], False, use_gate=False)
    for nm, g, r in zip(NAMES[:5], got[:5], ref[:5]):
        assert rel_inf(g, r) <= TOL, nm
    assert np.all(got[5] == 0)


def test_smha_backward_is_deterministic():
    a, _ = _run(CASES["three_tiles_causal_pad"], True)
    b, _ = _run(CASES["three_tiles_causal_pad"], True)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)


def test_smha_backward_unsupported_shapes():
    import paper_2503_02495_b200 as uoe
    w = _w(d=64)
    prob = problem_of(w, "att")
    x, Wr = to_dev(gen.make_x(w)), to_dev(gen.make_router(w, "att"))
    Wq, Wk, Wv, Wo = (to_dev(t) for t in gen.make_attn_weights(w))
    r = uoe.uoe_route(prob, x, Wr)
    with pytest.raises(uoe.UoeError) as ei:
        uoe.uoe_smha_backward(prob, x, Wq, Wk, Wv, Wo, Wr, r, x)
    assert ei.value.status == 2


def test_smha_forward_and_backward_on_dynamic_capacity_routing():
    """Two-stage routing (Eq. 15-16) leaves unused slots (-1) at the end of a pair's patch list: zero rows in the routed
    buffers, no keys, no gradient.  Forward and backward must match the oracle on the same routing."""
    import paper_2503_02495_b200 as uoe
    w = _w(B=4, L=512, L_valid=490, m=8, c=8, n=4, k=2, H=4, causal=True)
    x, Wr = gen.make_x(w), gen.store(gen.make_router(w, "att").f64 * 30, w.dtype)
    Wq, Wk, Wv, Wo = gen.make_attn_weights(w)
    dy = gen.make_dy(w)
    prob = problem_of(w, "att", residual=False, dynamic_c=True)
    xd, Wrd = to_dev(x), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    p_idx = r.patch_idx.cpu().numpy()
    assert (p_idx < 0).any() and (p_idx >= 0).any()          # the case really has unused slots
    wd = [to_dev(t) for t in (Wq, Wk, Wv, Wo)]
    y = uoe.uoe_smha_forward(prob, xd, *wd, r)
    got = uoe.uoe_smha_backward(prob, xd, *wd, Wrd, r, to_dev(dy))
    ro = orc.with_selection(x.f64, Wr.f64, r.expert_idx.cpu().numpy(), p_idx, w.m, w.L_valid)
    ref_y = orc.smha_forward(x.f64, Wq.f64, Wk.f64, Wv.f64, Wo.f64, ro, w.d_h, True, residual=False)
    assert rel_inf(to_f64(y), ref_y) <= TOL
    ref = orc.smha_backward(x.f64, Wq.f64, Wk.f64, Wv.f64, Wo.f64, Wr.f64, ro, dy.f64, w.d_h, True, False, True)
    for nm, g, rr in zip(NAMES, got, ref[:6]):
        assert rel_inf(to_f64(g), rr) <= TOL, nm
