"""Patches of exactly 128 tokens: the second expert layer and the combine (Eq. 39-40) run as one kernel walked by
output patch, with the combine weight applied in the first layer's epilogue, and the backward's dx takes the same
route.  Forward and backward against the float64 oracle on shapes small enough for it, with what that path has to
get right: pad tokens inside the last real patch and patches of pad tokens only, patches no expert selected and
patches all k experts selected, gates off (unit weights, Eq. 20 literally), the residual off, dynamic capacity
(unused slots), k = n."""
import numpy as np
import pytest

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2


def _w(**kw):
    base = dict(B=3, L=512, L_valid=512, m=4, c=2, d=256, n=4, k=2, d_ff=512, H=0, d_h=0, dtype="bf16", w_std=0.05,
                act="silu")
    base.update(kw)
    return gen.tiny(**base)


CASES = {
    "base": (_w(), {}),
    "pad_inside_and_whole_pad_patch": (_w(B=4, L=768, L_valid=530, m=6, c=3), {}),
    "gate_off": (_w(act="gelu_tanh"), dict(gate=False)),
    "all_experts": (_w(k=4, c=3), {}),
    "one_patch_per_expert": (_w(B=5, L=1024, L_valid=1000, m=8, c=1, k=3, n=5, d_ff=5 * 128), {}),
    "dynamic_capacity": (_w(B=4, L=1024, L_valid=1024, m=8, c=6, k=2), dict(dynamic_c=True)),
    "wide": (_w(B=2, d=512, d_ff=4 * 384, L=384, L_valid=384, m=3, c=2), {}),
}


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("residual", [True, False])
def test_forward_and_backward_match_oracle(name, residual):
    import paper_2503_02495_b200 as uoe
    w, kw = CASES[name]
    use_gate = kw.get("gate", True)
    Wr = gen.store(gen.make_router(w).f64 * 10, w.dtype)
    x = gen.make_x(w)
    W1, W2 = gen.make_mlp_weights(w)
    dy = gen.make_dy(w)
    prob = problem_of(w, "mlp", residual=residual, **kw)
    xd, W1d, W2d, Wrd = to_dev(x), to_dev(W1), to_dev(W2), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    saved_h = uoe.alloc_saved_h(prob)
    y = uoe.uoe_mlp_forward(prob, xd, W1d, W2d, r, saved_h=saved_h)
    got = uoe.uoe_mlp_backward(prob, xd, W1d, W2d, Wrd, r, saved_h, to_dev(dy))
    e_idx, p_idx = r.expert_idx.cpu().numpy(), r.patch_idx.cpu().numpy()
    ro = orc.with_selection(x.f64, Wr.f64, e_idx, p_idx, w.m, w.L_valid, use_gate)
    y_ref = orc.mlp_forward(x.f64, W1.f64, W2.f64, ro, w.act, residual=residual)
    yg = to_f64(y)
    assert rel_inf(yg, y_ref) <= TOL
    if residual:
        assert np.array_equal(yg[:, w.L_valid:], x.f64[:, w.L_valid:])       # pad tokens: y = x exactly
    else:
        assert np.all(yg[:, w.L_valid:] == 0)
    # a patch nobody selected carries x (or zero) through unchanged
    l_p = w.L // w.m
    for b in range(w.B):
        chosen = set(int(j) for j in p_idx[b].ravel() if j >= 0)
        for j in range(w.m):
            if j not in chosen:
                rows = slice(j * l_p, min((j + 1) * l_p, w.L_valid))
                want = x.f64[b, rows] if residual else np.zeros_like(x.f64[b, rows])
                assert np.array_equal(yg[b, rows], want)
    ref = orc.mlp_backward(x.f64, W1.f64, W2.f64, Wr.f64, ro, dy.f64, w.act, residual, use_gate)
    for nm, g, rr in zip(("dx", "dW1", "dW2", "dW_r"), got, ref[:4]):
        if nm == "dW_r" and not use_gate:
            assert np.all(to_f64(g) == 0)
            continue
        assert rel_inf(to_f64(g), rr) <= TOL, nm
    if name == "dynamic_capacity":
        assert (p_idx == -1).any()


def test_these_shapes_take_the_patch_major_kernels():
    """The launches of a forward + backward on the base shape: no combine, one block-weight kernel, the second layer
    and dx under their usual labels."""
    import torch

    import paper_2503_02495_b200 as uoe
    w, _ = CASES["base"]
    Wr = gen.store(gen.make_router(w).f64 * 10, w.dtype)
    x, dy = gen.make_x(w), gen.make_dy(w)
    W1, W2 = gen.make_mlp_weights(w)
    prob = problem_of(w, "mlp")
    xd, W1d, W2d, Wrd = to_dev(x), to_dev(W1), to_dev(W2), to_dev(Wr)
    r = uoe.uoe_route(prob, xd, Wrd)
    saved_h = uoe.alloc_saved_h(prob)
    uoe.uoe_profile_enable(True)
    try:
        uoe.uoe_mlp_forward(prob, xd, W1d, W2d, r, saved_h=saved_h)
        uoe.uoe_mlp_backward(prob, xd, W1d, W2d, Wrd, r, saved_h, to_dev(dy))
        torch.cuda.synchronize()
        names = [n for n, _ in uoe.uoe_profile_records()]
    finally:
        uoe.uoe_profile_enable(False)
    assert "combine" not in names
    assert names.count("block_gate") == 1 and names.count("gemm2") == 1 and names.count("bwd_dx") == 1
