"""GPU parity at full size on the scale workload (B=8, L=4096, d=4096, 16 experts of width 1024, k=4,
c=16 of 32 patches): forward and backward run in the launch configuration the benchmark times, and are
checked on outputs the float64 oracle can compute piece by piece:

  - routing: the whole oracle (cheap)
  - y and dx of one sample (samples are independent given the weights)
  - dW1 and dW2 of one expert (the oracle is run with every other expert's slots emptied)
  - dW_r: a single-sample GPU call against the oracle, and additivity of the full-batch result over
    single-sample GPU calls (a property that holds at any size)
"""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import check_routing, problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = 2e-2


def test_scale_workload_forward_and_backward():
    import paper_2503_02495_b200 as uoe
    w = gen.WORKLOADS["cfg5_scale"]
    x, Wr, dy = gen.make_x(w), gen.make_router(w), gen.make_dy(w)
    W1, W2 = gen.make_mlp_weights(w)
    prob = problem_of(w, "mlp")
    xd, W1d, W2d, Wrd, dyd = to_dev(x), to_dev(W1), to_dev(W2), to_dev(Wr), to_dev(dy)

    # ---- routing: full oracle ----
    r = uoe.uoe_route(prob, xd, Wrd)
    ro_full = orc.route(x.f64, Wr.f64, w.k, w.m, w.c)
    near_e, near_p = check_routing(r, ro_full)
    print(f"near-tie mismatches: experts {near_e}, patch sets {near_p}")
    assert np.abs(r.p_patch.cpu().numpy() - ro_full.p_patch).max() < 2e-6

    # ---- full-size GPU forward + backward ----
    saved_h = uoe.alloc_saved_h(prob)
    y = uoe.uoe_mlp_forward(prob, xd, W1d, W2d, r, saved_h=saved_h)
    dx, dW1, dW2, dWr = uoe.uoe_mlp_backward(prob, xd, W1d, W2d, Wrd, r, saved_h, dyd)
    e_gpu = r.expert_idx.cpu().numpy()
    p_gpu = r.patch_idx.cpu().numpy()

    # ---- one sample: y, dx (and dW_r of a single-sample call) ----
    b = 3
    ro1 = orc.with_selection(x.f64[b:b + 1], Wr.f64, e_gpu[b:b + 1], p_gpu[b:b + 1], w.m, w.L_valid)
    y_ref = orc.mlp_forward(x.f64[b:b + 1], W1.f64, W2.f64, ro1, w.act)
    assert rel_inf(to_f64(y[b]), y_ref[0]) <= TOL
    dx_ref, _, _, dWr_ref1, _ = orc.mlp_backward(x.f64[b:b + 1], W1.f64, W2.f64, Wr.f64, ro1, dy.f64[b:b + 1], w.act)
    assert rel_inf(to_f64(dx[b]), dx_ref[0]) <= TOL

    # y and dx are bf16 roundings of x + (small) and dy + (small): the small parts are compared with the
    # residual off, in single-sample GPU calls
    prob1 = problem_of(w.replace(B=1), "mlp", residual=False)
    acc_dWr = torch.zeros_like(dWr)
    for bb in range(w.B):
        xb, dyb = xd[bb:bb + 1].contiguous(), dyd[bb:bb + 1].contiguous()
        rb = uoe.uoe_route(prob1, xb, Wrd)
        assert torch.equal(rb.expert_idx, r.expert_idx[bb:bb + 1]) and torch.equal(rb.patch_idx, r.patch_idx[bb:bb + 1])
        sh = uoe.alloc_saved_h(prob1)
        yb = uoe.uoe_mlp_forward(prob1, xb, W1d, W2d, rb, saved_h=sh)
        dxb, _, _, dWrb = uoe.uoe_mlp_backward(prob1, xb, W1d, W2d, Wrd, rb, sh, dyb)
        acc_dWr += dWrb
        if bb == b:
            z_ref = orc.mlp_forward(x.f64[b:b + 1], W1.f64, W2.f64, ro1, w.act, residual=False)
            err = rel_inf(to_f64(yb[0]), z_ref[0])
            print(f"expert term of sample {b}: {err:.3e}")
            assert err <= TOL
            assert rel_inf(to_f64(dWrb), dWr_ref1) <= TOL
            assert rel_inf(to_f64(dxb[0]), dx_ref[0] - dy.f64[b]) <= TOL
    assert rel_inf(to_f64(dWr), to_f64(acc_dWr)) <= 1e-3            # additivity over samples

    # ---- dW1, dW2 of two experts: the least loaded and the most loaded (the weight-gradient kernel hands out the
    #      most loaded expert's tiles first and the least loaded one's last, so they take different ways through it) ----
    load = np.bincount(e_gpu.ravel(), minlength=w.n)
    i_min = int(np.argmin(np.where(load > 0, load, 10 ** 9)))
    i_max = int(np.argmax(load))
    ro_all = orc.with_selection(x.f64, Wr.f64, e_gpu, p_gpu, w.m, w.L_valid)
    for i_star in sorted({i_min, i_max}):
        p_only = p_gpu.copy()
        p_only[e_gpu != i_star] = -1
        ro_e = orc.with_selection(x.f64, Wr.f64, e_gpu, p_only, w.m, w.L_valid)
        ro_e.gate = np.where(p_only >= 0, ro_all.gate, 0.0)
        _, dW1_ref, dW2_ref, _, _ = orc.mlp_backward(x.f64, W1.f64, W2.f64, Wr.f64, ro_e, dy.f64, w.act)
        print(f"expert {i_star} (load {load[i_star]}):",
              rel_inf(to_f64(dW1[i_star]), dW1_ref[i_star]), rel_inf(to_f64(dW2[i_star]), dW2_ref[i_star]))
        assert rel_inf(to_f64(dW1[i_star]), dW1_ref[i_star]) <= TOL
        assert rel_inf(to_f64(dW2[i_star]), dW2_ref[i_star]) <= TOL
    # an expert nobody chose gets exactly zero gradients
    for i in np.nonzero(load == 0)[0]:
        assert torch.count_nonzero(dW1[i]) == 0 and torch.count_nonzero(dW2[i]) == 0
