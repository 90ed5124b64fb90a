"""GPU parity: uoe_mlp_forward against the float64 oracle (Eq. 18-20, 37-40).

The oracle is evaluated on the GPU's own selection (so that a near-tie in routing, which is checked
separately, does not leak into the layer comparison) with probabilities and gates recomputed in
float64.  Tolerances: float32  max|err| <= 1e-4 * max|ref|;  bfloat16  max|err| <= 2e-2 * max|ref|.
They are applied to the expert term alone (RESIDUAL off) and, with the residual on, to y.
"""
import numpy as np
import pytest
import torch

import uoe_inputs as gen
from oracle import uoe_oracle as orc
from tests.helpers import problem_of, rel_inf, to_dev, to_f64

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}

CASES = {
    "tiny_f32": gen.tiny(d=16, d_ff=32),
    "tiny_pad_f32": gen.tiny(L_valid=21, B=5, d=16, d_ff=32),
    "tiny_k1c1": gen.tiny(k=1, c=1, d=16, d_ff=32),
    "tiny_full": gen.tiny(k=4, c=6, d=16, d_ff=32),
    "odd_f32": gen.tiny(B=3, m=7, c=3, L=70, L_valid=64, d=36, n=3, k=2, d_ff=60, act="gelu_tanh"),
    "cfg1": gen.WORKLOADS["cfg1_small_f32"],
    "small_bf16": gen.tiny(B=3, L=96, L_valid=96, m=6, c=3, d=64, n=4, k=2, d_ff=256, dtype="bf16", w_std=0.05),
    "pad_bf16": gen.tiny(B=5, L=112, L_valid=100, m=7, c=4, d=128, n=3, k=2, d_ff=192, dtype="bf16", w_std=0.05,
                         act="gelu_erf"),
    # long K and many row tiles: 256-row tiles on CTA pairs, with regions of 3*load 128-row blocks (half tiles) ...
    "tall_tiles": gen.tiny(B=40, L=1152, L_valid=1152, m=9, c=3, d=1024, n=4, k=2, d_ff=4096, dtype="bf16", w_std=0.02),
    # ... and with a width that is not a multiple of 128 (17 K blocks): GEMM1 takes the 256-row tiles of one CTA
    "tall_tiles_k1088": gen.tiny(B=40, L=1152, L_valid=1152, m=9, c=3, d=1088, n=4, k=2, d_ff=4096, dtype="bf16",
                                 w_std=0.02),
    # CTA-pair tiles with x gathered in 16-token patches (eight boxes per 128-row block and K step, two K steps per round)
    "pair_tiles_short_patches": gen.tiny(B=80, L=256, L_valid=250, m=16, c=8, d=512, n=4, k=2, d_ff=4096, dtype="bf16",
                                         w_std=0.03),
    # narrow experts (d_e = 256): both GEMMs in one kernel; 64 output columns, a ragged second output half, pad
    # tokens, and a patch length the GEMM cannot gather by itself (routed copy of x as the A operand)
    "fused_d64": gen.tiny(B=3, L=96, L_valid=96, m=6, c=3, d=64, n=2, k=1, d_ff=512, dtype="bf16", w_std=0.05),
    "fused_d192_pad": gen.tiny(B=5, L=112, L_valid=100, m=7, c=4, d=192, n=3, k=2, d_ff=768, dtype="bf16", w_std=0.05,
                               act="gelu_erf"),
    "fused_d448": gen.tiny(B=4, L=256, L_valid=250, m=8, c=5, d=448, n=4, k=3, d_ff=1024, dtype="bf16", w_std=0.04,
                           act="gelu_tanh"),
    "fused_copy_a": gen.tiny(B=4, L=120, L_valid=115, m=10, c=4, d=128, n=2, k=2, d_ff=512, dtype="bf16", w_std=0.05),
    "cfg2": gen.WORKLOADS["cfg2_lm"],
    "cfg3": gen.WORKLOADS["cfg3_long"],
    "cfg4": gen.WORKLOADS["cfg4_vit"],
}


def _run(w, residual, use_gate, router_scale=1.0):
    import paper_2503_02495_b200 as uoe
    x, Wr = gen.make_x(w), gen.make_router(w)
    if router_scale != 1.0:
        Wr = gen.store(Wr.f64 * router_scale, w.dtype)
    W1, W2 = gen.make_mlp_weights(w)
    prob = problem_of(w, "mlp", residual=residual, gate=use_gate)
    xd = to_dev(x)
    r = uoe.uoe_route(prob, xd, to_dev(Wr))
    y = uoe.uoe_mlp_forward(prob, xd, to_dev(W1), to_dev(W2), r)
    ro = orc.with_selection(x.f64, Wr.f64, r.expert_idx.cpu().numpy(), r.patch_idx.cpu().numpy(), w.m, w.L_valid,
                            use_gate)
    ref = orc.mlp_forward(x.f64, W1.f64, W2.f64, ro, w.act, residual=residual)
    return to_f64(y), ref, x.f64, r


@pytest.mark.parametrize("name", list(CASES))
def test_expert_term_matches_oracle(name):
    w = CASES[name]
    scale = 20.0 if not (name.startswith("cfg") or name.startswith("tall_tiles")) else 1.0
    y, ref, x, r = _run(w, residual=False, use_gate=True, router_scale=scale)
    err = rel_inf(y, ref)
    print(f"{name}: max|err|/max|ref| = {err:.3e}")
    assert err <= TOL[w.dtype]
    # rows nobody selected, and pad rows, are exactly zero without the residual
    assert np.array_equal(y == 0, ref == 0) or np.all(y[ref == 0] == 0)


@pytest.mark.parametrize("name", ["tiny_f32", "tiny_pad_f32", "cfg1", "small_bf16", "cfg2", "cfg4"])
def test_residual_output_matches_oracle(name):
    w = CASES[name]
    y, ref, x, r = _run(w, residual=True, use_gate=True, router_scale=20.0 if not name.startswith("cfg") else 1.0)
    assert rel_inf(y, ref) <= TOL[w.dtype]
    if w.dtype == "f32":
        assert rel_inf(y - x, ref - x) <= TOL["f32"]
    # unselected patches and pad rows pass x through bit-exactly
    p = r.patch_idx.cpu().numpy()
    for b in range(w.B):
        used = set(int(j) for j in p[b].ravel() if j >= 0)
        for j in range(w.m):
            if j not in used:
                sl = slice(j * w.l_p, (j + 1) * w.l_p)
                assert np.array_equal(y[b, sl], x[b, sl])
        assert np.array_equal(y[b, w.L_valid:], x[b, w.L_valid:])


@pytest.mark.parametrize("name", ["tiny_f32", "small_bf16"])
def test_unit_weights_when_gate_flag_is_off(name):
    w = CASES[name]
    y, ref, _, _ = _run(w, residual=False, use_gate=False, router_scale=20.0)
    assert rel_inf(y, ref) <= TOL[w.dtype]


@pytest.mark.parametrize("name", ["tiny_full", "small_bf16"])
def test_full_selection_equals_dense_mlp(name):
    # k = n, c = m, unit weights: the union of experts is the dense MLP (Eq. 1, 5)
    w = CASES[name].replace(k=CASES[name].n, c=CASES[name].m)
    y, ref, x, _ = _run(w, residual=False, use_gate=False)
    W1, W2 = gen.make_mlp_weights(w)
    dense = orc.act_fn(x @ np.concatenate(list(W1.f64), axis=1), w.act) @ np.concatenate(list(W2.f64), axis=0)
    dense[:, w.L_valid:] = 0
    assert rel_inf(y, dense) <= TOL[w.dtype]


def test_caller_supplied_routing_and_determinism():
    import paper_2503_02495_b200 as uoe
    w = CASES["small_bf16"]
    x, Wr = gen.make_x(w), gen.make_router(w)
    W1, W2 = gen.make_mlp_weights(w)
    prob = problem_of(w, "mlp", residual=False)
    ro = orc.route(x.f64, Wr.f64 * 20, w.k, w.m, w.c)
    r = uoe.Routing(torch.from_numpy(ro.expert_idx.astype(np.int32)).cuda(),
                    torch.from_numpy(ro.patch_idx.astype(np.int32)).cuda(),
                    torch.from_numpy(ro.gate.astype(np.float32)).cuda(),
                    torch.from_numpy(ro.p_samp.astype(np.float32)).cuda(),
                    torch.from_numpy(ro.p_patch.astype(np.float32)).cuda(),
                    torch.from_numpy(ro.offsets.astype(np.int32)).cuda())
    args = (prob, to_dev(x), to_dev(W1), to_dev(W2), r)
    y1 = uoe.uoe_mlp_forward(*args)
    y2 = uoe.uoe_mlp_forward(*args)
    assert torch.equal(y1, y2)
    ref = orc.mlp_forward(x.f64, W1.f64, W2.f64, ro, w.act, residual=False)
    assert rel_inf(to_f64(y1), ref) <= TOL["bf16"]


def test_bad_arguments_return_codes():
    import paper_2503_02495_b200 as uoe
    w = CASES["tiny_f32"]
    prob = problem_of(w, "mlp")
    x, Wr = to_dev(gen.make_x(w)), to_dev(gen.make_router(w))
    with pytest.raises(uoe.UoeError) as ei:
        uoe.uoe_route(prob, x, Wr, ws=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert ei.value.status == 3
    r = uoe.uoe_route(prob, x, Wr)
    bad = uoe.Routing(r.expert_idx.clone().fill_(99), r.patch_idx, r.gate, r.p_samp, r.p_patch, r.expert_offsets)
    W1, W2 = gen.make_mlp_weights(w)
    ws = uoe.alloc_workspace(prob, uoe.UOE_OP_MLP_FWD)
    with pytest.raises(uoe.UoeError) as ei:
        uoe.uoe_mlp_forward(prob, x, to_dev(W1), to_dev(W2), bad, ws=ws)
    assert ei.value.status == 6      # recorded on the device, nothing faulted
    assert uoe.uoe_read_device_status(ws) == 0       # reporting an anomaly clears the sticky status word
    uoe.uoe_mlp_forward(prob, x, to_dev(W1), to_dev(W2), r, ws=ws)      # and the workspace is usable again
