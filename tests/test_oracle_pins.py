"""Pins for the float64 oracle: each test ties one part of it to something other than itself.

  - exhaustive subset search and planted ties          -> top-k / top-c selection (Eq. 17, 22)
  - dense MLP / textbook multi-head attention          -> expert math at k=n, c=m (Eq. 1, 5, 8-11)
  - mask identity of Fig. 4                            -> causal mask handling
  - special cases, bounds, symmetries                  -> routing structure (Eq. 20, 23, 26)
  - central finite differences                         -> backward
  - scalar-loop twin                                   -> array indexing
  - planted mistakes                                   -> the pins above do catch a wrong oracle
"""
import math

import numpy as np
import pytest

import uoe_inputs as gen
from oracle import loops
from oracle import uoe_oracle as orc


def _inputs(w, blocks=("mlp", "att")):
    x = gen.make_x(w).f64
    out = dict(x=x, Wr=gen.make_router(w, "mlp").f64, Wra=gen.make_router(w, "att").f64)
    if "mlp" in blocks:
        W1, W2 = gen.make_mlp_weights(w)
        out.update(W1=W1.f64, W2=W2.f64)
    if "att" in blocks:
        Wq, Wk, Wv, Wo = gen.make_attn_weights(w)
        out.update(Wq=Wq.f64, Wk=Wk.f64, Wv=Wv.f64, Wo=Wo.f64)
    return out


def _boost_router(Wr, scale=40.0):
    # larger router weights so that the gates are far from uniform in the tiny cases
    return Wr * scale


# ----------------------------------------------------------------------------------------------
# generator sanity (the pins below rely on these inputs)
# ----------------------------------------------------------------------------------------------

def test_generator_is_counter_based_and_normal():
    a = gen.normal(5, 2, (1000, 64))
    b = gen.normal(5, 2, (1000, 64), chunk=999)
    assert np.array_equal(a, b)
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1.0) < 0.02
    assert abs(np.mean(a ** 4) - 3.0) < 0.15
    assert not np.array_equal(a, gen.normal(5, 3, (1000, 64)))


def test_bf16_rounding_is_nearest_even():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -2.5, 3.140625], dtype=np.float32)
    got = gen.bf16_bits_to_f64(gen.f32_to_bf16_bits(v))
    # ties: 1+2^-8 is halfway between 1 and 1+2^-7 -> even mantissa (1.0); 1+3*2^-8 -> 1+2^-6
    assert got.tolist() == [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -2.5, 3.140625]


# ----------------------------------------------------------------------------------------------
# activations against closed forms
# ----------------------------------------------------------------------------------------------

def test_activation_closed_forms():
    h = np.array([0.0, 1.0, -1.0, 3.0])
    assert np.allclose(orc.act_fn(h, "silu"), [0.0, 1 / (1 + math.e ** -1), -1 / (1 + math.e), 3 / (1 + math.e ** -3)], atol=1e-15)
    # GELU(x) = x * Phi(x); Phi(1) = 0.841344746068543 (standard normal cdf)
    assert np.allclose(orc.act_fn(h, "gelu_erf"), [0.0, 0.841344746068543, -0.158655253931457, 3 * 0.998650101968370], atol=1e-14)
    assert np.allclose(orc.act_fn(h, "gelu_tanh"), orc.act_fn(h, "gelu_erf"), atol=2e-3)
    for act in ("silu", "gelu_erf", "gelu_tanh", "identity"):
        hh = np.linspace(-4, 4, 41)
        fd = (orc.act_fn(hh + 1e-6, act) - orc.act_fn(hh - 1e-6, act)) / 2e-6
        assert np.allclose(orc.act_grad(hh, act), fd, atol=1e-8)


# ----------------------------------------------------------------------------------------------
# selection: exhaustive search, ties, bounds
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n,k,m,c", [(4, 2, 6, 3), (5, 1, 5, 5), (3, 3, 4, 1), (5, 4, 6, 2)])
def test_selection_matches_exhaustive_search(n, k, m, c):
    w = gen.tiny(n=n, k=k, m=m, c=c, L=m * 4, L_valid=m * 4, d=8, d_ff=n * 4, H=0, d_h=0, B=4)
    x = gen.make_x(w).f64
    Wr = _boost_router(gen.make_router(w).f64)
    r = orc.route(x, Wr, k, m, c)
    for b in range(w.B):
        # the chosen set must maximise the score sum among all subsets of that size
        import itertools
        best = max(itertools.combinations(range(n), k), key=lambda s: sum(r.p_samp[b, i] for i in s))
        assert sorted(best) == r.expert_idx[b].tolist()
        for s, i in enumerate(r.expert_idx[b]):
            bestp = max(itertools.combinations(range(m), c), key=lambda q: sum(r.p_patch[b, i, j] for j in q))
            assert sorted(bestp) == r.patch_idx[b, s].tolist()


def test_selection_tie_goes_to_lower_index():
    p_samp = np.array([[0.2, 0.3, 0.3, 0.2]])
    p_patch = np.zeros((1, 4, 5))
    p_patch[0, 1] = [0.5, 0.1, 0.5, 0.5, 0.1]
    p_patch[0, 0] = [0.1, 0.1, 0.1, 0.1, 0.1]
    cnt = np.full(5, 4)
    e, p, em, pm = orc.select(p_samp, p_patch, cnt, k=3, c=2)
    assert e[0].tolist() == [0, 1, 2]           # 0.2 tie between experts 0 and 3 -> 0
    assert p[0, 1].tolist() == [0, 2]           # three-way tie at 0.5 -> patches 0 and 2
    assert p[0, 0].tolist() == [0, 1]
    assert em[0] == 0.0 and pm[0, 1] == 0.0
    # the exhaustive search in the scalar twin follows the same rule
    assert loops.best_subset(p_samp[0].tolist(), range(4), 3) == [0, 1, 2]
    assert loops.best_subset(p_patch[0, 1].tolist(), range(5), 2) == [0, 2]


def test_margin_definition():
    p = np.array([[0.4, 0.1, 0.3, 0.2]])
    e, _, em, _ = orc.select(p, np.full((1, 4, 2), 0.25), np.full(2, 1), k=2, c=2)
    assert e[0].tolist() == [0, 2]
    assert em[0] == pytest.approx((0.3 - 0.2) / 0.3)


@pytest.mark.parametrize("L_valid", [24, 21, 17])
def test_routing_bounds(L_valid):
    w = gen.tiny(B=7, L_valid=L_valid)
    x = gen.make_x(w).f64
    r = orc.route(x, _boost_router(gen.make_router(w).f64), w.k, w.m, w.c, L_valid=L_valid)
    assert np.allclose(r.p_samp.sum(axis=1), 1.0) and np.allclose(r.p_patch.sum(axis=1), 1.0)
    assert r.load.sum() == w.B * w.k and r.load.min() >= 0 and r.load.max() <= w.B
    cnt = orc.patch_valid_counts(w.L, w.m, L_valid)
    n_elig = int((cnt > 0).sum())
    for b in range(w.B):
        assert np.all(np.diff(r.expert_idx[b]) > 0)
        use = np.zeros(w.m, dtype=int)
        for s in range(w.k):
            sel = r.patch_idx[b, s][r.patch_idx[b, s] >= 0]
            assert len(sel) == min(w.c, n_elig)
            assert np.all(np.diff(sel) > 0) and sel.min() >= 0 and sel.max() < w.m
            assert np.all(cnt[sel] > 0)
            use[sel] += 1
        assert use.max() <= w.k
    assert np.all(np.diff(r.offsets) >= 0) and np.all(r.offsets % 128 == 0)
    r1 = orc.route(x, _boost_router(gen.make_router(w).f64), w.k, w.m, w.c, L_valid=L_valid, row_align=1)
    assert r1.offsets[-1] == w.B * w.k * w.c * w.l_p
    # buffer rows: every (sample, expert) pair gets its own disjoint run of c*l_p rows inside its expert
    seen = set()
    for b in range(w.B):
        for s in range(w.k):
            row = orc.buffer_row(r1, b, s)
            i = r1.expert_idx[b, s]
            assert r1.offsets[i] <= row and row + w.l_a <= r1.offsets[i + 1]
            assert row not in seen
            seen.add(row)


def test_patch_softmax_is_over_experts_not_patches():
    # Eq. 14 normalises each patch column over the n experts.
    w = gen.tiny()
    x = gen.make_x(w).f64
    Wr = _boost_router(gen.make_router(w).f64)
    p_samp, p_patch, pool, samp, cnt = orc.router_probs(x, Wr, w.m, w.L)
    b, j = 1, 2
    logits = x[b, j * w.l_p:(j + 1) * w.l_p].mean(0) @ Wr
    ref = np.exp(logits) / np.exp(logits).sum()
    assert np.allclose(p_patch[b, :, j], ref, atol=1e-14)
    sl = x[b].mean(0) @ Wr
    assert np.allclose(p_samp[b], np.exp(sl) / np.exp(sl).sum(), atol=1e-14)


# ----------------------------------------------------------------------------------------------
# lossless decomposition: k=n, c=m reproduces the dense layer (Eq. 1, 5; Eq. 8-11)
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("act", ["silu", "gelu_erf", "gelu_tanh", "identity"])
def test_uome_full_selection_equals_dense_mlp(act):
    w = gen.tiny(k=4, c=6, act=act)
    t = _inputs(w, ("mlp",))
    r = orc.route(t["x"], t["Wr"], w.k, w.m, w.c, use_gate=False)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, act)
    A_I = np.concatenate([t["W1"][i] for i in range(w.n)], axis=1)     # [d, d_ff]: column blocks
    A_O = np.concatenate([t["W2"][i] for i in range(w.n)], axis=0)     # [d_ff, d]: row blocks
    dense = orc.act_fn(t["x"].reshape(-1, w.d) @ A_I, act) @ A_O
    assert np.allclose(y - t["x"], dense.reshape(t["x"].shape), rtol=1e-12, atol=1e-13)


def test_uome_full_selection_with_gates_scales_hidden_blocks():
    w = gen.tiny(k=4, c=6)
    t = _inputs(w, ("mlp",))
    Wr = _boost_router(t["Wr"])
    r = orc.route(t["x"], Wr, w.k, w.m, w.c, use_gate=True)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
    A_I = np.concatenate(list(t["W1"]), axis=1)
    A_O = np.concatenate(list(t["W2"]), axis=0)
    hidden = orc.act_fn(t["x"] @ A_I, "silu")                          # [B, L, d_ff]
    for b in range(w.B):
        for tkn in range(w.L):
            j = tkn // w.l_p
            for i in range(w.n):
                hidden[b, tkn, i * w.d_e:(i + 1) * w.d_e] *= r.p_samp[b, i] * r.p_patch[b, i, j]
    assert np.allclose(y - t["x"], hidden @ A_O, rtol=1e-12, atol=1e-13)


def test_uome_full_selection_with_biases_equals_dense_mlp_with_bias():
    # the bias branch (the in-place bias of the batched product, Section III-D.2): at k=n, c=m with unit weights the
    # layer is the dense MLP whose first bias is the concatenation of the experts' b1 and whose second bias is the
    # SUM of the experts' b2 (every expert adds its own b2 to every token it serves, Eq. 5-7)
    w = gen.tiny(k=4, c=6, act="gelu_erf")
    t = _inputs(w, ("mlp",))
    b1 = gen.normal(500, 1, (w.n, w.d_e), 0.5)
    b2 = gen.normal(500, 2, (w.n, w.d), 0.5)
    r = orc.route(t["x"], t["Wr"], w.k, w.m, w.c, use_gate=False)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "gelu_erf", b1=b1, b2=b2)
    A_I = np.concatenate(list(t["W1"]), axis=1)
    A_O = np.concatenate(list(t["W2"]), axis=0)
    dense = orc.act_fn(t["x"] @ A_I + b1.reshape(-1), "gelu_erf") @ A_O + b2.sum(axis=0)
    assert np.allclose(y - t["x"], dense, rtol=1e-12, atol=1e-13)
    # a dropped or misplaced bias is visible at this size
    y_nob = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "gelu_erf")
    assert np.abs(y - y_nob).max() > 0.1
    # partial selection: a token served by q experts receives q second-layer biases, scaled by their gates
    w2 = gen.tiny(act="identity")
    t2 = _inputs(w2, ("mlp",))
    r2 = orc.route(t2["x"], _boost_router(t2["Wr"]), w2.k, w2.m, w2.c)
    zero = np.zeros_like(t2["W1"])
    b2s = gen.normal(500, 3, (w2.n, w2.d), 1.0)
    y2 = orc.mlp_forward(t2["x"], zero, t2["W2"], r2, "identity", b1=np.zeros((w2.n, w2.d_e)), b2=b2s, residual=False)
    for b in range(w2.B):
        want = np.zeros((w2.L, w2.d))
        for s, i in enumerate(r2.expert_idx[b]):
            for u, j in enumerate(r2.patch_idx[b, s]):
                if j >= 0:
                    want[j * w2.l_p:(j + 1) * w2.l_p] += r2.gate[b, s, u] * b2s[i]
        assert np.allclose(y2[b], want, rtol=1e-12, atol=1e-14)


def _textbook_mha(x, WI_q, WI_k, WI_v, WO, heads, d_h, causal, L_valid):
    """Plain multi-head attention on one sample, written independently of the oracle."""
    L = x.shape[0]
    q, k, v = x @ WI_q, x @ WI_k, x @ WI_v
    out = np.zeros_like(q)
    for h in range(heads):
        for a in range(L):
            w = np.full(L, -np.inf)
            for b in range(L):
                if b < L_valid and (not causal or b <= a):
                    w[b] = q[a, h * d_h:(h + 1) * d_h] @ k[b, h * d_h:(h + 1) * d_h] / math.sqrt(d_h)
            w = np.exp(w - w.max())
            w /= w.sum()
            out[a, h * d_h:(h + 1) * d_h] = w @ v[:, h * d_h:(h + 1) * d_h]
    return out @ WO


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("H,L_valid", [(4, 24), (8, 24), (4, 22)])
def test_smha_full_selection_equals_multihead_attention(causal, H, L_valid):
    w = gen.tiny(k=4, c=6, H=H, L_valid=L_valid, causal=causal)
    t = _inputs(w, ("att",))
    r = orc.route(t["x"], t["Wra"], w.k, w.m, w.c, L_valid=L_valid, use_gate=False)
    y = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, causal)
    cat = lambda W: np.concatenate(list(W), axis=1)
    WO = np.concatenate(list(t["Wo"]), axis=0)
    for b in range(w.B):
        ref = _textbook_mha(t["x"][b], cat(t["Wq"]), cat(t["Wk"]), cat(t["Wv"]), WO, H, w.d_h, causal, L_valid)
        assert np.allclose((y - t["x"])[b, :L_valid], ref[:L_valid], rtol=1e-11, atol=1e-12)
        assert np.array_equal(y[b, L_valid:], t["x"][b, L_valid:])


@pytest.mark.parametrize("causal,L_valid", [(False, 24), (True, 24), (False, 21)])
def test_smha_log_sum_exp_output_is_the_textbook_one(causal, L_valid):
    # return_lse: per (sample, chosen expert, head) the natural log of the sum over kept keys of exp(q.k / sqrt(d_h)),
    # written here from the definition with scalar loops over the gathered tokens
    w = gen.tiny(B=2, causal=causal, L_valid=L_valid, H=8)
    t = _inputs(w, ("att",))
    r = orc.route(t["x"], _boost_router(t["Wra"]), w.k, w.m, w.c, L_valid=L_valid)
    y, lse = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, causal, return_lse=True)
    assert np.array_equal(y, orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, causal))
    heads = w.d_g // w.d_h
    assert len(lse) == w.B * w.k * heads
    for b in range(w.B):
        for s, i in enumerate(r.expert_idx[b]):
            tok = orc.gathered_tokens(r, b, s)
            q, kk = t["x"][b, tok] @ t["Wq"][i], t["x"][b, tok] @ t["Wk"][i]
            for hd in range(heads):
                sl = slice(hd * w.d_h, (hd + 1) * w.d_h)
                got = lse[(b, s, hd)]
                assert got.shape == (len(tok),)
                for a in range(len(tok)):
                    tot = 0.0
                    for bb in range(len(tok)):
                        if tok[bb] < L_valid and (not causal or bb <= a):
                            tot += math.exp(float(q[a, sl] @ kk[bb, sl]) / math.sqrt(w.d_h))
                    assert abs(got[a] - math.log(tot)) <= 1e-12 * max(1.0, abs(math.log(tot)))


def test_fig4_mask_identity_and_its_negative():
    L, l_p = 24, 4
    full = np.tril(np.ones((L, L), dtype=bool))
    tok = np.concatenate([np.arange(j * l_p, (j + 1) * l_p) for j in (1, 3, 4)])
    assert np.array_equal(full[np.ix_(tok, tok)], np.tril(np.ones((len(tok),) * 2, dtype=bool)))
    bad = np.concatenate([np.arange(j * l_p, (j + 1) * l_p) for j in (3, 1, 4)])      # unsorted
    assert not np.array_equal(full[np.ix_(bad, bad)], np.tril(np.ones((len(bad),) * 2, dtype=bool)))


def test_smha_causal_partial_selection_uses_leading_triangle():
    # the oracle double-indexes the L x L mask; an attention over the gathered tokens with a plain
    # l_a x l_a lower triangle (Fig. 4) must give the same result
    w = gen.tiny(causal=True, B=2)
    t = _inputs(w, ("att",))
    r = orc.route(t["x"], _boost_router(t["Wra"]), w.k, w.m, w.c)
    y = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, True)
    for b in range(w.B):
        acc = t["x"][b].copy()
        for s, i in enumerate(r.expert_idx[b]):
            tok = orc.gathered_tokens(r, b, s)
            ref = _textbook_mha(t["x"][b, tok], t["Wq"][i], t["Wk"][i], t["Wv"][i], t["Wo"][i],
                                w.d_g // w.d_h, w.d_h, True, len(tok))
            g = np.repeat(r.gate[b, s], w.l_p)
            acc[tok] += g[:, None] * ref
        assert np.allclose(y[b], acc, rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------------------------
# special cases and symmetries
# ----------------------------------------------------------------------------------------------

def test_c_equals_m_is_pure_expert_selection():
    # Eq. 21-26: whole samples go to their top-k experts
    w = gen.tiny(c=6)
    t = _inputs(w, ("mlp",))
    Wr = _boost_router(t["Wr"])
    r = orc.route(t["x"], Wr, w.k, w.m, w.c, use_gate=False)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
    for b in range(w.B):
        sl = t["x"][b].mean(0) @ Wr
        top = np.sort(np.argsort(-sl, kind="stable")[:w.k])
        assert top.tolist() == r.expert_idx[b].tolist()
        ref = t["x"][b].copy()
        for i in top:
            ref += orc.act_fn(t["x"][b] @ t["W1"][i], "silu") @ t["W2"][i]      # Eq. 25-26
        assert np.allclose(y[b], ref, rtol=1e-12, atol=1e-13)


def test_k_equals_n_is_pure_data_selection():
    # Eq. 12-20: every expert takes its own top-c patches
    w = gen.tiny(k=4)
    t = _inputs(w, ("mlp",))
    Wr = _boost_router(t["Wr"])
    r = orc.route(t["x"], Wr, w.k, w.m, w.c, use_gate=False)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
    for b in range(w.B):
        ref = t["x"][b].copy()
        xp = t["x"][b].reshape(w.m, w.l_p, w.d)
        g = np.stack([orc.softmax(xp[j].mean(0) @ Wr, 0) for j in range(w.m)], axis=1)     # [n, m]
        for i in range(w.n):
            ids = np.sort(np.argsort(-g[i], kind="stable")[:w.c])                           # Eq. 17 + sort
            assert ids.tolist() == r.patch_idx[b, i].tolist()
            for j in ids:
                ref[j * w.l_p:(j + 1) * w.l_p] += orc.act_fn(xp[j] @ t["W1"][i], "silu") @ t["W2"][i]
        assert np.allclose(y[b], ref, rtol=1e-12, atol=1e-13)


def test_unselected_patches_and_pad_rows_pass_through():
    w = gen.tiny(L_valid=21)
    t = _inputs(w)
    r = orc.route(t["x"], _boost_router(t["Wr"]), w.k, w.m, w.c, L_valid=21)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
    y2 = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, False)
    for b in range(w.B):
        used = set(int(j) for j in r.patch_idx[b].ravel() if j >= 0)
        for j in range(w.m):
            sl = slice(j * w.l_p, (j + 1) * w.l_p)
            if j not in used:
                assert np.array_equal(y[b, sl], t["x"][b, sl]) and np.array_equal(y2[b, sl], t["x"][b, sl])
        assert np.array_equal(y[b, 21:], t["x"][b, 21:]) and np.array_equal(y2[b, 21:], t["x"][b, 21:])


def test_batch_permutation_and_expert_permutation():
    w = gen.tiny(B=5)
    t = _inputs(w)
    Wr = _boost_router(t["Wr"])
    r = orc.route(t["x"], Wr, w.k, w.m, w.c)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
    ya = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, True)
    perm = np.array([3, 0, 4, 2, 1])
    rp = orc.route(t["x"][perm], Wr, w.k, w.m, w.c)
    assert np.allclose(orc.mlp_forward(t["x"][perm], t["W1"], t["W2"], rp, "silu"), y[perm], atol=1e-14)
    ep = np.array([2, 0, 3, 1])
    re = orc.route(t["x"], Wr[:, ep], w.k, w.m, w.c)
    assert np.allclose(orc.mlp_forward(t["x"], t["W1"][ep], t["W2"][ep], re, "silu"), y, atol=1e-13)
    assert np.allclose(orc.smha_forward(t["x"], t["Wq"][ep], t["Wk"][ep], t["Wv"][ep], t["Wo"][ep], re, w.d_h, True),
                       ya, atol=1e-13)


def test_identity_activation_is_linear_for_fixed_routing():
    w = gen.tiny()
    t = _inputs(w, ("mlp",))
    r = orc.route(t["x"], _boost_router(t["Wr"]), w.k, w.m, w.c)
    f = lambda xx: orc.mlp_forward(xx, t["W1"], t["W2"], r, "identity", residual=False)
    x2 = gen.normal(99, 0, t["x"].shape)
    assert np.allclose(f(2.0 * t["x"] - 3.0 * x2), 2.0 * f(t["x"]) - 3.0 * f(x2), atol=1e-12)


def test_activation_sits_between_the_two_layers_only():
    # phi(Y1 + Y2) != phi(Y1) + phi(Y2): an oracle that applied phi after the second layer per expert
    # would break the dense equivalence; check the inequality the paper warns about on real numbers
    w = gen.tiny(k=4, c=6)
    t = _inputs(w, ("mlp",))
    Y = [t["x"][0] @ t["W1"][i] @ t["W2"][i] for i in range(w.n)]
    assert not np.allclose(orc.act_fn(sum(Y), "silu"), sum(orc.act_fn(v, "silu") for v in Y), atol=1e-6)


def test_theoretical_cost_ratio():
    # k/n = 1/2 in expert-selection mode, or c/m = 1/2 in data-selection mode, is half the dense rows
    B, L = 8, 64
    dense_rows = B * 4 * L                       # n experts x all tokens
    assert orc.routed_rows(B, k=2, c=8, l_p=8) * 2 == dense_rows
    assert orc.routed_rows(B, k=4, c=4, l_p=8) * 2 == dense_rows


# ----------------------------------------------------------------------------------------------
# scalar-loop twin
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("L_valid,causal,act", [(24, False, "silu"), (22, True, "gelu_erf"), (17, False, "gelu_tanh")])
def test_array_oracle_equals_scalar_loops(L_valid, causal, act):
    w = gen.tiny(B=2, L_valid=L_valid, causal=causal, act=act)
    t = _inputs(w)
    Wr = _boost_router(t["Wr"])
    r = orc.route(t["x"], Wr, w.k, w.m, w.c, L_valid=L_valid)
    lr = loops.route(t["x"].tolist(), Wr.tolist(), w.B, w.L, w.d, w.n, w.k, w.m, w.c, L_valid)
    for b in range(w.B):
        assert np.allclose(lr[b]["p_samp"], r.p_samp[b], atol=1e-13)
        assert np.allclose(np.array(lr[b]["p_patch"]), r.p_patch[b], atol=1e-13)
        assert [i for i, _, _ in lr[b]["sel"]] == r.expert_idx[b].tolist()
        for s, (i, patches, g) in enumerate(lr[b]["sel"]):
            got = [int(j) for j in r.patch_idx[b, s] if j >= 0]
            assert patches == got
            assert np.allclose(g, r.gate[b, s][:len(g)], atol=1e-14)
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, act)
    yl = loops.mlp_forward(t["x"].tolist(), t["W1"].tolist(), t["W2"].tolist(), lr, w.B, w.L, w.d, w.d_e, w.m,
                           L_valid, act)
    assert np.allclose(np.array(yl), y, rtol=1e-12, atol=1e-12)
    ya = orc.smha_forward(t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"], r, w.d_h, causal)
    yal = loops.smha_forward(t["x"].tolist(), t["Wq"].tolist(), t["Wk"].tolist(), t["Wv"].tolist(), t["Wo"].tolist(),
                             lr, w.B, w.L, w.d, w.d_g, w.d_h, w.m, L_valid, causal)
    assert np.allclose(np.array(yal), ya, rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------------------------
# two-stage dynamic capacity (Eq. 15-16) and load-balancing loss (Eq. 42-44)
# ----------------------------------------------------------------------------------------------

def test_balance_loss_and_dynamic_capacity_worked_by_hand():
    # n = 3 experts, k = 1, three patches; gate columns chosen by hand
    p = np.array([[[0.7, 0.1, 0.5],
                   [0.2, 0.6, 0.3],
                   [0.1, 0.3, 0.2]]])                     # [B=1, n, m]
    cnt = np.array([4, 4, 4])
    counts = orc.patch_expert_counts(p[0], cnt, 1)
    assert counts.tolist() == [2, 1, 0]                    # patches 0 and 2 -> expert 0, patch 1 -> expert 1
    assert orc.dynamic_capacity(p, cnt, 1).tolist() == [2]
    # f = n/(k l) * counts = [2, 1, 0];  P = row means = [1.3/3, 1.1/3, 0.6/3];  L = 2*1.3/3 + 1.1/3
    assert orc.balance_loss(p, cnt, 1, alpha=1.0)[0] == pytest.approx((2 * 1.3 + 1.1) / 3, rel=1e-14)
    assert orc.balance_loss(p, cnt, 1, alpha=0.01)[0] == pytest.approx(0.01 * (2 * 1.3 + 1.1) / 3, rel=1e-14)
    # k = 2: patch 0 -> {0,1}, patch 1 -> {1,2}, patch 2 -> {0,1}: counts [2,3,1], c = 3
    assert orc.patch_expert_counts(p[0], cnt, 2).tolist() == [2, 3, 1]
    assert orc.dynamic_capacity(p, cnt, 2).tolist() == [3]


def test_balance_loss_properties():
    w = gen.tiny(B=4, n=5, k=2, m=6, c=3)
    t = _inputs(w, ("mlp",))
    Wr = _boost_router(gen.normal(3, 9, (w.d, w.n)), 2.0)
    for L_valid in (24, 19):
        p_samp, p_patch, _, _, cnt = orc.router_probs(t["x"], Wr, w.m, L_valid)
        l = int((cnt > 0).sum())
        for b in range(w.B):
            counts = orc.patch_expert_counts(p_patch[b], cnt, w.k)
            assert counts.sum() == w.k * l and counts.max() <= l       # every real patch picks exactly k experts
        # sum_i f_i = n and sum_i P_i = 1, so a uniform gate gives exactly alpha (the loss's minimum over balanced loads)
        uniform = np.full_like(p_patch, 1.0 / w.n)
        assert np.allclose(orc.balance_loss(uniform, cnt, w.k, 2.5), 2.5, rtol=1e-13)
        # all the mass on one expert for every patch: f = [n/k, ...] on k experts, P = e_0 -> alpha * n / k
        one = np.zeros_like(p_patch)
        one[:, 0, :] = 1.0
        assert np.allclose(orc.balance_loss(one, cnt, w.k, 1.0), w.n / w.k, rtol=1e-13)
        c_dyn = orc.dynamic_capacity(p_patch, cnt, w.k)
        assert np.all(c_dyn >= -(-w.k * l // w.n)) and np.all(c_dyn <= l)   # pigeonhole bound and at most every patch


def test_dynamic_capacity_limits_the_patches_per_expert():
    w = gen.tiny(B=5, n=4, k=2, m=6, c=6)
    t = _inputs(w, ("mlp",))
    Wr = _boost_router(t["Wr"], 30.0)
    r_fix = orc.route(t["x"], Wr, w.k, w.m, w.c)
    r_dyn = orc.route(t["x"], Wr, w.k, w.m, w.c, dynamic_c=True)
    _, p_patch, _, _, cnt = orc.router_probs(t["x"], Wr, w.m, 24)
    c_dyn = orc.dynamic_capacity(p_patch, cnt, w.k)
    assert np.array_equal(r_fix.expert_idx, r_dyn.expert_idx)
    for b in range(w.B):
        for s in range(w.k):
            got = r_dyn.patch_idx[b, s]
            assert (got >= 0).sum() == min(w.c, c_dyn[b])
            # the dynamic selection is the head of the fixed one in gate order: same top patches, fewer of them
            i = r_dyn.expert_idx[b, s]
            best = np.argsort(-p_patch[b, i], kind="stable")[:(got >= 0).sum()]
            assert sorted(best.tolist()) == got[got >= 0].tolist()
    assert (c_dyn < w.c).any()          # the case really exercises a smaller capacity


@pytest.mark.parametrize("L_valid", [24, 19])
def test_balance_loss_backward_matches_finite_differences(L_valid):
    w = gen.tiny(B=3, n=5, k=2, m=6, c=3, d=8)
    x = gen.make_x(w).f64
    Wr = gen.normal(5, 4, (w.d, w.n)) * 0.8
    dloss = np.array([0.5, -1.25, 2.0])
    alpha = 0.3
    dx, dWr = orc.balance_loss_backward(x, Wr, w.m, L_valid, w.k, alpha, dloss)

    def loss(x_, Wr_):
        _, pp, _, _, cnt = orc.router_probs(x_, Wr_, w.m, L_valid)
        return float(np.dot(dloss, orc.balance_loss(pp, cnt, w.k, alpha)))

    eps = 1e-6
    for which, grad, arr in (("x", dx, x), ("Wr", dWr, Wr)):
        for trial in range(3):
            v = gen.normal(400 + trial, 0 if which == "x" else 1, arr.shape)
            if which == "x":
                v[:, L_valid:] = 0.0
            fd = (loss(x + eps * v, Wr) - loss(x - eps * v, Wr)) / (2 * eps) if which == "x" else \
                (loss(x, Wr + eps * v) - loss(x, Wr - eps * v)) / (2 * eps)
            an = float(np.sum(grad * v))
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (which, fd, an)
    assert np.all(dx[:, L_valid:] == 0.0)


# ----------------------------------------------------------------------------------------------
# backward: central finite differences with the selection frozen
# ----------------------------------------------------------------------------------------------

@pytest.mark.parametrize("act,L_valid,use_gate", [("silu", 24, True), ("gelu_erf", 21, True), ("gelu_tanh", 24, False)])
def test_backward_matches_finite_differences(act, L_valid, use_gate):
    w = gen.tiny(B=2, L_valid=L_valid, act=act, d=8, d_ff=16)
    t = _inputs(w, ("mlp",))
    x, W1, W2 = t["x"], t["W1"], t["W2"]
    Wr = _boost_router(t["Wr"], 10.0)
    r = orc.route(x, Wr, w.k, w.m, w.c, L_valid=L_valid, use_gate=use_gate)
    dy = gen.normal(7, 1, x.shape)
    dy[:, L_valid:] = 0.0
    dx, dW1, dW2, dWr, _ = orc.mlp_backward(x, W1, W2, Wr, r, dy, act, True, use_gate)

    def loss(x_, W1_, W2_, Wr_):
        rr = orc.with_selection(x_, Wr_, r.expert_idx, r.patch_idx, w.m, L_valid, use_gate)
        return float(np.sum(orc.mlp_forward(x_, W1_, W2_, rr, act) * dy))

    eps = 1e-5
    for which, grad, arr in (("x", dx, x), ("W1", dW1, W1), ("W2", dW2, W2), ("Wr", dWr, Wr)):
        for trial in range(3):
            v = gen.normal(100 + trial, {"x": 0, "W1": 1, "W2": 2, "Wr": 3}[which], arr.shape)
            if which == "x":
                v[:, L_valid:] = 0.0
            args_p = dict(x_=x, W1_=W1, W2_=W2, Wr_=Wr)
            args_m = dict(args_p)
            key = {"x": "x_", "W1": "W1_", "W2": "W2_", "Wr": "Wr_"}[which]
            args_p[key] = arr + eps * v
            args_m[key] = arr - eps * v
            fd = (loss(**args_p) - loss(**args_m)) / (2 * eps)
            an = float(np.sum(grad * v))
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (which, fd, an)
    if not use_gate:
        assert np.all(dWr == 0.0)


@pytest.mark.parametrize("causal,L_valid,use_gate,H", [(False, 24, True, 4), (True, 24, True, 4), (False, 21, True, 8),
                                                        (True, 21, False, 4)])
def test_smha_backward_matches_finite_differences(causal, L_valid, use_gate, H):
    w = gen.tiny(B=2, L_valid=L_valid, d=8, H=H, d_h=2)
    t = _inputs(w, ("att",))
    x, Wq, Wk, Wv, Wo = t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"]
    Wr = _boost_router(t["Wra"], 10.0)
    r = orc.route(x, Wr, w.k, w.m, w.c, L_valid=L_valid, use_gate=use_gate)
    dy = gen.normal(9, 1, x.shape)
    dy[:, L_valid:] = 0.0
    dx, dWq, dWk, dWv, dWo, dWr, _ = orc.smha_backward(x, Wq, Wk, Wv, Wo, Wr, r, dy, w.d_h, causal, True, use_gate)

    def loss(**a):
        rr = orc.with_selection(a["x"], a["Wr"], r.expert_idx, r.patch_idx, w.m, L_valid, use_gate)
        return float(np.sum(orc.smha_forward(a["x"], a["Wq"], a["Wk"], a["Wv"], a["Wo"], rr, w.d_h, causal) * dy))

    base = dict(x=x, Wq=Wq, Wk=Wk, Wv=Wv, Wo=Wo, Wr=Wr)
    grads = dict(x=dx, Wq=dWq, Wk=dWk, Wv=dWv, Wo=dWo, Wr=dWr)
    eps = 1e-5
    for si, which in enumerate(base):
        for trial in range(2):
            v = gen.normal(200 + trial, si, base[which].shape)
            if which == "x":
                v[:, L_valid:] = 0.0
            ap, am = dict(base), dict(base)
            ap[which] = base[which] + eps * v
            am[which] = base[which] - eps * v
            fd = (loss(**ap) - loss(**am)) / (2 * eps)
            an = float(np.sum(grads[which] * v))
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (which, fd, an)
    if not use_gate:
        assert np.all(dWr == 0.0)


def test_smha_backward_full_selection_equals_dense_attention_gradient():
    """k = n, c = m, unit weights: the layer is textbook multi-head attention (Eq. 8-11), so its input gradient
    must equal the gradient of that dense attention, derived here independently (per-head softmax backward)."""
    w = gen.tiny(B=2, k=4, c=6, d=8, H=4, d_h=2)
    t = _inputs(w, ("att",))
    x = t["x"]
    r = orc.route(x, t["Wra"], w.k, w.m, w.c, use_gate=False)
    dy = gen.normal(13, 2, x.shape)
    dx, dWq, dWk, dWv, dWo, dWr, _ = orc.smha_backward(x, t["Wq"], t["Wk"], t["Wv"], t["Wo"], t["Wra"], r, dy, w.d_h,
                                                       causal=True, residual=False, use_gate=False)
    WQ = np.concatenate(list(t["Wq"]), axis=1)
    WK = np.concatenate(list(t["Wk"]), axis=1)
    WV = np.concatenate(list(t["Wv"]), axis=1)
    WO = np.concatenate(list(t["Wo"]), axis=0)
    L = x.shape[1]
    mask = np.tril(np.ones((L, L), dtype=bool))
    dx_ref = np.zeros_like(x)
    dWO = np.zeros_like(WO)
    for b in range(x.shape[0]):
        q, k_, v = x[b] @ WQ, x[b] @ WK, x[b] @ WV
        do = dy[b] @ WO.T
        dq, dk, dv = np.zeros_like(q), np.zeros_like(k_), np.zeros_like(v)
        o = np.zeros_like(q)
        for hd in range(w.H):
            sl = slice(hd * w.d_h, (hd + 1) * w.d_h)
            sc = np.where(mask, q[:, sl] @ k_[:, sl].T / np.sqrt(w.d_h), -np.inf)
            P = np.exp(sc - sc.max(1, keepdims=True))
            P /= P.sum(1, keepdims=True)
            o[:, sl] = P @ v[:, sl]
            dP = do[:, sl] @ v[:, sl].T
            dS = P * (dP - (dP * P).sum(1, keepdims=True))
            dv[:, sl] = P.T @ do[:, sl]
            dq[:, sl] = dS @ k_[:, sl] / np.sqrt(w.d_h)
            dk[:, sl] = dS.T @ q[:, sl] / np.sqrt(w.d_h)
        dWO += o.T @ dy[b]
        dx_ref[b] = dq @ WQ.T + dk @ WK.T + dv @ WV.T
    assert np.allclose(dx, dx_ref, rtol=1e-10, atol=1e-12)
    assert np.allclose(np.concatenate(list(dWo), axis=0), dWO, rtol=1e-10, atol=1e-12)
    assert np.all(dWr == 0.0)


def test_rope_is_a_rotation_by_relative_position():
    """Eq. 32 against the complex form of rotary embeddings: with z_i = x_{2i} + j x_{2i+1}, RoPE multiplies z_i by
    exp(j t theta_i), so <RoPE(q, t), RoPE(k, s)> = Re sum_i q_i conj(k_i) exp(j (t - s) theta_i) (a function of t - s
    only), norms are kept, the constant part is untouched and the inverse undoes it."""
    d_h, d_r = 8, 6
    q = gen.normal(21, 0, (5, 2 * d_h))
    k = gen.normal(21, 1, (5, 2 * d_h))
    pos_q = np.array([0, 3, 7, 20, 21])
    pos_k = np.array([5, 3, 9, 2, 40])
    rq, rk = orc.rope(q, pos_q, d_h, d_r), orc.rope(k, pos_k, d_h, d_r)
    theta = 10000.0 ** (-2.0 * np.arange(d_r // 2) / d_r)
    for hd in range(2):
        c0 = hd * d_h
        assert np.array_equal(rq[:, c0:c0 + d_h - d_r], q[:, c0:c0 + d_h - d_r])
        zq = q[:, c0 + d_h - d_r:c0 + d_h:2] + 1j * q[:, c0 + d_h - d_r + 1:c0 + d_h:2]
        zk = k[:, c0 + d_h - d_r:c0 + d_h:2] + 1j * k[:, c0 + d_h - d_r + 1:c0 + d_h:2]
        for a in range(5):
            for b in range(5):
                want = np.real(np.sum(zq[a] * np.conj(zk[b]) * np.exp(1j * (pos_q[a] - pos_k[b]) * theta)))
                want += q[a, c0:c0 + d_h - d_r] @ k[b, c0:c0 + d_h - d_r]
                got = rq[a, c0:c0 + d_h] @ rk[b, c0:c0 + d_h]
                assert got == pytest.approx(want, rel=1e-12, abs=1e-12)
    assert np.allclose(np.linalg.norm(rq, axis=1), np.linalg.norm(q, axis=1), rtol=1e-13)
    assert np.allclose(orc.rope(rq, pos_q, d_h, d_r, inverse=True), q, rtol=1e-12, atol=1e-13)
    assert orc.rope(q, pos_q, d_h, 0) is q


def test_smha_with_rope_changes_the_output_and_backward_matches_finite_differences():
    w = gen.tiny(B=2, L_valid=24, d=8, H=4, d_h=4)
    t = _inputs(w, ("att",))
    x, Wq, Wk, Wv, Wo = t["x"], t["Wq"], t["Wk"], t["Wv"], t["Wo"]
    Wr = _boost_router(t["Wra"], 10.0)
    r = orc.route(x, Wr, w.k, w.m, w.c)
    y0 = orc.smha_forward(x, Wq, Wk, Wv, Wo, r, w.d_h, True, d_rope=0)
    y1 = orc.smha_forward(x, Wq, Wk, Wv, Wo, r, w.d_h, True, d_rope=2)
    assert not np.allclose(y0, y1)
    # backward: finite differences with the rotary part on
    dy = gen.normal(9, 1, x.shape)
    dx, dWq, dWk, dWv, dWo, dWr, _ = orc.smha_backward(x, Wq, Wk, Wv, Wo, Wr, r, dy, w.d_h, True, True, True, d_rope=2)

    def loss(**a):
        rr = orc.with_selection(a["x"], a["Wr"], r.expert_idx, r.patch_idx, w.m, 24, True)
        return float(np.sum(orc.smha_forward(a["x"], a["Wq"], a["Wk"], a["Wv"], a["Wo"], rr, w.d_h, True, d_rope=2) * dy))

    base = dict(x=x, Wq=Wq, Wk=Wk, Wv=Wv, Wo=Wo, Wr=Wr)
    grads = dict(x=dx, Wq=dWq, Wk=dWk, Wv=dWv, Wo=dWo, Wr=dWr)
    for si, which in enumerate(base):
        v = gen.normal(300, si, base[which].shape)
        ap, am = dict(base), dict(base)
        ap[which] = base[which] + 1e-5 * v
        am[which] = base[which] - 1e-5 * v
        fd = (loss(**ap) - loss(**am)) / 2e-5
        an = float(np.sum(grads[which] * v))
        assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)), (which, fd, an)


# ----------------------------------------------------------------------------------------------
# planted mistakes: the pins above must notice a wrong oracle
# ----------------------------------------------------------------------------------------------

def test_planted_mistakes_are_caught(monkeypatch):
    w = gen.tiny(k=4, c=6)
    t = _inputs(w)
    A_I = np.concatenate(list(t["W1"]), axis=1)
    A_O = np.concatenate(list(t["W2"]), axis=0)
    dense = (orc.act_fn(t["x"] @ A_I, "silu") @ A_O)
    r = orc.route(t["x"], t["Wr"], w.k, w.m, w.c, use_gate=False)

    def dense_ok():
        y = orc.mlp_forward(t["x"], t["W1"], t["W2"], r, "silu")
        return np.allclose(y - t["x"], dense, rtol=1e-12, atol=1e-13)

    assert dense_ok()
    # (1a) the activation applied twice to the hidden layer
    real_act = orc.act_fn
    monkeypatch.setattr(orc, "act_fn", lambda h, a: real_act(real_act(h, a), a))
    assert not dense_ok()
    monkeypatch.setattr(orc, "act_fn", real_act)
    # (1b) an activation after the second layer of every expert (the misprint in Eq. 39): the sum of the per-expert
    # phi(z_i) is not the dense layer (Eq. 5-7 put phi, if any, after the sum)
    y_phi = t["x"].copy()
    for b in range(w.B):
        for s, i in enumerate(r.expert_idx[b]):
            for j in r.patch_idx[b, s]:
                rows = slice(j * w.l_p, (j + 1) * w.l_p)
                y_phi[b, rows] += orc.act_fn(orc.act_fn(t["x"][b, rows] @ t["W1"][i], "silu") @ t["W2"][i], "silu")
    assert not np.allclose(y_phi - t["x"], dense, rtol=1e-9, atol=1e-10)
    # (2) experts' weight slices swapped between layers
    y = orc.mlp_forward(t["x"], t["W1"], t["W2"][::-1], r, "silu")
    assert not np.allclose(y - t["x"], dense, rtol=1e-9, atol=1e-10)
    # (3) softmax over patches instead of experts changes the selection of some sample
    w2 = gen.tiny(B=6)
    x2 = gen.make_x(w2).f64
    Wr2 = _boost_router(gen.make_router(w2).f64)
    good = orc.route(x2, Wr2, w2.k, w2.m, w2.c)
    real_sm = orc.softmax
    p_samp, p_patch, pool, samp, cnt = orc.router_probs(x2, Wr2, w2.m, w2.L)
    logits = np.einsum("bjd,dn->bnj", pool, Wr2)
    wrong = real_sm(logits, axis=2)              # normalised over patches: not Eq. 14
    _, pidx, _, _ = orc.select(p_samp, wrong, cnt, w2.k, w2.c)
    assert not np.array_equal(pidx, good.patch_idx)
