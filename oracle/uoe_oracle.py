"""CPU float64 oracle for the Union-of-Experts routed hot path.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer computes,
written from the paper's equations so that a reader can check it by eye.  It is used by the
tests, by the smoke check and by the benchmark's CPU-baseline leg; the product (the CUDA
library and its Python binding) never imports it and shares no code with it.

Everything is numpy float64 with explicit loops over samples, experts and patches.  No
blocking, fusion or reordering beyond what the equations state.

Notation (paper, Section III): b samples, l tokens, d channels, n experts, k experts per sample,
m patches per sample of l_p tokens, c patches per expert, l_a = c*l_p, d_e expert hidden width.

Functions and the passages they follow
  router_probs     Eq. 12-14 (patch gate) and Eq. 21 (sample gate)
  select           Eq. 17 (top-c patches, re-sorted), Eq. 22-23 (top-k experts, per-expert lists),
                   combined as in Fig. 3 / the "superposition" paragraph of Section III-B
  route            the two above + gate weights + buffer offsets
  patch_expert_counts, dynamic_capacity   Eq. 15-16 (two-stage routing: c = largest number of patches any
                   expert receives when every patch goes to its k best experts)
  balance_loss     Eq. 42-44 (sequence-wise load-balancing loss over the patches of one sample)
  balance_loss_backward   its gradient w.r.t. x and W_r (through P_i; pinned by finite differences)
  mlp_forward      Eq. 18-20 and Eq. 37-40 (UoME), decomposition Eq. 1-7
  smha_forward     Eq. 27-30, 33-36 (SMHA), masks Eq. 41 and Fig. 4, decomposition Eq. 8-11
  mlp_backward     derivative of mlp_forward with the selection held constant (no paper text;
                   pinned by finite differences)
  smha_backward    derivative of smha_forward with the selection held constant (no paper text;
                   pinned by finite differences)

Readings where the paper is silent or garbled are listed in the repository's design notes; the
ones that matter here: the router is one linear map W_r[d, n] applied to the mean token of a
patch (patch gate) or of the sample (sample gate); the combine weight is
P_samp[b,i] * P_patch[b,i,j] when gating is on, 1 otherwise (Eq. 20 literal); no activation
after the second linear layer (Eq. 5-7, against the misprint in Eq. 39); RoPE (Eq. 32; Eq. 31 is misprinted)
is optional: the last d_r channels of every head of q and k are rotated in interleaved pairs by the
token's position in its sample, base 10000 (the RoFormer form the paper cites).

Parity unpinned: the *choice* of router form and gate formula cannot be pinned to the paper
(it prints no worked example); everything else is pinned by tests/test_oracle_*.py.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
from scipy.special import erf as _erf

# ----------------------------------------------------------------------------------------------
# activations (Eq. 1: phi applied per column slice)
# ----------------------------------------------------------------------------------------------

_SQRT_2_OVER_PI = math.sqrt(2.0 / math.pi)


def act_fn(h: np.ndarray, act: str) -> np.ndarray:
    if act == "gelu_erf":
        return 0.5 * h * (1.0 + _erf(h / math.sqrt(2.0)))
    if act == "gelu_tanh":
        return 0.5 * h * (1.0 + np.tanh(_SQRT_2_OVER_PI * (h + 0.044715 * h ** 3)))
    if act == "silu":
        return h / (1.0 + np.exp(-h))
    if act == "identity":
        return h.copy()
    raise ValueError(act)


def act_grad(h: np.ndarray, act: str) -> np.ndarray:
    if act == "gelu_erf":
        cdf = 0.5 * (1.0 + _erf(h / math.sqrt(2.0)))
        pdf = np.exp(-0.5 * h * h) / math.sqrt(2.0 * math.pi)
        return cdf + h * pdf
    if act == "gelu_tanh":
        u = _SQRT_2_OVER_PI * (h + 0.044715 * h ** 3)
        t = np.tanh(u)
        du = _SQRT_2_OVER_PI * (1.0 + 3.0 * 0.044715 * h * h)
        return 0.5 * (1.0 + t) + 0.5 * h * (1.0 - t * t) * du
    if act == "silu":
        s = 1.0 / (1.0 + np.exp(-h))
        return s * (1.0 + h * (1.0 - s))
    if act == "identity":
        return np.ones_like(h)
    raise ValueError(act)


def softmax(v: np.ndarray, axis: int) -> np.ndarray:
    e = np.exp(v - np.max(v, axis=axis, keepdims=True))
    return e / np.sum(e, axis=axis, keepdims=True)


# ----------------------------------------------------------------------------------------------
# routing
# ----------------------------------------------------------------------------------------------

@dataclass
class Routing:
    expert_idx: np.ndarray      # [B, k]    int, ascending per sample               (Eq. 22)
    patch_idx: np.ndarray       # [B, k, c] int, ascending per (sample, expert), -1 = unused slot (Eq. 17)
    gate: np.ndarray            # [B, k, c] combine weight of each selected patch
    p_samp: np.ndarray          # [B, n]    sample gate                             (Eq. 21)
    p_patch: np.ndarray         # [B, n, m] patch gate, softmax over experts        (Eq. 14)
    load: np.ndarray            # [n]       samples routed to each expert           (Eq. 23)
    offsets: np.ndarray         # [n+1]     first row of each expert's region in the routed buffers
    expert_margin: np.ndarray   # [B]       relative gap between the last selected and first rejected expert
    patch_margin: np.ndarray    # [B, k]    same for the patch selection of each selected expert
    m: int
    l_p: int
    L_valid: int


def patch_valid_counts(L: int, m: int, L_valid: int) -> np.ndarray:
    """Number of real (non-pad) tokens in each patch (Eq. 12 splits l tokens into m patches of l_p)."""
    l_p = L // m
    return np.array([max(0, min((j + 1) * l_p, L_valid) - j * l_p) for j in range(m)], dtype=np.int64)


def router_probs(x: np.ndarray, W_r: np.ndarray, m: int, L_valid: int):
    """Patch gate (Eq. 13-14) and sample gate (Eq. 21).

    FFN_B is the linear map W_r applied per token and FFN_A averages the tokens of a patch, so the
    patch score is mean_{t in patch j} x[t] @ W_r; the sample score is the same map applied to
    the mean over all real tokens of the sample.  Pad tokens take no part in either mean.
    """
    B, L, d = x.shape
    n = W_r.shape[1]
    l_p = L // m
    cnt = patch_valid_counts(L, m, L_valid)
    pool = np.zeros((B, m, d))
    samp = np.zeros((B, d))
    p_patch = np.zeros((B, n, m))
    p_samp = np.zeros((B, n))
    for b in range(B):
        for j in range(m):
            if cnt[j] > 0:
                pool[b, j] = x[b, j * l_p: j * l_p + cnt[j]].mean(axis=0)
            g_prime = pool[b, j] @ W_r                        # Eq. 13, column j of g'
            p_patch[b, :, j] = softmax(g_prime, axis=0)       # Eq. 14: over the n experts
        samp[b] = x[b, :L_valid].mean(axis=0)
        p_samp[b] = softmax(samp[b] @ W_r, axis=0)            # Eq. 21
    return p_samp, p_patch, pool, samp, cnt


def _top(values: np.ndarray, candidates: np.ndarray, count: int):
    """The `count` candidates with the largest values; ties go to the lower index; result ascending.

    Also returns the relative margin between the last one taken and the first one left out.
    """
    order = candidates[np.argsort(-values[candidates], kind="stable")]
    take = order[:count]
    if count < len(order) and count > 0:
        v_in, v_out = values[take[-1]], values[order[count]]
        margin = (v_in - v_out) / abs(v_in) if v_in != 0 else 0.0
    else:
        margin = math.inf
    return np.sort(take), margin


def patch_expert_counts(p_patch_b: np.ndarray, cnt: np.ndarray, k: int) -> np.ndarray:
    """Eq. 15 and the inner sum of Eq. 16 / Eq. 43 for one sample: every patch that holds a real token goes to
    its k experts with the highest gate (ties: lower index); returns how many patches each expert receives."""
    n, m = p_patch_b.shape
    counts = np.zeros(n, dtype=np.int64)
    for j in range(m):
        if cnt[j] == 0:
            continue
        chosen, _ = _top(p_patch_b[:, j], np.arange(n), k)        # id'_j, Eq. 15
        counts[chosen] += 1
    return counts


def dynamic_capacity(p_patch: np.ndarray, cnt: np.ndarray, k: int) -> np.ndarray:
    """Eq. 16 per sample: c = max over experts of the number of patches routed to it in the first stage."""
    return np.array([patch_expert_counts(p_patch[b], cnt, k).max() for b in range(p_patch.shape[0])], dtype=np.int64)


def balance_loss(p_patch: np.ndarray, cnt: np.ndarray, k: int, alpha: float = 1.0) -> np.ndarray:
    """Eq. 42-44 per sample, the routed units t being the sample's patches that hold a real token (l of them):
    f_i = n / (k l) * #{t : expert i among the k best of t},  P_i = mean_t g_{i,t},  L = alpha * sum_i f_i P_i."""
    B, n, m = p_patch.shape
    elig = np.nonzero(cnt > 0)[0]
    l = len(elig)
    out = np.zeros(B)
    for b in range(B):
        f = n / (k * l) * patch_expert_counts(p_patch[b], cnt, k)        # Eq. 43
        P = p_patch[b][:, elig].mean(axis=1)                               # Eq. 44
        out[b] = alpha * float(np.sum(f * P))                              # Eq. 42
    return out


def balance_loss_backward(x: np.ndarray, W_r: np.ndarray, m: int, L_valid: int, k: int, alpha: float,
                          dloss: np.ndarray):
    """Gradient of sum_b dloss[b] * L_b (Eq. 42-44) with respect to x and W_r.  f_i (Eq. 43) counts top-k memberships
    and is piecewise constant, so the gradient flows through P_i (Eq. 44) only:
    dL_b/dg_{i,t} = alpha f_i / l on the real patches, then the softmax Jacobian of Eq. 14 and the mean-pooled
    linear router of Eq. 13."""
    B, L, d = x.shape
    n = W_r.shape[1]
    l_p = L // m
    p_samp, p_patch, pool, samp, cnt = router_probs(x, W_r, m, L_valid)
    l = int((cnt > 0).sum())
    dx = np.zeros_like(x)
    dW_r = np.zeros_like(W_r)
    for b in range(B):
        f = n / (k * l) * patch_expert_counts(p_patch[b], cnt, k)
        for j in range(m):
            if cnt[j] == 0:
                continue
            dg = dloss[b] * alpha * f / l                                  # d/dg_{:,j}
            pj = p_patch[b, :, j]
            dlogit = pj * (dg - np.dot(pj, dg))                            # softmax Jacobian, Eq. 14
            dW_r += np.outer(pool[b, j], dlogit)
            dx[b, j * l_p: j * l_p + cnt[j]] += (W_r @ dlogit)[None, :] / cnt[j]
    return dx, dW_r


def select(p_samp: np.ndarray, p_patch: np.ndarray, cnt: np.ndarray, k: int, c: int, dynamic_c: bool = False):
    """Top-k experts per sample (Eq. 22), then top-c patches for each chosen expert (Eq. 17), indices
    re-sorted ascending (text below Eq. 17).  With dynamic_c the number of patches
    per expert is the sample's own c of Eq. 16, capped by the given c (the width of the index array)."""
    B, n = p_samp.shape
    m = p_patch.shape[2]
    eligible = np.nonzero(cnt > 0)[0]
    expert_idx = np.zeros((B, k), dtype=np.int64)
    patch_idx = -np.ones((B, k, c), dtype=np.int64)
    e_margin = np.zeros(B)
    p_margin = np.zeros((B, k))
    for b in range(B):
        expert_idx[b], e_margin[b] = _top(p_samp[b], np.arange(n), k)
        c_b = min(c, int(patch_expert_counts(p_patch[b], cnt, k).max())) if dynamic_c else c
        for s, i in enumerate(expert_idx[b]):
            take, p_margin[b, s] = _top(p_patch[b, i], eligible, min(c_b, len(eligible)))
            patch_idx[b, s, :len(take)] = take
    return expert_idx, patch_idx, e_margin, p_margin


def gates(p_samp, p_patch, expert_idx, patch_idx, use_gate: bool) -> np.ndarray:
    """Combine weight of every selected (sample, expert, patch): P_samp * P_patch, or 1 (Eq. 20 literal)."""
    B, k, c = patch_idx.shape
    g = np.zeros((B, k, c))
    for b in range(B):
        for s in range(k):
            i = expert_idx[b, s]
            for u in range(c):
                j = patch_idx[b, s, u]
                if j >= 0:
                    g[b, s, u] = p_samp[b, i] * p_patch[b, i, j] if use_gate else 1.0
    return g


def buffer_offsets(expert_idx: np.ndarray, n: int, rows_per_pair: int, row_align: int):
    """Per-expert sample lists (Eq. 23) as row offsets: expert i's region starts at offsets[i], holds
    load[i]*rows_per_pair rows (samples ascending) and is padded up to a multiple of row_align."""
    load = np.zeros(n, dtype=np.int64)
    for b in range(expert_idx.shape[0]):
        for i in expert_idx[b]:
            load[i] += 1
    offsets = np.zeros(n + 1, dtype=np.int64)
    for i in range(n):
        rows = load[i] * rows_per_pair
        offsets[i + 1] = offsets[i] + ((rows + row_align - 1) // row_align) * row_align
    return load, offsets


def route(x, W_r, k: int, m: int, c: int, L_valid: int | None = None, use_gate: bool = True,
          row_align: int = 128, dynamic_c: bool = False) -> Routing:
    B, L, d = x.shape
    n = W_r.shape[1]
    L_valid = L if L_valid is None else L_valid
    p_samp, p_patch, _, _, cnt = router_probs(x, W_r, m, L_valid)
    expert_idx, patch_idx, e_margin, p_margin = select(p_samp, p_patch, cnt, k, c, dynamic_c)
    g = gates(p_samp, p_patch, expert_idx, patch_idx, use_gate)
    load, offsets = buffer_offsets(expert_idx, n, c * (L // m), row_align)
    return Routing(expert_idx, patch_idx, g, p_samp, p_patch, load, offsets, e_margin, p_margin,
                   m, L // m, L_valid)


def with_selection(x, W_r, expert_idx, patch_idx, m: int, L_valid: int, use_gate: bool = True,
                   row_align: int = 128) -> Routing:
    """Routing whose selection is given (for example the GPU's at a near-tie, or a frozen one for
    finite differences) and whose probabilities and gates are recomputed from x and W_r."""
    B, L, d = x.shape
    n = W_r.shape[1]
    p_samp, p_patch, _, _, cnt = router_probs(x, W_r, m, L_valid)
    g = gates(p_samp, p_patch, expert_idx, patch_idx, use_gate)
    load, offsets = buffer_offsets(expert_idx, n, patch_idx.shape[2] * (L // m), row_align)
    return Routing(np.asarray(expert_idx), np.asarray(patch_idx), g, p_samp, p_patch, load, offsets,
                   np.full(B, math.inf), np.full(patch_idx.shape[:2], math.inf), m, L // m, L_valid)


def buffer_row(r: Routing, b: int, s: int) -> int:
    """First buffer row of (sample b, its s-th selected expert): samples ascending inside the expert."""
    i = r.expert_idx[b, s]
    rank = sum(1 for bb in range(b) if i in r.expert_idx[bb])
    return int(r.offsets[i] + rank * r.patch_idx.shape[2] * r.l_p)


# ----------------------------------------------------------------------------------------------
# UoME forward (Eq. 37-40 with the selection of Eq. 17/22 and the index-add of Eq. 20)
# ----------------------------------------------------------------------------------------------

def mlp_forward(x, W1, W2, r: Routing, act: str = "silu", residual: bool = True, b1=None, b2=None,
                return_parts: bool = False):
    """y[b,t] = x[b,t] + sum over the (expert i, patch j) pairs that selected token t of
    gate[b,i,j] * ( phi(x[b,t] @ A^I_i + b1_i) @ A^O_i + b2_i ).   Pad rows and unselected rows: y = x."""
    B, L, d = x.shape
    y = x.copy() if residual else np.zeros_like(x)
    parts = {}
    for b in range(B):
        for s in range(r.expert_idx.shape[1]):
            i = r.expert_idx[b, s]
            for u in range(r.patch_idx.shape[2]):
                j = r.patch_idx[b, s, u]
                if j < 0:
                    continue
                t0, t1 = j * r.l_p, min((j + 1) * r.l_p, r.L_valid)
                h = x[b, t0:t1] @ W1[i]                      # Eq. 38: column slice of layer 1
                if b1 is not None:
                    h = h + b1[i]
                a = act_fn(h, act)
                z = a @ W2[i]                                # Eq. 39 without the misprinted phi
                if b2 is not None:
                    z = z + b2[i]
                y[b, t0:t1] += r.gate[b, s, u] * z           # Eq. 20 / 40: index-add
                if return_parts:
                    parts[(b, s, u)] = (h, a, z)
    return (y, parts) if return_parts else y


# ----------------------------------------------------------------------------------------------
# SMHA forward (Eq. 27-30, 33-36; masks Eq. 41, Fig. 4)
# ----------------------------------------------------------------------------------------------

def gathered_tokens(r: Routing, b: int, s: int) -> np.ndarray:
    """Token positions of the selected patches of (b, s), in ascending order (Eq. 18)."""
    toks = []
    for j in r.patch_idx[b, s]:
        if j >= 0:
            toks.extend(range(j * r.l_p, (j + 1) * r.l_p))
    return np.array(toks, dtype=np.int64)


def rope(t: np.ndarray, pos: np.ndarray, d_h: int, d_r: int, inverse: bool = False) -> np.ndarray:
    """Eq. 32: in every head of t [rows, heads*d_h] keep the first d_h - d_r channels (the constant part) and rotate
    the last d_r in pairs (2i, 2i+1) by the angle pos * 10000^(-2i/d_r); `inverse` rotates back."""
    if d_r == 0:
        return t
    out = t.copy()
    theta = 10000.0 ** (-2.0 * np.arange(d_r // 2) / d_r)
    ang = pos[:, None].astype(np.float64) * theta[None, :]
    if inverse:
        ang = -ang
    cs, sn = np.cos(ang), np.sin(ang)
    for hd in range(t.shape[1] // d_h):
        c0 = hd * d_h + (d_h - d_r)
        a, b = t[:, c0:c0 + d_r:2], t[:, c0 + 1:c0 + d_r:2]
        out[:, c0:c0 + d_r:2] = a * cs - b * sn
        out[:, c0 + 1:c0 + d_r:2] = a * sn + b * cs
    return out


def smha_forward(x, Wq, Wk, Wv, Wo, r: Routing, d_h: int, causal: bool, residual: bool = True,
                 return_lse: bool = False, d_rope: int = 0):
    """Each attention expert i owns the column slice W^{q,k,v}_i [d, d_g] and the row slice W^o_i
    [d_g, d] (Eq. 8-11); d_g = (heads per expert) * d_h.  Expert i of sample b attends only over the
    tokens of its selected patches."""
    B, L, d = x.shape
    d_g = Wq.shape[2]
    heads = d_g // d_h
    y = x.copy() if residual else np.zeros_like(x)
    full_causal = np.tril(np.ones((L, L), dtype=bool))
    pad_mask = np.arange(L) < r.L_valid                      # m^p: True = real token
    lse_out = {}
    for b in range(B):
        for s in range(r.expert_idx.shape[1]):
            i = r.expert_idx[b, s]
            tok = gathered_tokens(r, b, s)
            if len(tok) == 0:
                continue
            hp = x[b, tok]                                   # h' (Eq. 27)
            q, kk, v = hp @ Wq[i], hp @ Wk[i], hp @ Wv[i]    # Eq. 28-30
            q, kk = rope(q, tok, d_h, d_rope), rope(kk, tok, d_h, d_rope)      # Eq. 32, positions in the sample
            keep = np.broadcast_to(pad_mask[tok][None, :], (len(tok), len(tok))).copy()   # Eq. 41
            if causal:
                keep &= full_causal[np.ix_(tok, tok)]        # the mask indexed on both axes (Fig. 4)
            o = np.zeros((len(tok), d_g))
            for hd in range(heads):
                sl = slice(hd * d_h, (hd + 1) * d_h)
                sc = (q[:, sl] @ kk[:, sl].T) / math.sqrt(d_h)           # Eq. 33
                sc = np.where(keep, sc, -np.inf)
                mx = sc.max(axis=1, keepdims=True)
                e = np.exp(sc - mx)
                den = e.sum(axis=1, keepdims=True)
                o[:, sl] = (e / den) @ v[:, sl]                          # Eq. 34
                if return_lse:
                    lse_out[(b, s, hd)] = (mx + np.log(den))[:, 0]
            up = o @ Wo[i]                                   # Eq. 35
            # Eq. 36: index-add; gate is per patch, pad query rows are left as x
            for u, j in enumerate(r.patch_idx[b, s]):
                if j < 0:
                    continue
                t0, t1 = j * r.l_p, min((j + 1) * r.l_p, r.L_valid)
                y[b, t0:t1] += r.gate[b, s, u] * up[u * r.l_p: u * r.l_p + (t1 - t0)]
    return (y, lse_out) if return_lse else y


# ----------------------------------------------------------------------------------------------
# UoME backward (selection constant; gates differentiable when use_gate)
# ----------------------------------------------------------------------------------------------

def mlp_backward(x, W1, W2, W_r, r: Routing, dy, act: str = "silu", residual: bool = True,
                 use_gate: bool = True):
    """Gradients of sum(y * dy) for y = mlp_forward(x, ...) with expert_idx / patch_idx frozen.

    Returns dx [B,L,d], dW1 [n,d,d_e], dW2 [n,d_e,d], dW_r [d,n].
    """
    B, L, d = x.shape
    n = W_r.shape[1]
    m, l_p, L_valid = r.m, r.l_p, r.L_valid
    dx = dy.copy() if residual else np.zeros_like(dy)
    dx[:, L_valid:] = dy[:, L_valid:] if residual else 0.0
    dW1 = np.zeros_like(W1)
    dW2 = np.zeros_like(W2)
    dgate = np.zeros_like(r.gate)
    for b in range(B):
        for s in range(r.expert_idx.shape[1]):
            i = r.expert_idx[b, s]
            for u in range(r.patch_idx.shape[2]):
                j = r.patch_idx[b, s, u]
                if j < 0:
                    continue
                t0, t1 = j * l_p, min((j + 1) * l_p, L_valid)
                xp = x[b, t0:t1]
                h = xp @ W1[i]
                a = act_fn(h, act)
                z = a @ W2[i]
                g = r.gate[b, s, u]
                dyp = dy[b, t0:t1]
                dgate[b, s, u] = np.sum(dyp * z)
                dz = g * dyp
                dW2[i] += a.T @ dz
                da = dz @ W2[i].T
                dh = da * act_grad(h, act)
                dW1[i] += xp.T @ dh
                dx[b, t0:t1] += dh @ W1[i].T
    dW_r = np.zeros_like(W_r)
    if use_gate:
        p_samp, p_patch, pool, samp, cnt = router_probs(x, W_r, m, L_valid)
        for b in range(B):
            dP_samp = np.zeros(n)
            dP_patch = np.zeros((n, m))
            for s in range(r.expert_idx.shape[1]):
                i = r.expert_idx[b, s]
                for u in range(r.patch_idx.shape[2]):
                    j = r.patch_idx[b, s, u]
                    if j < 0:
                        continue
                    dP_samp[i] += dgate[b, s, u] * p_patch[b, i, j]
                    dP_patch[i, j] += dgate[b, s, u] * p_samp[b, i]
            # softmax Jacobians (over all n experts)
            dl_s = p_samp[b] * (dP_samp - np.dot(p_samp[b], dP_samp))
            dW_r += np.outer(samp[b], dl_s)
            dx[b, :L_valid] += (W_r @ dl_s)[None, :] / L_valid
            for j in range(m):
                if cnt[j] == 0:
                    continue
                pj = p_patch[b, :, j]
                dl_p = pj * (dP_patch[:, j] - np.dot(pj, dP_patch[:, j]))
                dW_r += np.outer(pool[b, j], dl_p)
                dx[b, j * l_p: j * l_p + cnt[j]] += (W_r @ dl_p)[None, :] / cnt[j]
    return dx, dW1, dW2, dW_r, dgate


# ----------------------------------------------------------------------------------------------
# SMHA backward (selection constant; gates differentiable when use_gate)
# ----------------------------------------------------------------------------------------------

def _gate_to_router_grads(x, W_r, r: Routing, dgate):
    """Chain rule from d(loss)/d(gate[b,s,u]) through gate = P_samp[b,i] * P_patch[b,i,j] and the two
    softmaxes (Eq. 14, 21) into W_r and x.  Returns (dW_r, dx_router)."""
    B, L, d = x.shape
    n = W_r.shape[1]
    m, l_p, L_valid = r.m, r.l_p, r.L_valid
    dW_r = np.zeros_like(W_r)
    dxr = np.zeros_like(x)
    p_samp, p_patch, pool, samp, cnt = router_probs(x, W_r, m, L_valid)
    for b in range(B):
        dP_samp = np.zeros(n)
        dP_patch = np.zeros((n, m))
        for s in range(r.expert_idx.shape[1]):
            i = r.expert_idx[b, s]
            for u in range(r.patch_idx.shape[2]):
                j = r.patch_idx[b, s, u]
                if j < 0:
                    continue
                dP_samp[i] += dgate[b, s, u] * p_patch[b, i, j]
                dP_patch[i, j] += dgate[b, s, u] * p_samp[b, i]
        dl_s = p_samp[b] * (dP_samp - np.dot(p_samp[b], dP_samp))          # softmax Jacobian, Eq. 21
        dW_r += np.outer(samp[b], dl_s)
        dxr[b, :L_valid] += (W_r @ dl_s)[None, :] / L_valid
        for j in range(m):
            if cnt[j] == 0:
                continue
            pj = p_patch[b, :, j]
            dl_p = pj * (dP_patch[:, j] - np.dot(pj, dP_patch[:, j]))      # softmax Jacobian, Eq. 14
            dW_r += np.outer(pool[b, j], dl_p)
            dxr[b, j * l_p: j * l_p + cnt[j]] += (W_r @ dl_p)[None, :] / cnt[j]
    return dW_r, dxr


def smha_backward(x, Wq, Wk, Wv, Wo, W_r, r: Routing, dy, d_h: int, causal: bool, residual: bool = True,
                  use_gate: bool = True, d_rope: int = 0):
    """Gradients of sum(y * dy) for y = smha_forward(x, ...) with expert_idx / patch_idx frozen.

    Per (sample b, chosen expert i), with h' the gathered tokens, P the masked softmax of Eq. 33 and
    o = P v (Eq. 34), u' = o W^o_i (Eq. 35), y += gate * u' on the real query rows (Eq. 36):
      du' = gate * dy (real query rows; pad query rows contribute nothing)
      dW^o_i += o^T du',  do = du' W^o_i^T
      dv = P^T do,  dP = do v^T,  dS = P * (dP - rowsum(dP * P)),  dq = dS k / sqrt(d_h),  dk = dS^T q / sqrt(d_h)
      dW^{q,k,v}_i += h'^T d{q,k,v},  dh' = dq W^q_i^T + dk W^k_i^T + dv W^v_i^T, index-added into dx
    Returns dx [B,L,d], dWq, dWk, dWv [n,d,d_g], dWo [n,d_g,d], dW_r [d,n], dgate [B,k,c].
    """
    B, L, d = x.shape
    d_g = Wq.shape[2]
    heads = d_g // d_h
    l_p, L_valid = r.l_p, r.L_valid
    dx = dy.copy() if residual else np.zeros_like(dy)
    dWq, dWk, dWv, dWo = np.zeros_like(Wq), np.zeros_like(Wk), np.zeros_like(Wv), np.zeros_like(Wo)
    dgate = np.zeros_like(r.gate)
    full_causal = np.tril(np.ones((L, L), dtype=bool))
    pad_mask = np.arange(L) < L_valid
    for b in range(B):
        for s in range(r.expert_idx.shape[1]):
            i = r.expert_idx[b, s]
            tok = gathered_tokens(r, b, s)
            if len(tok) == 0:
                continue
            la = len(tok)
            hp = x[b, tok]
            q, kk, v = hp @ Wq[i], hp @ Wk[i], hp @ Wv[i]
            q, kk = rope(q, tok, d_h, d_rope), rope(kk, tok, d_h, d_rope)
            keep = np.broadcast_to(pad_mask[tok][None, :], (la, la)).copy()
            if causal:
                keep &= full_causal[np.ix_(tok, tok)]
            P = np.zeros((heads, la, la))
            o = np.zeros((la, d_g))
            for hd in range(heads):
                sl = slice(hd * d_h, (hd + 1) * d_h)
                sc = np.where(keep, (q[:, sl] @ kk[:, sl].T) / math.sqrt(d_h), -np.inf)
                e = np.exp(sc - sc.max(axis=1, keepdims=True))
                P[hd] = e / e.sum(axis=1, keepdims=True)
                o[:, sl] = P[hd] @ v[:, sl]
            up = o @ Wo[i]
            dup = np.zeros((la, d))
            row = 0
            for u, j in enumerate(r.patch_idx[b, s]):
                if j < 0:
                    continue
                t0, t1 = j * l_p, min((j + 1) * l_p, L_valid)
                rows = slice(row, row + (t1 - t0))
                dgate[b, s, u] = np.sum(dy[b, t0:t1] * up[rows])
                dup[rows] = r.gate[b, s, u] * dy[b, t0:t1]
                row += l_p
            dWo[i] += o.T @ dup
            do = dup @ Wo[i].T
            dq, dk, dv = np.zeros_like(q), np.zeros_like(kk), np.zeros_like(v)
            for hd in range(heads):
                sl = slice(hd * d_h, (hd + 1) * d_h)
                dv[:, sl] = P[hd].T @ do[:, sl]
                dP = do[:, sl] @ v[:, sl].T
                dS = P[hd] * (dP - np.sum(dP * P[hd], axis=1, keepdims=True))
                dq[:, sl] = dS @ kk[:, sl] / math.sqrt(d_h)
                dk[:, sl] = dS.T @ q[:, sl] / math.sqrt(d_h)
            # a rotation is orthogonal: the gradient w.r.t. the unrotated q, k is the gradient rotated back
            dq, dk = rope(dq, tok, d_h, d_rope, inverse=True), rope(dk, tok, d_h, d_rope, inverse=True)
            dWq[i] += hp.T @ dq
            dWk[i] += hp.T @ dk
            dWv[i] += hp.T @ dv
            np.add.at(dx[b], tok, dq @ Wq[i].T + dk @ Wk[i].T + dv @ Wv[i].T)
    dW_r = np.zeros_like(W_r)
    if use_gate:
        dW_r, dxr = _gate_to_router_grads(x, W_r, r, dgate)
        dx += dxr
    return dx, dWq, dWk, dWv, dWo, dW_r, dgate


# ----------------------------------------------------------------------------------------------
# algorithmic work counts (used by the tests of the flop counter and by the benchmark's CPU leg)
# ----------------------------------------------------------------------------------------------

def routed_rows(B: int, k: int, c: int, l_p: int) -> int:
    return B * k * c * l_p
