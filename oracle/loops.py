"""Scalar-loop twin of the float64 oracle, for tiny inputs only.

TEST INFRASTRUCTURE ONLY (never imported by the product).  Every sum is written out as a Python
loop over scalars, with no numpy matmul, argsort or broadcasting, so that a slip in the array
version (a transposed operand, a wrong axis, an off-by-one slice) shows up as a disagreement.
Selections are found by exhaustive search over subsets rather than by sorting.

Follows the same passages as the array oracle: Eq. 12-14, 17, 21-23 (routing), Eq. 18-20 and 37-40
(UoME), Eq. 27-30, 33-36, 41 and Fig. 4 (SMHA).
"""
from __future__ import annotations

import itertools
import math


def _act(h: float, act: str) -> float:
    if act == "silu":
        return h / (1.0 + math.exp(-h))
    if act == "gelu_erf":
        return 0.5 * h * (1.0 + math.erf(h / math.sqrt(2.0)))
    if act == "gelu_tanh":
        return 0.5 * h * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (h + 0.044715 * h * h * h)))
    if act == "identity":
        return h
    raise ValueError(act)


def _softmax(v):
    mx = max(v)
    e = [math.exp(a - mx) for a in v]
    s = sum(e)
    return [a / s for a in e]


def best_subset(values, candidates, count):
    """Exhaustive search: the size-`count` subset of `candidates` with the largest value sum; among
    equal sums the lexicographically smallest index tuple (which is the lower-index tie rule)."""
    best, best_sum = None, None
    for comb in itertools.combinations(sorted(candidates), count):
        s = sum(values[j] for j in comb)
        if best is None or s > best_sum:   # strict: earlier (lexicographically smaller) tuples win ties
            best, best_sum = comb, s
    return list(best) if best is not None else []


def route(x, W_r, B, L, d, n, k, m, c, L_valid, use_gate=True):
    l_p = L // m
    cnt = [max(0, min((j + 1) * l_p, L_valid) - j * l_p) for j in range(m)]
    out = []
    for b in range(B):
        # patch gate
        p_patch = [[0.0] * m for _ in range(n)]
        for j in range(m):
            logits = []
            for i in range(n):
                acc = 0.0
                for t in range(j * l_p, j * l_p + cnt[j]):
                    for q in range(d):
                        acc += x[b][t][q] * W_r[q][i]
                logits.append(acc / cnt[j] if cnt[j] else 0.0)
            sm = _softmax(logits)
            for i in range(n):
                p_patch[i][j] = sm[i]
        # sample gate
        logits = []
        for i in range(n):
            acc = 0.0
            for t in range(L_valid):
                for q in range(d):
                    acc += x[b][t][q] * W_r[q][i]
            logits.append(acc / L_valid)
        p_samp = _softmax(logits)
        experts = best_subset(p_samp, range(n), k)
        elig = [j for j in range(m) if cnt[j] > 0]
        sel = []
        for i in experts:
            patches = best_subset(p_patch[i], elig, min(c, len(elig)))
            g = [(p_samp[i] * p_patch[i][j] if use_gate else 1.0) for j in patches]
            sel.append((i, patches, g))
        out.append(dict(p_samp=p_samp, p_patch=p_patch, sel=sel))
    return out


def mlp_forward(x, W1, W2, routing, B, L, d, d_e, m, L_valid, act, residual=True):
    l_p = L // m
    y = [[[x[b][t][q] if residual else 0.0 for q in range(d)] for t in range(L)] for b in range(B)]
    for b in range(B):
        for (i, patches, g) in routing[b]["sel"]:
            for u, j in enumerate(patches):
                for t in range(j * l_p, min((j + 1) * l_p, L_valid)):
                    a = []
                    for e in range(d_e):
                        acc = 0.0
                        for q in range(d):
                            acc += x[b][t][q] * W1[i][q][e]
                        a.append(_act(acc, act))
                    for q in range(d):
                        acc = 0.0
                        for e in range(d_e):
                            acc += a[e] * W2[i][e][q]
                        y[b][t][q] += g[u] * acc
    return y


def smha_forward(x, Wq, Wk, Wv, Wo, routing, B, L, d, d_g, d_h, m, L_valid, causal, residual=True):
    l_p = L // m
    heads = d_g // d_h
    y = [[[x[b][t][q] if residual else 0.0 for q in range(d)] for t in range(L)] for b in range(B)]
    for b in range(B):
        for (i, patches, g) in routing[b]["sel"]:
            tok = [t for j in patches for t in range(j * l_p, (j + 1) * l_p)]
            gate_of = [g[u] for u, j in enumerate(patches) for _ in range(l_p)]

            def proj(W):
                return [[sum(x[b][t][q] * W[i][q][e] for q in range(d)) for e in range(d_g)] for t in tok]
            Q, K, V = proj(Wq), proj(Wk), proj(Wv)
            for a_pos, ta in enumerate(tok):
                if ta >= L_valid:
                    continue                      # pad query: row of y stays x
                o = [0.0] * d_g
                for hd in range(heads):
                    lo = hd * d_h
                    sc, keys = [], []
                    for b_pos, tb in enumerate(tok):
                        if tb >= L_valid:
                            continue              # pad key (Eq. 41)
                        if causal and tb > ta:
                            continue              # original causal mask at (ta, tb)
                        sc.append(sum(Q[a_pos][lo + e] * K[b_pos][lo + e] for e in range(d_h)) / math.sqrt(d_h))
                        keys.append(b_pos)
                    p = _softmax(sc)
                    for w, b_pos in zip(p, keys):
                        for e in range(d_h):
                            o[lo + e] += w * V[b_pos][lo + e]
                for q in range(d):
                    y[b][ta][q] += gate_of[a_pos] * sum(o[e] * Wo[i][e][q] for e in range(d_g))
    return y
