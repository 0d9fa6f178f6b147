"""Literal scalar-loop writing of the SwitchHead forward pass (fp64, tiny shapes only).

TEST INFRASTRUCTURE ONLY.  A second, independent transcription of the equations of the
paper's Sec. 2.2, written token by token with Python floats and `math`, so that an index
or broadcasting slip in the vectorised oracle shows up as a disagreement.  It shares no
helper with the vectorised oracle.

Per sequence, per head h, per destination token t:
    y[t] += sum_{e in E_D^h(t)} sigmoid(z_D^h[t,e]) * (sum_{s<=t} A^h[t,s] V^h[s]) W_O^{h,e}
with V^h[s] = sum_{e in E_S^h(s)} sigmoid(z_S^h[s,e]) * x[s] W_V^{h,e}  and
     A^h[t,:] = softmax over visible keys of  Q^h[t].K^h[s] / sqrt(d_head)      (Eq. 1).
"""
from __future__ import annotations

import cmath
import math


def _sigmoid(z: float) -> float:
    if z >= 0:
        return 1.0 / (1.0 + math.exp(-z))
    ez = math.exp(z)
    return ez / (1.0 + ez)


def _select(z_row, k):
    """k best experts: repeatedly take the largest remaining logit, lowest index on ties."""
    chosen = []
    remaining = list(range(len(z_row)))
    for _ in range(k):
        best = remaining[0]
        for e in remaining[1:]:
            if z_row[e] > z_row[best]:
                best = e
        chosen.append(best)
        remaining.remove(best)
    return chosen


def _vecmat(v, W):
    """v [n], W [n][m] -> [m]"""
    m = len(W[0])
    out = [0.0] * m
    for i, vi in enumerate(v):
        row = W[i]
        for j in range(m):
            out[j] += vi * row[j]
    return out


def _rope_complex(vec, pos, base):
    """Rotary embedding written with complex numbers: the pair (v[2i], v[2i+1]) is one complex
    number, multiplied by exp(i * pos * base**(-2i/D)) (RoFormer's formulation)."""
    D = len(vec)
    out = [0.0] * D
    for i in range(D // 2):
        z = complex(vec[2 * i], vec[2 * i + 1]) * cmath.exp(1j * pos * base ** (-2.0 * i / D))
        out[2 * i], out[2 * i + 1] = z.real, z.imag
    return out


def switchhead_forward_loops(x, Wq, Wk, Wv, Wo, Ws, Wd, k, bias_s=None, bias_d=None, causal=True, rope_base=None, shared_selection=False):
    """Nested lists or arrays in, nested list y [B][T][M] out."""
    x = [[list(map(float, tok)) for tok in seq] for seq in x]
    B, T, M = len(x), len(x[0]), len(x[0][0])
    H, E = len(Wv), len(Wv[0])
    D = len(Wv[0][0][0])
    tolist = lambda a: a.tolist() if hasattr(a, "tolist") else a
    Wq, Wk, Wv, Wo, Ws, Wd = map(tolist, (Wq, Wk, Wv, Wo, Ws, Wd))
    bias_s = tolist(bias_s) if bias_s is not None else None
    bias_d = tolist(bias_d) if bias_d is not None else None
    y = [[[0.0] * M for _ in range(T)] for _ in range(B)]
    for b in range(B):
        for h in range(H):
            Q, K, V, selD = [], [], [], []
            for t in range(T):
                xt = x[b][t]
                moe_q, moe_k = isinstance(Wq[h][0][0], list), isinstance(Wk[h][0][0], list)   # [E][M][D] instead of [M][D]
                q_t = None if moe_q else _vecmat(xt, Wq[h])
                k_t = None if moe_k else _vecmat(xt, Wk[h])
                zs = _vecmat(xt, Ws[h])
                zd = _vecmat(xt, Ws[h] if shared_selection else Wd[h])
                if bias_s is not None:
                    zs = [a + c for a, c in zip(zs, bias_s[h])]
                bd = bias_s if shared_selection else bias_d
                if bd is not None:
                    zd = [a + c for a, c in zip(zd, bd[h])]
                v = [0.0] * D
                for e in _select(zs, k):
                    g = _sigmoid(zs[e])
                    pe = _vecmat(xt, Wv[h][e])
                    for d in range(D):
                        v[d] += g * pe[d]
                V.append(v)
                selD.append([(e, _sigmoid(zd[e])) for e in _select(zd, k)])
                if moe_k:                                   # key experts: the source side's selection and scores
                    k_t = [0.0] * D
                    for e in _select(zs, k):
                        pe = _vecmat(xt, Wk[h][e])
                        for d in range(D):
                            k_t[d] += _sigmoid(zs[e]) * pe[d]
                if moe_q:                                   # query experts: the destination side's
                    q_t = [0.0] * D
                    for e, g in selD[-1]:
                        pe = _vecmat(xt, Wq[h][e])
                        for d in range(D):
                            q_t[d] += g * pe[d]
                if rope_base is not None:
                    q_t, k_t = _rope_complex(q_t, t, rope_base), _rope_complex(k_t, t, rope_base)
                Q.append(q_t)
                K.append(k_t)
            for t in range(T):
                last = t if causal else T - 1
                logits = [sum(Q[t][d] * K[s][d] for d in range(D)) / math.sqrt(D)
                          for s in range(last + 1)]
                mx = max(logits)
                w = [math.exp(l - mx) for l in logits]
                tot = sum(w)
                a = [0.0] * D
                for s, ws_ in enumerate(w):
                    for d in range(D):
                        a[d] += (ws_ / tot) * V[s][d]
                for e, g in selD[t]:
                    contrib = _vecmat(a, Wo[h][e])
                    for c in range(M):
                        y[b][t][c] += g * contrib[c]
    return y
