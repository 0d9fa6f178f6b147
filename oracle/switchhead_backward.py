"""fp64 CPU oracle for the BACKWARD pass of one SwitchHead attention layer.

TEST INFRASTRUCTURE ONLY (same rules as switchhead_oracle.py: nothing in the product imports it).

The paper gives no backward formulas (its training runs rely on automatic differentiation of the
forward equations of Sec. 2.2); this file is the chain rule written out for those equations, in the
paper's notation, with the expert selection held fixed (top-k is piecewise constant: its gradient is
zero almost everywhere, which is also what automatic differentiation of the forward pass gives):

  y[t]      = sum_h sum_{e in E_D^h(t)} s_D^h[t,e] Ahat^h[t] W_O^{h,e}
  Ahat^h    = A^h V^h,   A^h = softmax(Q^h K^h^T / sqrt(d_head)) (causal),   Q^h = x W_Q^h, K^h = x W_K^h
  V^h[t]    = sum_{e in E_S^h(t)} s_S^h[t,e] x[t] W_V^{h,e},   s = sigmoid(x W_S^h), sigmoid(x W_D^h)

Given G = dL/dy it returns dL/dx and dL/dW for W_Q, W_K, W_V, W_O, W_S, W_D (and the gate biases, if any).
Pins (tests/test_oracle_backward_pins.py): central finite differences of the FORWARD oracle for every
returned gradient; linearity in G; zero gradient for experts nobody selected; the dense special case
(E = 1, gate weights zero) against the textbook attention backward.
"""
from __future__ import annotations

import numpy as np

from oracle.switchhead_oracle import gate_and_select


def switchhead_backward(x, Wq, Wk, Wv, Wo, Ws, Wd, k: int, G, bias_s=None, bias_d=None, causal: bool = True):
    """x [B, T, M]; Wq, Wk [H, M, D]; Wv [H, E, M, D]; Wo [H, E, D, M]; Ws, Wd [H, M, E]; G = dL/dy [B, T, M].
    Returns a dict: dx [B, T, M], dWq, dWk, dWv, dWo, dWs, dWd (shapes of the weights), dbias_s, dbias_d [H, E]."""
    f = lambda a: None if a is None else np.asarray(a, dtype=np.float64)
    x, Wq, Wk, Wv, Wo, Ws, Wd, G, bias_s, bias_d = map(f, (x, Wq, Wk, Wv, Wo, Ws, Wd, G, bias_s, bias_d))
    B, T, M = x.shape
    H, E, _, D = Wv.shape
    N = B * T
    x2d, G2d = x.reshape(N, M), G.reshape(N, M)
    scale = 1.0 / np.sqrt(D)

    # ---- forward quantities (recomputed: the oracle keeps no state) ----
    _, _, idxS, gateS = gate_and_select(x2d, Ws, bias_s, k)
    _, _, idxD, gateD = gate_and_select(x2d, Wd, bias_d, k)
    Q = np.einsum("nm,hmd->nhd", x2d, Wq)
    K = np.einsum("nm,hmd->nhd", x2d, Wk)
    XV = np.einsum("nm,hemd->nhed", x2d, Wv)                  # every expert's projection of every token
    V = np.zeros((N, H, D))
    for n in range(N):
        for h in range(H):
            for j in range(k):
                V[n, h] += gateS[n, h, j] * XV[n, h, idxS[n, h, j]]
    A = np.zeros((B, H, T, T))
    Ahat = np.zeros((N, H, D))
    for b in range(B):
        sl = slice(b * T, (b + 1) * T)
        for h in range(H):
            L = Q[sl, h] @ K[sl, h].T * scale
            if causal:
                L = np.where(np.triu(np.ones((T, T), dtype=bool), 1), -np.inf, L)
            P = np.exp(L - L.max(axis=1, keepdims=True))
            A[b, h] = P / P.sum(axis=1, keepdims=True)
            Ahat[sl, h] = A[b, h] @ V[sl, h]

    # ---- output experts: y[t] = sum_{h,j} gD * Ahat[t,h] Wo[h,e] ----
    dAhat = np.zeros((N, H, D))
    dWo = np.zeros_like(Wo)
    dgateD = np.zeros((N, H, k))
    for n in range(N):
        for h in range(H):
            for j in range(k):
                e, g = idxD[n, h, j], gateD[n, h, j]
                u = Ahat[n, h] @ Wo[h, e]                     # [M]
                dgateD[n, h, j] = u @ G2d[n]
                dAhat[n, h] += g * (Wo[h, e] @ G2d[n])
                dWo[h, e] += g * np.outer(Ahat[n, h], G2d[n])

    # ---- attention: Ahat = A V, A = softmax(S), S = Q K^T scale ----
    dQ, dK, dV = np.zeros((N, H, D)), np.zeros((N, H, D)), np.zeros((N, H, D))
    for b in range(B):
        sl = slice(b * T, (b + 1) * T)
        for h in range(H):
            dV[sl, h] = A[b, h].T @ dAhat[sl, h]
            dA = dAhat[sl, h] @ V[sl, h].T
            dS = A[b, h] * (dA - (dA * A[b, h]).sum(axis=1, keepdims=True))
            dQ[sl, h] = dS @ K[sl, h] * scale
            dK[sl, h] = dS.T @ Q[sl, h] * scale

    # ---- value experts: V[t,h] = sum_j gS * x[t] Wv[h,e] ----
    dx = np.zeros((N, M))
    dWv = np.zeros_like(Wv)
    dgateS = np.zeros((N, H, k))
    for n in range(N):
        for h in range(H):
            for j in range(k):
                e, g = idxS[n, h, j], gateS[n, h, j]
                dgateS[n, h, j] = XV[n, h, e] @ dV[n, h]
                dx[n] += g * (Wv[h, e] @ dV[n, h])
                dWv[h, e] += g * np.outer(x2d[n], dV[n, h])

    # ---- dense queries and keys ----
    dx += np.einsum("nhd,hmd->nm", dQ, Wq) + np.einsum("nhd,hmd->nm", dK, Wk)
    dWq = np.einsum("nm,nhd->hmd", x2d, dQ)
    dWk = np.einsum("nm,nhd->hmd", x2d, dK)

    # ---- gates: s = sigmoid(z), z = x W (+ b); only the selected entries reach the output ----
    out = {}
    for side, idx, gate, dgate, W in (("s", idxS, gateS, dgateS, Ws), ("d", idxD, gateD, dgateD, Wd)):
        dz = np.zeros((N, H, E))
        for j in range(k):
            np.put_along_axis(dz, idx[:, :, j][:, :, None], (dgate[:, :, j] * gate[:, :, j] * (1.0 - gate[:, :, j]))[:, :, None], 2)
        dx += np.einsum("nhe,hme->nm", dz, W)
        out["dW" + side] = np.einsum("nm,nhe->hme", x2d, dz)
        out["dbias_" + side] = dz.sum(axis=0)
    out.update(dx=dx.reshape(B, T, M), dWq=dWq, dWk=dWk, dWv=dWv, dWo=dWo)
    return out
