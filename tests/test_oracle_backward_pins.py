"""Pins of the backward oracle (oracle/switchhead_backward.py) against the FORWARD oracle and textbook
identities: central finite differences of L = sum(y * G) for every gradient it returns."""
import numpy as np
import pytest

from oracle.switchhead_backward import switchhead_backward
from oracle.switchhead_oracle import gate_and_select, switchhead_forward


def layer(rg, B, T, M, H, D, E, with_bias=False):
    W = dict(Wq=rg.standard_normal((H, M, D)) / np.sqrt(M), Wk=rg.standard_normal((H, M, D)) / np.sqrt(M),
             Wv=rg.standard_normal((H, E, M, D)) / np.sqrt(M), Wo=rg.standard_normal((H, E, D, M)) / np.sqrt(D),
             Ws=rg.standard_normal((H, M, E)), Wd=rg.standard_normal((H, M, E)))
    b = dict(bias_s=0.3 * rg.standard_normal((H, E)), bias_d=0.3 * rg.standard_normal((H, E))) if with_bias else dict(bias_s=None, bias_d=None)
    return rg.standard_normal((B, T, M)), W, b


def loss(x, W, b, k, G, causal):
    return float((switchhead_forward(x, W["Wq"], W["Wk"], W["Wv"], W["Wo"], W["Ws"], W["Wd"], k, b["bias_s"], b["bias_d"],
                                     causal=causal, return_stages=False)["y"] * G).sum())


def selection(x, W, b, k):
    M = x.shape[-1]
    return (gate_and_select(x.reshape(-1, M), W["Ws"], b["bias_s"], k)[2], gate_and_select(x.reshape(-1, M), W["Wd"], b["bias_d"], k)[2])


@pytest.mark.parametrize("causal,with_bias,E,k", [(True, False, 4, 2), (False, True, 3, 1), (True, True, 5, 3)])
def test_every_gradient_against_central_differences_of_the_forward_oracle(causal, with_bias, E, k):
    rg = np.random.default_rng(100 + E)
    B, T, M, H, D = 2, 5, 6, 2, 4
    x, W, b = layer(rg, B, T, M, H, D, E, with_bias)
    G = rg.standard_normal((B, T, M))
    g = switchhead_backward(x, W["Wq"], W["Wk"], W["Wv"], W["Wo"], W["Ws"], W["Wd"], k, G, b["bias_s"], b["bias_d"], causal=causal)
    sel0 = selection(x, W, b, k)
    eps = 1e-6
    checked = 0
    targets = [("dx", x, None), ("dWq", W["Wq"], "Wq"), ("dWk", W["Wk"], "Wk"), ("dWv", W["Wv"], "Wv"), ("dWo", W["Wo"], "Wo"),
               ("dWs", W["Ws"], "Ws"), ("dWd", W["Wd"], "Wd")]
    if with_bias:
        targets += [("dbias_s", b["bias_s"], "bias_s"), ("dbias_d", b["bias_d"], "bias_d")]
    for name, arr, key in targets:
        flat = arr.reshape(-1)
        for i in rg.choice(flat.size, size=min(flat.size, 25), replace=False):
            old = flat[i]
            flat[i] = old + eps
            same = all(np.array_equal(a, c) for a, c in zip(selection(x, W, b, k), sel0))
            lp = loss(x, W, b, k, G, causal)
            flat[i] = old - eps
            same = same and all(np.array_equal(a, c) for a, c in zip(selection(x, W, b, k), sel0))
            lm = loss(x, W, b, k, G, causal)
            flat[i] = old
            if not same:
                continue                                   # the step crossed a selection boundary: not differentiable there
            fd = (lp - lm) / (2 * eps)
            an = g[name].reshape(-1)[i]
            assert abs(fd - an) <= 1e-6 * (1 + abs(fd)), (name, int(i), fd, an)
            checked += 1
    assert checked > 100


def test_gradients_are_linear_in_the_output_gradient_and_vanish_for_unselected_experts():
    rg = np.random.default_rng(7)
    B, T, M, H, D, E, k = 1, 4, 6, 2, 4, 8, 2
    x, W, b = layer(rg, B, T, M, H, D, E)
    args = (x, W["Wq"], W["Wk"], W["Wv"], W["Wo"], W["Ws"], W["Wd"], k)
    G1, G2 = rg.standard_normal((B, T, M)), rg.standard_normal((B, T, M))
    a, c, s = switchhead_backward(*args, G1), switchhead_backward(*args, G2), switchhead_backward(*args, 2 * G1 - 3 * G2)
    for key in a:
        assert np.allclose(s[key], 2 * a[key] - 3 * c[key], rtol=1e-10, atol=1e-12), key
    idxS, idxD = selection(x, W, b, k)
    for h in range(H):
        for e in range(E):
            if e not in idxS[:, h, :]:
                assert not a["dWv"][h, e].any() and not a["dWs"][h, :, e].any()
            if e not in idxD[:, h, :]:
                assert not a["dWo"][h, e].any() and not a["dWd"][h, :, e].any()


def test_one_expert_with_zero_gate_weights_is_textbook_attention_backward():
    # E = 1, W_S = W_D = 0: both gates are 1/2, y = 1/4 * MHA(x); compare with the attention backward
    # written from the softmax Jacobian, head by head
    rg = np.random.default_rng(9)
    B, T, M, H, D = 1, 6, 5, 2, 3
    x, W, b = layer(rg, B, T, M, H, D, 1)
    W["Ws"][:] = 0; W["Wd"][:] = 0
    G = rg.standard_normal((B, T, M))
    g = switchhead_backward(x, W["Wq"], W["Wk"], W["Wv"], W["Wo"], W["Ws"], W["Wd"], 1, G)
    X, Gm = x[0], G[0]
    dx = np.zeros_like(X)
    for h in range(H):
        Wq, Wk, Wv, Wo = W["Wq"][h], W["Wk"][h], W["Wv"][h, 0], W["Wo"][h, 0]
        Q, K, V = X @ Wq, X @ Wk, X @ Wv
        S = Q @ K.T / np.sqrt(D)
        S[np.triu(np.ones((T, T), dtype=bool), 1)] = -np.inf
        A = np.exp(S - S.max(1, keepdims=True)); A /= A.sum(1, keepdims=True)
        dO = 0.25 * Gm @ Wo.T                               # d(A V)
        assert np.allclose(g["dWo"][h, 0], 0.5 * (0.5 * A @ V).T @ Gm, rtol=1e-10)     # destination gate 1/2, Ahat = A (x Wv / 2)
        dVm = A.T @ dO
        dA = dO @ V.T
        dS = np.zeros_like(A)
        for i in range(T):                                  # softmax Jacobian row by row
            J = np.diag(A[i]) - np.outer(A[i], A[i])
            dS[i] = J @ dA[i]
        dQ, dK = dS @ K / np.sqrt(D), dS.T @ Q / np.sqrt(D)
        assert np.allclose(g["dWq"][h], X.T @ dQ, rtol=1e-9, atol=1e-12)
        assert np.allclose(g["dWk"][h], X.T @ dK, rtol=1e-9, atol=1e-12)
        assert np.allclose(g["dWv"][h, 0], X.T @ dVm, rtol=1e-9, atol=1e-12)   # d(x Wv): the source gate 1/2 is inside dO's 1/4
        dx += dQ @ Wq.T + dK @ Wk.T + dVm @ Wv.T
    # with zero gate weights the gates pass no gradient to x
    assert np.allclose(g["dx"][0], dx, rtol=1e-9, atol=1e-12)
