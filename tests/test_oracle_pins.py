"""Pins for the fp64 oracle: every check compares it with something that is not itself
(a closed form, a textbook routine, torch's library attention, a brute-force rule, an
invariant of the equations, or values printed in the paper)."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import mac_count
from oracle.switchhead_loops import switchhead_forward_loops
from oracle.switchhead_oracle import (bucket_lists, dense_mha_forward, stable_sigmoid,
                                      switchhead_forward, topk_lower_index_wins)


def rand_layer(rng, B, T, M, H, D, E, gate_scale=1.0):
    f = lambda *s: rng.standard_normal(s)
    return dict(x=f(B, T, M), Wq=f(H, M, D) / np.sqrt(M), Wk=f(H, M, D) / np.sqrt(M),
                Wv=f(H, E, M, D) / np.sqrt(M), Wo=f(H, E, D, M) / np.sqrt(D),
                Ws=gate_scale * f(H, M, E) / np.sqrt(M), Wd=gate_scale * f(H, M, E) / np.sqrt(M))


def mha_sum_over_heads(x, Wq, Wk, Wv, Wo, causal=True):
    """Eq. 3: y = sum_h A^h V^h W_O^h, written independently with einsum."""
    B, T, M = x.shape
    H, _, D = Wq.shape
    Q = np.einsum("btm,hmd->bhtd", x, Wq)
    K = np.einsum("btm,hmd->bhtd", x, Wk)
    V = np.einsum("btm,hmd->bhtd", x, Wv)
    L = np.einsum("bhtd,bhsd->bhts", Q, K) / np.sqrt(D)
    if causal:
        t = np.arange(T)
        L = np.where(t[None, :] > t[:, None], -np.inf, L)
    L = L - L.max(-1, keepdims=True)
    A = np.exp(L)
    A /= A.sum(-1, keepdims=True)
    return np.einsum("bhts,bhsd,hdm->btm", A, V, Wo)


def torch_sdpa_mha(x, Wq, Wk, Wv, Wo):
    xt, q, k_, v, o = (torch.from_numpy(np.asarray(a)) for a in (x, Wq, Wk, Wv, Wo))
    Q = torch.einsum("btm,hmd->bhtd", xt, q)
    K = torch.einsum("btm,hmd->bhtd", xt, k_)
    V = torch.einsum("btm,hmd->bhtd", xt, v)
    R = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True)
    return torch.einsum("bhtd,hdm->btm", R, o).numpy()


# ---- P7: Eq. 2 (concatenation) == Eq. 3 (sum over heads) == library attention ----------
def test_dense_mha_eq2_equals_eq3_and_library():
    rng = np.random.default_rng(10)
    L = rand_layer(rng, 2, 19, 24, 3, 8, 1)
    Wv, Wo = L["Wv"][:, 0], L["Wo"][:, 0]
    y2 = dense_mha_forward(L["x"], L["Wq"], L["Wk"], Wv, Wo)
    y3 = mha_sum_over_heads(L["x"], L["Wq"], L["Wk"], Wv, Wo)
    yl = torch_sdpa_mha(L["x"], L["Wq"], L["Wk"], Wv, Wo)
    assert np.allclose(y2, y3, rtol=1e-12, atol=1e-13)
    assert np.allclose(y2, yl, rtol=1e-10, atol=1e-12)


# ---- P1: E=1, k=1 ------------------------------------------------------------------
def test_single_expert_zero_gate_weights_is_quarter_mha():
    rng = np.random.default_rng(11)
    L = rand_layer(rng, 2, 23, 16, 3, 8, 1)
    L["Ws"][:] = 0.0
    L["Wd"][:] = 0.0                      # every gate = sigmoid(0) = 0.5 exactly
    out = switchhead_forward(**L, k=1)
    ref = torch_sdpa_mha(L["x"], L["Wq"], L["Wk"], L["Wv"][:, 0], L["Wo"][:, 0])
    assert np.all(out["gateS"] == 0.5) and np.all(out["gateD"] == 0.5)
    assert np.allclose(out["y"], 0.25 * ref, rtol=1e-10, atol=1e-12)


def test_single_expert_gate_forced_to_one_is_mha():
    rng = np.random.default_rng(12)
    L = rand_layer(rng, 1, 17, 16, 2, 8, 1)
    out = switchhead_forward(**L, k=1, gate_override=1.0)
    ref = mha_sum_over_heads(L["x"], L["Wq"], L["Wk"], L["Wv"][:, 0], L["Wo"][:, 0])
    assert np.allclose(out["y"], ref, rtol=1e-11, atol=1e-12)


# ---- P2: k = E is the dense gate-weighted sum over all experts ------------------------
def test_k_equals_E_is_dense_weighted_sum():
    rng = np.random.default_rng(13)
    B, T, M, H, D, E = 2, 15, 12, 2, 4, 3
    L = rand_layer(rng, B, T, M, H, D, E)
    out = switchhead_forward(**L, k=E)
    x = L["x"]
    sS = 1.0 / (1.0 + np.exp(-np.einsum("btm,hme->bthe", x, L["Ws"])))
    sD = 1.0 / (1.0 + np.exp(-np.einsum("btm,hme->bthe", x, L["Wd"])))
    V = np.einsum("bthe,btm,hemd->bhtd", sS, x, L["Wv"])
    Q = np.einsum("btm,hmd->bhtd", x, L["Wq"])
    K = np.einsum("btm,hmd->bhtd", x, L["Wk"])
    Lg = np.einsum("bhtd,bhsd->bhts", Q, K) / np.sqrt(D)
    t = np.arange(T)
    Lg = np.where(t[None, :] > t[:, None], -np.inf, Lg)
    A = np.exp(Lg - Lg.max(-1, keepdims=True))
    A /= A.sum(-1, keepdims=True)
    R = np.einsum("bhts,bhsd->bthd", A, V)
    y = np.einsum("bthe,bthd,hedm->btm", sD, R, L["Wo"])
    assert np.allclose(out["y"], y, rtol=1e-11, atol=1e-12)


# ---- P3: top-k and the tie rule -------------------------------------------------------
def brute_topk(row, k):
    pairs = sorted(((-(v + 0.0), i) for i, v in enumerate(row)))
    return [i for _, i in pairs[:k]]


def test_topk_matches_brute_force_with_ties_and_signed_zero():
    rng = np.random.default_rng(14)
    for E in (1, 2, 5, 8):
        for k in range(1, E + 1):
            z = rng.integers(-2, 3, size=(200, E)).astype(np.float64)   # many exact ties
            z[::7] *= -0.0                                               # -0.0 / +0.0 rows
            z2 = rng.standard_normal((50, E))
            for zz in (z, z2):
                got = topk_lower_index_wins(zz, k)
                for r in range(zz.shape[0]):
                    assert got[r].tolist() == brute_topk(zz[r].tolist(), k)


def test_topk_constructed_ties():
    z = np.array([[1.0, 3.0, 3.0, 1.0, 3.0], [0.0, -0.0, 0.0, -1.0, -0.0]])
    assert topk_lower_index_wins(z, 2).tolist() == [[1, 2], [0, 1]]
    assert topk_lower_index_wins(z, 4).tolist() == [[1, 2, 4, 0], [0, 1, 2, 4]]


def test_sigmoid_closed_values():
    z = np.array([0.0, np.log(3.0), -np.log(3.0), 800.0, -800.0])
    s = stable_sigmoid(z)
    assert s[0] == 0.5 and abs(s[1] - 0.75) < 1e-15 and abs(s[2] - 0.25) < 1e-15
    assert s[3] == 1.0 and s[4] == 0.0 or s[4] < 1e-300


# ---- P4: causality ----------------------------------------------------------------------
def test_future_tokens_do_not_change_earlier_outputs():
    rng = np.random.default_rng(15)
    L = rand_layer(rng, 2, 20, 16, 2, 8, 4)
    y0 = switchhead_forward(**L, k=2)["y"]
    t0 = 11
    L2 = dict(L)
    L2["x"] = L["x"].copy()
    L2["x"][:, t0 + 1:] += rng.standard_normal(L2["x"][:, t0 + 1:].shape)
    y1 = switchhead_forward(**L2, k=2)["y"]
    assert np.array_equal(y0[:, :t0 + 1], y1[:, :t0 + 1])
    assert not np.allclose(y0[:, t0 + 1:], y1[:, t0 + 1:])
    # and without the mask the past does change
    y2 = switchhead_forward(**L, k=2, causal=False)["y"]
    y3 = switchhead_forward(**L2, k=2, causal=False)["y"]
    assert not np.allclose(y2[:, :t0 + 1], y3[:, :t0 + 1])


# ---- P5: softmax / mask closed form -----------------------------------------------------
def test_zero_queries_give_running_means_and_rows_sum_to_one():
    rng = np.random.default_rng(16)
    B, T, M, H, D, E, k = 1, 13, 10, 2, 4, 3, 2
    L = rand_layer(rng, B, T, M, H, D, E)
    L["Wq"][:] = 0.0
    out = switchhead_forward(**L, k=k)
    V = out["V"]                                        # [B,T,H,D]
    running = np.cumsum(V, axis=1) / np.arange(1, T + 1)[None, :, None, None]
    assert np.allclose(out["Ahat"], running, rtol=1e-12, atol=1e-13)
    # row 0 attends only to itself: y[0] = sum_h sum_e sD[0,e] V^h[0] W_O^{h,e}
    y0 = np.zeros(M)
    for h in range(H):
        for j in range(k):
            e = out["idxD"][0, h, j]
            y0 += out["sD"][0, h, e] * (V[0, 0, h] @ L["Wo"][h, e])
    assert np.allclose(out["y"][0, 0], y0, rtol=1e-12, atol=1e-13)


def test_constant_values_pass_through_attention():
    # if V^h[s] is the same vector for every s, any softmax row (summing to 1) returns it
    rng = np.random.default_rng(17)
    B, T, M, H, D, E = 1, 9, 6, 1, 3, 2
    L = rand_layer(rng, B, T, M, H, D, E)
    L["x"][:] = L["x"][:, :1]                           # identical tokens -> identical V rows
    out = switchhead_forward(**L, k=1)
    assert np.allclose(out["Ahat"], out["V"], rtol=1e-12, atol=1e-13)


# ---- P6: index bookkeeping ---------------------------------------------------------------
def test_expert_permutation_invariance():
    rng = np.random.default_rng(18)
    H, E = 2, 5
    L = rand_layer(rng, 2, 14, 12, H, 4, E)
    y0 = switchhead_forward(**L, k=2)["y"]
    L2 = {k_: v.copy() for k_, v in L.items()}
    for h in range(H):
        pS, pD = rng.permutation(E), rng.permutation(E)
        L2["Ws"][h] = L["Ws"][h][:, pS]
        L2["Wv"][h] = L["Wv"][h][pS]
        L2["Wd"][h] = L["Wd"][h][:, pD]
        L2["Wo"][h] = L["Wo"][h][pD]
    y1 = switchhead_forward(**L2, k=2)["y"]
    assert np.allclose(y0, y1, rtol=1e-11, atol=1e-12)
    # permuting only the gate columns (not the experts) must change the result
    L3 = {k_: v.copy() for k_, v in L.items()}
    L3["Ws"][0] = L["Ws"][0][:, ::-1]
    assert not np.allclose(y0, switchhead_forward(**L3, k=2)["y"])


def test_batch_permutation_and_linearity_in_Wo():
    rng = np.random.default_rng(19)
    L = rand_layer(rng, 3, 11, 8, 2, 4, 3)
    y0 = switchhead_forward(**L, k=2)["y"]
    perm = np.array([2, 0, 1])
    L2 = dict(L)
    L2["x"] = L["x"][perm]
    assert np.array_equal(switchhead_forward(**L2, k=2)["y"], y0[perm])
    L3 = dict(L)
    L3["Wo"] = 3.0 * L["Wo"]
    assert np.allclose(switchhead_forward(**L3, k=2)["y"], 3.0 * y0, rtol=1e-12)


def test_unselected_experts_contribute_nothing():
    rng = np.random.default_rng(20)
    H, E, k = 2, 4, 2
    L = rand_layer(rng, 1, 10, 8, H, 4, E)
    out = switchhead_forward(**L, k=k)
    # poison every expert that no token selected on either side; y must not move
    L2 = {k_: v.copy() for k_, v in L.items()}
    for h in range(H):
        for e in range(E):
            if not (out["idxS"][:, h] == e).any():
                L2["Wv"][h, e] = 1e6
            if not (out["idxD"][:, h] == e).any():
                L2["Wo"][h, e] = 1e6
    # force at least one fully unselected expert with a strongly negative gate column
    L2["Ws"][:, :, 0] = 0.0
    L2["Wd"][:, :, 0] = 0.0
    b = np.zeros((H, E)); b[:, 0] = -50.0
    o1 = switchhead_forward(**L2, k=k, bias_s=b, bias_d=b)
    L2["Wv"][:, 0] = 1e6
    L2["Wo"][:, 0] = -1e6
    o2 = switchhead_forward(**L2, k=k, bias_s=b, bias_d=b)
    assert not (o1["idxS"] == 0).any() and not (o1["idxD"] == 0).any()
    assert np.array_equal(o1["y"], o2["y"])


def test_gate_bias_enters_selection_and_score():
    rng = np.random.default_rng(21)
    L = rand_layer(rng, 1, 8, 8, 1, 4, 3)
    b = np.array([[0.0, 40.0, 0.0]])
    out = switchhead_forward(**L, k=1, bias_s=b, bias_d=b)
    assert (out["idxS"] == 1).all() and (out["idxD"] == 1).all()
    assert np.allclose(out["gateS"], 1.0) and np.allclose(out["gateD"], 1.0)


# ---- P8: bucket sort ---------------------------------------------------------------------
def test_bucket_lists_are_a_stable_counting_sort():
    rng = np.random.default_rng(22)
    n, H, E, k = 300, 3, 6, 3
    idx = np.stack([np.stack([rng.permutation(E)[:k] for _ in range(H)]) for _ in range(n)]).astype(np.int32)
    off, lists = bucket_lists(idx, E)
    for h in range(H):
        assert off[h, 0] == 0 and off[h, -1] == n * k
        counts = np.bincount(idx[:, h].ravel(), minlength=E)
        assert np.array_equal(np.diff(off[h]), counts)
        seen = np.zeros(n, dtype=int)
        for e in range(E):
            seg = lists[h, off[h, e]:off[h, e + 1]]
            assert np.all(np.diff(seg) > 0)
            for t in seg:
                assert e in idx[t, h]
            seen[seg] += 1
        assert np.all(seen == k)


# ---- vectorised oracle vs the literal loop writing ---------------------------------------
@pytest.mark.parametrize("B,T,M,H,D,E,k,bias", [(1, 7, 6, 1, 2, 1, 1, False), (2, 9, 8, 2, 4, 3, 2, False),
                                                (1, 12, 8, 2, 4, 5, 3, True), (1, 6, 4, 3, 2, 4, 4, False)])
def test_vectorised_equals_loops(B, T, M, H, D, E, k, bias):
    rng = np.random.default_rng(100 + T)
    L = rand_layer(rng, B, T, M, H, D, E)
    bs = rng.standard_normal((H, E)) if bias else None
    bd = rng.standard_normal((H, E)) if bias else None
    y = switchhead_forward(**L, k=k, bias_s=bs, bias_d=bd)["y"]
    yl = np.array(switchhead_forward_loops(**L, k=k, bias_s=bs, bias_d=bd))
    assert np.allclose(y, yl, rtol=1e-11, atol=1e-12)
    yn = switchhead_forward(**L, k=k, bias_s=bs, bias_d=bd, causal=False)["y"]
    yln = np.array(switchhead_forward_loops(**L, k=k, bias_s=bs, bias_d=bd, causal=False))
    assert np.allclose(yn, yln, rtol=1e-11, atol=1e-12)


# ---- P9: MAC accounting against the values the paper prints -------------------------------
def test_mac_formulas_reproduce_printed_table():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_mac_table.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 8
    for kind, H, D, M, T, E, k, macs, mem, tol in rows:
        H, D, M, T, E, k = map(int, (H, D, M, T, E, k))
        macs, mem, tol = float(macs), float(mem), float(tol)
        if kind == "dense":
            got, gotm = mac_count.xl_macs(H, T, D, M), mac_count.xl_mem(H, T, D)
        else:
            got = mac_count.switchhead_macs_as_tabulated(H, T, D, M, k, E)
            gotm = mac_count.switchhead_mem_as_tabulated(H, T, D)
        assert abs(got - macs) / macs < tol, (kind, H, got, macs)
        assert abs(gotm - mem) / mem < 0.07, (kind, H, gotm, mem)
    # headline ratios of the abstract: 44 % compute and 27 % memory at 262M
    r = mac_count.switchhead_macs_as_tabulated(4, 512, 112, 1024, 2, 4) / mac_count.xl_macs(16, 512, 64, 1024)
    m = mac_count.switchhead_mem_as_tabulated(4, 512, 112) / mac_count.xl_mem(16, 512, 64)
    assert round(100 * r) == 44 and round(100 * m) == 27
    # the printed SwitchHead equation exceeds the tabulated value (documented erratum)
    assert mac_count.switchhead_macs_printed(4, 512, 112, 1024, 2) > 2.45e9


# ---- rotary position embeddings (appendix "RoPE Positional Encodings") --------------------
def test_rope_closed_form_two_dimensions():
    """d_head = 2 has a single pair and theta_0 = 1: position p rotates (1, 0) to
    (cos p, sin p) and (0, 1) to (-sin p, cos p), whatever the base."""
    from oracle.switchhead_oracle import rope_rotate
    pos = np.array([0, 1, 2, 7])
    e0 = rope_rotate(np.tile([1.0, 0.0], (4, 1)), pos, 10000.0)
    e1 = rope_rotate(np.tile([0.0, 1.0], (4, 1)), pos, 123.0)
    assert np.allclose(e0, np.stack([np.cos(pos), np.sin(pos)], -1), atol=1e-15)
    assert np.allclose(e1, np.stack([-np.sin(pos), np.cos(pos)], -1), atol=1e-15)


def test_rope_angles_norms_and_relative_position():
    from oracle.switchhead_oracle import rope_rotate
    rng = np.random.default_rng(5)
    D, T, base = 8, 11, 10000.0
    a, b = rng.standard_normal((T, D)), rng.standard_normal((T, D))
    pos = np.arange(T)
    ra, rb = rope_rotate(a, pos, base), rope_rotate(b, pos, base)
    # position 0 is the identity; every pair keeps its norm
    assert np.array_equal(ra[0], a[0])
    assert np.allclose(ra[:, 0::2] ** 2 + ra[:, 1::2] ** 2, a[:, 0::2] ** 2 + a[:, 1::2] ** 2, rtol=1e-13)
    # pair i of the vector at position p is turned by p * base**(-2i/D): check the angle itself
    for i in range(D // 2):
        got = np.arctan2(ra[3, 2 * i + 1], ra[3, 2 * i]) - np.arctan2(a[3, 2 * i + 1], a[3, 2 * i])
        want = 3 * base ** (-2.0 * i / D)
        assert abs((got - want + np.pi) % (2 * np.pi) - np.pi) < 1e-12
    # scores depend on the two positions only through their difference
    s1 = rope_rotate(a, pos, base) @ rope_rotate(b, pos, base).T
    s2 = rope_rotate(a, pos + 37, base) @ rope_rotate(b, pos + 37, base).T
    assert np.allclose(s1, s2, rtol=1e-10, atol=1e-12)
    # and differ from the unrotated scores off the diagonal, agree on it
    s0 = a @ b.T
    assert np.allclose(np.diag(s1), np.diag(s0), rtol=1e-12)
    assert not np.allclose(s1, s0)


def test_rope_layer_is_shift_invariant_and_matches_the_complex_form():
    rng = np.random.default_rng(77)
    L = rand_layer(rng, 2, 9, 8, 2, 4, 3)
    y0 = switchhead_forward(**L, k=2, rope_base=10000.0)
    y1 = switchhead_forward(**L, k=2, rope_base=10000.0, rope_offset=1000)
    assert np.allclose(y0["y"], y1["y"], rtol=1e-9, atol=1e-11)          # only relative positions matter
    assert not np.allclose(y0["y"], switchhead_forward(**L, k=2)["y"])     # and it is not a no-op
    assert np.array_equal(y0["V"], switchhead_forward(**L, k=2)["V"])      # values are not rotated
    yl = np.array(switchhead_forward_loops(**L, k=2, rope_base=10000.0))   # complex-number writing
    assert np.allclose(y0["y"], yl, rtol=1e-11, atol=1e-12)
    # a single token sits at position 0: rotary embedding changes nothing
    L1 = rand_layer(rng, 3, 1, 8, 2, 4, 3)
    assert np.array_equal(switchhead_forward(**L1, k=2, rope_base=10000.0)["y"], switchhead_forward(**L1, k=2)["y"])


# ---- shared selection (appendix "Shared Selection") ---------------------------------------
def test_shared_selection_is_the_layer_with_one_gate_on_both_sides():
    rng = np.random.default_rng(91)
    L = rand_layer(rng, 2, 10, 8, 2, 4, 4)
    bs, bd = rng.standard_normal((2, 4)), rng.standard_normal((2, 4))
    sh = switchhead_forward(**L, k=2, bias_s=bs, bias_d=bd, shared_selection=True)
    # the same numbers as the ordinary layer whose destination gate is a copy of the source gate
    L2 = dict(L, Wd=L["Ws"])
    ref = switchhead_forward(**L2, k=2, bias_s=bs, bias_d=bs)
    assert np.array_equal(sh["y"], ref["y"])
    assert np.array_equal(sh["idxD"], sh["idxS"]) and np.array_equal(sh["gateD"], sh["gateS"])
    assert np.array_equal(sh["listsD"], sh["listsS"])
    # W_D and b_D play no part; the ordinary layer with a different W_D gives something else
    other = dict(L, Wd=rng.standard_normal(L["Wd"].shape))
    assert np.array_equal(switchhead_forward(**other, k=2, bias_s=bs, bias_d=None, shared_selection=True)["y"], sh["y"])
    assert not np.allclose(switchhead_forward(**L, k=2, bias_s=bs, bias_d=bd)["y"], sh["y"])
    # literal loop writing
    yl = np.array(switchhead_forward_loops(**L, k=2, bias_s=bs, bias_d=bd, shared_selection=True))
    assert np.allclose(sh["y"], yl, rtol=1e-11, atol=1e-12)
