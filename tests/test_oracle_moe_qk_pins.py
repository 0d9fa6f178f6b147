"""Pins of the oracle's MoE key / query projections (paper Sec. 2.2: K^h and Q^h written as expert sums
like V^h; its ablation over which projections are experts) against what the mathematics fixes."""
import numpy as np
import pytest

from oracle.switchhead_loops import switchhead_forward_loops
from oracle.switchhead_oracle import gate_and_select, switchhead_forward, switchhead_xl_forward


def weights(rg, H, E, M, D, moe_q, moe_k):
    Wq = rg.standard_normal((H, E, M, D) if moe_q else (H, M, D)) / np.sqrt(M)
    Wk = rg.standard_normal((H, E, M, D) if moe_k else (H, M, D)) / np.sqrt(M)
    Wv = rg.standard_normal((H, E, M, D)) / np.sqrt(M)
    Wo = rg.standard_normal((H, E, D, M)) / np.sqrt(D)
    Ws = rg.standard_normal((H, M, E))
    Wd = rg.standard_normal((H, M, E))
    return Wq, Wk, Wv, Wo, Ws, Wd


@pytest.mark.parametrize("moe_q,moe_k", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("shared", [False, True])
def test_vectorised_and_scalar_loop_writings_agree(moe_q, moe_k, shared):
    rg = np.random.default_rng(11)
    B, T, M, H, D, E, k = 2, 6, 8, 2, 4, 4, 2
    x = rg.standard_normal((B, T, M))
    W = weights(rg, H, E, M, D, moe_q, moe_k)
    a = switchhead_forward(x, *W, k, shared_selection=shared)["y"]
    b = np.array(switchhead_forward_loops(x, *W, k, shared_selection=shared))
    assert np.abs(a - b).max() < 1e-12


def test_identical_key_experts_scale_the_dense_keys_by_the_sum_of_the_selected_gates():
    rg = np.random.default_rng(12)
    B, T, M, H, D, E, k = 1, 9, 16, 2, 4, 5, 3
    x = rg.standard_normal((B, T, M))
    Wq, _, Wv, Wo, Ws, Wd = weights(rg, H, E, M, D, False, False)
    W = rg.standard_normal((H, M, D))
    Wk = np.repeat(W[:, None], E, axis=1)
    ref = switchhead_forward(x, Wq, Wk, Wv, Wo, Ws, Wd, k)
    _, _, idxS, gateS = gate_and_select(x.reshape(-1, M), Ws, None, k)
    want = gateS.sum(axis=2)[:, :, None] * np.einsum("nm,hmd->nhd", x.reshape(-1, M), W)
    assert np.allclose(ref["K"].reshape(-1, H, D), want, rtol=1e-12, atol=1e-12)
    # and the queries, with the destination side's gates
    Wq4 = np.repeat(W[:, None], E, axis=1)
    ref = switchhead_forward(x, Wq4, Wk, Wv, Wo, Ws, Wd, k)
    _, _, idxD, gateD = gate_and_select(x.reshape(-1, M), Wd, None, k)
    want = gateD.sum(axis=2)[:, :, None] * np.einsum("nm,hmd->nhd", x.reshape(-1, M), W)
    assert np.allclose(ref["Q"].reshape(-1, H, D), want, rtol=1e-12, atol=1e-12)


def test_all_experts_selected_with_a_constant_gate_is_a_dense_projection_with_the_summed_weights():
    rg = np.random.default_rng(13)
    B, T, M, H, D, E = 2, 7, 12, 2, 4, 3
    x = rg.standard_normal((B, T, M))
    Wq, Wk, Wv, Wo, Ws, Wd = weights(rg, H, E, M, D, True, True)
    c = 0.37
    moe = switchhead_forward(x, Wq, Wk, Wv, Wo, Ws, Wd, E, gate_override=c)["y"]
    dense = switchhead_forward(x, c * Wq.sum(axis=1), c * Wk.sum(axis=1), Wv, Wo, Ws, Wd, E, gate_override=c)["y"]
    assert np.allclose(moe, dense, rtol=1e-11, atol=1e-12)


def test_experts_nobody_selected_do_not_matter_and_selected_ones_do():
    rg = np.random.default_rng(14)
    B, T, M, H, D, E, k = 1, 5, 8, 2, 4, 8, 2
    x = rg.standard_normal((B, T, M))
    Wq, Wk, Wv, Wo, Ws, Wd = weights(rg, H, E, M, D, True, True)
    base = switchhead_forward(x, Wq, Wk, Wv, Wo, Ws, Wd, k)
    usedS = [set(base["idxS"].reshape(-1, H, k)[:, h, :].ravel()) for h in range(H)]
    usedD = [set(base["idxD"].reshape(-1, H, k)[:, h, :].ravel()) for h in range(H)]
    Wk2, Wq2 = Wk.copy(), Wq.copy()
    poisoned = 0
    for h in range(H):
        for e in range(E):
            if e not in usedS[h]:
                Wk2[h, e] = 1e6; poisoned += 1
            if e not in usedD[h]:
                Wq2[h, e] = -1e6; poisoned += 1
    assert poisoned > 0
    assert np.array_equal(switchhead_forward(x, Wq2, Wk2, Wv, Wo, Ws, Wd, k)["y"], base["y"])
    # a key expert some token did select changes the output; the keys use the SOURCE side's selection
    h0, e0 = 0, next(iter(usedS[0]))
    Wk3 = Wk.copy(); Wk3[h0, e0] *= 2.0
    assert not np.allclose(switchhead_forward(x, Wq, Wk3, Wv, Wo, Ws, Wd, k)["y"], base["y"])
    onlyD = [e for e in usedD[0] if e not in usedS[0]]
    if onlyD:                                   # selected on the destination side only: no key uses it
        Wk4 = Wk.copy(); Wk4[0, onlyD[0]] = 1e6
        assert np.array_equal(switchhead_forward(x, Wq, Wk4, Wv, Wo, Ws, Wd, k)["y"], base["y"])


def test_renumbering_the_experts_of_a_side_changes_nothing():
    rg = np.random.default_rng(15)
    B, T, M, H, D, E, k = 1, 8, 8, 2, 4, 5, 2
    x = rg.standard_normal((B, T, M))
    Wq, Wk, Wv, Wo, Ws, Wd = weights(rg, H, E, M, D, True, True)
    base = switchhead_forward(x, Wq, Wk, Wv, Wo, Ws, Wd, k)["y"]
    p = rg.permutation(E)
    src = switchhead_forward(x, Wq, Wk[:, p], Wv[:, p], Wo, Ws[:, :, p], Wd, k)["y"]      # source side: keys, values, W_S
    dst = switchhead_forward(x, Wq[:, p], Wk, Wv, Wo[:, p], Ws, Wd[:, :, p], k)["y"]      # destination side: queries, output, W_D
    assert np.allclose(src, base, rtol=1e-11, atol=1e-12) and np.allclose(dst, base, rtol=1e-11, atol=1e-12)


def test_context_form_without_a_cache_is_the_plain_layer_and_the_cache_keys_use_the_source_gate():
    rg = np.random.default_rng(16)
    B, T, Tc, M, H, D, E, k = 2, 5, 4, 8, 2, 4, 4, 2
    x = rg.standard_normal((B, T, M)); cache = rg.standard_normal((B, Tc, M))
    W = weights(rg, H, E, M, D, True, True)
    assert np.allclose(switchhead_xl_forward(x, None, *W, k)["y"], switchhead_forward(x, *W, k)["y"], rtol=1e-12, atol=1e-13)
    # with a cache: the chunk's outputs are those of the plain layer run over [cache; chunk]
    full = switchhead_forward(np.concatenate([cache, x], axis=1), *W, k)["y"][:, Tc:]
    assert np.allclose(switchhead_xl_forward(x, cache, *W, k)["y"], full, rtol=1e-11, atol=1e-12)
