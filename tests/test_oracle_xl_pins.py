"""Pins for the Transformer-XL-context oracle (switchhead_xl_forward): each check compares it with
something that is not itself - the plain layer, an identity of the equations, a closed form, a
brute-force scalar writing, or the paper's printed MAC / memory table."""
import numpy as np
import pytest

from oracle import mac_count
from oracle.switchhead_oracle import switchhead_forward, switchhead_xl_forward, xl_relative_embedding
from tests.test_oracle_pins import rand_layer


def xl_params(rng, H, M, D):
    return dict(Wr=rng.standard_normal((H, M, D)) / np.sqrt(M), u=0.3 * rng.standard_normal((H, D)),
                v=0.3 * rng.standard_normal((H, D)))


def layer_args(L):
    return (L["Wq"], L["Wk"], L["Wv"], L["Wo"], L["Ws"], L["Wd"])


def test_no_cache_no_positions_is_the_plain_layer():
    rng = np.random.default_rng(70)
    L = rand_layer(rng, 2, 23, 16, 2, 8, 4)
    a = switchhead_xl_forward(L["x"], None, *layer_args(L), 2)
    b = switchhead_forward(L["x"], *layer_args(L), 2)
    assert np.array_equal(a["idxS"], b["idxS"]) and np.array_equal(a["idxD"], b["idxD"])
    assert np.allclose(a["y"], b["y"], rtol=1e-12, atol=1e-13)
    assert np.allclose(a["Ahat"], b["Ahat"], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("with_positions", [False, True])
def test_cache_split_identity(with_positions):
    """One causal pass over 2T tokens equals a pass over the first T tokens followed by a pass over the
    second T tokens with the first chunk's layer input as the cache: with relative positions too, since
    the distances between a query and its keys are the same either way."""
    rng = np.random.default_rng(71)
    T = 13
    L = rand_layer(rng, 2, 2 * T, 16, 2, 8, 5)
    P = xl_params(rng, 2, 16, 8) if with_positions else {}
    whole = switchhead_xl_forward(L["x"], None, *layer_args(L), 3, **P)
    first = switchhead_xl_forward(L["x"][:, :T], None, *layer_args(L), 3, **P)
    second = switchhead_xl_forward(L["x"][:, T:], L["x"][:, :T], *layer_args(L), 3, **P)
    assert np.allclose(whole["y"][:, :T], first["y"], rtol=1e-11, atol=1e-12)
    assert np.allclose(whole["y"][:, T:], second["y"], rtol=1e-11, atol=1e-12)
    # the source side of the second pass covers the cache tokens as well, with the selections they had
    assert np.array_equal(second["idxS"], whole["idxS"])
    assert np.allclose(second["V"], whole["V"], rtol=1e-12, atol=1e-13)


def test_cache_is_visible_to_every_query_and_later_chunk_tokens_are_not():
    rng = np.random.default_rng(72)
    T, Tc = 9, 7
    L = rand_layer(rng, 1, T, 16, 2, 8, 4)
    cache = rng.standard_normal((1, Tc, 16))
    P = xl_params(rng, 2, 16, 8)
    base = switchhead_xl_forward(L["x"], cache, *layer_args(L), 2, **P)["y"]
    c2 = cache.copy()
    c2[:, 3] += 1.0                                          # a cache token: every output row moves
    moved = switchhead_xl_forward(L["x"], c2, *layer_args(L), 2, **P)["y"]
    assert np.all(np.abs(moved - base).max(axis=-1) > 1e-9)
    x2 = L["x"].copy()
    x2[:, 5:] += 1.0                                         # chunk tokens 5.. : rows 0..4 do not move
    later = switchhead_xl_forward(x2, cache, *layer_args(L), 2, **P)
    # (up to the last bit: the per-expert row groups change size, and with them the library's blocking)
    assert np.allclose(later["y"][:, :5], base[:, :5], rtol=1e-13, atol=1e-14)
    later = later["y"]
    assert not np.allclose(later[:, 5:], base[:, 5:])


def test_zero_queries_give_running_means_over_cache_and_chunk():
    """W_Q = 0 and no position term: every visible key has the same score, so Ahat[i] is the mean of
    V over the Tc + i + 1 context positions the query sees (a closed form)."""
    rng = np.random.default_rng(73)
    T, Tc = 6, 4
    L = rand_layer(rng, 2, T, 16, 2, 8, 3)
    L["Wq"] = np.zeros_like(L["Wq"])
    cache = rng.standard_normal((2, Tc, 16))
    r = switchhead_xl_forward(L["x"], cache, *layer_args(L), 2)
    csum = np.cumsum(r["V"], axis=1)                          # [B, Tc+T, H, D]
    want = csum[:, Tc:] / (Tc + 1 + np.arange(T))[None, :, None, None]
    assert np.allclose(r["Ahat"], want, rtol=1e-12, atol=1e-13)


def test_relative_embedding_closed_form():
    emb = xl_relative_embedding(5, 8)
    assert emb.shape == (5, 8)
    assert np.allclose(emb[0], [0, 0, 0, 0, 1, 1, 1, 1])      # distance 0: sin 0, cos 0
    w = 10000.0 ** (-2.0 * np.arange(4) / 8)
    assert np.allclose(emb[3, :4], np.sin(3 * w)) and np.allclose(emb[3, 4:], np.cos(3 * w))


def test_scalar_loop_writing_agrees_on_tiny_shapes():
    """The same layer written as plain loops over (batch, head, query, key), gathering r by distance
    one element at a time."""
    rng = np.random.default_rng(74)
    B, T, Tc, M, H, D, E, k = 2, 5, 3, 8, 2, 4, 3, 2
    L = rand_layer(rng, B, T, M, H, D, E)
    cache = rng.standard_normal((B, Tc, M))
    P = xl_params(rng, H, M, D)
    got = switchhead_xl_forward(L["x"], cache, *layer_args(L), k, **P)
    ctx = np.concatenate([cache, L["x"]], axis=1)
    emb = xl_relative_embedding(Tc + T, M)
    y = np.zeros((B, T, M))
    for b in range(B):
        for h in range(H):
            # source side, per context token
            Vc = np.zeros((Tc + T, D))
            Kc = ctx[b] @ L["Wk"][h]
            for s in range(Tc + T):
                z = ctx[b, s] @ L["Ws"][h]
                top = sorted(range(E), key=lambda e: (-z[e], e))[:k]
                for e in top:
                    Vc[s] += (1.0 / (1.0 + np.exp(-z[e]))) * (ctx[b, s] @ L["Wv"][h, e])
            for i in range(T):
                q = L["x"][b, i] @ L["Wq"][h]
                sc = []
                for j in range(Tc + i + 1):
                    r = emb[Tc + i - j] @ P["Wr"][h]
                    sc.append(((q + P["u"][h]) @ Kc[j] + (q + P["v"][h]) @ r) / np.sqrt(D))
                sc = np.array(sc)
                w = np.exp(sc - sc.max())
                a = (w / w.sum()) @ Vc[:Tc + i + 1]
                z = L["x"][b, i] @ L["Wd"][h]
                top = sorted(range(E), key=lambda e: (-z[e], e))[:k]
                for e in top:
                    y[b, i] += (1.0 / (1.0 + np.exp(-z[e]))) * (a @ L["Wo"][h, e])
    assert np.allclose(got["y"], y, rtol=1e-10, atol=1e-12)


def test_zero_position_weights_remove_the_position_term():
    rng = np.random.default_rng(75)
    L = rand_layer(rng, 1, 7, 16, 2, 8, 4)
    cache = rng.standard_normal((1, 5, 16))
    plain = switchhead_xl_forward(L["x"], cache, *layer_args(L), 2)["y"]
    zeroed = switchhead_xl_forward(L["x"], cache, *layer_args(L), 2, Wr=np.zeros((2, 16, 8)),
                                   u=np.zeros((2, 8)), v=np.zeros((2, 8)))["y"]
    assert np.allclose(plain, zeroed, rtol=1e-12, atol=1e-13)
    P = xl_params(rng, 2, 16, 8)
    assert not np.allclose(switchhead_xl_forward(L["x"], cache, *layer_args(L), 2, **P)["y"], plain)


def test_mac_and_memory_formulas_count_the_context_terms():
    """The appendix's cost model for the XL setting (C = 2) against the numbers its table prints:
    the context enters through the C T^2 attention terms and the C T position projection."""
    dense = mac_count.xl_macs(16, 512, 64, 1024, C=2)
    assert abs(dense - 5.37e9) / 5.37e9 < 5e-3                   # the "5.4G" row of the 262M models
    assert mac_count.xl_macs(16, 512, 64, 1024, C=1) < dense     # a single chunk costs less: the C terms
    assert abs(mac_count.xl_mem(16, 512, 64, C=2) - 21.0e6) / 21.0e6 < 5e-3   # "21M" floats of memory
