"""Host-side checks of the seeded synthetic input generator."""
import numpy as np

from paper_2312_07987_b200 import inputs as I


def test_bf16_rounding_is_nearest_even():
    a = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -3.1415926, 1e-30], dtype=np.float32)
    r = I.round_to_bf16(a)
    assert r[0] == 1.0 and r[1] == 1.0                       # tie -> even (1.0)
    assert r[2] == np.float32(1.0 + 2 ** -7)
    assert r[3] == np.float32(1.0 + 2 ** -6)                 # tie -> even (odd+1)
    assert abs(r[4] + 3.140625) < 1e-6
    bits = I.bf16_bits(r)
    assert bits.dtype == np.uint16 and bits[0] == 0x3F80


def test_inputs_are_deterministic_representable_and_gapped():
    cfg = I.CONFIGS["small_bf16"]
    a = I.make_inputs(cfg, batch=2)
    b = I.make_inputs(cfg, batch=2)
    for k_, v in a.arrays().items():
        if v is None:
            continue
        assert np.array_equal(v, b.arrays()[k_])
        assert v.dtype == np.float32
        assert np.array_equal(I.round_to_bf16(v), v)
    x2 = a.x.reshape(-1, cfg.d_model)
    for W in (a.Ws, a.Wd):
        assert I._rank_gap(x2, W, None, cfg.k).min() >= cfg.min_gap
    full = I.make_inputs(cfg, batch=1)
    assert np.array_equal(full.Wv, a.Wv)                     # weights do not depend on batch
    assert 0.9 < x2.std() < 1.1


def test_zipf_bias_profile_and_shapes():
    cfg = I.CONFIGS["wide_skew_bf16"]
    a = I.make_inputs(cfg, batch=1, seq=64)
    assert a.bias_s.shape == (cfg.n_heads, cfg.n_experts) and a.bias_s.dtype == np.float32
    assert np.allclose(a.bias_s.mean(axis=1), 0, atol=1e-6)
    assert np.allclose(np.sort(a.bias_s, axis=1)[:, -1] - np.sort(a.bias_s, axis=1)[:, 0],
                       1.2 * np.log(16), atol=1e-5)
    assert a.Wv.shape == (8, 16, 2048, 128) and a.Wo.shape == (8, 16, 128, 2048)


def test_useful_flop_matches_hand_count():
    f = I.useful_flop(I.CONFIGS["c4_262m_bf16"])
    assert abs(f["total"] / 1e9 - 55.83) < 0.01
    f = I.useful_flop(I.CONFIGS["long_ctx_bf16"])
    assert abs(f["total"] / 1e9 - 171.80) < 0.01
