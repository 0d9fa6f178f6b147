"""GPU parity of the layer with a Transformer-XL context (sh_configure_xl) against the oracle's
switchhead_xl_forward without the relative-position term: keys, values and the source side over
[cache; chunk], queries, destination side and output over the chunk."""
import numpy as np
import pytest
import torch

from oracle.switchhead_oracle import switchhead_xl_forward
from paper_2312_07987_b200 import binding, inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def xl_check(cfg, cache_len, batches=None):
    """cfg.seq = cache_len + chunk length: the inputs' sequences are [cache; chunk]."""
    inp = inputs.make_inputs(cfg)
    T = cfg.seq - cache_len
    layer = binding.layer_from_inputs(inp, cache_len=cache_len)
    x = binding.to_device(inp.x, cfg.dtype)
    y = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    assert tuple(y.shape) == (inp.x.shape[0], T, cfg.d_model)
    sel = slice(None) if batches is None else batches
    xs = inp.x[sel]
    ref = switchhead_xl_forward(xs[:, cache_len:], xs[:, :cache_len], inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd,
                                cfg.k, inp.bias_s, inp.bias_d)
    err = pu.rel_rms_err(y.cpu().numpy()[sel], ref["y"])
    assert err < pu.TOL_Y[cfg.dtype], f"output max-abs error / rms = {err:.3e}"
    # stage buffers: V over the whole context, Ahat for the chunk's tokens
    D = cfg.d_head
    rel = 2e-5 if cfg.dtype == inputs.DTYPE_F32 else 2.0 ** -10 * cfg.k
    V = layer.sh_debug_buffer("V").float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3)[sel]
    tolv = rel * np.abs(ref["V"]) + max(3e-4, rel) * np.sqrt((ref["V"] ** 2).mean())
    assert not (np.abs(V - ref["V"]) > tolv).any(), "V differs"
    A = layer.sh_debug_buffer("AHAT").float().cpu().numpy().astype(np.float64)
    A = A.reshape(inp.x.shape[0], cfg.seq, cfg.n_heads, D)[sel][:, cache_len:]
    r = 1e-2 if cfg.dtype != inputs.DTYPE_F32 else 4e-5
    tola = r * (np.abs(ref["Ahat"]) + 2 * np.sqrt((ref["Ahat"] ** 2).mean()))
    assert not (np.abs(A - ref["Ahat"]) > tola).any(), "Ahat differs"
    layer.sh_check_guards()
    layer.close()
    return err


@pytest.mark.parametrize("T,Tc,B,E,k,H,D,M", [(64, 64, 1, 4, 2, 2, 32, 128), (17, 5, 3, 5, 3, 2, 64, 128), (1, 40, 2, 3, 1, 1, 32, 64),
                                                (100, 200, 1, 8, 2, 3, 32, 64)])
def test_xl_context_f32(T, Tc, B, E, k, H, D, M):
    xl_check(inputs.LayerConfig("xl_f32", inputs.DTYPE_F32, B, Tc + T, M, H, D, E, k, seed=400 + T), Tc)


@pytest.mark.parametrize("T,Tc,B,E,k,H,D,M", [(128, 128, 2, 4, 2, 2, 64, 256),     # C = 2, one tile each
                                                (256, 256, 3, 5, 3, 2, 64, 512),     # the 47M-model shape with its cache (single-CTA... k = 3: pair kernel)
                                                (384, 128, 1, 4, 2, 3, 128, 384),    # odd number of query tiles
                                                (128, 512, 2, 16, 4, 2, 128, 256)])  # long cache, k = 4: single-CTA output kernel
def test_xl_context_bf16(T, Tc, B, E, k, H, D, M):
    xl_check(inputs.LayerConfig("xl_bf16", inputs.DTYPE_BF16, B, Tc + T, M, H, D, E, k, seed=500 + T), Tc)


def test_xl_context_c4_262m_shape_with_its_cache():
    # the 262M-scale model as the paper runs it: 512-token chunks with a 512-token cache (C = 2)
    c = inputs.CONFIGS["c4_262m_bf16"]
    cfg = inputs.LayerConfig("c4_xl", c.dtype, 4, 2 * c.seq, c.d_model, c.n_heads, c.d_head, c.n_experts, c.k, seed=c.seed)
    xl_check(cfg, c.seq)


def test_cache_split_identity_on_the_gpu():
    """One causal pass over 2T tokens against two passes of T tokens, the second with the first chunk's
    input as its cache: the same outputs for the second chunk (within the tolerance of the 16-bit
    intermediates; the two runs tile the work differently)."""
    c = inputs.CONFIGS["c4_262m_bf16"]
    T = 256
    cfg = inputs.LayerConfig("split", c.dtype, 2, 2 * T, c.d_model, c.n_heads, c.d_head, c.n_experts, c.k, seed=77)
    inp = inputs.make_inputs(cfg)
    x = binding.to_device(inp.x, cfg.dtype)
    whole = binding.layer_from_inputs(inp)
    y_whole = whole.sh_forward(x)[:, T:].clone()
    whole.close()
    xl = binding.layer_from_inputs(inp, cache_len=T)
    y_xl = xl.sh_forward(x)
    torch.cuda.synchronize()
    assert xl.sh_last_status() == 0
    rms = y_whole.double().pow(2).mean().sqrt().item()
    assert (y_xl - y_whole).abs().max().item() / rms < 2e-3
    xl.close()


def test_xl_argument_checks():
    L = binding.Layer(256, 2, 64, 4, 2)
    with pytest.raises(binding.SwitchHeadError) as e:
        L.sh_configure(binding.SH_BF16, 1, 128, cache_len=100)      # bf16: multiples of 128
    assert "multiples of 128" in str(e.value)
    L.sh_configure(binding.SH_BF16, 1, 128, cache_len=128)
    with pytest.raises(binding.SwitchHeadError):
        L.sh_set_rope(10000.0)
    L.close()
    Ld = binding.Layer(256, 2, 64, dense=True)
    with pytest.raises(binding.SwitchHeadError):
        Ld.sh_configure(binding.SH_F32, 1, 16, cache_len=16)
    Ld.close()


@pytest.mark.parametrize("T,Tc,B,E,k,H,D,M", [(64, 64, 1, 4, 2, 2, 32, 128), (33, 0, 2, 4, 2, 2, 32, 64), (17, 45, 2, 5, 3, 3, 22, 128),
                                                (130, 70, 1, 3, 1, 2, 64, 64)])
def test_xl_relative_positions_f32(T, Tc, B, E, k, H, D, M):
    """The full Transformer-XL layer of the paper's main models in the fp32 configuration: cache plus the
    relative-position term (q + u).k + (q + v).r_dist, against the oracle."""
    cfg = inputs.LayerConfig("xl_pos", inputs.DTYPE_F32, B, Tc + T, M, H, D, E, k, seed=600 + T)
    inp = inputs.make_inputs(cfg)
    rng = np.random.default_rng(601)
    Wr = (rng.standard_normal((H, M, D)) / np.sqrt(M)).astype(np.float32)
    u = (0.5 * rng.standard_normal((H, D))).astype(np.float32)
    v = (0.5 * rng.standard_normal((H, D))).astype(np.float32)
    layer = binding.layer_from_inputs(inp, cache_len=Tc)
    x = binding.to_device(inp.x, cfg.dtype)
    y_plain = layer.sh_forward(x).clone()
    layer.sh_set_xl_positions(*(torch.from_numpy(a).cuda() for a in (Wr, u, v)))
    y = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    ref = switchhead_xl_forward(inp.x[:, Tc:], inp.x[:, :Tc] if Tc else None, inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd,
                                cfg.k, inp.bias_s, inp.bias_d, Wr=Wr, u=u, v=v)
    err = pu.rel_rms_err(y.cpu().numpy(), ref["y"])
    assert err < 1e-4, f"output max-abs error / rms = {err:.3e}"
    assert not torch.allclose(y, y_plain, rtol=1e-3, atol=1e-3), "the position term changed nothing"
    layer.sh_set_xl_positions(None)                       # off again: the plain scores
    y_off = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert pu.rel_rms_err(y_off.cpu().numpy(), y_plain.cpu().numpy()) < 1e-5
    layer.close()


@pytest.mark.parametrize("T,Tc,B,E,k,H,D,M", [(128, 128, 2, 4, 2, 2, 64, 256), (256, 256, 2, 5, 3, 2, 64, 512),
                                                (384, 128, 1, 4, 2, 3, 128, 384), (128, 512, 1, 16, 4, 2, 128, 256),
                                                (1024, 1024, 1, 4, 2, 1, 128, 256)])   # the last: 2048 keys, the whole-S attention kernel
def test_xl_relative_positions_bf16(T, Tc, B, E, k, H, D, M):
    """The paper's main configuration on the tensor-core path: cache + Transformer-XL position term (score bias
    = Q R^T skewed to key order + v.r + u.k, added to the S tiles by the attention kernel)."""
    cfg = inputs.LayerConfig("xl_pos16", inputs.DTYPE_BF16, B, Tc + T, M, H, D, E, k, seed=700 + T)
    inp = inputs.make_inputs(cfg)
    rng = np.random.default_rng(701)
    Wr = (rng.standard_normal((H, M, D)) / np.sqrt(M)).astype(np.float32)
    u = (0.5 * rng.standard_normal((H, D))).astype(np.float32)
    v = (0.5 * rng.standard_normal((H, D))).astype(np.float32)
    layer = binding.layer_from_inputs(inp, cache_len=Tc)
    x = binding.to_device(inp.x, cfg.dtype)
    y_plain = layer.sh_forward(x).clone()
    layer.sh_set_xl_positions(*(torch.from_numpy(a).cuda() for a in (Wr, u, v)))
    y = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    ref = switchhead_xl_forward(inp.x[:, Tc:], inp.x[:, :Tc], inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd,
                                cfg.k, inp.bias_s, inp.bias_d, Wr=Wr, u=u, v=v)
    err = pu.rel_rms_err(y.cpu().numpy(), ref["y"])
    assert err < pu.TOL_Y[cfg.dtype], f"output max-abs error / rms = {err:.3e}"
    A = layer.sh_debug_buffer("AHAT").float().cpu().numpy().astype(np.float64).reshape(B, cfg.seq, H, D)[:, Tc:]
    tola = 1e-2 * (np.abs(ref["Ahat"]) + 2 * np.sqrt((ref["Ahat"] ** 2).mean()))
    assert not (np.abs(A - ref["Ahat"]) > tola).any(), "Ahat differs"
    assert not torch.allclose(y, y_plain, rtol=1e-2, atol=1e-2), "the position term changed nothing"
    layer.sh_set_xl_positions(None)
    y_off = layer.sh_forward(x)
    torch.cuda.synchronize()
    if cfg.k <= 2:
        assert torch.equal(y_off, y_plain)
    layer.sh_check_guards()
    layer.close()


def test_xl_relative_positions_bf16_need_a_cache():
    L = binding.Layer(256, 2, 64, 4, 2)
    L.sh_configure(binding.SH_BF16, 1, 128)
    with pytest.raises(binding.SwitchHeadError) as e:
        L.sh_set_xl_positions(torch.zeros((2, 256, 64), device="cuda"))
    assert "cache" in str(e.value)
    L.close()
