"""Query / key experts (sh_create_moe_qk, paper Sec. 2.2: K^h with the source side's selection, Q^h with the
destination side's) on the GPU, fp32 configuration, against the oracle: output, stages and selections."""
import numpy as np
import pytest
import torch

from paper_2312_07987_b200 import binding, inputs
from tests import parity_util as pu
from tests.test_gpu_parity import full_check

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("moe_q,moe_k", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("T,B,M,H,D,E,k", [(64, 1, 128, 2, 32, 4, 2), (150, 2, 192, 3, 40, 5, 3), (33, 3, 64, 1, 64, 2, 1)])
def test_moe_qk_f32_matches_the_oracle(moe_q, moe_k, T, B, M, H, D, E, k):
    cfg = inputs.LayerConfig("moe_qk", inputs.DTYPE_F32, B, T, M, H, D, E, k, seed=500 + T, moe_q=moe_q, moe_k=moe_k)
    full_check(inputs.make_inputs(cfg))


def test_moe_qk_f32_with_shared_selection_noncausal_and_gate_bias():
    cfg = inputs.LayerConfig("moe_qk_sh", inputs.DTYPE_F32, 2, 70, 128, 2, 32, 6, 2, seed=611, zipf_bias=1.2, moe_q=True, moe_k=True)
    inp = inputs.make_inputs(cfg)
    full_check(inp, shared_selection=True)
    layer = binding.layer_from_inputs(inp)
    layer.sh_set_causal(False)
    x = binding.to_device(inp.x, cfg.dtype)
    y = layer.sh_forward(x).cpu().numpy()
    ref = pu.oracle_for(inp, causal=False)
    assert pu.rel_rms_err(y, ref["y"]) < pu.TOL_Y[cfg.dtype]
    layer.close()


def test_moe_qk_f32_with_a_cache_and_relative_positions():
    from oracle.switchhead_oracle import switchhead_xl_forward
    cfg = inputs.LayerConfig("moe_qk_xl", inputs.DTYPE_F32, 2, 48 + 40, 128, 2, 32, 4, 2, seed=620, moe_q=True, moe_k=True)
    inp = inputs.make_inputs(cfg)
    Tc = 48
    layer = binding.layer_from_inputs(inp, cache_len=Tc)
    rg = np.random.default_rng(5)
    Wr = (rg.standard_normal((cfg.n_heads, cfg.d_model, cfg.d_head)) / np.sqrt(cfg.d_model)).astype(np.float32)
    u = (0.5 * rg.standard_normal((cfg.n_heads, cfg.d_head))).astype(np.float32)
    v = (0.5 * rg.standard_normal((cfg.n_heads, cfg.d_head))).astype(np.float32)
    layer.sh_set_xl_positions(torch.from_numpy(Wr).cuda(), torch.from_numpy(u).cuda(), torch.from_numpy(v).cuda())
    y = layer.sh_forward(binding.to_device(inp.x, cfg.dtype)).cpu().numpy()
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    ref = switchhead_xl_forward(inp.x[:, Tc:], inp.x[:, :Tc], inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, cfg.k,
                                Wr=Wr, u=u, v=v)
    assert pu.rel_rms_err(y, ref["y"]) < pu.TOL_Y[cfg.dtype]
    layer.close()


@pytest.mark.parametrize("moe_q,moe_k", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("T,B,M,H,D,E,k", [(300, 3, 256, 2, 128, 4, 2), (1000, 2, 384, 4, 100, 8, 2), (129, 1, 128, 2, 128, 2, 2)])
def test_moe_qk_bf16_matches_the_oracle(moe_q, moe_k, T, B, M, H, D, E, k):
    # tensor-core path: an expert projection of keys / queries is the pair-tiled value kernel with the key /
    # query experts' weights, on the source / destination side's (head, expert pair) tiles
    cfg = inputs.LayerConfig("moe_qk_bf16", inputs.DTYPE_BF16, B, T, M, H, D, E, k, seed=700 + T, moe_q=moe_q, moe_k=moe_k)
    full_check(inputs.make_inputs(cfg))


def test_moe_qk_bf16_odd_heads_both_experts_shared_selection_and_cache():
    cfg = inputs.LayerConfig("moe_qk_bf16_h3", inputs.DTYPE_BF16, 2, 260, 256, 3, 128, 4, 2, seed=731, moe_q=True, moe_k=True)
    inp = inputs.make_inputs(cfg)
    full_check(inp)
    full_check(inp, shared_selection=True)
    from oracle.switchhead_oracle import switchhead_xl_forward
    cfg = inputs.LayerConfig("moe_qk_bf16_xl", inputs.DTYPE_BF16, 2, 128 + 256, 256, 2, 128, 4, 2, seed=732, moe_q=True, moe_k=True)
    inp = inputs.make_inputs(cfg)
    layer = binding.layer_from_inputs(inp, cache_len=128)
    y = layer.sh_forward(binding.to_device(inp.x, cfg.dtype)).cpu().numpy()
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    ref = switchhead_xl_forward(inp.x[:, 128:], inp.x[:, :128], inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, cfg.k)
    assert pu.rel_rms_err(y, ref["y"]) < pu.TOL_Y[cfg.dtype]
    layer.sh_check_guards()
    layer.close()


def test_moe_qk_is_refused_for_bf16_shapes_the_pair_kernel_does_not_serve_and_with_rope():
    for args, kw in (((256, 2, 128, 4, 3), dict(moe_k=True)), ((256, 3, 128, 4, 2), dict(moe_q=True)), ((256, 2, 128, 16, 2), dict(moe_q=True, moe_k=True))):
        Lb = binding.Layer(*args, **kw)
        with pytest.raises(binding.SwitchHeadError):
            Lb.sh_configure(inputs.DTYPE_BF16, 1, 128)
        Lb.close()
    L = binding.Layer(256, 2, 64, 4, 2, moe_q=True)
    with pytest.raises(binding.SwitchHeadError) as e:
        L.sh_configure(inputs.DTYPE_BF16, 1, 128)
    assert "fp32 configuration" in str(e.value)
    L.sh_configure(inputs.DTYPE_F32, 1, 64)
    with pytest.raises(binding.SwitchHeadError):
        L.sh_set_rope(10000.0)
    L.close()
