"""Backward pass (sh_backward, fp32 configuration) on the GPU against the backward oracle: dx and the gradients of
all six weight tensors, on the tiny workload and on shapes with a padded d_head, one and three selections,
without the causal mask; argument checks."""
import numpy as np
import pytest
import torch

from oracle.switchhead_backward import switchhead_backward
from paper_2312_07987_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-4          # max-abs error / RMS of the gradient: fp32 products, sums and atomics against fp64


def check(cfg, causal=True, batch=None):
    inp = inputs.make_inputs(cfg, batch=batch)
    layer = binding.layer_from_inputs(inp)
    if not causal:
        layer.sh_set_causal(False)
    x = binding.to_device(inp.x, cfg.dtype)
    rg = np.random.default_rng(cfg.seed + 1)
    G = rg.standard_normal(inp.x.shape).astype(np.float32)
    layer.sh_forward(x)
    got = layer.sh_backward(x, torch.from_numpy(G).cuda())
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    ref = switchhead_backward(inp.x, inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, cfg.k, G, inp.bias_s, inp.bias_d, causal=causal)
    for name in ("dx", "dWq", "dWk", "dWv", "dWo", "dWs", "dWd"):
        a, r = got[name].cpu().numpy().astype(np.float64), ref[name]
        err = np.abs(a - r).max() / np.sqrt((r ** 2).mean())
        assert err < TOL, (name, err)
    layer.sh_check_guards()
    layer.close()


def test_backward_tiny_f32():
    check(inputs.CONFIGS["tiny_f32"])


@pytest.mark.parametrize("T,B,M,H,D,E,k,causal", [(70, 2, 128, 2, 40, 5, 3, True), (33, 3, 64, 3, 64, 4, 1, False), (150, 1, 192, 1, 132, 6, 2, True)])
def test_backward_shapes(T, B, M, H, D, E, k, causal):
    check(inputs.LayerConfig("bw", inputs.DTYPE_F32, B, T, M, H, D, E, k, seed=900 + T, zipf_bias=1.2 if E == 5 else 0.0), causal=causal)


def test_backward_argument_checks():
    inp = inputs.make_inputs(inputs.CONFIGS["tiny_f32"])
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, inp.cfg.dtype)
    G = torch.zeros(inp.x.shape, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.SwitchHeadError):          # no forward pass on this x yet
        layer.sh_backward(x, G)
    layer.sh_forward(x)
    layer.sh_backward(x, G)
    layer.close()
    bf = binding.layer_from_inputs(inputs.make_inputs(inputs.CONFIGS["small_bf16"], batch=1))
    xb = binding.to_device(inputs.make_inputs(inputs.CONFIGS["small_bf16"], batch=1).x, inputs.DTYPE_BF16)
    bf.sh_forward(xb)
    with pytest.raises(binding.SwitchHeadError):          # tensor-core path: forward only
        bf.sh_backward(xb, torch.zeros((1, 256, 512), dtype=torch.float32, device="cuda"))
    bf.close()
