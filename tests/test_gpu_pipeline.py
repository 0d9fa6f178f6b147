"""GPU test of the host-fed pipeline: copies overlapped with the forward pass on three streams
must give, step by step, what a plain forward pass of that step's input gives."""
import numpy as np
import pytest
import torch

from paper_2312_07987_b200 import binding, inputs, pipeline

pytestmark = pytest.mark.gpu


def test_host_fed_steps_match_direct_forward():
    # k = 2: the two-way fp16 sums of the value stage do not depend on arrival order, so every pass
    # over the same input gives the same bits
    inp = inputs.make_inputs(inputs.CONFIGS["c4_262m_bf16"], batch=2)
    layer = binding.layer_from_inputs(inp)
    x0 = binding.to_device(inp.x, inp.cfg.dtype)
    xs = [x0, (x0.float() * 0.5).to(x0.dtype), (x0.float().flip(1)).to(x0.dtype).contiguous()]
    want = [layer.sh_forward(x).clone().cpu() for x in xs]
    torch.cuda.synchronize()
    pipe = pipeline.HostFedLayer(layer, x0)
    xh = [x.cpu().pin_memory() for x in xs]
    n_steps = 9
    outh = [torch.empty(inp.x.shape, dtype=torch.float32).pin_memory() for _ in range(n_steps)]
    for i in range(n_steps):
        pipe.step(xh[i % 3], outh[i])
    pipe.wait()
    assert layer.sh_last_status() == 0
    for i in range(n_steps):
        ref = want[i % 3]
        assert torch.equal(outh[i], ref), f"step {i}: max abs difference {float((outh[i] - ref).abs().max()):.3e}"
    layer.close()
