"""The allocation-free gate entry point against the regular one.

sh_noalloc_gate_topk serves callers that cannot call cudaMalloc (no workspace to hand over):
its scratch memory is a set of fixed arrays inside the library.  This test drives it through
the C ABI twice in a row - the second call with different tokens, so that anything left in
the shared arrays by the first call would show - and checks every output against
sh_gate_topk on the same inputs.  It lives in a file that pytest collects last."""
import numpy as np
import pytest
import torch

from paper_2312_07987_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def stacked_gate_weights(inp):
    """[2*H*E, M]: W_S^h and W_D^h transposed, row (side*H + h)*E + e."""
    ws = np.transpose(inp.Ws, (0, 2, 1)).reshape(-1, inp.cfg.d_model)
    wd = np.transpose(inp.Wd, (0, 2, 1)).reshape(-1, inp.cfg.d_model)
    return np.concatenate([ws, wd], axis=0)


def canon(idx, gate):
    order = torch.argsort(idx.long(), dim=-1, stable=True)
    return torch.gather(idx.long(), -1, order), torch.gather(gate, -1, order)


@pytest.mark.parametrize("name,batch,gate_tol", [("tiny_f32", None, 0.0), ("small_bf16", 3, 2e-5)])
def test_noalloc_gate_topk_matches_regular_entry_point_twice(name, batch, gate_tol):
    cfg = inputs.CONFIGS[name]
    inp = inputs.make_inputs(cfg, batch=batch)
    layer = binding.layer_from_inputs(inp)
    H, E, k, M = cfg.n_heads, cfg.n_experts, cfg.k, cfg.d_model
    wg = binding.to_device(stacked_gate_weights(inp), cfg.dtype)
    x0 = binding.to_device(inp.x, cfg.dtype)
    perm = torch.randperm(x0.shape[0] * x0.shape[1], device="cuda")
    x1 = x0.reshape(-1, M)[perm].reshape(x0.shape).contiguous()      # same rows, other order: margins kept
    for x in (x0, x1):
        ref = [t.clone() for t in layer.sh_gate_topk(x)]
        got = binding.sh_noalloc_gate_topk(cfg.dtype, x.reshape(-1, M), wg, None, H, E, k)
        torch.cuda.synchronize()
        ri, rg = canon(ref[0], ref[1])
        gi, gg = canon(got[0], got[1])
        assert torch.equal(ri, gi), "selected experts differ"
        assert (rg - gg).abs().max().item() <= gate_tol, "gate values differ"
        assert torch.equal(ref[2], got[2]), "offsets differ"
        assert torch.equal(ref[3], got[3]), "token lists differ"
    # and against the fp64 oracle directly (selections, gates, offsets, lists of the unpermuted tokens)
    from tests import parity_util as pu
    got = binding.sh_noalloc_gate_topk(cfg.dtype, x0.reshape(-1, M), wg, None, H, E, k)
    torch.cuda.synchronize()
    want = pu.oracle_selection(inp)
    pu.check_selection(got[0].cpu().numpy(), got[1].cpu().numpy(), want, x0.shape[0] * x0.shape[1], max(gate_tol, 1e-6))
    pu.check_lists(got[2].cpu().numpy(), got[3].cpu().numpy(), want)
    layer.close()


def test_noalloc_gate_topk_with_bias_and_size_limits():
    cfg = inputs.LayerConfig("bias", inputs.DTYPE_F32, 2, 70, 128, 2, 32, 8, 3, seed=11, zipf_bias=1.2)
    inp = inputs.make_inputs(cfg)
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, cfg.dtype)
    wg = binding.to_device(stacked_gate_weights(inp), cfg.dtype)
    bias = torch.from_numpy(np.concatenate([inp.bias_s.ravel(), inp.bias_d.ravel()])).cuda()
    ref = layer.sh_gate_topk(x)
    got = binding.sh_noalloc_gate_topk(cfg.dtype, x.reshape(-1, cfg.d_model), wg, bias, cfg.n_heads, cfg.n_experts, cfg.k)
    torch.cuda.synchronize()
    for a, b in zip(ref, got):
        assert torch.equal(a, b)
    big = torch.zeros((16385, 128), device="cuda")
    with pytest.raises(binding.SwitchHeadError) as err:
        binding.sh_noalloc_gate_topk(binding.SH_F32, big, wg, None, cfg.n_heads, cfg.n_experts, cfg.k)
    assert "limited to" in str(err.value)
    layer.close()
