"""The one-grid front of the bf16 forward pass (gate logits, top-k, sort and the dense Q/K projection as one
cooperative grid of CTA pairs, sh_tc_front_kernel): that it is the path taken where the shape allows, that its
selections are those of the stand-alone gate entry point and of the oracle (Sec. 2.2: sigmoid gate, arg top-k),
that its sorted lists are valid, on the shapes that drive its branches (one or two 128-token blocks per CTA pair,
sequence lengths that are and are not a multiple of the TMA store's 32 rows, k = 2 pair buckets and k = 3 expert
buckets, a ragged last block), and that two layers may run their passes at the same time on two streams."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2312_07987_b200 import binding, inputs
from tests import parity_util as pu
from tests import test_gpu_parity as tp

pytestmark = pytest.mark.gpu


def _pair_id(a, b, E):
    a, b = np.minimum(a, b), np.maximum(a, b)
    return a * (2 * E - a - 1) // 2 + (b - a - 1)


def _cfg(name, B, T, M=1024, H=4, D=128, E=4, k=2, seed=811):
    return inputs.LayerConfig(name, inputs.DTYPE_BF16, B, T, M, H, D, E, k, seed=seed)


# (batch, seq, k): 8 blocks, one per pair | 80 blocks, two per pair | T not a multiple of 32 (epilogue without TMA
#  stores) and a ragged last block | k = 3: expert buckets, value rows cleared by the front
FRONT_SHAPES = [(2, 512, 2), (4, 2560, 2), (3, 1100, 2), (5, 300, 3)]


@pytest.mark.parametrize("B,T,k", FRONT_SHAPES)
def test_front_selections_and_lists(B, T, k):
    cfg = _cfg("front_bf16", B, T, k=k, E=4 if k == 2 else 5)
    inp = inputs.make_inputs(cfg)
    layer, x, y = pu.run_layer(inp)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    # front, V, attention, O (k = 3: one launch more behind them) - not the six or seven of the separate kernels
    assert binding.lib.sh_launch_count(layer.handle) == (4 if k == 2 else 5)
    N, H, E = B * T, cfg.n_heads, cfg.n_experts
    idx_f = layer.sh_debug_buffer("IDX").cpu().numpy().reshape(2, N, H, k).copy()
    gate_f = layer.sh_debug_buffer("GATE").cpu().numpy().reshape(2, N, H, k).copy()
    # the oracle's selections (bit-exact indices, gates to the logit tolerance of the tensor pipe)
    ref = pu.oracle_selection(inp, False)
    pu.check_selection(idx_f, gate_f, ref, N, 2e-5)
    # the stand-alone gate + sort entry point (kernels of their own) selects the same experts with the same gates
    idx_g, gate_g, off_g, lists_g = (t.cpu().numpy() for t in layer.sh_gate_topk(x))
    assert np.array_equal(idx_f.reshape(-1), idx_g.reshape(-1))
    assert np.allclose(gate_f.reshape(-1), gate_g.reshape(-1), rtol=0, atol=2e-6)   # (two UMMA shapes: the logits' sums may round apart)
    # the front's source-side lists: per head, every token once (k = 2: ordered by the pair of its experts, tokens
    # ascending inside a pair) or every selection once (other k: by expert, tokens ascending inside an expert)
    layer.sh_forward(x)                                             # (sh_gate_topk re-sorted by expert: run the front again)
    torch.cuda.synchronize()
    lists_f = layer.sh_debug_buffer("LISTS").cpu().numpy().reshape(-1)
    src = idx_f[0]                                                  # [N, H, k]
    for h in range(H):
        if k == 2:
            got = lists_f[h * N:(h + 1) * N]
            pid = _pair_id(src[:, h, 0].astype(np.int64), src[:, h, 1].astype(np.int64), E)
            want = np.lexsort((np.arange(N), pid))                 # stable: by pair, then by token
            assert np.array_equal(got, want), f"head {h}: pair-bucketed list differs"
        else:
            got = lists_f[h * N * k:(h + 1) * N * k]
            tok = np.repeat(np.arange(N), k)
            ex = src[:, h, :].reshape(-1)
            order = np.lexsort((tok, ex))
            assert np.array_equal(got, tok[order]), f"head {h}: expert-bucketed list differs"
    layer.sh_check_guards()
    layer.close()


@pytest.mark.parametrize("B,T,k", FRONT_SHAPES)
def test_front_shapes_against_the_oracle(B, T, k):
    cfg = _cfg("front_bf16", B, T, k=k, E=4 if k == 2 else 5, seed=823)
    tp.full_check(inputs.make_inputs(cfg), check_stage_buffers=(B * T <= 4096), batches=[0, B - 1] if B * T > 4096 else None)


def test_two_layers_run_their_passes_at_the_same_time():
    """Each front is a grid whose CTAs meet at a barrier; launched cooperatively, two of them on two streams take
    turns instead of holding each other's CTAs off the SMs."""
    cfg = _cfg("front_bf16", 4, 512, seed=829)
    inp_a, inp_b = inputs.make_inputs(cfg), inputs.make_inputs(dataclasses.replace(cfg, seed=830))
    la, xa, ya = pu.run_layer(inp_a)
    lb, xb, yb = pu.run_layer(inp_b)
    torch.cuda.synchronize()
    ya, yb = ya.clone(), yb.clone()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    outs = []
    for _ in range(20):
        with torch.cuda.stream(sa):
            oa = la.sh_forward(xa)
        with torch.cuda.stream(sb):
            ob = lb.sh_forward(xb)
        outs.append((oa, ob))
    torch.cuda.synchronize()
    assert la.sh_last_status() == 0 and lb.sh_last_status() == 0
    for oa, ob in outs:
        assert torch.equal(oa, ya) and torch.equal(ob, yb)
    la.close()
    lb.close()


# (batch, seq, d_model, heads, d_head, experts, k): the 2:4-sparse output projection | the CTA-pair kernel (k = 3) |
#  the single-CTA kernel (k = 4, 16 experts), a ragged last tile
F16_OUT_SHAPES = [(4, 512, 1024, 4, 128, 4, 2), (6, 256, 512, 2, 64, 5, 3), (2, 515, 512, 3, 128, 16, 4)]


@pytest.mark.parametrize("B,T,M,H,D,E,k", F16_OUT_SHAPES)
def test_fp16_output_is_the_fp32_output_rounded_once(B, T, M, H, D, E, k):
    cfg = inputs.LayerConfig("f16out_bf16", inputs.DTYPE_BF16, B, T, M, H, D, E, k, seed=907)
    inp = inputs.make_inputs(cfg)
    layer, x, y32 = pu.run_layer(inp)
    y32 = y32.clone()
    layer.sh_set_output_f16(True)
    y16 = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0 and y16.dtype == torch.float16
    if k == 2:        # (k >= 3: the value rows are summed in arrival order, two passes differ in the last bits)
        assert torch.equal(y16, y32.to(torch.float16))
    ref = pu.oracle_for(inp)
    err = pu.rel_rms_err(y16.float().cpu().numpy(), ref["y"])
    assert err < pu.TOL_Y[cfg.dtype], f"fp16 output: max-abs error / rms = {err:.3e}"
    layer.sh_set_output_f16(False)
    y = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert y.dtype == torch.float32
    if k == 2:
        assert torch.equal(y, y32)
    layer.sh_check_guards()
    layer.close()


def test_fp16_output_is_refused_where_no_kernel_writes_it():
    cfg = inputs.LayerConfig("f16out_f32", inputs.DTYPE_F32, 1, 64, 128, 2, 32, 4, 2, seed=908)
    layer, x, y = pu.run_layer(inputs.make_inputs(cfg))
    with pytest.raises(binding.SwitchHeadError):
        layer.sh_set_output_f16(True)
    layer.close()
