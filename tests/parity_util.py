"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding and
the fp64 oracle on the same seeded inputs, and compare stage by stage."""
import numpy as np
import torch

from oracle.switchhead_oracle import switchhead_forward
from paper_2312_07987_b200 import binding, inputs

# Tolerances.  Outputs: max-abs error relative to the RMS of the oracle output, 1e-4 for the
# fp32 configuration and 2e-2 for bf16 storage (fp32 accumulation, fp16 intermediates).
TOL_Y = {inputs.DTYPE_F32: 1e-4, inputs.DTYPE_BF16: 2e-2}


def oracle_for(inp, batches=None, rope_base=None, shared_selection=False, causal=True):
    x = inp.x if batches is None else inp.x[batches]
    return switchhead_forward(x, inp.Wq, inp.Wk, inp.Wv, inp.Wo, inp.Ws, inp.Wd, inp.cfg.k,
                              inp.bias_s, inp.bias_d, causal=causal, rope_base=rope_base,
                              shared_selection=shared_selection)


def oracle_selection(inp, shared_selection=False):
    """Selections, gates, offsets and token lists of ALL tokens of inp.x from the oracle's gate and
    bucket-sort steps alone (no attention: cheap at any size); same keys as the full oracle's stages."""
    from oracle.switchhead_oracle import bucket_lists, gate_and_select
    cfg = inp.cfg
    x2d = inp.x.reshape(-1, cfg.d_model).astype(np.float64)
    out = {}
    for side, W, b in (("S", inp.Ws, inp.bias_s), ("D", inp.Ws if shared_selection else inp.Wd,
                                                   inp.bias_s if shared_selection else inp.bias_d)):
        _, _, idx, gate = gate_and_select(x2d, W.astype(np.float64), b, cfg.k)
        off, lists = bucket_lists(idx, cfg.n_experts)
        out["idx" + side], out["gate" + side], out["offsets" + side], out["lists" + side] = idx, gate, off, lists
    return out


def rel_rms_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / np.sqrt((ref ** 2).mean()))


def check_selection(idx_gpu, gate_gpu, ref, N, gate_tol=1e-6):
    """idx_gpu, gate_gpu [2, N, H, k] (numpy); ref: oracle stages for the same N tokens.
    The selected SET must match bit-exactly; gates are compared per expert."""
    for side, (ik, gk) in enumerate((("idxS", "gateS"), ("idxD", "gateD"))):
        gi = idx_gpu[side].astype(np.int64)
        order = np.argsort(gi, axis=-1, kind="stable")
        gi_sorted = np.take_along_axis(gi, order, -1)
        gg_sorted = np.take_along_axis(gate_gpu[side].astype(np.float64), order, -1)
        ri = ref[ik].astype(np.int64)
        rorder = np.argsort(ri, axis=-1, kind="stable")
        ri_sorted = np.take_along_axis(ri, rorder, -1)
        rg_sorted = np.take_along_axis(ref[gk], rorder, -1)
        assert np.array_equal(gi_sorted, ri_sorted), f"side {side}: selected expert sets differ"
        gerr = np.abs(gg_sorted - rg_sorted).max()
        assert gerr <= gate_tol, f"side {side}: gate values differ by {gerr:.3e}"


def check_lists(off_gpu, lists_gpu, ref):
    for side, (ok, lk) in enumerate((("offsetsS", "listsS"), ("offsetsD", "listsD"))):
        assert np.array_equal(off_gpu[side], ref[ok]), f"side {side}: offsets differ"
        assert np.array_equal(lists_gpu[side], ref[lk]), f"side {side}: token lists differ"


def run_layer(inp, device="cuda", shared_selection=False):
    cfg = inp.cfg
    layer = binding.layer_from_inputs(inp, device=device, shared_selection=shared_selection)
    x = binding.to_device(inp.x, cfg.dtype, device)
    y = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0, f"device status word reports a failed kernel: status block {layer.sh_status_block()}"
    return layer, x, y


def check_stages(layer, ref, cfg, batches=None):
    """Q, K, V, Ahat of the CUDA path against the oracle (fp16 storage on the bf16 path)."""
    D = cfg.d_head
    qs = np.log2(np.e) / np.sqrt(D)
    sel = slice(None) if batches is None else batches
    rel = 2e-5 if cfg.dtype == inputs.DTYPE_F32 else 2.0 ** -10
    for name, key, scale in (("Q", "Q", qs), ("K", "K", 1.0), ("V", "V", 1.0)):
        got = layer.sh_debug_buffer(name).float().cpu().numpy().astype(np.float64)   # [B,H,T,D]
        got = got.transpose(0, 2, 1, 3)[sel]
        want = ref[key] * scale
        # V sums k gate-weighted fp16 contributions, each addition rounding to fp16
        r = rel * (cfg.k if name == "V" and cfg.dtype != inputs.DTYPE_F32 else 1)
        tol = r * np.abs(want) + max(3e-4, r) * np.sqrt((want ** 2).mean())
        bad = np.abs(got - want) > tol
        assert not bad.any(), f"{name}: {bad.sum()} elements off, worst {np.abs(got - want).max():.3e}"
    got = layer.sh_debug_buffer("AHAT").float().cpu().numpy().astype(np.float64)
    B, T, H, _ = ref["Ahat"].shape
    got = got.reshape(-1, T, H, D)[sel]
    want = ref["Ahat"]
    # Ahat inherits V's rounding (rows near t = 0 are single V rows) plus its own fp16 store
    # and the effect of fp16 Q, K on the softmax weights (logit error ~ 2^-11 |q.k|)
    r = 1e-2 if cfg.dtype != inputs.DTYPE_F32 else 4e-5
    tol = r * (np.abs(want) + 2 * np.sqrt((want ** 2).mean()))
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"Ahat: {bad.sum()} elements off, worst {np.abs(got - want).max():.3e}"
