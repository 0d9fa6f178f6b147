"""Error paths and measurement aids of the library that need a GPU but no fault: a bounded wait that
runs out, the status block and its reset, the guard words behind the workspace buffers, and the
in-pass time stamps."""
import numpy as np
import pytest
import torch

from paper_2312_07987_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_the_layer_recovers():
    inp = inputs.make_inputs(inputs.CONFIGS["c4_262m_bf16"], batch=1)
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, inp.cfg.dtype)
    y0 = layer.sh_forward(x).clone()
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    # a one-thread kernel waits 2 ms on a barrier nothing signals, through the library's own bounded wait
    layer.sh_selftest(0, 2_000_000)
    assert layer.sh_last_status() == -6                    # SH_ERR_TIMEOUT
    w = layer.sh_status_block()
    assert w[0] == -6
    assert w[1] == 0 and w[2] == 0                          # block 0, thread 0 gave up
    assert w[3] != 0 and w[4] == 0                          # the barrier's shared-memory address, parity 0
    assert w[5] == 1 and w[6] == 32                         # grid of 1 block, 32 threads
    # the status word is sticky until it is cleared; after that the layer works as before (k = 2: bit for bit)
    layer.sh_clear_status()
    y1 = layer.sh_forward(x)
    torch.cuda.synchronize()
    assert layer.sh_last_status() == 0
    assert torch.equal(y0, y1)
    with pytest.raises(binding.SwitchHeadError):
        layer.sh_selftest(0, 5_000_000_000)                 # limits above a second are refused
    if not binding.lib.sh_is_debug_build():
        with pytest.raises(binding.SwitchHeadError):
            layer.sh_selftest(1, 3)                         # the index self-test exists in the debug library only
    layer.close()


def test_guard_words_notice_a_write_past_a_buffer():
    inp = inputs.make_inputs(inputs.CONFIGS["small_bf16"], batch=1)
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, inp.cfg.dtype)
    layer.sh_forward(x)
    layer.sh_check_guards()
    # overwrite (from the host side, inside the workspace tensor the test owns) the first word behind the Q buffer
    p, n = binding.ctypes.c_void_p(), binding.ctypes.c_size_t()
    binding._check(binding.lib.sh_debug_buffer(layer.handle, binding.BUF["Q"], binding.ctypes.byref(p), binding.ctypes.byref(n)))
    off = p.value - layer.workspace.data_ptr() + (n.value + 255) // 256 * 256
    saved = layer.workspace[off:off + 4].clone()
    assert saved.tolist() == [0xC5] * 4
    layer.workspace[off:off + 4] = 0
    with pytest.raises(binding.SwitchHeadError) as err:
        layer.sh_check_guards()
    assert err.value.code == -7 and "1 guard words" in str(err.value)
    layer.workspace[off:off + 4] = saved
    layer.sh_check_guards()
    layer.close()


@pytest.mark.parametrize("name,batch", [("c4_262m_bf16", None), ("small_bf16", None), ("long_ctx_bf16", 1)])
def test_stamped_forward_is_the_same_pass_with_a_consistent_timeline(name, batch):
    cfg = inputs.CONFIGS[name]
    inp = inputs.make_inputs(cfg, batch=batch)
    layer = binding.layer_from_inputs(inp)
    x = binding.to_device(inp.x, cfg.dtype)
    y0 = layer.sh_forward(x).clone()
    out = torch.empty_like(y0)
    st = layer.sh_forward_stamped(x, out)
    assert layer.sh_last_status() == 0
    if cfg.k <= 2:
        assert torch.equal(out, y0)
    else:
        rms = y0.double().pow(2).mean().sqrt().item()
        assert (out - y0).abs().max().item() / rms < 6e-3       # k >= 3: arrival order of the value sums
    assert {"gate", "qk_a", "v", "attn", "o"} <= set(st), st.keys()
    for k, (res, start, end) in st.items():
        assert res <= start <= end, (k, res, start, end)
        assert end - res < 50_000_000                        # tens of ms at most
    # data dependencies show in the device clock: the value experts start after the selections are sorted,
    # attention after V and Q/K, the output projection after attention
    slack = 2000                                             # ns: the clock ticks coarsely
    sort_end = st["sort"][2] if "sort" in st else st["gate"][2]
    assert st["v"][1] + slack >= sort_end
    assert st["attn"][1] + slack >= st["v"][2] and st["attn"][1] + slack >= st["qk_a"][2]
    assert st["o"][1] + slack >= st["attn"][2]
    layer.close()
