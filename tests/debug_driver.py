"""Parity cases run against the DEBUG library (built with -DSH_DEBUG) in a process of their own.

The library is chosen when the binding is imported (environment variable SWITCHHEAD_LIB), and the
debug library reads its launch-structure switches from the environment when the weights are set, so
tests/test_gpu_debug_library.py starts this module as a child process with both in place:

    python -m tests.debug_driver CASE

Prints DEBUG_DRIVER_OK as its last line when every check of the case passed."""
import os
import sys

import torch

from paper_2312_07987_b200 import binding, inputs


def main(case: str) -> None:
    assert binding.lib.sh_is_debug_build() == 1, "this driver is meant for the debug library"
    from tests import test_gpu_parity as tp
    if case == "switches":
        # whatever switches the parent put into the environment: the numbers must not change
        tp.full_check(inputs.make_inputs(inputs.CONFIGS["small_bf16"]))
        tp.full_check(inputs.make_inputs(inputs.CONFIGS["c4_262m_bf16"], batch=3), check_stage_buffers=False)
        if "SH_SIMT_STAGES" not in os.environ:            # (the CUDA-core output stage sums with atomics: not bit for bit)
            tp.test_back_to_back_forward_passes_share_the_tile_counter_cleanly()
    elif case == "edges":
        # every index the kernels read from memory is range-checked here; a failed check sets the status
        # word, which full_check asserts to be zero - on ragged, tiny and skewed shapes
        for T, B, E, k, H, D in [(1, 2, 4, 2, 2, 64), (100, 3, 5, 3, 2, 64), (129, 1, 4, 4, 1, 128), (515, 1, 16, 4, 3, 128)]:
            tp.full_check(inputs.make_inputs(inputs.LayerConfig("edge_bf16", inputs.DTYPE_BF16, B, T, 256, H, D, E, k, seed=200 + T)))
        for M, T, B, E, k, H, D in [(384, 300, 3, 6, 2, 2, 128), (1024, 1100, 20, 4, 2, 2, 128), (512, 257, 1, 32, 4, 4, 64)]:
            tp.full_check(inputs.make_inputs(inputs.LayerConfig("edge_bf16_wide", inputs.DTYPE_BF16, B, T, M, H, D, E, k, seed=300 + T)))
        for cfg in tp._random_bf16_configs(4, 11):
            tp.full_check(inputs.make_inputs(cfg), check_stage_buffers=False)
    elif case == "sparse_o":
        # the shapes the 2:4-sparse output projection serves (or, with SH_O_MASKED, the masked kernel on them)
        for cfg in tp.SPARSE_O_CONFIGS:
            tp.full_check(inputs.make_inputs(cfg), check_stage_buffers=False)
    elif case == "moe_qk":
        # key / query experts on the pair-tiled kernel: both sides bucketed by expert pair, every list entry,
        # tile field and expert index range-checked
        for moe_q, moe_k in ((True, False), (False, True), (True, True)):
            cfg = inputs.LayerConfig("moe_qk_dbg", inputs.DTYPE_BF16, 2, 300, 256, 2, 128, 8, 2, seed=741, zipf_bias=1.2, moe_q=moe_q, moe_k=moe_k)
            tp.full_check(inputs.make_inputs(cfg))
    elif case == "index_selftest":
        inp = inputs.make_inputs(inputs.CONFIGS["small_bf16"], batch=1)
        layer = binding.layer_from_inputs(inp)
        layer.sh_selftest(1, 7)                           # inside the range: nothing recorded
        assert layer.sh_last_status() == 0
        layer.sh_selftest(1, 12345)                       # outside: SH_ERR_BOUNDS with site, value, limit, block
        assert layer.sh_last_status() == -7
        w = layer.sh_status_block()
        assert w[8:12] == [7, 12345, 10, 0], w
        layer.sh_clear_status()
        x = binding.to_device(inp.x, inp.cfg.dtype)
        layer.sh_forward(x)
        torch.cuda.synchronize()
        assert layer.sh_last_status() == 0
        layer.close()
    else:
        raise SystemExit(f"unknown case {case}")
    print("DEBUG_DRIVER_OK")


if __name__ == "__main__":
    main(sys.argv[1])
