"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, and validates arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2312_07987_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    text = open(os.path.join(ROOT, "include", "switchhead.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sh_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = header_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(binding.lib, n), n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) == set(binding.EXPORTS) | {n for n in names if n.startswith("sh_noalloc")}


@pytest.mark.parametrize("args,frag", [((100, 2, 32, 4, 2), "d_model"), ((128, 0, 32, 4, 2), "n_heads"),
                                       ((128, 2, 257, 4, 2), "d_head"), ((128, 2, 32, 33, 2), "n_experts"),
                                       ((128, 2, 32, 4, 0), "k must"), ((128, 2, 32, 4, 5), "k must")])
def test_create_rejects_bad_dimensions(args, frag):
    h = binding.lib.sh_create(*args)
    assert not h
    assert frag in binding.sh_last_error()


def test_call_order_and_argument_errors():
    lib = binding.lib
    h = ctypes.c_void_p(lib.sh_create(128, 2, 32, 4, 2))
    assert h
    assert lib.sh_workspace_bytes(h) == 0
    assert lib.sh_forward(h, None, None, None) == -3                 # not configured
    assert lib.sh_configure(h, 7, 1, 64) == -1
    assert lib.sh_configure(h, binding.SH_F32, 0, 64) == -1
    hb = ctypes.c_void_p(lib.sh_create(192, 2, 32, 4, 2))
    assert lib.sh_configure(hb, binding.SH_BF16, 1, 64) == -2        # d_model 192: not a multiple of 128
    assert "bf16" in binding.sh_last_error()
    lib.sh_destroy(hb)
    assert lib.sh_configure(h, binding.SH_F32, 1, 64) == 0
    need = lib.sh_workspace_bytes(h)
    assert need > 0
    assert lib.sh_set_workspace(h, None, need) == -4
    assert lib.sh_set_workspace(h, ctypes.c_void_p(0x1001), need) == -4   # misaligned
    assert lib.sh_set_workspace(h, ctypes.c_void_p(0x1000), need - 1) == -4
    assert "too small" in binding.sh_last_error()
    assert lib.sh_forward(h, None, None, None) == -4                 # no workspace
    assert lib.sh_set_weights(h, *([None] * 9)) == -4
    p, n = ctypes.c_void_p(), ctypes.c_size_t()
    assert lib.sh_debug_buffer(h, 0, ctypes.byref(p), ctypes.byref(n)) == -3
    assert lib.sh_last_status(None, None) == -1
    assert lib.sh_set_rope(None, 10000.0, None) == -1
    assert lib.sh_set_causal(None, 0) == -1 and lib.sh_set_causal(h, 0) == 0 and lib.sh_set_causal(h, 1) == 0
    assert lib.sh_set_rope(h, 10000.0, None) == -3                   # configured, but no workspace yet
    assert lib.sh_set_output_f16(None, 1) == -1
    assert lib.sh_set_output_f16(h, 1) == -2                         # fp32 configuration: unsupported
    assert lib.sh_set_output_f16(h, 0) == 0
    assert lib.sh_set_rope(h, -1.0, None) in (-3, -1)
    h2 = ctypes.c_void_p(lib.sh_create(128, 2, 32, 4, 2))
    assert lib.sh_set_rope(h2, 10000.0, None) == -3                  # not configured
    lib.sh_destroy(h2)
    lib.sh_destroy(h)
    lib.sh_destroy(None)                                             # NULL-safe
    assert lib.sh_configure(None, 0, 1, 1) == -1


def test_problem_size_limit():
    lib = binding.lib
    h = ctypes.c_void_p(lib.sh_create(1024, 16, 128, 32, 32))
    assert lib.sh_configure(h, binding.SH_BF16, 4096, 4096) == -2
    assert "2^31" in binding.sh_last_error()
    lib.sh_destroy(h)


def test_workspace_size_scales_with_tokens():
    lib = binding.lib
    h = ctypes.c_void_p(lib.sh_create(1024, 4, 128, 4, 2))
    assert lib.sh_configure(h, binding.SH_BF16, 1, 512) == 0
    a = lib.sh_workspace_bytes(h)
    assert lib.sh_configure(h, binding.SH_BF16, 16, 512) == 0
    b = lib.sh_workspace_bytes(h)
    weights = (2 * 4 * 128 * 1024 + 2 * 4 * 4 * 1024 + 2 * 4 * 4 * 128 * 1024) * 2
    assert a > weights and b > a
    # activations: Q, K, V, Ahat fp16 + idx/gate/lists
    per_tok = 4 * 4 * 128 * 2
    assert (b - a) >= 15 * 512 * per_tok
    lib.sh_destroy(h)
