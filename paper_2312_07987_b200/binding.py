"""ctypes binding of libswitchhead.so: argument marshalling only.

Every step of the forward pass runs in the library's CUDA kernels; torch is used here for
device memory and streams.  Function names mirror the C ABI (include/switchhead.h).
There is no CPU fallback: if the library cannot be loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

SH_F32, SH_BF16 = 0, 1
SH_OK = 0
ERROR_NAMES = {-1: "SH_ERR_INVALID_ARG", -2: "SH_ERR_UNSUPPORTED", -3: "SH_ERR_NOT_CONFIGURED",
               -4: "SH_ERR_WORKSPACE", -5: "SH_ERR_CUDA", -6: "SH_ERR_TIMEOUT", -7: "SH_ERR_BOUNDS"}
BUF = dict(Q=0, K=1, V=2, AHAT=3, IDX=4, GATE=5, OFFSETS=6, LISTS=7)

EXPORTS = ["sh_create", "sh_create_shared", "sh_create_moe_qk", "sh_create_dense", "sh_configure", "sh_configure_xl", "sh_workspace_bytes", "sh_set_workspace",
           "sh_set_weights", "sh_set_causal", "sh_set_rope", "sh_set_xl_positions", "sh_forward", "sh_backward", "sh_forward_timed", "sh_forward_stamped", "sh_gate_topk",
           "sh_noalloc_gate_topk", "sh_debug_buffer", "sh_last_status", "sh_status_block", "sh_clear_status", "sh_check_guards",
           "sh_selftest", "sh_set_output_f16", "sh_is_debug_build", "sh_launch_count", "sh_last_error", "sh_destroy"]
STAMP_KERNELS = ["gate", "sort", "qk_a", "qk_b", "v", "attn", "o"]


def _load() -> ctypes.CDLL:
    path = os.environ.get("SWITCHHEAD_LIB") or _build.LIB_PATH     # a custom build of the library
    if not os.path.exists(path):
        path = _build.build()
    lib = ctypes.CDLL(path)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.sh_create.restype = vp
    lib.sh_create.argtypes = [i32] * 5
    lib.sh_create_shared.restype = vp
    lib.sh_create_shared.argtypes = [i32] * 5
    lib.sh_create_moe_qk.restype = vp
    lib.sh_create_moe_qk.argtypes = [i32] * 8
    lib.sh_create_dense.restype = vp
    lib.sh_create_dense.argtypes = [i32] * 3
    lib.sh_configure.restype = i32
    lib.sh_configure.argtypes = [vp, i32, i32, i32]
    lib.sh_configure_xl.restype = i32
    lib.sh_configure_xl.argtypes = [vp, i32, i32, i32, i32]
    lib.sh_workspace_bytes.restype = sz
    lib.sh_workspace_bytes.argtypes = [vp]
    lib.sh_set_workspace.restype = i32
    lib.sh_set_workspace.argtypes = [vp, vp, sz]
    lib.sh_set_weights.restype = i32
    lib.sh_set_weights.argtypes = [vp] * 10
    lib.sh_forward.restype = i32
    lib.sh_forward.argtypes = [vp, vp, vp, vp]
    lib.sh_backward.restype = i32
    lib.sh_backward.argtypes = [vp] * 11
    lib.sh_forward_timed.restype = i32
    lib.sh_forward_timed.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float)]
    lib.sh_forward_stamped.restype = i32
    lib.sh_forward_stamped.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ctypes.c_uint64)]
    lib.sh_status_block.restype = i32
    lib.sh_status_block.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
    lib.sh_clear_status.restype = i32
    lib.sh_clear_status.argtypes = [vp, vp]
    lib.sh_check_guards.restype = i32
    lib.sh_check_guards.argtypes = [vp, vp]
    lib.sh_selftest.restype = i32
    lib.sh_selftest.argtypes = [vp, i32, ctypes.c_uint64, vp]
    lib.sh_is_debug_build.restype = i32
    lib.sh_is_debug_build.argtypes = []
    lib.sh_gate_topk.restype = i32
    lib.sh_gate_topk.argtypes = [vp] * 7
    lib.sh_noalloc_gate_topk.restype = i32
    lib.sh_noalloc_gate_topk.argtypes = [i32] * 6 + [vp] * 8
    lib.sh_set_causal.restype = i32
    lib.sh_set_causal.argtypes = [vp, i32]
    lib.sh_set_xl_positions.restype = i32
    lib.sh_set_xl_positions.argtypes = [vp, vp, vp, vp, vp]
    lib.sh_set_rope.restype = i32
    lib.sh_set_rope.argtypes = [vp, ctypes.c_double, vp]
    lib.sh_debug_buffer.restype = i32
    lib.sh_debug_buffer.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(sz)]
    lib.sh_last_status.restype = i32
    lib.sh_last_status.argtypes = [vp, vp]
    lib.sh_set_output_f16.restype = i32
    lib.sh_set_output_f16.argtypes = [vp, i32]
    lib.sh_launch_count.restype = i32
    lib.sh_launch_count.argtypes = [vp]
    lib.sh_last_error.restype = ctypes.c_char_p
    lib.sh_last_error.argtypes = []
    lib.sh_destroy.restype = None
    lib.sh_destroy.argtypes = [vp]
    return lib


lib = _load()


class SwitchHeadError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        msg = lib.sh_last_error().decode()
        super().__init__(f"{ERROR_NAMES.get(code, code)}: {msg}")


def _check(code: int) -> None:
    if code != SH_OK:
        raise SwitchHeadError(code)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def sh_last_error() -> str:
    return lib.sh_last_error().decode()


class Layer:
    """Owns one sh_layer handle plus the torch tensors that back its workspace."""

    def __init__(self, d_model: int, n_heads: int, d_head: int, n_experts: int = 1, k: int = 1,
                 dense: bool = False, shared_selection: bool = False, moe_q: bool = False, moe_k: bool = False):
        self.dense = dense
        self.shared_selection = shared_selection
        self.dims = (d_model, n_heads, d_head, n_experts, k)
        if dense:
            h = lib.sh_create_dense(d_model, n_heads, d_head)
        elif moe_q or moe_k:
            h = lib.sh_create_moe_qk(d_model, n_heads, d_head, n_experts, k, int(moe_q), int(moe_k), int(shared_selection))
        elif shared_selection:
            h = lib.sh_create_shared(d_model, n_heads, d_head, n_experts, k)
        else:
            h = lib.sh_create(d_model, n_heads, d_head, n_experts, k)
        if not h:
            raise SwitchHeadError(-1)
        self.handle = ctypes.c_void_p(h)
        self.workspace = None
        self.dtype = None
        self.batch = self.seq = 0

    def sh_configure(self, dtype: int, batch: int, seq: int, device="cuda", cache_len: int = 0) -> None:
        """cache_len > 0: Transformer-XL context (sh_configure_xl): x is [B, cache_len + seq, M], out [B, seq, M]."""
        if cache_len:
            _check(lib.sh_configure_xl(self.handle, dtype, batch, seq, cache_len))
        else:
            _check(lib.sh_configure(self.handle, dtype, batch, seq))
        # (self.seq: tokens per sequence the layer sees, cache included; self.seq_out: rows of out per sequence)
        self.dtype, self.batch, self.seq, self.seq_out = dtype, batch, cache_len + seq, seq
        nbytes = lib.sh_workspace_bytes(self.handle)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        _check(lib.sh_set_workspace(self.handle, ctypes.c_void_p(self._ws_ptr), nbytes))

    def sh_set_weights(self, Wq, Wk, Wv, Wo, Ws=None, Wd=None, bias_s=None, bias_d=None) -> None:
        ts = [Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d]
        for t in ts:
            assert t is None or (t.is_cuda and t.is_contiguous())
        _check(lib.sh_set_weights(self.handle, *[_ptr(t) for t in ts], _stream()))
        torch.cuda.current_stream().synchronize()   # the source tensors may now be released

    def sh_set_causal(self, causal: bool) -> None:
        _check(lib.sh_set_causal(self.handle, 1 if causal else 0))

    def sh_set_xl_positions(self, Wr, u=None, v=None) -> None:
        """Transformer-XL relative-position term (fp32 layers): Wr [H, M, D], u, v [H, D] fp32 device tensors; None switches it off."""
        for t in (Wr, u, v):
            assert t is None or (t.is_cuda and t.is_contiguous() and t.dtype == torch.float32)
        _check(lib.sh_set_xl_positions(self.handle, _ptr(Wr), _ptr(u), _ptr(v), _stream()))
        torch.cuda.current_stream().synchronize()   # the source tensors may now be released

    def sh_set_rope(self, base: float) -> None:
        _check(lib.sh_set_rope(self.handle, float(base), _stream()))

    def sh_set_output_f16(self, enable: bool) -> None:
        """sh_forward writes fp16 instead of fp32 from now on (bf16 storage configuration only)."""
        _check(lib.sh_set_output_f16(self.handle, 1 if enable else 0))
        self.out_dtype = torch.float16 if enable else torch.float32

    def sh_forward(self, x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        assert x.is_cuda and x.is_contiguous()
        if out is None:
            out = torch.empty((x.shape[0], self.seq_out, x.shape[2]), dtype=getattr(self, "out_dtype", torch.float32), device=x.device)
        assert out.dtype == getattr(self, "out_dtype", torch.float32), "out must have the layer's output dtype (see sh_set_output_f16)"
        _check(lib.sh_forward(self.handle, _ptr(x), _ptr(out), _stream()))
        return out

    def sh_forward_timed(self, x: torch.Tensor, out: torch.Tensor):
        """Returns the six stage times in ms: gate+sort, qk, v, attention, o, total."""
        ms = (ctypes.c_float * 6)()
        _check(lib.sh_forward_timed(self.handle, _ptr(x), _ptr(out), _stream(), ms))
        return list(ms)

    def sh_forward_stamped(self, x: torch.Tensor, out: torch.Tensor):
        """One forward pass launched as sh_forward launches it; returns {kernel: (resident, start, end)} in
        nanoseconds of the device clock for the kernels that ran (see STAMP_KERNELS)."""
        n = len(STAMP_KERNELS)
        buf = (ctypes.c_uint64 * (3 * n))()
        _check(lib.sh_forward_stamped(self.handle, _ptr(x), _ptr(out), _stream(), buf))
        return {name: (buf[i], buf[n + i], buf[2 * n + i]) for i, name in enumerate(STAMP_KERNELS) if buf[2 * n + i] != 0}

    def sh_status_block(self):
        w = (ctypes.c_int32 * 16)()
        _check(lib.sh_status_block(self.handle, w, _stream()))
        return list(w)

    def sh_clear_status(self) -> None:
        _check(lib.sh_clear_status(self.handle, _stream()))

    def sh_check_guards(self) -> None:
        _check(lib.sh_check_guards(self.handle, _stream()))

    def sh_selftest(self, which: int, arg: int) -> None:
        _check(lib.sh_selftest(self.handle, which, arg, _stream()))

    def sh_backward(self, x: torch.Tensor, dout: torch.Tensor) -> dict:
        """Gradients of sum(out * dout) with respect to x and every weight (fp32 configuration; call sh_forward(x) first)."""
        d_model, H, D, E, k = self.dims
        dev = x.device
        z = lambda *shape: torch.empty(shape, dtype=torch.float32, device=dev)
        g = dict(dx=z(self.batch, self.seq, d_model), dWq=z(H, d_model, D), dWk=z(H, d_model, D), dWv=z(H, E, d_model, D),
                 dWo=z(H, E, D, d_model), dWs=z(H, d_model, E), dWd=z(H, d_model, E))
        _check(lib.sh_backward(self.handle, _ptr(x), _ptr(dout), *[_ptr(g[n]) for n in ("dx", "dWq", "dWk", "dWv", "dWo", "dWs", "dWd")], _stream()))
        return g

    def sh_gate_topk(self, x: torch.Tensor):
        d_model, H, D, E, k = self.dims
        N = self.batch * self.seq
        dev = x.device
        idx = torch.empty((2, N, H, k), dtype=torch.int32, device=dev)
        gate = torch.empty((2, N, H, k), dtype=torch.float32, device=dev)
        offsets = torch.empty((2, H, E + 1), dtype=torch.int32, device=dev)
        lists = torch.empty((2, H, N * k), dtype=torch.int32, device=dev)
        _check(lib.sh_gate_topk(self.handle, _ptr(x), _ptr(idx), _ptr(gate), _ptr(offsets), _ptr(lists), _stream()))
        return idx, gate, offsets, lists

    def sh_debug_buffer(self, name: str) -> torch.Tensor:
        """Copy of an intermediate buffer as a torch tensor (Q, K, V [B,H,T,D]; AHAT [N,H,D])."""
        p, n = ctypes.c_void_p(), ctypes.c_size_t()
        _check(lib.sh_debug_buffer(self.handle, BUF[name], ctypes.byref(p), ctypes.byref(n)))
        off = p.value - self.workspace.data_ptr()
        raw = self.workspace[off:off + n.value].clone()
        d_model, H, D, E, k = self.dims
        if name in ("Q", "K", "V", "AHAT"):
            t = raw.view(torch.float32 if self.dtype == SH_F32 else torch.float16)
            # d_head is stored padded with zero columns (64 / 128 on the bf16 path, 32 / 64 / 128 on fp32)
            Dp = (64 if D <= 64 else 128 if D <= 128 else 256) if self.dtype != SH_F32 else (32 if D <= 32 else 64 if D <= 64 else 128 if D <= 128 else 256)
            t = t.view(self.batch, H, self.seq, Dp) if name != "AHAT" else t.view(self.batch * self.seq, H, Dp)
            return t[..., :D]
        return raw.view(torch.float32 if name == "GATE" else torch.int32)

    def sh_last_status(self) -> int:
        return lib.sh_last_status(self.handle, _stream())

    def sh_launch_count(self) -> int:
        return lib.sh_launch_count(self.handle)

    def close(self) -> None:
        if self.handle:
            lib.sh_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sh_noalloc_gate_topk(dtype: int, x: torch.Tensor, w_gate: torch.Tensor, bias: Optional[torch.Tensor],
                         n_heads: int, n_experts: int, k: int):
    """Gate + top-k + bucket sort without a layer handle or workspace (see switchhead.h).
    x [N, M]; w_gate [2*H*E, M] (one row per gate column); returns idx, gate, offsets, lists.
    The output tensors are allocated here, by torch, before the call; the call itself allocates nothing."""
    N, M = x.shape
    dev = x.device
    idx = torch.empty((2, N, n_heads, k), dtype=torch.int32, device=dev)
    gate = torch.empty((2, N, n_heads, k), dtype=torch.float32, device=dev)
    offsets = torch.empty((2, n_heads, n_experts + 1), dtype=torch.int32, device=dev)
    lists = torch.empty((2, n_heads, N * k), dtype=torch.int32, device=dev)
    _check(lib.sh_noalloc_gate_topk(dtype, N, M, n_heads, n_experts, k, _ptr(x), _ptr(w_gate), _ptr(bias),
                                    _ptr(idx), _ptr(gate), _ptr(offsets), _ptr(lists), _stream()))
    return idx, gate, offsets, lists


def to_device(a: Optional[np.ndarray], dtype: int, device="cuda") -> Optional[torch.Tensor]:
    """Host array (fp32 values already representable in the storage type) -> device tensor."""
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    if dtype == SH_BF16:
        t = t.to(torch.bfloat16)
    return t.to(device).contiguous()


def layer_from_inputs(inp, batch=None, seq=None, device="cuda", shared_selection=False, cache_len=0) -> "Layer":
    """Create, configure and load a Layer from a LayerInputs record (see inputs.py).
    shared_selection: the source gate (Ws, bias_s) serves both sides; Wd and bias_d are not used.
    cache_len: the first cache_len tokens of every sequence of inp.x are a Transformer-XL cache."""
    cfg = inp.cfg
    B, T = inp.x.shape[0], inp.x.shape[1]
    # (Wq / Wk given per expert, [H, E, M, D]: a layer with query / key experts)
    L = Layer(cfg.d_model, cfg.n_heads, cfg.d_head, cfg.n_experts, cfg.k, shared_selection=shared_selection,
              moe_q=inp.Wq.ndim == 4, moe_k=inp.Wk.ndim == 4)
    L.sh_configure(cfg.dtype, B, T - cache_len, device=device, cache_len=cache_len)
    dv = lambda a: to_device(a, cfg.dtype, device)
    bias = lambda a: None if a is None else torch.from_numpy(a).to(device)
    L.sh_set_weights(dv(inp.Wq), dv(inp.Wk), dv(inp.Wv), dv(inp.Wo), dv(inp.Ws),
                     None if shared_selection else dv(inp.Wd),
                     bias(inp.bias_s), None if shared_selection else bias(inp.bias_d))
    return L
