"""Seeded synthetic inputs for one SwitchHead attention layer (forward only).

This module is the only code shared by the CPU oracle's tests and the CUDA path's
tests/bench.  It draws random arrays, rounds them to the storage precision and
enforces a margin between the k-th and (k+1)-th gate logit of every token; it
contains none of the layer's arithmetic (no sigmoid, no top-k selection, no
attention, no expert sums).  The margin check needs the raw gate logits, which
it obtains with one plain fp64 matrix product followed by a sort.

Layouts (row-major, matching the C-ABI):
    x      [B, T, M]
    Wq, Wk [H, M, D]
    Wv     [H, E, M, D]
    Wo     [H, E, D, M]
    Ws, Wd [H, M, E]          source-side / destination-side gate weights
    bias_s, bias_d [H, E] fp32 or None

The five named workloads stand in for the language-model shapes of the paper's
hyper-parameter table (2 heads/E=5/k=3/T=256 for the 47M models, 4 heads/E=4/
k=2/T=512/d_model 1024 for the 262M models), with d_head rounded to a power of
two, plus a long-context and a wide skew-routed case.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

DTYPE_F32 = 0
DTYPE_BF16 = 1


@dataclass(frozen=True)
class LayerConfig:
    name: str
    dtype: int          # DTYPE_F32 or DTYPE_BF16: storage precision of x and weights
    batch: int
    seq: int
    d_model: int
    n_heads: int
    d_head: int
    n_experts: int
    k: int
    seed: int
    zipf_bias: float = 0.0   # exponent of the per-expert Zipf gate-bias profile (0 = no bias)
    min_gap: float = 1e-3    # required logit margin at rank k
    moe_q: bool = False      # query / key projections as experts too (Wq / Wk drawn as [H, E, M, D])
    moe_k: bool = False

    @property
    def n_tokens(self) -> int:
        return self.batch * self.seq


CONFIGS = {
    "tiny_f32": LayerConfig("tiny_f32", DTYPE_F32, 1, 64, 128, 2, 32, 4, 2, seed=0),
    "small_bf16": LayerConfig("small_bf16", DTYPE_BF16, 32, 256, 512, 2, 64, 5, 3, seed=1),
    "c4_262m_bf16": LayerConfig("c4_262m_bf16", DTYPE_BF16, 16, 512, 1024, 4, 128, 4, 2, seed=2),
    "long_ctx_bf16": LayerConfig("long_ctx_bf16", DTYPE_BF16, 4, 4096, 1024, 4, 128, 8, 2, seed=3),
    "wide_skew_bf16": LayerConfig("wide_skew_bf16", DTYPE_BF16, 8, 2048, 2048, 8, 128, 16, 4,
                                  seed=4, zipf_bias=1.2),
}
CONFIG_ORDER = ["tiny_f32", "small_bf16", "c4_262m_bf16", "long_ctx_bf16", "wide_skew_bf16"]


@dataclass
class LayerInputs:
    cfg: LayerConfig
    x: np.ndarray
    Wq: np.ndarray
    Wk: np.ndarray
    Wv: np.ndarray
    Wo: np.ndarray
    Ws: np.ndarray
    Wd: np.ndarray
    bias_s: Optional[np.ndarray] = None
    bias_d: Optional[np.ndarray] = None
    redrawn_rows: int = 0
    extra: dict = field(default_factory=dict)

    def arrays(self):
        return dict(x=self.x, Wq=self.Wq, Wk=self.Wk, Wv=self.Wv, Wo=self.Wo, Ws=self.Ws,
                    Wd=self.Wd, bias_s=self.bias_s, bias_d=self.bias_d)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays in an fp32 array."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an fp32 array whose values are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    assert not np.any(bits & 0xFFFF), "values are not bf16-representable"
    return (bits >> 16).astype(np.uint16).reshape(a.shape)


def _store(a: np.ndarray, dtype: int) -> np.ndarray:
    a32 = a.astype(np.float32)
    return round_to_bf16(a32) if dtype == DTYPE_BF16 else a32


def _zipf_bias(rng: np.random.Generator, n_heads: int, n_experts: int, s: float) -> np.ndarray:
    """Per (head) a seeded permutation of experts; p_e ~ rank^-s; bias = ln p - mean(ln p)."""
    out = np.empty((n_heads, n_experts), dtype=np.float32)
    for h in range(n_heads):
        perm = rng.permutation(n_experts)
        ranks = np.empty(n_experts, dtype=np.float64)
        ranks[perm] = np.arange(1, n_experts + 1, dtype=np.float64)
        lp = -s * np.log(ranks)
        out[h] = (lp - lp.mean()).astype(np.float32)
    return out


def _rank_gap(x2d: np.ndarray, W: np.ndarray, bias: Optional[np.ndarray], k: int) -> np.ndarray:
    """Smallest margin, over heads, between the k-th and (k+1)-th largest raw gate logit.

    x2d [n, M]; W [H, M, E].  A plain product and a sort: the margin is a property of the
    inputs, used only to decide which rows get redrawn."""
    n = x2d.shape[0]
    H, _, E = W.shape
    if k >= E:
        return np.full(n, np.inf)
    gap = np.full(n, np.inf)
    xd = x2d.astype(np.float64)
    for h in range(H):
        z = xd @ W[h].astype(np.float64)
        if bias is not None:
            z = z + bias[h].astype(np.float64)
        zs = np.sort(z, axis=1)[:, ::-1]
        gap = np.minimum(gap, zs[:, k - 1] - zs[:, k])
    return gap


def make_inputs(cfg: LayerConfig, *, batch: Optional[int] = None, seq: Optional[int] = None,
                enforce_gap: bool = True) -> LayerInputs:
    """Draw x and all weights for `cfg` (optionally with a smaller batch/seq: the weights
    drawn are identical, only x shrinks, because x is drawn last)."""
    B = cfg.batch if batch is None else batch
    T = cfg.seq if seq is None else seq
    M, H, D, E, k = cfg.d_model, cfg.n_heads, cfg.d_head, cfg.n_experts, cfg.k
    rng = np.random.Generator(np.random.PCG64(cfg.seed))

    def normal(shape, fan_in):
        return rng.standard_normal(shape, dtype=np.float64) / np.sqrt(fan_in)

    Wq = _store(normal((H, E, M, D) if cfg.moe_q else (H, M, D), M), cfg.dtype)
    Wk = _store(normal((H, E, M, D) if cfg.moe_k else (H, M, D), M), cfg.dtype)
    Wv = _store(normal((H, E, M, D), M), cfg.dtype)
    Wo = _store(normal((H, E, D, M), D), cfg.dtype)
    Ws = _store(normal((H, M, E), M), cfg.dtype)
    Wd = _store(normal((H, M, E), M), cfg.dtype)
    bias_s = bias_d = None
    if cfg.zipf_bias > 0:
        bias_s = _zipf_bias(rng, H, E, cfg.zipf_bias)
        bias_d = _zipf_bias(rng, H, E, cfg.zipf_bias)
    x = _store(rng.standard_normal((B * T, M), dtype=np.float64), cfg.dtype)

    redrawn = 0
    if enforce_gap and k < E:
        chunk = 4096
        for lo in range(0, B * T, chunk):
            hi = min(lo + chunk, B * T)
            rows = np.arange(lo, hi)
            for _ in range(64):
                g = np.minimum(_rank_gap(x[rows], Ws, bias_s, k), _rank_gap(x[rows], Wd, bias_d, k))
                bad = rows[g < cfg.min_gap]
                if bad.size == 0:
                    break
                x[bad] = _store(rng.standard_normal((bad.size, M), dtype=np.float64), cfg.dtype)
                redrawn += int(bad.size)
                rows = bad
            else:
                raise RuntimeError("gap enforcement did not converge")
    return LayerInputs(cfg, x.reshape(B, T, M), Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d, redrawn)


def make_dense_mha_weights(d_model: int, n_heads: int, d_head: int, seed: int, dtype: int):
    """Weights of the dense multi-head comparator: Wq, Wk, Wv [H, M, D], Wo [H, D, M]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    M, H, D = d_model, n_heads, d_head
    Wq = _store(rng.standard_normal((H, M, D)) / np.sqrt(M), dtype)
    Wk = _store(rng.standard_normal((H, M, D)) / np.sqrt(M), dtype)
    Wv = _store(rng.standard_normal((H, M, D)) / np.sqrt(M), dtype)
    Wo = _store(rng.standard_normal((H, D, M)) / np.sqrt(H * D), dtype)
    return Wq, Wk, Wv, Wo


def useful_flop(cfg: LayerConfig, batch: Optional[int] = None, seq: Optional[int] = None) -> dict:
    """Algorithmic FLOP of one forward pass: dense Q/K projections, the k selected V and O
    experts only, and half of the (QK^T + PV) attention FLOP (causal)."""
    B = cfg.batch if batch is None else batch
    T = cfg.seq if seq is None else seq
    N, M, H, D, k = B * T, cfg.d_model, cfg.n_heads, cfg.d_head, cfg.k
    qk = 2.0 * N * M * 2 * H * D
    v = 2.0 * N * H * k * M * D
    o = 2.0 * N * H * k * D * M
    attn = 2.0 * B * H * T * T * D
    return dict(qk=qk, v=v, o=o, attn_half=attn, total=qk + v + o + attn)
