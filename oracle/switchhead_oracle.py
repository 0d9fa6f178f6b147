"""fp64 CPU oracle for the forward pass of one SwitchHead attention layer.

TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA path is compared with; it
shares no code with the CUDA path and nothing in the product imports it (only tests/,
the smoke check and the benchmark's CPU-baseline leg do).

What it computes, following the paper's Sec. 2.2 ("From Dense to SwitchHead"):

  source-side gate        s_S^h = sigmoid(x W_S^h)            (first display eq. of Sec. 2.2)
  destination-side gate   s_D^h = sigmoid(x W_D^h)            (text after it)
  selections              E_S^h, E_D^h = arg top-k            (same place)
  value projection        V^h = sum_{e in E_S^h} s_S^h[e] x W_V^{h,e}
  dense queries / keys    Q^h = x W_Q^h, K^h = x W_K^h        (SwitchHead keeps one dense
                                                               Q/K per head, end of Sec. 2.2)
  attention               A^h = softmax(Q^h K^h^T / sqrt(d_head))     (Eq. 1), causal
  output                  y = sum_h sum_{e in E_D^h} s_D^h[e] A^h V^h W_O^{h,e}
                                                              (the MoE output equation)

Optional (off by default): rotary position embeddings on Q and K (the paper's appendix on
RoPE positional encodings: square causal attention, no cache), pairs (2i, 2i+1), angle
p * base**(-2i/d_head).

Readings where the paper is silent (each is listed in the design notes):
  * top-k is taken on the pre-sigmoid logits (sigmoid is strictly increasing, so the set
    is the same in exact arithmetic); ties go to the lower expert index; -0.0 == +0.0.
  * no renormalisation among the selected gates (non-competitive sigmoid gate).
  * causal mask: key s is visible to query t iff s <= t (language-model setting).
  * an optional per-expert gate bias b (z = x W + b) exists only for the skew-routed
    synthetic workload; None reproduces the paper exactly.
  * batch elements are independent sequences.

All arithmetic is fp64 on the values handed in (already rounded to their storage type);
no intermediate rounding.  Every stage is returned so that a failing comparison can be
localised.

Transformer-XL context (switchhead_xl_forward; the paper's main configuration): keys, values and the
source-side gate over [cache; chunk], queries and the destination side over the chunk, optional
relative-position term in Transformer-XL's form.  Pins (tests/test_oracle_xl_pins.py): no cache = the
plain layer; one 2T pass = two T passes with the cache (with and without positions); W_Q = 0 gives
running means over cache + chunk; cache visible to every query, later chunk tokens to none; a
scalar-loop writing; zero position weights = no position term; the appendix's MAC / memory table.

MoE key / query projections (expert_projection; Wk or Wq given as [H, E, M, D]): the K^h and Q^h expert
sums of Sec. 2.2, keys with the source side's selection and scores, queries with the destination
side's.  Pins (tests/test_oracle_moe_qk_pins.py): a scalar-loop writing; identical experts = the dense
projection times the sum of the selected gates; every expert selected with a constant gate = a dense
projection with the summed weights; experts nobody selected do not matter, selected ones do, and the
keys follow the SOURCE side; renumbering a side's experts; the context form against the plain layer.

Pins (tests/test_oracle_pins.py): E=1 with zero gate weights equals 0.25 x textbook MHA
(Eq. 2 and Eq. 3 forms, and torch's scaled_dot_product_attention); gate forced to 1 equals
MHA; k=E equals the dense gate-weighted einsum; top-k equals a brute-force stable sort;
causality; W_Q=0 gives running means of V; expert-permutation and batch-permutation
invariance; linearity in W_O; bucket lists are a stable counting sort.
Absolute output values for realistic trained weights: parity unpinned (the paper prints
no worked forward-pass example).
"""
from __future__ import annotations

from typing import Optional

import numpy as np


def stable_sigmoid(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    out = np.empty_like(z)
    pos = z >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-z[pos]))
    ez = np.exp(z[~pos])
    out[~pos] = ez / (1.0 + ez)
    return out


def topk_lower_index_wins(z: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest entries of each row of z [n, E]: value descending, and among
    equal values the lower index first.  Returns [n, k] int32."""
    z = np.asarray(z, dtype=np.float64) + 0.0      # -0.0 + 0.0 = +0.0: the two zeros tie
    # stable sort on the negated value keeps equal values in ascending index order
    order = np.argsort(-z, axis=1, kind="stable")
    return order[:, :k].astype(np.int32)


def gate_and_select(x2d, W, bias, k):
    """x2d [n, M], W [H, M, E], bias [H, E] or None.
    Returns logits z [n, H, E], scores s [n, H, E], idx [n, H, k] (rank order), gate [n, H, k]."""
    n = x2d.shape[0]
    H, _, E = W.shape
    z = np.empty((n, H, E))
    for h in range(H):
        z[:, h, :] = x2d @ W[h]
        if bias is not None:
            z[:, h, :] += bias[h]
    s = stable_sigmoid(z)
    idx = np.empty((n, H, k), dtype=np.int32)
    for h in range(H):
        idx[:, h, :] = topk_lower_index_wins(z[:, h, :], k)
    gate = np.take_along_axis(s, idx.astype(np.int64), axis=2)
    return z, s, idx, gate


def bucket_lists(idx: np.ndarray, n_experts: int):
    """Per (head, expert) lists of the tokens that selected the expert, token-ascending.

    idx [n, H, k].  Returns offsets [H, E+1] (exclusive scan of the counts, per head) and
    lists [H, n*k] of token ids (bucket e of head h occupies lists[h, offsets[h,e]:offsets[h,e+1]])."""
    n, H, k = idx.shape
    offsets = np.zeros((H, n_experts + 1), dtype=np.int32)
    lists = np.empty((H, n * k), dtype=np.int32)
    for h in range(H):
        pos = 0
        for e in range(n_experts):
            toks = np.nonzero((idx[:, h, :] == e).any(axis=1))[0]
            lists[h, pos:pos + toks.size] = toks
            pos += toks.size
            offsets[h, e + 1] = pos
        assert pos == n * k
    return offsets, lists


def rope_rotate(a: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotary position embedding (the RoPE variant of the paper's appendix "RoPE Positional
    Encodings", which takes it from RoFormer): feature pairs (2i, 2i+1) of the vector at
    position p are rotated by the angle p * base**(-2i/D).

    a [..., T, D] (D even), positions [T].  Written out pair by pair:
      a'[2i]   = a[2i] cos(p theta_i) - a[2i+1] sin(p theta_i)
      a'[2i+1] = a[2i] sin(p theta_i) + a[2i+1] cos(p theta_i)."""
    a = np.asarray(a, dtype=np.float64)
    D = a.shape[-1]
    if D % 2:
        raise ValueError("rotary embedding needs an even d_head")
    i = np.arange(D // 2, dtype=np.float64)
    theta = np.power(float(base), -2.0 * i / D)                       # [D/2]
    ang = np.asarray(positions, dtype=np.float64)[:, None] * theta[None, :]   # [T, D/2]
    c, s_ = np.cos(ang), np.sin(ang)
    out = np.empty_like(a)
    out[..., 0::2] = a[..., 0::2] * c - a[..., 1::2] * s_
    out[..., 1::2] = a[..., 0::2] * s_ + a[..., 1::2] * c
    return out


def expert_projection(x2d, W_he, idx_h, gate_h):
    """Gate-weighted sum of the selected experts' projections of every row (Sec. 2.2, the K^h / Q^h /
    V^h expert sums): out[t] = sum_j gate_h[t, j] * x2d[t] @ W_he[idx_h[t, j]].
    x2d [N, M]; W_he [E, M, D]: the experts of one head; idx_h, gate_h [N, k]."""
    N, k = idx_h.shape
    out = np.zeros((N, W_he.shape[2]))
    for e in range(W_he.shape[0]):
        for j in range(k):
            rows = np.nonzero(idx_h[:, j] == e)[0]
            if rows.size:
                out[rows] += gate_h[rows, j][:, None] * (x2d[rows] @ W_he[e])
    return out


def switchhead_forward(x, Wq, Wk, Wv, Wo, Ws, Wd, k: int, bias_s=None, bias_d=None,
                       causal: bool = True, gate_override: Optional[float] = None,
                       return_stages: bool = True, rope_base: Optional[float] = None,
                       rope_offset: int = 0, shared_selection: bool = False):
    """Forward pass of one SwitchHead layer in fp64.

    x [B, T, M]; Wq, Wk [H, M, D]; Wv [H, E, M, D]; Wo [H, E, D, M]; Ws, Wd [H, M, E].
    MoE key / query projections (the paper's Sec. 2.2 writes the key and query expert sums like the
    value one; its ablation over which projections are experts): Wk [H, E, M, D] makes the keys
    K^h[t] = sum_{e in E_S^h(t)} s_S^h[t,e] x[t] W_K^{h,e} (source-side selection, like the values);
    Wq [H, E, M, D] makes the queries Q^h[t] = sum_{e in E_D^h(t)} s_D^h[t,e] x[t] W_Q^{h,e}
    (destination-side selection, like the output).
    gate_override: if given, every selected expert's gate is replaced by this constant
    (used only to pin the E=1 case to plain multi-head attention).
    shared_selection: the "Shared Selection" variant of the paper's appendix: one gate serves
    both sides, i.e. the destination side uses the source side's selection and scores
    (Wd and bias_d are ignored).
    rope_base: if given, queries and keys are rotated by rotary position embeddings with
    this base before the attention scores (token t of a sequence sits at position
    rope_offset + t; no cache, square attention); None = no positional encoding.
    Returns a dict with y [B, T, M] and, if return_stages, the intermediate stages."""
    f = lambda a: None if a is None else np.asarray(a, dtype=np.float64)
    x, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d = map(f, (x, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d))
    B, T, M = x.shape
    H, E, _, D = Wv.shape
    N = B * T
    x2d = x.reshape(N, M)

    zS, sS, idxS, gateS = gate_and_select(x2d, Ws, bias_s, k)
    if shared_selection:
        zD, sD, idxD, gateD = zS, sS, idxS, gateS
    else:
        zD, sD, idxD, gateD = gate_and_select(x2d, Wd, bias_d, k)
    if gate_override is not None:
        gateS = np.full_like(gateS, gate_override)
        gateD = np.full_like(gateD, gate_override)

    Q = np.empty((N, H, D))
    K = np.empty((N, H, D))
    V = np.zeros((N, H, D))
    for h in range(H):
        Q[:, h, :] = x2d @ Wq[h] if Wq.ndim == 3 else expert_projection(x2d, Wq[h], idxD[:, h, :], gateD[:, h, :])
        K[:, h, :] = x2d @ Wk[h] if Wk.ndim == 3 else expert_projection(x2d, Wk[h], idxS[:, h, :], gateS[:, h, :])
        # value experts: only the rows that selected expert e are projected with it
        for e in range(E):
            for j in range(k):
                rows = np.nonzero(idxS[:, h, j] == e)[0]
                if rows.size:
                    V[rows, h, :] += gateS[rows, h, j][:, None] * (x2d[rows] @ Wv[h, e])

    if rope_base is not None:
        pos = rope_offset + np.arange(T)
        # [N, H, D] -> [B, H, T, D] so that the position axis sits next to the feature axis
        to_bhtd = lambda a: a.reshape(B, T, H, D).transpose(0, 2, 1, 3)
        back = lambda a: a.transpose(0, 2, 1, 3).reshape(N, H, D)
        Q = back(rope_rotate(to_bhtd(Q), pos, rope_base))
        K = back(rope_rotate(to_bhtd(K), pos, rope_base))

    Ahat = np.empty((N, H, D))
    scale = 1.0 / np.sqrt(D)
    mask = np.triu(np.ones((T, T), dtype=bool), k=1) if causal else None
    for b in range(B):
        sl = slice(b * T, (b + 1) * T)
        for h in range(H):
            L = (Q[sl, h, :] @ K[sl, h, :].T) * scale
            if causal:
                L = np.where(mask, -np.inf, L)
            L = L - L.max(axis=1, keepdims=True)
            P = np.exp(L)
            A = P / P.sum(axis=1, keepdims=True)
            Ahat[sl, h, :] = A @ V[sl, h, :]

    y = np.zeros((N, M))
    for h in range(H):
        for e in range(E):
            for j in range(k):
                rows = np.nonzero(idxD[:, h, j] == e)[0]
                if rows.size:
                    y[rows] += gateD[rows, h, j][:, None] * (Ahat[rows, h, :] @ Wo[h, e])

    out = {"y": y.reshape(B, T, M)}
    if return_stages:
        offS, listS = bucket_lists(idxS, E)
        offD, listD = bucket_lists(idxD, E)
        out.update(zS=zS, zD=zD, sS=sS, sD=sD, idxS=idxS, idxD=idxD, gateS=gateS, gateD=gateD,
                   Q=Q.reshape(B, T, H, D), K=K.reshape(B, T, H, D), V=V.reshape(B, T, H, D),
                   Ahat=Ahat.reshape(B, T, H, D), offsetsS=offS, listsS=listS,
                   offsetsD=offD, listsD=listD)
    return out


def dense_mha_forward(x, Wq, Wk, Wv, Wo, causal: bool = True):
    """Standard multi-head attention (Eq. 1-2) in the concatenated form: the per-head
    readouts are concatenated along the feature axis and multiplied by one W_O of shape
    [H*D, M].  x [B, T, M]; Wq, Wk, Wv [H, M, D]; Wo [H, D, M] (row blocks of W_O)."""
    x, Wq, Wk, Wv, Wo = (np.asarray(a, dtype=np.float64) for a in (x, Wq, Wk, Wv, Wo))
    B, T, M = x.shape
    H, _, D = Wq.shape
    WO = Wo.reshape(H * D, M)
    y = np.empty((B, T, M))
    for b in range(B):
        cat = np.empty((T, H * D))
        for h in range(H):
            Qh, Kh, Vh = x[b] @ Wq[h], x[b] @ Wk[h], x[b] @ Wv[h]
            L = Qh @ Kh.T / np.sqrt(D)
            if causal:
                L = np.where(np.triu(np.ones((T, T), dtype=bool), k=1), -np.inf, L)
            L = L - L.max(axis=1, keepdims=True)
            P = np.exp(L)
            cat[:, h * D:(h + 1) * D] = (P / P.sum(axis=1, keepdims=True)) @ Vh
        y[b] = cat @ WO
    return y


def xl_relative_embedding(n_dist: int, d_model: int) -> np.ndarray:
    """Sinusoidal embedding of the relative distances 0 .. n_dist-1, as Transformer-XL (which the
    paper's main models use: "Transformer-XL-style relative positional encoding") defines it:
    row d = [sin(d w_0) .. sin(d w_{M/2-1}), cos(d w_0) .. cos(d w_{M/2-1})], w_i = 10000^(-2i/M)."""
    if d_model % 2:
        raise ValueError("d_model must be even")
    w = np.power(10000.0, -2.0 * np.arange(d_model // 2, dtype=np.float64) / d_model)
    ang = np.arange(n_dist, dtype=np.float64)[:, None] * w[None, :]
    return np.concatenate([np.sin(ang), np.cos(ang)], axis=1)


def switchhead_xl_forward(x, cache, Wq, Wk, Wv, Wo, Ws, Wd, k: int, bias_s=None, bias_d=None,
                          Wr=None, u=None, v=None, return_stages: bool = True):
    """SwitchHead layer with a Transformer-XL context (the paper's main configuration, Sec. 3 and the
    appendix on resource usage: keys and values span C*T tokens, "C - 1 past chunks").

    x [B, T, M]: the current chunk.  cache [B, Tc, M]: the layer INPUT of the previous chunk(s)
    (Tc = (C-1)*T; Tc = 0 gives the plain layer).  The source side - keys, values, the source
    gate and its expert selection - is computed from the context ctx = [cache; x] (Tc + T tokens);
    the destination side - queries, the destination gate, the output - from x alone.  Query i
    (context position Tc + i) sees context positions j <= Tc + i.

    Relative positions (optional; Wr [H, M, D], u, v [H, D]): Transformer-XL's decomposition
        score[i, j] = ( (q_i + u) . k_j  +  (q_i + v) . r_{(Tc+i) - j} ) / sqrt(D),
        r_d = xl_relative_embedding(d) Wr^h,
    u and v being the two global bias vectors of each head.  With Wr None the score is the plain
    q_i . k_j / sqrt(D).  Returns y [B, T, M] and, if return_stages, Q [B,T,H,D], K, V [B,Tc+T,H,D],
    Ahat [B,T,H,D] and the selections of both sides."""
    f = lambda a: None if a is None else np.asarray(a, dtype=np.float64)
    x, cache, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d, Wr, u, v = map(
        f, (x, cache, Wq, Wk, Wv, Wo, Ws, Wd, bias_s, bias_d, Wr, u, v))
    B, T, M = x.shape
    Tc = 0 if cache is None else cache.shape[1]
    H, E, _, D = Wv.shape
    ctx = x if Tc == 0 else np.concatenate([cache, x], axis=1)             # [B, Tc + T, M]
    CT = Tc + T
    c2d, x2d = ctx.reshape(B * CT, M), x.reshape(B * T, M)

    _, _, idxS, gateS = gate_and_select(c2d, Ws, bias_s, k)                # source side: every context token
    _, _, idxD, gateD = gate_and_select(x2d, Wd, bias_d, k)                # destination side: the chunk's tokens

    Q = np.empty((B * T, H, D))
    K = np.empty((B * CT, H, D))
    V = np.zeros((B * CT, H, D))
    for h in range(H):
        Q[:, h, :] = x2d @ Wq[h] if Wq.ndim == 3 else expert_projection(x2d, Wq[h], idxD[:, h, :], gateD[:, h, :])
        K[:, h, :] = c2d @ Wk[h] if Wk.ndim == 3 else expert_projection(c2d, Wk[h], idxS[:, h, :], gateS[:, h, :])
        for e in range(E):
            for j in range(k):
                rows = np.nonzero(idxS[:, h, j] == e)[0]
                if rows.size:
                    V[rows, h, :] += gateS[rows, h, j][:, None] * (c2d[rows] @ Wv[h, e])

    R = None
    if Wr is not None:
        emb = xl_relative_embedding(CT, M)                                  # distances 0 .. CT-1
        R = np.stack([emb @ Wr[h] for h in range(H)])                       # [H, CT, D]
        u = np.zeros((H, D)) if u is None else u
        v = np.zeros((H, D)) if v is None else v

    Ahat = np.empty((B * T, H, D))
    scale = 1.0 / np.sqrt(D)
    qpos = Tc + np.arange(T)                                                # context position of query i
    jpos = np.arange(CT)
    hidden = jpos[None, :] > qpos[:, None]                                  # [T, CT]: keys after the query
    dist = np.clip(qpos[:, None] - jpos[None, :], 0, CT - 1)                # relative distance where visible
    for b in range(B):
        qs, cs = slice(b * T, (b + 1) * T), slice(b * CT, (b + 1) * CT)
        for h in range(H):
            if R is None:
                L = Q[qs, h, :] @ K[cs, h, :].T
            else:
                L = (Q[qs, h, :] + u[h]) @ K[cs, h, :].T                   # content terms
                BD = (Q[qs, h, :] + v[h]) @ R[h].T                          # [T, CT] over distances
                L = L + np.take_along_axis(BD, dist, axis=1)                # position terms, by distance
            L = np.where(hidden, -np.inf, L * scale)
            L = L - L.max(axis=1, keepdims=True)
            P = np.exp(L)
            A = P / P.sum(axis=1, keepdims=True)
            Ahat[qs, h, :] = A @ V[cs, h, :]

    y = np.zeros((B * T, M))
    for h in range(H):
        for e in range(E):
            for j in range(k):
                rows = np.nonzero(idxD[:, h, j] == e)[0]
                if rows.size:
                    y[rows] += gateD[rows, h, j][:, None] * (Ahat[rows, h, :] @ Wo[h, e])
    out = {"y": y.reshape(B, T, M)}
    if return_stages:
        out.update(idxS=idxS, idxD=idxD, gateS=gateS, gateD=gateD, Q=Q.reshape(B, T, H, D),
                   K=K.reshape(B, CT, H, D), V=V.reshape(B, CT, H, D), Ahat=Ahat.reshape(B, T, H, D))
    return out
