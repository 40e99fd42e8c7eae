"""Decoder forward that yields every layer's K and V for one logged prefix.

What is rebuilt (paper Sec. 4.2 step 5; Sec. 4.3): the K/V a worker held for a
request are a pure function of the request's logged tokens and the weights, so
a causal prefill over the prefix reproduces them.  The paper delegates the
model to its inference engine; the block below is the pre-norm decoder the
benchmark configurations name (RMSNorm, grouped-query attention, rotate-half
RoPE, SwiGLU, no biases), written as its textbook definition.

Two projection variants of the model families the paper trains (Sec. 6: Qwen3
for the end-to-end runs, Qwen2.5-1.5B for the re-prefill figure) are taken when
the weight set carries them: per-layer biases `bq`, `bk`, `bv` added to the
q/k/v projections, and per-head RMSNorm gains `qn`, `kn` [hd] applied to every
q and k head after the bias and before RoPE (same eps as the block norms).

All arrays are numpy float64.  Shapes: h [n, d]; q [n, Hq, hd]; k, v [n, Hkv, hd].
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Tuple

import numpy as np


def _f64(x) -> np.ndarray:
    """Weights may arrive as torch tensors (any float dtype) or numpy arrays."""
    if hasattr(x, "detach"):
        import torch
        return x.detach().cpu().to(torch.float64).numpy()
    return np.asarray(x, dtype=np.float64)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (ties to even, through fp32), returned as float64."""
    u = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32).astype(np.uint64)
    u = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def rmsnorm(h: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """a = h / sqrt(mean_i h_i^2 + eps) * g, row by row."""
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * g


def rope_cos_sin(positions: np.ndarray, head_dim: int, base: float) -> Tuple[np.ndarray, np.ndarray]:
    """theta[p, i] = p * base^(-2i/hd), i in [0, hd/2)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / head_dim)
    theta = positions.astype(np.float64)[:, None] * inv_freq[None, :]
    return np.cos(theta), np.sin(theta)


def apply_rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotate-half pairing: (x[i], x[i+hd/2]) turned by theta[p, i]."""
    hd = x.shape[-1]
    half = hd // 2
    cos, sin = rope_cos_sin(positions, hd, base)
    cos, sin = cos[:, None, :], sin[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    out = np.empty_like(x)
    out[..., :half] = x1 * cos - x2 * sin
    out[..., half:] = x2 * cos + x1 * sin
    return out


def causal_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, round_p=None) -> np.ndarray:
    """o_t[hq] = sum_{j<=t} softmax_j(q_t[hq].k_j[hq // G] / sqrt(hd)) v_j[hq // G].
    With `round_p`, the unnormalised weights exp(s - max) are rounded by it
    before they multiply V (the row sum stays unrounded), as a 16-bit
    materialisation of the weights does."""
    n, Hq, hd = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(hd)
    mask = np.triu(np.ones((n, n), dtype=bool), k=1)
    o = np.empty_like(q)
    for hq in range(Hq):
        hk = hq // G
        s = (q[:, hq, :] @ k[:, hk, :].T) * scale
        s[mask] = -np.inf
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        z = p.sum(axis=-1, keepdims=True)
        if round_p is not None:
            p = round_p(p)
        o[:, hq, :] = (p @ v[:, hk, :]) / z
    return o


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def _layer_weights(weights: Dict[str, object], l: int) -> Dict[str, np.ndarray]:
    w = {s: _f64(weights[s][l]) for s in ("ln1", "wq", "wk", "wv", "wo", "ln2", "wg", "wu", "wd")}
    for s in ("bq", "bk", "bv", "qn", "kn"):
        if weights.get(s) is not None:
            w[s] = _f64(weights[s][l])
    return w


def project_qkv(a: np.ndarray, w: Dict[str, np.ndarray], shape) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """q, k, v of normalised rows a [n, d] before RoPE: the three projections,
    plus the bias where the weight set has one, then the per-head RMSNorm of q
    and k where it has the gains."""
    n = a.shape[0]
    q, k, v = a @ w["wq"].T, a @ w["wk"].T, a @ w["wv"].T
    if "bq" in w:
        q = q + w["bq"]
    if "bk" in w:
        k = k + w["bk"]
    if "bv" in w:
        v = v + w["bv"]
    q = q.reshape(n, shape.n_q_heads, shape.head_dim)
    k = k.reshape(n, shape.n_kv_heads, shape.head_dim)
    v = v.reshape(n, shape.n_kv_heads, shape.head_dim)
    if "qn" in w:
        q = rmsnorm(q, w["qn"], shape.rms_eps)
    if "kn" in w:
        k = rmsnorm(k, w["kn"], shape.rms_eps)
    return q, k, v


def prefill_kv(weights: Dict[str, object], shape, tokens: np.ndarray,
               n_layers: Optional[int] = None, act_bf16: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """One-shot causal prefill of one request.

    `act_bf16=False` is the definition: no rounding anywhere.  `act_bf16=True`
    is the same forward under the bf16 mode's storage rule: every activation
    tensor that the mode materialises in bf16 (both norm outputs, q, the stored
    k and v that attention reads back, the attention weights and output, the
    SwiGLU output) is rounded to bf16 where it is produced; products and sums
    stay fp64 and the residual stream is never rounded.  It isolates what the
    storage format costs from what an implementation adds on top.

    Returns (K, V), each [L, n, Hkv, hd] float64 and unrounded: K after RoPE at
    position t = index in the prefix, V raw.  The last layer stops after its
    K/V (nothing downstream of them is part of the rebuilt state).
    `n_layers` limits the depth (layer l's K/V depend only on layers < l).
    """
    L = shape.n_layers if n_layers is None else n_layers
    tokens = np.asarray(tokens, dtype=np.int64)
    n = tokens.shape[0]
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    pos = np.arange(n)
    K = np.zeros((L, n, Hkv, hd))
    V = np.zeros((L, n, Hkv, hd))
    if n == 0:
        return K, V
    emb = weights["embed"]
    if hasattr(emb, "detach"):
        import torch
        h = _f64(emb[torch.as_tensor(tokens, device=emb.device)])
    else:
        h = _f64(emb[tokens])
    rb = round_bf16 if act_bf16 else (lambda x: x)
    for l in range(L):
        w = _layer_weights(weights, l)
        a = rb(rmsnorm(h, w["ln1"], shape.rms_eps))
        q, k, v = project_qkv(a, w, shape)
        q = apply_rope(q, pos, shape.rope_base)
        k = apply_rope(k, pos, shape.rope_base)
        K[l], V[l] = k, v
        if l == L - 1:
            break
        o = causal_attention(rb(q), rb(k), rb(v), round_p=rb if act_bf16 else None)
        o = rb(o).reshape(n, Hq * hd)
        h = h + o @ w["wo"].T
        b = rb(rmsnorm(h, w["ln2"], shape.rms_eps))
        h = h + rb(silu(b @ w["wg"].T) * (b @ w["wu"].T)) @ w["wd"].T
    return K, V


def resume_logits(weights: Dict[str, object], shape, tokens: np.ndarray, final_gain, lm_head,
                  act_bf16: bool = False) -> np.ndarray:
    """Next-token logits after the logged prefix: what a recovered request needs
    to resume generation (paper Sec. 4.2 step 5, Sec. 4.3).  The whole decoder,
    last layer included, over the whole prefix; final RMSNorm of the last
    position; product with the LM head [vocab, d].  `act_bf16` as in prefill_kv."""
    tokens = np.asarray(tokens, dtype=np.int64)
    n = tokens.shape[0]
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    pos = np.arange(n)
    emb = weights["embed"]
    if hasattr(emb, "detach"):
        import torch
        h = _f64(emb[torch.as_tensor(tokens, device=emb.device)])
    else:
        h = _f64(emb[tokens])
    rb = round_bf16 if act_bf16 else (lambda x: x)
    for l in range(shape.n_layers):
        w = _layer_weights(weights, l)
        a = rb(rmsnorm(h, w["ln1"], shape.rms_eps))
        q, k, v = project_qkv(a, w, shape)
        q = apply_rope(q, pos, shape.rope_base)
        k = apply_rope(k, pos, shape.rope_base)
        o = causal_attention(rb(q), rb(k), rb(v), round_p=rb if act_bf16 else None)
        h = h + rb(o).reshape(n, Hq * hd) @ w["wo"].T
        b = rb(rmsnorm(h, w["ln2"], shape.rms_eps))
        h = h + rb(silu(b @ w["wg"].T) * (b @ w["wu"].T)) @ w["wd"].T
    f = rb(rmsnorm(h[-1:], _f64(final_gain), shape.rms_eps))
    return (f @ _f64(lm_head).T)[0]


def prefill_kv_rows(weights: Dict[str, object], shape, tokens: np.ndarray, rows,
                    act_bf16: bool = False) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Sampled outputs of a long prefix, one row at a time: layer-0 K/V of every token (they need
    no attention) and layer-1 K/V of the tokens listed in `rows` only -- for those the layer-0
    attention row is written out as its definition (scores against keys 0..t, softmax, weighted sum
    of the values), followed by the rest of layer 0 and layer 1's projections.  Same mathematics
    as prefill_kv(n_layers=2) restricted to those rows, at a cost linear in the prefix length per
    sampled row; `act_bf16` applies the same storage rule as there (the same eight tensors rounded
    where they are produced).  Returns (K0 [n,Hkv,hd], V0 [n,Hkv,hd], K1 [len(rows),Hkv,hd],
    V1 [len(rows),Hkv,hd]), unrounded."""
    tokens = np.asarray(tokens, dtype=np.int64)
    rows = np.asarray(rows, dtype=np.int64)
    n = tokens.shape[0]
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    G = Hq // Hkv
    emb = weights["embed"]
    if hasattr(emb, "detach"):
        import torch
        h = _f64(emb[torch.as_tensor(tokens, device=emb.device)])
    else:
        h = _f64(emb[tokens])
    rb = round_bf16 if act_bf16 else (lambda x: x)
    w0, w1 = _layer_weights(weights, 0), _layer_weights(weights, 1)
    pos = np.arange(n)
    q, k, v = project_qkv(rb(rmsnorm(h, w0["ln1"], shape.rms_eps)), w0, shape)
    q = apply_rope(q, pos, shape.rope_base)
    k = apply_rope(k, pos, shape.rope_base)
    qs, ks, vs = rb(q), rb(k), rb(v)          # what attention reads (k, v themselves are returned unrounded)
    K1 = np.zeros((len(rows), Hkv, hd))
    V1 = np.zeros((len(rows), Hkv, hd))
    for i, t in enumerate(rows):
        o = np.zeros((Hq, hd))
        for hq in range(Hq):
            hk = hq // G
            sc = ks[:t + 1, hk, :] @ qs[t, hq, :] / math.sqrt(hd)
            pr = np.exp(sc - sc.max())
            o[hq] = (rb(pr) @ vs[:t + 1, hk, :]) / pr.sum()
        x = h[t] + w0["wo"] @ rb(o).reshape(-1)
        b = rb(rmsnorm(x[None], w0["ln2"], shape.rms_eps)[0])
        x = x + w0["wd"] @ rb(silu(w0["wg"] @ b) * (w0["wu"] @ b))
        a1 = rb(rmsnorm(x[None], w1["ln1"], shape.rms_eps))
        _, k1, v1 = project_qkv(a1, w1, shape)
        K1[i] = apply_rope(k1, np.array([t]), shape.rope_base)[0]
        V1[i] = v1[0]
    return k, v, K1, V1


def decode_incremental_kv(weights: Dict[str, object], shape, tokens: np.ndarray,
                          n_layers: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """The K/V a worker accumulates while generating: one token per step, each
    step appending its K/V row to a cache and attending over the cache so far.
    Written separately from `prefill_kv` (vector-at-a-time, explicit cache) so
    that agreement between the two is a real check of prefix consistency.
    """
    L = shape.n_layers if n_layers is None else n_layers
    tokens = np.asarray(tokens, dtype=np.int64)
    n = tokens.shape[0]
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    G = Hq // Hkv
    half = hd // 2
    inv_freq = np.array([shape.rope_base ** (-2.0 * i / hd) for i in range(half)])
    Kc = np.zeros((L, n, Hkv, hd))
    Vc = np.zeros((L, n, Hkv, hd))
    lw = [_layer_weights(weights, l) for l in range(L)]
    E = weights["embed"]
    for t in range(n):
        x = _f64(E[int(tokens[t])])
        c, s = np.cos(t * inv_freq), np.sin(t * inv_freq)
        for l in range(L):
            w = lw[l]
            a = x / math.sqrt(float(np.dot(x, x)) / x.shape[0] + shape.rms_eps) * w["ln1"]
            q = (w["wq"] @ a + w.get("bq", 0.0)).reshape(Hq, hd)
            k = (w["wk"] @ a + w.get("bk", 0.0)).reshape(Hkv, hd)
            v = (w["wv"] @ a + w.get("bv", 0.0)).reshape(Hkv, hd)
            for vec, gname in ((q, "qn"), (k, "kn")):
                if gname in w:
                    for hh in range(vec.shape[0]):
                        u = vec[hh].copy()
                        vec[hh] = u / math.sqrt(float(np.dot(u, u)) / hd + shape.rms_eps) * w[gname]
            for vec in (q, k):
                lo, hi = vec[:, :half].copy(), vec[:, half:].copy()
                vec[:, :half] = lo * c - hi * s
                vec[:, half:] = hi * c + lo * s
            Kc[l, t], Vc[l, t] = k, v
            if l == L - 1:
                break
            o = np.zeros((Hq, hd))
            for hq in range(Hq):
                hk = hq // G
                sc = Kc[l, :t + 1, hk, :] @ q[hq] / math.sqrt(hd)
                p = np.exp(sc - sc.max())
                p /= p.sum()
                o[hq] = p @ Vc[l, :t + 1, hk, :]
            x = x + w["wo"] @ o.reshape(-1)
            b = x / math.sqrt(float(np.dot(x, x)) / x.shape[0] + shape.rms_eps) * w["ln2"]
            gate, up = w["wg"] @ b, w["wu"] @ b
            x = x + w["wd"] @ (gate / (1.0 + np.exp(-gate)) * up)
    return Kc, Vc


def attention_bruteforce(q, k, v):
    """Dense n x n scores with an explicit mask, pure Python floats.  Tiny inputs only."""
    n, Hq, hd = len(q), len(q[0]), len(q[0][0])
    Hkv = len(k[0])
    G = Hq // Hkv
    out = [[[0.0] * hd for _ in range(Hq)] for _ in range(n)]
    for t in range(n):
        for hq in range(Hq):
            hk = hq // G
            scores = []
            for j in range(n):
                if j > t:
                    scores.append(None)
                else:
                    scores.append(sum(float(q[t][hq][i]) * float(k[j][hk][i]) for i in range(hd)) / math.sqrt(hd))
            m = max(s for s in scores if s is not None)
            e = [0.0 if s is None else math.exp(s - m) for s in scores]
            z = sum(e)
            for i in range(hd):
                out[t][hq][i] = sum(e[j] / z * float(v[j][hk][i]) for j in range(n))
    return out
