"""CPU oracle for one pipeline stage of a decoder-only LLM.  TEST INFRASTRUCTURE ONLY.

This file is the checker the GPU library is compared against.  It is plain numpy in
float64, un-paged, un-fused, one sequence at a time, written straight from the
definitions.  It shares no code with the CUDA path and must never be imported by it.

What the paper fixes (Section III-A, "Modeling of LLM Structure"): a decoder block is
RMSNorm -> grouped-query attention with rotary position encoding -> RMSNorm -> SwiGLU
feed-forward, the norm applied *before* each sub-layer; blocks are chained strictly in
order (B_i -> B_{i+1}); a stage is a contiguous index range of blocks (the index set
I_j(p) of Section III-C).  The paper gives no arithmetic beyond the operator names, so
each operator below is its standard definition; the readings taken where the paper is
silent are listed next to each function.

Parity against trained Phi-3-medium weights: parity unpinned (no such weights are used;
all inputs are seeded random-init tensors).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """RMS Norm (named in Section III-A).  y = x / sqrt(mean(x^2) + eps) * g, eps inside
    the root, mean over the hidden axis."""
    x = np.asarray(x, F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(g, F64)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position encoding (named in Section III-A as part of GQA).

    x: [T, heads, D]; pos: [T] absolute positions starting at 0.  Half-split pairing:
    element i pairs with i + D/2 for i in [0, D/2); the pair is rotated by the angle
    pos * theta^(-2i/D).  No scaling variants."""
    x = np.asarray(x, F64)
    T, nh, D = x.shape
    half = D // 2
    i = np.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * i / D)
    ang = np.asarray(pos, F64)[:, None] * inv_freq[None, :]          # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    """Row softmax with the row maximum subtracted first."""
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_probs(q: np.ndarray, k: np.ndarray, q_pos0: int = 0) -> np.ndarray:
    """Causal grouped-query attention weights.

    q: [Tq, Hq, D] (already rotated), k: [Tk, Hkv, D] (already rotated).  Query row t sits
    at absolute position q_pos0 + t and may see keys at positions <= its own.  Query head h
    reads KV head floor(h / (Hq/Hkv)).  Scale 1/sqrt(D).  Returns [Hq, Tq, Tk]."""
    Tq, Hq, D = q.shape
    Tk, Hkv, _ = k.shape
    G = Hq // Hkv
    P = np.zeros((Hq, Tq, Tk), F64)
    qpos = q_pos0 + np.arange(Tq)
    mask = np.arange(Tk)[None, :] <= qpos[:, None]                  # [Tq, Tk]
    for h in range(Hq):
        s = (q[:, h, :] @ k[:, h // G, :].T) / np.sqrt(F64(D))
        s = np.where(mask, s, -np.inf)
        P[h] = softmax_rows(s)
    return P


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, q_pos0: int = 0) -> np.ndarray:
    """softmax(q k^T / sqrt(D)) v with the causal mask and GQA head mapping above.
    Returns [Tq, Hq, D]."""
    Tq, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    P = attention_probs(q, k, q_pos0)
    out = np.empty((Tq, Hq, D), F64)
    for h in range(Hq):
        out[:, h, :] = P[h] @ v[:, h // G, :]
    return out


def silu(z: np.ndarray) -> np.ndarray:
    """SiLU(z) = z / (1 + exp(-z))."""
    return z / (1.0 + np.exp(-z))


def swiglu_ffn(h: np.ndarray, wgu: np.ndarray, wd: np.ndarray) -> np.ndarray:
    """SwiGLU feed-forward (named in Section III-A): (SiLU(h Wg^T) * (h Wu^T)) Wd^T.
    wgu rows are [gate (F); up (F)], every matrix stored [out, in]; no biases."""
    F = wgu.shape[0] // 2
    gu = h @ wgu.T
    return (silu(gu[:, :F]) * gu[:, F:]) @ wd.T


class Shape:
    """Decoder dimensions the oracle needs (its own record; nothing is shared with the library)."""

    def __init__(self, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab, rms_eps, rope_theta):
        self.hidden, self.n_q_heads, self.n_kv_heads = hidden, n_q_heads, n_kv_heads
        self.head_dim, self.ffn, self.vocab = head_dim, ffn, vocab
        self.rms_eps, self.rope_theta = rms_eps, rope_theta


def qkv_project(x: np.ndarray, w: dict, sh: Shape, pos: np.ndarray):
    """Pre-norm + QKV projection + rotation.  wqkv rows are [Q (Hq*D); K (Hkv*D); V (Hkv*D)]."""
    T = x.shape[0]
    Hq, Hkv, D = sh.n_q_heads, sh.n_kv_heads, sh.head_dim
    h = rmsnorm(x, w["g1"], sh.rms_eps)
    qkv = h @ w["wqkv"].T
    q = qkv[:, :Hq * D].reshape(T, Hq, D)
    k = qkv[:, Hq * D:(Hq + Hkv) * D].reshape(T, Hkv, D)
    v = qkv[:, (Hq + Hkv) * D:].reshape(T, Hkv, D)
    return rope(q, pos, sh.rope_theta), rope(k, pos, sh.rope_theta), v


def block_forward(x: np.ndarray, w: dict, sh: Shape, pos0: int = 0,
                  k_past: np.ndarray | None = None, v_past: np.ndarray | None = None):
    """One decoder block B_i on one sequence (Section III-A).

    x: [T, H] rows at absolute positions pos0 .. pos0+T-1.  k_past / v_past: rotated keys and
    values of positions 0 .. pos0-1 (None when pos0 == 0).  Residual placement is
    x + sublayer(norm(x)) for both sub-layers.  Returns (x_out, k_all, v_all)."""
    T = x.shape[0]
    x = np.asarray(x, F64)
    pos = pos0 + np.arange(T)
    q, k, v = qkv_project(x, w, sh, pos)
    if k_past is not None and k_past.shape[0] > 0:
        k = np.concatenate([k_past, k], axis=0)
        v = np.concatenate([v_past, v], axis=0)
    a = attention(q, k, v, q_pos0=pos0).reshape(T, -1)
    x = x + a @ w["wo"].T
    h = rmsnorm(x, w["g2"], sh.rms_eps)
    x = x + swiglu_ffn(h, w["wgu"], w["wd"])
    return x, k, v


def embed(ids: np.ndarray, E: np.ndarray) -> np.ndarray:
    """First-stage input: the token's embedding row, no scaling."""
    return np.asarray(E, F64)[np.asarray(ids, np.int64)]


def lm_head(x: np.ndarray, gf: np.ndarray, wlm: np.ndarray, eps: float) -> np.ndarray:
    """Last-stage output: logits = RMSNorm(x; gf) Wlm^T (head untied from the embedding)."""
    return rmsnorm(x, gf, eps) @ np.asarray(wlm, F64).T


def stage_forward(x: np.ndarray, layers, sh: Shape) -> np.ndarray:
    """Full-sequence causal pass of blocks `layers` (an iterable yielding the weight dict of
    each block of the stage in order) over one sequence x [T, H] starting at position 0.

    With teacher forcing, row t of the result is what a KV-cached decode step that feeds token
    t after caching tokens 0..t-1 must produce (see `stage_decode_cached` for the literal loop)."""
    x = np.asarray(x, F64)
    for w in layers:
        x, _, _ = block_forward(x, w, sh, 0)
    return x


class CachedStage:
    """Literal KV-cached evaluation of a stage on one sequence: a prefill call caches the keys
    and values of its rows; each later call appends rows and attends to the whole cache.  Used to
    prove that cached decode equals the full-sequence pass."""

    def __init__(self, layers, sh: Shape):
        self.layers = list(layers)
        self.sh = sh
        self.k = [None] * len(self.layers)
        self.v = [None] * len(self.layers)
        self.n_cached = 0

    def step(self, x: np.ndarray) -> np.ndarray:
        x = np.asarray(x, F64)
        for i, w in enumerate(self.layers):
            x, self.k[i], self.v[i] = block_forward(x, w, self.sh, self.n_cached, self.k[i], self.v[i])
        self.n_cached += x.shape[0]
        return x


def as_f64_weights(w: dict) -> dict:
    """Exact up-conversion of a dict of bf16-valued arrays (already numpy float) to float64."""
    return {k: np.asarray(v, F64) for k, v in w.items()}


def cosine(a: np.ndarray, b: np.ndarray) -> float:
    a = np.asarray(a, F64).ravel()
    b = np.asarray(b, F64).ravel()
    return float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))
