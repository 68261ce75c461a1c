"""CPU oracle for the stage downstream of the encoder: projector and language-model prefill up to the
first generated token (the remainder of the time-to-first-token the paper profiles).

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this module; the CUDA library never does, and the two share no code.  numpy only, float64 by default
(``dtype=np.float32`` for the wide one-layer case where matmul time matters).  ``np.matmul``, ``np.exp``,
``np.tanh``, ``np.cos`` and ``np.sin`` are the only library primitives; nothing is blocked or fused.

What the paper fixes (Sec. 3.1, "Video-LLM inference"): the encoder's tokens are aligned to the language
model's embedding space by a projector, concatenated with the text tokens and fed to the language model's
prefill; the first token ends the time-to-first-token.  The paper's model is LLaVA-OneVision-7B, whose
projector is a two-layer GELU MLP and whose language model is a Qwen2-style pre-norm decoder: RMSNorm,
grouped-query causal attention with rotary position embedding (rotate-half form, positions 0..n-1),
biases on the Q/K/V projections only, SwiGLU feed-forward, a final RMSNorm and an untied output head.
The paper prints none of these details; they are the public architecture of the named model and are
stated here as the reading this oracle follows.  Sequence order: text before the video, the visual
tokens in the encoder's output order, text after the video.

Pinning status (tests/test_oracle_prefill.py): every function is pinned against a composition of torch CPU
library ops (rms_norm, scaled_dot_product_attention with a causal mask and grouped heads, silu, gelu,
embedding, linear), the rotary embedding against complex multiplication and its closed forms (identity at
position 0, relative-position invariance of the logits, the printed angles of a 4-wide head), causality
against prefix truncation.
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np


def split_llm_weights(shape, blob: np.ndarray) -> Dict[str, np.ndarray]:
    """Views into the fp32 blob in the library's documented order (see include/earlytom_llm.h)."""
    H, V, M = shape.hidden, shape.vocab, shape.mlp_dim
    qkv = (shape.heads + 2 * shape.kv_heads) * shape.head_dim
    out: Dict[str, np.ndarray] = {}
    off = 0

    def take(name, *shp):
        nonlocal off
        n = int(np.prod(shp))
        out[name] = blob[off:off + n].reshape(shp)
        off += n

    take("embed", V, H)
    take("proj_w1", shape.vision_hidden, H); take("proj_b1", H); take("proj_w2", H, H); take("proj_b2", H)
    for i in range(shape.num_layers):
        p = f"l{i}."
        take(p + "rms1_g", H); take(p + "wqkv", H, qkv); take(p + "bqkv", qkv)
        take(p + "wo", shape.heads * shape.head_dim, H)
        take(p + "rms2_g", H); take(p + "wgu", H, 2 * M); take(p + "wd", M, H)
    take("final_g", H); take("lm_head", H, V)
    if off != blob.size:
        raise ValueError(f"weight blob has {blob.size} floats, layout needs {off}")
    return out


def rms_norm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = (x.astype(np.float64) ** 2).mean(axis=-1, keepdims=True)
    return (x.astype(np.float64) / np.sqrt(ms + eps) * g).astype(x.dtype)


def gelu(x: np.ndarray, tanh_approx: bool) -> np.ndarray:
    if tanh_approx:
        c = math.sqrt(2.0 / math.pi)
        return (0.5 * x * (1.0 + np.tanh(c * (x + 0.044715 * x ** 3)))).astype(x.dtype)
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return (0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))).astype(x.dtype)


def silu(x: np.ndarray) -> np.ndarray:
    return (x / (1.0 + np.exp(-x.astype(np.float64)))).astype(x.dtype)


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding, rotate-half form.  x [n, heads, d]; element i < d/2 pairs with i + d/2
    and the pair is rotated by the angle pos * theta^(-2i/d)."""
    n, h, d = x.shape
    half = d // 2
    inv_freq = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]          # [n, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half].astype(np.float64), x[..., half:].astype(np.float64)
    out = np.empty(x.shape, dtype=np.float64)
    out[..., :half] = a * c - b * s
    out[..., half:] = b * c + a * s
    return out.astype(x.dtype)


def causal_gqa_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """q [n, heads, d], k / v [n, kv_heads, d] -> [n, heads, d].  Query i sees keys 0..i; query head h reads
    key / value head h // (heads // kv_heads); softmax(q k^T / sqrt(d)) (Sec. 3.1)."""
    n, heads, d = q.shape
    group = heads // k.shape[1]
    out = np.empty_like(q)
    visible = np.tril(np.ones((n, n), dtype=bool))
    for h in range(heads):
        s = (q[:, h, :] @ k[:, h // group, :].T) / math.sqrt(d)
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        e = np.exp(s)
        p = e / e.sum(axis=-1, keepdims=True)
        out[:, h, :] = p @ v[:, h // group, :]
    return out


def projector(tokens: np.ndarray, w, shape) -> np.ndarray:
    """Two-layer GELU MLP from the encoder's width to the language model's width."""
    dt = tokens.dtype
    h = gelu(tokens @ w["proj_w1"].astype(dt) + w["proj_b1"].astype(dt), bool(shape.gelu_tanh))
    return h @ w["proj_w2"].astype(dt) + w["proj_b2"].astype(dt)


def decoder_layer(X: np.ndarray, w, layer: int, shape, kv_out: Optional[list] = None) -> np.ndarray:
    """One pre-norm decoder block on the whole sequence X [n, hidden].  kv_out, if given, receives this layer's
    (rotated keys [n, kv_heads, d], values [n, kv_heads, d]): what a decoder would cache."""
    p = f"l{layer}."
    n, dt = X.shape[0], X.dtype
    H, KV, d = shape.heads, shape.kv_heads, shape.head_dim
    xn = rms_norm(X, w[p + "rms1_g"], shape.rms_eps)
    qkv = xn @ w[p + "wqkv"].astype(dt) + w[p + "bqkv"].astype(dt)
    q = qkv[:, :H * d].reshape(n, H, d)
    k = qkv[:, H * d:(H + KV) * d].reshape(n, KV, d)
    v = qkv[:, (H + KV) * d:].reshape(n, KV, d)
    pos = np.arange(n)
    k_rot = rope(k, pos, shape.rope_theta)
    if kv_out is not None:
        kv_out.append((k_rot.copy(), v.copy()))
    ctx = causal_gqa_attention(rope(q, pos, shape.rope_theta), k_rot, v)
    X = X + ctx.reshape(n, H * d) @ w[p + "wo"].astype(dt)
    xn = rms_norm(X, w[p + "rms2_g"], shape.rms_eps)
    gu = xn @ w[p + "wgu"].astype(dt)
    M = shape.mlp_dim
    return X + (silu(gu[:, :M]) * gu[:, M:]) @ w[p + "wd"].astype(dt)


def assemble_sequence(shape, w, prefix_ids, visual_tokens: np.ndarray, suffix_ids, dtype) -> np.ndarray:
    """[embeddings of the text before | projected visual tokens | embeddings of the text after]."""
    parts = []
    if len(prefix_ids):
        parts.append(w["embed"][np.asarray(prefix_ids, dtype=np.int64)].astype(dtype))
    if len(visual_tokens):
        parts.append(projector(visual_tokens.astype(dtype), w, shape))
    if len(suffix_ids):
        parts.append(w["embed"][np.asarray(suffix_ids, dtype=np.int64)].astype(dtype))
    return np.concatenate(parts, axis=0)


def prefill(shape, w, prefix_ids, visual_tokens: np.ndarray, suffix_ids, dtype=np.float64,
            want_hidden: bool = False, want_kv: bool = False) -> dict:
    """Prefill of the whole sequence; the logits of the last position give the first generated token."""
    X = assemble_sequence(shape, w, prefix_ids, visual_tokens, suffix_ids, dtype)
    embeds = X.copy() if want_hidden else None
    kv = [] if want_kv else None
    for layer in range(shape.num_layers):
        X = decoder_layer(X, w, layer, shape, kv)
    last = rms_norm(X[-1:], w["final_g"], shape.rms_eps)
    logits = (last @ w["lm_head"].astype(dtype))[0]
    return dict(logits=logits, first_token=int(np.argmax(logits)), last_hidden=X[-1].copy(),
                hidden=X if want_hidden else None, embeds=embeds, n_tokens=X.shape[0], kv=kv)


def prefill_flops(shape, n_tokens: int, n_vis: int) -> float:
    """Multiply-add count x 2 of the downstream stage, in the manner of Eq. 8 (per-layer projections,
    attention products and feed-forward) with this model's grouped K/V width, causal attention (half of the
    n^2 products) and three feed-forward matrices; plus projector and output head of the last position."""
    H, M, d = shape.hidden, shape.mlp_dim, shape.head_dim
    n = float(n_tokens)
    per_layer = 2.0 * n * H * (shape.heads + 2 * shape.kv_heads) * d + 2.0 * n * shape.heads * d * H \
        + 2.0 * n * n * shape.heads * d + 6.0 * n * H * M
    proj = 2.0 * n_vis * (shape.vision_hidden * H + H * H)
    return shape.num_layers * per_layer + proj + 2.0 * H * shape.vocab
