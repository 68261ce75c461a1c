"""CPU oracle of the Qwen2.5-VL-style vision encoder (the architecture of the paper's generalisation study,
supplementary "Generalizability Analysis", Qwen2.5-VL-7B table).

TEST INFRASTRUCTURE ONLY, like `earlytom_oracle`: only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it; the CUDA library shares no code with it.  numpy only.

The paper names the model and prints nothing of its architecture, so the encoder follows the public description of
Qwen2.5-VL's vision tower (pinned against torch CPU library ops in tests/test_oracle_qwenvl.py, not against the paper):

  patch embedding     a convolution over (temporal_patch frames) x (patch x patch pixels) with stride = kernel, no bias:
                      `temporal_patch` input frames become ONE encoder frame of (H/p) * (W/p) tokens
  blocks              x += W_o MHA(RMSNorm(x)) + b_o ;  x += W_d (silu(gate) * up) + b_d, [gate | up] = RMSNorm(x) W_gu + b_gu
  positions           2-D rotary embedding on q and k: the first half of the rotated pairs turns with the token's row in
                      the patch grid, the second half with its column (rotate-half pairing: element i with i + dh/2),
                      frequencies theta^(-2i / (dh/2)), i = 0 .. dh/4 - 1
  attention           inside windows of `window` x `window` patches, except in the blocks of `full_attn_layers`, where
                      every token of an encoder frame attends to the whole frame (never across frames)
  output              RMSNorm with the final gain (the norm that precedes the model's patch merger); the 2 x 2 patch merger
                      itself is not part of this path: the paper does not say how token selection and the merger combine

Everything of the method (Stage I at the merge layers, Stage II at the output) is `earlytom_oracle`'s, applied to encoder
frames: `earlytom_oracle.encode_video` calls `embed` / `encoder_block` / `final_norm` of this module when
`shape.arch == 1`.  Tokens are kept in raster order throughout (a window is a set of indices, not a re-ordering).
"""
from __future__ import annotations

import math
from typing import Dict

import numpy as np


def split_weights(shape, blob: np.ndarray) -> Dict[str, np.ndarray]:
    """Views into the fp32 blob in the library's documented order for this architecture (include/earlytom.h)."""
    D, M = shape.hidden, shape.mlp_dim
    P = 3 * shape.temporal_patch * shape.patch_size * shape.patch_size
    out: Dict[str, np.ndarray] = {}
    off = 0

    def take(name, *shp):
        nonlocal off
        n = int(np.prod(shp))
        out[name] = blob[off:off + n].reshape(shp)
        off += n

    take("patch_w", P, D)
    for i in range(shape.num_layers):
        p = f"l{i}."
        take(p + "n1_g", D)
        take(p + "wqkv", D, 3 * D); take(p + "bqkv", 3 * D)
        take(p + "wo", D, D); take(p + "bo", D)
        take(p + "n2_g", D)
        take(p + "wgu", D, 2 * M); take(p + "bgu", 2 * M)
        take(p + "wd", M, D); take(p + "bd", D)
    take("post_g", D)
    if off != blob.size:
        raise ValueError(f"weight blob has {blob.size} floats, layout needs {off}")
    return out


def patchify3d(frames: np.ndarray, patch: int, tp: int) -> np.ndarray:
    """[B,3,H,W] -> [B/tp, L, 3*tp*p*p]; feature index c*tp*p*p + t*p*p + dy*p + dx (the flattening of a
    [D][3][tp][p][p] convolution weight); row-major patch grid over the top-left (H//p*p) x (W//p*p) crop."""
    B, C, H, W = frames.shape
    if B % tp:
        raise ValueError("the number of frames must be a multiple of the temporal patch")
    gh, gw = H // patch, W // patch
    x = frames[:, :, :gh * patch, :gw * patch].reshape(B // tp, tp, C, gh, patch, gw, patch)
    x = x.transpose(0, 3, 5, 2, 1, 4, 6)          # n, gy, gx, c, t, dy, dx
    return x.reshape(B // tp, gh * gw, C * tp * patch * patch)


def embed(frames: np.ndarray, shape, w) -> np.ndarray:
    return patchify3d(frames, shape.patch_size, shape.temporal_patch) @ w["patch_w"].astype(frames.dtype)


def rms_norm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = (x.astype(np.float64) ** 2).mean(axis=-1, keepdims=True)
    return (x.astype(np.float64) / np.sqrt(ms + eps) * g).astype(x.dtype)


def rope_angles(shape) -> np.ndarray:
    """[L, dh/2] rotation angle of pair i of the token at raster position l = gy * grid + gx."""
    dh, g = shape.head_dim, shape.grid
    if dh % 4:
        raise ValueError("2-D rotary positions need a head dim that is a multiple of 4")
    quarter = dh // 4
    inv_freq = np.array([shape.rope_theta ** (-2.0 * i / (dh // 2)) for i in range(quarter)], dtype=np.float64)
    gy, gx = np.divmod(np.arange(g * g), g)
    return np.concatenate([gy[:, None] * inv_freq[None, :], gx[:, None] * inv_freq[None, :]], axis=1)


def apply_rope(x: np.ndarray, ang: np.ndarray) -> np.ndarray:
    """x [L, dh]: pair (x[i], x[i + dh/2]) is turned by ang[:, i]."""
    h = x.shape[-1] // 2
    c, s = np.cos(ang), np.sin(ang)
    a, b = x[:, :h].astype(np.float64), x[:, h:].astype(np.float64)
    return np.concatenate([a * c - b * s, b * c + a * s], axis=1).astype(x.dtype)


def window_ids(shape) -> np.ndarray:
    """[L] window of each raster position: windows tile the patch grid in blocks of window x window patches (the
    last row / column of windows is smaller when the grid is not a multiple)."""
    g, ws = shape.grid, shape.window
    gy, gx = np.divmod(np.arange(g * g), g)
    per_row = -(-g // ws)
    return (gy // ws) * per_row + gx // ws


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def mha(xn: np.ndarray, w, p: str, shape, full: bool, want_scores: bool):
    """Self-attention of one encoder frame.  Returns (projected output [L, D], per-token attention score [L] or None):
    the score is the mean over heads and queries of the probability a key receives (0 from queries outside its window)."""
    L, D = xn.shape
    H, dh = shape.heads, shape.head_dim
    qkv = xn @ w[p + "wqkv"].astype(xn.dtype) + w[p + "bqkv"].astype(xn.dtype)
    q, k, v = qkv[:, :D], qkv[:, D:2 * D], qkv[:, 2 * D:]
    ang = rope_angles(shape)
    groups = [np.arange(L)] if full else [np.nonzero(window_ids(shape) == i)[0] for i in range(int(window_ids(shape).max()) + 1)]
    ctx = np.empty_like(xn)
    score = np.zeros(L, dtype=np.float64) if want_scores else None
    for h in range(H):
        sl = slice(h * dh, (h + 1) * dh)
        qh, kh = apply_rope(q[:, sl], ang), apply_rope(k[:, sl], ang)
        for idx in groups:
            P = softmax_rows((qh[idx] @ kh[idx].T) / math.sqrt(dh))
            ctx[idx, sl] = P @ v[idx, sl]
            if want_scores:
                score[idx] += P.astype(np.float64).sum(axis=0)
    if want_scores:
        score /= float(H * L)
    return ctx @ w[p + "wo"].astype(xn.dtype) + w[p + "bo"].astype(xn.dtype), score


def silu(x: np.ndarray) -> np.ndarray:
    return (x / (1.0 + np.exp(-x.astype(np.float64)))).astype(x.dtype)


def encoder_block(X: np.ndarray, w, layer: int, shape, want_scores: bool):
    """X [n, L, D] -> X after block `layer`; optionally the attention scores A [n, L]."""
    p = f"l{layer}."
    n, L, D = X.shape
    M = shape.mlp_dim
    full = (shape.window <= 0) or (layer in tuple(shape.full_attn_layers))
    A = np.zeros((n, L), dtype=np.float64) if want_scores else None
    out = np.empty_like(X)
    for f in range(n):
        x = X[f]
        a, sc = mha(rms_norm(x, w[p + "n1_g"], shape.ln_eps), w, p, shape, full, want_scores)
        x = x + a
        gu = rms_norm(x, w[p + "n2_g"], shape.ln_eps) @ w[p + "wgu"].astype(x.dtype) + w[p + "bgu"].astype(x.dtype)
        hmid = silu(gu[:, :M]) * gu[:, M:]
        x = x + (hmid @ w[p + "wd"].astype(x.dtype) + w[p + "bd"].astype(x.dtype))
        out[f] = x
        if want_scores:
            A[f] = sc
    return out, A


def final_norm(X: np.ndarray, w, shape) -> np.ndarray:
    return rms_norm(X, w["post_g"], shape.ln_eps) if shape.post_layernorm else X
