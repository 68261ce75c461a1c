"""Pins of the downstream oracle (projector + language-model prefill) against torch CPU library ops,
closed forms of the rotary embedding and structural invariants.  No GPU."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import prefill_oracle as P
from synthetic.llm import LLM_ODD, LLM_TINY, LlmShape, llm_blob_size, llm_weight_layout, make_llm_weights, make_prompt, make_visual_tokens

SHAPE = LlmShape(vision_hidden=24, hidden=32, num_layers=2, heads=4, kv_heads=2, head_dim=8, mlp_dim=48, vocab=50,
                 rope_theta=100.0)


def _setup(shape=SHAPE, n_prefix=3, n_vis=7, n_suffix=4, seed=5):
    blob = make_llm_weights(shape, seed)
    w = P.split_llm_weights(shape, blob)
    pre, suf = make_prompt(shape, n_prefix, n_suffix, seed)
    vis = make_visual_tokens(shape, n_vis, seed)
    return blob, w, pre, vis, suf


def test_blob_layout_matches_generator():
    blob = make_llm_weights(SHAPE, 1)
    assert blob.size == llm_blob_size(SHAPE)
    w = P.split_llm_weights(SHAPE, blob)
    for name, shp, off in llm_weight_layout(SHAPE):
        assert w[name].shape == shp
        assert np.shares_memory(w[name], blob) and w[name].ravel()[0] == blob[off]
    with pytest.raises(ValueError):
        P.split_llm_weights(SHAPE, blob[:-1])


def test_rms_norm_silu_gelu_against_torch():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 32)) * 3.0
    g = 1.0 + 0.1 * rng.standard_normal(32)
    ref = F.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), eps=1e-6).numpy()
    np.testing.assert_allclose(P.rms_norm(x, g, 1e-6), ref, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(P.silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(P.gelu(x, True), F.gelu(torch.from_numpy(x), approximate="tanh").numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(P.gelu(x, False), F.gelu(torch.from_numpy(x)).numpy(), rtol=1e-12, atol=1e-12)
    assert P.silu(np.zeros(1))[0] == 0.0 and abs(P.silu(np.array([30.0]))[0] - 30.0) < 1e-10


def test_rope_closed_forms():
    # a 2-wide head: one pair, angle = position (theta^0 = 1): (1, 0) -> (cos p, sin p)
    x = np.zeros((4, 1, 2)); x[..., 0] = 1.0
    pos = np.array([0, 1, 2, 5])
    y = P.rope(x, pos, 10000.0)
    np.testing.assert_allclose(y[:, 0, 0], np.cos(pos), atol=1e-15)
    np.testing.assert_allclose(y[:, 0, 1], np.sin(pos), atol=1e-15)
    # a 4-wide head, theta = 10000: pair (0, 2) turns by p, pair (1, 3) by p / 100
    x = np.zeros((1, 1, 4)); x[0, 0, 1] = 2.0
    y = P.rope(x, np.array([7]), 10000.0)
    np.testing.assert_allclose(y[0, 0], [0.0, 2.0 * math.cos(0.07), 0.0, 2.0 * math.sin(0.07)], atol=1e-15)
    # position 0 is the identity; rotation preserves the norm of every pair
    rng = np.random.default_rng(1)
    q = rng.standard_normal((6, 3, 8)); k = rng.standard_normal((6, 3, 8))
    np.testing.assert_array_equal(P.rope(q[:1], np.array([0]), 1e6), q[:1])
    np.testing.assert_allclose(np.linalg.norm(P.rope(q, np.arange(6), 50.0), axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    # the logit of (query at m, key at n) depends on m - n only
    a = np.einsum("ihd,jhd->hij", P.rope(q, np.arange(6), 50.0), P.rope(k, np.arange(6), 50.0))
    b = np.einsum("ihd,jhd->hij", P.rope(q, np.arange(6) + 11, 50.0), P.rope(k, np.arange(6) + 11, 50.0))
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-11)


def _rope_complex(x: torch.Tensor, theta: float) -> torch.Tensor:
    """Independent route: pairs (i, i + d/2) as complex numbers times exp(i * pos * theta^(-2i/d))."""
    n, h, d = x.shape
    half = d // 2
    freq = theta ** (-torch.arange(half, dtype=torch.float64) * 2.0 / d)
    ang = torch.arange(n, dtype=torch.float64)[:, None] * freq[None, :]
    z = torch.complex(x[..., :half], x[..., half:]) * torch.polar(torch.ones_like(ang), ang)[:, None, :]
    return torch.cat([z.real, z.imag], dim=-1)


def _torch_prefill(shape, w, pre, vis, suf):
    t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in w.items()}
    parts = []
    if len(pre):
        parts.append(F.embedding(torch.from_numpy(pre.astype(np.int64)), t["embed"]))
    if len(vis):
        h = F.gelu(F.linear(torch.from_numpy(vis.astype(np.float64)), t["proj_w1"].T, t["proj_b1"]),
                   approximate="tanh" if shape.gelu_tanh else "none")
        parts.append(F.linear(h, t["proj_w2"].T, t["proj_b2"]))
    if len(suf):
        parts.append(F.embedding(torch.from_numpy(suf.astype(np.int64)), t["embed"]))
    X = torch.cat(parts, dim=0)
    n, H, KV, d, M = X.shape[0], shape.heads, shape.kv_heads, shape.head_dim, shape.mlp_dim
    kv = []
    for i in range(shape.num_layers):
        p = f"l{i}."
        xn = F.rms_norm(X, (shape.hidden,), t[p + "rms1_g"], eps=shape.rms_eps)
        qkv = F.linear(xn, t[p + "wqkv"].T, t[p + "bqkv"])
        q = _rope_complex(qkv[:, :H * d].reshape(n, H, d), shape.rope_theta)
        k = _rope_complex(qkv[:, H * d:(H + KV) * d].reshape(n, KV, d), shape.rope_theta)
        v = qkv[:, (H + KV) * d:].reshape(n, KV, d)
        kv.append((k.numpy().copy(), v.numpy().copy()))
        ctx = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
                                             is_causal=True, enable_gqa=True)[0].transpose(0, 1).reshape(n, H * d)
        X = X + F.linear(ctx, t[p + "wo"].T)
        xn = F.rms_norm(X, (shape.hidden,), t[p + "rms2_g"], eps=shape.rms_eps)
        gu = F.linear(xn, t[p + "wgu"].T)
        X = X + F.linear(F.silu(gu[:, :M]) * gu[:, M:], t[p + "wd"].T)
    last = F.rms_norm(X[-1:], (shape.hidden,), t["final_g"], eps=shape.rms_eps)
    return X.numpy(), F.linear(last, t["lm_head"].T)[0].numpy(), kv


@pytest.mark.parametrize("shape", [SHAPE, LLM_TINY, LLM_ODD])
def test_prefill_against_torch_composition(shape):
    blob, w, pre, vis, suf = _setup(shape)
    got = P.prefill(shape, w, pre, vis, suf, want_hidden=True, want_kv=True)
    X, logits, kv = _torch_prefill(shape, w, pre, vis, suf)
    np.testing.assert_allclose(got["hidden"], X, rtol=1e-9, atol=1e-9)
    assert len(got["kv"]) == shape.num_layers
    for (k_o, v_o), (k_t, v_t) in zip(got["kv"], kv):         # what a decoder would cache: rotated keys, values
        np.testing.assert_allclose(k_o, k_t, rtol=1e-9, atol=1e-9)
        np.testing.assert_allclose(v_o, v_t, rtol=1e-9, atol=1e-9)
    np.testing.assert_allclose(got["logits"], logits, rtol=1e-9, atol=1e-9)
    assert got["first_token"] == int(np.argmax(logits)) and got["n_tokens"] == len(pre) + len(vis) + len(suf)


def test_sequence_order_and_projector():
    blob, w, pre, vis, suf = _setup()
    X = P.assemble_sequence(SHAPE, w, pre, vis, suf, np.float64)
    np.testing.assert_array_equal(X[:3], w["embed"][pre].astype(np.float64))
    np.testing.assert_array_equal(X[-4:], w["embed"][suf].astype(np.float64))
    mid = P.projector(vis.astype(np.float64), w, SHAPE)
    np.testing.assert_array_equal(X[3:10], mid)
    # text only and video only both work
    assert P.assemble_sequence(SHAPE, w, pre, vis[:0], suf, np.float64).shape[0] == 7
    assert P.assemble_sequence(SHAPE, w, pre[:0], vis, suf[:0], np.float64).shape[0] == 7


def test_causality_prefix_truncation():
    """Hidden states of the first m positions do not depend on what follows them."""
    blob, w, pre, vis, suf = _setup()
    full = P.prefill(SHAPE, w, pre, vis, suf, want_hidden=True)["hidden"]
    cut = P.prefill(SHAPE, w, pre, vis[:4], suf[:0], want_hidden=True)["hidden"]
    np.testing.assert_allclose(full[:7], cut, rtol=1e-12, atol=1e-12)
    other = P.prefill(SHAPE, w, pre, vis, (suf + 1) % SHAPE.vocab, want_hidden=True)["hidden"]
    np.testing.assert_allclose(full[:10], other[:10], rtol=1e-12, atol=1e-12)
    assert np.abs(full[10:] - other[10:]).max() > 1e-3


def test_grouped_heads_equal_repeated_heads():
    rng = np.random.default_rng(3)
    q = rng.standard_normal((9, 4, 8)); k = rng.standard_normal((9, 2, 8)); v = rng.standard_normal((9, 2, 8))
    a = P.causal_gqa_attention(q, k, v)
    b = P.causal_gqa_attention(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1))
    np.testing.assert_array_equal(a, b)
    # the first query sees only the first key: its output is that key's value row
    np.testing.assert_allclose(a[0], np.repeat(v[0], 2, axis=0), rtol=1e-14)


def test_flop_count_of_the_7b_shape():
    from synthetic.llm import QWEN2_7B
    n = 8000
    f = P.prefill_flops(QWEN2_7B, n, 7800)
    dense = 2.0 * n * (3584 * 4608 + 3584 * 3584 + 3 * 3584 * 18944) * 28
    attn = 2.0 * n * n * 3584 * 28
    assert abs(f - (dense + attn + 2.0 * 7800 * (1152 * 3584 + 3584 * 3584) + 2.0 * 3584 * 152064)) < 1e-6 * f
