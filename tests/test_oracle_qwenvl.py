"""Pins of the Qwen2.5-VL-style encoder oracle (oracle/qwenvl_oracle.py): every piece against a torch CPU library op or
a closed form, the assembled block and the whole uncompressed encoder against a composition of torch ops.  CPU only."""
import dataclasses
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import earlytom_oracle as O
from oracle import qwenvl_oracle as Q
from synthetic import EncoderShape, MergeParams, make_video, make_weights

SHAPE = EncoderShape(image_size=84, patch_size=14, num_layers=3, hidden=48, heads=3, mlp_dim=40, arch=1,
                     temporal_patch=2, window=4, full_attn_layers=(1,))          # grid 6: ragged windows (4 + 2)


def t64(a):
    return torch.from_numpy(np.ascontiguousarray(a)).double()


def test_patch_embedding_is_a_strided_3d_convolution():
    rng = np.random.default_rng(0)
    frames = rng.standard_normal((4, 3, 84, 84))
    w = Q.split_weights(SHAPE, make_weights(SHAPE, 1).astype(np.float64))
    got = Q.embed(frames, SHAPE, w)                                             # [2, 36, 48]
    kernel = t64(w["patch_w"]).T.reshape(48, 3, 2, 14, 14)                      # [D][c][t][dy][dx]
    vol = t64(frames).reshape(2, 2, 3, 84, 84).permute(0, 2, 1, 3, 4)           # [n, c, t, H, W]
    ref = F.conv3d(vol, kernel, stride=(2, 14, 14))                             # [n, D, 1, 6, 6]
    ref = ref.reshape(2, 48, 36).permute(0, 2, 1).numpy()
    np.testing.assert_allclose(got, ref, atol=1e-10)
    with pytest.raises(ValueError):
        Q.patchify3d(frames[:3], 14, 2)


def test_rms_norm_matches_torch():
    rng = np.random.default_rng(1)
    x, g = rng.standard_normal((7, 48)), rng.standard_normal(48)
    ref = F.rms_norm(t64(x), (48,), weight=t64(g), eps=1e-6).numpy()
    np.testing.assert_allclose(Q.rms_norm(x, g, 1e-6), ref, atol=1e-12)


def test_rope_is_complex_rotation_by_row_and_column():
    rng = np.random.default_rng(2)
    shape = dataclasses.replace(SHAPE, hidden=96, heads=3)                      # head dim 32: 8 row pairs + 8 column pairs
    ang = Q.rope_angles(shape)
    L, dh = shape.tokens_per_frame, 32
    assert ang.shape == (L, 16)
    g = shape.grid
    for l in (0, 5, 13, 35):
        gy, gx = divmod(l, g)
        for i in range(8):
            f = 10000.0 ** (-2.0 * i / 16)
            assert abs(ang[l, i] - gy * f) < 1e-12 and abs(ang[l, 8 + i] - gx * f) < 1e-12
    x = rng.standard_normal((L, dh))
    y = Q.apply_rope(x, ang)
    z = (x[:, :16] + 1j * x[:, 16:]) * np.exp(1j * ang)                         # pair (i, i + dh/2) as a complex number
    np.testing.assert_allclose(y, np.concatenate([z.real, z.imag], axis=1), atol=1e-12)
    np.testing.assert_allclose(y[0], x[0], atol=1e-15)                          # position (0, 0): identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), atol=1e-12)
    # relative positions: <rot(q, a), rot(k, b)> depends only on (row(a) - row(b), col(a) - col(b))
    q, k = rng.standard_normal(dh), rng.standard_normal(dh)
    def logit(a, b):
        return float(Q.apply_rope(q[None], ang[a:a + 1])[0] @ Q.apply_rope(k[None], ang[b:b + 1])[0])
    assert abs(logit(1 * g + 2, 0 * g + 1) - logit(4 * g + 5, 3 * g + 4)) < 1e-10     # both (+1, +1)
    assert abs(logit(1 * g + 2, 0 * g + 1) - logit(1 * g + 1, 0 * g + 2)) > 1e-3      # (+1, -1) differs


def test_window_ids_bruteforce():
    ids = Q.window_ids(SHAPE)                                                   # grid 6, windows of 4: 2 x 2 windows
    for gy in range(6):
        for gx in range(6):
            assert ids[gy * 6 + gx] == (gy >= 4) * 2 + (gx >= 4)
    assert np.bincount(ids).tolist() == [16, 8, 8, 4]


def torch_block(x, w, p, shape, full):
    """One block as a composition of torch CPU ops (fp64)."""
    D, H, dh, M = shape.hidden, shape.heads, shape.head_dim, shape.mlp_dim
    L = x.shape[0]
    xn = F.rms_norm(x, (D,), weight=t64(w[p + "n1_g"]), eps=shape.ln_eps)
    qkv = F.linear(xn, t64(w[p + "wqkv"]).T, t64(w[p + "bqkv"]))
    q, k, v = (t.reshape(L, H, dh).permute(1, 0, 2) for t in qkv.split(D, dim=1))          # [H, L, dh]
    ang = t64(Q.rope_angles(shape))
    rot = torch.polar(torch.ones_like(ang), ang)                                            # e^{i ang}
    def rope(t):
        z = torch.complex(t[..., :dh // 2], t[..., dh // 2:]) * rot
        return torch.cat([z.real, z.imag], dim=-1)
    ids = torch.from_numpy(Q.window_ids(shape))
    mask = None if full else (ids[:, None] == ids[None, :])
    ctx = F.scaled_dot_product_attention(rope(q), rope(k), v, attn_mask=mask)               # scale 1/sqrt(dh)
    x = x + F.linear(ctx.permute(1, 0, 2).reshape(L, D), t64(w[p + "wo"]).T, t64(w[p + "bo"]))
    gu = F.linear(F.rms_norm(x, (D,), weight=t64(w[p + "n2_g"]), eps=shape.ln_eps), t64(w[p + "wgu"]).T, t64(w[p + "bgu"]))
    return x + F.linear(F.silu(gu[:, :M]) * gu[:, M:], t64(w[p + "wd"]).T, t64(w[p + "bd"]))


def test_blocks_match_torch_composition_window_and_full():
    rng = np.random.default_rng(3)
    w = Q.split_weights(SHAPE, make_weights(SHAPE, 2).astype(np.float64))
    X = rng.standard_normal((2, 36, 48))
    for layer, full in ((0, False), (1, True)):
        got, A = Q.encoder_block(X, w, layer, SHAPE, want_scores=True)
        for f in range(2):
            ref = torch_block(t64(X[f]), w, f"l{layer}.", SHAPE, full).numpy()
            np.testing.assert_allclose(got[f], ref, atol=1e-10)
        np.testing.assert_allclose(A.sum(axis=1), 1.0, atol=1e-12)              # every query's probabilities sum to 1


def test_windows_isolate_tokens_and_full_layers_do_not():
    rng = np.random.default_rng(4)
    w = Q.split_weights(SHAPE, make_weights(SHAPE, 2).astype(np.float64))
    X = rng.standard_normal((1, 36, 48))
    Y = X.copy()
    Y[0, 0] += 1.0                                                              # a token of window 0
    ids = Q.window_ids(SHAPE)
    a, _ = Q.encoder_block(X, w, 0, SHAPE, False)
    b, _ = Q.encoder_block(Y, w, 0, SHAPE, False)
    assert np.array_equal(a[0][ids != 0], b[0][ids != 0]) and not np.allclose(a[0][ids == 0], b[0][ids == 0])
    a, _ = Q.encoder_block(X, w, 1, SHAPE, False)
    b, _ = Q.encoder_block(Y, w, 1, SHAPE, False)
    assert not np.allclose(a[0][ids == 3], b[0][ids == 3])


def test_whole_uncompressed_encoder_matches_torch_and_frames_pair_up():
    frames = make_video(6, 84, 14, 0.1, seed=5).astype(np.float64)
    blob = make_weights(SHAPE, 2).astype(np.float64)
    w = Q.split_weights(SHAPE, blob)
    p = MergeParams(merge_layers=(), selection=0, retain=1.0)
    res = O.encode_video(frames, SHAPE, blob, p, keep_features=True)
    assert res.features.shape == (3, 36, 48) and res.frames_per_block == [3, 3, 3]
    x = t64(Q.embed(frames, SHAPE, w))
    for f in range(3):
        y = x[f]
        for layer in range(3):
            y = torch_block(y, w, f"l{layer}.", SHAPE, layer in SHAPE.full_attn_layers)
        y = F.rms_norm(y, (48,), weight=t64(w["post_g"]), eps=SHAPE.ln_eps)
        np.testing.assert_allclose(res.features[f], y.numpy(), atol=1e-9)
    # the method on encoder frames: source ranges index temporal patches, Eq. 5 uses their count
    p = MergeParams(merge_layers=(1,), tau_seg=-2.0, tau_merge=-2.0, selection=1, retain_mode=1, retain=0.5)
    v = make_video(16, 84, 14, 0.05, seed=6).astype(np.float64)
    r = O.encode_video(v, SHAPE, blob, p)
    N = len(r.frame_dynamic)
    assert N < 8 and r.frame_src_hi[-1] == 7
    assert (r.k, r.w, r.M) == O.rescaled_keep(0.5, 8, N, 36, 1, p.window_mode)
