"""Pins of the oracle's encoder forward against independent library compositions (CPU only)."""
import dataclasses

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import earlytom_oracle as O
from synthetic import EncoderShape, MergeParams, make_video, make_weights
from synthetic.weights import views

SHAPE = EncoderShape(image_size=62, patch_size=14, num_layers=3, hidden=48, heads=4, mlp_dim=80)
OFF = MergeParams(merge_layers=(), selection=0, retain=1.0)


def torch_encoder(frames, shape, w, tanh=True):
    """The same architecture written with torch's own ops: conv2d, layer_norm, linear,
    scaled_dot_product_attention, gelu.  float64.  Returns (features [T,L,D], last-block probs)."""
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).double()
    D, p = shape.hidden, shape.patch_size
    x = t(frames)
    conv_w = t(w["patch_w"]).T.reshape(D, 3, p, p)           # [D, c, dy, dx]
    x = F.conv2d(x, conv_w, t(w["patch_b"]), stride=p)       # valid conv: crops the ragged border
    T = x.shape[0]
    x = x.flatten(2).transpose(1, 2) + t(w["pos"])[None]
    probs = None
    for i in range(shape.num_layers):
        g = lambda n: t(w[f"l{i}.{n}"])
        h = F.layer_norm(x, (D,), g("ln1_g"), g("ln1_b"), shape.ln_eps)
        qkv = F.linear(h, g("wqkv").T, g("bqkv"))
        q, k, v = [z.reshape(T, -1, shape.heads, shape.head_dim).transpose(1, 2) for z in qkv.chunk(3, dim=-1)]
        a = F.scaled_dot_product_attention(q, k, v)
        if i == shape.num_layers - 1:
            probs = torch.softmax(q @ k.transpose(-1, -2) / shape.head_dim ** 0.5, dim=-1)
        a = a.transpose(1, 2).reshape(T, -1, D)
        x = x + F.linear(a, g("wo").T, g("bo"))
        h = F.layer_norm(x, (D,), g("ln2_g"), g("ln2_b"), shape.ln_eps)
        h = F.gelu(F.linear(h, g("w1").T, g("b1")), approximate="tanh" if tanh else "none")
        x = x + F.linear(h, g("w2").T, g("b2"))
    x = F.layer_norm(x, (D,), t(w["post_g"]), t(w["post_b"]), shape.ln_eps)
    return x.numpy(), probs.numpy()


@pytest.mark.parametrize("tanh", [1, 0])
def test_uncompressed_encoder_equals_torch_composition(tanh):
    shape = dataclasses.replace(SHAPE, gelu_tanh=tanh)
    frames = make_video(3, shape.image_size, shape.patch_size, 0.3, seed=5)
    blob = make_weights(shape, 11)
    w = views(shape, blob)
    ref, probs = torch_encoder(frames, shape, w, tanh=bool(tanh))
    r = O.encode_video(frames, shape, blob, OFF, keep_features=True)
    assert r.features.shape == ref.shape == (3, 16, 48)
    np.testing.assert_allclose(r.features, ref, rtol=0, atol=1e-10)
    # with nothing compressed the token list is the feature map itself, in order
    np.testing.assert_array_equal(r.tokens.reshape(ref.shape), r.features)
    np.testing.assert_array_equal(r.token_pos, np.tile(np.arange(16), 3))
    # per-token attention score = mean over heads and queries of the attention each key receives
    a_ref = probs.mean(axis=(1, 2))
    np.testing.assert_allclose(r.scores, a_ref, rtol=0, atol=1e-12)


def test_patchify_is_a_strided_valid_convolution():
    rng = np.random.default_rng(0)
    fr = rng.standard_normal((2, 3, 31, 31))
    wgt = rng.standard_normal((3 * 49, 5))
    mine = O.patchify(fr, 7) @ wgt
    ref = F.conv2d(torch.from_numpy(fr), torch.from_numpy(wgt).T.reshape(5, 3, 7, 7).contiguous(), stride=7)
    np.testing.assert_allclose(mine, ref.flatten(2).transpose(1, 2).numpy(), atol=1e-12)


def test_attention_scores_sum_to_one_and_uniform_case():
    shape = SHAPE
    frames = make_video(2, shape.image_size, shape.patch_size, 0.5, seed=1)
    blob = make_weights(shape, 3)
    r = O.encode_video(frames, shape, blob, OFF)
    np.testing.assert_allclose(r.scores.sum(axis=1), 1.0, atol=1e-12)
    # zero query projection and bias in the last block -> all logits equal -> uniform attention
    w = views(shape, blob)
    D = shape.hidden
    w[f"l{shape.num_layers - 1}.wqkv"][:, :D] = 0
    w[f"l{shape.num_layers - 1}.bqkv"][:D] = 0
    r = O.encode_video(frames, shape, blob, OFF)
    np.testing.assert_allclose(r.scores, 1.0 / shape.tokens_per_frame, atol=1e-14)


def test_fp32_variant_tracks_fp64():
    frames = make_video(2, SHAPE.image_size, SHAPE.patch_size, 0.3, seed=2)
    blob = make_weights(SHAPE, 4)
    a = O.encode_video(frames, SHAPE, blob, OFF, keep_features=True).features
    b = O.encode_video(frames, SHAPE, blob, OFF, keep_features=True, dtype=np.float32).features
    assert b.dtype == np.float32
    assert np.abs(a - b).max() / np.abs(a).max() < 1e-5


def test_frames_are_independent_inside_the_encoder():
    """Attention is per frame: encoding a frame alone gives the same features as inside a video."""
    frames = make_video(3, SHAPE.image_size, SHAPE.patch_size, 0.6, seed=9)
    blob = make_weights(SHAPE, 4)
    full = O.encode_video(frames, SHAPE, blob, OFF, keep_features=True).features
    one = O.encode_video(frames[1:2], SHAPE, blob, OFF, keep_features=True).features
    np.testing.assert_allclose(full[1], one[0], atol=1e-12)


def test_eq8_cost_model():
    # 4 L D^2 + 2 L^2 D + 2 L D M per frame-block, worked by hand for L=2, D=3, M=5: 72 + 24 + 60 = 156
    assert O.eq8_macs(2, [1], 3, 5) == 156
    assert O.eq8_macs(2, [3, 2], 3, 5) == 156 * 5
    # SigLIP-so400m shapes, one frame, one block (the three terms printed in Eq. 8)
    L, D, M = 729, 1152, 4304
    assert O.eq8_macs(L, [1], D, M) == 4 * L * D * D + 2 * L * L * D + 2 * L * D * M


def test_weight_blob_layout_matches_generator():
    blob = make_weights(SHAPE, 1)
    a = O.split_weights(SHAPE, blob)
    b = views(SHAPE, blob)
    assert list(a.keys()) == list(b.keys())
    for k in a:
        assert a[k].shape == b[k].shape and a[k].__array_interface__["data"][0] == b[k].__array_interface__["data"][0]
    with pytest.raises(ValueError):
        O.split_weights(SHAPE, blob[:-1])
