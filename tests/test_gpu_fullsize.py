"""Parity at the full benchmark sizes (32, 64 and 8 x 32 frames of SigLIP-so400m shapes), in the launch
configuration bench.py times.

`test_full_size_against_oracle` puts the whole compressed path through the comparison protocol of tests/helpers.py
against the oracle's results for the same seeded inputs: similarities, EMA, segments and merged pairs of every
merge layer, attention scores, kept sets (near-ties inside the measured band logged and counted), then tokens and
index map under identical decisions.  The numpy oracle needs 4 to 50 minutes per workload, so its results are read
from tests/golden/fullsize_<name>.npz, written on CPU by tests/golden/make_fullsize_goldens.py (which imports only
the oracle and the input generators); the test first checks the stored fingerprint of the oracle's inputs against
the generators.

`test_full_size_workload` adds what needs no stored values:

  * values: frames are independent in the uncompressed encoder, hence sampled frames of the full-size
    uncompressed run are compared with the oracle's encoding of those frames alone (<= 2e-2);
  * a frame that Stage I never merged goes through exactly the per-frame arithmetic of the
    uncompressed run, so its kept tokens must be bit-identical to that run's rows;
  * decisions: every decision the library took (segments, merged pairs, Eq. 5 amounts, kept sets) is
    re-derived by the oracle's own decision functions from the similarities / scores the library
    reports, and must be equal bit for bit;
  * structure: source ranges partition every video in order, positions ascend inside a frame, the
    ragged offsets match the kept counts, dynamic frames are the heads / tails of the last segmentation.
"""
import numpy as np
import pytest

from oracle import earlytom_oracle as O
from synthetic import make_batch, make_weights, workload
from tests import helpers as H

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2
BF16_SIM, BF16_SCORE = 5e-4, 1e-2     # hard ceilings on similarity / score error (see tests/test_gpu_encode.py)
NEAR_TIE_SHARE = 0.005
FULL_SIZE = ["so400m_32f", "so400m_32f_cal", "so400m_64f_p50", "so400m_64f_p10", "so400m_64f_p90", "serve_8x32", "qwenvl_768f"]


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2605_30010_b200 import binding
    return binding


def _np(t):
    return t.detach().cpu().numpy().copy()


def _snapshot(res):
    """Results live in encoder-owned memory until the next call: copy what the checks need."""
    return dict(tokens=_np(res.tokens), token_pos=_np(res.token_pos), frame_offsets=_np(res.frame_offsets),
                src_lo=_np(res.frame_src_lo), src_hi=_np(res.frame_src_hi), dynamic=_np(res.frame_dynamic).astype(bool),
                vfo=_np(res.video_frame_offsets), n_frames=res.n_frames_out, n_tokens=res.n_tokens,
                fpb=list(res.frames_per_block), trace=res.trace)


def _check_decisions(run, wl, offs):
    """Oracle decision functions on the library's reported similarities / scores -> identical decisions."""
    p, L = wl.params, wl.shape.tokens_per_frame
    tr = run["trace"]
    cur = np.asarray(offs, dtype=np.int64)
    last_starts = None
    for i in range(len(p.merge_layers)):
        assert tr.n_in[i] == cur[-1]
        new = [0]
        starts_all = []
        for v in range(len(cur) - 1):
            g0, g1 = int(cur[v]), int(cur[v + 1])
            c = tr.sim[i][g0:g1 - 1].astype(np.float64)
            st, _ = O.segment_by_similarity(c, g1 - g0, p.ema_alpha, p.tau_seg)
            mw = O.merge_pairs(c, O.segments_from_starts(st), p.tau_merge)
            np.testing.assert_array_equal(tr.seg_start[i][g0:g1].astype(bool), st, err_msg=f"layer {i} video {v} segments")
            np.testing.assert_array_equal(tr.merge_next[i][g0:g1].astype(bool), mw, err_msg=f"layer {i} video {v} pairs")
            new.append(new[-1] + (g1 - g0) - int(mw.sum()))
            starts_all.append((st, mw))
        assert tr.n_out[i] == new[-1]
        cur = np.asarray(new, dtype=np.int64)
        last_starts = starts_all
    np.testing.assert_array_equal(run["vfo"], cur)
    # dynamic flags: heads and tails of the last layer's segments, carried over the merge
    for v, (st, mw) in enumerate(last_starts):
        _, role = O.roles_of_segments(st)
        keep_frame = np.ones(len(st), dtype=bool)
        keep_frame[1:][mw[:-1]] = False                   # the second frame of a pair disappears
        role_out = np.where(mw, 1, role)[keep_frame]      # a merged pair is a middle frame
        np.testing.assert_array_equal(run["dynamic"][cur[v]:cur[v + 1]], role_out != 1)
    # Stage II amounts and kept sets
    for v in range(len(cur) - 1):
        f0, f1 = int(cur[v]), int(cur[v + 1])
        Bv = int(offs[v + 1] - offs[v])                  # encoder frames of the video
        k, w, M = O.rescaled_keep(p.retain, Bv, f1 - f0, L, p.retain_mode, p.window_mode)
        assert tr.video_k[v] == k and tr.video_w[v] == w
        keep = O.select_tokens(tr.scores[f0:f1].astype(np.float64), run["dynamic"][f0:f1], k, w, p.selection, p.window_mode)
        np.testing.assert_array_equal(tr.keep[f0:f1].astype(bool), keep, err_msg=f"video {v} kept set")
        np.testing.assert_allclose(tr.scores[f0:f1].sum(axis=1), 1.0, atol=2e-3)
    return cur


def _check_structure(run, offs, L):
    tr = run["trace"]
    vfo = run["vfo"]
    for v in range(len(vfo) - 1):
        lo, hi = run["src_lo"][vfo[v]:vfo[v + 1]], run["src_hi"][vfo[v]:vfo[v + 1]]
        assert lo[0] == 0 and hi[-1] == offs[v + 1] - offs[v] - 1
        assert (lo[1:] == hi[:-1] + 1).all() and (hi >= lo).all()
    counts = tr.keep.astype(bool).sum(axis=1)
    np.testing.assert_array_equal(np.diff(run["frame_offsets"]), counts)
    assert run["n_tokens"] == counts.sum() == len(run["token_pos"])
    for f in range(run["n_frames"]):
        pos = run["token_pos"][run["frame_offsets"][f]:run["frame_offsets"][f + 1]]
        np.testing.assert_array_equal(pos, np.nonzero(tr.keep[f])[0])


@pytest.mark.parametrize("name", FULL_SIZE)
def test_full_size_against_oracle(B, name):
    import os
    import torch
    wl = workload(name)
    assert os.path.exists(H.golden_path(name)), f"missing {H.golden_path(name)}: run tests/golden/make_fullsize_goldens.py {name}"
    ob = H.batch_from_golden(name, len(wl.params.merge_layers))
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed, wl.pos_std)
    assert H.input_sha(frames, blob) == ob.input_sha, "the stored oracle results were computed from other inputs"
    enc = B.Encoder(wl.shape, blob, B.ET_BF16, wl.total_frames, len(wl.videos))
    try:
        stats, log = H.check_parity(B, enc, torch.from_numpy(frames).cuda(), offs, wl.params, ob, BF16_TOL, BF16_SIM,
                                    BF16_SCORE, name)
    finally:
        enc.close()
    assert stats["near_ties"] <= max(1, NEAR_TIE_SHARE * stats["decisions"]), stats
    # the budget of Eq. 5: with k near-equal windows on static frames the kept total is N*k per video
    L = wl.shape.tokens_per_frame
    target = wl.params.retain * wl.encoder_frames * L
    assert abs(ob.n_tokens - target) <= len(ob.dynamic), (ob.n_tokens, target)


@pytest.mark.parametrize("name", FULL_SIZE)
def test_full_size_workload(B, name):
    import torch
    wl = workload(name)
    shape, L, tp = wl.shape, wl.shape.tokens_per_frame, wl.shape.temporal_patch
    frames, in_offs = make_batch(wl)
    offs = [int(o) // tp for o in in_offs]              # every index the library reports is in encoder frames
    blob = make_weights(shape, wl.weight_seed, wl.pos_std)
    enc = B.Encoder(shape, blob, B.ET_BF16, wl.total_frames, len(wl.videos))
    try:
        fr = torch.from_numpy(frames).cuda()
        unc = _snapshot(enc.encode_batch(fr, in_offs, wl.uncompressed().params))
        run = _snapshot(enc.encode_batch(fr, in_offs, wl.params, want_trace=True))
        again = _snapshot(enc.encode_batch(fr, in_offs, wl.params))
    finally:
        enc.close()
    assert unc["n_tokens"] == wl.encoder_frames * L
    assert np.array_equal(run["tokens"], again["tokens"]) and np.array_equal(run["token_pos"], again["token_pos"]), \
        "two runs of the same call must agree bit for bit"

    # values: sampled frames of the uncompressed run against the oracle on those frames alone
    w = O.split_weights(shape, blob)
    samples = [0, wl.encoder_frames - 1] if name in ("so400m_32f", "serve_8x32") else [wl.encoder_frames // 2]
    if name == "so400m_32f_cal":
        samples = [6]                       # the first scene cut
    if name == "qwenvl_768f":
        samples = [0, 24, 383]              # first frame, a scene cut, last frame
    for fidx in samples:
        ref = O.encode_video(frames[fidx * tp:(fidx + 1) * tp], shape, w, wl.uncompressed().params, dtype=np.float32)
        err = H.token_error(unc["tokens"][fidx * L:(fidx + 1) * L], ref.tokens)
        assert err <= BF16_TOL, f"{name} frame {fidx}: token error {err:.3e}"

    # decisions and structure
    _check_decisions(run, wl, offs)
    _check_structure(run, offs, L)
    expect_blocks, alive, m = [], wl.encoder_frames, 0
    for layer in range(shape.num_layers):
        if m < len(wl.params.merge_layers) and wl.params.merge_layers[m] == layer:
            alive = run["trace"].n_out[m]; m += 1
        expect_blocks.append(alive)
    assert run["fpb"] == expect_blocks

    # frames never merged: bit-identical to the uncompressed run's rows at the kept positions
    vfo, checked = run["vfo"], 0
    for v in range(len(vfo) - 1):
        for f in range(vfo[v], vfo[v + 1]):
            if run["src_lo"][f] != run["src_hi"][f]:
                continue
            orig = int(offs[v]) + int(run["src_lo"][f])
            a, b = run["frame_offsets"][f], run["frame_offsets"][f + 1]
            rows = orig * L + run["token_pos"][a:b]
            assert np.array_equal(run["tokens"][a:b], unc["tokens"][rows]), f"{name}: un-merged frame {f} differs"
            checked += 1
    assert checked > 0
    retained = run["n_tokens"] / (wl.encoder_frames * L)
    print(f"{name}: frames {wl.encoder_frames} -> {run['n_frames']}, tokens kept {retained:.3f}, un-merged frames checked {checked}")
