"""Pins of the oracle's Stage II (Eq. 4-7, Algorithm 2) and of the assembled path.  CPU only."""
import dataclasses
import itertools
import os

import numpy as np
import pytest

from oracle import earlytom_oracle as O
from synthetic import EncoderShape, MergeParams, make_video, make_weights
from tests.test_oracle_stage1 import golden, fl

SHAPE = EncoderShape(image_size=56, patch_size=14, num_layers=3, hidden=32, heads=2, mlp_dim=48)


def test_eq56_golden():
    for inp, exp in golden("eq56"):
        r, B, N, L = fl(inp)
        assert list(O.rescaled_keep(r, int(B), int(N), int(L), 1)) == [int(x) for x in exp.split()]


def test_eq5_restores_target_ratio():
    for B, N, L, r in itertools.product([8, 32, 64], [1, 5, 8, 24], [16, 64, 729], [0.1, 0.25, 0.5, 1.0]):
        if N > B:
            continue
        k, w, M = O.rescaled_keep(r, B, N, L, 1)
        assert 1 <= k <= L and w >= 1 and M == -(-L // w)
        if k < L:
            assert abs(N * k - r * B * L) < N + 1e-6       # N*k is the budget r*B*L up to rounding
        assert M >= k or w == 1                            # windows never keep fewer than k unless w = 1
        if N == B:
            assert k == max(1, int(np.floor(r * L + 1e-9)))
    assert O.rescaled_keep(0.5, 8, 8, 64, 0) == (32, 2, 32)
    assert O.rescaled_keep(1.0, 8, 4, 64, 1)[0] == 64      # clamp at L: identity selection


def test_topk_bruteforce_rank_count():
    rng = np.random.default_rng(0)
    for trial in range(200):
        L = int(rng.integers(1, 17))
        a = rng.integers(0, 6, L).astype(np.float64) / 7.0      # many exact ties
        k = int(rng.integers(1, L + 1))
        m = O.topk_mask(a, k)
        rank = [sum((a[i] > a[j]) or (a[i] == a[j] and i < j) for i in range(L)) for j in range(L)]
        assert m.tolist() == [r < k for r in rank]
        assert m.sum() == k
        if k < L:
            assert a[m].min() >= a[~m].max()


def test_window_bruteforce():
    rng = np.random.default_rng(1)
    for trial in range(200):
        L = int(rng.integers(1, 17))
        w = int(rng.integers(1, L + 1))
        a = rng.integers(0, 4, L).astype(np.float64)
        m = O.window_mask(a, w)
        assert m.sum() == -(-L // w)
        for lo in range(0, L, w):
            win = a[lo:lo + w]
            assert m[lo:lo + w].sum() == 1
            assert np.nonzero(m[lo:lo + w])[0][0] == int(np.argmax(win))   # first maximum


def test_balanced_windows_closed_form_and_budget():
    """window_mode 1: k windows [floor(m L / k), floor((m+1) L / k)).  Pinned by the closed form of the window
    a position falls into, m(j) = ceil((j+1) k / L) - 1, which never uses the edges; by the widths; by equality
    with Eq. 6 as printed whenever k divides L; and by the kept total N*k against the budget r*B*L."""
    rng = np.random.default_rng(11)
    for trial in range(300):
        L = int(rng.integers(1, 40))
        k = int(rng.integers(1, L + 1))
        w = L // k
        e = O.window_edges(L, k, w, 1)
        assert e[0] == 0 and e[-1] == L and len(e) == k + 1
        widths = np.diff(e)
        assert widths.min() >= 1 and set(widths.tolist()) <= {w, w + 1}
        a = rng.integers(0, 4, L).astype(np.float64)
        m = O.window_mask(a, w, k, 1)
        assert m.sum() == k
        win_of = [-(-((j + 1) * k) // L) - 1 for j in range(L)]
        for mm in range(k):
            members = [j for j in range(L) if win_of[j] == mm]
            best = max(members, key=lambda j: (a[j], -j))                   # first maximum
            assert m[members].sum() == 1 and m[best]
        if L % k == 0:
            assert e == O.window_edges(L, k, w, 0)
            np.testing.assert_array_equal(m, O.window_mask(a, w))
    # the budget: static and dynamic frames both keep k, so the total is N*k, within N of r*B*L
    for B, N, L, r in [(32, 13, 729, 0.25), (32, 24, 729, 0.25), (32, 12, 729, 0.10), (64, 40, 729, 0.25)]:
        k, w, M = O.rescaled_keep(r, B, N, L, 1, window_mode=1)
        assert M == k and abs(N * k - r * B * L) < N
    # Eq. 6 as printed misses it as soon as k > L/2: every static frame keeps all L tokens
    k, w, M = O.rescaled_keep(0.25, 32, 13, 729, 1, window_mode=0)
    assert (k, w, M) == (448, 1, 729)
    assert O.rescaled_keep(0.25, 32, 13, 729, 1, window_mode=1) == (448, 1, 448)


def test_selection_counts_and_roles():
    rng = np.random.default_rng(2)
    A = rng.random((5, 16))
    dyn = np.array([1, 0, 0, 1, 1], dtype=bool)
    keep = O.select_tokens(A, dyn, 4, 4, 1)
    assert keep.sum(axis=1).tolist() == [4, 4, 4, 4, 4]
    keep = O.select_tokens(A, dyn, 5, 3, 1)          # w = 16 // 5 = 3 -> M = 6 windows on static frames
    assert keep.sum(axis=1).tolist() == [5, 6, 6, 5, 5]
    assert O.select_tokens(A, dyn, 5, 3, 1, window_mode=1).sum(axis=1).tolist() == [5] * 5
    assert O.select_tokens(A, dyn, 5, 3, 2).sum(axis=1).tolist() == [5] * 5
    assert O.select_tokens(A, dyn, 5, 3, 0).all()


def _run(frames, blob, **kw):
    p = MergeParams(**{**dict(merge_layers=(1,), tau_seg=0.8, tau_merge=0.8, selection=1, retain_mode=1, retain=0.5), **kw})
    return O.encode_video(frames, SHAPE, blob, p, keep_features=True), p


def test_disabled_compression_equals_plain_encoder():
    frames = make_video(6, 56, 14, 0.2, seed=3)
    blob = make_weights(SHAPE, 5)
    plain = O.encode_video(frames, SHAPE, blob, MergeParams(merge_layers=(), selection=0, retain=1.0), keep_features=True)
    for kw in (dict(tau_seg=1.5), dict(tau_merge=2.0)):
        r, _ = _run(frames, blob, retain=1.0, **kw)
        assert len(r.frame_dynamic) == 6
        np.testing.assert_array_equal(r.features, plain.features)
        np.testing.assert_array_equal(r.tokens, plain.tokens)        # rho = 1 -> k = L -> identity
    # tau_seg > 1: all frames are 1-frame segments -> all dynamic
    r, _ = _run(frames, blob, tau_seg=1.5)
    assert r.frame_dynamic.all()


def test_end_to_end_bookkeeping():
    frames = make_video(10, 56, 14, 0.1, seed=4)
    blob = make_weights(SHAPE, 5)
    r, p = _run(frames, blob, tau_seg=0.2, tau_merge=0.2, merge_layers=(1, 2))
    N = len(r.frame_dynamic)
    B, L = 10, SHAPE.tokens_per_frame
    assert N < B, "workload must actually merge"
    assert N == B - sum(int(t.merge_with_next.sum()) for t in r.merge_trace)
    assert r.frames_per_block == [10, r.merge_trace[0].n_out, r.merge_trace[1].n_out]
    # Eq. 7: frames in temporal order, positions ascending inside a frame
    for f in range(N):
        pos = r.token_pos[r.frame_offsets[f]:r.frame_offsets[f + 1]]
        assert (np.diff(pos) > 0).all()
        np.testing.assert_array_equal(r.tokens[r.frame_offsets[f]:r.frame_offsets[f + 1]], r.features[f][pos])
    # dynamic = head/tail of the segments of the last merge layer
    T = int(r.frame_dynamic.sum())
    assert r.tokens.shape[0] == T * r.k + (N - T) * r.M
    assert (r.k, r.w, r.M) == O.rescaled_keep(p.retain, B, N, L, 1, p.window_mode)
    assert r.frame_src_lo[0] == 0 and r.frame_src_hi[-1] == B - 1
    assert (r.frame_src_hi[:-1] + 1 == r.frame_src_lo[1:]).all()


def test_decisions_invariant_to_hidden_permutation_of_merge_input():
    """Permuting the feature axis of all frames changes no Stage-I decision and permutes the output."""
    rng = np.random.default_rng(3)
    base = rng.standard_normal((5, 12))
    F = np.stack([base + 0.3 * t * rng.standard_normal((5, 12)) for t in range(8)])
    perm = rng.permutation(12)
    meta = [O.FrameMeta(t, t) for t in range(8)]
    a, _, ta = O.stage1_one_video(F, meta, 0.9, 0.3, 0.3, True, 0)
    b, _, tb = O.stage1_one_video(F[:, :, perm], meta, 0.9, 0.3, 0.3, True, 0)
    assert (ta.merge_with_next == tb.merge_with_next).all() and (ta.starts == tb.starts).all()
    np.testing.assert_allclose(a[:, :, perm], b, atol=1e-12)


def test_forced_replay_reproduces_free_run():
    frames = make_video(9, 56, 14, 0.15, seed=6)
    blob = make_weights(SHAPE, 5)
    r, p = _run(frames, blob, tau_seg=0.3, tau_merge=0.3)
    forced = {"merge": {t.layer: (t.starts, t.merge_with_next) for t in r.merge_trace}, "keep": r.keep}
    r2 = O.encode_video(frames, SHAPE, blob, p, forced=forced)
    np.testing.assert_array_equal(r.tokens, r2.tokens)
    np.testing.assert_array_equal(r.frame_dynamic, r2.frame_dynamic)


def test_batch_is_independent_videos():
    blob = make_weights(SHAPE, 5)
    v0 = make_video(5, 56, 14, 0.2, seed=1)
    v1 = make_video(7, 56, 14, 0.4, seed=2)
    p = MergeParams(merge_layers=(1,), tau_seg=0.3, tau_merge=0.3, retain=0.5)
    rs = O.encode_batch(np.concatenate([v0, v1]), [0, 5, 12], SHAPE, blob, p)
    np.testing.assert_array_equal(rs[1].tokens, O.encode_video(v1, SHAPE, blob, p).tokens)
    np.testing.assert_array_equal(rs[0].tokens, O.encode_video(v0, SHAPE, blob, p).tokens)


def test_main_setting_matches_paper_table():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_hyperparameters.txt")
    kv = {}
    for line in open(path):
        if line.startswith("#") or "=" not in line:
            continue
        k, v = line.split(";")[0].split("=")
        kv[k.strip()] = v.strip()
    from synthetic import WORKLOADS
    p = WORKLOADS["so400m_32f"].params
    assert p.ema_alpha == float(kv["ema_alpha"]) and p.tau_seg == float(kv["tau_seg_mvbench_25"])
    assert list(p.merge_layers) == [int(x) for x in kv["merge_layers_mvbench_25"].split(",")]
    assert WORKLOADS["so400m_32f"].total_frames == int(kv["frames_per_video"])
    assert p.retain in [float(x) for x in kv["retain_ratios"].split(",")]


# ------------------------------------------------------------------ random-sampling ablation (selection 3)

def test_philox_known_answers():
    """The counter-based generator behind the random-sampling baseline, against the published vectors."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        out = O.philox4x32_10(np.array(w[0:4], dtype=np.uint32), (w[4], w[5]))
        assert [int(x) for x in out] == w[6:10]


def test_random_scores_are_uniform_and_counter_based():
    a = O.random_scores(seed=7, video=2, n_frames=5, L=729)
    assert a.shape == (5, 729) and a.min() >= 0.0 and a.max() < 1.0
    assert abs(a.mean() - 0.5) < 0.02 and abs(a.var() - 1 / 12) < 0.01
    # a token's number depends only on (seed, video, frame, position)
    b = O.random_scores(seed=7, video=2, n_frames=3, L=100)
    np.testing.assert_array_equal(a[:3, :100], b)
    assert not np.array_equal(a, O.random_scores(seed=8, video=2, n_frames=5, L=729))
    assert not np.array_equal(a, O.random_scores(seed=7, video=3, n_frames=5, L=729))


def test_random_sampling_keeps_k_per_frame():
    a = O.random_scores(seed=1, video=0, n_frames=6, L=64)
    keep = O.select_tokens(a, np.zeros(6, dtype=bool), 16, 4, 2)
    assert (keep.sum(axis=1) == 16).all()
    # every position is kept about k/L of the time over many frames
    big = O.select_tokens(O.random_scores(3, 0, 400, 32), np.zeros(400, dtype=bool), 8, 4, 2)
    freq = big.mean(axis=0)
    assert np.abs(freq - 0.25).max() < 0.1
