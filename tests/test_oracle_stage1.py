"""Pins of the oracle's Stage I (frame similarity, Eq. 1-3, Algorithm 1).  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import earlytom_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden(name):
    out = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = [p.strip() for p in line.split("|")]
        if parts[0] == name:
            out.append(parts[1:])
    assert out, name
    return out


def fl(s):
    return [float(x) for x in s.split()]


# ---------------------------------------------------------------- similarity

def test_similarity_closed_forms():
    rng = np.random.default_rng(0)
    a = rng.standard_normal((5, 8))
    F = np.stack([a, 3.0 * a, -a, a])            # scaled copy -> 1, negated -> -1, back -> -1
    np.testing.assert_allclose(O.frame_similarity(F), [1.0, -1.0, -1.0], atol=1e-12)
    e = np.eye(4)[None].repeat(2, 0)             # tokens = unit vectors
    e[1] = np.roll(e[1], 1, axis=-1)             # orthogonal at every position
    np.testing.assert_allclose(O.frame_similarity(e), [0.0], atol=1e-12)
    # 45 degrees at half of the positions, identical at the others: mean of cos
    F = np.zeros((2, 4, 2)); F[:, :, 0] = 1.0; F[1, :2, 1] = 1.0
    np.testing.assert_allclose(O.frame_similarity(F), [(2 * np.sqrt(0.5) + 2) / 4], atol=1e-12)


def test_similarity_zero_token_contributes_zero():
    F = np.ones((2, 4, 3)); F[0, 1] = 0.0
    np.testing.assert_allclose(O.frame_similarity(F), [0.75], atol=1e-12)


def test_similarity_is_per_position_not_per_frame_vector():
    """A dropped mean-over-positions (cosine of the flattened frames) would give another value."""
    F = np.zeros((2, 2, 2))
    F[0, 0] = [10, 0]; F[1, 0] = [10, 0]      # big identical token
    F[0, 1] = [1, 0];  F[1, 1] = [0, 1]       # small orthogonal token
    np.testing.assert_allclose(O.frame_similarity(F), [0.5], atol=1e-12)


def test_similarity_invariant_to_feature_permutation():
    rng = np.random.default_rng(1)
    F = rng.standard_normal((6, 7, 16))
    perm = rng.permutation(16)
    np.testing.assert_allclose(O.frame_similarity(F), O.frame_similarity(F[:, :, perm]), atol=1e-13)


# ---------------------------------------------------------------- Eq. 1

def test_eq1_golden():
    (inp, exp), = golden("eq1_ema")
    alpha, sims = inp.split(";")
    _, ema = O.segment_by_similarity(fl(sims), len(fl(sims)) + 1, float(alpha), -2.0)
    np.testing.assert_allclose(ema[1:], fl(exp), atol=1e-12)
    for name in ("eq1_nobreak", "eq1_break"):
        (inp, exp), = golden(name)
        head, sims = inp.split(";")
        alpha, tau = fl(head)
        starts, _ = O.segment_by_similarity(fl(sims), len(fl(sims)) + 1, alpha, tau)
        assert starts.astype(int).tolist() == [int(x) for x in exp.split()]


def test_eq1_alpha_one_is_plain_thresholding_exhaustive():
    """With alpha = 1 the EMA is the raw similarity: frame t opens a segment iff c[t-1] < tau.
    All 2^(n-1) low/high patterns for n <= 8."""
    for n in range(1, 9):
        for bits in itertools.product([0, 1], repeat=n - 1):
            c = [0.9 if b else 0.1 for b in bits]
            starts, _ = O.segment_by_similarity(c, n, 1.0, 0.5)
            assert starts.tolist() == [True] + [not b for b in bits]


def test_eq1_extreme_thresholds():
    c = np.random.default_rng(0).uniform(-1, 1, 9)
    s, _ = O.segment_by_similarity(c, 10, 0.9, -1.5)
    assert s.tolist() == [True] + [False] * 9
    s, _ = O.segment_by_similarity(c, 10, 0.9, 1.5)
    assert s.all()


def test_eq1_ema_resets_after_break_bruteforce():
    """Independent restatement: within a segment the EMA is the explicit weighted sum
    alpha * sum_j (1-alpha)^j s_{t-j} + (1-alpha)^(t-t0) * s_{t0} (first similarity of the segment)."""
    rng = np.random.default_rng(3)
    for trial in range(200):
        n = int(rng.integers(2, 9))
        c = rng.uniform(0.3, 1.0, n - 1)
        alpha, tau = float(rng.uniform(0.1, 1.0)), float(rng.uniform(0.4, 0.9))
        starts, ema = O.segment_by_similarity(c, n, alpha, tau)
        first = None      # index t of the first similarity folded into the running segment
        for t in range(1, n):
            if first is None:
                first = t
            m = t - first
            val = (1 - alpha) ** m * c[first - 1] + sum(alpha * (1 - alpha) ** j * c[t - 1 - j] for j in range(m))
            assert abs(val - ema[t]) < 1e-12
            assert starts[t] == (val < tau)
            if val < tau:
                first = None


# ---------------------------------------------------------------- Eq. 2

def merged_recursive(c, g, tau):
    """Restatement of the rule as a recursion over the local index (no loop state):
    pair starts at i  <=>  no pair started at i-1, both frames are middle frames, and Eq. 2 holds."""
    k = len(g) - 1
    m = {}
    for i in range(0, k + 1):
        m[i] = (i >= 1 and not m.get(i - 1, False) and i <= k - 2
                and c[g[i]] > tau and c[g[i]] > c[g[i + 1]])
    return [g[i] for i in range(k + 1) if m[i]]


def test_eq2_golden():
    for inp, exp in golden("eq2_pairs"):
        tau, sims = inp.split(";")
        sims = fl(sims)
        n = len(sims) + 1
        mw = O.merge_pairs(sims, [list(range(n))], float(tau))
        assert mw.astype(int).tolist() == [int(x) for x in exp.split()]


def test_eq2_matches_recursion_and_invariants_random():
    rng = np.random.default_rng(7)
    for trial in range(500):
        n = int(rng.integers(1, 12))
        c = rng.uniform(0, 1, max(n - 1, 0))
        starts = rng.random(n) < 0.3
        starts[0] = True
        segs = O.segments_from_starts(starts)
        tau = float(rng.uniform(0, 1))
        mw = O.merge_pairs(c, segs, tau)
        exp = np.zeros(n, dtype=bool)
        for g in segs:
            exp[merged_recursive(c, g, tau)] = True
        assert (mw == exp).all()
        for g in segs:
            # head and tail are never part of a pair; segments of <= 3 frames never merge
            assert not mw[g[0]] and not mw[g[-1]]
            if len(g) >= 2:
                assert not mw[g[-2]]
            if len(g) <= 3:
                assert not mw[g].any()
        assert not (mw[:-1] & mw[1:]).any()      # pairs do not overlap


def test_eq2_monotone_cases():
    n = 9
    dec = np.linspace(0.95, 0.55, n - 1)
    mw = O.merge_pairs(dec, [list(range(n))], 0.5)
    assert np.nonzero(mw)[0].tolist() == [1, 3, 5]        # (1,2) (3,4) (5,6); frame 7 is the last middle
    mw = O.merge_pairs(dec, [list(range(n))], 0.75)
    assert np.nonzero(mw)[0].tolist() == [1, 3]           # c[3] = 0.779 passes, c[5] = 0.664 fails the threshold
    inc = dec[::-1]
    assert not O.merge_pairs(inc, [list(range(n))], 0.0).any()
    eq = np.full(n - 1, 0.9)
    assert not O.merge_pairs(eq, [list(range(n))], 0.0).any()   # strict '>' : equal neighbours do not merge


# ---------------------------------------------------------------- Eq. 3 and the assembled step

def test_eq3_golden_weights():
    (inp, exp), = golden("eq3_weights")
    sa, sb = fl(inp)
    a, b = np.full((2, 3), 1.0), np.full((2, 3), 2.0)
    m, wa, wb = O.weighted_merge(a, b, sa, sb, True)
    np.testing.assert_allclose([wa, wb], fl(exp), atol=1e-12)
    np.testing.assert_allclose(m, 1.4, atol=1e-12)
    m, wa, wb = O.weighted_merge(a, b, sa, sb, False)
    np.testing.assert_allclose(m, 1.5, atol=1e-12)
    m, wa, wb = O.weighted_merge(a, b, 1e-9, -1e-9, True)      # guarded denominator -> mean
    np.testing.assert_allclose(m, 1.5, atol=1e-12)


def _rotated_frames(angles, L=6, D=8, seed=0):
    """Frames whose token at every position is r_l * (cos(theta_t) e1 + sin(theta_t) e2) for a fixed orthonormal
    pair (e1, e2) and positive per-position lengths r_l (differing between frames): the cosine of every position of
    frames t, t+1 is cos(theta_{t+1} - theta_t), hence so is their similarity -- known without running any code."""
    rng = np.random.default_rng(seed)
    q, _ = np.linalg.qr(rng.standard_normal((D, 2)))
    e1, e2 = q[:, 0], q[:, 1]
    frames = []
    for th in angles:
        r = rng.uniform(0.5, 2.0, size=(L, 1))
        frames.append(r * (np.cos(th) * e1 + np.sin(th) * e2)[None, :])
    return np.stack(frames)


def test_assembled_step_uses_similarity_to_the_following_frame_as_eq3_weights():
    """One segment [H, X, Y, Z, T] with similarities c = cos(.3), cos(.2), cos(.5), cos(.1).  Eq. 2 picks the pair
    (X, Y) (c_1 > tau and c_1 > c_2); Eq. 3 then weights X by c_1 = Sim(X, Y) and Y by c_2 = Sim(Y, Z): each frame by
    its similarity with the frame after it.  A step that took (c_0, c_1) or (c_1, c_3) instead gives other weights."""
    import math
    th = np.cumsum([0.0, 0.3, 0.2, 0.5, 0.1])
    F = _rotated_frames(th)
    c = [math.cos(0.3), math.cos(0.2), math.cos(0.5), math.cos(0.1)]
    wa, wb = c[1] / (c[1] + c[2]), c[2] / (c[1] + c[2])
    expect = wa * F[1] + wb * F[2]
    meta = [O.FrameMeta(t, t) for t in range(5)]
    for run in ("free", "forced"):
        if run == "free":
            Fo, mo, tr = O.stage1_one_video(F, meta, 0.9, -2.0, 0.5, True, 0)
        else:
            decision = (np.array([1, 0, 0, 0, 0], bool), np.array([0, 1, 0, 0, 0], bool))
            Fo, mo, tr = O._stage1_forced(F, meta, decision, True, 0)
        np.testing.assert_allclose(tr.c, c, atol=1e-12)
        assert np.nonzero(tr.merge_with_next)[0].tolist() == [1] and tr.n_out == 4
        np.testing.assert_allclose(tr.w_a, [1.0, wa, 1.0, 1.0], atol=1e-12)
        np.testing.assert_allclose(tr.w_b, [0.0, wb, 0.0, 0.0], atol=1e-12)
        assert tr.src_a.tolist() == [0, 1, 3, 4] and tr.src_b.tolist() == [-1, 2, -1, -1]
        np.testing.assert_allclose(Fo[1], expect, atol=1e-12)
        np.testing.assert_array_equal(Fo[[0, 2, 3]], F[[0, 3, 4]])
        # the plausible wrong choices are far outside the tolerance
        for sa, sb in ((c[0], c[1]), (c[1], c[3]), (c[2], c[1])):
            wrong = (sa * F[1] + sb * F[2]) / (sa + sb)
            assert np.abs(wrong - expect).max() > 1e-3
    # unweighted variant: plain mean, whatever the similarities
    Fo, _, tr = O.stage1_one_video(F, meta, 0.9, -2.0, 0.5, False, 0)
    np.testing.assert_allclose(Fo[1], 0.5 * (F[1] + F[2]), atol=1e-12)
    np.testing.assert_allclose(tr.w_a[1], 0.5)


def test_assembled_step_two_pairs_and_later_layer():
    """Seven frames, decreasing similarities inside one segment: pairs (1,2) and (3,4) merge, each with its own two
    similarities; a second pass over the merged list (the way several merge layers compose) uses the similarities of
    the merged list, again known in closed form because a merged frame stays in the (e1, e2) plane."""
    import math
    d = [0.10, 0.15, 0.20, 0.25, 0.30, 0.05]
    th = np.cumsum([0.0] + d)
    F = _rotated_frames(th, seed=3)
    c = [math.cos(x) for x in d]
    Fo, mo, tr = O.stage1_one_video(F, [O.FrameMeta(t, t) for t in range(7)], 0.9, -2.0, 0.5, True, 0)
    assert np.nonzero(tr.merge_with_next)[0].tolist() == [1, 3]
    np.testing.assert_allclose(Fo[1], (c[1] * F[1] + c[2] * F[2]) / (c[1] + c[2]), atol=1e-12)
    np.testing.assert_allclose(Fo[2], (c[3] * F[3] + c[4] * F[4]) / (c[3] + c[4]), atol=1e-12)
    assert [(m.src_lo, m.src_hi) for m in mo] == [(0, 0), (1, 2), (3, 4), (5, 5), (6, 6)]


def test_identical_middle_pair_collapses():
    """[H, X, X, Y, T] in one segment: the two X have similarity 1 > the next similarity, so they
    merge into one frame equal to X; every other frame is copied."""
    rng = np.random.default_rng(0)
    H, X, Y, T = (rng.standard_normal((6, 8)) for _ in range(4))
    F = np.stack([H, X, X, Y, T])
    meta = [O.FrameMeta(t, t) for t in range(5)]
    Fo, mo, tr = O.stage1_one_video(F, meta, 0.9, -2.0, 0.5, True, 0)
    assert tr.n_out == 4 and np.nonzero(tr.merge_with_next)[0].tolist() == [1]
    np.testing.assert_allclose(Fo[1], X, atol=1e-12)
    np.testing.assert_array_equal(Fo[[0, 2, 3]], F[[0, 3, 4]])
    assert [(m.src_lo, m.src_hi) for m in mo] == [(0, 0), (1, 2), (3, 3), (4, 4)]
    assert [m.role for m in mo] == [0, 1, 1, 2]


def test_all_identical_frames_do_not_merge():
    """Consequence of the strict inequality in Eq. 2: a run of bit-identical frames has equal
    similarities everywhere, so no pair is 'more similar than the next pair'."""
    X = np.random.default_rng(0).standard_normal((4, 8))
    F = np.stack([X] * 6)
    Fo, mo, tr = O.stage1_one_video(F, [O.FrameMeta(t, t) for t in range(6)], 0.9, 0.8, 0.5, True, 0)
    assert tr.n_out == 6


def test_merged_frame_lies_between_its_sources():
    rng = np.random.default_rng(5)
    a, b = rng.standard_normal((2, 5, 7))
    m, wa, wb = O.weighted_merge(a, b, 0.7, 0.4, True)
    assert ((m >= np.minimum(a, b) - 1e-12) & (m <= np.maximum(a, b) + 1e-12)).all()
    assert abs(wa + wb - 1) < 1e-12 and wa > wb


def test_stage1_partition_invariants_random():
    rng = np.random.default_rng(11)
    for trial in range(100):
        n = int(rng.integers(1, 14))
        base = rng.standard_normal((3, 6))
        F = np.stack([base + rng.uniform(0, 1.5) * rng.standard_normal((3, 6)) for _ in range(n)])
        meta = [O.FrameMeta(t, t) for t in range(n)]
        for layer in range(2):       # two merge layers composed
            F, meta, tr = O.stage1_one_video(F, meta, 0.9, float(rng.uniform(0, 0.8)), float(rng.uniform(0, 0.8)), True, layer)
            assert tr.n_out == tr.n_in - int(tr.merge_with_next.sum()) == F.shape[0]
        lo = [m.src_lo for m in meta]; hi = [m.src_hi for m in meta]
        assert lo[0] == 0 and hi[-1] == n - 1
        assert all(hi[i] + 1 == lo[i + 1] for i in range(len(meta) - 1))
        assert all(l <= h for l, h in zip(lo, hi))


def test_merging_disabled_by_thresholds():
    rng = np.random.default_rng(2)
    F = rng.standard_normal((7, 4, 8))
    meta = [O.FrameMeta(t, t) for t in range(7)]
    Fo, _, tr = O.stage1_one_video(F, meta, 0.9, 1.5, 0.0, True, 0)       # every frame its own segment
    assert tr.n_out == 7 and np.array_equal(Fo, F)
    Fo, _, tr = O.stage1_one_video(F, meta, 0.9, -2.0, 2.0, True, 0)      # nothing passes tau_merge
    assert tr.n_out == 7 and np.array_equal(Fo, F)
