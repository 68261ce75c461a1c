"""The comparison protocol of the GPU parity tests: the oracle's results (computed in the test, or read from a
tests/golden/fullsize_*.npz file that tests/golden/make_fullsize_goldens.py wrote with the oracle alone) on one
side, the C-ABI library on the other.

One flipped decision changes every later value, so the protocol is:
  1. run the library free and compare the decision trace layer by layer.  Similarities must agree within a hard
     ceiling.  A decision that differs is accepted as a near-tie only if the oracle's margin lies inside the band
     1e-3 (absolute for similarities, relative for scores) widened by the numeric error MEASURED in this run on the
     quantity that decides (twice that error where two quantities are compared); it is logged.  Anything else fails;
  2. after a near-tie the library is re-run with the oracle's decisions forced, and the comparison continues;
  3. values (tokens, index map) are always compared under identical decisions.
The function returns the counts and errors so that callers can assert ceilings and report them.
"""
from __future__ import annotations

import hashlib
import json
import os
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

SIM_TIE = 1e-3       # absolute near-tie margin for similarity decisions (similarities lie in [-1, 1])
SCORE_TIE = 1e-3     # relative near-tie margin for attention scores (they are O(1/L))
GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def token_error(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max over tokens of ||g - o||_inf / ||o||_inf."""
    if ref.shape[0] == 0:
        return 0.0
    num = np.abs(gpu.astype(np.float64) - ref.astype(np.float64)).max(axis=1)
    den = np.abs(ref.astype(np.float64)).max(axis=1)
    return float((num / np.maximum(den, 1e-30)).max())


@dataclass
class OracleBatch:
    """Oracle results of all videos of one call, concatenated in call order."""
    sim: List[np.ndarray]            # per merge layer [n_in], 0 at the last frame of a video
    ema: List[np.ndarray]            # per merge layer [n_in], 0 at first frames
    starts: List[np.ndarray]         # per merge layer bool [n_in]
    merge: List[np.ndarray]          # per merge layer bool [n_in]
    scores: Optional[np.ndarray]     # [N, L]
    keep: np.ndarray                 # bool [N, L]
    dynamic: np.ndarray              # bool [N]
    video_frame_offsets: np.ndarray  # [V+1]
    video_k: np.ndarray
    video_w: np.ndarray
    token_pos: np.ndarray
    frame_offsets: np.ndarray
    src_lo: np.ndarray
    src_hi: np.ndarray
    frames_per_block: List[int]
    tokens: Optional[np.ndarray] = None          # [n_tokens, D] when the oracle ran in the test
    sample_rows: Optional[np.ndarray] = None     # else: rows of the token list stored in full ...
    sample_tokens: Optional[np.ndarray] = None
    token_absmax: Optional[np.ndarray] = None    # ... and two summaries of every row
    token_mean: Optional[np.ndarray] = None
    input_sha: Optional[str] = None

    @property
    def n_tokens(self) -> int:
        return int(self.frame_offsets[-1])


def batch_from_results(results) -> OracleBatch:
    nm = len(results[0].merge_trace)
    sim, ema, starts, merge = [], [], [], []
    for i in range(nm):
        ss, ee = [], []
        for r in results:
            tr = r.merge_trace[i]
            s = np.zeros(tr.n_in)
            s[:tr.n_in - 1] = tr.c
            e = tr.ema.copy()
            e[0] = 0.0
            ss.append(s); ee.append(e)
        sim.append(np.concatenate(ss)); ema.append(np.concatenate(ee))
        starts.append(np.concatenate([r.merge_trace[i].starts for r in results]))
        merge.append(np.concatenate([r.merge_trace[i].merge_with_next for r in results]))
    fo = [0]
    for r in results:
        fo += list(fo[-1] + r.frame_offsets[1:])
    return OracleBatch(
        sim=sim, ema=ema, starts=starts, merge=merge,
        scores=np.concatenate([r.scores for r in results], axis=0) if results[0].scores is not None else None,
        keep=np.concatenate([r.keep for r in results], axis=0),
        dynamic=np.concatenate([r.frame_dynamic for r in results]),
        video_frame_offsets=np.concatenate([[0], np.cumsum([len(r.frame_dynamic) for r in results])]),
        video_k=np.array([r.k for r in results]), video_w=np.array([r.w for r in results]),
        token_pos=np.concatenate([r.token_pos for r in results]), frame_offsets=np.array(fo),
        src_lo=np.concatenate([r.frame_src_lo for r in results]), src_hi=np.concatenate([r.frame_src_hi for r in results]),
        frames_per_block=[int(sum(r.frames_per_block[i] for r in results)) for i in range(len(results[0].frames_per_block))],
        tokens=np.concatenate([r.tokens for r in results], axis=0))


def golden_path(name: str) -> str:
    return os.path.join(GOLDEN_DIR, f"fullsize_{name}.npz")


def batch_from_golden(name: str, n_merge_layers: int) -> OracleBatch:
    g = np.load(golden_path(name))
    shp = tuple(int(x) for x in g["keep_shape"])
    keep = np.unpackbits(g["keep_bits"], axis=1)[:, :shp[1]].astype(bool)
    return OracleBatch(
        sim=[g[f"sim_{i}"] for i in range(n_merge_layers)], ema=[g[f"ema_{i}"] for i in range(n_merge_layers)],
        starts=[g[f"starts_{i}"] for i in range(n_merge_layers)], merge=[g[f"merge_{i}"] for i in range(n_merge_layers)],
        scores=g["scores"].astype(np.float64), keep=keep, dynamic=g["dynamic"].astype(bool),
        video_frame_offsets=g["video_frame_offsets"], video_k=g["video_k"], video_w=g["video_w"],
        token_pos=g["token_pos"].astype(np.int64), frame_offsets=g["frame_offsets"], src_lo=g["src_lo"], src_hi=g["src_hi"],
        frames_per_block=[int(x) for x in g["frames_per_block"]],
        sample_rows=g["sample_rows"], sample_tokens=g["sample_tokens"], token_absmax=g["token_absmax"],
        token_mean=g["token_mean"], input_sha=str(g["input_sha"]))


def input_sha(frames: np.ndarray, blob: np.ndarray) -> str:
    """Fingerprint of the oracle's inputs, as stored in a golden file."""
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(frames).tobytes())
    h.update(np.ascontiguousarray(blob).tobytes())
    return h.hexdigest()


def compare_stage1(gpu_trace, ob: OracleBatch, params, sim_ceiling, log, stats):
    """Walk the merge layers in order.  Returns True if every decision agrees; a disagreement whose oracle margin
    is inside the near-tie band is logged and makes the function return False (the caller re-runs with the oracle's
    decisions forced); anything else raises.  Layers after the first disagreement see different lists and are
    not compared here."""
    for i in range(len(params.merge_layers)):
        sim, st, mw, ema = ob.sim[i], ob.starts[i], ob.merge[i], ob.ema[i]
        assert gpu_trace.n_in[i] == len(sim), f"merge layer {i}: list length {gpu_trace.n_in[i]} vs oracle {len(sim)}"
        gs = gpu_trace.sim[i].astype(np.float64)
        err = float(np.abs(gs - sim).max()) if len(sim) else 0.0
        ema_err = float(np.abs(gpu_trace.ema[i].astype(np.float64) - ema).max()) if len(sim) else 0.0
        stats["sim_err"] = max(stats["sim_err"], err)
        assert err <= sim_ceiling, f"merge layer {i}: similarity error {err:.3e} > {sim_ceiling}"
        stats["decisions"] += 2 * len(sim)
        bad_s = np.nonzero(gpu_trace.seg_start[i].astype(bool) != st)[0]
        bad_m = np.nonzero(gpu_trace.merge_next[i].astype(bool) != mw)[0]
        if len(bad_s) == 0 and len(bad_m) == 0:
            assert ema_err <= sim_ceiling, f"merge layer {i}: EMA error {ema_err:.3e}"
            continue
        for t in bad_s:
            margin = abs(ema[t] - params.tau_seg)
            if margin > SIM_TIE + err:
                raise AssertionError(f"layer {i} frame {t}: segmentation differs, margin {margin:.3e}, measured error {err:.3e}")
            log.append(f"near-tie: layer {i} frame {t} segmentation, |ema - tau_seg| = {margin:.2e} (error {err:.1e})")
        for t in bad_m:
            cands = []
            for u in (t - 2, t - 1, t, t + 1):
                if 0 <= u and u + 1 < len(sim):
                    cands.append(abs(sim[u] - sim[u + 1]) - err)          # two similarities compared: twice the error
                if 0 <= u < len(sim):
                    cands.append(abs(sim[u] - params.tau_merge))
            margin = min(cands)
            if len(bad_s) == 0 and margin > SIM_TIE + err:
                raise AssertionError(f"layer {i} frame {t}: merge decision differs, margin {margin:.3e}, measured error {err:.3e}")
            log.append(f"near-tie: layer {i} frame {t} merge, margin = {margin:.2e} (error {err:.1e})")
        return False
    return True


def window_of(j, L, k, w, window_mode):
    """[lo, hi) of the local window position j of a static frame falls into."""
    if window_mode == 1:
        m = -(-((j + 1) * k) // L) - 1
        return (m * L) // k, ((m + 1) * L) // k
    lo = (j // w) * w
    return lo, min(lo + w, L)


def compare_keep(gpu_keep, gpu_scores, ora_keep, ora_scores, dynamic, k, w, log, window_mode=0):
    """Kept sets must be equal except where the oracle's score is within the near-tie band of the cut (the k-th
    score on dynamic frames, the window's maximum on static frames): 1e-3 relative, widened by twice the largest
    score error measured on that frame (both scores of the comparison carry it)."""
    N, L = ora_keep.shape
    exact = True
    for f in range(N):
        diff = np.nonzero(gpu_keep[f].astype(bool) != ora_keep[f])[0]
        if len(diff) == 0:
            continue
        exact = False
        a = ora_scores[f]
        e_f = float(np.abs(gpu_scores[f].astype(np.float64) - a).max())
        if dynamic[f]:
            kth = np.sort(a)[::-1][k - 1]
            for j in diff:
                margin = abs(a[j] - kth)
                if margin > SCORE_TIE * abs(kth) + 2 * e_f:
                    raise AssertionError(f"frame {f} token {j}: top-k differs, |a - a_k| = {margin:.3e}, a_k = {kth:.3e}, "
                                         f"measured score error {e_f:.3e}")
                log.append(f"near-tie: frame {f} token {j} top-k, |a - a_k|/a_k = {margin / abs(kth):.2e}")
        else:
            for j in diff:
                lo, hi = window_of(int(j), L, k, w, window_mode)
                top = a[lo:hi].max()
                margin = abs(a[j] - top)
                if margin > SCORE_TIE * abs(top) + 2 * e_f:
                    raise AssertionError(f"frame {f} token {j}: window argmax differs, margin {margin:.3e}, "
                                         f"measured score error {e_f:.3e}")
                log.append(f"near-tie: frame {f} token {j} window, rel margin {margin / abs(top):.2e}")
    return exact


def check_parity(B, enc, frames_dev, offs, params, ob: OracleBatch, tol, sim_ceiling, score_ceiling, name=""):
    """The whole protocol (see the module docstring).  Returns (stats, log); stats = {"config", "decisions",
    "near_ties", "sim_err", "score_err", "token_err", "forced_stage1", "forced_keep"}."""
    log: List[str] = []
    stats = {"config": name, "decisions": 0, "near_ties": 0, "sim_err": 0.0, "score_err": 0.0, "token_err": 0.0,
             "forced_stage1": False, "forced_keep": False}
    free = enc.encode_batch(frames_dev, offs, params, want_trace=True)
    stage1_same = compare_stage1(free.trace, ob, params, sim_ceiling, log, stats) if params.merge_layers else True
    run = free
    if not stage1_same:
        stats["forced_stage1"] = True
        run = enc.encode_batch(frames_dev, offs, params, want_trace=True, forced=B.ForcedPlan(ob.starts, ob.merge, None))
        for i in range(len(params.merge_layers)):       # under the oracle's decisions every layer sees the oracle's list
            assert run.trace.n_in[i] == len(ob.sim[i])
            err = float(np.abs(run.trace.sim[i].astype(np.float64) - ob.sim[i]).max())
            stats["sim_err"] = max(stats["sim_err"], err)
            assert err <= sim_ceiling, f"merge layer {i} (forced decisions): similarity error {err:.3e}"
    # Stage II decisions under identical Stage I decisions
    np.testing.assert_array_equal(run.frame_dynamic.cpu().numpy().astype(bool), ob.dynamic)
    np.testing.assert_array_equal(run.video_frame_offsets.cpu().numpy(), ob.video_frame_offsets)
    keep_same = True
    if ob.scores is not None:
        rel = float(np.abs(run.trace.scores - ob.scores).max() / ob.scores.max())
        stats["score_err"] = rel
        assert rel <= score_ceiling, f"attention scores differ by {rel:.3e} of the maximum"
        vfo = ob.video_frame_offsets
        for v in range(len(vfo) - 1):
            f0, f1 = int(vfo[v]), int(vfo[v + 1])
            assert run.trace.video_k[v] == ob.video_k[v] and run.trace.video_w[v] == ob.video_w[v]
            if params.selection in (1, 2):
                stats["decisions"] += (f1 - f0) * ob.keep.shape[1]
                dynv = ob.dynamic[f0:f1] if params.selection == 1 else np.ones(f1 - f0, dtype=bool)
                keep_same &= compare_keep(run.trace.keep[f0:f1], run.trace.scores[f0:f1], ob.keep[f0:f1], ob.scores[f0:f1],
                                          dynv, int(ob.video_k[v]), int(ob.video_w[v]), log, params.window_mode)
            elif params.selection == 3:
                keep_same &= bool(np.array_equal(run.trace.keep[f0:f1].astype(bool), ob.keep[f0:f1]))
                assert keep_same, "random sampling draws the same numbers on both sides: kept sets must be identical"
    final = run
    if not keep_same:
        stats["forced_keep"] = True
        final = enc.encode_batch(frames_dev, offs, params, want_trace=True, forced=B.ForcedPlan(ob.starts, ob.merge, ob.keep))
    stats["near_ties"] = len(log)
    # values and index map under identical decisions
    assert final.n_tokens == ob.n_tokens
    got = final.tokens.cpu().numpy()
    if ob.tokens is not None:
        err = token_error(got, ob.tokens)
    else:
        err = token_error(got[ob.sample_rows], ob.sample_tokens)
        # every row: its largest magnitude and its mean, each within the tolerance scaled by the row's magnitude
        am = np.abs(got).max(axis=1)
        e_am = float((np.abs(am - ob.token_absmax) / ob.token_absmax).max())
        e_mean = float((np.abs(got.mean(axis=1, dtype=np.float64) - ob.token_mean) / ob.token_absmax).max())
        assert e_am <= tol and e_mean <= tol, f"row summaries differ: absmax {e_am:.3e}, mean {e_mean:.3e}"
        stats["row_summary_err"] = max(e_am, e_mean)
    stats["token_err"] = err
    assert err <= tol, f"token error {err:.3e} > {tol}"
    np.testing.assert_array_equal(final.token_pos.cpu().numpy(), ob.token_pos)
    np.testing.assert_array_equal(final.frame_offsets.cpu().numpy(), ob.frame_offsets)
    np.testing.assert_array_equal(final.frame_src_lo.cpu().numpy(), ob.src_lo)
    np.testing.assert_array_equal(final.frame_src_hi.cpu().numpy(), ob.src_hi)
    assert list(final.frames_per_block) == list(ob.frames_per_block)
    for line in log:
        print(line)
    print("parity " + json.dumps(stats))
    return stats, log
