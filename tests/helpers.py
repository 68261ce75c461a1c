"""Shared comparison helpers for the GPU parity tests (oracle on one side, C-ABI library on the other)."""
from __future__ import annotations

import numpy as np

SIM_TIE = 1e-3       # absolute near-tie margin for similarity decisions (similarities lie in [-1, 1])
SCORE_TIE = 1e-3     # relative near-tie margin for attention scores (they are O(1/L))


def token_error(gpu: np.ndarray, ref: np.ndarray) -> float:
    """max over tokens of ||g - o||_inf / ||o||_inf."""
    if ref.shape[0] == 0:
        return 0.0
    num = np.abs(gpu.astype(np.float64) - ref.astype(np.float64)).max(axis=1)
    den = np.abs(ref.astype(np.float64)).max(axis=1)
    return float((num / np.maximum(den, 1e-30)).max())


def oracle_trace_arrays(res, layer_idx):
    """(sim [n_in] with 0 at the end, starts, merge_next) of the oracle's trace entry."""
    tr = res.merge_trace[layer_idx]
    sim = np.zeros(tr.n_in)
    sim[:tr.n_in - 1] = tr.c
    return sim, tr.starts, tr.merge_with_next


def compare_stage1(gpu_trace, oracle_results, params, sim_tol, log):
    """Walk the merge layers in order.  Returns True if every decision agrees; a disagreement
    whose oracle margin is inside the near-tie band is logged and makes the function return False
    (caller re-runs with the oracle's decisions forced); anything else raises."""
    nm = len(params.merge_layers)
    for i in range(nm):
        sims, starts, mws, emas = [], [], [], []
        for res in oracle_results:
            s, st, mw = oracle_trace_arrays(res, i)
            sims.append(s); starts.append(st); mws.append(mw)
            e = res.merge_trace[i].ema.copy(); e[0] = 0.0
            emas.append(e)
        sim = np.concatenate(sims); st = np.concatenate(starts); mw = np.concatenate(mws); ema = np.concatenate(emas)
        assert gpu_trace.n_in[i] == len(sim), f"merge layer {i}: list length {gpu_trace.n_in[i]} vs oracle {len(sim)}"
        gs = gpu_trace.sim[i].astype(np.float64)
        err = np.abs(gs - sim).max() if len(sim) else 0.0
        assert err <= sim_tol, f"merge layer {i}: similarity error {err:.3e} > {sim_tol}"
        bad_s = np.nonzero(gpu_trace.seg_start[i] != st)[0]
        bad_m = np.nonzero(gpu_trace.merge_next[i] != mw)[0]
        if len(bad_s) == 0 and len(bad_m) == 0:
            continue
        # classify the first disagreement
        for t in bad_s:
            margin = abs(ema[t] - params.tau_seg)
            if margin > SIM_TIE + sim_tol:
                raise AssertionError(f"layer {i} frame {t}: segmentation differs, margin {margin:.3e}")
            log.append(f"near-tie: layer {i} frame {t} segmentation, |ema - tau_seg| = {margin:.2e}")
        for t in bad_m:
            cands = [abs(sim[t] - params.tau_merge)]
            for u in (t - 2, t - 1, t, t + 1):
                if 0 <= u and u + 1 < len(sim):
                    cands.append(abs(sim[u] - sim[u + 1]))
                if 0 <= u < len(sim):
                    cands.append(abs(sim[u] - params.tau_merge))
            margin = min(cands)
            if len(bad_s) == 0 and margin > SIM_TIE + 2 * sim_tol:
                raise AssertionError(f"layer {i} frame {t}: merge decision differs, margin {margin:.3e}")
            log.append(f"near-tie: layer {i} frame {t} merge, margin = {margin:.2e}")
        return False
    return True


def window_of(j, L, k, w, window_mode):
    """[lo, hi) of the local window position j of a static frame falls into."""
    if window_mode == 1:
        m = -(-((j + 1) * k) // L) - 1
        return (m * L) // k, ((m + 1) * L) // k
    lo = (j // w) * w
    return lo, min(lo + w, L)


def compare_keep(gpu_keep, gpu_scores, ora_keep, ora_scores, dynamic, k, w, score_tol, log, window_mode=0):
    """Kept sets must be equal except where the oracle's score is within the near-tie band of the
    cut (k-th score on dynamic frames, the window's maximum on static frames)."""
    N, L = ora_keep.shape
    exact = True
    for f in range(N):
        diff = np.nonzero(gpu_keep[f] != ora_keep[f])[0]
        if len(diff) == 0:
            continue
        exact = False
        a = ora_scores[f]
        if dynamic[f]:
            kth = np.sort(a)[::-1][k - 1]
            for j in diff:
                rel = abs(a[j] - kth) / abs(kth)
                if rel > SCORE_TIE + score_tol:
                    raise AssertionError(f"frame {f} token {j}: top-k differs, |a - a_k|/a_k = {rel:.3e}")
                log.append(f"near-tie: frame {f} token {j} top-k, rel margin {rel:.2e}")
        else:
            for j in diff:
                lo, hi = window_of(int(j), L, k, w, window_mode)
                win = a[lo:hi]
                rel = abs(a[j] - win.max()) / abs(win.max())
                if rel > SCORE_TIE + score_tol:
                    raise AssertionError(f"frame {f} token {j}: window argmax differs, rel margin {rel:.3e}")
                log.append(f"near-tie: frame {f} token {j} window, rel margin {rel:.2e}")
    return exact
