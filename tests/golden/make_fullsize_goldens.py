"""Writes the oracle's results for the full-size workloads to tests/golden/fullsize_<name>.npz.

    python tests/golden/make_fullsize_goldens.py [workload ...]        (default: every full-size workload)

The numpy oracle needs about ten seconds per frame of SigLIP-so400m shape, i.e. minutes to an hour per
workload, which is too slow to repeat inside every GPU test run; so it is run once, here, on CPU, and the GPU
parity tests compare the library with the stored values.  This script imports only `oracle` and `synthetic`
(never the CUDA package), so no stored value can come from the GPU path.

Stored per workload (all videos of the call concatenated in call order):
  input_sha        sha256 of the fp32 frames and of the weight blob the oracle consumed (the tests recompute it
                   from the seeded generators, so a drift of the generators is noticed)
  per merge layer i: sim_i, ema_i (float64), starts_i, merge_i (bool), w_a_i, w_b_i (float64), n_in_i, n_out_i
  scores           float32 [N, L] attention scores A of the output frames
  keep_bits        np.packbits of the kept mask [N, L]
  dynamic, src_lo, src_hi, frame_offsets, token_pos, video_frame_offsets, video_k, video_w, video_M
  frames_per_block frames alive in every block (summed over videos)
  token_absmax, token_mean   float32 [n_tokens] row summaries of EVERY output token
  sample_rows, sample_tokens full rows chosen by a fixed rule: every 3rd token of the first merged frame and of
                   the first static frame of video 0, plus every 97th row of the whole list
"""
from __future__ import annotations

import hashlib
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import earlytom_oracle as O  # noqa: E402
from synthetic import make_batch, make_weights, workload  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))
FULL_SIZE = ("so400m_32f", "so400m_32f_cal", "so400m_64f_p10", "so400m_64f_p50", "so400m_64f_p90", "serve_8x32",
             "qwenvl_768f")
ROW_STRIDE = 97


def input_sha(frames: np.ndarray, blob: np.ndarray) -> str:
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(frames).tobytes())
    h.update(np.ascontiguousarray(blob).tobytes())
    return h.hexdigest()


def sample_rows(results) -> np.ndarray:
    """Indices into the concatenated token list (see the module docstring)."""
    r = results[0]
    N = len(r.frame_dynamic)
    merged = [f for f in range(N) if r.frame_src_hi[f] > r.frame_src_lo[f]]
    static = [f for f in range(N) if not r.frame_dynamic[f]]
    rows = []
    for f in {merged[0] if merged else 0, static[0] if static else N - 1}:
        rows.extend(range(int(r.frame_offsets[f]), int(r.frame_offsets[f + 1]), 3))
    total = sum(x.tokens.shape[0] for x in results)
    rows.extend(range(0, total, ROW_STRIDE))
    return np.unique(np.asarray(rows, dtype=np.int64))


def build(name: str) -> str:
    wl = workload(name)
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed, wl.pos_std)
    w = O.split_weights(wl.shape, blob)
    t0 = time.time()
    results = []
    for v in range(len(offs) - 1):
        results.append(O.encode_video(frames[offs[v]:offs[v + 1]], wl.shape, w, wl.params, dtype=np.float32, video_index=v))
        print(f"{name}: video {v} done, {len(results[-1].frame_dynamic)} frames out, {time.time() - t0:.0f} s", flush=True)
    out = dict(input_sha=np.array(input_sha(frames, blob)), oracle_seconds=np.array(time.time() - t0))
    for i in range(len(wl.params.merge_layers)):
        trs = [r.merge_trace[i] for r in results]
        sims, emas = [], []
        for tr in trs:
            s = np.zeros(tr.n_in)
            s[:tr.n_in - 1] = tr.c
            e = tr.ema.copy()
            e[0] = 0.0
            sims.append(s); emas.append(e)
        out[f"sim_{i}"] = np.concatenate(sims)
        out[f"ema_{i}"] = np.concatenate(emas)
        out[f"starts_{i}"] = np.concatenate([tr.starts for tr in trs])
        out[f"merge_{i}"] = np.concatenate([tr.merge_with_next for tr in trs])
        out[f"w_a_{i}"] = np.concatenate([tr.w_a for tr in trs])
        out[f"w_b_{i}"] = np.concatenate([tr.w_b for tr in trs])
        out[f"n_in_{i}"] = np.array([tr.n_in for tr in trs])
        out[f"n_out_{i}"] = np.array([tr.n_out for tr in trs])
    keep = np.concatenate([r.keep for r in results], axis=0)
    toks = np.concatenate([r.tokens for r in results], axis=0).astype(np.float32)
    fo = [0]
    for r in results:
        fo += list(fo[-1] + r.frame_offsets[1:])
    rows = sample_rows(results)
    out.update(
        scores=np.concatenate([r.scores for r in results], axis=0).astype(np.float32),
        keep_bits=np.packbits(keep, axis=1), keep_shape=np.array(keep.shape),
        dynamic=np.concatenate([r.frame_dynamic for r in results]),
        src_lo=np.concatenate([r.frame_src_lo for r in results]).astype(np.int32),
        src_hi=np.concatenate([r.frame_src_hi for r in results]).astype(np.int32),
        frame_offsets=np.array(fo, dtype=np.int64),
        token_pos=np.concatenate([r.token_pos for r in results]).astype(np.int16),
        video_frame_offsets=np.concatenate([[0], np.cumsum([len(r.frame_dynamic) for r in results])]),
        video_k=np.array([r.k for r in results]), video_w=np.array([r.w for r in results]),
        video_M=np.array([r.M for r in results]),
        frames_per_block=np.sum([r.frames_per_block for r in results], axis=0),
        token_absmax=np.abs(toks).max(axis=1), token_mean=toks.mean(axis=1, dtype=np.float64).astype(np.float32),
        sample_rows=rows, sample_tokens=toks[rows])
    path = os.path.join(HERE, f"fullsize_{name}.npz")
    np.savez_compressed(path, **out)
    print(f"{name}: wrote {path} ({os.path.getsize(path) / 1e6:.1f} MB), {toks.shape[0]} tokens, "
          f"{len(rows)} sampled rows, oracle {time.time() - t0:.0f} s", flush=True)
    return path


if __name__ == "__main__":
    for nm in (sys.argv[1:] or FULL_SIZE):
        build(nm)
