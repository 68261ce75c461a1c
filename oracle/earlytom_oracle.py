"""CPU oracle for the compressed video vision-encoder (EarlyTom).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the hot path
computes.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it;
the CUDA library never does, and the two share no code.  numpy only; every floating-point
quantity is float64 by default (``dtype=np.float32`` gives the fp32 variant used for the
large workloads, where matmul time matters); all decision quantities (similarities, EMA,
comparisons, attention scores) are float64 in both variants.  ``np.matmul`` (BLAS), ``np.exp``,
``np.tanh`` and ``math.erf`` are the only library primitives; there is no blocking or fusion.

The method is a heuristic pipeline, so the oracle is the algorithm's steps in the paper's order:

  encoder forward            Sec. 3.1 (attention QK^T / sqrt(d)); SigLIP-style pre-LN ViT
  frame similarity           Sec. 3.2, "Streaming frame segmentation" (mean token-wise cosine)
  streaming segmentation     Eq. 1, Algorithm 1 ("SegmentBySimilarity")
  middle-frame merge         Eq. 2, Algorithm 1 (while loop over the middle frames)
  weighted frame merge       Eq. 3
  dynamic / static split     Sec. 3.3, Algorithm 2 (head and tail of each segment are dynamic)
  re-scaled amount           Eq. 5 (read as a per-frame token count, see ``rescaled_keep``)
  global top-K               Eq. 4
  local-window top-1         Eq. 6
  gather in temporal order   Eq. 7
  cost model                 Eq. 8

Pinning status (tests/test_oracle_*.py): encoder forward pinned against a composition of
torch CPU library ops; similarity, segmentation, merge rule, weights (the formula and the assembled
step, on frames whose similarities are known cosines), top-k, windows (both window modes) pinned by
closed forms, brute force and invariants.  Readings with no external pin ("parity unpinned"):
which tensor is compared and merged (the residual stream entering the block), the value of
tau_merge (a parameter), the definition of the per-token attention score A (mean over heads and
queries of the last block's attention probabilities; only its row sum and the uniform case are
pinned), which segmentation feeds Stage II (that of the last merge layer), composition of
several merge layers (re-run from scratch on the merged list).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

COS_EPS = 1e-8      # clamp of the cosine denominator (zero-norm tokens contribute 0)
WSUM_EPS = 1e-6     # Eq. 3 denominator guard: below it the merge is a plain mean


# ----------------------------------------------------------------------------------------------
# Weights
# ----------------------------------------------------------------------------------------------

def split_weights(shape, blob: np.ndarray) -> Dict[str, np.ndarray]:
    """Views into the fp32 blob in the library's documented order (see include/earlytom.h)."""
    if int(getattr(shape, "arch", 0)) == 1:
        from oracle import qwenvl_oracle as Q
        return Q.split_weights(shape, blob)
    D, M, L = shape.hidden, shape.mlp_dim, shape.tokens_per_frame
    P = 3 * shape.patch_size * shape.patch_size
    out: Dict[str, np.ndarray] = {}
    off = 0

    def take(name, *shp):
        nonlocal off
        n = int(np.prod(shp))
        out[name] = blob[off:off + n].reshape(shp)
        off += n

    take("patch_w", P, D); take("patch_b", D); take("pos", L, D)
    for i in range(shape.num_layers):
        p = f"l{i}."
        take(p + "ln1_g", D); take(p + "ln1_b", D)
        take(p + "wqkv", D, 3 * D); take(p + "bqkv", 3 * D)
        take(p + "wo", D, D); take(p + "bo", D)
        take(p + "ln2_g", D); take(p + "ln2_b", D)
        take(p + "w1", D, M); take(p + "b1", M)
        take(p + "w2", M, D); take(p + "b2", D)
    take("post_g", D); take("post_b", D)
    if off != blob.size:
        raise ValueError(f"weight blob has {blob.size} floats, layout needs {off}")
    return out


# ----------------------------------------------------------------------------------------------
# Encoder pieces (SigLIP-style ViT: patch embedding, pre-LN blocks, per-frame attention)
# ----------------------------------------------------------------------------------------------

def patchify(frames: np.ndarray, patch: int) -> np.ndarray:
    """[T,3,H,W] -> [T, L, 3*p*p]; non-overlapping patches of the top-left (H//p*p)^2 crop,
    row-major patch grid, feature index c*p*p + dy*p + dx (a stride-p valid convolution)."""
    T, C, H, W = frames.shape
    gh, gw = H // patch, W // patch
    x = frames[:, :, :gh * patch, :gw * patch].reshape(T, C, gh, patch, gw, patch)
    x = x.transpose(0, 2, 4, 1, 3, 5)             # T, gy, gx, c, dy, dx
    return x.reshape(T, gh * gw, C * patch * patch)


def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True, dtype=np.float64)
    var = ((x.astype(np.float64) - mu) ** 2).mean(axis=-1, keepdims=True)
    y = (x.astype(np.float64) - mu) / np.sqrt(var + eps)
    return (y * g + b).astype(x.dtype)


def gelu(x: np.ndarray, tanh_approx: bool) -> np.ndarray:
    if tanh_approx:
        c = math.sqrt(2.0 / math.pi)
        return (0.5 * x * (1.0 + np.tanh(c * (x + 0.044715 * x ** 3)))).astype(x.dtype)
    erf = np.vectorize(math.erf, otypes=[np.float64])
    return (0.5 * x * (1.0 + erf(x / math.sqrt(2.0)))).astype(x.dtype)


def attention_probs(q: np.ndarray, k: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(d)) over the keys; q, k [L, d]  (Sec. 3.1)."""
    s = (q @ k.T) / math.sqrt(q.shape[-1])
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def mha(xn: np.ndarray, w, p: str, heads: int, want_scores: bool):
    """Multi-head self-attention of one frame (tokens attend only inside their frame).
    Returns (projected output [L, D], per-token attention score [L] float64 or None)."""
    L, D = xn.shape
    dh = D // heads
    qkv = xn @ w[p + "wqkv"].astype(xn.dtype) + w[p + "bqkv"].astype(xn.dtype)
    q, k, v = qkv[:, :D], qkv[:, D:2 * D], qkv[:, 2 * D:]
    ctx = np.empty_like(xn)
    score = np.zeros(L, dtype=np.float64) if want_scores else None
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        P = attention_probs(q[:, sl], k[:, sl])
        ctx[:, sl] = P @ v[:, sl]
        if want_scores:
            score += P.astype(np.float64).sum(axis=0)       # attention received by key j
    if want_scores:
        score /= float(heads * L)                            # mean over heads and queries
    out = ctx @ w[p + "wo"].astype(xn.dtype) + w[p + "bo"].astype(xn.dtype)
    return out, score


def encoder_block(X: np.ndarray, w, layer: int, shape, want_scores: bool):
    """X [n, L, D] -> X after block `layer`; optionally the attention scores A [n, L]."""
    p = f"l{layer}."
    n, L, D = X.shape
    A = np.zeros((n, L), dtype=np.float64) if want_scores else None
    out = np.empty_like(X)
    for f in range(n):
        x = X[f]
        a, sc = mha(layer_norm(x, w[p + "ln1_g"], w[p + "ln1_b"], shape.ln_eps), w, p, shape.heads, want_scores)
        x = x + a
        hmid = layer_norm(x, w[p + "ln2_g"], w[p + "ln2_b"], shape.ln_eps) @ w[p + "w1"].astype(x.dtype) \
            + w[p + "b1"].astype(x.dtype)
        hmid = gelu(hmid, bool(shape.gelu_tanh))
        x = x + (hmid @ w[p + "w2"].astype(x.dtype) + w[p + "b2"].astype(x.dtype))
        out[f] = x
        if want_scores:
            A[f] = sc
    return out, A


# ----------------------------------------------------------------------------------------------
# Stage I: inner-encoder frame merging (Sec. 3.2, Algorithm 1)
# ----------------------------------------------------------------------------------------------

def frame_similarity(F: np.ndarray) -> np.ndarray:
    """c[t] = Sim(F_t, F_{t+1}): mean over the L positions of the cosine between the two tokens at
    the same position (Sec. 3.2).  F [n, L, D] -> float64 [n-1]."""
    F = F.astype(np.float64)
    n = F.shape[0]
    c = np.zeros(max(n - 1, 0), dtype=np.float64)
    for t in range(n - 1):
        a, b = F[t], F[t + 1]
        dot = (a * b).sum(axis=-1)
        den = np.sqrt((a * a).sum(axis=-1)) * np.sqrt((b * b).sum(axis=-1))
        c[t] = (dot / np.maximum(den, COS_EPS)).mean()
    return c


def segment_by_similarity(c: Sequence[float], n: int, alpha: float, tau_seg: float):
    """Eq. 1.  s_t = c[t-1] is the similarity of frames t-1 and t; the EMA starts at the first
    similarity of a segment and restarts after every break; frame t opens a new segment when the
    smoothed value is below tau_seg.  Returns (starts: bool [n], ema: float64 [n], ema[0] = nan)."""
    starts = np.zeros(n, dtype=bool)
    ema = np.full(n, np.nan, dtype=np.float64)
    if n == 0:
        return starts, ema
    starts[0] = True
    prev = None
    for t in range(1, n):
        s = float(c[t - 1])
        cur = s if prev is None else alpha * s + (1.0 - alpha) * prev
        ema[t] = cur
        if cur < tau_seg:
            starts[t] = True
            prev = None
        else:
            prev = cur
    return starts, ema


def segments_from_starts(starts: np.ndarray) -> List[List[int]]:
    segs: List[List[int]] = []
    for t, s in enumerate(starts):
        if s:
            segs.append([])
        segs[-1].append(t)
    return segs


def merge_pairs(c: Sequence[float], segs: List[List[int]], tau_merge: float) -> np.ndarray:
    """Eq. 2 inside each segment, Algorithm 1's loop over the middle frames g_1..g_{k-1}.
    Both frames of a merged pair are middle frames (the paper's text excludes head and tail),
    so a pair may start at local index i only while i <= k-2; the similarity to the following
    frame, c[g_{i+1}], then always lies inside the segment.  All similarities are those of the
    un-merged frames of this layer.  Returns merge_with_next: bool [n]."""
    n = sum(len(s) for s in segs)
    mw = np.zeros(n, dtype=bool)
    for g in segs:
        k = len(g) - 1
        i = 1
        while i <= k - 1:
            if i <= k - 2 and c[g[i]] > tau_merge and c[g[i]] > c[g[i + 1]]:
                mw[g[i]] = True
                i += 2
            else:
                i += 1
    return mw


@dataclass
class MergeLayerTrace:
    layer: int
    n_in: int
    c: np.ndarray                 # [n_in-1] similarities (concatenated over videos; cross-video gaps = nan)
    ema: np.ndarray               # [n_in]
    starts: np.ndarray            # [n_in] bool, frame opens a segment
    merge_with_next: np.ndarray   # [n_in] bool
    w_a: np.ndarray               # [n_out] weight of the first source frame
    w_b: np.ndarray               # [n_out] weight of the second (0 if a copy)
    src_a: np.ndarray             # [n_out]
    src_b: np.ndarray             # [n_out], -1 if a copy
    n_out: int = 0


def weighted_merge(Fa, Fb, sa: float, sb: float, weighted: bool):
    """Eq. 3: (s_a F_a + s_b F_b) / (s_a + s_b); plain mean when unweighted or the sum is ~0."""
    den = sa + sb
    if (not weighted) or den <= WSUM_EPS:
        wa, wb = 0.5, 0.5
    else:
        wa, wb = sa / den, sb / den
    return (wa * Fa.astype(np.float64) + wb * Fb.astype(np.float64)).astype(Fa.dtype), wa, wb


@dataclass
class FrameMeta:
    src_lo: int          # first original frame merged into this frame (index inside its video)
    src_hi: int          # last one
    seg_id: int = 0      # segment of the last merge layer (per video)
    role: int = 0        # 0 head, 1 middle, 2 tail, 3 head==tail (1-frame segment)


def stage1_one_video(F: np.ndarray, meta: List[FrameMeta], alpha, tau_seg, tau_merge, weighted: bool, layer: int):
    """Algorithm 1 on one video's current frame list.  Returns (F', meta', trace)."""
    n = F.shape[0]
    c = frame_similarity(F)
    starts, ema = segment_by_similarity(c, n, alpha, tau_seg)
    segs = segments_from_starts(starts)
    mw = merge_pairs(c, segs, tau_merge)
    out_frames, out_meta = [], []
    w_a, w_b, s_a, s_b = [], [], [], []
    for sid, g in enumerate(segs):
        k = len(g) - 1
        j = 0
        while j <= k:
            t = g[j]
            role = 3 if k == 0 else (0 if j == 0 else (2 if j == k else 1))
            if mw[t]:
                merged, wa, wb = weighted_merge(F[t], F[t + 1], float(c[t]), float(c[t + 1]), weighted)
                out_frames.append(merged)
                out_meta.append(FrameMeta(meta[t].src_lo, meta[t + 1].src_hi, sid, 1))
                w_a.append(wa); w_b.append(wb); s_a.append(t); s_b.append(t + 1)
                j += 2
            else:
                out_frames.append(F[t])
                out_meta.append(FrameMeta(meta[t].src_lo, meta[t].src_hi, sid, role))
                w_a.append(1.0); w_b.append(0.0); s_a.append(t); s_b.append(-1)
                j += 1
    Fo = np.stack(out_frames, axis=0) if out_frames else F[:0]
    tr = MergeLayerTrace(layer, n, c, ema, starts, mw, np.array(w_a), np.array(w_b),
                         np.array(s_a, dtype=np.int64), np.array(s_b, dtype=np.int64), len(out_frames))
    return Fo, out_meta, tr


def roles_of_segments(starts: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(seg_id [n], role [n]) of an un-merged list given its segment starts."""
    segs = segments_from_starts(starts)
    n = len(starts)
    sid = np.zeros(n, dtype=np.int64)
    role = np.zeros(n, dtype=np.int64)
    for s, g in enumerate(segs):
        for j, t in enumerate(g):
            sid[t] = s
            role[t] = 3 if len(g) == 1 else (0 if j == 0 else (2 if j == len(g) - 1 else 1))
    return sid, role


# ----------------------------------------------------------------------------------------------
# Stage II: decoupled spatial token selection (Sec. 3.3, Algorithm 2)
# ----------------------------------------------------------------------------------------------

def rescaled_keep(r: float, B: int, N: int, L: int, retain_mode: int, window_mode: int = 0) -> Tuple[int, int, int]:
    """Eq. 5-6.  The printed Eq. 5 cannot be used literally (it yields ~1e-3 where Eq. 6 needs a
    token amount), so r-hat is read as the per-frame token amount that restores the target ratio
    after Stage I removed B-N frames:  k = floor(r*B*L / N)  (mode 1) or floor(r*L) (mode 0),
    clamped to [1, L];  window width w = floor(L / k) >= 1.
    Window count M of a static frame: Eq. 6 as printed (window_mode 0) cuts windows of exactly w
    positions, M = ceil(L / w), which is >= k and equals L as soon as k > L/2 (static frames then keep
    every token and the target ratio is missed); window_mode 1 cuts M = k windows of near-equal width
    (see `window_edges`), so that a static frame keeps exactly as many tokens as a dynamic one."""
    if retain_mode == 1:
        k = int(math.floor(r * B * L / N + 1e-9))
    else:
        k = int(math.floor(r * L + 1e-9))
    k = max(1, min(L, k))
    w = max(1, L // k)
    M = k if window_mode == 1 else -(-L // w)
    return k, w, M


def window_edges(L: int, k: int, w: int, window_mode: int = 0) -> List[int]:
    """Boundaries e_0 = 0 < e_1 < ... < e_M = L of the local windows of a static frame (window m is
    [e_m, e_{m+1})).  window_mode 0: Eq. 6 as printed, consecutive windows of w positions, the last one
    possibly shorter.  window_mode 1: k windows with e_m = floor(m*L/k), widths floor(L/k) or that plus
    one; identical to mode 0 whenever k divides L."""
    if window_mode == 1:
        return [(m * L) // k for m in range(k + 1)]
    return list(range(0, L, w)) + [L]


def topk_mask(a: np.ndarray, k: int) -> np.ndarray:
    """Eq. 4: the k largest scores; ties broken towards the lower index."""
    order = sorted(range(len(a)), key=lambda j: (-float(a[j]), j))
    m = np.zeros(len(a), dtype=bool)
    m[order[:k]] = True
    return m


def window_mask(a: np.ndarray, w: int, k: int = 0, window_mode: int = 0) -> np.ndarray:
    """Eq. 6: the maximum of each local window is kept, the lowest index among equals.  The windows
    are those of `window_edges` (consecutive runs of w positions over the flattened token index in
    mode 0, k near-equal runs in mode 1)."""
    L = len(a)
    m = np.zeros(L, dtype=bool)
    edges = window_edges(L, k, w, window_mode)
    for lo, hi in zip(edges[:-1], edges[1:]):
        best = lo
        for j in range(lo + 1, hi):
            if a[j] > a[best]:
                best = j
        m[best] = True
    return m


def philox4x32_10(counter: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox-4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11),
    written from its published definition.  counter uint32 [..., 4] -> uint32 [..., 4]."""
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    mask = np.uint64(0xFFFFFFFF)
    c = [counter[..., i].astype(np.uint64) for i in range(4)]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0 = np.uint64(M0) * c[0]
        p1 = np.uint64(M1) * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c = [hi1 ^ c[1] ^ np.uint64(k0), lo1, hi0 ^ c[3] ^ np.uint64(k1), lo0]
        k0, k1 = (k0 + W0) & 0xFFFFFFFF, (k1 + W1) & 0xFFFFFFFF
    return np.stack(c, axis=-1).astype(np.uint32)


def random_scores(seed: int, video: int, n_frames: int, L: int) -> np.ndarray:
    """Scores of the random-sampling baseline (the paper's sampling ablation): token j of output frame f of
    video v gets the uniform number (x >> 8) / 2^24, x = first word of Philox(counter (j, f, v, 0), key = seed)."""
    ctr = np.zeros((n_frames, L, 4), dtype=np.uint32)
    ctr[..., 0] = np.arange(L, dtype=np.uint32)[None, :]
    ctr[..., 1] = np.arange(n_frames, dtype=np.uint32)[:, None]
    ctr[..., 2] = np.uint32(video)
    x = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))[..., 0]
    return (x >> np.uint32(8)).astype(np.float64) / float(1 << 24)


def select_tokens(A: np.ndarray, dynamic: np.ndarray, k: int, w: int, selection: int, window_mode: int = 0) -> np.ndarray:
    """keep mask [N, L].  selection: 0 keep all, 1 decoupled (dynamic: top-k, static: windows),
    2 plain per-frame top-k on every frame (3, random sampling, is selection 2 applied to `random_scores`)."""
    N, L = A.shape
    keep = np.zeros((N, L), dtype=bool)
    for f in range(N):
        if selection == 0:
            keep[f] = True
        elif selection == 2 or dynamic[f]:
            keep[f] = topk_mask(A[f], k)
        else:
            keep[f] = window_mask(A[f], w, k, window_mode)
    return keep


# ----------------------------------------------------------------------------------------------
# Whole path
# ----------------------------------------------------------------------------------------------

@dataclass
class VideoResult:
    tokens: np.ndarray            # [n_tokens, D] compressed tokens, frames in temporal order
    frame_offsets: np.ndarray     # [N+1] into tokens
    token_pos: np.ndarray         # [n_tokens] spatial index of each kept token (kept-index map)
    frame_src_lo: np.ndarray      # [N]
    frame_src_hi: np.ndarray      # [N]
    frame_dynamic: np.ndarray     # [N] bool
    keep: np.ndarray              # [N, L] bool
    scores: Optional[np.ndarray]  # [N, L] float64 attention scores A
    k: int
    w: int
    M: int
    merge_trace: List[MergeLayerTrace] = field(default_factory=list)
    features: Optional[np.ndarray] = None    # [N, L, D] post-LN features before selection
    frames_per_block: List[int] = field(default_factory=list)


def encode_video(frames: np.ndarray, shape, blob_or_w, params, dtype=np.float64,
                 keep_features: bool = False, forced: Optional[dict] = None, video_index: int = 0) -> VideoResult:
    """frames [B,3,H,W] of ONE video -> compressed tokens + index map.

    `forced` (tests only) replays given decisions instead of taking them:
      {"merge": {layer: (starts bool[n], merge_with_next bool[n])}, "keep": bool [N, L]}.
    """
    arch = int(getattr(shape, "arch", 0))
    if arch == 1:
        # Qwen2.5-VL-style encoder (the paper's generalisation study): same method, another encoder.  A "frame" is an
        # encoder frame (temporal_patch input frames); the encoder's pieces live in oracle/qwenvl_oracle.py.
        from oracle import qwenvl_oracle as Q
        w = blob_or_w if isinstance(blob_or_w, dict) else Q.split_weights(shape, blob_or_w)
        X = Q.embed(frames.astype(dtype), shape, w)
        block = Q.encoder_block
    else:
        w = blob_or_w if isinstance(blob_or_w, dict) else split_weights(shape, blob_or_w)
        X = patchify(frames.astype(dtype), shape.patch_size) @ w["patch_w"].astype(dtype) \
            + w["patch_b"].astype(dtype) + w["pos"].astype(dtype)[None]
        block = encoder_block
    B = X.shape[0]
    L, D = shape.tokens_per_frame, shape.hidden
    meta = [FrameMeta(t, t) for t in range(B)]
    traces: List[MergeLayerTrace] = []
    A = None
    fpb: List[int] = []
    merge_layers = tuple(params.merge_layers)
    for layer in range(shape.num_layers):
        if layer in merge_layers:
            if forced is not None and "merge" in forced:
                X, meta, tr = _stage1_forced(X, meta, forced["merge"][layer], bool(params.weighted_merge), layer)
            else:
                X, meta, tr = stage1_one_video(X, meta, params.ema_alpha, params.tau_seg, params.tau_merge,
                                               bool(params.weighted_merge), layer)
            traces.append(tr)
        fpb.append(X.shape[0])
        last = layer == shape.num_layers - 1
        X, sc = block(X, w, layer, shape, want_scores=last)
        if last:
            A = sc
    N = X.shape[0]
    if arch == 1:
        feats = Q.final_norm(X, w, shape)
    else:
        feats = layer_norm(X, w["post_g"], w["post_b"], shape.ln_eps) if shape.post_layernorm else X
    if not merge_layers:
        # Stage I is off: the segment list for Stage II comes from running the streaming segmentation
        # of Sec. 3.2 on the final features (Sec. 3.3 says the division follows that segmentation).
        starts, _ = segment_by_similarity(frame_similarity(X), N, params.ema_alpha, params.tau_seg)
        sid, role = roles_of_segments(starts)
        for f in range(N):
            meta[f].seg_id, meta[f].role = int(sid[f]), int(role[f])
    dynamic = np.array([m.role != 1 for m in meta], dtype=bool)
    wmode = int(getattr(params, "window_mode", 0))
    k, wdt, M = rescaled_keep(params.retain, B, N, L, params.retain_mode, wmode)
    if forced is not None and "keep" in forced:
        keep = np.asarray(forced["keep"], dtype=bool)
    elif params.selection == 3:
        # random sampling (paper's sampling ablation): k tokens per frame, uniformly at random
        keep = select_tokens(random_scores(int(getattr(params, "sample_seed", 0)), video_index, N, L), dynamic, k, wdt, 2)
    else:
        keep = select_tokens(A, dynamic, k, wdt, params.selection, wmode)
    counts = keep.sum(axis=1)
    offs = np.zeros(N + 1, dtype=np.int64)
    offs[1:] = np.cumsum(counts)
    pos = np.concatenate([np.nonzero(keep[f])[0] for f in range(N)]) if N else np.zeros(0, np.int64)
    toks = np.concatenate([feats[f][keep[f]] for f in range(N)], axis=0) if N else feats.reshape(0, D)
    return VideoResult(tokens=toks, frame_offsets=offs, token_pos=pos.astype(np.int64),
                       frame_src_lo=np.array([m.src_lo for m in meta]), frame_src_hi=np.array([m.src_hi for m in meta]),
                       frame_dynamic=dynamic, keep=keep, scores=A, k=k, w=wdt, M=M, merge_trace=traces,
                       features=feats if keep_features else None, frames_per_block=fpb)


def _stage1_forced(F, meta, decision, weighted: bool, layer: int):
    """Stage I with the segmentation and the merged pairs given; similarities (hence the Eq. 3
    weights) are still computed from F."""
    starts, mw = (np.asarray(d, dtype=bool) for d in decision)
    n = F.shape[0]
    c = frame_similarity(F)
    sid_in, role_in = roles_of_segments(starts)
    out_frames, out_meta, w_a, w_b, s_a, s_b = [], [], [], [], [], []
    t = 0
    while t < n:
        if mw[t]:
            merged, wa, wb = weighted_merge(F[t], F[t + 1], float(c[t]), float(c[t + 1]) if t + 1 < n - 1 else 0.0, weighted)
            out_frames.append(merged)
            out_meta.append(FrameMeta(meta[t].src_lo, meta[t + 1].src_hi, int(sid_in[t]), 1))
            w_a.append(wa); w_b.append(wb); s_a.append(t); s_b.append(t + 1)
            t += 2
        else:
            out_frames.append(F[t])
            out_meta.append(FrameMeta(meta[t].src_lo, meta[t].src_hi, int(sid_in[t]), int(role_in[t])))
            w_a.append(1.0); w_b.append(0.0); s_a.append(t); s_b.append(-1)
            t += 1
    _, ema = segment_by_similarity(c, n, 1.0, -2.0)
    tr = MergeLayerTrace(layer, n, c, ema, starts, mw, np.array(w_a), np.array(w_b),
                         np.array(s_a, dtype=np.int64), np.array(s_b, dtype=np.int64), len(out_frames))
    return np.stack(out_frames, axis=0), out_meta, tr


def encode_batch(frames: np.ndarray, video_offsets: Sequence[int], shape, blob_or_w, params,
                 dtype=np.float64, **kw) -> List[VideoResult]:
    """Independent videos: each one goes through `encode_video` on its own."""
    if isinstance(blob_or_w, dict):
        w = blob_or_w
    elif int(getattr(shape, "arch", 0)) == 1:
        from oracle import qwenvl_oracle as Q
        w = Q.split_weights(shape, blob_or_w)
    else:
        w = split_weights(shape, blob_or_w)
    return [encode_video(frames[video_offsets[v]:video_offsets[v + 1]], shape, w, params, dtype=dtype, video_index=v, **kw)
            for v in range(len(video_offsets) - 1)]


# ----------------------------------------------------------------------------------------------
# Cost model
# ----------------------------------------------------------------------------------------------

def eq8_macs(tokens_per_frame: int, frames_per_block: Sequence[int], D: int, M: int) -> int:
    """Eq. 8 summed over the executed blocks: 4 L D^2 + 2 L^2 D + 2 L D M multiply-accumulates
    per frame per block (attention is per frame, so L_i is the per-frame token count)."""
    L = tokens_per_frame
    per = 4 * L * D * D + 2 * L * L * D + 2 * L * D * M
    return int(sum(frames_per_block)) * per
