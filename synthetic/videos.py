"""Seeded synthetic videos with controllable temporal redundancy.

Recipe (stands in for the paper's benchmark videos, which are not available):
frame 0 is smooth uniform[0, 1] noise (one uniform value per 7x7-pixel cell and
channel, bilinearly interpolated); every following frame copies its predecessor
and replaces exactly round(p * P) of the P = (H // patch)**2 patches by fresh
smooth noise.  An optional per-frame global brightness offset, uniform in
[-jitter, +jitter], is added to that frame only (it does not accumulate).
With cut_every = c > 0 every c-th frame (t = c, 2c, ...) is a scene cut: all of its
patches are fresh, so the similarity to its predecessor drops to that of unrelated
images.  Pixels are finally mapped from [0, 1] to [-1, 1].  Output: float32 [T, 3, H, W].
"""
from __future__ import annotations

import numpy as np

CELL = 7


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def _smooth_field(rng: np.random.Generator, size: int) -> np.ndarray:
    """[3, size, size] float32 in [0, 1]: bilinear interpolation of a coarse uniform grid."""
    g = size // CELL + 2
    coarse = rng.random((3, g, g), dtype=np.float32)
    pos = (np.arange(size, dtype=np.float32) + 0.5) / CELL
    i0 = np.floor(pos).astype(np.int64)
    f = (pos - i0).astype(np.float32)
    rows = coarse[:, i0, :] * (1 - f)[None, :, None] + coarse[:, i0 + 1, :] * f[None, :, None]
    out = rows[:, :, i0] * (1 - f)[None, None, :] + rows[:, :, i0 + 1] * f[None, None, :]
    return out.astype(np.float32)


def make_video(n_frames: int, image_size: int, patch_size: int, resample_p: float,
               seed: int, jitter: float = 0.0, cut_every: int = 0) -> np.ndarray:
    grid = image_size // patch_size
    n_patches = grid * grid
    n_swap = int(round(resample_p * n_patches))
    base = _smooth_field(_rng(seed, 0), image_size)
    pick = _rng(seed, 1)
    jit = _rng(seed, 2)
    frames = np.empty((n_frames, 3, image_size, image_size), dtype=np.float32)
    for t in range(n_frames):
        cut = cut_every > 0 and t > 0 and t % cut_every == 0
        if t > 0 and (n_swap > 0 or cut):
            fresh = _smooth_field(_rng(seed, 16 + t), image_size)
            chosen = pick.permutation(n_patches)[:n_patches if cut else n_swap]
            for pidx in chosen:
                y0 = (int(pidx) // grid) * patch_size
                x0 = (int(pidx) % grid) * patch_size
                base[:, y0:y0 + patch_size, x0:x0 + patch_size] = \
                    fresh[:, y0:y0 + patch_size, x0:x0 + patch_size]
        delta = np.float32(jit.uniform(-jitter, jitter)) if jitter > 0 else np.float32(0)
        frames[t] = (base + delta) * np.float32(2.0) - np.float32(1.0)
    return frames


def make_batch(workload) -> tuple[np.ndarray, np.ndarray]:
    """All videos of a workload concatenated along the frame axis, plus int32 offsets [V+1]."""
    s = workload.shape
    vids = [make_video(v.n_frames, s.image_size, s.patch_size, v.resample_p, v.seed, v.jitter, v.cut_every)
            for v in workload.videos]
    offs = np.zeros(len(vids) + 1, dtype=np.int32)
    offs[1:] = np.cumsum([v.shape[0] for v in vids])
    return np.ascontiguousarray(np.concatenate(vids, axis=0)), offs
