"""The workload configurations (shapes and parameters only, no arithmetic).

Five workloads mirror the benchmark definition of this repository:

  tiny        2-layer fp32 ViT, 8 frames of 112x112, merge after layer 1, per-frame top-k 50 %
  so400m_8f   SigLIP-so400m shapes, bf16, 8 frames, 30 % patch resampling
  so400m_32f  same encoder, 32 frames (LLaVA-OneVision's frame count), 20 % resampling + brightness jitter
  so400m_32f_cal  the same with a scene cut every 6 frames (frame retention of Stage I near the paper's 73.9 %)
  so400m_64f_p{10,50,90}  64 frames at three levels of temporal redundancy
  serve_8x32  eight independent 32-frame videos encoded in one call, 25 % total retention
  qwenvl_*    a Qwen2.5-VL-style encoder (windows, 2-D rotary positions, two input frames per encoder frame),
              the architecture of the paper's generalisation study, at 15 % retention

The "main setting" is the hyper-parameter row of the paper's appendix table for
25 % retention (EMA factor 0.9, segmentation threshold 0.8, merge layers
[6, 14, 20]); the merge threshold, which the paper never prints, is a free
parameter of the library and defaults to the segmentation threshold.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Tuple

import numpy as np


@dataclass(frozen=True)
class EncoderShape:
    image_size: int
    patch_size: int
    num_layers: int
    hidden: int
    heads: int
    mlp_dim: int
    ln_eps: float = 1e-6
    gelu_tanh: int = 1
    post_layernorm: int = 1
    # arch 0: SigLIP-style (LayerNorm, GELU MLP, learned position table, full per-frame attention).
    # arch 1: Qwen2.5-VL-style (RMSNorm, gated SiLU MLP, 2-D rotary positions, attention inside windows of
    #         `window` x `window` patches except in the blocks of `full_attn_layers`, `temporal_patch` input frames
    #         per encoder frame, no position table, no patch-embedding bias)
    arch: int = 0
    temporal_patch: int = 1
    window: int = 0
    full_attn_layers: Tuple[int, ...] = ()
    rope_theta: float = 10000.0

    @property
    def grid(self) -> int:
        return self.image_size // self.patch_size

    @property
    def tokens_per_frame(self) -> int:
        return self.grid * self.grid

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    @property
    def patch_dim(self) -> int:
        return 3 * self.temporal_patch * self.patch_size * self.patch_size

    @property
    def full_attn_mask(self) -> int:
        m = 0
        for layer in self.full_attn_layers:
            m |= 1 << layer
        return m


@dataclass(frozen=True)
class MergeParams:
    merge_layers: Tuple[int, ...] = (6, 14, 20)
    ema_alpha: float = 0.9
    tau_seg: float = 0.8
    tau_merge: float = 0.8
    weighted_merge: int = 1
    selection: int = 1      # 0 none, 1 decoupled, 2 plain per-frame top-k, 3 random sampling (ablation)
    retain_mode: int = 1    # 0 per-frame fraction, 1 total budget
    retain: float = 0.25
    sample_seed: int = 0    # seed of the random-sampling ablation (selection 3)
    window_mode: int = 1    # static frames: 0 = windows of floor(L/k) positions (Eq. 6 as printed), 1 = k near-equal windows


@dataclass(frozen=True)
class VideoSpec:
    n_frames: int
    resample_p: float
    seed: int
    jitter: float = 0.0
    cut_every: int = 0      # > 0: every cut_every-th frame is a scene cut (all patches fresh)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: EncoderShape
    dtype: str                      # "f32" or "bf16": the arithmetic type of the CUDA path
    videos: Tuple[VideoSpec, ...]
    params: MergeParams
    weight_seed: int
    pos_std: float = 0.5

    @property
    def total_frames(self) -> int:
        return sum(v.n_frames for v in self.videos)

    @property
    def encoder_frames(self) -> int:
        """Frames as the encoder sees them (temporal patches): the unit of Stage I and of every frame index."""
        return self.total_frames // self.shape.temporal_patch

    def uncompressed(self) -> "Workload":
        p = replace(self.params, merge_layers=(), selection=0, retain=1.0)
        return replace(self, name=self.name + "_uncompressed", params=p)


TINY = EncoderShape(image_size=112, patch_size=14, num_layers=2, hidden=64, heads=4, mlp_dim=256)
SO400M = EncoderShape(image_size=384, patch_size=14, num_layers=27, hidden=1152, heads=16, mlp_dim=4304)

# Qwen2.5-VL's vision tower (public architecture): 32 blocks of width 1280, 16 heads of 80, gated MLP 3420, patches of
# 14 x 14 pixels over 2 frames, windows of 8 x 8 patches, full attention in blocks 7, 15, 23, 31
QWENVL = EncoderShape(image_size=224, patch_size=14, num_layers=32, hidden=1280, heads=16, mlp_dim=3420, arch=1,
                      temporal_patch=2, window=8, full_attn_layers=(7, 15, 23, 31))
QWENVL_TINY = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=64, heads=4, mlp_dim=100, arch=1,
                           temporal_patch=2, window=2, full_attn_layers=(1, 3))

MAIN = MergeParams()


def _serve_videos() -> Tuple[VideoSpec, ...]:
    out = []
    for s in range(8):
        p = float(np.random.Generator(np.random.Philox(key=1000 + s)).uniform(0.1, 0.6))
        out.append(VideoSpec(32, round(p, 4), s))
    return tuple(out)


WORKLOADS = {
    "tiny": Workload(
        "tiny", TINY, "f32", (VideoSpec(8, 0.3, 0),),
        MergeParams(merge_layers=(1,), selection=1, retain_mode=0, retain=0.5), 1234 + 1),
    "so400m_8f": Workload("so400m_8f", SO400M, "bf16", (VideoSpec(8, 0.3, 0),), MAIN, 1234 + 2),
    "so400m_32f": Workload("so400m_32f", SO400M, "bf16", (VideoSpec(32, 0.2, 0, jitter=0.05),), MAIN, 1234 + 2),
    # the same video with a scene cut every 6 frames: Stage I then leaves 22-24 of the 32 frames, close to the 73.9 %
    # frame retention the paper reports for Stage I alone; without cuts one long segment merges down to 11-13
    "so400m_32f_cal": Workload("so400m_32f_cal", SO400M, "bf16", (VideoSpec(32, 0.2, 0, jitter=0.05, cut_every=6),), MAIN, 1234 + 2),
    "so400m_64f_p10": Workload("so400m_64f_p10", SO400M, "bf16", (VideoSpec(64, 0.1, 0),), MAIN, 1234 + 2),
    "so400m_64f_p50": Workload("so400m_64f_p50", SO400M, "bf16", (VideoSpec(64, 0.5, 0),), MAIN, 1234 + 2),
    "so400m_64f_p90": Workload("so400m_64f_p90", SO400M, "bf16", (VideoSpec(64, 0.9, 0),), MAIN, 1234 + 2),
    "serve_8x32": Workload("serve_8x32", SO400M, "bf16", _serve_videos(), MAIN, 1234 + 2),
    # Qwen2.5-VL-style encoder (the paper's generalisation study): fp32 tiny case, 32 and 768 input frames of 224 x 224
    # (16 / 384 encoder frames of 256 tokens; 768 frames -> 24 576 tokens after a 2 x 2 merger, the paper's 23k context)
    "qwenvl_tiny": Workload("qwenvl_tiny", QWENVL_TINY, "f32", (VideoSpec(24, 0.1, 0),),
                            MergeParams(merge_layers=(1, 2), tau_seg=0.6, tau_merge=0.65, retain=0.4), 1234 + 5),
    "qwenvl_32f": Workload("qwenvl_32f", QWENVL, "bf16", (VideoSpec(32, 0.03, 0, jitter=0.05),),
                           MergeParams(retain=0.15), 1234 + 6),
    "qwenvl_768f": Workload("qwenvl_768f", QWENVL, "bf16", (VideoSpec(768, 0.03, 0, jitter=0.05, cut_every=48),),
                            MergeParams(retain=0.15), 1234 + 6),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name]
