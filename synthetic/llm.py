"""Shapes, workloads and seeded random-init weight blobs of the stage downstream of the encoder:
the projector and the language model's prefill (shapes and random numbers only, no arithmetic).

Blob order (all float32, row-major, a linear layer is y = x @ W + b with W [in, out]):

  embed   [vocab, hidden]
  proj_w1 [vision_hidden, hidden], proj_b1 [hidden], proj_w2 [hidden, hidden], proj_b2 [hidden]
  for each layer:  rms1_g [hidden],
                   wqkv [hidden, (heads + 2*kv_heads)*head_dim], bqkv [(heads + 2*kv_heads)*head_dim],
                   wo [heads*head_dim, hidden],
                   rms2_g [hidden], wgu [hidden, 2*mlp_dim]  (gate columns first, then up), wd [mlp_dim, hidden]
  final_g [hidden]
  lm_head [hidden, vocab]

wqkv's output columns are [Q | K | V]: heads*head_dim, then kv_heads*head_dim twice; query head h
uses key / value head h // (heads // kv_heads).

Distributions: embedding rows N(0, 1); linear weights N(0, 1/fan_in), the two residual-branch output
projections additionally scaled by 1/sqrt(2*layers); biases N(0, 0.02^2); RMSNorm gains 1 + N(0, 0.1^2).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np


@dataclass(frozen=True)
class LlmShape:
    vision_hidden: int
    hidden: int
    num_layers: int
    heads: int
    kv_heads: int
    head_dim: int
    mlp_dim: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    gelu_tanh: int = 1

    @property
    def q_dim(self) -> int:
        return self.heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.kv_heads * self.head_dim

    @property
    def qkv_dim(self) -> int:
        return self.q_dim + 2 * self.kv_dim


# LLaVA-OneVision-7B's language model (Qwen2-7B shapes) behind a two-layer GELU projector.
QWEN2_7B = LlmShape(vision_hidden=1152, hidden=3584, num_layers=28, heads=28, kv_heads=4, head_dim=128,
                    mlp_dim=18944, vocab=152064)
# One layer at the full width and a small vocabulary: what the CPU oracle can follow in seconds.
QWEN2_7B_1L = LlmShape(vision_hidden=1152, hidden=3584, num_layers=1, heads=28, kv_heads=4, head_dim=128,
                       mlp_dim=18944, vocab=1024)
LLM_TINY = LlmShape(vision_hidden=64, hidden=256, num_layers=2, heads=2, kv_heads=1, head_dim=128, mlp_dim=512,
                    vocab=512, rope_theta=1e4)
# mlp_dim not a multiple of 128 (the feed-forward gating runs as a kernel of its own) and as many key / value heads as
# query heads (plain multi-head attention)
LLM_ODD = LlmShape(vision_hidden=72, hidden=384, num_layers=2, heads=3, kv_heads=3, head_dim=128, mlp_dim=328, vocab=264,
                   rope_theta=5e5, gelu_tanh=0)
LLM_SMALL = LlmShape(vision_hidden=1152, hidden=512, num_layers=3, heads=4, kv_heads=2, head_dim=128, mlp_dim=1408,
                     vocab=1000)


def llm_weight_layout(shape: LlmShape) -> List[Tuple[str, Tuple[int, ...], int]]:
    H, V, M = shape.hidden, shape.vocab, shape.mlp_dim
    items: List[Tuple[str, Tuple[int, ...]]] = [
        ("embed", (V, H)), ("proj_w1", (shape.vision_hidden, H)), ("proj_b1", (H,)), ("proj_w2", (H, H)), ("proj_b2", (H,))]
    for i in range(shape.num_layers):
        pre = f"l{i}."
        items += [(pre + "rms1_g", (H,)), (pre + "wqkv", (H, shape.qkv_dim)), (pre + "bqkv", (shape.qkv_dim,)),
                  (pre + "wo", (shape.q_dim, H)), (pre + "rms2_g", (H,)), (pre + "wgu", (H, 2 * M)), (pre + "wd", (M, H))]
    items += [("final_g", (H,)), ("lm_head", (H, V))]
    out, off = [], 0
    for name, shp in items:
        out.append((name, shp, off))
        off += int(np.prod(shp))
    return out


def llm_blob_size(shape: LlmShape) -> int:
    name, shp, off = llm_weight_layout(shape)[-1]
    return off + int(np.prod(shp))


def _std(leaf: str, shp, num_layers: int) -> float:
    if leaf == "embed":
        return 1.0
    if leaf in ("proj_w1", "proj_w2", "wqkv", "wgu", "lm_head"):
        return 1.0 / float(np.sqrt(shp[0]))
    if leaf in ("wo", "wd"):
        return 1.0 / float(np.sqrt(shp[0])) / float(np.sqrt(2.0 * num_layers))
    return 0.02          # linear biases


def make_llm_weights(shape: LlmShape, seed: int) -> np.ndarray:
    """Host blob (numpy, Philox): the one the oracle and the library both read in the parity tests."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 11]))
    blob = np.empty(llm_blob_size(shape), dtype=np.float32)
    for name, shp, off in llm_weight_layout(shape):
        n = int(np.prod(shp))
        leaf = name.split(".")[-1]
        z = rng.standard_normal(n, dtype=np.float32)
        if leaf.endswith("_g"):
            z = np.float32(1.0) + np.float32(0.1) * z
        else:
            z *= np.float32(_std(leaf, shp, shape.num_layers))
        blob[off:off + n] = z
    return blob


def make_llm_weights_device(shape: LlmShape, seed: int, device="cuda"):
    """The same layout and distributions drawn on the GPU (torch generator): for sizes whose blob is too
    large to draw and copy from the host in benchmark time.  Not bit-identical to ``make_llm_weights``."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    blob = torch.empty(llm_blob_size(shape), dtype=torch.float32, device=device)
    for name, shp, off in llm_weight_layout(shape):
        n = int(np.prod(shp))
        leaf = name.split(".")[-1]
        view = blob[off:off + n]
        view.normal_(0.0, 1.0, generator=gen)
        if leaf.endswith("_g"):
            view.mul_(0.1).add_(1.0)
        else:
            view.mul_(_std(leaf, shp, shape.num_layers))
    return blob


def llm_views(shape: LlmShape, blob: np.ndarray) -> dict:
    return {name: blob[off:off + int(np.prod(shp))].reshape(shp) for name, shp, off in llm_weight_layout(shape)}


def make_prompt(shape: LlmShape, n_prefix: int, n_suffix: int, seed: int):
    """Token ids of the text before and after the visual tokens (uniform over the vocabulary)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 13]))
    return (rng.integers(0, shape.vocab, size=n_prefix, dtype=np.int32),
            rng.integers(0, shape.vocab, size=n_suffix, dtype=np.int32))


def make_visual_tokens(shape: LlmShape, n_vis: int, seed: int) -> np.ndarray:
    """Stand-in for the encoder's output rows (post-LayerNorm features are O(1) per element)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 17]))
    return rng.standard_normal((n_vis, shape.vision_hidden), dtype=np.float32)
