"""Seeded random-init weight blobs in the library's documented order.

Blob order (all float32, row-major, a linear layer is y = x @ W + b with W [in, out]):

  patch_w [3*p*p, D]   (row index = c*p*p + dy*p + dx)
  patch_b [D]
  pos     [L, D]
  for each layer:  ln1_g [D], ln1_b [D], wqkv [D, 3D], bqkv [3D], wo [D, D], bo [D],
                   ln2_g [D], ln2_b [D], w1 [D, M], b1 [M], w2 [M, D], b2 [D]
  post_g [D], post_b [D]

wqkv's output columns are [Q | K | V], each D wide, head h at columns h*dh..(h+1)*dh of its third.

Qwen2.5-VL-style encoders (shape.arch == 1) have no position table, no patch bias and no norm shifts:

  patch_w [3*tp*p*p, D]   (row index = c*tp*p*p + t*p*p + dy*p + dx, tp = frames per temporal patch)
  for each layer:  n1_g [D], wqkv [D, 3D], bqkv [3D], wo [D, D], bo [D],
                   n2_g [D], wgu [D, 2M] (columns [gate | up]), bgu [2M], wd [M, D], bd [D]
  post_g [D]

Distributions: linear weights N(0, 1/fan_in) (attention logits come out O(1), so the
attention scores are well separated); the two residual-branch output projections are
additionally scaled by 1/sqrt(2*layers); biases N(0, 0.02^2); LayerNorm gains
1 + N(0, 0.1^2) and shifts N(0, 0.05^2) (non-trivial, so that a dropped gain or shift shows
up in parity); position embedding N(0, pos_std^2).
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def weight_layout(shape) -> List[Tuple[str, Tuple[int, ...], int]]:
    D, M, L, P = shape.hidden, shape.mlp_dim, shape.tokens_per_frame, shape.patch_dim
    if getattr(shape, "arch", 0) == 1:
        items = [("patch_w", (P, D))]
        for i in range(shape.num_layers):
            pre = f"l{i}."
            items += [(pre + "n1_g", (D,)), (pre + "wqkv", (D, 3 * D)), (pre + "bqkv", (3 * D,)),
                      (pre + "wo", (D, D)), (pre + "bo", (D,)), (pre + "n2_g", (D,)),
                      (pre + "wgu", (D, 2 * M)), (pre + "bgu", (2 * M,)), (pre + "wd", (M, D)), (pre + "bd", (D,))]
        items += [("post_g", (D,))]
        out, off = [], 0
        for name, shp in items:
            out.append((name, shp, off))
            off += int(np.prod(shp))
        return out
    items: List[Tuple[str, Tuple[int, ...]]] = [("patch_w", (P, D)), ("patch_b", (D,)), ("pos", (L, D))]
    for i in range(shape.num_layers):
        pre = f"l{i}."
        items += [(pre + "ln1_g", (D,)), (pre + "ln1_b", (D,)),
                  (pre + "wqkv", (D, 3 * D)), (pre + "bqkv", (3 * D,)),
                  (pre + "wo", (D, D)), (pre + "bo", (D,)),
                  (pre + "ln2_g", (D,)), (pre + "ln2_b", (D,)),
                  (pre + "w1", (D, M)), (pre + "b1", (M,)),
                  (pre + "w2", (M, D)), (pre + "b2", (D,))]
    items += [("post_g", (D,)), ("post_b", (D,))]
    out, off = [], 0
    for name, shp in items:
        out.append((name, shp, off))
        off += int(np.prod(shp))
    return out


def blob_size(shape) -> int:
    name, shp, off = weight_layout(shape)[-1]
    return off + int(np.prod(shp))


def make_weights(shape, seed: int, pos_std: float = 0.5) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[seed, 7]))
    blob = np.empty(blob_size(shape), dtype=np.float32)
    branch_scale = 1.0 / np.sqrt(2.0 * shape.num_layers)
    for name, shp, off in weight_layout(shape):
        n = int(np.prod(shp))
        leaf = name.split(".")[-1]
        z = rng.standard_normal(n, dtype=np.float32)
        if leaf in ("patch_w", "wqkv", "wo", "w1", "w2", "wgu", "wd"):
            std = 1.0 / np.sqrt(shp[0])
            if leaf in ("wo", "w2", "wd"):
                std *= branch_scale
            z *= np.float32(std)
        elif leaf == "pos":
            z *= np.float32(pos_std)
        elif leaf.endswith("_g"):
            z = np.float32(1.0) + np.float32(0.1) * z
        elif leaf in ("ln1_b", "ln2_b", "post_b"):
            z *= np.float32(0.05)
        else:  # linear biases
            z *= np.float32(0.02)
        blob[off:off + n] = z
    return blob


def views(shape, blob: np.ndarray) -> dict:
    """Name -> ndarray view into the blob (no copy)."""
    return {name: blob[off:off + int(np.prod(shp))].reshape(shp) for name, shp, off in weight_layout(shape)}
