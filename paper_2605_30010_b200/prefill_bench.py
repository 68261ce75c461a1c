"""Times the projector + language-model prefill stage alone, per kernel category, on random-init weights drawn on the
device (Qwen2-7B widths by default; --layers / --vocab shrink the model so that a profiler capture stays small).

    python -m paper_2605_30010_b200.prefill_bench [--layers 28] [--vocab 152064] [--visual-tokens 7621] [--iters 5]

Prints one JSON line: ms per prefill, ms per category, TFLOP/s of the dense layers and of the attention kernel
(causal: half of the n^2 products are counted), GB/s of the bandwidth kernels.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
from dataclasses import replace

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=28)
    ap.add_argument("--vocab", type=int, default=152064)
    ap.add_argument("--visual-tokens", type=int, default=7621)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    args = ap.parse_args()

    import torch
    from paper_2605_30010_b200 import binding as B
    from synthetic.llm import QWEN2_7B, make_llm_weights_device, make_prompt, make_visual_tokens

    shape = replace(QWEN2_7B, num_layers=args.layers, vocab=args.vocab)
    blob = make_llm_weights_device(shape, 5)
    llm = B.LanguageModel(shape, blob, max_tokens=args.visual_tokens + 64, keep_kv_cache=True)
    del blob
    torch.cuda.empty_cache()
    pre, suf = make_prompt(shape, 14, 40, 6)
    vis = torch.from_numpy(make_visual_tokens(shape, args.visual_tokens, 6)).cuda()
    for _ in range(args.warmup):
        B.et_llm_prefill(llm, pre, vis, suf, copy_logits=False)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.iters):
        r = B.et_llm_prefill(llm, pre, vis, suf, copy_logits=False)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.iters
    B.et_llm_profile_enable(llm, True)
    for _ in range(args.iters):
        B.et_llm_prefill(llm, pre, vis, suf, copy_logits=False)
    p = B.et_llm_profile_read(llm)
    llm.close()

    n, calls = r.n_tokens, p["calls"]
    H, M, L = shape.hidden, shape.mlp_dim, shape.num_layers
    per = {k: v / calls for k, v in p["ms"].items()}
    gemm_flops = L * 2.0 * n * (H * shape.qkv_dim + shape.q_dim * H + 3 * H * M) \
        + 2.0 * args.visual_tokens * (shape.vision_hidden * H + H * H) + 2.0 * H * shape.vocab
    attn_flops = L * 2.0 * n * n * shape.q_dim
    norm_bytes = 2 * L * n * H * (4 + 2)                      # fp32 row in, bf16 row out
    rope_bytes = L * n * (shape.q_dim + shape.kv_dim) * 2 * 2   # Q and K parts read and written
    out = {"tokens": n, "layers": L, "vocab": shape.vocab, "ms_per_prefill": round(ms, 3), "tokens_per_s": round(n / (ms * 1e-3), 1),
           "ms_per_category": {k: round(v, 4) for k, v in per.items()},
           "launches_per_prefill": {k: v // calls for k, v in p["launches"].items()},
           "gemm_tflops": round(gemm_flops / (per["gemm"] * 1e-3) / 1e12, 1),
           "attention_tflops": round(attn_flops / (per["attention"] * 1e-3) / 1e12, 1),
           "rmsnorm_gbs": round(norm_bytes / (per["norm"] * 1e-3) / 1e9, 1),
           "rope_gbs": round(rope_bytes / (per["rope"] * 1e-3) / 1e9, 1)}
    print(json.dumps(out))


if __name__ == "__main__":
    main()
