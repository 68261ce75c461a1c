"""GPU parity of the stage downstream of the encoder (projector + language-model prefill) against the
numpy oracle, through the C ABI: every step kernel on its own, then the whole prefill on two small models,
on one decoder layer at the full Qwen2-7B width, and properties of the full 28-layer model.

Tolerances: the step kernels read bf16 inputs (the oracle gets the same rounded values) and write bf16, so
they are held to a few bf16 ulps; the whole path to the bf16 bound of the encoder tests, max over tokens of
||gpu - oracle||_inf / ||oracle||_inf <= 2e-2."""
import numpy as np
import pytest

from oracle import prefill_oracle as P
from synthetic.llm import (LLM_ODD, LLM_SMALL, LLM_TINY, QWEN2_7B, QWEN2_7B_1L, LlmShape, make_llm_weights, make_llm_weights_device,
                           make_prompt, make_visual_tokens)
from tests import helpers as H

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2
BF16_ULP = 2.0 ** -8


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2605_30010_b200 import binding
    return binding


def _bf16(a: np.ndarray):
    """(torch bf16 CUDA tensor, the same values as float64 numpy)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)
    return t, t.float().cpu().numpy().astype(np.float64)


def _close_bf16(got, ref, ulps=2.0, atol=1e-6):
    got = got.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    bound = ulps * BF16_ULP * np.abs(ref) + atol
    assert (err <= bound).all(), f"max excess {(err - bound).max():.3e} at {np.unravel_index(np.argmax(err - bound), err.shape)}"


@pytest.mark.parametrize("rows,D", [(1, 3584), (300, 3584), (37, 256), (129, 100), (5, 4096), (64, 1152)])
def test_rmsnorm(B, rows, D):
    import torch
    rng = np.random.default_rng(rows * 7 + D)
    x = (rng.standard_normal((rows, D)) * rng.uniform(0.1, 5.0, size=(rows, 1))).astype(np.float32)
    g = (1.0 + 0.1 * rng.standard_normal(D)).astype(np.float32)
    y = B.et_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda(), 1e-6)
    _close_bf16(y, P.rms_norm(x.astype(np.float64), g.astype(np.float64), 1e-6), ulps=1.25)


@pytest.mark.parametrize("rows,L,heads,kv,dh,theta", [(300, 300, 4, 2, 128, 1e6), (300, 150, 3, 1, 128, 1e4),
                                                      (9000, 9000, 1, 1, 128, 1e6), (70, 70, 2, 2, 64, 1e4), (33, 33, 1, 1, 16, 50.0)])
def test_rope(B, rows, L, heads, kv, dh, theta):
    rng = np.random.default_rng(rows + heads)
    width = (heads + 2 * kv) * dh
    t, ref_in = _bf16(rng.standard_normal((rows, width)))
    B.et_rope(t, L, heads, kv, dh, theta)
    pos = np.arange(rows) % L
    ref = ref_in.copy()
    qk = ref_in[:, :(heads + kv) * dh].reshape(rows, heads + kv, dh)
    ref[:, :(heads + kv) * dh] = P.rope(qk, pos, theta).reshape(rows, -1)
    # a rotated element is a sum of two products: bound by ulps of the pair's magnitude
    got = t.float().cpu().numpy().astype(np.float64)
    mag = np.abs(ref_in[:, :(heads + kv) * dh].reshape(rows, heads + kv, 2, dh // 2)).max(axis=2, keepdims=True)
    bound = np.broadcast_to(1.5 * BF16_ULP * mag * 1.5 + 1e-6, (rows, heads + kv, 2, dh // 2)).reshape(rows, -1)
    err = np.abs(got - ref)
    assert (err[:, :(heads + kv) * dh] <= bound).all(), f"rope error {err.max():.3e}"
    np.testing.assert_array_equal(got[:, (heads + kv) * dh:], ref_in[:, (heads + kv) * dh:])     # V untouched


@pytest.mark.parametrize("rows,M", [(1, 8), (77, 1408), (300, 18944)])
def test_swiglu(B, rows, M):
    rng = np.random.default_rng(M)
    t, ref_in = _bf16(rng.standard_normal((rows, 2 * M)) * 3.0)
    h = B.et_swiglu(t)
    _close_bf16(h, P.silu(ref_in[:, :M]) * ref_in[:, M:], ulps=1.5)


@pytest.mark.parametrize("rows,K,M", [(300, 256, 128), (1000, 512, 1408), (77, 64, 256)])
def test_gated_dense_layer(B, rows, K, M):
    """Dense layer with the SwiGLU epilogue: weight rows and bias in the interleaved order, output
    silu(gate + b_gate) * (up + b_up)."""
    import torch
    rng = np.random.default_rng(K + M)
    a, a_ref = _bf16(rng.standard_normal((rows, K)))
    wg, wg_ref = _bf16(rng.standard_normal((M, K)) / np.sqrt(K))        # [out][in]
    wu, wu_ref = _bf16(rng.standard_normal((M, K)) / np.sqrt(K))
    j = np.arange(M)
    row_gate = (j >> 7) * 256 + ((j & 127) >> 5) * 64 + (j & 31)
    w = torch.empty((2 * M, K), dtype=torch.bfloat16, device="cuda")
    w[torch.from_numpy(row_gate).cuda()] = wg
    w[torch.from_numpy(row_gate + 32).cuda()] = wu
    bg, bu = (0.3 * rng.standard_normal(M)).astype(np.float32), (0.3 * rng.standard_normal(M)).astype(np.float32)
    bias = torch.zeros(2 * M, dtype=torch.float32, device="cuda")
    bias[torch.from_numpy(row_gate).cuda()] = torch.from_numpy(bg).cuda()
    bias[torch.from_numpy(row_gate + 32).cuda()] = torch.from_numpy(bu).cuda()
    h, status = B.et_linear_bf16(a, w, bias, epilogue=4)
    assert int(status.item()) == 0 and tuple(h.shape) == (rows, M)
    ref = P.silu(a_ref @ wg_ref.T + bg) * (a_ref @ wu_ref.T + bu)
    got = h.float().cpu().numpy().astype(np.float64)
    assert np.abs(got - ref).max() <= 1.5 * BF16_ULP * np.abs(ref).max() + 1e-5, f"error {np.abs(got - ref).max():.3e}"
    err = np.abs(got - ref)
    assert (err <= 2 * BF16_ULP * np.abs(ref) + 2e-3).all()


@pytest.mark.parametrize("n_seq,L,heads,kv", [(1, 1, 1, 1), (1, 100, 2, 1), (1, 128, 1, 1), (1, 129, 2, 2), (1, 300, 4, 2),
                                              (2, 257, 2, 2), (1, 777, 4, 1), (3, 64, 7, 1), (1, 1500, 2, 1)])
def test_attention_causal(B, n_seq, L, heads, kv):
    rng = np.random.default_rng(L * 3 + heads)
    dh = 128
    width = (heads + 2 * kv) * dh
    t, ref_in = _bf16(rng.standard_normal((n_seq * L, width)) * 1.5)
    out, status = B.et_attention_causal(t, n_seq, L, heads, kv, dh)
    assert int(status.item()) == 0
    got = out.float().cpu().numpy()
    for s in range(n_seq):
        rows = ref_in[s * L:(s + 1) * L]
        q = rows[:, :heads * dh].reshape(L, heads, dh)
        k = rows[:, heads * dh:(heads + kv) * dh].reshape(L, kv, dh)
        v = rows[:, (heads + kv) * dh:].reshape(L, kv, dh)
        ref = P.causal_gqa_attention(q, k, v).reshape(L, heads * dh)
        err = H.token_error(got[s * L:(s + 1) * L].reshape(L * heads, dh), ref.reshape(L * heads, dh))
        assert err <= BF16_TOL, f"sequence {s}: attention error {err:.3e}"


def _run_prefill(B, shape, blob, n_prefix, n_vis, n_suffix, seed, dtype):
    import torch
    pre, suf = make_prompt(shape, n_prefix, n_suffix, seed)
    vis = make_visual_tokens(shape, n_vis, seed)
    llm = B.LanguageModel(shape, blob, max_tokens=n_prefix + n_vis + n_suffix)
    try:
        r = llm.prefill(pre, torch.from_numpy(vis).cuda() if n_vis else None, suf, want_hidden=True)
        r2 = llm.prefill(pre, torch.from_numpy(vis).cuda() if n_vis else None, suf, want_hidden=True)
    finally:
        llm.close()
    w = P.split_llm_weights(shape, blob)
    ref = P.prefill(shape, w, pre, vis, suf, dtype=dtype, want_hidden=True)
    return r, r2, ref


def _check_prefill(r, r2, ref):
    import torch
    assert r.n_tokens == ref["n_tokens"]
    assert torch.equal(r.hidden, r2.hidden) and torch.equal(r.logits, r2.logits), "two runs of the same call must agree bit for bit"
    err = H.token_error(r.hidden.cpu().numpy(), ref["hidden"])
    assert err <= BF16_TOL, f"hidden-state error {err:.3e}"
    lg, lo = r.logits.cpu().numpy().astype(np.float64), ref["logits"].astype(np.float64)
    lerr = np.abs(lg - lo).max() / np.abs(lo).max()
    assert lerr <= BF16_TOL, f"logit error {lerr:.3e}"
    assert r.first_token == int(np.argmax(lg)), "first token is the argmax of the library's own logits"
    top2 = np.sort(lo)[-2:]
    if (top2[1] - top2[0]) > 2 * BF16_TOL * np.abs(lo).max():        # otherwise a near-tie: either id is acceptable
        assert r.first_token == ref["first_token"]
    return err, lerr


@pytest.mark.parametrize("shape,n_prefix,n_vis,n_suffix", [(LLM_TINY, 5, 300, 9), (LLM_TINY, 0, 130, 0), (LLM_TINY, 3, 0, 4),
                                                           (LLM_SMALL, 14, 500, 21), (LLM_SMALL, 1, 255, 0),
                                                           (LLM_ODD, 7, 290, 3), (LLM_ODD, 1, 0, 0), (LLM_TINY, 0, 256, 0)])
def test_prefill_small_models(B, shape, n_prefix, n_vis, n_suffix):
    blob = make_llm_weights(shape, 3)
    r, r2, ref = _run_prefill(B, shape, blob, n_prefix, n_vis, n_suffix, 1, np.float64)
    err, lerr = _check_prefill(r, r2, ref)
    print(f"{shape.hidden}x{shape.num_layers}: n = {r.n_tokens}, hidden error {err:.2e}, logit error {lerr:.2e}")


def test_prefill_one_layer_at_full_width(B):
    """One decoder layer with the widths of the 7B model (3584 / 28 heads / 4 key-value heads / 18944), several
    row tiles and a ragged tail, against the fp32 oracle."""
    shape = QWEN2_7B_1L
    blob = make_llm_weights(shape, 4)
    r, r2, ref = _run_prefill(B, shape, blob, 14, 650, 31, 2, np.float32)
    err, lerr = _check_prefill(r, r2, ref)
    print(f"full width, one layer: n = {r.n_tokens}, hidden error {err:.2e}, logit error {lerr:.2e}")


def test_kv_cache(B):
    """Keys (after the rotary embedding) and values of every layer, as kept for decoding, against the oracle's."""
    import torch
    shape = LLM_SMALL
    blob = make_llm_weights(shape, 3)
    pre, suf = make_prompt(shape, 6, 11, 4)
    vis = make_visual_tokens(shape, 300, 4)
    llm = B.LanguageModel(shape, blob, max_tokens=400, keep_kv_cache=True)
    plain = B.LanguageModel(shape, blob, max_tokens=400)
    try:
        r = llm.prefill(pre, torch.from_numpy(vis).cuda(), suf, want_hidden=True, want_kv=True)
        r0 = plain.prefill(pre, torch.from_numpy(vis).cuda(), suf, want_hidden=True)
        with pytest.raises(B.EarlyTomError):
            plain.prefill(pre, torch.from_numpy(vis).cuda(), suf, want_kv=True)
    finally:
        llm.close(); plain.close()
    assert torch.equal(r.hidden, r0.hidden), "keeping the cache must not change the result"
    ref = P.prefill(shape, P.split_llm_weights(shape, blob), pre, vis, suf, want_kv=True)
    n, kvd = r.n_tokens, shape.kv_heads * shape.head_dim
    assert tuple(r.kv_cache.shape) == (shape.num_layers, n, 2 * kvd)
    got = r.kv_cache.float().cpu().numpy()
    for layer, (k, v) in enumerate(ref["kv"]):
        ek = H.token_error(got[layer, :, :kvd], k.reshape(n, kvd))
        ev = H.token_error(got[layer, :, kvd:], v.reshape(n, kvd))
        assert ek <= BF16_TOL and ev <= BF16_TOL, f"layer {layer}: key error {ek:.3e}, value error {ev:.3e}"


def test_errors(B):
    import torch
    shape = LLM_TINY
    blob = make_llm_weights(shape, 3)
    with pytest.raises(B.EarlyTomError) as ei:
        B.LanguageModel(shape, blob[:-1], max_tokens=16)
    assert ei.value.status == 7
    bad = LlmShape(vision_hidden=64, hidden=256, num_layers=1, heads=2, kv_heads=1, head_dim=64, mlp_dim=512, vocab=512)
    with pytest.raises(B.EarlyTomError) as ei:
        B.LanguageModel(bad, make_llm_weights(bad, 0), max_tokens=16)
    assert ei.value.status == 2
    llm = B.LanguageModel(shape, blob, max_tokens=16)
    try:
        with pytest.raises(B.EarlyTomError) as ei:
            llm.prefill(np.arange(17), None, [])
        assert ei.value.status == 3
        with pytest.raises(B.EarlyTomError) as ei:
            llm.prefill([], None, [])
        assert ei.value.status == 1
        with pytest.raises(B.EarlyTomError) as ei:
            llm.prefill([shape.vocab], None, [])
        assert ei.value.status == 1
        ok = llm.prefill([1, 2, 3], torch.zeros((4, shape.vision_hidden), device="cuda"), [4])
        assert ok.n_tokens == 8
    finally:
        llm.close()


def test_full_model_properties(B):
    """The 28-layer model at the benchmark's sequence length (weights drawn on the device): finite logits, the
    first token is their argmax, and causality -- the hidden states of a prefix do not depend on what follows."""
    import torch
    shape = QWEN2_7B
    blob = make_llm_weights_device(shape, 5)
    n_vis = 7621
    llm = B.LanguageModel(shape, blob, max_tokens=8192)
    del blob
    torch.cuda.empty_cache()
    try:
        pre, suf = make_prompt(shape, 14, 40, 6)
        vis = torch.from_numpy(make_visual_tokens(shape, n_vis, 6)).cuda()
        full = llm.prefill(pre, vis, suf, want_hidden=True)
        assert full.n_tokens == 14 + n_vis + 40
        assert bool(torch.isfinite(full.logits).all()) and bool(torch.isfinite(full.hidden).all())
        assert full.first_token == int(torch.argmax(full.logits).item())
        cut = llm.prefill(pre, vis[:3000], [], want_hidden=True)
        a, b = full.hidden[:3014].cpu().numpy(), cut.hidden.cpu().numpy()
        err = H.token_error(a, b)
        assert err <= 1e-2, f"prefix rows changed with the suffix: {err:.3e}"
        assert float(full.hidden.abs().max()) < 1e4
    finally:
        llm.close()
