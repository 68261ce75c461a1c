"""Per-kernel parity: every single-step entry point of the C ABI against the oracle (needs a B200)."""
import math

import numpy as np
import pytest

from oracle import earlytom_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2605_30010_b200 import binding
    return binding


def cuda(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


# ------------------------------------------------------------------ Stage I

@pytest.mark.parametrize("n,L,D", [(8, 64, 64), (5, 37, 100), (2, 16, 8), (11, 729, 1152), (3, 50, 2048)])
def test_frame_similarity(B, n, L, D):
    rng = np.random.default_rng(n * 1000 + L)
    base = rng.standard_normal((L, D)).astype(np.float32)
    x = np.stack([base + rng.uniform(0.1, 1.5) * rng.standard_normal((L, D)).astype(np.float32) for _ in range(n)])
    x[0, 3] = 0.0                                   # a zero-norm token: contributes 0
    sim, cosb = B.et_frame_similarity(cuda(x))
    ref = O.frame_similarity(x)
    np.testing.assert_allclose(sim.cpu().numpy(), ref, atol=2e-6)
    assert cosb[0, 3].item() == 0.0
    sim2, _ = B.et_frame_similarity(cuda(x))
    assert (sim2 == sim).all(), "fixed-order reductions must be bit-reproducible"


def test_frame_similarity_single_frame(B):
    sim, _ = B.et_frame_similarity(cuda(np.ones((1, 4, 8), dtype=np.float32)))
    assert sim.numel() == 0


def oracle_plan(sim64, offs, alpha, tau_seg, tau_merge, weighted):
    starts, mws, emas, src_a, src_b, w_a, w_b, new_off = [], [], [], [], [], [], [], [0]
    for v in range(len(offs) - 1):
        g0, g1 = offs[v], offs[v + 1]
        c = sim64[g0:g1 - 1]
        st, ema = O.segment_by_similarity(c, g1 - g0, alpha, tau_seg)
        mw = O.merge_pairs(c, O.segments_from_starts(st), tau_merge)
        ema[0] = 0.0
        starts.append(st); mws.append(mw); emas.append(ema)
        t = 0
        while t < g1 - g0:
            if mw[t]:
                dummy = np.zeros((1, 1))
                _, wa, wb = O.weighted_merge(dummy, dummy, float(c[t]), float(c[t + 1]), bool(weighted))
                src_a.append(g0 + t); src_b.append(g0 + t + 1); w_a.append(wa); w_b.append(wb)
                t += 2
            else:
                src_a.append(g0 + t); src_b.append(-1); w_a.append(1.0); w_b.append(0.0)
                t += 1
        new_off.append(len(src_a))
    return (np.concatenate(starts), np.concatenate(mws), np.concatenate(emas), np.array(src_a), np.array(src_b),
            np.array(w_a), np.array(w_b), np.array(new_off))


@pytest.mark.parametrize("seed", range(8))
def test_merge_plan_matches_oracle(B, seed):
    rng = np.random.default_rng(seed)
    V = int(rng.integers(1, 6))
    lens = rng.integers(1, 40, V)
    if seed == 6:                       # more videos than lanes, single-frame videos among them
        V, lens = 70, rng.integers(1, 6, 70)
    if seed == 7:                       # a list longer than the shared-memory staging area of the plan
        V, lens = 3, np.array([1500, 1, 1700])
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n = int(offs[-1])
    sim = rng.uniform(0.5, 1.0, n).astype(np.float32)
    if seed % 2:
        sim = np.round(sim * 8) / 8            # exact ties between neighbours and with the thresholds
    alpha, tau_seg, tau_merge = [(0.9, 0.7, 0.75), (1.0, 0.75, 0.625), (0.5, 0.8, 0.6)][seed % 3]
    for weighted in (1, 0):
        o = B.et_merge_plan(cuda(sim), cuda(offs), alpha, tau_seg, tau_merge, weighted)
        st, mw, ema, sa, sb, wa, wb, noff = oracle_plan(sim.astype(np.float64), offs, alpha, tau_seg, tau_merge, weighted)
        n_out = int(o["n_out"].item())
        assert n_out == len(sa)
        np.testing.assert_array_equal(o["seg_start"].cpu().numpy().astype(bool), st)
        np.testing.assert_array_equal(o["merge_next"].cpu().numpy().astype(bool), mw)
        np.testing.assert_allclose(o["ema"].cpu().numpy(), ema, atol=1e-6)
        np.testing.assert_array_equal(o["src_a"].cpu().numpy()[:n_out], sa)
        np.testing.assert_array_equal(o["src_b"].cpu().numpy()[:n_out], sb)
        np.testing.assert_allclose(o["w_a"].cpu().numpy()[:n_out], wa, atol=1e-6)
        np.testing.assert_allclose(o["w_b"].cpu().numpy()[:n_out], wb, atol=1e-6)
        np.testing.assert_array_equal(o["new_video_offsets"].cpu().numpy(), noff)


def test_merge_frames_matches_eq3(B):
    import torch
    rng = np.random.default_rng(3)
    n, L, D = 9, 33, 20
    x = rng.standard_normal((n, L, D)).astype(np.float32)
    sim = np.array([0.9, 0.85, 0.8, 0.7, 0.95, 0.9, 0.6, 0.5, 0.0], dtype=np.float32)
    offs = np.array([0, n], dtype=np.int32)
    plan = B.et_merge_plan(cuda(sim), cuda(offs), 0.9, 0.1, 0.3)
    y = B.et_merge_frames(cuda(x), plan).cpu().numpy()
    n_out = int(plan["n_out"].item())
    assert n_out < n
    sa, sb = plan["src_a"].cpu().numpy(), plan["src_b"].cpu().numpy()
    for j in range(n_out):
        if sb[j] < 0:
            np.testing.assert_array_equal(y[j], x[sa[j]])
        else:
            ref, _, _ = O.weighted_merge(x[sa[j]].astype(np.float64), x[sb[j]].astype(np.float64),
                                         float(sim[sa[j]]), float(sim[sb[j]]), True)
            np.testing.assert_allclose(y[j], ref, rtol=1e-6, atol=1e-6)


# ------------------------------------------------------------------ Stage II

@pytest.mark.parametrize("window_mode", [0, 1])
@pytest.mark.parametrize("N,L", [(6, 64), (3, 729), (4, 17), (1, 1), (40, 729)])
def test_select_tokens_exact(B, N, L, window_mode):
    rng = np.random.default_rng(N * 100 + L)
    a = rng.random((N, L)).astype(np.float32)
    a[:, ::3] = np.round(a[:, ::3] * 4) / 4          # exact ties
    dyn = (rng.random(N) < 0.5).astype(np.uint8)
    dyn[0] = 1
    k = rng.integers(1, L + 1, N).astype(np.int32)
    if N > 2:
        k[1], k[2] = L, 1                            # the extremes: keep everything / one token
    w = np.maximum(1, L // k).astype(np.int32)
    keep, count = B.et_select_tokens(cuda(a), cuda(dyn), cuda(k), cuda(w), window_mode)
    keep = keep.cpu().numpy().astype(bool)
    for f in range(N):
        ref = O.topk_mask(a[f], int(k[f])) if dyn[f] else O.window_mask(a[f], int(w[f]), int(k[f]), window_mode)
        np.testing.assert_array_equal(keep[f], ref)
        assert int(count[f].item()) == ref.sum()


def test_select_tokens_degenerate_inputs(B):
    """Out-of-range amounts are clamped to [1, L]; a NaN score ranks below every number, so the kept count never
    exceeds k and count[] always equals the bytes set in the mask (what the gather's offsets rely on)."""
    L = 50
    rng = np.random.default_rng(0)
    a = rng.random((4, L)).astype(np.float32)
    a[0, [3, 7, 20]] = np.nan
    a[1, :] = np.nan
    dyn = np.array([1, 1, 0, 0], dtype=np.uint8)
    k = np.array([10, 5, 0, 99], dtype=np.int32)
    w = np.array([5, 10, 0, -3], dtype=np.int32)
    for mode in (0, 1):
        keep, count = B.et_select_tokens(cuda(a), cuda(dyn), cuda(k), cuda(w), mode)
        keep = keep.cpu().numpy().astype(bool)
        np.testing.assert_array_equal(keep.sum(axis=1), count.cpu().numpy())
        finite = np.where(np.isnan(a[0]), -np.inf, a[0])
        np.testing.assert_array_equal(keep[0], O.topk_mask(finite, 10))
        assert not keep[0, [3, 7, 20]].any()
        assert np.nonzero(keep[1])[0].tolist() == [0, 1, 2, 3, 4]     # all equal: lowest indices
        assert count[2].item() == (1 if mode == 1 else L)              # k = 0 -> 1 ; w = 0 -> 1
        assert count[3].item() == L                                    # k = 99 -> L ; w < 1 -> 1


@pytest.mark.parametrize("N,L,D,ln", [(5, 64, 64, True), (3, 729, 1152, True), (4, 30, 12, False), (2, 100, 2048, True)])
def test_gather_tokens(B, N, L, D, ln):
    rng = np.random.default_rng(L)
    x = rng.standard_normal((N, L, D)).astype(np.float32)
    keep = rng.random((N, L)) < 0.3
    keep[1] = False                                  # a frame that keeps nothing
    if N > 2:
        keep[2] = True                               # a frame that keeps everything
    g = (1 + 0.1 * rng.standard_normal(D)).astype(np.float32)
    b = (0.1 * rng.standard_normal(D)).astype(np.float32)
    toks, offs, pos = B.et_gather_tokens(cuda(x), cuda(keep.astype(np.uint8)), cuda(g) if ln else None,
                                         cuda(b) if ln else None, 1e-6)
    counts = keep.sum(axis=1)
    np.testing.assert_array_equal(offs.cpu().numpy(), np.concatenate([[0], np.cumsum(counts)]))
    ref_pos = np.concatenate([np.nonzero(keep[f])[0] for f in range(N)])
    np.testing.assert_array_equal(pos.cpu().numpy(), ref_pos)
    rows = np.concatenate([x[f][keep[f]] for f in range(N)]).astype(np.float64)
    ref = O.layer_norm(rows, g.astype(np.float64), b.astype(np.float64), 1e-6) if ln else rows
    np.testing.assert_allclose(toks.cpu().numpy(), ref, rtol=2e-5, atol=2e-5)


def test_gather_capacity_error(B):
    x = np.zeros((2, 8, 8), dtype=np.float32)
    keep = np.ones((2, 8), dtype=np.uint8)
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_gather_tokens(cuda(x), cuda(keep), capacity_rows=3)
    assert ei.value.status == 3


# ------------------------------------------------------------------ dense layers on tcgen05

def bf16_round(a):
    import torch
    return torch.from_numpy(a).to(torch.bfloat16)


def gelu_ref(x, tanh):
    return O.gelu(x, bool(tanh))


@pytest.mark.parametrize("M,N,K", [(300, 1152, 1152), (257, 4304, 1152), (200, 3456, 1152), (333, 1152, 4304),
                                    (130, 1152, 592), (1, 256, 64), (128, 128, 128), (1000, 512, 72),
                                    (2100, 4304, 1152), (1555, 3456, 256), (40000, 192, 64),
                                    (300, 72, 64), (513, 1160, 200), (256, 384, 1152), (777, 264, 8)])
@pytest.mark.parametrize("epi", [0, 1, 2, 3])
def test_linear_bf16(B, M, N, K, epi):
    import torch
    rng = np.random.default_rng(M + N + K + epi)
    a = bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    w = bf16_round((rng.standard_normal((N, K)) / math.sqrt(K)).astype(np.float32))
    bias = rng.standard_normal(N).astype(np.float32)
    acc = a.double().numpy() @ w.double().numpy().T + bias.astype(np.float64)
    table_rows = 7
    table = rng.standard_normal((table_rows, N)).astype(np.float32)
    c0 = rng.standard_normal((M, N)).astype(np.float32)
    if epi == 0:
        ref, c = acc, None
    elif epi == 1:
        ref, c = gelu_ref(acc, 1), None
    elif epi == 2:
        ref, c = acc + c0, cuda(c0)
    else:
        ref, c = acc + table[np.arange(M) % table_rows], torch.empty((M, N), dtype=torch.float32, device="cuda")
    out, status = B.et_linear_bf16(a.cuda(), w.cuda(), cuda(bias), epi, 1, c, cuda(table) if epi == 3 else None)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded wait expired inside the kernel"
    got = out.float().cpu().numpy().astype(np.float64)
    scale = np.abs(ref).max()
    tol = (2.0 ** -8 if epi in (0, 1) else 1e-4) * scale + 1e-3   # bf16 output rounding vs fp32 output
    err = np.abs(got - ref).max()
    assert err <= tol, f"max abs err {err:.3e} > {tol:.3e} (scale {scale:.2f})"


def test_linear_bf16_erf_gelu(B):
    rng = np.random.default_rng(0)
    a = bf16_round(rng.standard_normal((64, 64)).astype(np.float32))
    w = bf16_round((rng.standard_normal((64, 64)) / 8).astype(np.float32))
    bias = np.zeros(64, dtype=np.float32)
    out, status = B.et_linear_bf16(a.cuda(), w.cuda(), cuda(bias), 1, 0)
    ref = gelu_ref(a.double().numpy() @ w.double().numpy().T, 0)
    assert int(status.item()) == 0
    assert np.abs(out.float().cpu().numpy() - ref).max() < 2.0 ** -7 * max(1.0, np.abs(ref).max())


# ------------------------------------------------------------------ attention

def attention_ref(qkv, n, L, H, dh):
    """fp64 per-frame attention written with the oracle's softmax; returns (out, lse, score)."""
    D = H * dh
    q = qkv.reshape(n, L, 3 * D).astype(np.float64)
    out = np.zeros((n, L, D)); lse = np.zeros((n, H, L)); score = np.zeros((n, L))
    for f in range(n):
        for h in range(H):
            Q, K, V = (q[f][:, i * D + h * dh:i * D + (h + 1) * dh] for i in range(3))
            P = O.attention_probs(Q, K)
            out[f][:, h * dh:(h + 1) * dh] = P @ V
            s = Q @ K.T / math.sqrt(dh)
            lse[f, h] = np.log(np.exp(s - s.max(1, keepdims=True)).sum(1)) + s.max(1)
            score[f] += P.sum(axis=0)
    return out.reshape(n * L, D), lse, score / (H * L)


@pytest.mark.parametrize("n,L,H,dh", [(2, 64, 4, 16), (1, 729, 2, 72), (2, 50, 3, 24), (1, 33, 1, 128)])
def test_attention_f32(B, n, L, H, dh):
    rng = np.random.default_rng(L + dh)
    qkv = rng.standard_normal((n * L, 3 * H * dh)).astype(np.float32)
    out, lse = B.et_attention(cuda(qkv), n, L, H, dh)
    ref, lse_ref, score_ref = attention_ref(qkv, n, L, H, dh)
    np.testing.assert_allclose(out.cpu().numpy(), ref, rtol=0, atol=2e-5)
    np.testing.assert_allclose(lse.cpu().numpy(), lse_ref, rtol=0, atol=2e-5)
    score = B.et_attention_scores(cuda(qkv), lse, n, L, H, dh)
    np.testing.assert_allclose(score.cpu().numpy() * L, score_ref * L, rtol=0, atol=2e-5)
    np.testing.assert_allclose(score.cpu().numpy().sum(1), 1.0, atol=1e-5)


@pytest.mark.parametrize("n,L,H,dh", [(2, 729, 16, 72), (1, 64, 4, 16), (1, 100, 2, 64), (3, 130, 2, 72),
                                      (1, 17, 1, 32), (1, 200, 1, 128), (1, 70, 2, 40),
                                      (2, 128, 1, 72), (1, 257, 2, 72), (3, 1, 1, 72), (5, 16, 3, 64), (1, 513, 1, 72),
                                      (40, 729, 2, 72), (2, 256, 4, 80), (1, 729, 2, 80), (3, 64, 2, 80), (2, 300, 1, 80)])
def test_attention_bf16(B, n, L, H, dh):
    import torch
    rng = np.random.default_rng(L + dh)
    qkv = bf16_round(rng.standard_normal((n * L, 3 * H * dh)).astype(np.float32))
    out, lse = B.et_attention(qkv.cuda(), n, L, H, dh)
    ref, lse_ref, score_ref = attention_ref(qkv.float().numpy(), n, L, H, dh)
    err = np.abs(out.float().cpu().numpy() - ref).max()
    assert err <= 2e-2 * np.abs(ref).max(), err         # P and the output are rounded to bf16
    np.testing.assert_allclose(lse.cpu().numpy(), lse_ref, rtol=0, atol=1e-4)
    score = B.et_attention_scores(qkv.cuda(), lse, n, L, H, dh).cpu().numpy()
    np.testing.assert_allclose(score * L, score_ref * L, rtol=1e-3, atol=1e-4)
    s2 = B.et_attention_scores(qkv.cuda(), lse, n, L, H, dh).cpu().numpy()
    assert (s2 == score).all(), "score pass must be bit-reproducible"


@pytest.mark.parametrize("n,L,H,dh,w,bf", [(2, 256, 2, 80, 64, True), (3, 64, 2, 80, 16, True), (1, 512, 1, 72, 128, True),
                                          (2, 384, 2, 64, 96, True), (1, 256, 1, 80, 256, True), (2, 36, 3, 16, 9, False),
                                          (1, 320, 2, 40, 64, True)])
def test_attention_windowed(B, n, L, H, dh, w, bf):
    """Windows are runs of w consecutive rows: the result equals plain attention over each window on its own."""
    rng = np.random.default_rng(L + dh + w)
    qkv = rng.standard_normal((n * L, 3 * H * dh)).astype(np.float32)
    if bf:
        qkv = bf16_round(qkv)
        out = B.et_attention_windowed(qkv.cuda(), n, L, H, dh, w).float().cpu().numpy()
        ref, _, _ = attention_ref(qkv.float().numpy(), n * (L // w), w, H, dh)
        assert np.abs(out - ref).max() <= 2e-2 * np.abs(ref).max()
    else:
        out = B.et_attention_windowed(cuda(qkv), n, L, H, dh, w).cpu().numpy()
        ref, _, _ = attention_ref(qkv, n * (L // w), w, H, dh)
        np.testing.assert_allclose(out, ref, rtol=0, atol=2e-5)


@pytest.mark.parametrize("rows,D,bf", [(100, 64, False), (333, 1152, True), (5, 2048, False), (17, 12, True)])
def test_layernorm(B, rows, D, bf):
    rng = np.random.default_rng(D)
    x = (3 + 2 * rng.standard_normal((rows, D))).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(D)).astype(np.float32)
    b = (0.1 * rng.standard_normal(D)).astype(np.float32)
    y = B.et_layernorm(cuda(x), cuda(g), cuda(b), 1e-6, bf).float().cpu().numpy()
    ref = O.layer_norm(x.astype(np.float64), g.astype(np.float64), b.astype(np.float64), 1e-6)
    tol = 2.0 ** -8 * np.abs(ref).max() if bf else 2e-5
    assert np.abs(y - ref).max() <= tol
