"""End-to-end parity of the C-ABI encode calls against the oracle (needs a B200)."""
import dataclasses

import numpy as np
import pytest

from oracle import earlytom_oracle as O
from synthetic import EncoderShape, MergeParams, VideoSpec, Workload, make_batch, make_video, make_weights, workload
from tests import helpers as H

pytestmark = pytest.mark.gpu

F32_TOL = 1e-4       # max relative token error, fp32 arithmetic path
BF16_TOL = 2e-2      # bf16 operands, fp32 accumulate


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2605_30010_b200 import binding
    return binding


def to_cuda(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# Hard ceilings on the numeric error of the decision quantities (the near-tie band itself is widened by the error
# MEASURED in the run, see tests/helpers.py).  Measured on B200: fp32 path similarity error <= 7e-8, score error
# <= 4e-7 of the largest score (rounding order only); bf16 path similarity error <= 7.2e-5 (the cosines come from
# the fp32 residual stream and the errors of 729 positions average out), score error <= 3.5e-3 of the largest
# score.  The ceilings are those figures times 7 (similarity) and 3 (scores), rounded.
F32_SIM, F32_SCORE = 1e-6, 5e-6
BF16_SIM, BF16_SCORE = 5e-4, 1e-2
NEAR_TIE_SHARE = 0.005       # at most 0.5 % of the decisions of a workload may be logged near-ties (measured: <= 0.2 %)


def run_workload(B, wl, oracle_dtype, tol, sim_ceiling, score_ceiling, params=None):
    params = params or wl.params
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed, wl.pos_std)
    w = O.split_weights(wl.shape, blob)
    results = O.encode_batch(frames, offs, wl.shape, w, params, dtype=oracle_dtype)
    enc = B.Encoder(wl.shape, blob, B.ET_F32 if wl.dtype == "f32" else B.ET_BF16, wl.total_frames, len(wl.videos))
    try:
        stats, log = H.check_parity(B, enc, to_cuda(frames), offs, params, H.batch_from_results(results), tol,
                                    sim_ceiling, score_ceiling, wl.name)
    finally:
        enc.close()
    assert stats["near_ties"] <= max(1, NEAR_TIE_SHARE * stats["decisions"]), stats
    return stats["token_err"], log


# ------------------------------------------------------------------ fp32 path

def test_tiny_fp32_workload(B):
    err, log = run_workload(B, workload("tiny"), np.float64, F32_TOL, F32_SIM, F32_SCORE)
    assert not log, "no near-tie expected on the fp32 tiny workload"


def test_tiny_fp32_uncompressed(B):
    wl = workload("tiny").uncompressed()
    run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE)


@pytest.mark.parametrize("selection,mode,retain", [(2, 0, 0.25), (1, 1, 0.3), (0, 1, 1.0), (3, 0, 0.25)])
def test_tiny_fp32_variants(B, selection, mode, retain):
    wl = workload("tiny")
    p = dataclasses.replace(wl.params, selection=selection, retain_mode=mode, retain=retain, tau_seg=0.895, tau_merge=0.85)
    run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE, params=p)


def test_tiny_fp32_unweighted_merge_and_erf_gelu(B):
    wl = workload("tiny")
    wl = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, gelu_tanh=0, post_layernorm=0))
    run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE, params=dataclasses.replace(wl.params, weighted_merge=0))


def test_fp32_batch_of_ragged_videos(B):
    shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
    vids = (VideoSpec(5, 0.1, 1), VideoSpec(1, 0.2, 2), VideoSpec(9, 0.05, 3), VideoSpec(2, 0.5, 4), VideoSpec(12, 0.15, 5))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.6, tau_merge=0.7, selection=1, retain_mode=1, retain=0.4)
    wl = Workload("ragged", shape, "f32", vids, p, 77)
    run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE)


def test_random_sampling_ablation_on_ragged_batch(B):
    """selection 3: both sides draw the same Philox numbers per (video, output frame, position) -> identical kept sets."""
    shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
    vids = (VideoSpec(5, 0.1, 1), VideoSpec(1, 0.2, 2), VideoSpec(9, 0.05, 3), VideoSpec(12, 0.15, 5))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.6, tau_merge=0.7, selection=3, retain_mode=1, retain=0.4,
                    sample_seed=0x1234567890ABCDEF)
    wl = Workload("ragged_random", shape, "f32", vids, p, 77)
    err, log = run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE)
    assert not log


def test_identical_middle_frames_collapse(B):
    """[H, X, X, Y, T]: the two identical frames merge into one frame equal to X."""
    wl = workload("tiny")
    v = make_video(5, 112, 14, 0.6, seed=3)
    v[2] = v[1]
    blob = make_weights(wl.shape, wl.weight_seed)
    p = MergeParams(merge_layers=(1,), tau_seg=-2.0, tau_merge=0.5, selection=0, retain=1.0)
    res = O.encode_video(v, wl.shape, blob, p)
    assert np.nonzero(res.merge_trace[0].merge_with_next)[0].tolist() == [1]
    enc = B.Encoder(wl.shape, blob, B.ET_F32, 5)
    out = enc.encode_video(to_cuda(v), p, want_trace=True)
    assert out.n_frames_out == 4 and np.nonzero(out.trace.merge_next[0])[0].tolist() == [1]
    assert out.trace.sim[0][1] == 1.0
    assert H.token_error(out.tokens.cpu().numpy(), res.tokens) <= F32_TOL
    enc.close()


# ------------------------------------------------------------------ bf16 tensor-core path

@pytest.mark.parametrize("window_mode", [0, 1])
def test_stage2_only_decoupled_selection(B, window_mode):
    """No merge layer: the dynamic / static split comes from the streaming segmentation of the final features, and
    the decoupled selection runs on it (the 'only stage 2' ablation)."""
    shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
    vids = (VideoSpec(9, 0.05, 3), VideoSpec(1, 0.2, 2), VideoSpec(12, 0.15, 5))
    p = MergeParams(merge_layers=(), tau_seg=0.93, tau_merge=0.7, selection=1, retain_mode=1, retain=0.4,
                    window_mode=window_mode)
    wl = Workload("stage2_only", shape, "f32", vids, p, 77)
    frames, offs = make_batch(wl)
    res = O.encode_batch(frames, offs, shape, make_weights(shape, 77), p)
    dyn = np.concatenate([r.frame_dynamic for r in res])
    assert dyn.any() and not dyn.all(), "the case must have both dynamic and static frames"
    err, log = run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE)
    assert not log


def test_stage2_only_bf16(B):
    shape = EncoderShape(image_size=70, patch_size=14, num_layers=4, hidden=144, heads=2, mlp_dim=304)
    vids = (VideoSpec(12, 0.1, 1), VideoSpec(7, 0.3, 2))
    p = MergeParams(merge_layers=(), tau_seg=0.5, tau_merge=0.6, selection=1, retain_mode=1, retain=0.4)
    run_workload(B, Workload("stage2_only_bf16", shape, "bf16", vids, p, 5), np.float64, BF16_TOL, BF16_SIM, BF16_SCORE)


def test_small_bf16_encoder(B):
    """so400m-like odd shapes at a small size: head dim 72, MLP width not a multiple of 64, ragged batch."""
    shape = EncoderShape(image_size=70, patch_size=14, num_layers=4, hidden=144, heads=2, mlp_dim=304)
    vids = (VideoSpec(12, 0.1, 1), VideoSpec(7, 0.3, 2))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.5, tau_merge=0.6, selection=1, retain_mode=1, retain=0.4)
    wl = Workload("small_bf16", shape, "bf16", vids, p, 5)
    run_workload(B, wl, np.float64, BF16_TOL, BF16_SIM, BF16_SCORE)


def test_so400m_8f_bf16(B):
    run_workload(B, workload("so400m_8f"), np.float32, BF16_TOL, BF16_SIM, BF16_SCORE)


# ------------------------------------------------------------------ host entry point and errors

def test_host_entry_point_matches_device_entry_point(B):
    import torch
    wl = workload("tiny")
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed)
    enc = B.Encoder(wl.shape, blob, B.ET_F32, 8)
    dev = enc.encode_batch(to_cuda(frames), offs, wl.params)
    dst = B.HostBuffers(8 * 64, 8, wl.shape.hidden)
    host = B.et_encode_batch_host(enc, torch.from_numpy(frames).pin_memory(), offs, wl.params, dst)
    assert host.n_tokens == dev.n_tokens and host.n_frames_out == dev.n_frames_out
    assert torch.equal(host.tokens, dev.tokens.cpu())
    assert torch.equal(host.token_pos, dev.token_pos.cpu())
    assert torch.equal(host.frame_offsets, dev.frame_offsets.cpu())
    small = B.HostBuffers(4, 8, wl.shape.hidden)
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_encode_batch_host(enc, torch.from_numpy(frames).pin_memory(), offs, wl.params, small)
    assert ei.value.status == 3
    enc.close()


def test_pipelined_host_calls_match_synchronous_calls(B):
    """Two host calls in flight (submit, submit, collect, submit, ...) give bit for bit what the synchronous host call
    gives, on videos of different lengths and content, in both architectures' slot rotation; misuse is refused."""
    import torch
    from synthetic.videos import make_video
    wl = workload("tiny")
    s = wl.shape
    blob = make_weights(s, wl.weight_seed)
    enc = B.Encoder(s, blob, B.ET_F32, 8)
    vids = [torch.from_numpy(make_video(n, s.image_size, s.patch_size, p, seed)).pin_memory()
            for n, p, seed in ((8, 0.3, 0), (5, 0.6, 1), (7, 0.1, 2), (8, 0.9, 3), (3, 0.3, 4))]
    want = []
    for v in vids:
        dst = B.HostBuffers(8 * 64, 8, s.hidden)
        r = B.et_encode_batch_host(enc, v, [0, v.shape[0]], wl.params, dst)
        want.append((r.n_tokens, r.n_frames_out, r.tokens.clone(), r.token_pos.clone(), r.frame_offsets.clone(),
                     r.frame_src_lo.clone(), r.frame_src_hi.clone(), r.frame_dynamic.clone()))
    assert len({w[0] for w in want}) > 1                      # the calls really differ
    bufs = [B.HostBuffers(8 * 64, 8, s.hidden) for _ in range(2)]
    stream = torch.cuda.Stream()
    got, calls = [], []
    for i, v in enumerate(vids):
        calls.append(B.et_encode_batch_host_submit(enc, v, [0, v.shape[0]], wl.params, bufs[i % 2], stream))
        if len(calls) == 2:
            r = B.et_encode_batch_host_collect(enc, calls.pop(0))
            got.append((r.n_tokens, r.n_frames_out, r.tokens.clone(), r.token_pos.clone(), r.frame_offsets.clone(),
                        r.frame_src_lo.clone(), r.frame_src_hi.clone(), r.frame_dynamic.clone()))
    r = B.et_encode_batch_host_collect(enc, calls.pop(0))
    got.append((r.n_tokens, r.n_frames_out, r.tokens.clone(), r.token_pos.clone(), r.frame_offsets.clone(),
                r.frame_src_lo.clone(), r.frame_src_hi.clone(), r.frame_dynamic.clone()))
    assert len(got) == len(want)
    for g, w in zip(got, want):
        assert g[0] == w[0] and g[1] == w[1]
        for a, b in zip(g[2:], w[2:]):
            assert torch.equal(a, b)

    # misuse: a third call in flight, collecting out of order, an unknown ticket, a synchronous call in between,
    # another stream, a trace request
    c1 = B.et_encode_batch_host_submit(enc, vids[0], [0, 8], wl.params, bufs[0], stream)
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_encode_batch_host_submit(enc, vids[1], [0, 5], wl.params, bufs[1], torch.cuda.Stream())
    assert ei.value.status == 1
    c2 = B.et_encode_batch_host_submit(enc, vids[1], [0, 5], wl.params, bufs[1], stream)
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_encode_batch_host_submit(enc, vids[2], [0, 7], wl.params, B.HostBuffers(8 * 64, 8, s.hidden), stream)
    assert ei.value.status == 3
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_encode_batch_host_collect(enc, c2)
    assert ei.value.status == 1
    with pytest.raises(B.EarlyTomError) as ei:
        enc.encode_video(to_cuda(vids[0].numpy()), wl.params)
    assert ei.value.status == 1
    r1 = B.et_encode_batch_host_collect(enc, c1)
    assert r1.n_tokens == want[0][0] and torch.equal(r1.tokens, want[0][2])
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_encode_batch_host_collect(enc, c1)
    assert ei.value.status == 1
    r2 = B.et_encode_batch_host_collect(enc, c2)
    assert r2.n_tokens == want[1][0] and torch.equal(r2.tokens, want[1][2])
    import ctypes as C
    q, _keep = B.make_params(wl.params, None, True)           # a trace request, through the raw entry point
    offs8 = np.array([0, 8], dtype=np.int32)
    ticket = C.c_ulonglong(0)
    st = B.lib().et_encode_batch_host_submit(enc.handle, C.c_void_p(vids[0].data_ptr()),
                                             offs8.ctypes.data_as(C.POINTER(C.c_int32)), 1, C.byref(q), None,
                                             C.byref(bufs[0].c), C.byref(ticket))
    assert st == 1
    # the encoder still serves synchronous calls afterwards
    dev = enc.encode_video(to_cuda(vids[0].numpy()), wl.params)
    assert dev.n_tokens == want[0][0] and torch.equal(dev.tokens.cpu(), want[0][2])
    enc.close()


def test_argument_errors(B):
    wl = workload("tiny")
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed)
    with pytest.raises(B.EarlyTomError) as ei:
        B.Encoder(wl.shape, blob[:-1], B.ET_F32, 8)
    assert ei.value.status == 7
    poisoned = blob.copy()
    poisoned[len(poisoned) // 2] = np.inf
    with pytest.raises(B.EarlyTomError) as ei:
        B.Encoder(wl.shape, poisoned, B.ET_F32, 8)
    assert ei.value.status == 7                                      # non-finite weight
    enc = B.Encoder(wl.shape, blob, B.ET_F32, 4)
    with pytest.raises(B.EarlyTomError) as ei:
        enc.encode_batch(to_cuda(frames), offs, wl.params)          # 8 frames > capacity 4
    assert ei.value.status == 3
    for bad in (dict(merge_layers=(0,)), dict(merge_layers=(2,)), dict(ema_alpha=0.0), dict(retain=0.0), dict(selection=5)):
        with pytest.raises(B.EarlyTomError) as ei:
            enc.encode_batch(to_cuda(frames[:4]), [0, 4], dataclasses.replace(wl.params, **bad))
        assert ei.value.status == 1
    # a forced plan that does not fit the list is reported, not executed blindly
    forced = B.ForcedPlan([np.array([1, 0, 0], dtype=bool)], [np.zeros(3, dtype=bool)], None)
    with pytest.raises(B.EarlyTomError):
        enc.encode_batch(to_cuda(frames[:4]), [0, 4], wl.params, forced=forced)
    ok = enc.encode_batch(to_cuda(frames[:4]), [0, 4], wl.params)    # the encoder stays usable
    assert ok.n_frames_out >= 1
    enc.close()


def test_launch_counter_and_reproducibility(B):
    import torch
    wl = workload("tiny")
    frames, offs = make_batch(wl)
    enc = B.Encoder(wl.shape, make_weights(wl.shape, wl.weight_seed), B.ET_F32, 8)
    before = B.et_kernel_launch_count()
    a = enc.encode_batch(to_cuda(frames), offs, wl.params)
    assert B.et_kernel_launch_count() - before > 10
    b = enc.encode_batch(to_cuda(frames), offs, wl.params)
    assert torch.equal(a.tokens, b.tokens) and torch.equal(a.token_pos, b.token_pos)
    enc.close()


# ------------------------------------------------------------------ Qwen2.5-VL-style encoder (windows, 2-D rotary positions)

def test_qwenvl_tiny_fp32(B):
    err, log = run_workload(B, workload("qwenvl_tiny"), np.float64, F32_TOL, F32_SIM, F32_SCORE)
    assert not log


def test_qwenvl_tiny_fp32_uncompressed_and_full_attention_only(B):
    wl = workload("qwenvl_tiny")
    run_workload(B, wl.uncompressed(), np.float64, F32_TOL, F32_SIM, F32_SCORE)
    nowin = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, window=0, full_attn_layers=()))
    run_workload(B, nowin, np.float64, F32_TOL, F32_SIM, F32_SCORE)


def test_qwenvl_fp32_ragged_batch_three_frames_per_patch(B):
    shape = EncoderShape(image_size=84, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=52, arch=1,
                         temporal_patch=3, window=3, full_attn_layers=(0, 3))
    vids = (VideoSpec(15, 0.05, 1), VideoSpec(3, 0.2, 2), VideoSpec(27, 0.03, 3))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.55, tau_merge=0.6, selection=1, retain_mode=1, retain=0.4)
    wl = Workload("qwenvl_ragged", shape, "f32", vids, p, 78)
    run_workload(B, wl, np.float64, F32_TOL, F32_SIM, F32_SCORE)


def test_qwenvl_small_bf16(B):
    """Head dim 80 and an MLP width that is padded on the tensor-core path (200 -> 256)."""
    shape = EncoderShape(image_size=112, patch_size=14, num_layers=4, hidden=160, heads=2, mlp_dim=200, arch=1,
                         temporal_patch=2, window=4, full_attn_layers=(1, 3))
    vids = (VideoSpec(24, 0.03, 1), VideoSpec(14, 0.1, 2))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.5, tau_merge=0.6, selection=1, retain_mode=1, retain=0.3)
    wl = Workload("qwenvl_small_bf16", shape, "bf16", vids, p, 6)
    run_workload(B, wl, np.float64, BF16_TOL, BF16_SIM, BF16_SCORE)


def test_qwenvl_32f_bf16(B):
    """Qwen2.5-VL's own widths (1280, 16 heads of 80, gated MLP 3420, 32 blocks, windows of 64 tokens in frames of 256):
    16 encoder frames; the oracle runs in the test (about half a minute)."""
    run_workload(B, workload("qwenvl_32f"), np.float32, BF16_TOL, BF16_SIM, BF16_SCORE)


def test_qwenvl_argument_errors(B):
    wl = workload("qwenvl_tiny")
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed)
    for bad in (dict(window=3), dict(full_attn_layers=(1,)), dict(heads=32)):      # grid 4 % 3, last block windowed, head dim 2
        with pytest.raises(B.EarlyTomError) as ei:
            shape = dataclasses.replace(wl.shape, **bad)
            B.Encoder(shape, make_weights(shape, 1), B.ET_F32, 24)
        assert ei.value.status == 2
    enc = B.Encoder(wl.shape, blob, B.ET_F32, 24)
    with pytest.raises(B.EarlyTomError) as ei:
        enc.encode_batch(to_cuda(frames[:5]), [0, 5], wl.params)                    # 5 frames: not a multiple of 2
    assert ei.value.status == 1
    enc.close()
