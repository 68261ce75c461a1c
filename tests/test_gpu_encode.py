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


def oracle_forced(results):
    """Oracle decisions of all videos, concatenated in the layout the library's forced plan uses."""
    nm = len(results[0].merge_trace)
    seg = [np.concatenate([r.merge_trace[i].starts for r in results]) for i in range(nm)]
    mrg = [np.concatenate([r.merge_trace[i].merge_with_next for r in results]) for i in range(nm)]
    keep = np.concatenate([r.keep for r in results], axis=0)
    return seg, mrg, keep


def check_against_oracle(B, enc, frames, offs, params, results, tol, sim_tol, score_tol):
    """The comparison protocol: decisions first (near-ties logged), then values under identical decisions."""
    log = []
    fr = to_cuda(frames)
    free = enc.encode_batch(fr, offs, params, want_trace=True)
    seg, mrg, keep = oracle_forced(results)
    stage1_same = H.compare_stage1(free.trace, results, params, sim_tol, log) if params.merge_layers else True
    run = free if stage1_same else enc.encode_batch(fr, offs, params, want_trace=True,
                                                    forced=B.ForcedPlan(seg, mrg, None))
    # Stage II decisions under identical Stage I decisions
    ora_scores = np.concatenate([r.scores for r in results], axis=0)
    dyn = np.concatenate([r.frame_dynamic for r in results])
    np.testing.assert_array_equal(run.frame_dynamic.cpu().numpy().astype(bool), dyn)
    rel = np.abs(run.trace.scores - ora_scores).max() / ora_scores.max()
    assert rel <= score_tol, f"attention scores differ by {rel:.3e} of the maximum"
    f0 = 0
    keep_same = True
    for v, r in enumerate(results):
        N = len(r.frame_dynamic)
        assert run.trace.video_k[v] == r.k and run.trace.video_w[v] == r.w
        if params.selection != 0:
            dynv = r.frame_dynamic if params.selection == 1 else np.ones(N, dtype=bool)
            keep_same &= H.compare_keep(run.trace.keep[f0:f0 + N], run.trace.scores[f0:f0 + N], r.keep, r.scores,
                                        dynv, r.k, r.w, score_tol, log, params.window_mode)
        f0 += N
    final = run if (stage1_same and keep_same) else enc.encode_batch(fr, offs, params, want_trace=True,
                                                                      forced=B.ForcedPlan(seg, mrg, keep))
    # values and index map under identical decisions
    toks = np.concatenate([r.tokens for r in results], axis=0)
    assert final.n_tokens == toks.shape[0]
    err = H.token_error(final.tokens.cpu().numpy(), toks)
    assert err <= tol, f"token error {err:.3e} > {tol}"
    np.testing.assert_array_equal(final.token_pos.cpu().numpy(), np.concatenate([r.token_pos for r in results]))
    fo = [0]
    for r in results:
        fo += list(fo[-1] + r.frame_offsets[1:])
    np.testing.assert_array_equal(final.frame_offsets.cpu().numpy(), np.array(fo))
    np.testing.assert_array_equal(final.frame_src_lo.cpu().numpy(), np.concatenate([r.frame_src_lo for r in results]))
    np.testing.assert_array_equal(final.frame_src_hi.cpu().numpy(), np.concatenate([r.frame_src_hi for r in results]))
    vfo = np.concatenate([[0], np.cumsum([len(r.frame_dynamic) for r in results])])
    np.testing.assert_array_equal(final.video_frame_offsets.cpu().numpy(), vfo)
    assert final.frames_per_block == [sum(r.frames_per_block[i] for r in results) for i in range(len(final.frames_per_block))]
    for line in log:
        print(line)
    return err, log


def run_workload(B, wl, oracle_dtype, tol, sim_tol, score_tol, params=None):
    params = params or wl.params
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed, wl.pos_std)
    w = O.split_weights(wl.shape, blob)
    results = O.encode_batch(frames, offs, wl.shape, w, params, dtype=oracle_dtype)
    enc = B.Encoder(wl.shape, blob, B.ET_F32 if wl.dtype == "f32" else B.ET_BF16, wl.total_frames, len(wl.videos))
    try:
        return check_against_oracle(B, enc, frames, offs, params, results, tol, sim_tol, score_tol)
    finally:
        enc.close()


# ------------------------------------------------------------------ fp32 path

def test_tiny_fp32_workload(B):
    err, log = run_workload(B, workload("tiny"), np.float64, F32_TOL, 1e-5, 1e-4)
    assert not log, "no near-tie expected on the fp32 tiny workload"


def test_tiny_fp32_uncompressed(B):
    wl = workload("tiny").uncompressed()
    run_workload(B, wl, np.float64, F32_TOL, 1e-5, 1e-4)


@pytest.mark.parametrize("selection,mode,retain", [(2, 0, 0.25), (1, 1, 0.3), (0, 1, 1.0), (3, 0, 0.25)])
def test_tiny_fp32_variants(B, selection, mode, retain):
    wl = workload("tiny")
    p = dataclasses.replace(wl.params, selection=selection, retain_mode=mode, retain=retain, tau_seg=0.895, tau_merge=0.85)
    run_workload(B, wl, np.float64, F32_TOL, 1e-5, 1e-4, params=p)


def test_tiny_fp32_unweighted_merge_and_erf_gelu(B):
    wl = workload("tiny")
    wl = dataclasses.replace(wl, shape=dataclasses.replace(wl.shape, gelu_tanh=0, post_layernorm=0))
    run_workload(B, wl, np.float64, F32_TOL, 1e-5, 1e-4, params=dataclasses.replace(wl.params, weighted_merge=0))


def test_fp32_batch_of_ragged_videos(B):
    shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
    vids = (VideoSpec(5, 0.1, 1), VideoSpec(1, 0.2, 2), VideoSpec(9, 0.05, 3), VideoSpec(2, 0.5, 4), VideoSpec(12, 0.15, 5))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.6, tau_merge=0.7, selection=1, retain_mode=1, retain=0.4)
    wl = Workload("ragged", shape, "f32", vids, p, 77)
    run_workload(B, wl, np.float64, F32_TOL, 1e-5, 1e-4)


def test_random_sampling_ablation_on_ragged_batch(B):
    """selection 3: both sides draw the same Philox numbers per (video, output frame, position) -> identical kept sets."""
    shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
    vids = (VideoSpec(5, 0.1, 1), VideoSpec(1, 0.2, 2), VideoSpec(9, 0.05, 3), VideoSpec(12, 0.15, 5))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.6, tau_merge=0.7, selection=3, retain_mode=1, retain=0.4,
                    sample_seed=0x1234567890ABCDEF)
    wl = Workload("ragged_random", shape, "f32", vids, p, 77)
    err, log = run_workload(B, wl, np.float64, F32_TOL, 1e-5, 1e-4)
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

def test_small_bf16_encoder(B):
    """so400m-like odd shapes at a small size: head dim 72, MLP width not a multiple of 64, ragged batch."""
    shape = EncoderShape(image_size=70, patch_size=14, num_layers=4, hidden=144, heads=2, mlp_dim=304)
    vids = (VideoSpec(12, 0.1, 1), VideoSpec(7, 0.3, 2))
    p = MergeParams(merge_layers=(1, 3), tau_seg=0.5, tau_merge=0.6, selection=1, retain_mode=1, retain=0.4)
    wl = Workload("small_bf16", shape, "bf16", vids, p, 5)
    run_workload(B, wl, np.float64, BF16_TOL, 1e-2, 5e-2)


def test_so400m_8f_bf16(B):
    run_workload(B, workload("so400m_8f"), np.float32, BF16_TOL, 1e-2, 5e-2)


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


def test_argument_errors(B):
    wl = workload("tiny")
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed)
    with pytest.raises(B.EarlyTomError) as ei:
        B.Encoder(wl.shape, blob[:-1], B.ET_F32, 8)
    assert ei.value.status == 7
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
