"""Failure detection without a fault: a bounded device-side wait that runs out is reported as ET_ERR_TIMEOUT and the
context stays usable; the checked build of the library (index checks that record instead of faulting) runs the
small-shape path with no check failing.  Needs a B200."""
import os
import subprocess
import sys
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bounded_wait_runs_out_and_is_reported():
    import torch
    from paper_2605_30010_b200 import binding as B
    B.et_selftest_bounded_wait(1_000_000, arrive=True)                 # the barrier completes: ET_OK
    t0 = time.perf_counter()
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_selftest_bounded_wait(1_000_000, arrive=False)            # nothing arrives: the 1 ms limit runs out
    dt = time.perf_counter() - t0
    assert ei.value.status == 6                                        # ET_ERR_TIMEOUT
    assert dt < 1.0, f"the wait should have given up after a millisecond, took {dt:.3f} s"
    with pytest.raises(B.EarlyTomError) as ei:
        B.et_selftest_bounded_wait(2_000_000_000, arrive=False)        # limits above one second are refused
    assert ei.value.status == 1
    # the context is intact: ordinary work still runs and gives right answers
    x = torch.arange(1024, device="cuda", dtype=torch.float32)
    assert float(x.sum().item()) == 1023 * 1024 / 2
    B.et_selftest_bounded_wait(1_000_000, arrive=True)


DRIVER = r"""
import numpy as np, torch
from oracle import earlytom_oracle as O
from paper_2605_30010_b200 import binding as B
from synthetic import EncoderShape, MergeParams, VideoSpec, Workload, make_batch, make_weights, workload
from tests import helpers as H
assert B.et_debug_build(), "this run must use the checked build"
shape = EncoderShape(image_size=56, patch_size=14, num_layers=4, hidden=48, heads=3, mlp_dim=100)
vids = (VideoSpec(5, 0.1, 1), VideoSpec(1, 0.2, 2), VideoSpec(9, 0.05, 3), VideoSpec(2, 0.5, 4), VideoSpec(12, 0.15, 5))
cases = [workload("tiny"),
         Workload("ragged", shape, "f32", vids, MergeParams(merge_layers=(1, 3), tau_seg=0.6, tau_merge=0.7, selection=1,
                                                            retain_mode=1, retain=0.4), 77),
         Workload("ragged_w0", shape, "f32", vids, MergeParams(merge_layers=(2,), tau_seg=0.6, tau_merge=0.7, selection=1,
                                                               retain_mode=1, retain=0.3, window_mode=0), 77),
         Workload("stage2_only", shape, "f32", vids, MergeParams(merge_layers=(), tau_seg=0.93, selection=1, retain=0.4), 77)]
for wl in cases:
    frames, offs = make_batch(wl)
    blob = make_weights(wl.shape, wl.weight_seed, wl.pos_std)
    res = O.encode_batch(frames, offs, wl.shape, blob, wl.params)
    enc = B.Encoder(wl.shape, blob, B.ET_F32, wl.total_frames, len(wl.videos))
    H.check_parity(B, enc, torch.from_numpy(frames).cuda(), offs, wl.params, H.batch_from_results(res), 1e-4, 1e-6, 5e-6, wl.name)
    enc.close()
rng = np.random.default_rng(0)
a = torch.from_numpy(rng.random((7, 729)).astype(np.float32)).cuda()
dyn = torch.tensor([1, 0, 1, 0, 0, 1, 0], dtype=torch.uint8).cuda()
k = torch.tensor([1, 729, 300, 448, 2, 729, 97], dtype=torch.int32).cuda()
w = torch.clamp(729 // k, min=1).to(torch.int32)
for mode in (0, 1):
    keep, count = B.et_select_tokens(a, dyn, k, w, mode)
    x = torch.from_numpy(rng.standard_normal((7, 729, 64)).astype(np.float32)).cuda()
    toks, offs_, pos = B.et_gather_tokens(x, keep, None, None, 1e-6)
    assert int(offs_[-1].item()) == int(count.sum().item())
torch.cuda.synchronize()
assert B.et_debug_status() == 0, f"an index check failed in the checked build: status {B.et_debug_status()}"
print("checked build ok")
"""


def test_checked_build_runs_the_small_shapes_clean():
    from paper_2605_30010_b200 import build
    lib = build.LIB_DEBUG
    assert os.path.exists(lib), f"{lib} is missing: python -m paper_2605_30010_b200.build --debug"
    env = dict(os.environ, EARLYTOM_LIB=lib, PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-c", DRIVER], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "checked build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_regular_build_reports_no_checked_status():
    from paper_2605_30010_b200 import binding as B
    assert not B.et_debug_build() and B.et_debug_status() == 0
