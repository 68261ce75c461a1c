"""The N > 1 host path of bench.py (replicas, max-over-ranks timing) as two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    seeds = bench.rank_video_seeds(rank, 4)
    # rank 1 is the slow one: the job's time is its time
    local_ms = 100.0 if rank == 0 else 160.0
    value, ms_step = bench.job_throughput(local_ms, steps=4, frames_per_step_per_rank=32, world=world, dist=dist, device="cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, seeds)
    out.put((rank, value, ms_step, gathered))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_aggregate_with_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=100) for _ in procs]
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    for rank, value, ms_step, gathered in results:
        assert ms_step == pytest.approx(40.0)                       # 160 ms / 4 steps, on both ranks
        assert value == pytest.approx(2 * 32 / 0.040)               # whole-job frames/s
        flat = [s for per_rank in gathered for s in per_rank]
        assert len(set(flat)) == len(flat), "replicas must encode different videos"


def test_single_process_needs_no_process_group():
    import bench
    value, ms_step = bench.job_throughput(50.0, steps=5, frames_per_step_per_rank=32, world=1, dist=None, device="cpu")
    assert ms_step == pytest.approx(10.0) and value == pytest.approx(3200.0)
