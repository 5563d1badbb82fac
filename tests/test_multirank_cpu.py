"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks, no data-path collective.

Each rank owns its own copy of the weight set (different seed); the only exchange is the reduction
of the timing (max over ranks) and the whole-job throughput is computed from it.
"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def _worker(rank, world, port, out):
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
        seeds = [None] * world
        dist.all_gather_object(seeds, bench.rank_seed(rank))
        if rank == 0:
            out.put((ms, seeds, bench.whole_job_value(1000, world, ms, steps=5)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_disjoint_inputs():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, seeds, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0
    assert len(set(seeds)) == 2
    assert value == pytest.approx(2 * 1000 / (15.0e-3 / 5))


def test_single_rank_helpers_are_identity():
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_value(100, 1, 1000.0, 10) == pytest.approx(1000.0)


def test_reference_arm_prints_one_json_line_on_rank_zero_only(tmp_path):
    import json
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
