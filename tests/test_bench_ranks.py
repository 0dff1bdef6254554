"""bench.py's multi-rank accounting, on CPU with the gloo backend and two processes: the job's
time is the MAX over the ranks' device times and `value` counts every rank's steps."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slow one: 30 ms against 20 ms for 100 steps each
    value, ms = bench.whole_job_rate(20.0 + 10.0 * rank, 100, world, dist, "cpu")
    out.put((rank, value, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_value_is_all_ranks_steps_over_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, ms in res:
        assert ms == pytest.approx(30.0)
        assert value == pytest.approx(2 * 100 / 0.030)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.whole_job_rate(50.0, 10, 1)
    assert ms == 50.0 and value == pytest.approx(200.0)


def test_algorithmic_bytes_match_the_benchmark_table():
    sys.path.insert(0, ROOT)
    import bench
    from paper_1805_10032_b200 import synthetic as syn
    w = syn.make_config(2, dims=(3072, 512, 512, 10), m=2, b=1, faults=[(1, "noise200")])
    w.m, w.b = 20, 8          # the byte count depends on the sizes only
    score, agg = bench.algorithmic_bytes(w)
    assert abs(score - 155.1e6) < 0.2e6 and abs(agg - 95.7e6) < 0.2e6   # 250.8 MB per step
