"""The N > 1 path of bench.py is "replicas only": ranks do not exchange data, the job time is the
maximum over ranks.  Exercised here with two gloo ranks on CPU."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 0.010 * (rank + 1)                      # rank 1 is the slow replica
        t = bench.max_over_ranks(mine, world, torch.device("cpu"))
        out.put((rank, t, bench.job_us_per_layer(t, steps=5, layers=80, world=world)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    for _, t, us in res:
        assert t == pytest.approx(0.020)                # both ranks see the maximum
        assert us == pytest.approx(0.020 / 5 / 80 / 2 * 1e6)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.5, 1, None) == 0.5
    assert bench.job_us_per_layer(0.004, 1, 80, 1) == pytest.approx(50.0)
