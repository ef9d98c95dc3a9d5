"""Host-side logic of bench.py that does not need a GPU: the replicas-only aggregation over ranks (two gloo processes on
CPU) and the reference arm's rank rule."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, torch.device("cpu"), dist, torch)
    rate = bench.replica_rate(world, 1.0e9, 4, ms)     # 1 GB per rank per step, 4 steps
    out.put((rank, ms, rate))
    dist.barrier()
    dist.destroy_process_group()


def test_replicas_report_the_slowest_rank_and_the_sum_of_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in res:
        assert ms == pytest.approx(15.0)                               # max over ranks, on every rank
        assert rate == pytest.approx(2 * 1.0e9 * 4 / 15.0e-3)          # both replicas' bytes over the slowest rank's time


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5, 1, torch.device("cpu"), None, torch) == 7.5
    assert bench.replica_rate(1, 2.0, 3, 1000.0) == pytest.approx(6.0)


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import argparse
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(argparse.Namespace(decode_m=16, steps=1, warmup=0, gpus=2))
    assert capsys.readouterr().out == ""                                # the other ranks print nothing and do no work
