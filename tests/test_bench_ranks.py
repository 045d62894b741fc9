"""The multi-rank bookkeeping of bench.py (independent replicas, no data-path collective): the job's
time is the slowest rank's, the job's rate sums the replicas' work.  Run as two gloo ranks on CPU."""

import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, "cpu")
    dist.barrier()
    out.put((rank, ms, bench.job_rate(1000 * 20, ms, world)))
    dist.destroy_process_group()


def test_slowest_rank_sets_the_time_and_work_adds_up():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in res:
        assert ms == pytest.approx(15.0)
        assert rate == pytest.approx(2 * 1000 * 20 / 15.0e-3)


def test_single_process_is_a_no_op():
    import bench
    assert bench.max_over_ranks(7.5, "cpu") == 7.5
    assert bench.job_rate(100, 50.0, 1) == pytest.approx(2000.0)


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import argparse
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    args = argparse.Namespace(workload="cfg1_al108", steps=1, warmup=1, cpu_seconds=1.0, gpus=2, impl="reference", modes=-1)
    bench.run_reference(args)                           # returns at once, prints nothing
    assert capsys.readouterr().out == ""
