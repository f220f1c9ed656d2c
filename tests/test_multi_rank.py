"""The N > 1 arithmetic of bench.py on CPU: two gloo ranks, each with its own duration, must agree on
the slowest rank's time and on the whole-job throughput; the reference arm runs on rank 0 only."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = [10.0, 12.5][rank]                      # rank 1 is the slow one
        slowest = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
        value = bench.whole_job_value(world, 1024, slowest)
        dist.barrier()
        out.put((rank, slowest, value))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_value():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 12.5
        assert abs(value - 2 * 1024 / 12.5e-3) < 1e-6
    assert [g[0] for g in got] == [0, 1]


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.25, 1, torch.device("cpu")) == 3.25
    assert bench.whole_job_value(1, 100, 50.0) == 2000.0


def test_reference_arm_is_silent_on_other_ranks(monkeypatch, capsys):
    import argparse
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(argparse.Namespace(workload="llama2_7b_ffn_r20_b1", warmup=0, steps=1, gpus=2))
    assert capsys.readouterr().out == ""
