"""Replicas only: the N > 1 path of the benchmark has no data-path collective, just a barrier and a
max-over-ranks of the measured time.  Two gloo ranks on the CPU exercise that host logic."""
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
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    dist.barrier()
    slowest = bench.max_over_ranks(mine, "cpu")
    dist.barrier()
    out.put((rank, slowest, bench.whole_job_throughput(world, 32, 100, slowest)))
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_report_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=100) for _ in range(world))
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    for rank, slowest, value in res:
        assert slowest == 15.0                                    # the max, on every rank
        assert value == pytest.approx(2 * 32 * 100 / 15e-3)      # images of both replicas over the slowest time


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    """Under torchrun the CPU reference arm prints one line from rank 0; the other ranks leave without work."""
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--steps", "1", "--warmup", "0"])
    bench.main()
    assert capsys.readouterr().out.strip() == ""
