"""The multi-GPU mode is "replicas only": ranks exchange nothing but their step times. Two CPU ranks over gloo check
that exchange and the whole-job figure computed from it."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_02470_b200 import replicas


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 100.0 + 25.0 * rank                       # rank 1 is the slower replica
        slowest = replicas.max_over_ranks(local_ms)
        dist.barrier()
        out.put((rank, slowest, replicas.whole_job_rows_per_s(50000, world, slowest)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_step_and_the_sum_of_rows():
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
        assert slowest == 125.0
        assert value == pytest.approx(2 * 50000 / 0.125)


def test_single_process_is_its_own_maximum():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rows_per_s(1000, 1, 10.0) == pytest.approx(1e5)
