"""The N > 1 plumbing of bench.py (independent replicas: barrier, max over ranks, whole-job rate),
run as two gloo ranks on CPU."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_11248_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        slowest = replicas.max_over_ranks(ms)
        rate = replicas.whole_job_rate(100.0, slowest / 1e3, world)
        out.put((rank, slowest, rate))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, slowest, rate in got:
        assert slowest == 15.0                       # every rank sees the maximum
        assert abs(rate - 2 * 100.0 / 0.015) < 1e-6  # both replicas' work over the slowest time


def test_single_process_needs_no_group():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(10.0, 2.0, 1) == 5.0
