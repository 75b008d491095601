"""world_size-2 check (gloo, CPU) of the only multi-GPU logic the path has: replicas agree on the
slowest rank's time and the whole-job rate is computed from it."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_26515_b200.replicas import max_over_ranks, whole_job_rate
    my_ms = 10.0 + 5.0 * rank
    worst = max_over_ranks(my_ms)
    rate = whole_job_rate(units_per_rank_per_step=100.0, steps=4, max_ms=worst, world=world)
    out[rank] = (worst, rate)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_agree_on_the_slowest_rank():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    worst, rate = out[0]
    assert worst == 15.0
    assert rate == 2 * 100.0 * 4 / 15e-3


def test_single_process_needs_no_group():
    from paper_2607_26515_b200.replicas import max_over_ranks
    assert max_over_ranks(3.5) == 3.5
