"""The N > 1 path of the bench (independent replicas, max-over-ranks timing) on CPU: two gloo ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_24270_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [0.8, 1.25][rank]                                  # rank 1 is the slow replica
        value, job_ms = replicas.job_throughput(ms, 1.0e12)
        # every rank sees the slowest rank's time and the work of both ranks (a failed assert fails the spawn)
        assert abs(job_ms - 1.25) < 1e-12 and abs(replicas.slowest_rank_ms(ms) - 1.25) < 1e-12
        assert abs(value - 2 * 1.0e12 / 1.25e-3) < 1e-3
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_ranks_time():
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port), nprocs=world, join=True)


def test_single_process_is_identity():
    value, ms = replicas.job_throughput(0.5, 4.0)
    assert ms == 0.5 and value == pytest.approx(4.0 / 0.5e-3)
