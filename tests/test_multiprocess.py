"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks agree on the slowest rank's time,
and the whole-job figure counts every rank's tokens (replicas, no data-path collective)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from bench import max_over_ranks, whole_job_tokens_per_s


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 1.5 + rank            # rank 1 is the slow one
    got = max_over_ranks(mine)
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_max_over_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        assert dict(out) == {0: 2.5, 1: 2.5}


def test_single_process_and_weak_scaling_figure():
    assert max_over_ranks(3.25) == 3.25
    assert whole_job_tokens_per_s(256, 1, 2.0) == 128000.0
    assert whole_job_tokens_per_s(256, 8, 2.0) == 8 * 128000.0
