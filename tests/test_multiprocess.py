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


# ---- the benchmark's own rank starter, driven with two gloo ranks and a wave that needs no GPU ----
class OracleWave:
    """The tensor-parallel wave of one rank with the float64 oracle in place of the kernels (same interface
    as bench.KernelWave): shrink on the rank's rows of A, all-reduce of m over the process group, expand on
    its columns of B."""

    def __init__(self, wl, rank, world, local):
        import numpy as np
        import oracle
        from paper_2608_05483_b200.tp import shard_adapter, shard_bounds
        from workloads import gen_adapter, gen_x, gen_y_in
        self.np, self.oracle, self.wl, self.rank, self.world = np, oracle, wl, rank, world
        self.pool = wl.pools[0]
        p = self.pool
        self.lo_i, self.hi_i = shard_bounds(p.d_in, rank, world)
        self.lo_o, self.hi_o = shard_bounds(p.d_out, rank, world)
        full = [gen_adapter(wl, p, a) for a in range(wl.n_adapters)]
        self.full = full
        shards = [shard_adapter(a, b, rank, world) for a, b in full]
        self.A, self.B = [s[0] for s in shards], [s[1] for s in shards]
        self.x = gen_x(wl, p)
        self.y_in = gen_y_in(wl, p)
        self.pool_bytes = sum(a.nbytes + b.nbytes for a, b in shards)
        self.ldm = int(max(wl.ranks))
        self.allreduce_bytes_per_wave = wl.n_tok * self.ldm * 4
        self.calls = 0

    def _wave(self):
        np, wl = self.np, self.wl
        m = self.oracle.shrink(np.ascontiguousarray(self.x[:, self.lo_i:self.hi_i]), wl.ids, wl.ranks, self.A, self.ldm)
        t = torch.from_numpy(m)
        if dist.is_initialized() and dist.get_world_size() > 1:
            dist.all_reduce(t)
        self.calls += 1
        return self.oracle.expand(t.numpy(), wl.ids, wl.ranks, wl.scales, self.B, self.hi_o - self.lo_o,
                                  np.ascontiguousarray(self.y_in[:, self.lo_o:self.hi_o]))

    def check(self):
        np, wl, p = self.np, self.wl, self.pool
        want = self.oracle.lora_delta(self.x, wl.ids, wl.ranks, wl.scales, [f[0] for f in self.full],
                                      [f[1] for f in self.full], p.d_out, self.y_in)[:, self.lo_o:self.hi_o]
        got = self._wave()
        return float(np.max(np.abs(got - want)) / np.max(np.abs(want)))

    def step(self):
        self._wave()

    def timed(self, steps):
        import time
        t0 = time.perf_counter()
        for _ in range(steps):
            self.step()
        return (time.perf_counter() - t0) * 1e3 / steps

    def launches(self):
        return self.calls

    def close(self):
        pass


def oracle_wave(wl, rank, world, local):
    return OracleWave(wl, rank, world, local)


def test_bench_starts_its_own_ranks(tmp_path):
    import argparse
    import json

    import bench
    args = argparse.Namespace(config=1, layers=None, steps=2, warmup=1, tp_backend="gloo")
    out = tmp_path / "line.json"
    bench.spawn_local(2, bench.tp_job, (args, oracle_wave, str(out)))
    line = json.loads(out.read_text())
    assert line["n_gpus"] == 2 and line["config"]["parallelism"] == "tp2"
    assert line["parity_max_rel_err"] <= 1e-12
    # Finding 5: a rank holds half of every adapter, and the only exchange is n_tok x rank floats per wave
    assert line["per_gpu_pool_bytes"] == 16 * (512 * 8 + 8 * 512) * 2 // 2
    assert line["allreduce_bytes_per_wave"] == 64 * 8 * 4
    assert line["gpu_launches"] == 2 and line["steps"] == 2
