"""Tensor-parallel adapter wave (paper Finding 5: row-parallel A, an R-wide all-reduce, column-parallel B).

CPU: the shard arithmetic, and the wave on two gloo ranks with the oracle standing in for each
rank's shrink and expand.  GPU (one device): both ranks' shards run one after the other through the
library's shrink and expand kernels, the all-reduce replaced by a sum on the device; kernels of
different ranks never wait for one another here."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from helpers import TOL_FP32_PATH, random_problem, rel_err
from paper_2608_05483_b200.tp import TensorParallelDelta, shard_adapter, shard_bounds


def test_shard_bounds_cover_the_dimension_in_aligned_pieces():
    for d, world in [(4096, 4), (5120, 8), (13824, 64), (328, 3), (8, 1), (64, 8)]:
        cuts = [shard_bounds(d, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == d
        for (lo, hi), (lo2, _) in zip(cuts, cuts[1:]):
            assert hi == lo2
        sizes = [hi - lo for lo, hi in cuts]
        assert all(s % 8 == 0 and s > 0 for s in sizes) and max(sizes) - min(sizes) <= 8
    with pytest.raises(ValueError):
        shard_bounds(100, 0, 2)        # not a multiple of 8
    with pytest.raises(ValueError):
        shard_bounds(16, 0, 4)         # fewer blocks than ranks
    with pytest.raises(ValueError):
        shard_bounds(64, 2, 2)


def _problem():
    return random_problem(91, T=37, d_in=328, d_out=200, ranks=[8, 16, 5, 64, 33, 128], with_minus_one=True)


def _rank_wave_on_the_oracle(p, rank, world, all_reduce):
    """One rank's part of the wave: oracle shrink on its rows of A, the exchange, oracle expand on its columns of B."""
    lo_i, hi_i = shard_bounds(p["d_in"], rank, world)
    lo_o, hi_o = shard_bounds(p["d_out"], rank, world)
    shards = [shard_adapter(a, b, rank, world) for a, b in zip(p["A"], p["B"])]
    ldm = int(max(p["ranks"]))
    m = oracle.shrink(np.ascontiguousarray(p["x"][:, lo_i:hi_i]), p["ids"], p["ranks"], [s[0] for s in shards], ldm)
    m = all_reduce(m)
    y = oracle.expand(m, p["ids"], p["ranks"], p["scales"], [s[1] for s in shards], hi_o - lo_o,
                      np.ascontiguousarray(p["y_in"][:, lo_o:hi_o]))
    return (lo_o, hi_o), y


def test_the_wave_equals_the_unsharded_delta():
    # sum of the ranks' partial m = the full m, so the column shards of y are the columns of the full y
    p = _problem()
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], p["y_in"])
    for world in (2, 3):
        parts = []
        for r in range(world):
            lo_i, hi_i = shard_bounds(p["d_in"], r, world)
            shards = [shard_adapter(a, b, r, world) for a, b in zip(p["A"], p["B"])]
            parts.append(oracle.shrink(np.ascontiguousarray(p["x"][:, lo_i:hi_i]), p["ids"], p["ranks"],
                                       [s[0] for s in shards], int(max(p["ranks"]))))
        m = np.sum(parts, axis=0)
        got = np.empty_like(ref)
        for r in range(world):
            (lo, hi), y = _rank_wave_on_the_oracle(p, r, world, lambda _m: m)
            got[:, lo:hi] = y
        assert np.max(np.abs(got - ref)) <= 1e-12 * np.max(np.abs(ref))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _gloo_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    p = _problem()

    def all_reduce(m):
        t = torch.from_numpy(m)
        dist.all_reduce(t)            # sums in place over the two ranks
        return t.numpy()

    (lo, hi), y = _rank_wave_on_the_oracle(p, rank, world, all_reduce)
    out[rank] = (lo, hi, y)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_run_the_wave():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_gloo_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    p = _problem()
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], p["y_in"])
    got = np.empty_like(ref)
    for r in range(world):
        lo, hi, y = res[r]
        got[:, lo:hi] = y
    assert np.max(np.abs(got - ref)) <= 1e-12 * np.max(np.abs(ref))


@pytest.mark.gpu
@pytest.mark.parametrize("world", [2, 4])
def test_both_shards_through_the_kernels_on_one_gpu(world):
    import paper_2608_05483_b200 as P
    from gpu_util import DEV, bits_to_dev

    p = random_problem(93, T=150, d_in=512, d_out=384, ranks=[16, 8, 64, 128, 30, 16, 16, 100], with_minus_one=True)
    ref = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"], p["y_in"])
    ids = torch.from_numpy(p["ids"]).to(DEV)
    ranks_tp, pending = [], []

    # every rank's all-reduce hands back the same sum; it is formed once all ranks have shrunk
    class Exchange:
        def __init__(self):
            self.parts, self.total = [], None

    ex = Exchange()
    for r in range(world):
        ctx = P.Context(p["T"], p["N"])
        tp = TensorParallelDelta(ctx, r, world, all_reduce=None)
        tp.register_pool(0, 0, p["d_in"], p["d_out"], p["ranks"], p["scales"], p["A"], p["B"])
        ranks_tp.append(tp)
    # phase 1: every rank's shrink (what TensorParallelDelta.lora_delta does up to the exchange)
    for r, tp in enumerate(ranks_tp):
        lo_i, hi_i = shard_bounds(p["d_in"], r, world)
        x_shard = bits_to_dev(np.ascontiguousarray(p["x"][:, lo_i:hi_i]))
        m = torch.zeros((p["T"], tp.ctx.pool_max_rank(0, 0)), dtype=torch.float32, device=DEV)
        tp.ctx.bucket(ids, p["N"])
        tp.ctx.shrink(x_shard, ids, 0, 0, m)
        ex.parts.append(m)
        pending.append(x_shard)
    torch.cuda.synchronize()
    ex.total = torch.stack(ex.parts).sum(dim=0)
    # phase 2: the whole wave per rank through the class, its all-reduce returning the sum of all ranks' m
    got = np.empty((p["T"], p["d_out"]), np.float32)
    for r, tp in enumerate(ranks_tp):
        lo_o, hi_o = shard_bounds(p["d_out"], r, world)

        def all_reduce(m, mine=ex.parts[r]):
            assert torch.equal(m, mine)          # the class's shrink gives the same partial m again
            m.copy_(ex.total)

        tp.all_reduce = all_reduce
        y = torch.from_numpy(np.ascontiguousarray(p["y_in"][:, lo_o:hi_o])).to(DEV)
        tp.lora_delta(pending[r], ids, 0, 0, y)
        torch.cuda.synchronize()
        got[:, lo_o:hi_o] = y.cpu().numpy()
        assert tp.ctx.device_status() == 0
    delta = np.max(np.abs(ref - p["y_in"]))
    assert np.max(np.abs(got - ref)) <= TOL_FP32_PATH * delta + 1e-6 * np.max(np.abs(ref))
    for tp in ranks_tp:
        tp.ctx.close()


def test_the_wave_runs_its_three_steps_in_order_on_the_callers_stream(monkeypatch):
    """The all-reduce must be called between the two kernels while the caller's stream is the current one
    (torch.distributed orders a collective against the current stream)."""
    import contextlib

    log = []

    class FakeCtx:
        def pool_max_rank(self, layer, proj):
            return 8

        def shrink(self, x, ids, layer, proj, m, stream=None):
            log.append(("shrink", stream, current[0]))

        def expand(self, m, ids, layer, proj, y, stream=None):
            log.append(("expand", stream, current[0]))

    current = [None]

    @contextlib.contextmanager
    def fake_stream_ctx(s):
        prev, current[0] = current[0], s
        try:
            yield
        finally:
            current[0] = prev

    monkeypatch.setattr(torch.cuda, "stream", fake_stream_ctx)
    tp = TensorParallelDelta(FakeCtx(), 0, 2, all_reduce=lambda m: log.append(("all_reduce", None, current[0])))
    x = torch.zeros((4, 16))
    ids = torch.zeros(4, dtype=torch.int32)
    y = torch.zeros((4, 16))
    mine = object()
    tp.lora_delta(x, ids, 0, 0, y, stream=mine)
    assert [e[0] for e in log] == ["shrink", "all_reduce", "expand"]
    assert all(e[2] is mine for e in log) and log[0][1] is mine and log[2][1] is mine
    log.clear()
    tp.lora_delta(x, ids, 0, 0, y)            # no stream given: nothing is made current
    assert [e[0] for e in log] == ["shrink", "all_reduce", "expand"] and all(e[2] is None for e in log)
