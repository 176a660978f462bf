"""Tensor-parallel adapter wave (paper Section VIII, Finding 5): partition the LoRA delta with the
base model's tensor parallelism instead of replicating the activation on every GPU.

Rank p of P holds, for every adapter, the rows [lo_in, hi_in) of A (row-parallel A: the activation
arrives already split along d_in, as after a column-parallel layer) and the columns
[lo_out, hi_out) of B (column-parallel B).  One wave is

    m_p = x[:, lo_in:hi_in] A[lo_in:hi_in, :]      plora_shrink on the rank's pool
    m   = sum_p m_p                                 an R-wide all-reduce (n_tok x rank floats)
    y[:, lo_out:hi_out] += s m B[:, lo_out:hi_out]  plora_expand on the rank's pool

so the pool traffic of a GPU and its share of the activation both shrink as 1/P and the only
exchange is the small m.  Everything numerical runs in the library's shrink and expand kernels;
this module holds the index arithmetic and the call sequence, and takes the all-reduce as a
callable (torch.distributed.all_reduce on an NCCL group in production, anything else in a test).

The benchmark's --tp mode runs this wave with torch.distributed.all_reduce on an NCCL group, one rank per
GPU.  Covered by a two-rank gloo test of the arithmetic on CPU, by a one-GPU test that runs both ranks'
shards one after the other, and by a CPU test that the wave's three steps run in order on the caller's
stream.
"""
from __future__ import annotations

from typing import Callable, Sequence

import numpy as np

ALIGN = 8   # the library wants d_in and d_out in multiples of 8 (16-byte rows of bf16)


def shard_bounds(d: int, rank: int, world: int, align: int = ALIGN) -> tuple[int, int]:
    """[lo, hi) of dimension d owned by `rank`: contiguous, multiples of `align`, sizes differing by at
    most one block, the first d / align % world ranks taking the larger share."""
    if d % align or world < 1 or not 0 <= rank < world:
        raise ValueError(f"cannot shard d={d} over {world} ranks in blocks of {align} (rank {rank})")
    blocks = d // align
    if blocks < world:
        raise ValueError(f"d={d} has fewer blocks of {align} than ranks ({world})")
    base, extra = divmod(blocks, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo * align, hi * align


def shard_adapter(A, B, rank: int, world: int):
    """The rank's slices of one adapter: rows of A [d_in, r], columns of B [r, d_out] (numpy arrays or
    torch tensors; contiguous copies, as the registration wants row-major matrices)."""
    lo_i, hi_i = shard_bounds(A.shape[0], rank, world)
    lo_o, hi_o = shard_bounds(B.shape[1], rank, world)
    a, b = A[lo_i:hi_i, :], B[:, lo_o:hi_o]
    if isinstance(a, np.ndarray):
        return np.ascontiguousarray(a), np.ascontiguousarray(b)
    return a.contiguous(), b.contiguous()


class TensorParallelDelta:
    """The wave on one rank.  `ctx` is a paper_2608_05483_b200.Context whose pools were registered with
    this rank's shards (register_pool below does the slicing); `all_reduce(m)` sums the fp32 tensor m
    in place over the ranks of the tensor-parallel group."""

    def __init__(self, ctx, rank: int, world: int, all_reduce: Callable):
        self.ctx, self.rank, self.world, self.all_reduce = ctx, rank, world, all_reduce
        self._m = {}

    def register_pool(self, layer: int, proj: int, d_in: int, d_out: int, ranks, scales, A: Sequence, B: Sequence):
        """A[a]: the full [d_in, r_a], B[a]: the full [r_a, d_out]; only this rank's slices are kept."""
        lo_i, hi_i = shard_bounds(d_in, self.rank, self.world)
        lo_o, hi_o = shard_bounds(d_out, self.rank, self.world)
        shards = [shard_adapter(a, b, self.rank, self.world) for a, b in zip(A, B)]
        return self.ctx.register_pool(layer, proj, hi_i - lo_i, hi_o - lo_o, ranks, scales,
                                      [s[0] for s in shards], [s[1] for s in shards])

    def lora_delta(self, x_shard, ids, layer: int, proj: int, y_shard, stream=None):
        """x_shard: [n_tok, d_in / P] (this rank's columns of x); y_shard: fp32 [n_tok, d_out / P],
        accumulated.  The all-reduce is queued between the two kernels by its own library."""
        import torch

        n_tok = int(ids.numel())
        ldm = self.ctx.pool_max_rank(layer, proj)
        key = (n_tok, ldm, x_shard.device)
        m = self._m.get(key)
        if m is None:
            m = self._m[key] = torch.empty((n_tok, ldm), dtype=torch.float32, device=x_shard.device)
        # All three steps are queued on one stream, in this order.  torch.distributed orders a collective
        # against the stream that is current when it is called, so a caller's stream is made current for the
        # whole wave: the all-reduce then starts after the shrink kernel and the expand kernel after the sum.
        import contextlib
        with (torch.cuda.stream(stream) if stream is not None else contextlib.nullcontext()):
            self.ctx.shrink(x_shard, ids, layer, proj, m, stream=stream)
            self.all_reduce(m)
            self.ctx.expand(m, ids, layer, proj, y_shard, stream=stream)
