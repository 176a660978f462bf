"""Seeded generators for the benchmark-shaped workloads.

Every array is a pure function of (config number, overrides, seed): a test can
regenerate any single adapter, activation block or id vector without building
the rest.  Values are drawn in fp32 and rounded to bf16 once (round to nearest
even, by integer arithmetic on the bit pattern); the raw 16-bit patterns are
what both the GPU path and the CPU oracle consume.

Workload recipes (shapes follow the paper's evaluation: 1000 adapters, ranks
from a power-of-two set, uniform or skewed adapter popularity, Llama-2 7B/13B
projection shapes — Section VII-A and its workload table):

  1 tiny      64 tokens, 512->512, rank 8, 16 adapters, ids uniform, s = 2
  2 decode7b  256 tokens (one per request), q/k/v/o 4096->4096 per layer,
              rank 16, 1000 adapters, ids ~ bounded Zipf(1.0), s = 32/16
  3 decode13b 512 tokens, q/k/v/o 5120->5120, up/gate 5120->13824,
              down 13824->5120, rank 64, 1000 adapters, ids uniform, s = 32/64
  4 prefill   32 requests x 512 contiguous tokens, q/k/v/o 4096->4096,
              rank 32, 1000 adapters, request adapter ~ bounded Zipf(1.2), s = 1
  5 mixed     2048 tokens: 1024 one-token requests + prefill requests of
              length U[2,256] filling 1024 more tokens, request order shuffled,
              q/o 8192->8192, per-adapter rank ~ U{8,16,32,64}, ids ~ bounded
              Zipf(0.8), s_a = 32/r_a
  6 skew7b    the paper's own skewed request mix on the decode shapes of 2: 256
              one-token requests, 80 % of them to 50 hot adapters (uniform inside
              the hot and inside the cold set), per-adapter rank ~ U{8,16,32,64,128}
              (the evaluation's rank set), q/k/v/o 4096->4096, s_a = 32/r_a

Distributions: x ~ N(0,1); A ~ N(0, 1/d_in) (variance); B ~ N(0, 1/r)
(variance); y_in ~ N(0,1).  Bounded Zipf: p_k proportional to k^-alpha for
k = 1..N, sampled by inverse CDF; popularity rank k is mapped to an adapter id
through a seeded permutation so hot adapters are not neighbours in memory.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20260805 * 10

CONFIG_NAMES = {1: "tiny", 2: "decode7b", 3: "decode13b", 4: "prefill", 5: "mixed", 6: "skew7b"}

PROJ_NAMES = ("q", "k", "v", "o", "up", "gate", "down")
# projections that read the same activation tensor share an x group
_X_GROUP = {0: 0, 1: 0, 2: 0, 3: 1, 4: 2, 5: 2, 6: 3}

_TAG_X, _TAG_A, _TAG_B, _TAG_Y, _TAG_IDS, _TAG_RANKS, _TAG_POP, _TAG_MIX = range(1, 9)


# --------------------------------------------------------------------------
# bf16 bit helpers (storage format only, no arithmetic of the method)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def f32_to_fp16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to IEEE half (nearest even) and return the uint16 bit patterns."""
    return np.ascontiguousarray(a, dtype=np.float32).astype(np.float16).view(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------
# workload description
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class PoolSpec:
    """One (layer, projection) adapter pool."""

    layer: int
    proj: int
    d_in: int
    d_out: int

    @property
    def name(self) -> str:
        return f"L{self.layer}.{PROJ_NAMES[self.proj]}"

    @property
    def x_group(self) -> int:
        return _X_GROUP[self.proj]


@dataclass
class Workload:
    cfg: int
    name: str
    seed: int
    n_tok: int
    n_adapters: int
    pools: list
    ranks: np.ndarray  # int32 [n_adapters]
    scales: np.ndarray  # float32 [n_adapters]
    ids: np.ndarray  # int32 [n_tok]
    meta: dict = field(default_factory=dict)

    def pool(self, layer: int, proj: int) -> PoolSpec:
        for p in self.pools:
            if p.layer == layer and p.proj == proj:
                return p
        raise KeyError((layer, proj))

    def distinct_adapters(self) -> np.ndarray:
        return np.unique(self.ids[self.ids >= 0])


def _rng(seed: int, *tags: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([seed, *[int(t) for t in tags]]))


def bounded_zipf_pmf(n: int, alpha: float) -> np.ndarray:
    k = np.arange(1, n + 1, dtype=np.float64)
    w = k ** (-float(alpha))
    return w / w.sum()


def _zipf_ids(rng_draw, rng_perm, n_draw: int, n_adapters: int, alpha: float) -> np.ndarray:
    cdf = np.cumsum(bounded_zipf_pmf(n_adapters, alpha))
    cdf[-1] = 1.0
    pop_rank = np.searchsorted(cdf, rng_draw.random(n_draw), side="right")
    pop_rank = np.minimum(pop_rank, n_adapters - 1)
    id_of_rank = rng_perm.permutation(n_adapters)
    return id_of_rank[pop_rank].astype(np.int32)


def _pools(n_layers: int, projs, dims) -> list:
    out = []
    for layer in range(n_layers):
        for p in projs:
            d_in, d_out = dims[p]
            out.append(PoolSpec(layer, p, d_in, d_out))
    return out


def make_workload(cfg: int, *, n_layers: int | None = None, n_adapters: int | None = None,
                  n_tok: int | None = None, d_model: int | None = None, d_ff: int | None = None,
                  rank: int | None = None, seed: int | None = None) -> Workload:
    """Build workload `cfg` (1..5).  Keyword overrides shrink a config for tests
    without changing its structure (id distribution, rank mix, segment mix)."""
    if cfg not in CONFIG_NAMES:
        raise ValueError(f"unknown config {cfg}")
    seed = BASE_SEED + cfg if seed is None else int(seed)
    meta: dict = {}

    if cfg == 1:
        T, N, D, r, L = n_tok or 64, n_adapters or 16, d_model or 512, rank or 8, n_layers or 1
        pools = _pools(L, (0,), {0: (D, D)})
        ranks = np.full(N, r, np.int32)
        scales = np.full(N, 2.0, np.float32)
        ids = _rng(seed, _TAG_IDS).integers(0, N, size=T).astype(np.int32)
        meta["ids"] = "uniform"
    elif cfg == 2:
        T, N, D, r, L = n_tok or 256, n_adapters or 1000, d_model or 4096, rank or 16, n_layers or 32
        pools = _pools(L, (0, 1, 2, 3), {p: (D, D) for p in range(4)})
        ranks = np.full(N, r, np.int32)
        scales = np.full(N, 32.0 / r, np.float32)
        ids = _zipf_ids(_rng(seed, _TAG_IDS), _rng(seed, _TAG_POP), T, N, 1.0)
        meta["ids"] = "zipf(1.0)"
    elif cfg == 3:
        T, N, D, r, L = n_tok or 512, n_adapters or 1000, d_model or 5120, rank or 64, n_layers or 1
        F = d_ff or (13824 if D == 5120 else (D * 27 // 10 + 255) // 256 * 256)
        dims = {0: (D, D), 1: (D, D), 2: (D, D), 3: (D, D), 4: (D, F), 5: (D, F), 6: (F, D)}
        pools = _pools(L, (0, 1, 2, 3, 4, 5, 6), dims)
        ranks = np.full(N, r, np.int32)
        scales = np.full(N, 32.0 / r, np.float32)
        ids = _rng(seed, _TAG_IDS).integers(0, N, size=T).astype(np.int32)
        meta["ids"] = "uniform"
    elif cfg == 4:
        n_req, req_len = 32, 512
        if n_tok is not None:
            req_len = max(1, n_tok // n_req)
        T, N, D, r, L = n_req * req_len, n_adapters or 1000, d_model or 4096, rank or 32, n_layers or 1
        pools = _pools(L, (0, 1, 2, 3), {p: (D, D) for p in range(4)})
        ranks = np.full(N, r, np.int32)
        scales = np.full(N, 32.0 / r, np.float32)
        req_ids = _zipf_ids(_rng(seed, _TAG_IDS), _rng(seed, _TAG_POP), n_req, N, 1.2)
        ids = np.repeat(req_ids, req_len).astype(np.int32)
        meta.update(ids="zipf(1.2) per request", n_requests=n_req, request_len=req_len)
    elif cfg == 6:
        T, N, D, L = n_tok or 256, n_adapters or 1000, d_model or 4096, n_layers or 8
        pools = _pools(L, (0, 1, 2, 3), {p: (D, D) for p in range(4)})
        if rank is None:
            ranks = _rng(seed, _TAG_RANKS).choice(np.array([8, 16, 32, 64, 128], np.int32), size=N).astype(np.int32)
        else:
            ranks = np.full(N, rank, np.int32)
        scales = (32.0 / ranks.astype(np.float64)).astype(np.float32)
        n_hot = min(50, max(1, N // 20))
        order = _rng(seed, _TAG_POP).permutation(N)           # the first n_hot of it are the hot adapters
        draw = _rng(seed, _TAG_IDS)
        to_hot = draw.random(T) < 0.8
        pick_hot = draw.integers(0, n_hot, size=T)
        pick_cold = draw.integers(n_hot, N, size=T) if N > n_hot else pick_hot
        ids = order[np.where(to_hot, pick_hot, pick_cold)].astype(np.int32)
        meta.update(ids="80 % of requests to 50 hot adapters", n_hot=int(n_hot))
    else:  # cfg == 5
        T, N, D, L = n_tok or 2048, n_adapters or 1000, d_model or 8192, n_layers or 1
        pools = _pools(L, (0, 3), {0: (D, D), 3: (D, D)})
        if rank is None:
            ranks = _rng(seed, _TAG_RANKS).choice(np.array([8, 16, 32, 64], np.int32), size=N).astype(np.int32)
        else:
            ranks = np.full(N, rank, np.int32)
        scales = (32.0 / ranks.astype(np.float64)).astype(np.float32)
        rmix = _rng(seed, _TAG_MIX)
        half = T // 2
        lens = [1] * half
        left = T - half
        max_len = min(256, max(2, T // 8))
        while left > 0:
            n = int(rmix.integers(2, max_len + 1))
            n = min(n, left)
            lens.append(n)
            left -= n
        lens = np.array(lens, np.int64)
        rmix.shuffle(lens)
        req_ids = _zipf_ids(_rng(seed, _TAG_IDS), _rng(seed, _TAG_POP), len(lens), N, 0.8)
        ids = np.repeat(req_ids, lens).astype(np.int32)
        meta.update(ids="zipf(0.8) per request", n_requests=int(len(lens)),
                    n_decode_requests=int(half), max_prefill_len=int(max_len))

    assert ids.shape == (T,)
    return Workload(cfg=cfg, name=CONFIG_NAMES[cfg], seed=seed, n_tok=T, n_adapters=N, pools=pools,
                    ranks=ranks, scales=scales, ids=ids, meta=meta)


# --------------------------------------------------------------------------
# host (numpy) payload generators: any piece can be regenerated on its own
# --------------------------------------------------------------------------
def gen_x(wl: Workload, pool: PoolSpec) -> np.ndarray:
    """bf16 bit patterns, uint16 [n_tok, d_in]; q/k/v (and up/gate) of a layer share it."""
    r = _rng(wl.seed, _TAG_X, pool.layer, pool.x_group)
    return f32_to_bf16_bits(r.standard_normal((wl.n_tok, pool.d_in), dtype=np.float32))


def gen_y_in(wl: Workload, pool: PoolSpec) -> np.ndarray:
    """fp32 [n_tok, d_out]: stands for the base projection output the delta adds to."""
    r = _rng(wl.seed, _TAG_Y, pool.layer, pool.proj)
    return r.standard_normal((wl.n_tok, pool.d_out), dtype=np.float32)


def gen_adapter(wl: Workload, pool: PoolSpec, a: int):
    """(A bits uint16 [d_in, r_a], B bits uint16 [r_a, d_out]) of adapter `a` in `pool`."""
    r_a = int(wl.ranks[a])
    ra = _rng(wl.seed, _TAG_A, pool.layer, pool.proj, a)
    rb = _rng(wl.seed, _TAG_B, pool.layer, pool.proj, a)
    A = ra.standard_normal((pool.d_in, r_a), dtype=np.float32) * np.float32(1.0 / np.sqrt(pool.d_in))
    B = rb.standard_normal((r_a, pool.d_out), dtype=np.float32) * np.float32(1.0 / np.sqrt(r_a))
    return f32_to_bf16_bits(A), f32_to_bf16_bits(B)


# --------------------------------------------------------------------------
# device payload generator for full-size pools (tens of GB: too slow on host)
# --------------------------------------------------------------------------
def gen_pool_device(wl: Workload, pool: PoolSpec, device, fp16: bool = False):
    """Draw a whole pool on `device` with torch's seeded generator.

    Returns (A_list, B_list): per-adapter bf16 tensors, A_a [d_in, r_a] and
    B_a [r_a, d_out], row-major contiguous (views into one block per rank
    class).  Same distributions as gen_adapter; the bits differ from the host
    generator's, so a test that uses this path copies the adapters it checks
    back to the host before handing them to the oracle.
    """
    import torch

    dt = torch.float16 if fp16 else torch.bfloat16     # fp16: the same draws rounded to IEEE half instead
    g = torch.Generator(device=device)
    g.manual_seed((wl.seed * 1000003 + pool.layer * 101 + pool.proj) & 0x7FFFFFFFFFFF)
    n = wl.n_adapters
    A_list = [None] * n
    B_list = [None] * n
    for r in sorted({int(v) for v in wl.ranks}):
        idx = np.nonzero(wl.ranks == r)[0]
        cnt = len(idx)
        A_blk = torch.empty((cnt, pool.d_in, r), dtype=dt, device=device)
        B_blk = torch.empty((cnt, r, pool.d_out), dtype=dt, device=device)
        # draw in slices so the fp32 temporaries stay small
        step = max(1, (64 << 20) // max(1, pool.d_in * r, r * pool.d_out))
        for s in range(0, cnt, step):
            e = min(cnt, s + step)
            t = torch.randn((e - s, pool.d_in, r), generator=g, device=device, dtype=torch.float32)
            A_blk[s:e] = (t * (1.0 / float(np.sqrt(pool.d_in)))).to(dt)
            t = torch.randn((e - s, r, pool.d_out), generator=g, device=device, dtype=torch.float32)
            B_blk[s:e] = (t * (1.0 / float(np.sqrt(r)))).to(dt)
        for j, a in enumerate(idx):
            A_list[int(a)] = A_blk[j]
            B_list[int(a)] = B_blk[j]
    return A_list, B_list
