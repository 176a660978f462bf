"""The seeded generators: shapes, determinism, distributions' coarse statistics."""
import numpy as np
import pytest

from workloads import (bf16_bits_to_f32, bounded_zipf_pmf, f32_to_bf16_bits, gen_adapter, gen_x, make_workload)


def test_bf16_round_to_nearest_even():
    # 1 + 2^-8 is halfway between two bf16 values: ties go to the even mantissa
    vals = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], np.float32)
    back = bf16_bits_to_f32(f32_to_bf16_bits(vals))
    assert back.tolist() == [1.0, 1.0, 1.0 + 2.0 ** -6, -2.5, 0.0]
    torch = pytest.importorskip("torch")
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(f32_to_bf16_bits(x), want)


@pytest.mark.parametrize("cfg,T,N", [(1, 64, 16), (2, 256, 1000), (3, 512, 1000), (4, 16384, 1000), (5, 2048, 1000),
                                      (6, 256, 1000)])
def test_shapes_and_determinism(cfg, T, N):
    a, b = make_workload(cfg), make_workload(cfg)
    assert a.n_tok == T and a.n_adapters == N and a.ids.shape == (T,)
    assert np.array_equal(a.ids, b.ids) and np.array_equal(a.ranks, b.ranks)
    assert a.ids.min() >= 0 and a.ids.max() < N
    assert np.allclose(a.scales * a.ranks, 32.0) or cfg == 1


def test_pool_shapes():
    assert len(make_workload(2).pools) == 128
    dims = {(p.proj): (p.d_in, p.d_out) for p in make_workload(3).pools}
    assert dims[4] == (5120, 13824) and dims[6] == (13824, 5120) and dims[0] == (5120, 5120)
    assert {(p.d_in, p.d_out) for p in make_workload(5).pools} == {(8192, 8192)}


def test_zipf_distinct_count_near_expectation():
    pmf = bounded_zipf_pmf(1000, 1.0)
    expect = float(np.sum(1.0 - (1.0 - pmf) ** 256))  # about 130 distinct adapters in 256 draws
    assert 125 < expect < 135
    got = [len(make_workload(2, seed=s).distinct_adapters()) for s in range(20)]
    assert abs(np.mean(got) - expect) < 6


def test_prefill_runs_are_contiguous():
    wl = make_workload(4)
    runs = wl.ids.reshape(32, 512)
    assert np.all(runs == runs[:, :1])


def test_mixed_has_decode_and_prefill_segments():
    wl = make_workload(5)
    change = np.flatnonzero(np.diff(wl.ids)) + 1
    lens = np.diff(np.concatenate([[0], change, [wl.n_tok]]))
    assert lens.max() > 32 and (lens == 1).sum() > 100
    assert set(np.unique(wl.ranks)) == {8, 16, 32, 64}


def test_adapter_regenerates_alone_with_right_variance():
    wl = make_workload(2, n_layers=1)
    pool = wl.pools[1]
    A1, B1 = gen_adapter(wl, pool, 7)
    A2, B2 = gen_adapter(wl, pool, 7)
    assert np.array_equal(A1, A2) and np.array_equal(B1, B2)
    assert A1.shape == (4096, 16) and B1.shape == (16, 4096)
    assert abs(bf16_bits_to_f32(A1).std() * 64.0 - 1.0) < 0.02
    assert abs(bf16_bits_to_f32(B1).std() * 4.0 - 1.0) < 0.02
    assert not np.array_equal(A1, gen_adapter(wl, wl.pools[0], 7)[0])
    x = gen_x(wl, pool)
    assert np.array_equal(x, gen_x(wl, wl.pools[0]))  # q and k read the same activations
    assert not np.array_equal(x, gen_x(wl, wl.pools[3]))


def test_skewed_mix_sends_four_fifths_of_the_requests_to_fifty_adapters():
    # the paper's skewed request distribution (its workload table): 80 % of the requests go to 50 adapters
    shares = []
    for seed in range(20):
        wl = make_workload(6, n_tok=4096, seed=1000 + seed)
        counts = np.sort(np.bincount(wl.ids, minlength=wl.n_adapters))[::-1]
        shares.append(counts[:50].sum() / wl.n_tok)
        assert set(np.unique(wl.ranks)) <= {8, 16, 32, 64, 128}
        assert np.allclose(wl.scales * wl.ranks, 32.0)
    assert abs(np.mean(shares) - 0.8) < 0.01
    wl = make_workload(6)
    assert wl.n_tok == 256 and len(wl.pools) == 8 * 4 and {(p.d_in, p.d_out) for p in wl.pools} == {(4096, 4096)}
    assert set(np.unique(wl.ranks)) == {8, 16, 32, 64, 128}
