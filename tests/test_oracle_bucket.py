"""Pins for the oracle's bucketing: the stable sort of tokens by adapter id and
the segment list (segment length = the per-adapter request count B_i of the
cost model, Section VI-B).  Pinned against numpy's stable argsort, Python's
sorted() on (key, index) tuples, bincount/cumsum, and structural invariants.
"""
import numpy as np
import pytest

import oracle
from workloads import make_workload


def _reference(ids, N):
    ids = np.asarray(ids, np.int32)
    T = len(ids)
    key = np.where(ids == -1, N, ids).astype(np.int64)
    perm = np.argsort(key, kind="stable").astype(np.int32)
    cap = min(T, N)
    cnt = np.bincount(ids[ids >= 0], minlength=N)
    present = np.nonzero(cnt)[0]
    n_seg = len(present)
    n_active = int((ids >= 0).sum())
    seg_adapter = np.full(cap, -1, np.int32)
    seg_adapter[:n_seg] = present
    starts = np.concatenate([[0], np.cumsum(cnt)])[:-1]
    seg_start = np.full(cap + 1, n_active, np.int32)
    seg_start[:n_seg] = starts[present]
    return perm, seg_adapter, seg_start, n_seg, n_active


def _check(ids, N):
    ids = np.asarray(ids, np.int32)
    got = oracle.bucket(ids, N)
    perm, seg_adapter, seg_start, n_seg, n_active = _reference(ids, N)
    assert np.array_equal(got["perm"], perm)
    assert np.array_equal(got["seg_adapter"], seg_adapter)
    assert np.array_equal(got["seg_start"], seg_start)
    assert got["n_seg"] == n_seg and got["n_active"] == n_active
    # independent second statement: Python sorted on (key, index)
    key = [N if v == -1 else int(v) for v in ids]
    assert list(got["perm"]) == sorted(range(len(ids)), key=lambda t: (key[t], t))
    # structure
    T = len(ids)
    assert sorted(got["perm"].tolist()) == list(range(T))
    act = ids[got["perm"][:n_active]]
    assert np.all(np.diff(act) >= 0) and np.all(act >= 0)
    assert np.all(ids[got["perm"][n_active:]] == -1)
    for k in range(n_seg):
        s, e = got["seg_start"][k], got["seg_start"][k + 1]
        assert e > s
        assert np.all(ids[got["perm"][s:e]] == got["seg_adapter"][k])
        assert np.all(np.diff(got["perm"][s:e]) > 0)  # stable: ascending token index inside a segment
    assert np.all(np.diff(got["seg_adapter"][:n_seg]) > 0)


@pytest.mark.parametrize("T", [0, 1, 31, 32, 33, 64, 256, 1000, 16384])
@pytest.mark.parametrize("N", [1, 16, 1000])
def test_random_ids(T, N):
    rng = np.random.default_rng(T * 7919 + N)
    _check(rng.integers(0, N, size=T), N)
    _check(rng.integers(-1, N, size=T), N)


def test_adversarial_sets():
    N = 37
    _check(np.full(100, 5), N)                       # all the same id
    _check(np.arange(N), N)                          # all distinct, ascending
    _check(np.arange(N)[::-1].copy(), N)             # descending
    _check(np.full(50, -1), N)                       # nobody has an adapter
    _check(np.full(9, N - 1), N)                     # last id only
    _check(np.array([N - 1, 0, -1, N - 1, 0, -1]), N)
    _check(np.array([3]), N)
    _check(np.array([], np.int32), N)
    _check(np.tile(np.array([2, 1, 0]), 40), 3)      # T > N: cap = N


def test_worked_example():
    # ids:   t=0:2  1:0  2:2  3:-1  4:0  5:1
    got = oracle.bucket(np.array([2, 0, 2, -1, 0, 1], np.int32), 4)
    assert got["perm"].tolist() == [1, 4, 5, 0, 2, 3]
    assert got["seg_adapter"].tolist() == [0, 1, 2, -1]
    assert got["seg_start"].tolist() == [0, 2, 3, 5, 5]
    assert got["n_seg"] == 3 and got["n_active"] == 5


def test_bad_ids_rejected():
    for bad in ([0, 4], [0, -2]):
        with pytest.raises(oracle.OracleError) as e:
            oracle.bucket(np.array(bad, np.int32), 4)
        assert e.value.code == oracle.ERR_BAD_ADAPTER_ID


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_benchmark_id_vectors(cfg):
    wl = make_workload(cfg)
    _check(wl.ids, wl.n_adapters)
