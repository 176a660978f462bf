"""Pins for the float64 oracle's LoRA delta: closed forms, library routines,
brute force and invariants.  Each pin is chosen so that a dropped term, wrong
index, transposed operand or wrong sign in the oracle fails at least one.

Definition pinned: y = x (W + A B) with A [D1, R], B [R, D2] (Section II-A),
delta Y = X A B (Section III-A), shrink m = x A / expand y = m B (Section V-A).
"""
import numpy as np
import pytest

import oracle
from helpers import bits_of, random_problem
from workloads import bf16_bits_to_f64, make_workload, gen_adapter, gen_x, gen_y_in

RTOL = 1e-12


def _delta(p, y_in=None, ids=None):
    return oracle.lora_delta(p["x"], p["ids"] if ids is None else ids, p["ranks"], p["scales"], p["A"], p["B"],
                             p["d_out"], y_in)


def _close(a, b, rtol=RTOL):
    scale = max(1.0, float(np.max(np.abs(b))))
    assert np.max(np.abs(np.asarray(a) - np.asarray(b))) <= rtol * scale


# -- pin 1: merged dense delta  x (s A B) with W = 0 (Section II-A) -------------
@pytest.mark.parametrize("seed", range(4))
def test_merged_dense_delta(seed):
    p = random_problem(seed, T=7, d_in=12, d_out=10, ranks=[1, 2, 3, 4])
    y = _delta(p)
    for t in range(p["T"]):
        a = int(p["ids"][t])
        dW = float(p["scales"][a]) * (p["Af"][a] @ p["Bf"][a])  # [d_in, d_out]
        _close(y[t], p["xf"][t] @ dW)


# -- pin 2: all-same-adapter batch is two library matrix products ---------------
def test_same_adapter_is_one_gemm():
    p = random_problem(11, T=9, d_in=24, d_out=16, ranks=[4, 5, 6])
    ids = np.full(p["T"], 1, np.int32)
    y = _delta(p, y_in=p["y_in"], ids=ids)
    ref = p["y_in"].astype(np.float64) + float(p["scales"][1]) * ((p["xf"] @ p["Af"][1]) @ p["Bf"][1])
    _close(y, ref)


# -- pin 3: brute force, independent loop order (j outer, i inner, k innermost) -
def test_brute_force_loops():
    p = random_problem(5, T=5, d_in=6, d_out=4, ranks=[2, 3], with_minus_one=True)
    p["ids"][0] = -1
    y = _delta(p, y_in=p["y_in"])
    for t in range(p["T"]):
        a = int(p["ids"][t])
        for j in range(p["d_out"]):
            acc = 0.0
            if a >= 0:
                for i in range(p["d_in"]):
                    for k in range(int(p["ranks"][a])):
                        acc += p["xf"][t, i] * p["Af"][a][i, k] * p["Bf"][a][k, j]
                acc *= float(p["scales"][a])
            assert abs(y[t, j] - (float(p["y_in"][t, j]) + acc)) <= 1e-12 * max(1.0, abs(acc))


# -- pin 4: closed forms --------------------------------------------------------
def test_all_ones_closed_form_tiny_config_shape():
    # x, A, B all ones: every delta element is s * d_in * r (2 * 512 * 8 = 8192)
    T, D, r, N = 3, 512, 8, 2
    x = bits_of(np.ones((T, D)))
    A = [bits_of(np.ones((D, r))) for _ in range(N)]
    B = [bits_of(np.ones((r, D))) for _ in range(N)]
    y = oracle.lora_delta(x, np.array([0, 1, 0], np.int32), np.full(N, r, np.int32), np.full(N, 2.0, np.float32),
                          A, B, D)
    assert np.all(y == 8192.0)


def test_one_hot_routes_single_element():
    # A = e_i e_k^T, B = e_k e_j^T  =>  y[t, j] += s x[t, i], nothing else moves.
    rng = np.random.default_rng(3)
    T, d_in, d_out, r = 4, 7, 9, 3
    i0, k0, j0 = 5, 2, 6
    xf = rng.integers(-8, 9, size=(T, d_in)).astype(np.float64)
    A = np.zeros((d_in, r)); A[i0, k0] = 1.0
    B = np.zeros((r, d_out)); B[k0, j0] = 1.0
    y = oracle.lora_delta(bits_of(xf), np.zeros(T, np.int32), np.array([r], np.int32), np.array([4.0], np.float32),
                          [bits_of(A)], [bits_of(B)], d_out)
    ref = np.zeros((T, d_out)); ref[:, j0] = 4.0 * xf[:, i0]
    assert np.array_equal(y, ref)


def test_asymmetric_A_B_detects_transposes():
    # Distinct small integers everywhere: a transposed A or B, or swapped d_in/d_out, changes the answer.
    d_in, r, d_out = 3, 2, 4
    xf = np.array([[1.0, 2.0, 3.0]])
    A = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]])
    B = np.array([[1.0, 2.0, 3.0, 4.0], [5.0, 6.0, 7.0, 8.0]])
    # m = [22, 28];  y = [22+140, 44+168, 66+196, 88+224]
    y = oracle.lora_delta(bits_of(xf), np.zeros(1, np.int32), np.array([r], np.int32), np.array([1.0], np.float32),
                          [bits_of(A)], [bits_of(B)], d_out)
    assert np.array_equal(y, np.array([[162.0, 212.0, 262.0, 312.0]]))
    m = oracle.shrink(bits_of(xf), np.zeros(1, np.int32), np.array([r], np.int32), [bits_of(A)])
    assert np.array_equal(m, np.array([[22.0, 28.0]]))


def test_zero_B_and_zero_scale_give_zero_delta():
    p = random_problem(2, T=6, d_in=8, d_out=8, ranks=[2, 4])
    zB = [np.zeros_like(b) for b in p["B"]]
    y = oracle.lora_delta(p["x"], p["ids"], p["ranks"], p["scales"], p["A"], zB, p["d_out"], p["y_in"])
    assert np.array_equal(y, p["y_in"].astype(np.float64))
    y = oracle.lora_delta(p["x"], p["ids"], p["ranks"], np.zeros(2, np.float32), p["A"], p["B"], p["d_out"], p["y_in"])
    assert np.array_equal(y, p["y_in"].astype(np.float64))


# -- pin 5: invariants ----------------------------------------------------------
def test_token_permutation_permutes_outputs():
    p = random_problem(8, T=11, d_in=16, d_out=8, ranks=[2, 2, 4], with_minus_one=True)
    y = _delta(p, y_in=p["y_in"])
    perm = np.random.default_rng(0).permutation(p["T"])
    y2 = oracle.lora_delta(p["x"][perm], p["ids"][perm], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"],
                           p["y_in"][perm])
    assert np.array_equal(y2, y[perm])


def test_linearity_in_x_and_scale():
    p = random_problem(9, T=6, d_in=16, d_out=8, ranks=[4, 2])
    y1 = _delta(p)
    x2 = bits_of(2.0 * p["xf"])  # doubling is exact in bf16
    y2 = oracle.lora_delta(x2, p["ids"], p["ranks"], p["scales"], p["A"], p["B"], p["d_out"])
    _close(y2, 2.0 * y1)
    y3 = oracle.lora_delta(p["x"], p["ids"], p["ranks"], 4.0 * p["scales"], p["A"], p["B"], p["d_out"])
    _close(y3, 4.0 * y1)


def test_minus_one_rows_untouched_and_other_tokens_do_not_matter():
    p = random_problem(10, T=8, d_in=8, d_out=8, ranks=[2, 2, 2], with_minus_one=True)
    p["ids"][3] = -1
    y = _delta(p, y_in=p["y_in"])
    assert np.array_equal(y[3], p["y_in"][3].astype(np.float64))
    ids2 = p["ids"].copy()
    ids2[4] = (ids2[4] + 1) % 3 if ids2[4] >= 0 else 0
    y2 = _delta(p, y_in=p["y_in"], ids=ids2)
    keep = np.arange(p["T"]) != 4
    assert np.array_equal(y2[keep], y[keep])


def test_independent_of_unused_adapters():
    p = random_problem(12, T=6, d_in=8, d_out=8, ranks=[2, 4])
    y = _delta(p)
    rng = np.random.default_rng(1)
    extra_A = rng.integers(0, 2 ** 15, size=(8, 3)).astype(np.uint16)
    extra_B = rng.integers(0, 2 ** 15, size=(3, 8)).astype(np.uint16)
    y2 = oracle.lora_delta(p["x"], p["ids"], np.append(p["ranks"], 3).astype(np.int32),
                           np.append(p["scales"], 7.0).astype(np.float32), p["A"] + [extra_A], p["B"] + [extra_B],
                           p["d_out"])
    assert np.array_equal(y, y2)


def test_shrink_then_expand_equals_delta():
    p = random_problem(13, T=9, d_in=20, d_out=12, ranks=[1, 3, 5], with_minus_one=True)
    m = oracle.shrink(p["x"], p["ids"], p["ranks"], p["A"])
    assert m.shape == (9, 5)
    for t in range(p["T"]):
        a = int(p["ids"][t])
        if a < 0:
            assert np.all(m[t] == 0)
        else:
            r = int(p["ranks"][a])
            _close(m[t, :r], p["xf"][t] @ p["Af"][a])
            assert np.all(m[t, r:] == 0)
    y = oracle.expand(m, p["ids"], p["ranks"], p["scales"], p["B"], p["d_out"], p["y_in"])
    _close(y, _delta(p, y_in=p["y_in"]))


def test_error_codes():
    p = random_problem(14, T=4, d_in=8, d_out=8, ranks=[2, 2])
    bad = p["ids"].copy(); bad[1] = 2
    with pytest.raises(oracle.OracleError) as e:
        _delta(p, ids=bad)
    assert e.value.code == oracle.ERR_BAD_ADAPTER_ID
    bad[1] = -2
    with pytest.raises(oracle.OracleError) as e:
        _delta(p, ids=bad)
    assert e.value.code == oracle.ERR_BAD_ADAPTER_ID


def test_empty_batch():
    p = random_problem(15, T=0, d_in=8, d_out=8, ranks=[2])
    assert _delta(p).shape == (0, 8)


# -- the tiny benchmark config against numpy float64 matmul ----------------------
def test_tiny_config_against_numpy():
    wl = make_workload(1)
    pool = wl.pools[0]
    x = gen_x(wl, pool)
    AB = [gen_adapter(wl, pool, a) for a in range(wl.n_adapters)]
    A = [ab[0] for ab in AB]; B = [ab[1] for ab in AB]
    y_in = gen_y_in(wl, pool)
    y = oracle.lora_delta(x, wl.ids, wl.ranks, wl.scales, A, B, pool.d_out, y_in)
    xf = bf16_bits_to_f64(x)
    for t in range(wl.n_tok):
        a = int(wl.ids[t])
        ref = y_in[t].astype(np.float64) + 2.0 * ((xf[t] @ bf16_bits_to_f64(A[a])) @ bf16_bits_to_f64(B[a]))
        _close(y[t], ref)


def test_input_conversions_match_numpy_for_every_bit_pattern():
    # both 16-bit input types widen exactly; numpy's float16 and the bf16-as-upper-half-of-fp32 view are the references
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    try:
        oracle.set_input_type(True)
        got = oracle.input_to_double(bits)
        with np.errstate(invalid="ignore"):
            want = bits.view(np.float16).astype(np.float64)
        assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
        assert np.array_equal(np.signbit(got), np.signbit(want))
    finally:
        oracle.set_input_type(False)
    got = oracle.input_to_double(bits)
    with np.errstate(invalid="ignore"):
        want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])


def test_half_inputs_reduce_to_a_matmul():
    # same-adapter batch with IEEE-half inputs == two numpy float64 products of the widened matrices
    rng = np.random.default_rng(5)
    x = rng.standard_normal((7, 40)).astype(np.float16)
    A = (rng.standard_normal((40, 5)) / 6).astype(np.float16)
    B = (rng.standard_normal((5, 24)) / 2).astype(np.float16)
    try:
        oracle.set_input_type(True)
        got = oracle.lora_delta(x.view(np.uint16), np.zeros(7, np.int32), [5], [0.5], [A.view(np.uint16)], [B.view(np.uint16)], 24)
    finally:
        oracle.set_input_type(False)
    want = 0.5 * (x.astype(np.float64) @ A.astype(np.float64)) @ B.astype(np.float64)
    assert np.max(np.abs(got - want)) <= 1e-12 * np.max(np.abs(want))
    # read as bf16 the same bits mean something else entirely
    other = oracle.lora_delta(x.view(np.uint16), np.zeros(7, np.int32), [5], [0.5], [A.view(np.uint16)], [B.view(np.uint16)], 24)
    assert np.max(np.abs(other - want)) > 1e-3 * np.max(np.abs(want))
