"""Shared test helpers: tiny random problems and the parity measure."""
from __future__ import annotations

import numpy as np

from workloads import bf16_bits_to_f64, f32_to_bf16_bits, f32_to_fp16_bits

# Contract: max|gpu - ref| <= 5e-3 * max|ref| (bf16 inputs, fp32 accumulation).
TOL_CONTRACT = 5e-3
# fp32 accumulation of at most ~14k bf16 products and a rank-sized second sum sits
# near 1e-6 of max|ref|; anything above 1e-4 on the fp32-m paths is an indexing bug.
TOL_FP32_PATH = 1e-4


def rel_err(got, ref) -> float:
    ref = np.asarray(ref, np.float64)
    got = np.asarray(got, np.float64)
    denom = np.max(np.abs(ref))
    if denom == 0.0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / denom)


def random_problem(seed, T, d_in, d_out, ranks, n_adapters=None, with_minus_one=False, scales=None, fp16=False):
    """Small random instance: dict with bit-pattern inputs and float64 views.  fp16: x, A and B are IEEE
    half instead of bf16 (the problem carries the flag; the oracle and the device are told by the callers)."""
    rng = np.random.default_rng(seed)
    to_bits = f32_to_fp16_bits if fp16 else f32_to_bf16_bits
    to_f64 = (lambda b: b.view(np.float16).astype(np.float64)) if fp16 else bf16_bits_to_f64
    ranks = np.asarray(ranks, np.int32)
    N = len(ranks) if n_adapters is None else n_adapters
    assert len(ranks) == N
    lo = -1 if with_minus_one else 0
    ids = rng.integers(lo, N, size=T).astype(np.int32)
    x = to_bits(rng.standard_normal((T, d_in), dtype=np.float32))
    A = [to_bits(rng.standard_normal((d_in, int(r)), dtype=np.float32) / np.float32(np.sqrt(d_in)))
         for r in ranks]
    B = [to_bits(rng.standard_normal((int(r), d_out), dtype=np.float32) / np.float32(np.sqrt(r)))
         for r in ranks]
    if scales is None:
        scales = rng.choice(np.array([0.5, 1.0, 2.0, 4.0], np.float32), size=N).astype(np.float32)
    else:
        scales = np.asarray(scales, np.float32)
    y_in = rng.standard_normal((T, d_out), dtype=np.float32)
    return dict(T=T, d_in=d_in, d_out=d_out, N=N, ranks=ranks, scales=scales, ids=ids, x=x, A=A, B=B, y_in=y_in, fp16=fp16,
                xf=to_f64(x), Af=[to_f64(a) for a in A], Bf=[to_f64(b) for b in B])


def bits_of(a64):
    """float values that are exactly representable in bf16 -> bit patterns."""
    b = f32_to_bf16_bits(np.asarray(a64, np.float32))
    assert np.array_equal(bf16_bits_to_f64(b), np.asarray(a64, np.float64)), "not bf16-representable"
    return b
