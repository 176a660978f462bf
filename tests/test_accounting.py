"""The byte / throughput accounting the benchmark reports, pinned to numbers the paper prints
(tests/golden/paper_accounting.txt) and to its cost-model formulas (Section VI-B, Table IV)."""
from pathlib import Path

import numpy as np

from bench import algorithmic_bytes, algorithmic_flops, hbm_floor_ms


def _golden():
    out = {}
    for line in (Path(__file__).parent / "golden" / "paper_accounting.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        name, value = [c.strip() for c in line.split("|")][:2]
        out[name] = float(value)
    return out


def test_cached_matrix_pool_size():
    g = _golden()
    # one matrix of every adapter per layer and injected weight: D * R * S bytes each
    mean_rank = np.mean([8, 16, 32, 64, 128])
    total = 7 * 4096 * mean_rank * g["value_bytes_fp16"] * 32 * 1000
    assert round(total / 1e9) == g["e4_cached_matrix_pool"]
    # the same count through the benchmark's accounting: 1000 one-token adapters, A only = half of (A + B)
    ids = np.arange(1000, dtype=np.int32)
    ranks = np.resize(np.array([8, 16, 32, 64, 128], np.int32), 1000)
    per_weight = algorithmic_bytes(ids, ranks, 4096, 4096)["adapter"] / 2
    assert abs(per_weight * 7 * 32 - total) < 1e-6 * total


def test_hbm_floor_of_a_decode_step():
    g = _golden()
    assert round(hbm_floor_ms(14e9, 3350.0), 2) == g["decode_step_7b"]
    assert round(hbm_floor_ms(26e9, 3350.0), 2) == g["decode_step_13b"]
    assert round(32 / (14e9 / 3350e9)) == g["decode_tokens_per_s_7b"]
    assert round(32 / (26e9 / 3350e9)) == g["decode_tokens_per_s_13b"]


def test_flops_follow_the_cost_model():
    # E1 compute term: 4 * sum_i B_i * D * R_i flops for square projections
    ids = np.array([0, 0, 1, 2, 2, 2], np.int32)
    ranks = np.array([8, 16, 64], np.int32)
    D = 4096
    assert algorithmic_flops(ids, ranks, D, D) == 4 * D * (2 * 8 + 1 * 16 + 3 * 64)
    b = algorithmic_bytes(ids, ranks, D, D)
    # E1 memory term: 2 * D * S * sum of the ranks of the adapters present
    assert b["adapter"] == 2 * D * 2 * (8 + 16 + 64) and b["distinct"] == 3
    assert algorithmic_bytes(np.array([-1, 1], np.int32), ranks, D, D)["y"] == 1 * D * 8
