"""The paper's LoRA cost model (Section VI-B, table of per-strategy cost terms; T_LoRA equation).

The oracle (oracle/cost_model.py) is pinned by what the table fixes independently of any code:
hand-worked single-adapter cases in round numbers, the ratios between strategies the table
implies, which terms are zero, and scaling laws.  The library's C entry point is then compared
with the oracle on random inputs.  Host arithmetic only: no GPU involved."""
import numpy as np
import pytest

import paper_2608_05483_b200 as P
from oracle.cost_model import cost_terms

# the evaluation's hardware (paper Section VII-A, hardware table): one H100, four devices
HW = dict(C_GPU=989e12, W_GPU=3350e9, C_dev=2e12, W_DRAM=1.1e12, N_dev=4, L_link=200e-9, W_link=128e9)


def _lib_hw(hw):
    return dict(c_gpu=hw["C_GPU"], w_gpu=hw["W_GPU"], c_dev=hw["C_dev"], w_dram=hw["W_DRAM"], n_dev=hw["N_dev"],
                l_link=hw["L_link"], w_link=hw["W_link"])


def _one(strategy, batch, R=16, D=4096, hw=HW, S=2.0, T_base=0.0):
    B = [[0.0] * 4]
    B[0][strategy] = batch
    return cost_terms(hw, [R], B, D, S, T_base)


def test_hand_worked_single_adapter_in_round_numbers():
    # C = 1e12 flop/s, W = 1e9 B/s, D = 1000, R = 10, S = 2, one request under E1:
    # compute 4 * 1 * 1000 * 10 / 1e12 = 4e-8 s; memory 2 * 1000 * 2 * 10 / 1e9 = 4e-5 s
    hw = dict(C_GPU=1e12, W_GPU=1e9, C_dev=1e11, W_DRAM=1e9, N_dev=2, L_link=1e-6, W_link=1e8)
    t = _one(0, 1, R=10, D=1000, hw=hw)
    assert t["T_GPU"][0] == pytest.approx(4e-5) and t["T_LoRA"] == pytest.approx(4e-5)
    # 2000 requests: compute 4 * 2000 * 1e4 / 1e12 = 8e-5 s now exceeds the memory term
    assert _one(0, 2000, R=10, D=1000, hw=hw)["T_GPU"][0] == pytest.approx(8e-5)
    # E3, one request: devices compute max(4e4 / 2e11, 4e4 / 2e9) = 2e-5 s; return 2e-6 + 2 * 1000 * 2 / 1e8 = 4.2e-5 s
    t = _one(2, 1, R=10, D=1000, hw=hw)
    assert t["T_dev_cpt"][2] == pytest.approx(2e-5) and t["T_dev_trs"][2] == pytest.approx(4.2e-5)
    assert t["T_GPU"] == [0.0] * 4 and t["T_LoRA"] == pytest.approx(6.2e-5)
    # E4, one request: GPU half max(2e4 / 1e12, 2e4 / 1e9) = 2e-5; device half max(2e4 / 2e11, 2e4 / 2e9) = 1e-5;
    # return 2e-6 + 2 * (1000 + 10) / 1e8 = 2.22e-5; total = devices 3.22e-5 + GPU 2e-5
    t = _one(3, 1, R=10, D=1000, hw=hw)
    assert t["T_GPU"][3] == pytest.approx(2e-5) and t["T_dev_cpt"][3] == pytest.approx(1e-5)
    assert t["T_dev_trs"][3] == pytest.approx(2.22e-5) and t["T_LoRA"] == pytest.approx(5.22e-5)


def test_relations_between_strategies():
    for batch in (1, 7, 300, 5000):
        e1, e2, e3, e4 = (_one(j, batch) for j in range(4))
        # E4 keeps one of the two matrices on the GPU: exactly half of E1's GPU work and bytes
        assert e4["T_GPU"][3] == pytest.approx(e1["T_GPU"][0] / 2)
        # E3 and E4 split the same device work 2 : 1
        assert e4["T_dev_cpt"][3] == pytest.approx(e3["T_dev_cpt"][2] / 2)
        # E2 does E1's arithmetic but pays the link for the matrices: never faster than E1 while the link is slower than HBM
        assert e2["T_GPU"][1] >= e1["T_GPU"][0]
        # nothing but the GPU works under E1 and E2; the GPU is idle under E3
        assert e1["T_LoRA_dev"] == 0 and e2["T_LoRA_dev"] == 0 and e3["T_LoRA_GPU"] == 0
    # the memory argument does not grow with the batch (matrices load once per step), the compute argument does
    assert _one(0, 1)["T_GPU"][0] == _one(0, 100)["T_GPU"][0]
    crossover = HW["C_GPU"] * 2.0 / (2 * HW["W_GPU"])       # batch at which E1 turns compute-bound: S * C / (2 W)
    assert _one(0, crossover * 0.99)["T_GPU"][0] == _one(0, 1)["T_GPU"][0]
    assert _one(0, crossover * 2)["T_GPU"][0] == pytest.approx(2 * _one(0, 1)["T_GPU"][0])


def test_sums_run_over_adapters_present_and_total_overlaps_base():
    R = [8, 16, 64, 128]
    B = [[3, 0, 0, 0], [0, 0, 0, 0], [1, 0, 2, 0], [0, 0, 0, 5]]
    t = cost_terms(HW, R, B, 4096, 2.0, 0.0)
    # adapter 1 serves nobody: dropping it changes nothing; E1's bytes count ranks 8 + 64 only
    assert t == cost_terms(HW, [8, 64, 128], [B[0], B[2], B[3]], 4096, 2.0, 0.0)
    assert t["T_GPU"][0] == pytest.approx(2 * 4096 * 2.0 * (8 + 64) / HW["W_GPU"])
    assert t["T_GPU"][1] == 0 and t["T_dev_cpt"][1] == 0 and t["T_dev_trs"][1] == 0      # nobody uses E2: no latency either
    dev = t["T_LoRA_dev"]
    assert dev == pytest.approx(sum(t["T_dev_cpt"]) + sum(t["T_dev_trs"]))
    # base-model time hides device time up to its own length
    assert cost_terms(HW, R, B, 4096, 2.0, dev / 2)["T_LoRA"] == pytest.approx(t["T_LoRA"])
    assert cost_terms(HW, R, B, 4096, 2.0, 3 * dev)["T_LoRA"] == pytest.approx(3 * dev + t["T_LoRA_GPU"])
    # doubling every bandwidth and throughput and removing latency halves every term
    fast = {k: (v * 2 if k not in ("L_link", "N_dev") else v) for k, v in HW.items()}
    slow0, fast0 = dict(HW, L_link=0.0), dict(fast, L_link=0.0)
    assert cost_terms(fast0, R, B, 4096, 2.0, 0.0)["T_LoRA"] == pytest.approx(cost_terms(slow0, R, B, 4096, 2.0, 0.0)["T_LoRA"] / 2)


def test_roofline_of_the_benchmark_is_e1_memory_term():
    from bench import algorithmic_bytes
    ids = np.array([0, 0, 1, 2, 2, 2], np.int32)
    ranks = np.array([8, 16, 64], np.int32)
    counts = np.bincount(ids, minlength=3)
    t = cost_terms(dict(HW, C_GPU=1e30), list(ranks), [[float(c), 0, 0, 0] for c in counts], 4096, 2.0, 0.0)
    assert t["T_GPU"][0] * HW["W_GPU"] == pytest.approx(algorithmic_bytes(ids, ranks, 4096, 4096)["adapter"])


def test_library_matches_the_oracle():
    rng = np.random.default_rng(7)
    for _ in range(200):
        n = int(rng.integers(1, 40))
        R = rng.choice([1, 2, 8, 16, 32, 64, 128], size=n)
        B = rng.integers(0, 50, size=(n, 4)).astype(np.float64) * (rng.random((n, 4)) < 0.4)
        hw = {k: v * float(rng.uniform(0.2, 5.0)) for k, v in HW.items()}
        D, S, T_base = float(rng.choice([1024, 4096, 5120, 8192])), float(rng.choice([1, 2, 4])), float(rng.uniform(0, 1e-3))
        want = cost_terms(hw, [int(r) for r in R], B.tolist(), D, S, T_base)
        rc, got = P.plora_cost_model(_lib_hw(hw), R, B, D, S, T_base)
        assert rc == 0
        for a, b in (("t_gpu", "T_GPU"), ("t_dev_cpt", "T_dev_cpt"), ("t_dev_trs", "T_dev_trs")):
            assert got[a] == pytest.approx(want[b], rel=1e-12, abs=0)
        assert got["t_lora"] == pytest.approx(want["T_LoRA"], rel=1e-12)
        assert got["t_lora_gpu"] == pytest.approx(want["T_LoRA_GPU"], rel=1e-12)
        assert got["t_lora_dev"] == pytest.approx(want["T_LoRA_dev"], rel=1e-12)


def test_library_rejects_bad_arguments():
    hw = _lib_hw(HW)
    assert P.plora_cost_model(dict(hw, w_gpu=0.0), [8], [[1, 0, 0, 0]], 4096, 2, 0)[0] == -1
    assert P.plora_cost_model(hw, [0], [[1, 0, 0, 0]], 4096, 2, 0)[0] == -1
    assert P.plora_cost_model(hw, [8], [[-1, 0, 0, 0]], 4096, 2, 0)[0] == -1
    assert P.plora_cost_model(hw, [8], [[1, 0, 0, 0]], 0, 2, 0)[0] == -1
    rc, t = P.plora_cost_model(hw, [], np.zeros((0, 4)), 4096, 2, 1e-3)
    assert rc == 0 and t["t_lora"] == 1e-3
