"""Plain restatement of the paper's LoRA cost model (Section VI-B: the table of per-strategy cost
terms, and T_LoRA = max{T_Base, T_LoRA_dev} + T_LoRA_GPU), in the paper's notation.

Test infrastructure, like everything under oracle/: only tests may import it.  Python floats
(float64), one loop per sum, no shortcuts, so that it can be checked against the table by eye.
"""
from __future__ import annotations


def cost_terms(hw: dict, R, B, D: float, S: float, T_base: float) -> dict:
    """hw: C_GPU, W_GPU, C_dev, W_DRAM, N_dev, L_link, W_link.  R[i]: rank of adapter i.
    B[i][j]: requests of adapter i under strategy E(j+1).  Returns the three terms of every
    strategy, their sums and T_LoRA."""
    N = len(R)
    T_GPU, T_dev_cpt, T_dev_trs = [0.0] * 4, [0.0] * 4, [0.0] * 4

    def sum_BDR(j):              # sum_i B_ij * D * R_i
        return sum(B[i][j] * D * R[i] for i in range(N))

    def sum_R_present(j):        # sum of R_i over the adapters with B_ij > 0
        return sum(R[i] for i in range(N) if B[i][j] > 0)

    def used(j):
        return any(B[i][j] > 0 for i in range(N))

    if used(0):
        T_GPU[0] = max(4 * sum_BDR(0) / hw["C_GPU"], 2 * D * S * sum_R_present(0) / hw["W_GPU"])
    if used(1):
        T_GPU[1] = max(4 * sum_BDR(1) / hw["C_GPU"], 2 * hw["L_link"] + 2 * D * S * sum_R_present(1) / hw["W_link"])
    if used(2):
        T_dev_cpt[2] = max(4 * sum_BDR(2) / (hw["C_dev"] * hw["N_dev"]),
                           2 * D * S * sum_R_present(2) / (hw["W_DRAM"] * hw["N_dev"]))
        T_dev_trs[2] = 2 * hw["L_link"] + 2 * D * S * sum(B[i][2] for i in range(N)) / hw["W_link"]
    if used(3):
        T_GPU[3] = max(2 * sum_BDR(3) / hw["C_GPU"], D * S * sum_R_present(3) / hw["W_GPU"])
        T_dev_cpt[3] = max(2 * sum_BDR(3) / (hw["C_dev"] * hw["N_dev"]),
                           D * S * sum_R_present(3) / (hw["W_DRAM"] * hw["N_dev"]))
        T_dev_trs[3] = 2 * hw["L_link"] + S * sum(B[i][3] * (D + R[i]) for i in range(N)) / hw["W_link"]
    T_LoRA_GPU = sum(T_GPU)
    T_LoRA_dev = sum(T_dev_cpt) + sum(T_dev_trs)
    return dict(T_GPU=T_GPU, T_dev_cpt=T_dev_cpt, T_dev_trs=T_dev_trs, T_LoRA_GPU=T_LoRA_GPU,
                T_LoRA_dev=T_LoRA_dev, T_LoRA=max(T_base, T_LoRA_dev) + T_LoRA_GPU)
