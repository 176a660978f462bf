// Cost model of the LoRA computation (paper Section VI-B, the table of per-strategy cost terms and
// the equation T_LoRA = max{T_Base, T_LoRA_dev} + T_LoRA_GPU).  Host arithmetic only.
#include <algorithm>

#include "plora.h"

namespace {

// Sums a strategy needs: total batch, batch-weighted ranks, batch-weighted (D + R_i), and the
// ranks of the adapters that serve at least one request under the strategy.
struct Sums {
    double b = 0, br = 0, b_d_plus_r = 0, r_present = 0;
};

}  // namespace

extern "C" PLORA_API plora_status plora_cost_model(const plora_cost_hw* hw, int32_t n_adapters, const int32_t* ranks,
                                                   const double* batch, double d, double value_bytes, double t_base,
                                                   plora_cost_terms* out) {
    if (!hw || !out || n_adapters < 0 || (n_adapters > 0 && (!ranks || !batch))) return PLORA_ERR_INVALID_ARG;
    if (!(hw->c_gpu > 0 && hw->w_gpu > 0 && hw->c_dev > 0 && hw->w_dram > 0 && hw->n_dev > 0 && hw->l_link >= 0 &&
          hw->w_link > 0 && d > 0 && value_bytes > 0 && t_base >= 0))
        return PLORA_ERR_INVALID_ARG;
    Sums s[4];
    for (int i = 0; i < n_adapters; ++i) {
        if (ranks[i] < 1) return PLORA_ERR_INVALID_ARG;
        for (int j = 0; j < 4; ++j) {
            const double b = batch[(size_t)i * 4 + j];
            if (!(b >= 0)) return PLORA_ERR_INVALID_ARG;
            s[j].b += b;
            s[j].br += b * ranks[i];
            s[j].b_d_plus_r += b * (d + ranks[i]);
            if (b > 0) s[j].r_present += ranks[i];
        }
    }
    const double S = value_bytes;
    plora_cost_terms t = {};
    // E1: both matrices cached on the GPU, which computes x A B
    if (s[0].b > 0) t.t_gpu[0] = std::max(4 * s[0].br * d / hw->c_gpu, 2 * d * S * s[0].r_present / hw->w_gpu);
    // E2: the GPU fetches both matrices over the link, then computes
    if (s[1].b > 0)
        t.t_gpu[1] = std::max(4 * s[1].br * d / hw->c_gpu, 2 * hw->l_link + 2 * d * S * s[1].r_present / hw->w_link);
    // E3: the devices compute x A B and return the result
    if (s[2].b > 0) {
        t.t_dev_cpt[2] = std::max(4 * s[2].br * d / (hw->c_dev * hw->n_dev), 2 * d * S * s[2].r_present / (hw->w_dram * hw->n_dev));
        t.t_dev_trs[2] = 2 * hw->l_link + 2 * d * S * s[2].b / hw->w_link;
    }
    // E4: one half on the GPU from one cached matrix, the other half on the devices
    if (s[3].b > 0) {
        t.t_gpu[3] = std::max(2 * s[3].br * d / hw->c_gpu, d * S * s[3].r_present / hw->w_gpu);
        t.t_dev_cpt[3] = std::max(2 * s[3].br * d / (hw->c_dev * hw->n_dev), d * S * s[3].r_present / (hw->w_dram * hw->n_dev));
        t.t_dev_trs[3] = 2 * hw->l_link + S * s[3].b_d_plus_r / hw->w_link;
    }
    for (int j = 0; j < 4; ++j) {
        t.t_lora_gpu += t.t_gpu[j];
        t.t_lora_dev += t.t_dev_cpt[j] + t.t_dev_trs[j];
    }
    t.t_lora = std::max(t_base, t.t_lora_dev) + t.t_lora_gpu;
    *out = t;
    return PLORA_OK;
}
