// Unit scoring on tcgen05 tensor cores (bf16, head dim 128).
#include "common.cuh"

omni_status omni_score_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_cache,
                          const int32_t* n_hist_dev, int n_hist_max, const omni_unit* units,
                          const int32_t* n_units_dev, int n_units_max, const float* w, float scale,
                          float* scores_out, float* mass_out) {
    return omni_score_simple(ctx, st, q, t, k_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max, w, scale,
                             scores_out, mass_out);
}
