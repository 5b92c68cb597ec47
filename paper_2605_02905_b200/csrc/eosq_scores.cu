// Entry of the score path (Remark 6.4): the centroid table shared by the score and decode kernels,
// and the hand-over to the warp-specialised tensor-core kernel.
#include <algorithm>
#include <cmath>

#include "eosq_common.cuh"

namespace eosq {

// Scale factor kappa in [8, 16) for which the fp16 roundings of kappa * centroid are, jointly, as
// close to exact as possible (searched over 4096 mantissas); with four levels the worst relative
// rounding error drops from 2.4e-4 to the 1e-6 range.
float best_table_scale(const Codebook &cb, uint16_t (&table)[16]) {
    const int levels = 1 << cb.bits;
    double best_err = 1e30;
    float best = 8.0f;
    for (int m = 0; m < 4096; ++m) {
        const float kappa = 8.0f * (1.0f + static_cast<float>(m) / 4096.0f);
        double worst = 0.0;
        for (int k = 0; k < levels; ++k) {
            const double exact = static_cast<double>(kappa) * static_cast<double>(cb.centroid[k]);
            const double got = static_cast<double>(__half2float(__float2half_rn(static_cast<float>(exact))));
            worst = std::max(worst, std::fabs(got - exact) / std::fabs(exact));
        }
        if (worst < best_err) {
            best_err = worst;
            best = kappa;
        }
    }
    for (int k = 0; k < levels; ++k) table[k] = __half_as_ushort(__float2half_rn(best * cb.centroid[k]));
    return best;
}

bool launch_scores_ws(const eosq_cache_t &cache, int bits, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const uint16_t (&table)[16], float kappa, const __half *q, int G, float scale, float *scores, int *err,
                      int sm_count, void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s);

// The kernel reads codes, norms and factors with 16-byte bulk copies and vector loads.
bool scores_tc_supported(const eosq_cache_t &cache, int bits, int n) {
    auto aligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    return bits >= 1 && bits <= 4 && n >= 128 && (n % 8) == 0 && aligned(cache.codes) && aligned(cache.norms) && aligned(cache.P) && aligned(cache.V);
}

bool launch_scores_tc(const eosq_cache_t &cache, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const Codebook &cb, const __half *q, int G, float scale, float *scores, int *err, int sm_count,
                      void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s) {
    // the table depends only on the codebook: search once per bit width
    static uint16_t tables[5][16];
    static float kappas[5] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    if (cb.bits < 1 || cb.bits > 4) return false;
    if (kappas[cb.bits] == 0.0f) kappas[cb.bits] = best_table_scale(cb, tables[cb.bits]);
    return launch_scores_ws(cache, cb.bits, heads, bph, head_stride, n, rot, tables[cb.bits], kappas[cb.bits], q, G, scale, scores, err,
                            sm_count, scratch, scratch_bytes, kernels, s);
}

}  // namespace eosq
