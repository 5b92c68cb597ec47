// Host-side pure functions of the eosq library: pilot parameter, Lloyd-Max codebook,
// seeded Haar rotation, storage layout and bit accounting.  No CUDA here.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#include "eosq.h"

namespace {

// Standard normal density and the probability of an interval, tail-safe.
inline double phi_density(double x) {
    return std::isinf(x) ? 0.0 : std::exp(-0.5 * x * x) * 0.3989422804014326779;
}
inline double upper_tail(double x) { return 0.5 * std::erfc(x * 0.7071067811865475244); }
inline double interval_mass(double lo, double hi) {
    // both tails measured from the side where they are small
    if (lo >= 0.0) return upper_tail(lo) - upper_tail(hi);
    if (hi <= 0.0) return upper_tail(-hi) - upper_tail(-lo);
    return 1.0 - upper_tail(hi) - upper_tail(-lo);
}

// SplitMix64 output for a given counter (stateless form).
inline uint64_t mix64(uint64_t seed, uint64_t counter) {
    uint64_t x = seed + (counter + 1) * 0x9E3779B97F4A7C15ull;
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}
inline double to_unit(uint64_t x) { return (static_cast<double>(x >> 11) + 0.5) * 0x1.0p-53; }

}  // namespace

extern "C" int eosq_pilot_k(int d) {
    if (d < 3) return -1;
    const double ll = std::log(std::log(static_cast<double>(d)));
    double c = 1.0 / 2.01;
    if (ll > 0.0) c = std::fmin(c, 1.0 / ll);
    return static_cast<int>(std::floor(std::pow(static_cast<double>(d), c)));
}

// Lloyd's fixed point on the N(0,1) density, scaled by 1/sqrt(d) at the end.  Symmetry is
// imposed (only the positive half is iterated), which also makes the middle threshold exactly 0.
extern "C" int eosq_codebook(int bits, int d, double *centroids, double *thresholds) {
    if (bits < 1 || bits > 8 || d < 1 || centroids == nullptr) return EOSQ_ERR_INVALID_ARG;
    const int levels = 1 << bits;
    const int half = levels / 2;
    std::vector<double> pos(half), cut(half + 1);
    for (int i = 0; i < half; ++i) pos[i] = 3.0 * (i + 0.5) / half;
    for (int iter = 0; iter < 2000000; ++iter) {
        cut[0] = 0.0;
        for (int i = 1; i < half; ++i) cut[i] = 0.5 * (pos[i - 1] + pos[i]);
        cut[half] = INFINITY;
        double moved = 0.0;
        for (int i = 0; i < half; ++i) {
            const double mean = (phi_density(cut[i]) - phi_density(cut[i + 1])) / interval_mass(cut[i], cut[i + 1]);
            moved = std::fmax(moved, std::fabs(mean - pos[i]));
            pos[i] = mean;
        }
        if (moved < 1e-15) break;
    }
    const double s = 1.0 / std::sqrt(static_cast<double>(d));
    for (int i = 0; i < half; ++i) {
        centroids[half + i] = s * pos[i];
        centroids[half - 1 - i] = -s * pos[i];
    }
    if (thresholds != nullptr)
        for (int i = 0; i + 1 < levels; ++i) thresholds[i] = 0.5 * (centroids[i] + centroids[i + 1]);
    return EOSQ_OK;
}

// Orthonormalise the columns of the seeded Gaussian matrix in order (Gram-Schmidt, each
// projection done twice).  Because the diagonal of the implied R is a norm, hence positive, the
// result is the unique positive-diagonal QR factor, i.e. a Haar-distributed matrix.
extern "C" int eosq_rotation(int d, uint64_t seed, double *Pi) {
    if (d < 1 || Pi == nullptr) return EOSQ_ERR_INVALID_ARG;
    const size_t dd = static_cast<size_t>(d) * d;
    std::vector<double> col(dd);  // col[j*d + i] = A[i][j]
    for (size_t e = 0; e < dd; ++e) {
        const double u1 = to_unit(mix64(seed, 2 * e));
        const double u2 = to_unit(mix64(seed, 2 * e + 1));
        const double g = std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586477 * u2);
        col[(e % d) * d + (e / d)] = g;
    }
    for (int j = 0; j < d; ++j) {
        double *cj = &col[static_cast<size_t>(j) * d];
        for (int pass = 0; pass < 2; ++pass)
            for (int p = 0; p < j; ++p) {
                const double *cp = &col[static_cast<size_t>(p) * d];
                long double dot = 0.0L;
                for (int i = 0; i < d; ++i) dot += static_cast<long double>(cp[i]) * cj[i];
                for (int i = 0; i < d; ++i) cj[i] -= static_cast<double>(dot) * cp[i];
            }
        long double nn = 0.0L;
        for (int i = 0; i < d; ++i) nn += static_cast<long double>(cj[i]) * cj[i];
        const double inv = 1.0 / std::sqrt(static_cast<double>(nn));
        for (int i = 0; i < d; ++i) cj[i] *= inv;
    }
    for (int i = 0; i < d; ++i)
        for (int j = 0; j < d; ++j) Pi[static_cast<size_t>(i) * d + j] = col[static_cast<size_t>(j) * d + i];
    return EOSQ_OK;
}

extern "C" int eosq_layout(int n, int d, int bits, eosq_layout_t *out) {
    if (out == nullptr) return EOSQ_ERR_INVALID_ARG;
    if (d != 128 || bits < 1 || bits > 4 || n < d || n > 4096 || (n % 8) != 0) return EOSQ_ERR_UNSUPPORTED;
    std::memset(out, 0, sizeof(*out));
    out->k = eosq_pilot_k(d);
    out->rmax = EOSQ_RMAX;
    out->row_bytes = d * bits / 8;
    out->codes_bytes = static_cast<int64_t>(n) * out->row_bytes;
    out->norms_bytes = static_cast<int64_t>(n) * 2;
    out->P_bytes = static_cast<int64_t>(EOSQ_RMAX) * n * 2;
    out->V_bytes = static_cast<int64_t>(EOSQ_RMAX) * d * 2;
    out->sigma_bytes = EOSQ_RMAX * 4;
    out->phi_bytes = EOSQ_RMAX * 4;
    out->eig_bytes = static_cast<int64_t>(d) * 4;
    out->stored_bytes = out->codes_bytes + out->norms_bytes + out->P_bytes + out->V_bytes + out->phi_bytes;
    return EOSQ_OK;
}

extern "C" double eosq_bits_per_entry(int bits, double rank, int n, int d, double b_s, int prod) {
    return bits + rank * (static_cast<double>(n) + d) * b_s / (static_cast<double>(n) * d) + (prod ? 1.0 : 0.0);
}
