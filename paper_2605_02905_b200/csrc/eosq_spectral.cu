// Spectral stage of eosq_encode: symmetric eigen-decomposition of the d x d Gram matrix
// (the block's singular values and right singular vectors, Sec. 2.3) and Algorithm 2
// (bulk edge, rank, imputed noise spectrum, D-transform estimators, Frobenius shrinker).
//
// All arithmetic here is double precision: the bulk eigenvalues sit two to three orders of
// magnitude below the largest outlier, and the rank test and the shrunk values must agree with a
// double-precision reference to 1e-4 relative or better.
#include <algorithm>

#include "eosq_common.cuh"

namespace eosq {

// ------------------------------------------------------------------------------------------
// Eigenvalues of a symmetric tridiagonal matrix from Sturm sequences: with
//   p_0 = 1, p_1 = d_0 - x, p_{i+1} = (d_i - x) p_i - e_{i-1}^2 p_{i-1},
// the number of sign changes in p_0 .. p_d is the number of eigenvalues below x, and p_d(x) is the
// characteristic polynomial.  One thread per eigenvalue.  A first pass evaluates at 128 points
// spaced geometrically below the Gershgorin bound (the spectrum of a Gram matrix spans many
// decades), which brackets every eigenvalue to 18 %.  Each thread then shrinks its bracket until
// it is below 1e-8 relative (2e-15 of the matrix scale for the smallest ones): by bisection on
// the counts while the bracket holds several eigenvalues, and once it holds exactly one, by
// regula falsi on p_d (Illinois variant: an end that survives twice has its value halved), which
// needs a third of the evaluations.  The count still decides which end every new point replaces,
// so a bracket never loses its eigenvalue; a step that would fall outside it is bisected instead.
// ------------------------------------------------------------------------------------------
constexpr double EV_E2_FLOOR = 1e-60;   // keeps the recurrence alive across an exactly decoupled entry
constexpr int EV_MAX_ITER = 96;
constexpr double EV_SECANT_WIDTH = 2e-3;   // relative bracket width below which p_d is interpolated
constexpr int EV_PE_INVALID = -(1 << 28);   // exponent marking a p_d whose magnitude was lost

constexpr int EV_GROUP = 8;               // recurrence steps between two range checks
constexpr int EV_PAD = EV_GROUP;          // entries past the end that the look-ahead may read

template <bool COUNT>
__device__ __forceinline__ void sturm_step(const double2 de, double x, double &p0, double &p1, unsigned &cnt) {
    const double t = de.y * p0;
    const double p2 = fma(de.x - x, p1, -t);
    if (COUNT) cnt += static_cast<unsigned>(__double2hiint(p1) ^ __double2hiint(p2)) >> 31;
    p0 = p1;
    p1 = p2;
}

// sde[i] = (d_i, e_{i-1}^2), scaled so that every entry is at most 1 in magnitude, followed by
// EV_PAD entries that are read but not used.  Returns the count; p_d(x) = pm 2^pe.  The entries
// of the next group are fetched before the current group's chain of dependent multiply-adds
// starts, and the pair is brought back to within 2^+-300 of one after every group: eight steps
// move it by at most 2^13 upwards and, even with full cancellation in every step, 2^-424 downwards.
// Without COUNT only p_d(x) is worked out (its sign is all a bracket around a single eigenvalue needs).
template <bool COUNT = true>
__device__ __forceinline__ int sturm_eval(const double2 *__restrict__ sde, double x, double &pm, int &pe) {
    double p0 = 1.0, p1 = sde[0].x - x;
    unsigned cnt = static_cast<unsigned>(__double2hiint(p1)) >> 31;
    int esum = 0;
    constexpr int NG = (D - 1) / EV_GROUP;
    double2 cur[EV_GROUP], nxt[EV_GROUP];
#pragma unroll
    for (int i = 0; i < EV_GROUP; ++i) cur[i] = sde[1 + i];
#pragma unroll 1
    for (int g = 0; g < NG; ++g) {
        const double2 *q = sde + 1 + (g + 1) * EV_GROUP;
#pragma unroll
        for (int i = 0; i < EV_GROUP; ++i) nxt[i] = q[i];
#pragma unroll
        for (int i = 0; i < EV_GROUP; ++i) sturm_step<COUNT>(cur[i], x, p0, p1, cnt);
        const int e0 = (__double2hiint(p0) >> 20) & 0x7ff, e1 = (__double2hiint(p1) >> 20) & 0x7ff;
        const int em = max(e0, e1);
        if (static_cast<unsigned>(em - 723) > 600u) {
            if (em == 0) {   // both vanished: restart with the current sign
                p0 = 0.0;
                p1 = (__double2hiint(p1) < 0) ? -1.0 : 1.0;
                esum = EV_PE_INVALID;
            } else if (em < 2047) {
                const double sc = __hiloint2double((2046 - em) << 20, 0);   // 2^(1023 - em)
                p0 *= sc;
                p1 *= sc;
                esum += em - 1023;
            }
        }
#pragma unroll
        for (int i = 0; i < EV_GROUP; ++i) cur[i] = nxt[i];
    }
#pragma unroll
    for (int i = 0; i < (D - 1) - NG * EV_GROUP; ++i) sturm_step<COUNT>(cur[i], x, p0, p1, cnt);
    pm = p1;
    pe = esum;
    return static_cast<int>(cnt);
}

// Which eigenvalues are resolved.  Algorithm 2 reads individually only lambda_1 .. lambda_{k+r+1} and
// lambda_{2k+1}, lambda_{2k+r+1} (Steps 1 and 2; r <= k); the rest of the spectrum enters through sums
// that the spectral kernel takes from the characteristic polynomial.  The fast kernel resolves the
// EV_EXPL = 32 largest (one lane each) and, for the rare ranks 10 and 11, lambda_{2k+r+1} (index 32 or
// 33) in a second round; the full kernel resolves every eigenvalue (the optional `eig` output).
constexpr int EV_EXPL = 32;
constexpr int EV_TOP = 3 * KPILOT + 1;   // entries of lam the spectral kernel may read without the full spectrum
static_assert(2 * KPILOT + 9 < EV_EXPL && EV_TOP <= EV_EXPL + 2, "ranks up to 9 find lambda_{2k+r+1} among the first 32");

// With `mark_list` set (first pass over tensor-core Gram matrices), a block whose smallest
// eigenvalue is not at least REDO_RATIO of the largest (this includes non-finite spectra) is queued
// in mark_list[atomicAdd(mark_count)] for a second pass with the exact Gram matrix.
// This is the full-spectrum kernel (D threads, thread t resolves lambda_{t+1}); it serves caches that
// ask for the `eig` output.
__device__ __forceinline__ void eigvals_block(const double *__restrict__ diag, const double *__restrict__ off,
                                              double *__restrict__ lam, int blk, int *__restrict__ mark_list,
                                              int *__restrict__ mark_count) {
    constexpr int NT = D, NWARP = NT / 32, PER = 1;
    __shared__ __align__(16) double2 sde[D + EV_PAD];
    __shared__ double s_e2[D];
    __shared__ double s_red[3][4];
    __shared__ int s_cnt[D], s_pe[D];
    __shared__ double s_pm[D];
    const int tid = threadIdx.x;
    const size_t base = static_cast<size_t>(blk) * D;
    // every thread loads PER rows of the tridiagonal matrix: rows tid, tid + NT, ..
    double dv[PER], ev[PER];
    double m = 0.0;
    bool nonfinite = false;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        const int i = tid + NT * q;
        dv[q] = diag[base + i];
        ev[q] = (i < D - 1) ? off[base + i] : 0.0;
        m = fmax(m, fmax(fabs(dv[q]), fabs(ev[q])));
        nonfinite |= !(fabs(dv[q]) < 1e300) || !(fabs(ev[q]) < 1e300);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) s_red[0][tid >> 5] = m;
    // a non-finite entry anywhere poisons the whole spectrum: report NaN instead of a bracket
    const int bad = __syncthreads_or(nonfinite);
    if (bad) {
#pragma unroll
        for (int q = 0; q < PER; ++q) lam[base + tid + NT * q] = nan("");
        if (mark_list && tid == 0) mark_list[atomicAdd(mark_count, 1)] = blk;
        return;
    }
    m = s_red[0][0];
#pragma unroll
    for (int w = 1; w < NWARP; ++w) m = fmax(m, s_red[0][w]);
    if (m == 0.0) {
#pragma unroll
        for (int q = 0; q < PER; ++q) lam[base + tid + NT * q] = 0.0;
        return;
    }
    const double scale = 1.0 / m;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        const int i = tid + NT * q;
        const double se = fabs(ev[q] * scale);
        s_e2[i] = (i < D - 1) ? fmax(se * se, EV_E2_FLOOR) : 0.0;
    }
    __syncthreads();
    // Gershgorin bounds of the scaled matrix
    double glo = 1e300, ghi = -1e300;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        const int i = tid + NT * q;
        const double sd = dv[q] * scale, se = fabs(ev[q] * scale);
        const double se_prev = (i > 0) ? fabs(off[base + i - 1] * scale) : 0.0;
        sde[i] = make_double2(sd, (i > 0) ? s_e2[i - 1] : 0.0);
        glo = fmin(glo, sd - se - se_prev);
        ghi = fmax(ghi, sd + se + se_prev);
    }
    if (tid < EV_PAD) sde[D + tid] = make_double2(0.0, 0.0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        glo = fmin(glo, __shfl_xor_sync(0xffffffffu, glo, o));
        ghi = fmax(ghi, __shfl_xor_sync(0xffffffffu, ghi, o));
    }
    if ((tid & 31) == 0) {
        s_red[1][tid >> 5] = glo;
        s_red[2][tid >> 5] = ghi;
    }
    __syncthreads();
    glo = s_red[1][0];
    ghi = s_red[2][0];
#pragma unroll
    for (int w = 1; w < NWARP; ++w) {
        glo = fmin(glo, s_red[1][w]);
        ghi = fmax(ghi, s_red[2][w]);
    }
    glo -= 1e-10 * (fabs(glo) + 1.0);
    ghi += 1e-10 * (fabs(ghi) + 1.0);

    // first pass: counts at D points, geometric below ghi when ghi > 0 (nine decades), else uniform
    const bool geometric = ghi > 0.0;
    auto point = [&](int t) -> double {
        if (t < 0) return glo;
        if (geometric) return ghi * exp2(-(9.0 * 3.321928094887362 / (D - 1)) * static_cast<double>(D - 1 - t));
        return glo + (ghi - glo) * static_cast<double>(t + 1) / static_cast<double>(D);
    };
#pragma unroll 1
    for (int q = 0; q < PER; ++q) {
        const int i = tid + NT * q;
        double pm;
        int pe;
        s_cnt[i] = sturm_eval(sde, point(i), pm, pe);
        s_pm[i] = pm;
        s_pe[i] = pe;
    }
    __syncthreads();
    // ascending index of the eigenvalue this thread brackets, and where it goes
    const bool active = true;
    const int slot = tid;   // descending position in lam
    const int target = D - 1 - slot;
    int t = -1;                      // largest grid index with count <= target
#pragma unroll
    for (int step = D / 2; step > 0; step >>= 1)
        if (t + step < D && s_cnt[t + step] <= target) t += step;
    double lo = point(t), hi = (t + 1 < D) ? point(t + 1) : ghi;
    if (t == D - 1) lo = hi;   // cannot happen (every eigenvalue is below the last point); keeps the bracket sane
    // counts and p_d at both ends (ends that are not grid points carry no value).  flo / fhi steer
    // the interpolation and may be halved (Illinois); tlo / thi stay the true values.
    int clo = (t >= 0) ? s_cnt[t] : 0, chi = (t + 1 < D) ? s_cnt[t + 1] : D;
    double flo = (t >= 0) ? s_pm[t] : 0.0, fhi = (t + 1 < D) ? s_pm[t + 1] : 0.0;
    double tlo = flo, thi = fhi;
    int elo = (t >= 0) ? s_pe[t] : EV_PE_INVALID, ehi = (t + 1 < D) ? s_pe[t + 1] : EV_PE_INVALID;
    int replaced = 0;   // +1: the last point became hi, -1: it became lo
    int poor = 0;
    for (int it = 0; it < EV_MAX_ITER; ++it) {
        const double mid = 0.5 * (lo + hi);
        const bool done = !active || (hi - lo) <= fmax(2e-15, 1e-8 * fabs(mid));
        if (__all_sync(0xffffffffu, done)) break;
        double x = mid;
        // p_d varies like x^d over a wide bracket, far from linear: interpolate only in a narrow one
        if (chi - clo == 1 && poor < 3 && (hi - lo) <= EV_SECANT_WIDTH * fabs(mid) && elo > EV_PE_INVALID / 2 &&
            ehi > EV_PE_INVALID / 2 && flo != 0.0) {
            const double r = scalbn(fhi / flo, max(-2000, min(2000, ehi - elo)));   // p_d(hi) / p_d(lo), negative
            if (r < 0.0) {
                const double xs = lo + (hi - lo) / (1.0 - r);
                if (xs > lo && xs < hi) x = xs;
            }
        }
        const bool secant = x != mid;
        const double width = hi - lo;
        double pm;
        int pe;
        const int c = sturm_eval(sde, x, pm, pe);
        if (c > target) {
            hi = x;
            chi = c;
            fhi = pm;
            thi = pm;
            ehi = pe;
            if (secant && replaced > 0) flo *= 0.5;
            replaced = 1;
        } else {
            lo = x;
            clo = c;
            flo = pm;
            tlo = pm;
            elo = pe;
            if (secant && replaced < 0) fhi *= 0.5;
            replaced = -1;
        }
        poor = (hi - lo > 0.5 * width) ? poor + 1 : 0;   // three steps in a row that fail to halve the bracket force a bisection
    }
    // The bracket is 1e-8 wide; one more interpolation of p_d between its ends (no further
    // evaluation) lands within the square of that of the root, which the spectral kernel's
    // sums near a kept eigenvalue need.
    double xr = 0.5 * (lo + hi);
    if (chi - clo == 1 && elo > EV_PE_INVALID / 2 && ehi > EV_PE_INVALID / 2 && tlo != 0.0) {
        const double r = scalbn(thi / tlo, max(-2000, min(2000, ehi - elo)));
        if (r < 0.0) {
            const double xs = lo + (hi - lo) / (1.0 - r);
            if (xs >= lo && xs <= hi) xr = xs;
        }
    }
    const double evv = xr * m;
    if (active) lam[base + slot] = evv;
    if (mark_list) {   // uniform over the CTA
        if (tid == 0) s_red[0][0] = evv;   // the largest eigenvalue
        __syncthreads();
        if (slot == D - 1 && active && !(evv >= REDO_RATIO * s_red[0][0])) mark_list[atomicAdd(mark_count, 1)] = blk;
    }
}

__global__ void __launch_bounds__(D) eigvals_kernel(const double *__restrict__ diag, const double *__restrict__ off,
                                                               double *__restrict__ lam, const int *__restrict__ list,
                                                               const int *__restrict__ count, int *__restrict__ mark_list,
                                                               int *__restrict__ mark_count) {
    // without a list: block blockIdx.x; with one: the listed blocks, shared out over the grid
    for (int li = blockIdx.x; !list || li < *count; li += gridDim.x) {
        eigvals_block(diag, off, lam, list ? list[li] : li, mark_list, mark_count);
        if (!list) break;
        __syncthreads();   // the shared state is reused by the next listed block
    }
}

// ------------------------------------------------------------------------------------------
// The fast eigenvalue kernel: one warp per block, lane t resolves lambda_{t+1}.  Same method as
// above (first pass on a geometric grid, here of 64 points; bisection on Sturm counts; regula falsi
// on p_d once a bracket holds one eigenvalue), with two savings: while every lane of the warp
// interpolates, the evaluations skip the sign counting (the sign of p_d tells the side), and nothing
// beyond the 32 largest eigenvalues is resolved unless the rank turns out to be 10 or 11.
// ------------------------------------------------------------------------------------------
constexpr int EVT_WARPS = 4;     // blocks per CTA
constexpr int EVT_GRID = 64;     // points of the first pass

struct EvtShared {
    double2 sde[D + EV_PAD];
    double pm[EVT_GRID];
    int cnt[EVT_GRID], pe[EVT_GRID];
};

// Shrinks the bracket of the eigenvalue with ascending index `target` (lanes with active = false only
// keep the warp's evaluations company) and returns the polished root, in the scaled units of sde.
__device__ __forceinline__ double evt_refine(const EvtShared &sh, int target, bool active, double glo, double ghi, bool geometric) {
    auto point = [&](int t) -> double {
        if (t < 0) return glo;
        if (geometric) return ghi * exp2(-(9.0 * 3.321928094887362 / (EVT_GRID - 1)) * static_cast<double>(EVT_GRID - 1 - t));
        return glo + (ghi - glo) * static_cast<double>(t + 1) / static_cast<double>(EVT_GRID);
    };
    int t = -1;                      // largest grid index with count <= target
#pragma unroll
    for (int step = EVT_GRID / 2; step > 0; step >>= 1)
        if (t + step < EVT_GRID && sh.cnt[t + step] <= target) t += step;
    double lo = point(t), hi = (t + 1 < EVT_GRID) ? point(t + 1) : ghi;
    if (t == EVT_GRID - 1) lo = hi;
    int clo = (t >= 0) ? sh.cnt[t] : 0, chi = (t + 1 < EVT_GRID) ? sh.cnt[t + 1] : D;
    double flo = (t >= 0) ? sh.pm[t] : 0.0, fhi = (t + 1 < EVT_GRID) ? sh.pm[t + 1] : 0.0;
    double tlo = flo, thi = fhi;
    int elo = (t >= 0) ? sh.pe[t] : EV_PE_INVALID, ehi = (t + 1 < EVT_GRID) ? sh.pe[t + 1] : EV_PE_INVALID;
    int replaced = 0, poor = 0;
    for (int it = 0; it < EV_MAX_ITER; ++it) {
        const double mid = 0.5 * (lo + hi);
        const bool done = !active || (hi - lo) <= fmax(2e-15, 1e-8 * fabs(mid));
        if (__all_sync(0xffffffffu, done)) break;
        double x = mid;
        const bool single = chi - clo == 1 && elo > EV_PE_INVALID / 2 && ehi > EV_PE_INVALID / 2 && tlo != 0.0 && thi != 0.0;
        if (single && poor < 3 && (hi - lo) <= EV_SECANT_WIDTH * fabs(mid)) {
            const double r = scalbn(fhi / flo, max(-2000, min(2000, ehi - elo)));   // p_d(hi) / p_d(lo), negative
            if (r < 0.0) {
                const double xs = lo + (hi - lo) / (1.0 - r);
                if (xs > lo && xs < hi) x = xs;
            }
        }
        const bool secant = x != mid;
        const double width = hi - lo;
        double pmv;
        int pev, c;
        // a lane that is done or holds a single eigenvalue with both end values can do without the count
        if (__all_sync(0xffffffffu, done || single)) {
            sturm_eval<false>(sh.sde, x, pmv, pev);
            const bool same_as_lo = (__double2hiint(pmv) < 0) == (__double2hiint(tlo) < 0);
            c = (pev > EV_PE_INVALID / 2 && pmv != 0.0) ? (same_as_lo ? clo : chi) : chi;
            if (!(pev > EV_PE_INVALID / 2 && pmv != 0.0)) c = sturm_eval<true>(sh.sde, x, pmv, pev);   // the value was lost: count after all
        } else {
            c = sturm_eval<true>(sh.sde, x, pmv, pev);
        }
        if (c > target) {
            hi = x;
            chi = c;
            fhi = pmv;
            thi = pmv;
            ehi = pev;
            if (secant && replaced > 0) flo *= 0.5;
            replaced = 1;
        } else {
            lo = x;
            clo = c;
            flo = pmv;
            tlo = pmv;
            elo = pev;
            if (secant && replaced < 0) fhi *= 0.5;
            replaced = -1;
        }
        poor = (hi - lo > 0.5 * width) ? poor + 1 : 0;
    }
    double xr = 0.5 * (lo + hi);
    if (chi - clo == 1 && elo > EV_PE_INVALID / 2 && ehi > EV_PE_INVALID / 2 && tlo != 0.0) {
        const double r = scalbn(thi / tlo, max(-2000, min(2000, ehi - elo)));
        if (r < 0.0) {
            const double xs = lo + (hi - lo) / (1.0 - r);
            if (xs >= lo && xs <= hi) xr = xs;
        }
    }
    return xr;
}

__global__ void __launch_bounds__(32 * EVT_WARPS) eigvals_top_kernel(const double *__restrict__ diag, const double *__restrict__ off,
                                                                     double *__restrict__ lam, int nb, const int *__restrict__ list,
                                                                     const int *__restrict__ count, int *__restrict__ mark_list,
                                                                     int *__restrict__ mark_count) {
    __shared__ __align__(16) EvtShared shs[EVT_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    EvtShared &sh = shs[warp];
    const int total = list ? *count : nb;
    for (int li = blockIdx.x * EVT_WARPS + warp; li < total; li += gridDim.x * EVT_WARPS) {
        const int blk = list ? list[li] : li;
        const size_t base = static_cast<size_t>(blk) * D;
        double dv[4], ev[4], m = 0.0;
        bool nonfinite = false;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lane + 32 * q;
            dv[q] = diag[base + i];
            ev[q] = (i < D - 1) ? off[base + i] : 0.0;
            m = fmax(m, fmax(fabs(dv[q]), fabs(ev[q])));
            nonfinite |= !(fabs(dv[q]) < 1e300) || !(fabs(ev[q]) < 1e300);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (__any_sync(0xffffffffu, nonfinite) || m == 0.0) {
            // a non-finite entry poisons the whole spectrum (NaN, and a second pass if there is one); a zero matrix has a zero spectrum
            const bool bad = m != 0.0;
            lam[base + lane] = bad ? nan("") : 0.0;
            if (lane < 2) lam[base + EV_EXPL + lane] = bad ? nan("") : 0.0;
            if (bad && mark_list && lane == 0) mark_list[atomicAdd(mark_count, 1)] = blk;
            continue;
        }
        const double scale = 1.0 / m;
        __syncwarp();   // the previous block's last reads of sde are over
        double glo = 1e300, ghi = -1e300;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int i = lane + 32 * q;
            const double sd = dv[q] * scale, se = fabs(ev[q] * scale);
            double se_prev = __shfl_up_sync(0xffffffffu, se, 1);
            if (lane == 0) se_prev = (q > 0) ? fabs(off[base + i - 1] * scale) : 0.0;
            sh.sde[i] = make_double2(sd, (i > 0) ? fmax(se_prev * se_prev, EV_E2_FLOOR) : 0.0);
            glo = fmin(glo, sd - se - se_prev);
            ghi = fmax(ghi, sd + se + se_prev);
        }
        if (lane < EV_PAD) sh.sde[D + lane] = make_double2(0.0, 0.0);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            glo = fmin(glo, __shfl_xor_sync(0xffffffffu, glo, o));
            ghi = fmax(ghi, __shfl_xor_sync(0xffffffffu, ghi, o));
        }
        glo -= 1e-10 * (fabs(glo) + 1.0);
        ghi += 1e-10 * (fabs(ghi) + 1.0);
        __syncwarp();
        const bool geometric = ghi > 0.0;
#pragma unroll 1
        for (int q = 0; q < EVT_GRID / 32; ++q) {
            const int t = lane + 32 * q;
            const double x = geometric ? ghi * exp2(-(9.0 * 3.321928094887362 / (EVT_GRID - 1)) * static_cast<double>(EVT_GRID - 1 - t))
                                       : glo + (ghi - glo) * static_cast<double>(t + 1) / static_cast<double>(EVT_GRID);
            double pmv;
            int pev;
            sh.cnt[t] = sturm_eval<true>(sh.sde, x, pmv, pev);
            sh.pm[t] = pmv;
            sh.pe[t] = pev;
        }
        __syncwarp();
        const double xs = evt_refine(sh, D - 1 - lane, true, glo, ghi, geometric);
        lam[base + lane] = xs * m;
        // Is the smallest eigenvalue below REDO_RATIO of the largest?  One count tells.
        const double x_top = __shfl_sync(0xffffffffu, xs, 0);
        if (mark_list) {
            double pmv;
            int pev;
            const int below = sturm_eval<true>(sh.sde, REDO_RATIO * x_top, pmv, pev);
            if (lane == 0 && (below > 0 || !(x_top > 0.0))) mark_list[atomicAdd(mark_count, 1)] = blk;
        }
        // Ranks 10 and 11 make Step 2 read lambda_{2k+r+1}, index 32 or 33: resolve both then.
        const double edge_c = 1.0 / (cbrt(4.0) - 1.0);
        const double l_k = __shfl_sync(0xffffffffu, xs, KPILOT), l_2k = __shfl_sync(0xffffffffu, xs, 2 * KPILOT);
        const double lam_plus = l_k + edge_c * (l_k - l_2k);
        const unsigned passing = __ballot_sync(0xffffffffu, lane <= KPILOT && (xs / lam_plus - 1.0 > 1.0 / cbrt(static_cast<double>(D))));
        if (__popc(passing) >= 10) {
            const double x2 = evt_refine(sh, D - 1 - (EV_EXPL + (lane & 1)), lane < 2, glo, ghi, geometric);
            if (lane < 2) lam[base + EV_EXPL + lane] = x2 * m;
        }
    }
}

// 1 / x to about 2^-80 relative: the hardware's 20-bit estimate and two Newton steps.  Shorter than
// the full division, which sits on the critical path of the factorisation; x is a clamped pivot,
// far from the subnormal range the estimate flushes.
__device__ __forceinline__ double sp_rcp(double x) {
    double r;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
    double e = fma(-x, r, 1.0);
    r = fma(r, e, r);
    e = fma(-x, r, 1.0);
    return fma(r, e, r);
}

// Sums over the whole spectrum from the characteristic polynomial p(x) = det(T - x I) and its first
// two derivatives, by the three-term recurrences
//   p_{i+1} = (d_i - x) p_i - e_{i-1}^2 p_{i-1},   p'_{i+1} = (d_i - x) p'_i - p_i - e_{i-1}^2 p'_{i-1},
//   p''_{i+1} = (d_i - x) p''_i - 2 p'_i - e_{i-1}^2 p''_{i-1}:
//   s1 = sum_j 1 / (lambda_j - x) = -p'/p,   s2 = sum_j 1 / (lambda_j - x)^2 = (p'/p)^2 - p''/p.
// sde[i] = (d_i, e_{i-1}^2) as for the Sturm counts.  The six running values are brought back to
// within range together after every group of eight rows (the ratios do not change).
__device__ __forceinline__ void charpoly_sums(const double2 *__restrict__ sde, double x, double &s1, double &s2) {
    double p0 = 1.0, p1 = sde[0].x - x, q0 = 0.0, q1 = -1.0, r0 = 0.0, r1 = 0.0;
    auto row = [&](int i) {
        const double2 de = sde[i];
        const double t = de.x - x;
        const double p2 = fma(t, p1, -de.y * p0);
        const double q2 = fma(t, q1, fma(-de.y, q0, -p1));
        const double r2 = fma(t, r1, fma(-de.y, r0, -2.0 * q1));
        p0 = p1;
        p1 = p2;
        q0 = q1;
        q1 = q2;
        r0 = r1;
        r1 = r2;
    };
    auto rescale = [&]() {
        const int e0 = (__double2hiint(p0) >> 20) & 0x7ff, e1 = (__double2hiint(p1) >> 20) & 0x7ff;
        const int em = max(e0, e1);
        if (em > 0 && em < 2047) {
            const double sc = __hiloint2double((2046 - em) << 20, 0);   // 2^(1023 - em)
            p0 *= sc;
            p1 *= sc;
            q0 *= sc;
            q1 *= sc;
            r0 *= sc;
            r1 *= sc;
        }
    };
    constexpr int NG = (D - 1) / 8;
#pragma unroll 1
    for (int g = 0; g < NG; ++g) {
#pragma unroll
        for (int i = 0; i < 8; ++i) row(1 + 8 * g + i);
        rescale();
    }
#pragma unroll
    for (int i = 1 + 8 * NG; i < D; ++i) row(i);
    const double ip = sp_rcp(p1);
    s1 = -q1 * ip;
    s2 = fma(s1, s1, -r1 * ip);
}

// ------------------------------------------------------------------------------------------
// Algorithm 2 on the spectrum, then the kept eigenvectors from the twisted factorisation of the
// tridiagonal matrix and back-transformation through the stored reflectors.
// ------------------------------------------------------------------------------------------
//
// Every phase here is a chain of dependent latencies (a pivot after a pivot, a reflector after a
// reflector) that leaves most of the CTA idle, so the kernel is laid out for four CTAs of four warps
// per SM, whose chains overlap (measured: 3.4 / 2.4 / 1.9 ms at two / three / four CTAs per SM).
// Shared memory (33 KB: 12 columns of factor storage - the rank never exceeds the pilot k = 11 - in
// two arrays that the vectors and the reflector stages take over in turn) would allow six, but the
// 80 or 90 registers per thread that five or six CTAs leave cost more than the extra CTAs bring
// (2.5 ms against 1.8 ms).
constexpr int SP_THREADS = 128, SP_WARPS = SP_THREADS / 32;
constexpr int FAC_LANES = 12;
static_assert(KPILOT < FAC_LANES && KPILOT <= 3 * SP_WARPS, "one factor column and one warp slot per kept vector");

// Back-transformation x = H_0 H_1 ... H_{D-3} y of the kept vectors, normalisation, and the stores of
// the right singular vectors.  The reflectors (rows of R, 1 KB each) are staged through shared memory
// by the CTA's last warp, six rows per stage and two stages, handed over with named barriers.
// The other three warps apply them: a group of eight lanes owns one vector (sixteen entries per
// lane: rows 16 m + 2 sub, + 1), so a dot product needs three shuffle stages and four vectors share
// every instruction.  Reflector k is zero up to index k, and whole 16-row chunks of zeros are skipped.
constexpr int BT_ROWS = 6;                  // reflector rows per stage: two stages fill one factor array
static_assert((D - 2) % BT_ROWS == 0 && 2 * BT_ROWS * D <= D * FAC_LANES, "the stages take the place of the second factor array");
// dynamic shared memory: two arrays [D][12].  The first holds e_i / D+_i and then, in place, the vectors;
// the second D+_i, then e_i / D-_{i+1}, then the two reflector stages.
constexpr size_t SPECTRAL_DYN_SMEM = sizeof(double) * 2 * D * FAC_LANES;
constexpr int BT_BAR_FULL = 2, BT_BAR_EMPTY = 4;   // named barriers: + stage


// (barrier numbers are spelled out: a number in a register makes the compiler reserve all sixteen)
__device__ __forceinline__ void bt_bar_sync(int id) {
    if (id == 2) asm volatile("bar.sync 2, 128;" ::: "memory");
    else if (id == 3) asm volatile("bar.sync 3, 128;" ::: "memory");
    else if (id == 4) asm volatile("bar.sync 4, 128;" ::: "memory");
    else asm volatile("bar.sync 5, 128;" ::: "memory");
}
__device__ __forceinline__ void bt_bar_arrive(int id) {
    if (id == 2) asm volatile("bar.arrive 2, 128;" ::: "memory");
    else if (id == 3) asm volatile("bar.arrive 3, 128;" ::: "memory");
    else if (id == 4) asm volatile("bar.arrive 4, 128;" ::: "memory");
    else asm volatile("bar.arrive 5, 128;" ::: "memory");
}

__device__ __forceinline__ void sp_back_transform(const double *__restrict__ R, const double *__restrict__ tt,
                                                  const double *__restrict__ yv, double *__restrict__ ring, int rank, int warp,
                                                  int lane, float *__restrict__ vr, const eosq_cache_t &out, long long gb) {
    constexpr int NSTAGE = (D - 2 + BT_ROWS - 1) / BT_ROWS;
    double2 *ring2 = reinterpret_cast<double2 *>(ring);
    if (warp == SP_WARPS - 1) {
        // producer: rows klo .. khi of R are contiguous in global memory
        const double2 *R2 = reinterpret_cast<const double2 *>(R);
#pragma unroll 1
        for (int j = 0; j < NSTAGE; ++j) {
            const int st = j & 1;
            const int khi = D - 3 - BT_ROWS * j, klo = max(khi - (BT_ROWS - 1), 0);
            const int cnt2 = (khi - klo + 1) * (D / 2);
            if (j >= 2) bt_bar_sync(BT_BAR_EMPTY + st);
            const double2 *src = R2 + static_cast<size_t>(klo) * (D / 2);
            double2 *dst = ring2 + st * (BT_ROWS * D / 2);
#pragma unroll 1
            for (int e0 = 0; e0 < cnt2; e0 += 32 * 8) {
                double2 v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int e = e0 + 32 * q + lane;
                    v[q] = (e < cnt2) ? __ldg(src + e) : make_double2(0.0, 0.0);
                }
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const int e = e0 + 32 * q + lane;
                    if (e < cnt2) dst[e] = v[q];
                }
            }
            bt_bar_arrive(BT_BAR_FULL + st);
        }
        return;
    }
    const int grp = lane >> 3, sub = lane & 7;
    const int vi = 4 * warp + grp;
    const bool live = vi < rank;
    double y[16];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
        y[2 * m] = live ? yv[(16 * m + 2 * sub) * FAC_LANES + vi] : 0.0;
        y[2 * m + 1] = live ? yv[(16 * m + 2 * sub + 1) * FAC_LANES + vi] : 0.0;
    }
#pragma unroll 1
    for (int j = 0; j < NSTAGE; ++j) {
        const int st = j & 1;
        const int khi = D - 3 - BT_ROWS * j, klo = max(khi - (BT_ROWS - 1), 0);
        bt_bar_sync(BT_BAR_FULL + st);
        if (4 * warp < rank) {   // a warp without vectors only keeps the barriers going
            const double2 *stage = ring2 + st * (BT_ROWS * D / 2);
#pragma unroll 1
            for (int k = khi; k >= klo; --k) {
                const double2 *urow = stage + (k - klo) * (D / 2) + sub;
                const int m0 = (k + 1) >> 4;   // chunks below it hold only zeros of the reflector
                double2 u[8];
                double d0 = 0.0, d1 = 0.0;
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    if (m >= m0) {
                        u[m] = urow[8 * m];
                        d0 = fma(u[m].x, y[2 * m], d0);
                        d1 = fma(u[m].y, y[2 * m + 1], d1);
                    }
                }
                double dot = d0 + d1;
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                const double g = tt[k] * dot;
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    if (m >= m0) {
                        y[2 * m] = fma(-g, u[m].x, y[2 * m]);
                        y[2 * m + 1] = fma(-g, u[m].y, y[2 * m + 1]);
                    }
                }
            }
        }
        if (j + 2 < NSTAGE) bt_bar_arrive(BT_BAR_EMPTY + st);
    }
    double nn = 0.0;
#pragma unroll
    for (int e = 0; e < 16; ++e) nn = fma(y[e], y[e], nn);
    nn += __shfl_xor_sync(0xffffffffu, nn, 1);
    nn += __shfl_xor_sync(0xffffffffu, nn, 2);
    nn += __shfl_xor_sync(0xffffffffu, nn, 4);
    const double rn = (nn > 0.0) ? rsqrt(nn) : 0.0;
    if (live) {
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            const int jrow = 16 * m + 2 * sub;
            const float f0 = static_cast<float>(y[2 * m] * rn), f1 = static_cast<float>(y[2 * m + 1] * rn);
            *reinterpret_cast<float2 *>(vr + vi * D + jrow) = make_float2(f0, f1);
            *reinterpret_cast<uint32_t *>(out.V + (gb * RMAX + vi) * D + jrow) =
                static_cast<uint32_t>(__half_as_ushort(__float2half_rn(f0))) | (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(f1))) << 16);
            if (out.vr32) *reinterpret_cast<float2 *>(out.vr32 + (gb * RMAX + vi) * D + jrow) = make_float2(f0, f1);
        }
    }
}

__global__ void __launch_bounds__(SP_THREADS, 4) spectral_kernel(int n, Workspace ws, eosq_cache_t out, long long block0, bool full) {
    __shared__ double lam[D], dd[D], ee[D], tt[D], atoms[D];
    __shared__ __align__(16) double2 sde[D];  // (d_i, e_{i-1}^2) of the scaled matrix, for the characteristic polynomial
    __shared__ double st1[6 * KPILOT], st2[6 * KPILOT];   // weighted samples of the tail sums around each kept eigenvalue
    __shared__ double s_max[SP_WARPS];
    __shared__ double s_phi[RMAX], s_sig[RMAX];
    __shared__ unsigned s_flags;
    extern __shared__ double dyn[];
    double *yv = dyn;                        // e_i / D+_i, then the vectors                       [D][12]
    double *fb = dyn + D * FAC_LANES;         // D+_i, then e_i / D-_{i+1}                          [D][12]
    double *ring = dyn + D * FAC_LANES;       // the back-transformation's reflector stages take the place of fb

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const long long gb = block0 + b;
    const size_t base = static_cast<size_t>(b) * D;
    {
        // lam[EV_TOP .. D-2] holds eigenvalues only when the full spectrum was asked for
        lam[tid] = (full || tid < EV_TOP) ? ws.lam[base + tid] : 0.0;   // (indices 32, 33: only meaningful, and only read, for ranks 10, 11)
        dd[tid] = ws.diag[base + tid];
        ee[tid] = ws.off[base + tid];
        tt[tid] = ws.tau[base + tid];
        double mx = fmax(fabs(dd[tid]), fabs(ee[tid]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) s_max[warp] = mx;
    }
    if (tid < RMAX) {
        s_phi[tid] = 0.0;
        s_sig[tid] = 0.0;
    }
    if (tid == 0) s_flags = 0u;
    __syncthreads();
    const double mscale = fmax(fmax(s_max[0], s_max[1]), fmax(s_max[2], s_max[3]));

    // Step 1: bulk edge from lambda_{k+1}, lambda_{2k+1} (1-based) and the rank test.
    const double edge_c = 1.0 / (cbrt(4.0) - 1.0);
    const double cut = 1.0 / cbrt(static_cast<double>(D));
    const double lam_plus = lam[KPILOT] + edge_c * (lam[KPILOT] - lam[2 * KPILOT]);
    const bool pass = (tid <= KPILOT) && (lam[tid] / lam_plus - 1.0 > cut);
    int rank = __syncthreads_count(pass);
    if (tid == 0) {
        unsigned f = 0u;
        if (!(lam[0] == lam[0]) || !(lam[0] < 1e300) || !(lam_plus == lam_plus)) f |= EOSQ_BLOCK_NONFINITE;
        if (rank > KPILOT) f |= EOSQ_BLOCK_NONFINITE;
        if (f) atomicOr(&s_flags, f);
    }
    if (rank > KPILOT) rank = KPILOT;

    if (rank > 0) {
        // Step 2: k imputed atoms behind the outliers; the observed eigenvalues after them are known
        // one by one up to lambda_EV_EXPL, the rest (the tail) only through sums.
        {
            double a = 0.0;
            if (tid >= rank + KPILOT && tid < EV_EXPL) a = lam[tid];
            else if (tid >= rank && tid < rank + KPILOT) {
                const int jj = tid - rank + 1;
                const double bs = lam[KPILOT + rank];
                const double gap = bs - lam[2 * KPILOT + rank];
                a = bs + (1.0 - pow(static_cast<double>(jj) / KPILOT, 2.0 / 3.0)) * edge_c * gap;
            }
            atoms[tid] = a;
        }
        const double floor_piv = 1.2e-16 * fmax(fabs(lam[0]), 1e-300);
        {
            const double is = (mscale > 0.0) ? 1.0 / mscale : 0.0;
            const double se = (tid > 0) ? fabs(ee[tid - 1] * is) : 0.0;
            sde[tid] = make_double2(dd[tid] * is, (tid > 0) ? fmax(se * se, EV_E2_FLOOR) : 0.0);
        }
        __syncthreads();
        // Tail sums  sum_{j > EV_EXPL} 1 / (lambda_j - z)  and  sum 1 / (lambda_j - z)^2  at z = lambda_i:
        // the sums over the whole spectrum have a pole at z, so they are taken at six points
        // z + m h, m = -3 .. 3 without 0, the known eigenvalues are subtracted there, and what is left
        // (smooth: the tail lies well below z) is interpolated to z, exact for polynomials of degree 5.
        // h = z / 64, or a little less when a known eigenvalue would sit on a sample point.
        // Warps 1 .. 3 take these sums and Step 3 while warp 0 factorises for the eigenvectors below.
        if (warp > 0) {
            const int e = tid - 32;
            if (e < 6 * rank) {
                const int i = e / 6, m6 = e % 6;
                const int mm = (m6 < 3) ? m6 - 3 : m6 - 2;   // -3, -2, -1, 1, 2, 3
                const double z = lam[i];
                // A known eigenvalue right at a sample point would be subtracted with a large
                // cancellation error: shrink h until every other known eigenvalue keeps a quarter
                // step away from all six points (the six threads of a vector find the same h).
                double h = z * (1.0 / 64.0);
#pragma unroll 1
                for (int attempt = 0; attempt < 8; ++attempt) {
                    double nearest = 1e300;
#pragma unroll 1
                    for (int j = 0; j < EV_EXPL; ++j) {
                        if (j == i) continue;
                        const double t = fabs(lam[j] - z) / h;   // in steps
                        if (t < 3.5) nearest = fmin(nearest, fabs(t - rint(t)) + ((t < 0.5) ? 1.0 : 0.0));
                    }
                    if (nearest >= 0.25) break;
                    h *= 0.8125;
                }
                const double x = fma(static_cast<double>(mm), h, z);
                const double is = sp_rcp(mscale);
                double f1, f2;
                charpoly_sums(sde, x * is, f1, f2);
                f1 *= is;
                f2 *= is * is;
#pragma unroll 2
                for (int j = 0; j < EV_EXPL; ++j) {
                    const double inv = sp_rcp(lam[j] - x);
                    f1 -= inv;
                    f2 = fma(-inv, inv, f2);
                }
                const int am = (mm < 0) ? -mm : mm;
                const double w = (am == 1) ? 15.0 / 20.0 : ((am == 2) ? -6.0 / 20.0 : 1.0 / 20.0);
                st1[e] = w * f1;
                st2[e] = w * f2;
            }
            asm volatile("bar.sync 1, 96;" ::: "memory");
            // Step 3: Stieltjes transforms of F_e at z = lambda_i, D-transform, Eq. 9, Eq. 6.
            for (int i = warp - 1; i < rank; i += SP_WARPS - 1) {
                const double z = lam[i];
                double ms = 0.0, msp = 0.0;
                for (int j = rank + lane; j < EV_EXPL; j += 32) {
                    const double inv = sp_rcp(atoms[j] - z);
                    ms += inv;
                    msp = fma(inv, inv, msp);
                }
                if (lane < 6) {
                    ms += st1[6 * i + lane];
                    msp += st2[6 * i + lane];
                }
                ms = warp_sum(ms);
                msp = warp_sum(msp);
                if (lane == 0) {
                    const double nn = static_cast<double>(D - rank);
                    ms /= nn;
                    msp /= nn;
                    const double ratio = static_cast<double>(D) / static_cast<double>(n);
                    const double m1 = ratio * ms - (1.0 - ratio) / z;  // n x n side: n - d extra zeros
                    const double m1p = ratio * msp + (1.0 - ratio) / (z * z);
                    const double m2 = ms, m2p = msp;                   // d x d side
                    const double T = z * m1 * m2;
                    const double Tp = m1 * m2 + z * (m1p * m2 + m1 * m2p);
                    const double dh = 1.0 / sqrt(T);
                    const double a1 = m1 / (dh * dh * Tp), a2 = m2 / (dh * dh * Tp);
                    double ph = dh * sqrt(a1 * a2);
                    const double sg = sqrt(z);
                    if (!(ph >= 0.0) || !(ph < 1e300)) {
                        ph = 0.0;
                        atomicOr(&s_flags, EOSQ_BLOCK_CLAMPED);
                    } else if (ph > sg) {
                        ph = sg;
                        atomicOr(&s_flags, EOSQ_BLOCK_CLAMPED);
                    }
                    s_phi[i] = ph;
                    s_sig[i] = sg;
                    if (i > 0 && (lam[i - 1] - z) < 1e-9 * lam[i - 1]) atomicOr(&s_flags, EOSQ_BLOCK_CLUSTERED);
                }
            }
        }

        // Kept eigenvectors of the tridiagonal matrix from its twisted factorisation: with the
        // pivots of T - mu I = L+ D+ L+^T taken from the top,  D+_{i+1} = (d_{i+1} - mu) - e_i^2 / D+_i,
        // and of U- D- U-^T taken from the bottom,  D-_i = (d_i - mu) - e_i^2 / D-_{i+1},
        // gamma_i = D+_i + D-_i - (d_i - mu) is the residual of the vector z that starts with z_r = 1
        // at index r and runs  z_i = -(e_i / D+_i) z_{i+1}  upwards and  z_{i+1} = -(e_i / D-_{i+1}) z_i
        // downwards: (T - mu I) z = gamma_r e_r.  r = argmin |gamma| gives a residual of the order of
        // the error of mu, which is at rounding level here, so one such vector is as good as inverse
        // iteration converged.  Lane i of warp 0 owns vector i (column i of the arrays).
        if (warp == 0 && lane < rank) {
            const int c = lane;
            const double mu = lam[c];
            // forward pivots: the ratios go where the vector will be, D+ where the backward ratios will be
            double dp = dd[0] - mu;
#pragma unroll 4
            for (int i = 0; i < D - 1; ++i) {
                if (!(fabs(dp) >= floor_piv)) dp = (dp < 0.0) ? -floor_piv : floor_piv;
                const double e = ee[i];
                const double lp = e * sp_rcp(dp);
                fb[i * FAC_LANES + c] = dp;
                yv[i * FAC_LANES + c] = lp;
                dp = fma(-lp, e, dd[i + 1] - mu);
            }
            // backward pivots, and the twist index on the way
            double dm = dd[D - 1] - mu;
            double gbest = fabs(dp);   // gamma_{D-1} = D+_{D-1} (D-_{D-1} is d - mu itself)
            int rbest = D - 1;
#pragma unroll 4
            for (int i = D - 2; i >= 0; --i) {
                if (!(fabs(dm) >= floor_piv)) dm = (dm < 0.0) ? -floor_piv : floor_piv;
                const double e = ee[i];
                const double um = e * sp_rcp(dm);
                const double dpi = fb[i * FAC_LANES + c];   // D+_i, read before its place is taken
                fb[i * FAC_LANES + c] = um;
                const double t = dd[i] - mu;
                dm = fma(-um, e, t);
                const double gam = fabs(dpi + dm - t);
                if (gam < gbest) {
                    gbest = gam;
                    rbest = i;
                }
            }
            // the vector, left unnormalised (the back-transformation normalises at the end)
            double ss = 1.0;
            yv[rbest * FAC_LANES + c] = 1.0;
            double z = 1.0;
            for (int i = rbest - 1; i >= 0; --i) {
                z = -yv[i * FAC_LANES + c] * z;   // the ratio's place becomes the entry's
                yv[i * FAC_LANES + c] = z;
                ss = fma(z, z, ss);
            }
            z = 1.0;
            for (int i = rbest; i < D - 1; ++i) {
                z = -fb[i * FAC_LANES + c] * z;
                yv[(i + 1) * FAC_LANES + c] = z;
                ss = fma(z, z, ss);
            }
            if (!(ss > 0.0 && ss < 1e300)) atomicOr(&s_flags, EOSQ_BLOCK_NOT_CONVERGED);
        }
    }
    __syncthreads();

    // Back-transformation of the kept vectors (the ring takes the place of the factorisations, which
    // are no longer needed after the barrier above).
    const double *R = ws.gram + static_cast<size_t>(b) * D * D;
    float *vr = ws.vr + static_cast<size_t>(b) * RMAX * D;
    if (rank > 0) sp_back_transform(R, tt, yv, ring, rank, warp, lane, vr, out, gb);
    // rows >= rank of V are zero; scalars
    for (int e = tid; e < RMAX * D; e += SP_THREADS) {
        if (e / D >= rank) {
            out.V[gb * RMAX * D + e] = 0;
            vr[e] = 0.0f;
            if (out.vr32) out.vr32[gb * RMAX * D + e] = 0.0f;
        }
    }
    if (tid < RMAX) {
        const float sg = static_cast<float>(s_sig[tid]);
        const float ph = static_cast<float>(s_phi[tid]);
        const float cf = (tid < rank && s_sig[tid] > 0.0) ? static_cast<float>(s_phi[tid] / s_sig[tid]) : 0.0f;
        out.sigma[gb * RMAX + tid] = sg;
        out.phi[gb * RMAX + tid] = ph;
        ws.coef[static_cast<size_t>(b) * RMAX + tid] = cf;
        if (out.coef) out.coef[gb * RMAX + tid] = cf;
    }
    if (full && out.eig) out.eig[gb * D + tid] = static_cast<float>(lam[tid]);
    if (tid == 0) {
        if (b == 0) *ws.redo_count = 0;   // the second pass of this chunk is over: empty its queue for the next chunk
        out.rank[gb] = rank;
        ws.rank[b] = rank;
        out.status[gb] = static_cast<int32_t>(s_flags);
        if (out.lambda_plus) out.lambda_plus[gb] = static_cast<float>(lam_plus);
    }
}

void launch_eigvals(int64_t nb, const Workspace &ws, const int *list, const int *count, int *mark_list, bool full, cudaStream_t s) {
    if (full) {
        eigvals_kernel<<<list_grid(nb, list), D, 0, s>>>(ws.diag, ws.off, ws.lam, list, count, mark_list, ws.redo_count);
    } else {
        const int64_t work = list ? std::min<int64_t>(nb, LIST_GRID) : nb;
        const unsigned grid = static_cast<unsigned>(std::max<int64_t>(1, (work + EVT_WARPS - 1) / EVT_WARPS));
        eigvals_top_kernel<<<grid, 32 * EVT_WARPS, 0, s>>>(ws.diag, ws.off, ws.lam, static_cast<int>(nb), list, count, mark_list, ws.redo_count);
    }
}

void launch_spectral(int64_t nb, int n, const Workspace &ws, const eosq_cache_t &out, int64_t block0, bool full,
                     cudaStream_t s) {
    ensure_dynamic_smem(reinterpret_cast<const void *>(spectral_kernel), SPECTRAL_DYN_SMEM);
    spectral_kernel<<<static_cast<unsigned>(nb), SP_THREADS, SPECTRAL_DYN_SMEM, s>>>(n, ws, out, static_cast<long long>(block0), full);
}

}  // namespace eosq
