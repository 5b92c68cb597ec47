// Spectral stage of eosq_encode: symmetric eigen-decomposition of the d x d Gram matrix
// (the block's singular values and right singular vectors, Sec. 2.3) and Algorithm 2
// (bulk edge, rank, imputed noise spectrum, D-transform estimators, Frobenius shrinker).
//
// All arithmetic here is double precision: the bulk eigenvalues sit two to three orders of
// magnitude below the largest outlier, and the rank test and the shrunk values must agree with a
// double-precision reference to 1e-4 relative or better.
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

__device__ __forceinline__ void sturm_step(const double2 de, double x, double &p0, double &p1, unsigned &cnt) {
    const double t = de.y * p0;
    const double p2 = fma(de.x - x, p1, -t);
    cnt += static_cast<unsigned>(__double2hiint(p1) ^ __double2hiint(p2)) >> 31;
    p0 = p1;
    p1 = p2;
}

// sde[i] = (d_i, e_{i-1}^2), scaled so that every entry is at most 1 in magnitude, followed by
// EV_PAD entries that are read but not used.  Returns the count; p_d(x) = pm 2^pe.  The entries
// of the next group are fetched before the current group's chain of dependent multiply-adds
// starts, and the pair is brought back to within 2^+-300 of one after every group: eight steps
// move it by at most 2^13 upwards and, even with full cancellation in every step, 2^-424 downwards.
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
        for (int i = 0; i < EV_GROUP; ++i) sturm_step(cur[i], x, p0, p1, cnt);
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
    for (int i = 0; i < (D - 1) - NG * EV_GROUP; ++i) sturm_step(cur[i], x, p0, p1, cnt);
    pm = p1;
    pe = esum;
    return static_cast<int>(cnt);
}

// With `mark_list` set (first pass over tensor-core Gram matrices), a block whose smallest
// eigenvalue is not at least REDO_RATIO of the largest (this includes non-finite spectra) is queued
// in mark_list[atomicAdd(mark_count)] for a second pass with the exact Gram matrix.
__device__ __forceinline__ void eigvals_block(const double *__restrict__ diag, const double *__restrict__ off,
                                              double *__restrict__ lam, int blk, int *__restrict__ mark_list,
                                              int *__restrict__ mark_count) {
    __shared__ __align__(16) double2 sde[D + EV_PAD];
    __shared__ double s_e2[D];
    __shared__ double s_red[3][4];
    __shared__ int s_cnt[D], s_pe[D];
    __shared__ double s_pm[D];
    const int tid = threadIdx.x;
    const size_t base = static_cast<size_t>(blk) * D;
    const double d0 = diag[base + tid];
    const double e0 = (tid < D - 1) ? off[base + tid] : 0.0;
    double m = fmax(fabs(d0), fabs(e0));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) s_red[0][tid >> 5] = m;
    // a non-finite entry anywhere poisons the whole spectrum: report NaN instead of a bracket
    const int bad = __syncthreads_or(!(fabs(d0) < 1e300) || !(fabs(e0) < 1e300));
    if (bad) {
        lam[base + tid] = nan("");
        if (mark_list && tid == 0) mark_list[atomicAdd(mark_count, 1)] = blk;
        return;
    }
    m = fmax(fmax(s_red[0][0], s_red[0][1]), fmax(s_red[0][2], s_red[0][3]));
    if (m == 0.0) {
        lam[base + tid] = 0.0;
        return;
    }
    const double scale = 1.0 / m;
    const double sd = d0 * scale, se = fabs(e0 * scale);
    s_e2[tid] = (tid < D - 1) ? fmax(se * se, EV_E2_FLOOR) : 0.0;
    __syncthreads();
    const double se_prev = (tid > 0) ? fabs(off[base + tid - 1] * scale) : 0.0;
    sde[tid] = make_double2(sd, (tid > 0) ? s_e2[tid - 1] : 0.0);
    if (tid < EV_PAD) sde[D + tid] = make_double2(0.0, 0.0);
    // Gershgorin bounds of the scaled matrix
    double glo = sd - se - se_prev, ghi = sd + se + se_prev;
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
    glo = fmin(fmin(s_red[1][0], s_red[1][1]), fmin(s_red[1][2], s_red[1][3]));
    ghi = fmax(fmax(s_red[2][0], s_red[2][1]), fmax(s_red[2][2], s_red[2][3]));
    glo -= 1e-10 * (fabs(glo) + 1.0);
    ghi += 1e-10 * (fabs(ghi) + 1.0);

    // first pass: counts at D points, geometric below ghi when ghi > 0 (nine decades), else uniform
    const bool geometric = ghi > 0.0;
    auto point = [&](int t) -> double {
        if (t < 0) return glo;
        if (geometric) return ghi * exp2(-(9.0 * 3.321928094887362 / (D - 1)) * static_cast<double>(D - 1 - t));
        return glo + (ghi - glo) * static_cast<double>(t + 1) / static_cast<double>(D);
    };
    {
        double pm;
        int pe;
        s_cnt[tid] = sturm_eval(sde, point(tid), pm, pe);
        s_pm[tid] = pm;
        s_pe[tid] = pe;
    }
    __syncthreads();
    const int target = D - 1 - tid;  // ascending index of the eigenvalue this thread brackets
    int t = -1;                      // largest grid index with count <= target
#pragma unroll
    for (int step = D / 2; step > 0; step >>= 1)
        if (t + step < D && s_cnt[t + step] <= target) t += step;
    double lo = point(t), hi = (t + 1 < D) ? point(t + 1) : ghi;
    if (t == D - 1) lo = hi;   // cannot happen (every eigenvalue is below the last point); keeps the bracket sane
    // counts and p_d at both ends (ends that are not grid points carry no value)
    int clo = (t >= 0) ? s_cnt[t] : 0, chi = (t + 1 < D) ? s_cnt[t + 1] : D;
    double flo = (t >= 0) ? s_pm[t] : 0.0, fhi = (t + 1 < D) ? s_pm[t + 1] : 0.0;
    int elo = (t >= 0) ? s_pe[t] : EV_PE_INVALID, ehi = (t + 1 < D) ? s_pe[t + 1] : EV_PE_INVALID;
    int replaced = 0;   // +1: the last point became hi, -1: it became lo
    int poor = 0;
    for (int it = 0; it < EV_MAX_ITER; ++it) {
        const double mid = 0.5 * (lo + hi);
        const bool done = (hi - lo) <= fmax(2e-15, 1e-8 * fabs(mid));
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
            ehi = pe;
            if (secant && replaced > 0) flo *= 0.5;
            replaced = 1;
        } else {
            lo = x;
            clo = c;
            flo = pm;
            elo = pe;
            if (secant && replaced < 0) fhi *= 0.5;
            replaced = -1;
        }
        poor = (hi - lo > 0.5 * width) ? poor + 1 : 0;   // three steps in a row that fail to halve the bracket force a bisection
    }
    const double ev = 0.5 * (lo + hi) * m;
    lam[base + tid] = ev;
    if (mark_list) {   // uniform over the CTA
        if (tid == 0) s_red[0][0] = ev;   // the largest eigenvalue
        __syncthreads();
        if (tid == D - 1 && !(ev >= REDO_RATIO * s_red[0][0])) mark_list[atomicAdd(mark_count, 1)] = blk;
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
// Algorithm 2 on the spectrum, then the kept eigenvectors by inverse iteration on the
// tridiagonal matrix and back-transformation through the stored reflectors.
// ------------------------------------------------------------------------------------------
//
// Every phase here is a chain of dependent latencies (a pivot after a pivot, a reflector after a
// reflector) that leaves most of the CTA idle, so the kernel is laid out for four CTAs of four warps
// per SM, whose chains overlap: 12 columns of LU storage (the rank never exceeds the pilot k = 11)
// and registers for three vectors per warp.
constexpr int SP_THREADS = 128, SP_WARPS = SP_THREADS / 32;
constexpr int LU_LANES = 12;
static_assert(KPILOT < LU_LANES && KPILOT <= 3 * SP_WARPS, "one LU column and one warp slot per kept vector");
constexpr size_t SPECTRAL_DYN_SMEM = sizeof(double) * 4 * D * LU_LANES;

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

// Back-transformation of the NV vectors warp, warp + 4, .. of `yv` through the reflectors stored in
// the rows of R, normalisation, and the stores of the kept right singular vectors.
// Reflectors are applied two at a time, H_{k-1} H_k y = y - g_k u_k - g_{k-1} u_{k-1} with
//   g_k = t_k (u_k . y),   g_{k-1} = t_{k-1} ((u_{k-1} . y) - g_k (u_{k-1} . u_k)),
// so that one round of warp reductions serves two steps, and their rows are fetched from global
// memory two pairs ahead of use.
template <int NV>
__device__ __forceinline__ void sp_back_transform(const double *__restrict__ R, const double *__restrict__ tt,
                                                  const double *__restrict__ yv, int warp, int lane, float *__restrict__ vr,
                                                  const eosq_cache_t &out, long long gb) {
    double y[NV][4];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int m = 0; m < 4; ++m) y[v][m] = yv[(lane + 32 * m) * LU_LANES + warp + SP_WARPS * v];
    double ring[2][2][4];
    auto load_pair = [&](int k, double (&dst)[2][4]) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            dst[0][m] = __ldg(R + static_cast<size_t>(k) * D + lane + 32 * m);
            dst[1][m] = __ldg(R + static_cast<size_t>(k - 1) * D + lane + 32 * m);
        }
    };
    load_pair(D - 3, ring[0]);
    load_pair(D - 5, ring[1]);
#pragma unroll 1
    for (int k0 = D - 3; k0 >= 1; k0 -= 4) {
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2) {
            const int k = k0 - 2 * s2;
            if (k >= 1) {
                double ua[4], ub[4];
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    ua[m] = ring[s2][0][m];
                    ub[m] = ring[s2][1][m];
                }
                if (k - 4 >= 1) load_pair(k - 4, ring[s2]);
                const double ta = tt[k], tb = tt[k - 1];
                double dots[2 * NV + 1];
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    dots[2 * v] = fma(ua[0], y[v][0], ua[1] * y[v][1]) + fma(ua[2], y[v][2], ua[3] * y[v][3]);
                    dots[2 * v + 1] = fma(ub[0], y[v][0], ub[1] * y[v][1]) + fma(ub[2], y[v][2], ub[3] * y[v][3]);
                }
                dots[2 * NV] = fma(ua[0], ub[0], ua[1] * ub[1]) + fma(ua[2], ub[2], ua[3] * ub[3]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                    for (int q = 0; q < 2 * NV + 1; ++q) dots[q] += __shfl_xor_sync(0xffffffffu, dots[q], o);
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const double ga = ta * dots[2 * v];
                    const double gbb = tb * fma(-ga, dots[2 * NV], dots[2 * v + 1]);
#pragma unroll
                    for (int m = 0; m < 4; ++m) y[v][m] = fma(-gbb, ub[m], fma(-ga, ua[m], y[v][m]));
                }
            }
        }
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int vi = warp + SP_WARPS * v;
        double nn = fma(y[v][0], y[v][0], y[v][1] * y[v][1]) + fma(y[v][2], y[v][2], y[v][3] * y[v][3]);
        nn = warp_sum(nn);
        const double rn = (nn > 0.0) ? rsqrt(nn) : 0.0;
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int j = lane + 32 * m;
            const float f = static_cast<float>(y[v][m] * rn);
            vr[vi * D + j] = f;
            out.V[(gb * RMAX + vi) * D + j] = __half_as_ushort(__float2half_rn(f));
            if (out.vr32) out.vr32[(gb * RMAX + vi) * D + j] = f;
        }
    }
}

__global__ void __launch_bounds__(SP_THREADS, 4) spectral_kernel(int n, Workspace ws, eosq_cache_t out, long long block0) {
    __shared__ double lam[D], dd[D], ee[D], tt[D], atoms[D];
    __shared__ double inv_e[D];              // reciprocals of the (clamped) subdiagonal entries
    __shared__ double s_phi[RMAX], s_sig[RMAX];
    __shared__ unsigned s_flags;
    extern __shared__ double dyn[];
    double *lu_l = dyn;                      // multipliers                      [D][12]
    double *lu_d = dyn + D * LU_LANES;       // reciprocal pivots                [D][12]
    double *lu_u = dyn + 2 * D * LU_LANES;   // first superdiagonal of U         [D][12]
    double *yv = dyn + 3 * D * LU_LANES;     // iteration vectors                [D][12]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const long long gb = block0 + b;
    const size_t base = static_cast<size_t>(b) * D;
    if (tid < D) {
        lam[tid] = ws.lam[base + tid];
        dd[tid] = ws.diag[base + tid];
        ee[tid] = ws.off[base + tid];
        tt[tid] = ws.tau[base + tid];
    }
    if (tid < RMAX) {
        s_phi[tid] = 0.0;
        s_sig[tid] = 0.0;
    }
    if (tid == 0) s_flags = 0u;
    __syncthreads();

    // Step 1: bulk edge from lambda_{k+1}, lambda_{2k+1} (1-based) and the rank test.
    const double edge_c = 1.0 / (cbrt(4.0) - 1.0);
    const double cut = 1.0 / cbrt(static_cast<double>(D));
    const double lam_plus = lam[KPILOT] + edge_c * (lam[KPILOT] - lam[2 * KPILOT]);
    const bool pass = (tid < D) && (lam[tid] / lam_plus - 1.0 > cut);
    int rank = __syncthreads_count(pass);
    if (tid == 0) {
        unsigned f = 0u;
        if (!(lam[0] == lam[0]) || !(lam[0] < 1e300) || !(lam_plus == lam_plus)) f |= EOSQ_BLOCK_NONFINITE;
        if (rank > KPILOT) f |= EOSQ_BLOCK_NONFINITE;
        if (f) atomicOr(&s_flags, f);
    }
    if (rank > KPILOT) rank = KPILOT;

    if (rank > 0) {
        // Step 2: k imputed atoms behind the outliers, observed eigenvalues after them.
        if (tid < D) {
            double a = 0.0;
            if (tid >= rank + KPILOT) a = lam[tid];
            else if (tid >= rank) {
                const int jj = tid - rank + 1;
                const double bs = lam[KPILOT + rank];
                const double gap = bs - lam[2 * KPILOT + rank];
                a = bs + (1.0 - pow(static_cast<double>(jj) / KPILOT, 2.0 / 3.0)) * edge_c * gap;
            }
            atoms[tid] = a;
        }
        const double floor_piv = 1.2e-16 * fmax(fabs(lam[0]), 1e-300);
        if (tid < D) {   // pivots taken from the subdiagonal do not depend on the vector: their reciprocals are shared
            double l = ee[tid];
            if (!(fabs(l) >= floor_piv)) l = (l < 0.0) ? -floor_piv : floor_piv;
            inv_e[tid] = sp_rcp(l);
        }
        __syncthreads();
        // Step 3: Stieltjes transforms of F_e at z = lambda_i, D-transform, Eq. 9, Eq. 6.
        for (int i = warp; i < rank; i += SP_WARPS) {
            const double z = lam[i];
            double ms = 0.0, msp = 0.0;
            for (int j = rank + lane; j < D; j += 32) {
                const double inv = 1.0 / (atoms[j] - z);
                ms += inv;
                msp += inv * inv;
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

        // Kept eigenvectors of the tridiagonal matrix: (T - mu I) = P L U with partial pivoting,
        // two steps of inverse iteration (the kept eigenvalues are separated from their
        // neighbours by far more than their error, so each step gains many digits).  Lane i of
        // warp 0 owns vector i (column i of the arrays).  The iterate is left unnormalised: it can
        // grow by at most 1 / floor_piv per step, and the back-transformation normalises at the end.
        if (warp == 0 && lane < rank) {
            // A lone warp pays the full latency of every instruction, so these loops are written for
            // few instructions per row: selects instead of branches, pointers that advance by
            // constants, the pivot bits of 32 rows in one register.
            const int c = lane;
            const double mu = lam[c];
            unsigned piv[4];
            double d_i = dd[0] - mu, u_i = ee[0];
            {
                double *pl = lu_l + c, *pd = lu_d + c, *pu = lu_u + c;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    unsigned word = 0u;
#pragma unroll 1
                    for (int ii = 0; ii < 32; ii += 4) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int i = 32 * q + ii + j;
                            if (i < D - 1) {
                                const double l = ee[i];
                                const double d_next = dd[i + 1] - mu;
                                const double u_next = ee[i + 1];   // ee[D - 1] is zero
                                // the reciprocal of the diagonal candidate starts before the pivot choice is known
                                const double ds = (fabs(d_i) >= floor_piv) ? d_i : ((d_i < 0.0) ? -floor_piv : floor_piv);
                                const double inv_d = sp_rcp(ds);
                                const bool keep = fabs(d_i) >= fabs(l);
                                // keep: row i stays.  Otherwise rows i and i + 1 change places and U gets a
                                // second superdiagonal entry, e_{i+1}.
                                const double inv = keep ? inv_d : inv_e[i];   // serves the elimination and the back substitution
                                const double fact = (keep ? l : d_i) * inv;
                                const double uu = keep ? u_i : d_next, other = keep ? d_next : u_i;
                                pl[j * LU_LANES] = fact;
                                pd[j * LU_LANES] = inv;
                                pu[j * LU_LANES] = uu * inv;   // U's superdiagonal over its pivot
                                d_i = fma(-fact, uu, other);
                                u_i = keep ? u_next : -fact * u_next;
                                word |= (keep ? 0u : 1u) << j;
                            }
                        }
                        word = (word << 28) | (word >> 4);   // rotate: after eight groups bit r belongs to row 32 q + r
                        pl += 4 * LU_LANES;
                        pd += 4 * LU_LANES;
                        pu += 4 * LU_LANES;
                    }
                    piv[q] = word;
                }
            }
            if (!(fabs(d_i) >= floor_piv)) d_i = (d_i < 0.0) ? -floor_piv : floor_piv;
            lu_d[(D - 1) * LU_LANES + c] = 1.0 / d_i;
            lu_u[(D - 1) * LU_LANES + c] = 0.0;
            for (int i = 0; i < D; ++i) {
                const double f = (i + 1) * 0.6180339887498949;
                yv[i * LU_LANES + c] = 0.5 + (f - floor(f));
            }
            double ss = 0.0;
            for (int it = 0; it < 2; ++it) {
                // forward: apply the row interchanges and L^-1.  Entries are fetched a group of four
                // ahead (the stores of a group never reach the entries already fetched).
                double carry = yv[c];
                {
                    double *py = yv + c;
                    const double *pl = lu_l + c;
                    double ny[4], nl[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        ny[j] = py[(1 + j) * LU_LANES];
                        nl[j] = pl[j * LU_LANES];
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        unsigned word = piv[q];
#pragma unroll 1
                        for (int ii = 0; ii < 32; ii += 4) {
                            double cy[4], cl[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                cy[j] = ny[j];
                                cl[j] = nl[j];
                                if (32 * q + ii + 4 + j < D - 1) {   // false only in the very last group
                                    ny[j] = py[(5 + j) * LU_LANES];
                                    nl[j] = pl[(4 + j) * LU_LANES];
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (32 * q + ii + j < D - 1) {
                                    const bool swap = (word >> j) & 1u;
                                    const double a = swap ? cy[j] : carry, other = swap ? carry : cy[j];
                                    py[j * LU_LANES] = a;
                                    carry = fma(-cl[j], a, other);
                                }
                            }
                            word >>= 4;
                            py += 4 * LU_LANES;
                            pl += 4 * LU_LANES;
                        }
                    }
                }
                // backward: U^-1, as x_i = a_i - b_i x_{i+1} - c_i x_{i+2} with the coefficients
                // prepared off the chain, so that one multiply-add separates consecutive entries.
                // Rows go down from D - 2 in groups of four, row 32 q + ii + 3 - j in slot j.
                double x1 = carry * lu_d[(D - 1) * LU_LANES + c];
                yv[(D - 1) * LU_LANES + c] = x1;
                double x2 = 0.0;
                ss = x1 * x1;
                {
                    double *py = yv + (D - 4) * LU_LANES + c;   // row 32 q + ii of the current group
                    const double *pd = lu_d + (D - 4) * LU_LANES + c, *pu = lu_u + (D - 4) * LU_LANES + c;
                    const double *pe = ee + (D - 4) + 1;         // pe[r] = e_{i+1} for row i = 32 q + ii + r
                    double ny[4], nd[4], nb[4], ne[4];
#pragma unroll
                    for (int j = 1; j < 4; ++j) {   // slot 0 of the first group would be row D - 1
                        ny[j] = py[(3 - j) * LU_LANES];
                        nd[j] = pd[(3 - j) * LU_LANES];
                        nb[j] = pu[(3 - j) * LU_LANES];
                        ne[j] = pe[3 - j];
                    }
                    ny[0] = nd[0] = nb[0] = ne[0] = 0.0;
#pragma unroll
                    for (int q = 3; q >= 0; --q) {
                        const unsigned word = piv[q];
#pragma unroll 1
                        for (int ii = 28; ii >= 0; ii -= 4) {
                            const unsigned bits = word >> ii;
                            double ca[4], cb[4], cc[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                ca[j] = ny[j] * nd[j];
                                cb[j] = nb[j];
                                cc[j] = ((bits >> (3 - j)) & 1u) ? ne[j] * nd[j] : 0.0;
                                if (32 * q + ii >= 4) {   // false only in the very last group
                                    ny[j] = py[(-1 - j) * LU_LANES];
                                    nd[j] = pd[(-1 - j) * LU_LANES];
                                    nb[j] = pu[(-1 - j) * LU_LANES];
                                    ne[j] = pe[-1 - j];
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (32 * q + ii + 3 - j <= D - 2) {
                                    const double x = fma(-cb[j], x1, fma(-cc[j], x2, ca[j]));
                                    py[(3 - j) * LU_LANES] = x;
                                    ss = fma(x, x, ss);
                                    x2 = x1;
                                    x1 = x;
                                }
                            }
                            py -= 4 * LU_LANES;
                            pd -= 4 * LU_LANES;
                            pu -= 4 * LU_LANES;
                            pe -= 4;
                        }
                    }
                }
            }
            if (!(ss > 0.0 && ss < 1e300)) atomicOr(&s_flags, EOSQ_BLOCK_NOT_CONVERGED);
        }
    }
    __syncthreads();

    // Back-transformation x = H_0 H_1 ... H_{D-3} y; warp w takes those of the vectors w, w + 4, w + 8
    // that exist (the instruction count follows the number of vectors, so it is a template argument).
    const double *R = ws.gram + static_cast<size_t>(b) * D * D;
    float *vr = ws.vr + static_cast<size_t>(b) * RMAX * D;
    if (warp < rank) {
        const int nv = (rank - warp + SP_WARPS - 1) / SP_WARPS;
        if (nv == 1) sp_back_transform<1>(R, tt, yv, warp, lane, vr, out, gb);
        else if (nv == 2) sp_back_transform<2>(R, tt, yv, warp, lane, vr, out, gb);
        else sp_back_transform<3>(R, tt, yv, warp, lane, vr, out, gb);
    }
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
    if (tid < D && out.eig) out.eig[gb * D + tid] = static_cast<float>(lam[tid]);
    if (tid == 0) {
        if (b == 0) *ws.redo_count = 0;   // the second pass of this chunk is over: empty its queue for the next chunk
        out.rank[gb] = rank;
        ws.rank[b] = rank;
        out.status[gb] = static_cast<int32_t>(s_flags);
        if (out.lambda_plus) out.lambda_plus[gb] = static_cast<float>(lam_plus);
    }
}

void launch_eigvals(int64_t nb, const Workspace &ws, const int *list, const int *count, int *mark_list, cudaStream_t s) {
    eigvals_kernel<<<list_grid(nb, list), D, 0, s>>>(ws.diag, ws.off, ws.lam, list, count, mark_list, ws.redo_count);
}

void launch_spectral(int64_t nb, int n, const Workspace &ws, const eosq_cache_t &out, int64_t block0,
                     cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaFuncSetAttribute(spectral_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(SPECTRAL_DYN_SMEM));
        configured = true;
    }
    spectral_kernel<<<static_cast<unsigned>(nb), SP_THREADS, SPECTRAL_DYN_SMEM, s>>>(n, ws, out, static_cast<long long>(block0));
}

}  // namespace eosq
