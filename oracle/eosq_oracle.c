/*
 * eOptShrinkQ reference oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, double-precision CPU statement of what the eOptShrinkQ hot
 * path computes, written from the paper's algorithms so that it can be checked
 * against them by eye.  It shares no code, tables or constants with the CUDA
 * library; only tests, the smoke check and the benchmark's CPU-baseline leg may
 * load it.  No blocking, fusion or reordering beyond what each algorithm states.
 *
 * Passages followed (paper section / equation / algorithm):
 *   - SVD of the block and lambda_i = sigma_i^2 ............ Sec. 2.3 (text before Eq. 3)
 *   - pilot k, bulk edge, rank test ........................ Algorithm 2, Step 1
 *   - imputed noise spectrum F_e ........................... Algorithm 2, Step 2; Eq. 8
 *   - Stieltjes / D-transform, d_hat, a_hat ................ Eq. 7, Eq. 9
 *   - Frobenius shrinker phi = d sqrt(a1 a2) ............... Eq. 6 (first case)
 *   - residual R = S - S_hat (or S when rank = 0) .......... Algorithm 3
 *   - norm, Haar rotation, Lloyd-Max code, reconstruction .. Algorithm 1 (TQ_MSE)
 *   - score decomposition <y,x> = <y,x_lowrank> + <y,r> .... Remark 6.4
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *   - Algorithm 2 prints "lambda^2"; lambda_i already denotes sigma_i^2 (Sec. 2.3), so
 *     every "lambda^2" there is read as the eigenvalue sigma_i^2.
 *   - F_e has N = q - rank atoms (q = min(n,d)) and is normalised by 1/N.
 *   - m_2 is the Stieltjes transform of the d x d side, m_1 of the n x n side; the larger
 *     side carries |n-d| extra zero eigenvalues (companion transform).
 *   - T'(z) is the analytic derivative of z m_1(z) m_2(z).
 *   - log is the natural logarithm (reproduces k = 11 at d = 128 and k = 7 at d = 64).
 *   - Quantiser: thresholds at centroid midpoints, index ascending in centroid value,
 *     a value exactly on a threshold takes the lower index.
 *   - Bit packing (paper silent): coordinate j of a row occupies bits [j*b, (j+1)*b) of
 *     the row's little-endian bit string.
 *
 * Pins (tests, no GPU): 1-bit centroids, Lloyd-Max distortions, orthogonality of Pi,
 * k = 11 / 7, rank 0 on pure noise, white-noise closed forms for outlier locations and
 * the Frobenius shrinker, the identity phi = -T/(sigma T'), brute force on tiny blocks.
 * Parity unpinned (conventions fixed here, not by the paper): the 1/N normaliser of F_e
 * and taking R against the unrounded factors.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif
#ifndef M_SQRT2
#define M_SQRT2 1.41421356237309504880
#endif

/* ------------------------------------------------------------------------- */
/* Lloyd-Max codebook for N(0, 1/d)  (Algorithm 1, REQUIRE line; Sec. 2.2 item 3) */
/* ------------------------------------------------------------------------- */

static double std_normal_pdf(double x)
{
    if (isinf(x)) return 0.0;
    return exp(-0.5 * x * x) / sqrt(2.0 * M_PI);
}

/* P(a < X < b) for X ~ N(0,1), written so that tail cells keep their digits. */
static double std_normal_mass(double a, double b)
{
    if (a >= 0.0) return 0.5 * (erfc(a / M_SQRT2) - erfc(b / M_SQRT2));
    if (b <= 0.0) return 0.5 * (erfc(-b / M_SQRT2) - erfc(-a / M_SQRT2));
    return 0.5 * (erf(b / M_SQRT2) + erf(-a / M_SQRT2));
}

/*
 * Lloyd iteration on the density of N(0, 1/d): thresholds are midpoints of neighbouring
 * centroids; each centroid is the conditional mean of its cell,
 *     E[X | a < X < b] = sigma (pdf(a/sigma) - pdf(b/sigma)) / P(a/sigma < X/sigma < b/sigma).
 * centroids: 2^bits values ascending; thresholds: 2^bits - 1 midpoints.
 * Returns the number of iterations used.
 */
int orc_codebook(int bits, int d, double *centroids, double *thresholds)
{
    const int L = 1 << bits;
    const double sigma = 1.0 / sqrt((double)d);
    double *c = (double *)malloc(sizeof(double) * (size_t)L);
    double *t = (double *)malloc(sizeof(double) * (size_t)(L + 1));
    int it, i;
    for (i = 0; i < L; ++i) c[i] = -3.0 + 6.0 * (i + 0.5) / L; /* symmetric start, units of sigma */
    for (it = 0; it < 1000000; ++it) {
        double change = 0.0;
        t[0] = -INFINITY;
        t[L] = INFINITY;
        for (i = 1; i < L; ++i) t[i] = 0.5 * (c[i - 1] + c[i]);
        for (i = 0; i < L; ++i) {
            double mass = std_normal_mass(t[i], t[i + 1]);
            double mean = (std_normal_pdf(t[i]) - std_normal_pdf(t[i + 1])) / mass;
            double diff = fabs(mean - c[i]);
            if (diff > change) change = diff;
            c[i] = mean;
        }
        if (change < 1e-15) { ++it; break; }
    }
    for (i = 0; i < L; ++i) centroids[i] = sigma * c[i];
    for (i = 0; i + 1 < L; ++i) thresholds[i] = 0.5 * (centroids[i] + centroids[i + 1]);
    free(c);
    free(t);
    return it;
}

/* Mean squared error per unit variance of the codebook, E[(X - Q(X))^2] / sigma^2, by the
 * closed-form Gaussian cell integrals  int (x-c)^2 pdf = (1 + c^2) mass + ... */
double orc_codebook_distortion(int bits, int d, const double *centroids)
{
    const int L = 1 << bits;
    const double sigma = 1.0 / sqrt((double)d);
    double total = 0.0;
    int i;
    for (i = 0; i < L; ++i) {
        double c = centroids[i] / sigma;
        double a = (i == 0) ? -INFINITY : 0.5 * (centroids[i - 1] + centroids[i]) / sigma;
        double b = (i == L - 1) ? INFINITY : 0.5 * (centroids[i] + centroids[i + 1]) / sigma;
        double mass = std_normal_mass(a, b);
        /* int_a^b x pdf = pdf(a) - pdf(b);  int_a^b x^2 pdf = mass + a pdf(a) - b pdf(b) */
        double m1 = std_normal_pdf(a) - std_normal_pdf(b);
        double apa = isinf(a) ? 0.0 : a * std_normal_pdf(a);
        double bpb = isinf(b) ? 0.0 : b * std_normal_pdf(b);
        double m2 = mass + apa - bpb;
        total += m2 - 2.0 * c * m1 + c * c * mass;
    }
    return total;
}

/* ------------------------------------------------------------------------- */
/* Seeded Haar rotation  (Algorithm 1: "shared Haar rotation Pi")             */
/* ------------------------------------------------------------------------- */

/* Counter-based generator: SplitMix64 finaliser of seed + (counter+1) * golden ratio. */
static uint64_t splitmix64_at(uint64_t seed, uint64_t counter)
{
    uint64_t z = seed + (counter + 1ULL) * 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static double uniform_open01(uint64_t bits)
{
    return ((double)(bits >> 11) + 0.5) * (1.0 / 9007199254740992.0); /* 2^-53 */
}

/* d x d matrix of iid N(0,1): entry e = i*d + j uses counters 2e, 2e+1 through Box-Muller. */
void orc_gaussian_matrix(int d, uint64_t seed, double *A)
{
    int64_t e, total = (int64_t)d * d;
    for (e = 0; e < total; ++e) {
        double u1 = uniform_open01(splitmix64_at(seed, 2ULL * (uint64_t)e));
        double u2 = uniform_open01(splitmix64_at(seed, 2ULL * (uint64_t)e + 1ULL));
        A[e] = sqrt(-2.0 * log(u1)) * cos(2.0 * M_PI * u2);
    }
}

/*
 * Pi = Q diag(sign R_ii) with A = Q R the Householder QR of the seeded Gaussian matrix:
 * the unique QR factor with positive diagonal of R, which is Haar distributed.
 * Pi is written row-major, z = Pi u.
 */
void orc_rotation(int d, uint64_t seed, double *Pi)
{
    double *A = (double *)malloc(sizeof(double) * (size_t)d * d);
    double *V = (double *)calloc((size_t)d * d, sizeof(double)); /* reflector k in column k */
    double *alpha = (double *)malloc(sizeof(double) * (size_t)d);
    int i, j, k;
    orc_gaussian_matrix(d, seed, A);
    for (k = 0; k < d; ++k) {
        double norm = 0.0, vnorm = 0.0;
        for (i = k; i < d; ++i) norm += A[i * d + k] * A[i * d + k];
        norm = sqrt(norm);
        alpha[k] = (A[k * d + k] >= 0.0) ? -norm : norm; /* R_kk */
        for (i = k; i < d; ++i) V[i * d + k] = A[i * d + k];
        V[k * d + k] -= alpha[k];
        for (i = k; i < d; ++i) vnorm += V[i * d + k] * V[i * d + k];
        vnorm = sqrt(vnorm);
        if (vnorm > 0.0)
            for (i = k; i < d; ++i) V[i * d + k] /= vnorm;
        for (j = k; j < d; ++j) { /* A <- (I - 2 v v^T) A */
            double dot = 0.0;
            for (i = k; i < d; ++i) dot += V[i * d + k] * A[i * d + j];
            for (i = k; i < d; ++i) A[i * d + j] -= 2.0 * V[i * d + k] * dot;
        }
    }
    /* Q = H_0 H_1 ... H_{d-1}: apply the reflectors to the identity, last first. */
    for (i = 0; i < d; ++i)
        for (j = 0; j < d; ++j) Pi[i * d + j] = (i == j) ? 1.0 : 0.0;
    for (k = d - 1; k >= 0; --k) {
        for (j = 0; j < d; ++j) {
            double dot = 0.0;
            for (i = k; i < d; ++i) dot += V[i * d + k] * Pi[i * d + j];
            for (i = k; i < d; ++i) Pi[i * d + j] -= 2.0 * V[i * d + k] * dot;
        }
    }
    for (j = 0; j < d; ++j)
        if (alpha[j] < 0.0)
            for (i = 0; i < d; ++i) Pi[i * d + j] = -Pi[i * d + j];
    free(A);
    free(V);
    free(alpha);
}

/* ------------------------------------------------------------------------- */
/* SVD by one-sided (Hestenes) Jacobi  (Sec. 2.3; Algorithm 2 REQUIRE)        */
/* ------------------------------------------------------------------------- */

/*
 * S is n x d row-major with n >= d.  On return sigma[0..d) holds the singular values in
 * descending order, U (n x d, row-major, column i = left vector i) and V (d x d, row-major,
 * column i = right vector i).  Columns of W = S V are rotated in pairs until every pair is
 * orthogonal to 1e-15 relative.  Returns the number of sweeps.
 */
int orc_svd(int n, int d, const double *S, double *sigma, double *U, double *V)
{
    /* work column-major: W[j*n + t] = column j */
    double *W = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *Vc = (double *)calloc((size_t)d * d, sizeof(double)); /* Vc[j*d + i] = V[i][j] */
    int *order = (int *)malloc(sizeof(int) * (size_t)d);
    int sweeps = 0, p, q, t, i, j, rotated = 1;
    for (j = 0; j < d; ++j) {
        for (t = 0; t < n; ++t) W[(size_t)j * n + t] = S[(size_t)t * d + j];
        Vc[(size_t)j * d + j] = 1.0;
    }
    while (rotated && sweeps < 60) {
        rotated = 0;
        ++sweeps;
        for (p = 0; p < d - 1; ++p) {
            for (q = p + 1; q < d; ++q) {
                double *wp = W + (size_t)p * n, *wq = W + (size_t)q * n;
                double a = 0.0, b = 0.0, g = 0.0;
                for (t = 0; t < n; ++t) {
                    a += wp[t] * wp[t];
                    b += wq[t] * wq[t];
                    g += wp[t] * wq[t];
                }
                if (g == 0.0 || fabs(g) <= 1e-15 * sqrt(a * b)) continue;
                {
                    double zeta = (b - a) / (2.0 * g);
                    double tn = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                    double c = 1.0 / sqrt(1.0 + tn * tn), s = c * tn;
                    double *vp = Vc + (size_t)p * d, *vq = Vc + (size_t)q * d;
                    for (t = 0; t < n; ++t) {
                        double x = wp[t], y = wq[t];
                        wp[t] = c * x - s * y;
                        wq[t] = s * x + c * y;
                    }
                    for (i = 0; i < d; ++i) {
                        double x = vp[i], y = vq[i];
                        vp[i] = c * x - s * y;
                        vq[i] = s * x + c * y;
                    }
                    rotated = 1;
                }
            }
        }
    }
    {
        double *norms = (double *)malloc(sizeof(double) * (size_t)d);
        for (j = 0; j < d; ++j) {
            double a = 0.0;
            for (t = 0; t < n; ++t) a += W[(size_t)j * n + t] * W[(size_t)j * n + t];
            norms[j] = sqrt(a);
            order[j] = j;
        }
        for (i = 1; i < d; ++i) { /* insertion sort, descending */
            int oi = order[i];
            j = i - 1;
            while (j >= 0 && norms[order[j]] < norms[oi]) {
                order[j + 1] = order[j];
                --j;
            }
            order[j + 1] = oi;
        }
        for (i = 0; i < d; ++i) {
            int src = order[i];
            sigma[i] = norms[src];
            for (t = 0; t < n; ++t)
                U[(size_t)t * d + i] = (norms[src] > 0.0) ? W[(size_t)src * n + t] / norms[src] : 0.0;
            for (j = 0; j < d; ++j) V[(size_t)j * d + i] = Vc[(size_t)src * d + j];
        }
        free(norms);
    }
    free(W);
    free(Vc);
    free(order);
    return sweeps;
}

/* ------------------------------------------------------------------------- */
/* eOptShrink on the spectrum  (Algorithm 2; Eq. 7-9; Eq. 6 Frobenius case)   */
/* ------------------------------------------------------------------------- */

/* Pilot parameter k = floor(d^c), c = min(1/2.01, 1/log log d)  (Algorithm 2, REQUIRE and Step 1). */
int orc_pilot_k(int d)
{
    double c = 1.0 / 2.01;
    double loglog = log(log((double)d));
    if (loglog > 0.0 && 1.0 / loglog < c) c = 1.0 / loglog;
    return (int)floor(pow((double)d, c));
}

/*
 * Inputs: n, d, the q = min(n,d) singular values (descending), k (pass <= 0 for the
 * paper's pilot value).  Outputs (arrays of length q unless noted):
 *   out_scalars[0] = k, [1] = lambda_plus, [2] = rank, [3] = margin (smallest distance of
 *   any lambda_i/lambda_plus - 1 from the cut d^(-1/3)), [4] = number of clamped shrunk values
 *   atoms[q]   : estimated noise eigenvalues; entries [0, rank) are unused (0)
 *   m1,m2,T,Tp,dhat,a1,a2,phi : entries [0, rank) filled, rest 0
 * Returns rank, or -1 when the indices of Step 2 would leave the spectrum (3k+1 > q).
 */
int orc_eoptshrink_spectrum(int n, int d, const double *sigma, int k_in, double *out_scalars,
                            double *atoms, double *m1, double *m2, double *T, double *Tp,
                            double *dhat, double *a1, double *a2, double *phi)
{
    const int q = (n < d) ? n : d;
    const int Q = (n < d) ? d : n;
    const int k = (k_in > 0) ? k_in : orc_pilot_k(d);
    const double edge_c = 1.0 / (pow(2.0, 2.0 / 3.0) - 1.0);
    const double cut = pow((double)d, -1.0 / 3.0);
    double *lam = (double *)malloc(sizeof(double) * (size_t)q);
    double lambda_plus, margin = INFINITY;
    int rank = 0, clamped = 0, i, j;
    for (i = 0; i < q; ++i) {
        lam[i] = sigma[i] * sigma[i];
        atoms[i] = m1[i] = m2[i] = T[i] = Tp[i] = dhat[i] = a1[i] = a2[i] = phi[i] = 0.0;
    }
    if (3 * k + 1 > q) {
        free(lam);
        return -1;
    }
    /* Step 1 (1-based lambda_{k+1}, lambda_{2k+1} are lam[k], lam[2k]) */
    lambda_plus = lam[k] + edge_c * (lam[k] - lam[2 * k]);
    for (i = 0; i < q; ++i) {
        double excess = lam[i] / lambda_plus - 1.0;
        if (excess > cut) ++rank;
        if (fabs(excess - cut) < margin) margin = fabs(excess - cut);
    }
    out_scalars[0] = (double)k;
    out_scalars[1] = lambda_plus;
    out_scalars[2] = (double)rank;
    out_scalars[3] = margin;
    out_scalars[4] = 0.0;
    if (rank == 0 || 2 * k + rank + 1 > q) {
        free(lam);
        return rank;
    }
    /* Step 2: k imputed atoms after the rank outliers, observed values after those. */
    {
        double base = lam[k + rank];              /* lambda_{k + rank + 1} */
        double gap = lam[k + rank] - lam[2 * k + rank]; /* minus lambda_{2k + rank + 1} */
        for (j = 1; j <= k; ++j)
            atoms[rank + j - 1] = base + (1.0 - pow((double)j / k, 2.0 / 3.0)) * edge_c * gap;
        for (i = rank + k; i < q; ++i) atoms[i] = lam[i];
    }
    /* Step 3: Stieltjes transforms of F_e at z = lambda_i, D-transform, Eq. 9, Eq. 6. */
    {
        const int N = q - rank;
        const double ratio = (double)q / (double)Q;
        for (i = 0; i < rank; ++i) {
            double z = lam[i];
            double ms = 0.0, msp = 0.0; /* small (q x q) side and its derivative */
            double ml, mlp, m_1, m_2, m_1p, m_2p, t, tp, dh, x1, x2, ph;
            for (j = rank; j < q; ++j) {
                double inv = 1.0 / (atoms[j] - z);
                ms += inv;
                msp += inv * inv;
            }
            ms /= N;
            msp /= N;
            ml = ratio * ms - (1.0 - ratio) / z; /* large (Q x Q) side: Q - q extra zeros */
            mlp = ratio * msp + (1.0 - ratio) / (z * z);
            if (n >= d) { m_1 = ml; m_1p = mlp; m_2 = ms; m_2p = msp; } /* m_1: n x n, m_2: d x d */
            else        { m_1 = ms; m_1p = msp; m_2 = ml; m_2p = mlp; }
            t = z * m_1 * m_2;
            tp = m_1 * m_2 + z * (m_1p * m_2 + m_1 * m_2p);
            dh = 1.0 / sqrt(t);
            x1 = m_1 / (dh * dh * tp);
            x2 = m_2 / (dh * dh * tp);
            ph = dh * sqrt(x1 * x2);
            if (!(ph >= 0.0) || !isfinite(ph)) { ph = 0.0; ++clamped; }
            else if (ph > sigma[i]) { ph = sigma[i]; ++clamped; }
            m1[i] = m_1; m2[i] = m_2; T[i] = t; Tp[i] = tp;
            dhat[i] = dh; a1[i] = x1; a2[i] = x2; phi[i] = ph;
        }
    }
    out_scalars[4] = (double)clamped;
    free(lam);
    return rank;
}

/* ------------------------------------------------------------------------- */
/* Residual, TQ_MSE rows, packing  (Algorithm 3; Algorithm 1)                 */
/* ------------------------------------------------------------------------- */

/*
 * R = S - sum_i coef_i (S v_i) v_i^T with coef_i = phi_i / sigma_i, i.e. the shrunk estimate
 * written through the right vectors (xi_i sigma_i = S zeta_i).  Vr is d x r row-major
 * (column i = zeta_i).  With r = 0, R = S.  Also writes Pfac[i*n + t] = coef_i (S v_i)[t].
 */
void orc_residual(int n, int d, int r, const double *S, const double *Vr, const double *coef,
                  double *R, double *Pfac)
{
    int t, i, j;
    for (t = 0; t < n; ++t) {
        for (j = 0; j < d; ++j) R[(size_t)t * d + j] = S[(size_t)t * d + j];
        for (i = 0; i < r; ++i) {
            double proj = 0.0;
            for (j = 0; j < d; ++j) proj += S[(size_t)t * d + j] * Vr[(size_t)j * r + i];
            proj *= coef[i];
            if (Pfac) Pfac[(size_t)i * n + t] = proj;
            for (j = 0; j < d; ++j) R[(size_t)t * d + j] -= proj * Vr[(size_t)j * r + i];
        }
    }
}

/*
 * TQ_MSE forward pass on each row of R (Algorithm 1): rho = ||r||, u = r / rho, z = Pi u,
 * code_j = number of thresholds strictly below z_j.  A zero row gives u = 0.
 * rho[n], z[n*d], codes[n*d] (one byte per coordinate, unpacked).
 */
void orc_tq_rows(int n, int d, int bits, const double *R, const double *Pi,
                 const double *thresholds, double *rho, double *z, uint8_t *codes)
{
    const int nthr = (1 << bits) - 1;
    int t, j, c, i;
    for (t = 0; t < n; ++t) {
        const double *r = R + (size_t)t * d;
        double nrm = 0.0;
        for (j = 0; j < d; ++j) nrm += r[j] * r[j];
        nrm = sqrt(nrm);
        rho[t] = nrm;
        for (c = 0; c < d; ++c) {
            double acc = 0.0;
            int code = 0;
            if (nrm > 0.0)
                for (j = 0; j < d; ++j) acc += Pi[(size_t)c * d + j] * (r[j] / nrm);
            for (i = 0; i < nthr; ++i)
                if (thresholds[i] < acc) ++code;
            z[(size_t)t * d + c] = acc;
            codes[(size_t)t * d + c] = (uint8_t)code;
        }
    }
}

/* Row bit string, little-endian: coordinate j at bits [j*bits, (j+1)*bits). */
void orc_pack(int n, int d, int bits, const uint8_t *codes, uint8_t *packed)
{
    const int row_bytes = (d * bits + 7) / 8;
    int t, j, b;
    memset(packed, 0, (size_t)n * row_bytes);
    for (t = 0; t < n; ++t)
        for (j = 0; j < d; ++j)
            for (b = 0; b < bits; ++b)
                if ((codes[(size_t)t * d + j] >> b) & 1) {
                    int pos = j * bits + b;
                    packed[(size_t)t * row_bytes + pos / 8] |= (uint8_t)(1u << (pos % 8));
                }
}

void orc_unpack(int n, int d, int bits, const uint8_t *packed, uint8_t *codes)
{
    const int row_bytes = (d * bits + 7) / 8;
    int t, j, b;
    for (t = 0; t < n; ++t)
        for (j = 0; j < d; ++j) {
            int code = 0;
            for (b = 0; b < bits; ++b) {
                int pos = j * bits + b;
                if ((packed[(size_t)t * row_bytes + pos / 8] >> (pos % 8)) & 1) code |= 1 << b;
            }
            codes[(size_t)t * d + j] = (uint8_t)code;
        }
}

/*
 * Reconstruction from stored values (Algorithm 1 last TQ_MSE line; Algorithm 2 Return):
 *   x_hat[t] = sum_i Pfac[i][t] Vfac[i][:] + rho[t] * Pi^T zhat_t,   zhat = centroids[code].
 * Pfac is [r][n], Vfac is [r][d], both as stored (already rounded by the caller).
 */
void orc_decode(int n, int d, int bits, int r, const uint8_t *codes, const double *rho,
                const double *Pfac, const double *Vfac, const double *Pi,
                const double *centroids, double *X)
{
    int t, j, c, i;
    (void)bits;
    for (t = 0; t < n; ++t)
        for (j = 0; j < d; ++j) {
            double acc = 0.0, low = 0.0;
            for (c = 0; c < d; ++c) acc += Pi[(size_t)c * d + j] * centroids[codes[(size_t)t * d + c]];
            for (i = 0; i < r; ++i) low += Pfac[(size_t)i * n + t] * Vfac[(size_t)i * d + j];
            X[(size_t)t * d + j] = low + rho[t] * acc;
        }
}

/* scores[g][t] = scale <y_g, x_hat_t>  (attention logits, Sec. 2.1; Remark 6.4). */
void orc_scores(int n, int d, int G, const double *X, const double *Y, double scale, double *scores)
{
    int g, t, j;
    for (g = 0; g < G; ++g)
        for (t = 0; t < n; ++t) {
            double acc = 0.0;
            for (j = 0; j < d; ++j) acc += Y[(size_t)g * d + j] * X[(size_t)t * d + j];
            scores[(size_t)g * n + t] = scale * acc;
        }
}

/* ------------------------------------------------------------------------- */
/* Whole block, Algorithm 3, and a batch loop over independent blocks         */
/* ------------------------------------------------------------------------- */

/*
 * One block.  RMAX = capacity of the factor outputs (rank never exceeds the pilot k).
 * Outputs: sigma[d]; scal[5] as in orc_eoptshrink_spectrum; phi[d], dhat[d], a1[d], a2[d];
 * Vr[RMAX*d] (row i = zeta_i); Pfac[RMAX*n]; rho[n]; z[n*d]; codes[n*d]; packed[n*row_bytes].
 * Requires n >= d.  Returns rank (or -1).
 */
int orc_encode_block(int n, int d, int bits, int rmax, const double *S, const double *Pi,
                     const double *thresholds, double *sigma, double *scal, double *phi,
                     double *dhat, double *a1, double *a2, double *Vr_out, double *Pfac,
                     double *rho, double *z, uint8_t *codes, uint8_t *packed)
{
    double *U = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *V = (double *)malloc(sizeof(double) * (size_t)d * d);
    double *R = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *tmp = (double *)malloc(sizeof(double) * (size_t)d * 5);
    double *Vr = NULL, *coef = NULL;
    int rank, i, j;
    orc_svd(n, d, S, sigma, U, V);
    rank = orc_eoptshrink_spectrum(n, d, sigma, 0, scal, tmp, tmp + d, tmp + 2 * d, tmp + 3 * d,
                                   tmp + 4 * d, dhat, a1, a2, phi);
    if (rank < 0 || rank > rmax) {
        free(U); free(V); free(R); free(tmp);
        return -1;
    }
    Vr = (double *)malloc(sizeof(double) * (size_t)d * (rank > 0 ? rank : 1));
    coef = (double *)malloc(sizeof(double) * (size_t)(rank > 0 ? rank : 1));
    for (i = 0; i < rank; ++i) {
        coef[i] = phi[i] / sigma[i];
        for (j = 0; j < d; ++j) {
            Vr[(size_t)j * rank + i] = V[(size_t)j * d + i];
            Vr_out[(size_t)i * d + j] = V[(size_t)j * d + i];
        }
    }
    orc_residual(n, d, rank, S, Vr, coef, R, Pfac);
    orc_tq_rows(n, d, bits, R, Pi, thresholds, rho, z, codes);
    orc_pack(n, d, bits, codes, packed);
    free(U); free(V); free(R); free(tmp); free(Vr); free(coef);
    return rank;
}

/* Independent blocks, one after another (threads over blocks when built with OpenMP). */
int orc_encode_batch(int64_t num_blocks, int n, int d, int bits, int rmax, const double *S,
                     const double *Pi, const double *thresholds, double *sigma, double *scal,
                     double *phi, double *dhat, double *a1, double *a2, double *Vr, double *Pfac,
                     double *rho, double *z, uint8_t *codes, uint8_t *packed, int32_t *ranks)
{
    const size_t row_bytes = (size_t)(d * bits + 7) / 8;
    int64_t b;
    int bad = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad)
#endif
    for (b = 0; b < num_blocks; ++b) {
        int r = orc_encode_block(n, d, bits, rmax, S + (size_t)b * n * d, Pi, thresholds,
                                 sigma + (size_t)b * d, scal + (size_t)b * 5, phi + (size_t)b * d,
                                 dhat + (size_t)b * d, a1 + (size_t)b * d, a2 + (size_t)b * d,
                                 Vr + (size_t)b * rmax * d, Pfac + (size_t)b * rmax * n,
                                 rho + (size_t)b * n, z + (size_t)b * n * d,
                                 codes + (size_t)b * n * d, packed + (size_t)b * n * row_bytes);
        ranks[b] = r;
        if (r < 0) ++bad;
    }
    return bad;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
