// Householder tridiagonalisation of the d x d Gram matrices (the first half of the symmetric
// eigen-decomposition that stands in for the block's SVD, Sec. 2.3 and Algorithm 2 REQUIRE line),
// in double precision, with the matrix resident in tensor memory.
//
// Why tensor memory.  Every step of the reduction is a chain of dependent latencies (publish a row,
// barrier, norm, matrix-vector product, reduction, barrier, rank-2 update), so one matrix cannot
// keep the double-precision pipe of an SM busy: several matrices per SM have to be in flight, each
// worked on by enough warps to keep its own steps short.  A 128 x 128 fp64 matrix is 128 KB, half
// of the register file, so registers hold one.  Tensor memory (256 KB per SM, 128 lanes x 512
// columns of 32 bits) is otherwise idle here and is addressed per thread: a thread of warp w reads
// and writes lane 32 (w % 4) + its lane index, any columns, with tcgen05.ld / tcgen05.st.  With the
// matrix there, a thread needs registers only for the vectors of a step, 128 registers are enough,
// and sixteen warps fit on an SM: two matrices of order 128 (256 threads each), or eight of order
// 64 (64 threads each).
//
// Layout.  A team of G x G threads (G = order / 8) works on one matrix; thread (tr, tc) =
// (t / G, t % G) holds A[tr + G a][tc + G b], a, b < 8, so every thread keeps an equal share of the
// shrinking trailing matrix.  Row slot a of a thread's tile is 16 consecutive tensor-memory columns
// (eight doubles), one load or store instruction.
//
// One step k reflects with H = I - gamma u u^T, u = x - beta e_{k+1}, x = A[k][k+1..],
// beta = -sign(x_{k+1}) ||x||, gamma = 1 / (beta (beta - x_{k+1})):
//     p = gamma A u,  2K = gamma (u . p),  A <- A - u p^T - (p - 2K u) u^T.
// The rank-2 update of step k is not applied when it becomes known but folded into the sweep of
// step k + 1, which reads every live element once, brings it up to date, writes it back and uses it
// for the next matrix-vector product: one pass over tensor memory per step instead of two.  Only
// the row that defines the next reflector is brought up to date early, by the G threads that hold
// it.  x and p travel through shared memory (double buffered by the parity of k, two team-wide
// barriers per step) in a permuted order that makes a thread's eight columns contiguous.
// Finished tile slots are skipped at compile time (one instantiation of the step per value of
// (k + 1) / G).
#include <algorithm>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"
#include "eosq_tridiag.cuh"

namespace eosq {

using namespace sm100;

namespace {

constexpr int TT_PSTRIDE = 10;   // doubles per column residue in the permuted vectors (8 used, 2 pad)

// Barrier over the threads of one team (the whole CTA when it is one team).
template <int TEAMS, int TEAM_THREADS>
__device__ __forceinline__ void tt_sync(int team) {
    // the barrier number is spelled out: a number in a register makes the compiler reserve all sixteen
    // barriers for the CTA, and the SM then holds two CTAs instead of four
    if (TEAMS == 1) __syncthreads();
    else if (team == 0) asm volatile("bar.sync 1, %0;" ::"n"(TEAM_THREADS) : "memory");
    else if (team == 1) asm volatile("bar.sync 2, %0;" ::"n"(TEAM_THREADS) : "memory");
    else if (team == 2) asm volatile("bar.sync 3, %0;" ::"n"(TEAM_THREADS) : "memory");
    else asm volatile("bar.sync 4, %0;" ::"n"(TEAM_THREADS) : "memory");
}
// The sweep token of a CTA with two teams.  Two reductions that share an SM slow each other down
// most when both sweep at once (the sweep is the one phase that fills the double-precision pipe) and
// left alone they fall into exactly that rhythm.  So the teams take turns: a team sweeps only while
// it holds the token and passes it on when its sweep is done; the rest of its step (reductions,
// barriers, the next reflector) then runs under the other team's sweep.  Barrier 5 carries the token
// to team 0 and barrier 6 to team 1: the receiver syncs, the giver only arrives.  Both teams take
// the token the same number of times (a team without work passes it on at once), team 1 gives it
// away once before its first step, and team 0 takes it once more at the very end.
template <int TEAM_THREADS>
__device__ __forceinline__ void tt_token_take(int team) {
    if (team == 0) asm volatile("bar.sync 5, %0;" ::"n"(2 * TEAM_THREADS) : "memory");
    else asm volatile("bar.sync 6, %0;" ::"n"(2 * TEAM_THREADS) : "memory");
}
template <int TEAM_THREADS>
__device__ __forceinline__ void tt_token_give(int team) {
    if (team == 0) asm volatile("bar.arrive 6, %0;" ::"n"(2 * TEAM_THREADS) : "memory");
    else asm volatile("bar.arrive 5, %0;" ::"n"(2 * TEAM_THREADS) : "memory");
}
template <int G>
__device__ __forceinline__ int tt_pos(int j) {
    return (j & (G - 1)) * TT_PSTRIDE + (j / G);
}

// Shared-memory state of one reduction of order 8 G.
template <int G>
struct TtShared {
    double xu[2][G * TT_PSTRIDE];   // published row x (zero up to its own index), permuted
    double pp[2][G * TT_PSTRIDE];   // p, permuted (zero for finished indices)
    double scal[2][4];              // per parity of k: beta_k, gamma_k, 2K_k (the first two from the publisher of row k)
    double wsum[2][8];              // per-warp parts of u . A u
    double dg[8 * G], of[8 * G], ta[8 * G];
};

// The G threads that hold row r (row slot AR = r / G of their tiles) turn it into reflector r and
// publish that: x = A[r][r+1..], beta = -sign(x_{r+1}) ||x||, gamma = 1 / (beta (beta - x_{r+1})),
// u = x - beta e_{r+1} into buffer `nxt` (zero up to index r), beta and gamma into scal[nxt], the
// tridiagonal entries d_r, beta into dg / of / ta, and u into row r of the matrix in global memory
// (`grow`).  With UPDATE the pending rank-2 update of step r - 1 (vectors in buffer nxt ^ 1,
// u_{r-1}[r] = uown, (p - 2K u)[r] = sown) is applied to the row first; the stored row is left as it
// is, the next sweep brings it up to date like every other row.  Tensor-memory loads and shuffles
// are warp-wide, so the whole warp of the holders runs this and `mine` marks the holders (they are
// G consecutive lanes).
template <int G, int AR, bool UPDATE>
__device__ __forceinline__ void tt_publish(uint32_t tb, int r, int nxt, int lane, int tc, bool mine, TtShared<G> &sh, double uown,
                                           double sown, double *__restrict__ grow) {
    uint32_t raw[16];
    tmem_ld16(tb + 16u * AR, raw);
    double uj[8], pj[8];
    if (UPDATE) {
        const double2 *us = reinterpret_cast<const double2 *>(&sh.xu[nxt ^ 1][tc * TT_PSTRIDE]);
        const double2 *ps = reinterpret_cast<const double2 *>(&sh.pp[nxt ^ 1][tc * TT_PSTRIDE]);
#pragma unroll
        for (int q = AR / 2; q < 4; ++q) {
            const double2 v = us[q], w = ps[q];
            uj[2 * q] = v.x;
            uj[2 * q + 1] = v.y;
            pj[2 * q] = w.x;
            pj[2 * q + 1] = w.y;
        }
    }
    tt_wait16(raw);
    double x[8], ss0 = 0.0, ss1 = 0.0;
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        if (b < AR) {
            x[b] = 0.0;
            continue;
        }
        const int col = tc + G * b;
        double t = tt_get(raw, b);
        if (UPDATE) t = fma(-uown, pj[b], fma(-sown, uj[b], t));
        if (b == AR && mine && col == r) sh.dg[r] = t;
        x[b] = (col > r) ? t : 0.0;
        const double s = (col > r + 1) ? t : 0.0;
        if (b & 1) ss1 = fma(s, s, ss1);
        else ss0 = fma(s, s, ss0);
    }
    // ||x[r+2..]||^2 over the holders, x_{r+1} from the holder of that column
    double ss = ss0 + ss1;
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const bool next_slot = ((r + 1) / G) != AR;   // column r + 1 sits in column slot AR or AR + 1
    const double xsel = next_slot ? x[(AR + 1) & 7] : x[AR];
    const double alpha = __shfl_sync(0xffffffffu, xsel, (lane & ~(G - 1)) | ((r + 1) & (G - 1)));
    double beta = alpha, gamma = 0.0;
    if (ss > 0.0) {
        const double sq = fma(alpha, alpha, ss);
        const double nrm = sq * tt_rsqrt(sq);
        beta = (alpha >= 0.0) ? -nrm : nrm;
        gamma = tt_rcp(fma(fabs(alpha), nrm, sq));   // 1 / (beta (beta - alpha))
    }
    if (tc == ((r + 1) & (G - 1))) {
        if (next_slot) x[(AR + 1) & 7] -= beta;
        else x[AR] -= beta;
    }
    if (mine) {
        double2 *dst = reinterpret_cast<double2 *>(&sh.xu[nxt][tc * TT_PSTRIDE]);
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_double2(x[2 * q], x[2 * q + 1]);
#pragma unroll
        for (int b = 0; b < 8; ++b) grow[tc + G * b] = x[b];
        if (tc == 0) {
            sh.scal[nxt][0] = beta;
            sh.scal[nxt][1] = gamma;
            sh.of[r] = beta;
            sh.ta[r] = gamma;
        }
    }
}

// One step k of a team, with (k + 1) / G == K0: the sweep with reflector k (published before the
// first barrier, together with beta_k and gamma_k), p_k, and then, by the warp that holds row k + 1,
// 2K_k and reflector k + 1.  `trow0` is row 0 of the matrix in global memory; t is the thread's index
// within its team.
template <int G, int K0, int TEAMS, bool TOKEN>
__device__ __forceinline__ void tt_step(uint32_t tb, int k, int kend, int t, int team, TtShared<G> &sh, double *__restrict__ trow0) {
    constexpr int TEAM_THREADS = G * G, NW = TEAM_THREADS / 32;
    const int lane = t & 31, warp = t >> 5, tr = t / G, tc = t & (G - 1);
    const int cur = k & 1, prv = cur ^ 1;
    // What does not depend on reflector k is fetched while its publisher is still at work: the
    // vectors u' and p' of the pending update (complete since the last barrier).
    double ujn[8], ujp[8], pjp[8];
    {
        const double2 *up = reinterpret_cast<const double2 *>(&sh.xu[prv][tc * TT_PSTRIDE]);
        const double2 *pq = reinterpret_cast<const double2 *>(&sh.pp[prv][tc * TT_PSTRIDE]);
#pragma unroll
        for (int q = K0 / 2; q < 4; ++q) {
            const double2 b = up[q], c = pq[q];
            ujp[2 * q] = b.x;
            ujp[2 * q + 1] = b.y;
            pjp[2 * q] = c.x;
            pjp[2 * q + 1] = c.y;
        }
    }
    uint32_t raw0[16];
    tmem_ld16(tb + 16u * K0, raw0);   // the first live row slot of the tile, too
    tt_sync<TEAMS, TEAM_THREADS>(team);
    const double gamma = sh.scal[cur][1], twoK_prev = sh.scal[prv][2];   // 2K' comes from the publisher, like gamma
    {
        const double2 *un = reinterpret_cast<const double2 *>(&sh.xu[cur][tc * TT_PSTRIDE]);
#pragma unroll
        for (int q = K0 / 2; q < 4; ++q) {
            const double2 a = un[q];
            ujn[2 * q] = a.x;
            ujn[2 * q + 1] = a.y;
        }
    }
    // The sweep: every live element is brought up to date, written back and used for A u.
    if (TOKEN) tt_token_take<TEAM_THREADS>(team);
    double acc[8];
    const double *ur = &sh.xu[prv][tr * TT_PSTRIDE], *pr = &sh.pp[prv][tr * TT_PSTRIDE];
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        acc[a] = 0.0;
        if (a < K0) continue;
        uint32_t raw[16];
        if (a == K0) {
#pragma unroll
            for (int e = 0; e < 16; ++e) raw[e] = raw0[e];
        } else {
            tmem_ld16(tb + 16u * a, raw);
        }
        const double uip = ur[a];
        const double sip = fma(-twoK_prev, uip, pr[a]);
        tt_wait16(raw);
        double s0 = 0.0, s1 = 0.0;
#pragma unroll
        for (int b = K0; b < 8; ++b) {
            double v = tt_get(raw, b);
            v = fma(-uip, pjp[b], v);
            v = fma(-sip, ujp[b], v);
            tt_put(raw, b, v);
            if ((b - K0) & 1) s1 = fma(v, ujn[b], s1);
            else s0 = fma(v, ujn[b], s0);
        }
        tt_st16(tb + 16u * a, raw);
        acc[a] = s0 + s1;
    }
    if (TOKEN) tt_token_give<TEAM_THREADS>(team);
    // u . A u (parts), then the sums of the partial rows over the G column residues: each stage
    // keeps half of the rows
    double tloc = 0.0;
    {
        const double2 *un = reinterpret_cast<const double2 *>(&sh.xu[cur][tr * TT_PSTRIDE]);
#pragma unroll
        for (int q = K0 / 2; q < 4; ++q) {
            const double2 v = un[q];
            tloc = fma(v.x, acc[2 * q], tloc);
            tloc = fma(v.y, acc[2 * q + 1], tloc);
        }
    }
    // (the five butterfly stages of u . A u are interleaved with the tree by hand: both are chains of
    // shuffles and additions, and neither depends on the other)
    const bool hA = tc & (G / 2), hB = tc & (G / 4), hC = tc & (G / 8);
    double v4[4], v2[2], v1;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const double keep = hA ? acc[q + 4] : acc[q], send = hA ? acc[q] : acc[q + 4];
        v4[q] = keep + __shfl_xor_sync(0xffffffffu, send, G / 2);
    }
    tloc += __shfl_xor_sync(0xffffffffu, tloc, 16);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const double keep = hB ? v4[q + 2] : v4[q], send = hB ? v4[q] : v4[q + 2];
        v2[q] = keep + __shfl_xor_sync(0xffffffffu, send, G / 4);
    }
    tloc += __shfl_xor_sync(0xffffffffu, tloc, 8);
    {
        const double keep = hC ? v2[1] : v2[0], send = hC ? v2[0] : v2[1];
        v1 = keep + __shfl_xor_sync(0xffffffffu, send, G / 8);
    }
    tloc += __shfl_xor_sync(0xffffffffu, tloc, 4);
    if (G == 16) v1 += __shfl_xor_sync(0xffffffffu, v1, 1);   // two threads per row are left: both get the sum
    tloc += __shfl_xor_sync(0xffffffffu, tloc, 2);
    const int arow = (hA ? 4 : 0) + (hB ? 2 : 0) + (hC ? 1 : 0);
    const int irow = tr + G * arow;
    if (G == 8 || !(tc & 1)) sh.pp[cur][tt_pos<G>(irow)] = (irow > k) ? gamma * v1 : 0.0;
    tloc += __shfl_xor_sync(0xffffffffu, tloc, 1);
    if (lane == 0) sh.wsum[cur][warp] = tloc;
    tmem_st_wait();   // this thread's own stores; nobody else reads its lane
    tt_sync<TEAMS, TEAM_THREADS>(team);
    // The warp that holds row k + 1 (row slot K0 of G of its lanes) finishes the step: 2K from the
    // warps' parts of u . A u, then the next reflector.
    if (warp == (((k + 1) & (G - 1)) * G) / 32) {
        double uAu;
        {
            const double2 *wp = reinterpret_cast<const double2 *>(&sh.wsum[cur][0]);
            const double2 w0 = wp[0];
            uAu = w0.x + w0.y;
            if (NW == 8) {
                const double2 w1 = wp[1], w2 = wp[2], w3 = wp[3];
                uAu = (uAu + (w1.x + w1.y)) + ((w2.x + w2.y) + (w3.x + w3.y));
            }
        }
        const double twoK = gamma * gamma * uAu;
        if (lane == 0) sh.scal[cur][2] = twoK;
        if (k + 1 < kend) {
            const int p1 = tt_pos<G>(k + 1);
            const double uown = sh.xu[cur][p1];
            const double sown = fma(-twoK, uown, sh.pp[cur][p1]);
            tt_publish<G, K0, true>(tb, k + 1, prv, lane, tc, tr == ((k + 1) & (G - 1)), sh, uown, sown,
                                    trow0 + static_cast<size_t>(k + 1) * D);
        }
    }
}

template <int G, int K0, int LO, int HI, int TEAMS, bool TOKEN>
__device__ __forceinline__ void tt_step_if(uint32_t tb, int k, int kend, int t, int team, TtShared<G> &sh, double *__restrict__ trow0) {
    if constexpr (K0 >= LO && K0 <= HI) tt_step<G, K0, TEAMS, TOKEN>(tb, k, kend, t, team, sh, trow0);
}

// Steps [0, KE) of the reduction of the order-8G matrix whose element (i, j) sits at
// gram[(ORIGIN + i) D + ORIGIN + j]; KE is a multiple of G, or 8 G - 2 (the last step).  Reflector
// k goes to row ORIGIN + k (full width, zero up to column ORIGIN + k); diag / off / tau receive
// d_k, the new off-diagonal entry and gamma_k.  When steps remain the trailing matrix is written
// back to its own place.  A CTA holds TEAMS teams, each working through its own matrices.
template <int G, int ORIGIN, int KE, int TEAMS, int MINB, bool TOKEN>
__global__ void __launch_bounds__(G *G *TEAMS, MINB) tridiag_tm_kernel(double *__restrict__ gram, double *__restrict__ diag,
                                                                        double *__restrict__ off, double *__restrict__ tau, int nb,
                                                                        const int *__restrict__ list, const int *__restrict__ count) {
    constexpr int N = 8 * G, TEAM_THREADS = G * G, THREADS = TEAM_THREADS * TEAMS;
    // columns per CTA: a thread's tile is 128 columns, and warps w, w + 4 share the lanes of a quadrant
    constexpr uint32_t COLS = 128u * ((THREADS / 32 + 3) / 4);
    constexpr bool LAST = (KE == N - 2);
    static_assert(LAST || KE % G == 0, "ranges end on tile-slot boundaries");
    static_assert(COLS >= 32 && (COLS & (COLS - 1)) == 0 && COLS <= 512, "tensor-memory allocations are powers of two");
    static_assert(TEAM_THREADS % 32 == 0, "teams are whole warps");
    static_assert(!TOKEN || TEAMS == 2, "the sweep token goes back and forth between two teams");
    __shared__ __align__(16) TtShared<G> shs[TEAMS];
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, cwarp = tid >> 5;
    const int team = tid / TEAM_THREADS, t = tid % TEAM_THREADS;
    const int tr = t / G, tc = t & (G - 1);
    TtShared<G> &sh = shs[team];
    if (cwarp == 0) {
        tmem_alloc(&tmem_base_s, COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tb = tmem_base_s + (static_cast<uint32_t>(32 * (cwarp & 3)) << 16) + 128u * static_cast<uint32_t>(cwarp >> 2);
    const int total = list ? *count : nb;
    if (TOKEN && team == 1) tt_token_give<TEAM_THREADS>(1);
    for (int li = blockIdx.x * TEAMS + team; li < total; li += gridDim.x * TEAMS) {
        const int blk = list ? list[li] : li;
        double *Gm = gram + static_cast<size_t>(blk) * D * D;
        double *T = Gm + static_cast<size_t>(ORIGIN) * D + ORIGIN;
        // the matrix into tensor memory
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            uint32_t raw[16];
#pragma unroll
            for (int b = 0; b < 8; ++b) tt_put(raw, b, T[static_cast<size_t>(tr + G * a) * D + tc + G * b]);
            tt_st16(tb + 16u * a, raw);
        }
        for (int e = t; e < G * TT_PSTRIDE; e += TEAM_THREADS) {
            sh.xu[0][e] = 0.0;
            sh.xu[1][e] = 0.0;
            sh.pp[0][e] = 0.0;
            sh.pp[1][e] = 0.0;
        }
        if (t < 8) sh.scal[t >> 2][t & 3] = 0.0;
        if constexpr (ORIGIN > 0) {   // the reflector rows of this range are full-width rows: zero left of the matrix
            for (int e = t; e < KE * (ORIGIN / 2); e += TEAM_THREADS) {
                const int r = e / (ORIGIN / 2), c2 = e % (ORIGIN / 2);
                reinterpret_cast<double2 *>(Gm + static_cast<size_t>(ORIGIN + r) * D)[c2] = make_double2(0.0, 0.0);
            }
        }
        tmem_st_wait();
        tt_sync<TEAMS, TEAM_THREADS>(team);
        if ((t >> 5) == 0) tt_publish<G, 0, false>(tb, 0, 0, t & 31, tc, tr == 0, sh, 0.0, 0.0, T);
        constexpr int HI = KE / G;
#pragma unroll 1
        for (int k = 0; k < KE; ++k) {
            switch ((k + 1) / G) {
                case 0: tt_step_if<G, 0, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 1: tt_step_if<G, 1, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 2: tt_step_if<G, 2, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 3: tt_step_if<G, 3, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 4: tt_step_if<G, 4, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 5: tt_step_if<G, 5, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                case 6: tt_step_if<G, 6, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
                default: tt_step_if<G, 7, 0, HI, TEAMS, TOKEN>(tb, k, KE, t, team, sh, T); break;
            }
        }
        // The update of the last step is still pending: apply it to what is left of the matrix
        // (rows and columns from KE on) and hand that on: to global memory for the next kernel, or,
        // at the very end, as the last diagonal and off-diagonal entries.
        {
            constexpr int AF = KE / G;
            tt_sync<TEAMS, TEAM_THREADS>(team);   // 2K of the last step comes from another warp
            const int kl = KE - 1, cur = kl & 1;
            const double twoK_prev = sh.scal[cur][2];
            double uj[8], pj[8];
#pragma unroll
            for (int b = AF; b < 8; ++b) {
                uj[b] = sh.xu[cur][tc * TT_PSTRIDE + b];
                pj[b] = sh.pp[cur][tc * TT_PSTRIDE + b];
            }
#pragma unroll
            for (int a = AF; a < 8; ++a) {
                const int row = tr + G * a;
                const double ui = sh.xu[cur][tr * TT_PSTRIDE + a];
                const double si = fma(-twoK_prev, ui, sh.pp[cur][tr * TT_PSTRIDE + a]);
                uint32_t raw[16];
                tmem_ld16(tb + 16u * a, raw);
                tt_wait16(raw);
#pragma unroll
                for (int b = AF; b < 8; ++b) {
                    const int col = tc + G * b;
                    const double v = fma(-ui, pj[b], fma(-si, uj[b], tt_get(raw, b)));
                    if (LAST) {
                        if (row == N - 2 && col == N - 2) sh.dg[N - 2] = v;
                        if (row == N - 2 && col == N - 1) sh.of[N - 2] = v;
                        if (row == N - 1 && col == N - 1) sh.dg[N - 1] = v;
                    } else if (row >= KE && col >= KE) {
                        T[static_cast<size_t>(row) * D + col] = v;
                    }
                }
            }
            if (LAST && t == 0) {
                sh.of[N - 1] = 0.0;
                sh.ta[N - 2] = 0.0;
                sh.ta[N - 1] = 0.0;
            }
        }
        tt_sync<TEAMS, TEAM_THREADS>(team);
        constexpr int KOUT = LAST ? N : KE;
        for (int k = t; k < KOUT; k += TEAM_THREADS) {
            const size_t o = static_cast<size_t>(blk) * D + ORIGIN + k;
            diag[o] = sh.dg[k];
            off[o] = sh.of[k];
            tau[o] = sh.ta[k];
        }
        tt_sync<TEAMS, TEAM_THREADS>(team);   // the shared state is reused by the team's next block
    }
    if (TOKEN) {
        // Team 0 is never behind team 1 in matrices and at most one ahead: then team 1 passes the
        // token through once for every step of that matrix.  The last token goes back to team 0.
        if (team == 1) {
            const int first0 = blockIdx.x * TEAMS, stride = gridDim.x * TEAMS;
            const int n0 = first0 < total ? (total - first0 + stride - 1) / stride : 0;
            const int n1 = first0 + 1 < total ? (total - first0 - 1 + stride - 1) / stride : 0;
            for (int i = 0; i < (n0 - n1) * KE; ++i) {
                tt_token_take<TEAM_THREADS>(1);
                tt_token_give<TEAM_THREADS>(1);
            }
        } else {
            tt_token_take<TEAM_THREADS>(0);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (cwarp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base_s, COLS);
    }
}


// ------------------------------------------------------------------------------------------
// The last 30 steps, on the trailing 32 x 32 matrix: one warp per matrix, lane i keeps row i in
// registers.  At this size a team's barriers and reductions cost more than its arithmetic, and a
// matrix is 8 KB, so a warp does a step on its own (two warp sums, two broadcasts through shared
// memory) and sixteen of them share an SM.  The step is the one of the header comment; column k of
// the symmetric matrix is read as element k of every lane's row, and the loop over k is unrolled so
// that finished columns drop out at compile time.
// ------------------------------------------------------------------------------------------
constexpr int TW_N = 32, TW_ORIGIN = D - TW_N, TW_WARPS = 4;

__device__ __forceinline__ double tw_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int K>
__device__ __forceinline__ void tw_step(double (&a)[TW_N], int lane, double *ub, double *pb, double &dg, double &of, double &ta,
                                        double *__restrict__ grow) {
    // reflector K from column K (= row K): x_j = A[j][K], j > K
    const double xj = (lane > K) ? a[K] : 0.0;
    if (lane == K) dg = a[K];
    const double alpha = __shfl_sync(0xffffffffu, xj, K + 1);
    const double ss = tw_sum((lane > K + 1) ? xj * xj : 0.0);
    double beta = alpha, gamma = 0.0;
    if (ss > 0.0) {
        const double sq = fma(alpha, alpha, ss);
        const double nrm = sq * tt_rsqrt(sq);
        beta = (alpha >= 0.0) ? -nrm : nrm;
        gamma = tt_rcp(fma(fabs(alpha), nrm, sq));
    }
    const double uj = (lane == K + 1) ? xj - beta : xj;
    if (lane == K) {
        of = beta;
        ta = gamma;
    }
    grow[lane] = uj;   // row TW_ORIGIN + K of the matrix in global memory, from its column TW_ORIGIN on
    ub[lane] = uj;
    __syncwarp();
    // p = gamma A u over the live columns
    constexpr int J0 = (K + 1) & ~1;   // pairs of columns; u is zero at K + 1 - 1 = K when that one is dragged in
    double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0;
#pragma unroll
    for (int j = J0; j < TW_N; j += 2) {
        const double2 u2 = *reinterpret_cast<const double2 *>(ub + j);
        if ((j - J0) & 2) {
            p2 = fma(a[j], u2.x, p2);
            p3 = fma(a[j + 1], u2.y, p3);
        } else {
            p0 = fma(a[j], u2.x, p0);
            p1 = fma(a[j + 1], u2.y, p1);
        }
    }
    const double pi = (lane > K) ? gamma * ((p0 + p1) + (p2 + p3)) : 0.0;
    const double twoK = gamma * tw_sum(uj * pi);
    const double si = fma(-twoK, uj, pi);
    pb[lane] = pi;
    __syncwarp();
    // A <- A - u p^T - (p - 2K u) u^T on the rows and columns beyond K (u and s vanish on the others)
#pragma unroll
    for (int j = J0; j < TW_N; j += 2) {
        const double2 u2 = *reinterpret_cast<const double2 *>(ub + j);
        const double2 p2 = *reinterpret_cast<const double2 *>(pb + j);
        a[j] = fma(-uj, p2.x, fma(-si, u2.x, a[j]));
        a[j + 1] = fma(-uj, p2.y, fma(-si, u2.y, a[j + 1]));
    }
    __syncwarp();   // the broadcasts are overwritten by the next step
}

template <int K>
__device__ __forceinline__ void tw_steps(double (&a)[TW_N], int lane, double *ub, double *pb, double &dg, double &of, double &ta,
                                         double *__restrict__ trow0) {
    if constexpr (K < TW_N - 2) {
        tw_step<K>(a, lane, ub, pb, dg, of, ta, trow0 + static_cast<size_t>(K) * D);
        tw_steps<K + 1>(a, lane, ub, pb, dg, of, ta, trow0);
    }
}

__global__ void __launch_bounds__(32 * TW_WARPS, 4) tridiag_warp_kernel(double *__restrict__ gram, double *__restrict__ diag,
                                                                        double *__restrict__ off, double *__restrict__ tau, int nb,
                                                                        const int *__restrict__ list, const int *__restrict__ count) {
    __shared__ __align__(16) double bc[TW_WARPS][2][TW_N];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int total = list ? *count : nb;
    for (int li = blockIdx.x * TW_WARPS + warp; li < total; li += gridDim.x * TW_WARPS) {
        const int blk = list ? list[li] : li;
        double *T = gram + static_cast<size_t>(blk) * D * D + static_cast<size_t>(TW_ORIGIN) * D + TW_ORIGIN;
        double a[TW_N];
        {
            const double2 *row = reinterpret_cast<const double2 *>(T + static_cast<size_t>(lane) * D);
#pragma unroll
            for (int q = 0; q < TW_N / 2; ++q) {
                const double2 v = row[q];
                a[2 * q] = v.x;
                a[2 * q + 1] = v.y;
            }
        }
        __syncwarp();   // every row is in registers before the reflectors overwrite the rows in memory
        double dg = 0.0, of = 0.0, ta = 0.0;
        tw_steps<0>(a, lane, bc[warp][0], bc[warp][1], dg, of, ta, T);
        // what is left is the 2 x 2 block of the last two rows
        if (lane == TW_N - 2) {
            dg = a[TW_N - 2];
            of = a[TW_N - 1];
        }
        if (lane == TW_N - 1) dg = a[TW_N - 1];
        const size_t o = static_cast<size_t>(blk) * D + TW_ORIGIN + lane;
        diag[o] = dg;
        off[o] = of;
        tau[o] = ta;
    }
}

}  // namespace

// Three ranges: the 128 x 128 matrix through its first 64 steps (two teams of 256 threads and all of
// the tensor memory per CTA), the trailing 64 x 64 matrix through 32 more (teams of 64 threads, two
// per CTA, four CTAs per SM), and the last 32 x 32 matrix by one warp each.
void launch_tridiag(int part, int64_t nb, const Workspace &ws, const int *list, const int *count, int sm_count, cudaStream_t s) {
    double *g0 = ws.gram, *d0 = ws.diag, *o0 = ws.off, *t0 = ws.tau;
    const int n = static_cast<int>(nb);
    const int64_t work = list ? std::min<int64_t>(nb, LIST_GRID) : nb;
    if (part == 0) {
        const int grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((work + 1) / 2, static_cast<int64_t>(sm_count))));
        tridiag_tm_kernel<16, 0, 64, 2, 1, true><<<grid, 512, 0, s>>>(g0, d0, o0, t0, n, list, count);
    } else if (part == 1) {
        const int grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((work + 1) / 2, 4 * static_cast<int64_t>(sm_count))));
        tridiag_tm_kernel<8, 64, 32, 2, 4, false><<<grid, 128, 0, s>>>(g0, d0, o0, t0, n, list, count);
    } else {
        const int grid = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>((work + TW_WARPS - 1) / TW_WARPS, 4 * static_cast<int64_t>(sm_count))));
        tridiag_warp_kernel<<<grid, 32 * TW_WARPS, 0, s>>>(g0, d0, o0, t0, n, list, count);
    }
}

}  // namespace eosq
