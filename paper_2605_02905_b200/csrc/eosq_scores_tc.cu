// Attention logits straight from the compressed keys on the tensor cores (Remark 6.4):
//   s[g][t] = scale ( rho_t <Pi q_g, centroid[code_t]> + <q_g V^T, P[:, t]> ).
// Per 128-token tile the two inner products are two small MMAs (N = 16 query columns):
//   D1 = Z W^T,  Z = centroids of the codes (128 x 128),  W = Pi q (16 x 128);
//   D2 = P^T Aq^T, P^T the stored left factors of the tile (128 x 16), Aq = q V^T (16 x 16).
// The A operands never touch shared memory: every thread owns one token, expands its packed
// codes to fp16 centroids with byte permutes (the four 2-bit levels are a four-entry byte table
// that fits a register pair) and stores the row into tensor memory.  The query-side operands are
// split into a high and a low fp16 plane so that they enter with about 2^-22 precision; the
// centroid table is scaled by a factor chosen on the host so that every level is (almost) exactly
// an fp16 number.
#include <algorithm>
#include <cmath>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

constexpr int TC_ERR_SCORES_TIMEOUT = 4;

constexpr int SC_THREADS = 256;           // two groups of four warps, each group works on its own tiles
constexpr int SC_NQ = 16;                 // query columns per pass (MMA N)
constexpr uint32_t SC_TMEM_COLS = 256;    // 128 columns per warp group
constexpr uint32_t SC_COL_A = 0;          // code operand: 64 columns (128 fp16)
constexpr uint32_t SC_COL_P = 64;         // factor operand: 8 columns (16 fp16)
constexpr uint32_t SC_COL_D1 = 80;        // 16 columns
constexpr uint32_t SC_COL_D2 = 96;        // 16 columns
constexpr float SC_QSCALE = 256.0f;       // scaling of the query-side operands before the hi/lo split

// Byte offset of element (row, k) of a K-major, 128-byte-swizzled operand whose 64-wide K boxes
// hold `rows` rows each.
__device__ __forceinline__ uint32_t sc_b_offset(int row, int k, int rows) {
    const int box = k >> 6, kk = k & 63;
    return box * rows * 128 + row * 128 + ((((kk >> 3) ^ (row & 7)) << 4) | ((kk & 7) << 1));
}

__device__ __forceinline__ void sc_split(float v, __half &hi, __half &lo) {
    hi = __float2half_rn(v);
    lo = __float2half_rn(v - __half2float(hi));
}

__device__ __forceinline__ uint32_t sc_prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Sixteen 2-bit codes (one word) -> eight words of fp16 pairs.  `lo_tab` / `hi_tab` hold the low
// and the high bytes of the four centroids.
__device__ __forceinline__ void sc_expand16(uint32_t w, uint32_t lo_tab, uint32_t hi_tab, uint32_t *out) {
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        uint32_t t = (w >> (16 * part)) & 0xFFFFu;
        t = (t | (t << 8)) & 0x00FF00FFu;
        t = (t | (t << 4)) & 0x0F0F0F0Fu;
        t = (t | (t << 2)) & 0x33333333u;   // one nibble per code
#pragma unroll
        for (int quad = 0; quad < 2; ++quad) {
            const uint32_t sel = t >> (16 * quad);
            const uint32_t lows = sc_prmt(lo_tab, 0u, sel), highs = sc_prmt(hi_tab, 0u, sel);
            out[4 * part + 2 * quad] = sc_prmt(lows, highs, 0x5140u);
            out[4 * part + 2 * quad + 1] = sc_prmt(lows, highs, 0x7362u);
        }
    }
}

struct ScoresArgs {
    eosq_cache_t cache;
    long long bph, head_stride, items;   // items = heads * bph
    int n, G, g0;                        // this pass handles query columns [g0, g0 + min(16, G - g0))
    float scale;                         // softmax scale
    float inv_code;                      // 1 / (centroid table scale * SC_QSCALE)
    uint32_t lo_tab, hi_tab;             // bytes of the scaled fp16 centroids
    const float *pi_t;
    const __half *q;
    float *scores;
    int *err;
};

__global__ void __launch_bounds__(SC_THREADS, 2) scores_tc_kernel(const ScoresArgs a) {
    extern __shared__ uint8_t sc_smem_raw[];
    __shared__ __align__(8) uint64_t done_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(sc_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *b1_hi = base, *b1_lo = base + 4096;            // W  : two 64-wide K boxes of 16 rows x 128 bytes per plane
    uint8_t *b2_hi = base + 8192, *b2_lo = base + 10240;    // Aq : one box per plane
    float *qs = reinterpret_cast<float *>(base + 12288);    // [16][128] queries of the current head
    __half *vs = reinterpret_cast<__half *>(base + 20480);  // [16][128] right vectors of the current block
    const int tid = threadIdx.x, warp = tid >> 5;
    const int wg = tid >> 7, wt = tid & 127, lw = warp & 3;
    const int n = a.n, tiles = (n + 127) / 128;
    const int gcount = min(SC_NQ, a.G - a.g0);

    if (tid == 0) {
        mbar_init(&done_bar[0], 1);
        mbar_init(&done_bar[1], 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, SC_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_wg = tmem_base_s + 128u * wg;                                  // lane 0 view (MMA operands)
    const uint32_t tmem_me = tmem_wg + (static_cast<uint32_t>(32 * lw) << 16);           // this warp's lanes

    const long long ipc = (a.items + gridDim.x - 1) / gridDim.x;
    const long long it0 = ipc * blockIdx.x, it1 = min(a.items, it0 + ipc);
    long long cur_head = -1;
    uint32_t done_cnt = 0;
    constexpr uint32_t idesc = umma_idesc_f16(128, SC_NQ, false, false);

    for (long long item = it0; item < it1; ++item) {
        const long long head = item / a.bph, jb = item % a.bph;
        const long long gb = head * a.head_stride + jb;
        if (head != cur_head) {
            __syncthreads();
            for (int e = tid; e < SC_NQ * D; e += SC_THREADS) {
                const int g = e / D;
                qs[e] = (g < gcount) ? __half2float(a.q[(head * a.G + a.g0 + g) * D + (e % D)]) : 0.0f;
            }
            __syncthreads();
            const int c = tid & (D - 1), half = tid >> 7;
            float w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = 0.0f;
            for (int j = 0; j < D; ++j) {
                const float pv = a.pi_t[j * D + c];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = fmaf(pv, qs[(8 * half + i) * D + j], w[i]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                __half hi, lo;
                sc_split(w[i] * SC_QSCALE, hi, lo);
                const uint32_t off = sc_b_offset(8 * half + i, c, SC_NQ);
                *reinterpret_cast<__half *>(b1_hi + off) = hi;
                *reinterpret_cast<__half *>(b1_lo + off) = lo;
            }
            cur_head = head;
        }
        const int rank = a.cache.rank[gb];
        reinterpret_cast<uint4 *>(vs)[tid] = reinterpret_cast<const uint4 *>(a.cache.V + gb * RMAX * D)[tid];
        __syncthreads();   // every group is past the previous block; vs and qs are in place
        if (abort_flag) break;
        {
            const int g = tid >> 4, i = tid & 15;
            float dot = 0.0f;
            if (i < rank) {
#pragma unroll 8
                for (int j = 0; j < D; ++j) dot = fmaf(qs[g * D + j], __half2float(vs[i * D + j]), dot);
            }
            __half hi, lo;
            sc_split(dot * SC_QSCALE, hi, lo);
            const uint32_t off = sc_b_offset(g, i, SC_NQ);
            *reinterpret_cast<__half *>(b2_hi + off) = hi;
            *reinterpret_cast<__half *>(b2_lo + off) = lo;
        }
        fence_proxy_async_smem();
        __syncthreads();

        for (int tile = wg; tile < tiles; tile += 2) {
            const int tok = tile * 128 + wt;
            const bool valid = tok < n;
            uint32_t cw[8];
            float rho = 0.0f;
            uint32_t pw[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                cw[i] = 0u;
                pw[i] = 0u;
            }
            if (valid) {
                const uint4 *src = reinterpret_cast<const uint4 *>(a.cache.codes + (static_cast<size_t>(gb) * n + tok) * 32);
                const uint4 c0 = src[0], c1 = src[1];
                cw[0] = c0.x; cw[1] = c0.y; cw[2] = c0.z; cw[3] = c0.w;
                cw[4] = c1.x; cw[5] = c1.y; cw[6] = c1.z; cw[7] = c1.w;
                rho = __half2float(__ushort_as_half(a.cache.norms[static_cast<size_t>(gb) * n + tok]));
#pragma unroll
                for (int i = 0; i < RMAX; ++i) {
                    if (i < rank) {
                        const uint32_t v = a.cache.P[(static_cast<size_t>(gb) * RMAX + i) * n + tok];
                        pw[i >> 1] |= v << (16 * (i & 1));
                    }
                }
            }
            {
                uint32_t av[32];
#pragma unroll
                for (int q = 0; q < 4; ++q) sc_expand16(cw[q], a.lo_tab, a.hi_tab, &av[8 * q]);
                tmem_st32(tmem_me + SC_COL_A, av);
#pragma unroll
                for (int q = 0; q < 4; ++q) sc_expand16(cw[4 + q], a.lo_tab, a.hi_tab, &av[8 * q]);
                tmem_st32(tmem_me + SC_COL_A + 32, av);
            }
            tmem_st8(tmem_me + SC_COL_P, pw);
            tmem_st_wait();
            tc_fence_before_sync();
            asm volatile("bar.sync %0, %1;" ::"r"(1 + wg), "r"(128) : "memory");
            if (wt == 0) {
                tc_fence_after_sync();
                const uint32_t h1 = smem_u32(b1_hi), l1 = smem_u32(b1_lo);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t kb = (ks >> 2) * (SC_NQ * 128) + (ks & 3) * 32;
                    umma_f16_ts(tmem_wg + SC_COL_D1, tmem_wg + SC_COL_A + 8 * ks, umma_desc_sw128(h1 + kb, 16, 1024), idesc, ks ? 1u : 0u);
                    umma_f16_ts(tmem_wg + SC_COL_D1, tmem_wg + SC_COL_A + 8 * ks, umma_desc_sw128(l1 + kb, 16, 1024), idesc, 1u);
                }
                umma_f16_ts(tmem_wg + SC_COL_D2, tmem_wg + SC_COL_P, umma_desc_sw128(smem_u32(b2_hi), 16, 1024), idesc, 0u);
                umma_f16_ts(tmem_wg + SC_COL_D2, tmem_wg + SC_COL_P, umma_desc_sw128(smem_u32(b2_lo), 16, 1024), idesc, 1u);
                umma_commit(&done_bar[wg]);
            }
            const bool ok = mbar_wait(&done_bar[wg], done_cnt & 1u, &abort_flag);
            done_cnt += 1;
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t d1[16], d2[16];
            tmem_ld16(tmem_me + SC_COL_D1, d1);
            tmem_ld16(tmem_me + SC_COL_D2, d2);
            tmem_ld_wait();
            if (valid) {
                const float f1 = a.scale * rho * a.inv_code, f2 = a.scale * (1.0f / SC_QSCALE);
                float *dst = a.scores + (head * a.G + a.g0) * (a.bph * n) + jb * n + tok;
#pragma unroll
                for (int g = 0; g < SC_NQ; ++g)
                    if (g < gcount) dst[static_cast<size_t>(g) * (a.bph * n)] = fmaf(f1, __uint_as_float(d1[g]), f2 * __uint_as_float(d2[g]));
            }
            tc_fence_before_sync();
            asm volatile("bar.sync %0, %1;" ::"r"(1 + wg), "r"(128) : "memory");
        }
    }

    __syncthreads();
    if (abort_flag && tid == 0) atomicOr(a.err, TC_ERR_SCORES_TIMEOUT);
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base_s, SC_TMEM_COLS);
    }
}

// Scale factor kappa in [8, 16) for which the fp16 roundings of kappa * centroid are, jointly, as
// close to exact as possible (searched over 4096 mantissas); with four levels the worst relative
// rounding error drops from 2.4e-4 to the 1e-6 range.
static float best_table_scale(const Codebook &cb, uint16_t (&table)[16]) {
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

bool scores_tc_supported(int bits, int n) { return bits == 2 && n >= 128; }

bool launch_scores_tc(const eosq_cache_t &cache, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const Codebook &cb, const __half *q, int G, float scale, float *scores, int *err, int sm_count,
                      cudaStream_t s) {
    static bool configured = false;
    constexpr size_t smem = 24576 + 1024;
    if (!configured) {
        if (cudaFuncSetAttribute(scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
            return false;
        configured = true;
    }
    uint16_t table[16];
    const float kappa = best_table_scale(cb, table);
    ScoresArgs a;
    a.cache = cache;
    a.bph = bph;
    a.head_stride = head_stride;
    a.items = heads * bph;
    a.n = n;
    a.G = G;
    a.scale = scale;
    a.inv_code = 1.0f / (kappa * SC_QSCALE);
    a.lo_tab = 0u;
    a.hi_tab = 0u;
    for (int k = 0; k < 4; ++k) {
        a.lo_tab |= static_cast<uint32_t>(table[k] & 0xFFu) << (8 * k);
        a.hi_tab |= static_cast<uint32_t>(table[k] >> 8) << (8 * k);
    }
    a.pi_t = rot.pi_t;
    a.q = q;
    a.scores = scores;
    a.err = err;
    const int grid = static_cast<int>(std::min<int64_t>(a.items, 2 * static_cast<int64_t>(sm_count)));
    for (int g0 = 0; g0 < G; g0 += SC_NQ) {
        a.g0 = g0;
        scores_tc_kernel<<<grid, SC_THREADS, smem, s>>>(a);
    }
    return true;
}

}  // namespace eosq
