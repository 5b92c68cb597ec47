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

constexpr int SC_THREADS = 128;           // one token per thread, one tensor-memory lane per token
constexpr int SC_NQ = 16;                 // query columns per pass (MMA N)
constexpr uint32_t SC_TMEM_COLS = 128;
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

// What a thread fetches from global memory for one token of one tile.  The values stay exactly as
// loaded (nothing here depends on a load's result), so a fetch issued one tile ahead does not
// stall the thread; they are unpacked when the tile is processed.
constexpr int SC_PMAX = 12;   // factor rows fetched per token: the rank never exceeds the pilot k = 11
struct ScTokenData {
    uint4 c0, c1;               // 128 packed 2-bit codes
    unsigned short p[SC_PMAX];  // fp16 factor entries, rows below the rank
    unsigned short rho;         // fp16 row norm
};

__device__ __forceinline__ void sc_fetch(const ScoresArgs &a, long long gb, int rank, int tok, ScTokenData &t) {
    const bool valid = tok < a.n;
    const int tk = valid ? tok : 0;
    const uint4 *src = reinterpret_cast<const uint4 *>(a.cache.codes + (static_cast<size_t>(gb) * a.n + tk) * 32);
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    t.c0 = valid ? __ldg(src) : zero;
    t.c1 = valid ? __ldg(src + 1) : zero;
    t.rho = valid ? __ldg(a.cache.norms + static_cast<size_t>(gb) * a.n + tk) : static_cast<unsigned short>(0);
    const unsigned short *prow = a.cache.P + static_cast<size_t>(gb) * RMAX * a.n + tk;
#pragma unroll
    for (int i = 0; i < SC_PMAX; ++i) t.p[i] = (valid && i < rank) ? __ldg(prow + static_cast<size_t>(i) * a.n) : static_cast<unsigned short>(0);
}

// One CTA of four warps works through a contiguous range of (head, block) items; four CTAs share
// an SM.  Everything a tile needs from global memory is fetched one tile ahead into registers.
__global__ void __launch_bounds__(SC_THREADS, 4) scores_tc_kernel(const ScoresArgs a) {
    extern __shared__ uint8_t sc_smem_raw[];
    __shared__ __align__(8) uint64_t done_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(sc_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *b1_hi = base, *b1_lo = base + 4096;            // W  : two 64-wide K boxes of 16 rows x 128 bytes per plane
    uint8_t *b2_hi = base + 8192, *b2_lo = base + 10240;    // Aq : one box per plane
    float *qs = reinterpret_cast<float *>(base + 12288);    // [16][128] queries of the current head
    __half *vs = reinterpret_cast<__half *>(base + 20480);  // [16][128] right vectors of the current block
    const int tid = threadIdx.x, warp = tid >> 5;
    const int n = a.n, tiles = (n + 127) / 128;
    const int gcount = min(SC_NQ, a.G - a.g0);

    if (tid == 0) {
        mbar_init(&done_bar, 1);
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
    const uint32_t tmem0 = tmem_base_s;                                           // lane 0 view (MMA operands)
    const uint32_t tmem_me = tmem0 + (static_cast<uint32_t>(32 * warp) << 16);    // this warp's lanes

    const long long ipc = (a.items + gridDim.x - 1) / gridDim.x;
    const long long it0 = ipc * blockIdx.x, it1 = min(a.items, it0 + ipc);
    long long cur_head = -1;
    uint32_t done_cnt = 0;
    constexpr uint32_t idesc = umma_idesc_f16(128, SC_NQ, false, false);

    auto block_of = [&](long long item) { return (item / a.bph) * a.head_stride + (item % a.bph); };
    // prefetch state: the next tile's token data, the next block's rank and right vectors
    ScTokenData nxt;
    int rank = 0, rank_next = 0;
    uint4 v_next[2];
    if (it0 < it1) {
        const long long gb0 = block_of(it0);
        rank = __ldg(a.cache.rank + gb0);
        const uint4 *vsrc = reinterpret_cast<const uint4 *>(a.cache.V + gb0 * RMAX * D);
        v_next[0] = __ldg(vsrc + tid);
        v_next[1] = __ldg(vsrc + SC_THREADS + tid);
        sc_fetch(a, gb0, rank, tid, nxt);
    }

    for (long long item = it0; item < it1; ++item) {
        const long long head = item / a.bph, jb = item % a.bph;
        const long long gb = block_of(item);
        __syncthreads();   // the previous block's MMAs have been waited for: the shared operands are free
        if (abort_flag) break;
        if (head != cur_head) {
            for (int e = tid; e < SC_NQ * D; e += SC_THREADS) {
                const int g = e / D;
                qs[e] = (g < gcount) ? __half2float(a.q[(head * a.G + a.g0 + g) * D + (e % D)]) : 0.0f;
            }
            __syncthreads();
            const int c = tid;   // SC_THREADS == D
            float w[SC_NQ];
#pragma unroll
            for (int i = 0; i < SC_NQ; ++i) w[i] = 0.0f;
            for (int j = 0; j < D; ++j) {
                const float pv = a.pi_t[j * D + c];
#pragma unroll
                for (int i = 0; i < SC_NQ; ++i) w[i] = fmaf(pv, qs[i * D + j], w[i]);
            }
#pragma unroll
            for (int i = 0; i < SC_NQ; ++i) {
                __half hi, lo;
                sc_split(w[i] * SC_QSCALE, hi, lo);
                const uint32_t off = sc_b_offset(i, c, SC_NQ);
                *reinterpret_cast<__half *>(b1_hi + off) = hi;
                *reinterpret_cast<__half *>(b1_lo + off) = lo;
            }
            cur_head = head;
        }
        reinterpret_cast<uint4 *>(vs)[tid] = v_next[0];
        reinterpret_cast<uint4 *>(vs)[SC_THREADS + tid] = v_next[1];
        const bool more = item + 1 < it1;
        const long long gb_next = more ? block_of(item + 1) : gb;
        if (more) {
            rank_next = __ldg(a.cache.rank + gb_next);
            const uint4 *vsrc = reinterpret_cast<const uint4 *>(a.cache.V + gb_next * RMAX * D);
            v_next[0] = __ldg(vsrc + tid);
            v_next[1] = __ldg(vsrc + SC_THREADS + tid);
        }
        __syncthreads();
        for (int e = tid; e < SC_NQ * RMAX; e += SC_THREADS) {   // Aq[g][i] = q_g . zeta_i
            const int g = e >> 4, i = e & 15;
            float dot = 0.0f;
            if (i < rank && g < gcount) {
                const uint4 *vrow = reinterpret_cast<const uint4 *>(vs + i * D);
                const float4 *qrow = reinterpret_cast<const float4 *>(qs + g * D);
                float d0 = 0.0f, d1 = 0.0f;
#pragma unroll 4
                for (int j = 0; j < D / 8; ++j) {
                    const uint4 v = vrow[j];
                    const float4 qa = qrow[2 * j], qb = qrow[2 * j + 1];
                    const float2 v0 = __half22float2(*reinterpret_cast<const __half2 *>(&v.x));
                    const float2 v1 = __half22float2(*reinterpret_cast<const __half2 *>(&v.y));
                    const float2 v2 = __half22float2(*reinterpret_cast<const __half2 *>(&v.z));
                    const float2 v3 = __half22float2(*reinterpret_cast<const __half2 *>(&v.w));
                    d0 = fmaf(qa.x, v0.x, d0);
                    d1 = fmaf(qa.y, v0.y, d1);
                    d0 = fmaf(qa.z, v1.x, d0);
                    d1 = fmaf(qa.w, v1.y, d1);
                    d0 = fmaf(qb.x, v2.x, d0);
                    d1 = fmaf(qb.y, v2.y, d1);
                    d0 = fmaf(qb.z, v3.x, d0);
                    d1 = fmaf(qb.w, v3.y, d1);
                }
                dot = d0 + d1;
            }
            __half hi, lo;
            sc_split(dot * SC_QSCALE, hi, lo);
            const uint32_t off = sc_b_offset(g, i, SC_NQ);
            *reinterpret_cast<__half *>(b2_hi + off) = hi;
            *reinterpret_cast<__half *>(b2_lo + off) = lo;
        }
        fence_proxy_async_smem();
        __syncthreads();

        bool ok = true;
        for (int tile = 0; tile < tiles; ++tile) {
            const ScTokenData cur = nxt;
            const int tok = tile * 128 + tid;
            if (tile + 1 < tiles) sc_fetch(a, gb, rank, tok + 128, nxt);
            else if (more) sc_fetch(a, gb_next, rank_next, tid, nxt);
            {
                uint32_t av[32];
#pragma unroll
                const uint32_t w0[4] = {cur.c0.x, cur.c0.y, cur.c0.z, cur.c0.w}, w1[4] = {cur.c1.x, cur.c1.y, cur.c1.z, cur.c1.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) sc_expand16(w0[q], a.lo_tab, a.hi_tab, &av[8 * q]);
                tmem_st32(tmem_me + SC_COL_A, av);
#pragma unroll
                for (int q = 0; q < 4; ++q) sc_expand16(w1[q], a.lo_tab, a.hi_tab, &av[8 * q]);
                tmem_st32(tmem_me + SC_COL_A + 32, av);
            }
            {
                uint32_t pw[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t lo = (2 * i < SC_PMAX) ? cur.p[2 * i] : 0u, hi = (2 * i + 1 < SC_PMAX) ? cur.p[2 * i + 1] : 0u;
                    pw[i] = lo | (hi << 16);
                }
                tmem_st8(tmem_me + SC_COL_P, pw);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after_sync();
                const uint32_t h1 = smem_u32(b1_hi), l1 = smem_u32(b1_lo);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t kb = (ks >> 2) * (SC_NQ * 128) + (ks & 3) * 32;
                    umma_f16_ts(tmem0 + SC_COL_D1, tmem0 + SC_COL_A + 8 * ks, umma_desc_sw128(h1 + kb, 16, 1024), idesc, ks ? 1u : 0u);
                    umma_f16_ts(tmem0 + SC_COL_D1, tmem0 + SC_COL_A + 8 * ks, umma_desc_sw128(l1 + kb, 16, 1024), idesc, 1u);
                }
                umma_f16_ts(tmem0 + SC_COL_D2, tmem0 + SC_COL_P, umma_desc_sw128(smem_u32(b2_hi), 16, 1024), idesc, 0u);
                umma_f16_ts(tmem0 + SC_COL_D2, tmem0 + SC_COL_P, umma_desc_sw128(smem_u32(b2_lo), 16, 1024), idesc, 1u);
                umma_commit(&done_bar);
            }
            ok = mbar_wait(&done_bar, done_cnt & 1u, &abort_flag);
            done_cnt += 1;
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t d1[16], d2[16];
            tmem_ld16(tmem_me + SC_COL_D1, d1);
            tmem_ld16(tmem_me + SC_COL_D2, d2);
            tmem_ld_wait();
            if (tok < n) {
                const float f1 = a.scale * __half2float(__ushort_as_half(cur.rho)) * a.inv_code, f2 = a.scale * (1.0f / SC_QSCALE);
                float *dst = a.scores + (head * a.G + a.g0) * (a.bph * n) + jb * n + tok;
#pragma unroll
                for (int g = 0; g < SC_NQ; ++g)
                    if (g < gcount) dst[static_cast<size_t>(g) * (a.bph * n)] = fmaf(f1, __uint_as_float(d1[g]), f2 * __uint_as_float(d2[g]));
            }
            tc_fence_before_sync();
            __syncthreads();
        }
        rank = rank_next;
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

bool scores_ws_supported(const eosq_cache_t &cache, int bits, int n);
bool launch_scores_ws(const eosq_cache_t &cache, int bits, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const uint16_t (&table)[16], float kappa, const __half *q, int G, float scale, float *scores, int *err,
                      int sm_count, void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s);

// 2-bit codes always (the simpler kernel below takes what the warp-specialised one cannot); the other
// widths where the warp-specialised kernel applies.
bool scores_tc_supported(const eosq_cache_t &cache, int bits, int n) {
    return n >= 128 && (bits == 2 || scores_ws_supported(cache, bits, n));
}

bool launch_scores_tc(const eosq_cache_t &cache, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const Codebook &cb, const __half *q, int G, float scale, float *scores, int *err, int sm_count,
                      void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s) {
    static bool configured = false;
    constexpr size_t smem = 24576 + 1024;
    if (!configured) {
        if (cudaFuncSetAttribute(scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
            return false;
        configured = true;
    }
    // the table depends only on the codebook: search once per bit width
    static uint16_t tables[5][16];
    static float kappas[5] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    if (cb.bits < 1 || cb.bits > 4) return false;
    if (kappas[cb.bits] == 0.0f) kappas[cb.bits] = best_table_scale(cb, tables[cb.bits]);
    const uint16_t (&table)[16] = tables[cb.bits];
    const float kappa = kappas[cb.bits];
    if (scores_ws_supported(cache, cb.bits, n))
        return launch_scores_ws(cache, cb.bits, heads, bph, head_stride, n, rot, table, kappa, q, G, scale, scores, err, sm_count, scratch,
                                scratch_bytes, kernels, s);
    if (cb.bits != 2) return false;
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
    const int grid = static_cast<int>(std::min<int64_t>(a.items, 4 * static_cast<int64_t>(sm_count)));
    for (int g0 = 0; g0 < G; g0 += SC_NQ) {
        a.g0 = g0;
        scores_tc_kernel<<<grid, SC_THREADS, smem, s>>>(a);
        *kernels += 1;
    }
    return true;
}

}  // namespace eosq
