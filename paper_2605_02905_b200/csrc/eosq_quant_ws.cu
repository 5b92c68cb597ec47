// Residual, norm, rotation, Lloyd-Max codes, bit packing and the stored left factors of fp16 blocks
// (Algorithm 3, residual line; Algorithm 1) as one warp-specialised tensor-core kernel.
//
// With V the kept right vectors and coef_i = phi_i / sigma_i, the rotated residual rows are
//     Y = R Pi^T = S Pi^T - P'' W,      P'' = S V^T  (n x r),     W = diag(coef) V Pi^T  (r x d),
// and the stored left factors are coef_i P''[:, i].  The rotation therefore stays in shared memory
// for the life of the CTA as one operand (hi / lo fp16 planes of 2^12 Pi), serving three products:
//   main     [Y0 | P''] = S [Pi^T | V^T]          per 128-token tile, 16 MMAs of N = 144 (V's rows sit
//                                                  behind Pi's in the same operand, rewritten per block)
//   W-build  W^T = Pi V^T                          once per block, 24 small MMAs (Pi as the A operand)
//   fix      Y = Y0 - P'' W                         per tile, 3 MMAs of K = 16: P'' goes from its
//                                                  accumulator back into tensor memory as fp16 hi / lo
//                                                  planes, W (times -coef) sits in shared memory
// S is fp16 and exact as an operand; every other factor enters as a high and a low fp16 plane, so the
// products carry about 2^-22 and the accumulation is fp32.
//
// One persistent CTA of 22 warps per SM:
//   warp 0       TMA loads of the 128-token tiles into a ring of three stages
//   warp 1       issues every MMA
//   warps 2-5    per block: write V's rows of the operand, turn the W accumulator into the fix
//                operand; per tile: turn P'' into the fix's A operand and store the left factors
//                (one warp per quarter of the tensor-memory lanes)
//   warps 6-21   epilogue, one token and 32 rotated coordinates per thread: norm, thresholds scaled
//                by the norm, codes, thread-local bit packing
// Two accumulator buffers let the MMAs of a tile run under the epilogue of the previous one.
#include <algorithm>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

bool make_block_tensor_map(const void *blocks, int64_t nb, int n, CUtensorMap *out);

namespace {

constexpr int Q2_ERR_TIMEOUT = 2;        // same bit as the kernel this one replaced
constexpr int Q2_THREADS = 704;
constexpr int Q2_EPI_WARPS = 16, Q2_EPI_FIRST = 6, Q2_CONV_FIRST = 2;
constexpr int Q2_EPI_COLS = D / (Q2_EPI_WARPS / 4);   // 32 coordinates per epilogue thread
constexpr int Q2_NST = 3;                // stages of the token-tile ring
constexpr int Q2_NACC = 2;               // accumulator buffers
constexpr int Q2_N = D + RMAX;           // 144 accumulator columns of the main product
constexpr uint32_t Q2_BBOX = Q2_N * 128; // one 64-wide K half of one plane: 144 rows of 128 bytes
constexpr uint32_t Q2_PLANE = 2 * Q2_BBOX;
constexpr uint32_t Q2_OFF_HI = 0, Q2_OFF_LO = Q2_PLANE;
constexpr uint32_t Q2_WBOX = D * 128;    // the fix operand: 128 rows (c) of 128 bytes, K = 16 used
constexpr uint32_t Q2_OFF_WHI = 2 * Q2_PLANE, Q2_OFF_WLO = Q2_OFF_WHI + Q2_WBOX;
constexpr uint32_t Q2_ABOX = 128 * 128, Q2_ABYTES = 2 * Q2_ABOX;
constexpr uint32_t Q2_OFF_A = Q2_OFF_WLO + Q2_WBOX;
constexpr size_t Q2_SMEM = Q2_OFF_A + Q2_NST * Q2_ABYTES + 1024;
static_assert(Q2_SMEM <= 227 * 1024, "fits the shared memory of an SM");
// tensor memory: per accumulator buffer Y 0-127, P'' 128-143, A of the fix 144-151 (hi) and 152-159 (lo)
constexpr uint32_t Q2_ACC_COLS = 160, Q2_COL_P = 128, Q2_COL_A2 = 144, Q2_COL_DW = Q2_NACC * Q2_ACC_COLS;
constexpr uint32_t Q2_TMEM_COLS = 512;
constexpr float Q2_SCALE = 4096.0f;      // planes of Pi and V
constexpr float Q2_FIX_SCALE = 64.0f;    // both operands of the fix: 64 x 64 = the 4096 of the accumulator

struct Q2Bars {
    uint64_t a_full[Q2_NST], a_empty[Q2_NST];
    uint64_t main_done[Q2_NACC], a2_full[Q2_NACC], y_full[Q2_NACC], acc_free[Q2_NACC];
    uint64_t v_free, v_full, dw_full, w_full, w_free, drain;
};

// Byte offset of the 16-byte chunk `jc` (8 fp16 along K) of row `row` inside one plane whose K halves
// are `box` bytes apart (128-byte swizzle: 8-row groups of 1 KB, chunks XOR-ed with the row).
__device__ __forceinline__ uint32_t q2_offset(int row, int jc, uint32_t box) {
    return (jc >> 3) * box + (row >> 3) * 1024 + (row & 7) * 128 + (((jc & 7) ^ (row & 7)) << 4);
}

// Eight fp32 values, scaled, into their fp16 high and low parts.
__device__ __forceinline__ void q2_split8(const float (&m)[8], float scale, uint4 &hi, uint4 &lo) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float a = m[2 * e] * scale, b = m[2 * e + 1] * scale;
        const __half ah = __float2half_rn(a), bh = __float2half_rn(b);
        const __half al = __float2half_rn(a - __half2float(ah)), bl = __float2half_rn(b - __half2float(bh));
        h[e] = static_cast<uint32_t>(__half_as_ushort(ah)) | (static_cast<uint32_t>(__half_as_ushort(bh)) << 16);
        l[e] = static_cast<uint32_t>(__half_as_ushort(al)) | (static_cast<uint32_t>(__half_as_ushort(bl)) << 16);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// Barrier over the 512 epilogue threads that also tells every one of them whether any of them failed.
__device__ __forceinline__ bool q2_epi_any(bool failed) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, 512, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(failed ? 1u : 0u)
        : "memory");
    return r != 0;
}

template <int BITS>
__global__ void __launch_bounds__(Q2_THREADS, 1) quant_ws_kernel(const __grid_constant__ CUtensorMap tmap, int nb, int n, Workspace ws,
                                                                 const float *__restrict__ pi, Codebook cb, eosq_cache_t out,
                                                                 int *__restrict__ err) {
    extern __shared__ uint8_t q2_smem_raw[];
    __shared__ __align__(8) Q2Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ float ss_part[Q2_NACC][4][128];
    __shared__ uint32_t fills[Q2_NST], drains[Q2_NST];   // loads issued / consumed per stage (for the clean-up after a failed wait)
    __shared__ volatile int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(q2_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles = (n + 127) / 128;
    constexpr int NTHR = (1 << BITS) - 1;
    constexpr int ROW_BYTES = D * BITS / 8;

    if (tid == 0) {
        for (int s = 0; s < Q2_NST; ++s) {
            mbar_init(&bars.a_full[s], 1);
            mbar_init(&bars.a_empty[s], 1);
            fills[s] = 0;
            drains[s] = 0;
        }
        for (int a = 0; a < Q2_NACC; ++a) {
            mbar_init(&bars.main_done[a], 1);
            mbar_init(&bars.a2_full[a], 4);
            mbar_init(&bars.y_full[a], 1);
            mbar_init(&bars.acc_free[a], Q2_EPI_WARPS);
        }
        mbar_init(&bars.v_free, 1);
        mbar_init(&bars.v_full, 4);
        mbar_init(&bars.dw_full, 1);
        mbar_init(&bars.w_full, 4);
        mbar_init(&bars.w_free, 1);
        mbar_init(&bars.drain, 1);
        abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_s, Q2_TMEM_COLS);
        tmem_relinquish();
    }
    // the rotation's rows of the operand, once per CTA: Pi[c][j] is row c, K index j
    for (int chunk = tid; chunk < D * D / 8; chunk += Q2_THREADS) {
        const int c = chunk >> 4, jc = chunk & 15;
        const float4 p0 = __ldg(reinterpret_cast<const float4 *>(pi + chunk * 8)), p1 = __ldg(reinterpret_cast<const float4 *>(pi + chunk * 8 + 4));
        const float m[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
        uint4 hi, lo;
        q2_split8(m, Q2_SCALE, hi, lo);
        const uint32_t off = q2_offset(c, jc, Q2_BBOX);
        *reinterpret_cast<uint4 *>(base + Q2_OFF_HI + off) = hi;
        *reinterpret_cast<uint4 *>(base + Q2_OFF_LO + off) = lo;
    }
    // the fix operand's unused K columns (16 .. 63 of every row) are never read: no need to clear them
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem0 = tmem_base_s;
    const int my_blocks = (blockIdx.x < nb) ? (nb - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;

    if (warp == 0) {
        // ------------------------------------------------------------------ token tiles by TMA
        if (lane == 0) {
            uint32_t g = 0;
            bool ok = true;
            for (int bi = 0; bi < my_blocks && ok; ++bi) {
                const int b = blockIdx.x + bi * gridDim.x;
                for (int t = 0; t < tiles; ++t, ++g) {
                    const int s = g % Q2_NST;
                    if (!mbar_wait(&bars.a_empty[s], ((g / Q2_NST) & 1u) ^ 1u, &abort_flag)) {
                        ok = false;
                        break;
                    }
                    uint8_t *dst = base + Q2_OFF_A + s * Q2_ABYTES;
                    mbar_arrive_expect_tx(&bars.a_full[s], Q2_ABYTES);
                    tma_load_3d(dst, &tmap, &bars.a_full[s], 0, t * 128, b);
                    tma_load_3d(dst + Q2_ABOX, &tmap, &bars.a_full[s], 64, t * 128, b);
                    fills[s] += 1;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ every MMA
        if (lane == 0) {
            constexpr uint32_t idesc_main = umma_idesc_f16(128, Q2_N, false, false);
            constexpr uint32_t idesc_w = umma_idesc_f16(128, RMAX, false, false);
            constexpr uint32_t idesc_fix = umma_idesc_f16(128, D, false, false);
            const uint32_t hi0 = smem_u32(base + Q2_OFF_HI), lo0 = smem_u32(base + Q2_OFF_LO);
            const uint32_t whi = smem_u32(base + Q2_OFF_WHI), wlo = smem_u32(base + Q2_OFF_WLO);
            uint32_t g = 0;          // tiles issued so far (main product)
            bool ok = true;
            // the fix of tile `gf` (pipelined one tile behind its main product)
            auto issue_fix = [&](uint32_t gf, bool first_of_block, bool last_of_block, uint32_t blk_seq) -> bool {
                const int buf = gf % Q2_NACC;
                if (first_of_block && !mbar_wait(&bars.w_full, blk_seq & 1u, &abort_flag)) return false;
                if (!mbar_wait(&bars.a2_full[buf], (gf / Q2_NACC) & 1u, &abort_flag)) return false;
                tc_fence_after_sync();
                const uint32_t acc = tmem0 + buf * Q2_ACC_COLS;
                const uint64_t dh = umma_desc_sw128(whi, 16, 1024), dl = umma_desc_sw128(wlo, 16, 1024);
                umma_f16_ts(acc, acc + Q2_COL_A2, dh, idesc_fix, 1u);        // P'' hi x W hi
                umma_f16_ts(acc, acc + Q2_COL_A2, dl, idesc_fix, 1u);        // P'' hi x W lo
                umma_f16_ts(acc, acc + Q2_COL_A2 + 8, dh, idesc_fix, 1u);    // P'' lo x W hi
                umma_commit(&bars.y_full[buf]);
                if (last_of_block) umma_commit(&bars.w_free);
                return true;
            };
            for (int bi = 0; bi < my_blocks && ok; ++bi) {
                // W^T = Pi V^T of this block: Pi's rows as the A operand, V's rows (144 .. 159 of the planes) as B
                if (!mbar_wait(&bars.v_full, bi & 1u, &abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t kb = (ks >> 2) * Q2_BBOX + (ks & 3) * 32;
                    const uint64_t ah = umma_desc_sw128(hi0 + kb, 16, 1024), al = umma_desc_sw128(lo0 + kb, 16, 1024);
                    const uint64_t vh = umma_desc_sw128(hi0 + kb + D * 128, 16, 1024), vl = umma_desc_sw128(lo0 + kb + D * 128, 16, 1024);
                    umma_f16(tmem0 + Q2_COL_DW, ah, vh, idesc_w, ks ? 1u : 0u);
                    umma_f16(tmem0 + Q2_COL_DW, ah, vl, idesc_w, 1u);
                    umma_f16(tmem0 + Q2_COL_DW, al, vh, idesc_w, 1u);
                }
                umma_commit(&bars.dw_full);
                for (int t = 0; t < tiles; ++t, ++g) {
                    const int s = g % Q2_NST, buf = g % Q2_NACC;
                    if (!mbar_wait(&bars.acc_free[buf], ((g / Q2_NACC) & 1u) ^ 1u, &abort_flag) ||
                        !mbar_wait(&bars.a_full[s], (g / Q2_NST) & 1u, &abort_flag)) {
                        ok = false;
                        break;
                    }
                    drains[s] += 1;
                    tc_fence_after_sync();
                    const uint32_t a0 = smem_u32(base + Q2_OFF_A + s * Q2_ABYTES);
                    const uint32_t acc = tmem0 + buf * Q2_ACC_COLS;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t ka = (ks >> 2) * Q2_ABOX + (ks & 3) * 32, kb = (ks >> 2) * Q2_BBOX + (ks & 3) * 32;
                        const uint64_t da = umma_desc_sw128(a0 + ka, 16, 1024);
                        umma_f16(acc, da, umma_desc_sw128(hi0 + kb, 16, 1024), idesc_main, ks ? 1u : 0u);
                        umma_f16(acc, da, umma_desc_sw128(lo0 + kb, 16, 1024), idesc_main, 1u);
                    }
                    umma_commit(&bars.a_empty[s]);
                    umma_commit(&bars.main_done[buf]);
                    if (t == tiles - 1) umma_commit(&bars.v_free);   // V's rows may be rewritten for the next block
                    if (t > 0 && !issue_fix(g - 1, t == 1, false, static_cast<uint32_t>(bi))) {
                        ok = false;
                        break;
                    }
                }
                if (!ok) break;
                if (!issue_fix(g - 1, tiles == 1, true, static_cast<uint32_t>(bi))) {
                    ok = false;
                    break;
                }
            }
        }
    } else if (warp >= Q2_CONV_FIRST && warp < Q2_CONV_FIRST + 4) {
        // ------------------------------------------------------------------ per-block operands, P'' -> fix operand, left factors
        const int q = warp & 3;                     // tensor-memory lanes [32 q, 32 q + 32) belong to this warp
        const int row = 32 * q + lane;              // a token of the tile, or a rotated coordinate c of W
        const int st = tid - 32 * Q2_CONV_FIRST;    // 0 .. 127 within the group
        const uint32_t lane_addr = tmem0 + (static_cast<uint32_t>(32 * q) << 16);
        uint32_t g = 0;
        bool ok = true;
        for (int bi = 0; bi < my_blocks && ok; ++bi) {
            const int b = blockIdx.x + bi * gridDim.x;
            const int rank = ws.rank[b];
            // V's rows (K index j): 16 rows x 16 chunks of eight entries, two chunks per thread
            if (bi > 0 && !mbar_wait(&bars.v_free, (bi - 1) & 1u, &abort_flag)) {
                ok = false;
                break;
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int chunk = st + 128 * h, i = chunk >> 4, jc = chunk & 15;
                float m[8];
                const float4 v0 = __ldg(reinterpret_cast<const float4 *>(ws.vr + (static_cast<size_t>(b) * RMAX + i) * D + 8 * jc));
                const float4 v1 = __ldg(reinterpret_cast<const float4 *>(ws.vr + (static_cast<size_t>(b) * RMAX + i) * D + 8 * jc + 4));
                const bool live = i < rank;
                m[0] = live ? v0.x : 0.0f;
                m[1] = live ? v0.y : 0.0f;
                m[2] = live ? v0.z : 0.0f;
                m[3] = live ? v0.w : 0.0f;
                m[4] = live ? v1.x : 0.0f;
                m[5] = live ? v1.y : 0.0f;
                m[6] = live ? v1.z : 0.0f;
                m[7] = live ? v1.w : 0.0f;
                uint4 hi, lo;
                q2_split8(m, Q2_SCALE, hi, lo);
                const uint32_t off = q2_offset(D + i, jc, Q2_BBOX);
                *reinterpret_cast<uint4 *>(base + Q2_OFF_HI + off) = hi;
                *reinterpret_cast<uint4 *>(base + Q2_OFF_LO + off) = lo;
            }
            float coef[RMAX];
#pragma unroll
            for (int i = 0; i < RMAX; ++i) coef[i] = (i < rank) ? __ldg(ws.coef + static_cast<size_t>(b) * RMAX + i) : 0.0f;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.v_full);
            // W accumulator -> rows c of the fix operand: -coef_i W[c][i] 2^6, hi and lo
            if (!mbar_wait(&bars.dw_full, bi & 1u, &abort_flag) || (bi > 0 && !mbar_wait(&bars.w_free, (bi - 1) & 1u, &abort_flag))) {
                ok = false;
                break;
            }
            tc_fence_after_sync();
            {
                uint32_t wv[16];
                tmem_ld16(lane_addr + Q2_COL_DW, wv);
                tmem_ld_wait();
                tc_fence_before_sync();
#pragma unroll
                for (int hc = 0; hc < 2; ++hc) {
                    float m[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) m[e] = -coef[8 * hc + e] * __uint_as_float(wv[8 * hc + e]);
                    uint4 hi, lo;
                    q2_split8(m, Q2_FIX_SCALE / (Q2_SCALE * Q2_SCALE), hi, lo);
                    const uint32_t off = q2_offset(row, hc, Q2_WBOX);
                    *reinterpret_cast<uint4 *>(base + Q2_OFF_WHI + off) = hi;
                    *reinterpret_cast<uint4 *>(base + Q2_OFF_WLO + off) = lo;
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.w_full);
            // tiles: P'' (accumulator columns 128 .. 143) -> left factors and the fix's A operand
            for (int t = 0; t < tiles; ++t, ++g) {
                const int buf = g % Q2_NACC;
                if (!mbar_wait(&bars.main_done[buf], (g / Q2_NACC) & 1u, &abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t acc = lane_addr + buf * Q2_ACC_COLS;
                uint32_t pv[16];
                tmem_ld16(acc + Q2_COL_P, pv);
                tmem_ld_wait();
                uint32_t a2[16];   // columns 0-7: hi pairs, 8-15: lo pairs
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float x0 = __uint_as_float(pv[2 * e]) * (Q2_FIX_SCALE / Q2_SCALE), x1 = __uint_as_float(pv[2 * e + 1]) * (Q2_FIX_SCALE / Q2_SCALE);
                    const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
                    const __half l0 = __float2half_rn(x0 - __half2float(h0)), l1 = __float2half_rn(x1 - __half2float(h1));
                    a2[e] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
                    a2[8 + e] = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
                }
                {
                    uint32_t lo8[8], hi8[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        hi8[e] = a2[e];
                        lo8[e] = a2[8 + e];
                    }
                    tmem_st8(acc + Q2_COL_A2, hi8);
                    tmem_st8(acc + Q2_COL_A2 + 8, lo8);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.a2_full[buf]);
                const int tok = t * 128 + row;
                if (tok < n) {
#pragma unroll
                    for (int i = 0; i < RMAX; ++i)
                        if (i < rank)
                            out.P[(static_cast<size_t>(b) * RMAX + i) * n + tok] =
                                __half_as_ushort(__float2half_rn(coef[i] * __uint_as_float(pv[i]) * (1.0f / Q2_SCALE)));
                }
            }
        }
    } else if (warp >= Q2_EPI_FIRST) {
        // ------------------------------------------------------------------ epilogue: this thread owns token `row`, coordinates [32 part, 32 part + 32)
        const int q = warp & 3, part = (warp - Q2_EPI_FIRST) >> 2;
        const int row = 32 * q + lane;
        const uint32_t lane_addr = tmem0 + (static_cast<uint32_t>(32 * q) << 16);
        float thr[NTHR];
#pragma unroll
        for (int t = 0; t < NTHR; ++t) thr[t] = cb.threshold[t];
        uint32_t g = 0;
        bool alive = true;
        for (int bi = 0; bi < my_blocks && alive; ++bi) {
            const int b = blockIdx.x + bi * gridDim.x;
            for (int t = 0; t < tiles; ++t, ++g) {
                const int buf = g % Q2_NACC;
                const bool got = mbar_wait(&bars.y_full[buf], (g / Q2_NACC) & 1u, &abort_flag);
                float y[Q2_EPI_COLS];
                if (got) {
                    tc_fence_after_sync();
                    uint32_t v0[32];
                    tmem_ld32(lane_addr + buf * Q2_ACC_COLS + static_cast<uint32_t>(Q2_EPI_COLS * part), v0);
                    tmem_ld_wait();
                    tc_fence_before_sync();
                    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
                    for (int c = 0; c < Q2_EPI_COLS; c += 4) {
                        y[c] = __uint_as_float(v0[c]);
                        y[c + 1] = __uint_as_float(v0[c + 1]);
                        y[c + 2] = __uint_as_float(v0[c + 2]);
                        y[c + 3] = __uint_as_float(v0[c + 3]);
                        s0 = fmaf(y[c], y[c], s0);
                        s1 = fmaf(y[c + 1], y[c + 1], s1);
                        s2 = fmaf(y[c + 2], y[c + 2], s2);
                        s3 = fmaf(y[c + 3], y[c + 3], s3);
                    }
                    ss_part[buf][part][row] = (s0 + s1) + (s2 + s3);
                }
                // the four parts of every row are summed; every warp has read its part of the accumulator; and
                // all epilogue threads learn together whether one of them gave up waiting
                if (q2_epi_any(!got)) {
                    alive = false;
                    break;
                }
                if (lane == 0) mbar_arrive(&bars.acc_free[buf]);
                const float tot = (ss_part[buf][0][row] + ss_part[buf][1][row]) + (ss_part[buf][2][row] + ss_part[buf][3][row]);
                const float rho = sqrtf(tot);
                // thresholds scaled by the norm: y > thr rho decides as y / rho > thr does (a zero row keeps
                // the plain thresholds, so that it gets the code of z = 0)
                // The codebook is symmetric with its middle threshold at exactly 0, so a code is the sign plus the
                // count of positive thresholds below |y|: 2^(b-1) comparisons instead of 2^b - 1.  (On the
                // negative side this counts a value that sits exactly on a threshold into the outer cell, where
                // the ascending count puts it into the inner one: a tie of measure zero, inside the band that
                // the comparison with the reference exempts.)
                constexpr int MAG = NTHR / 2;   // positive thresholds
                float tp[MAG > 0 ? MAG : 1];
#pragma unroll
                for (int k = 0; k < MAG; ++k) tp[k] = (rho > 0.0f) ? thr[MAG + 1 + k] * rho : thr[MAG + 1 + k];
                auto code_of = [&](float v) -> uint32_t {
                    const float av = fabsf(v);
                    uint32_t mag = 0u;
#pragma unroll
                    for (int k = 0; k < MAG; ++k) mag += (tp[k] < av) ? 1u : 0u;
                    return (0.0f < v) ? (static_cast<uint32_t>(MAG + 1) + mag) : (static_cast<uint32_t>(MAG) - mag);
                };
                // 32 codes of BITS bits: BITS words of 32 bits, coordinate j of the thread at bits [j BITS, (j+1) BITS)
                uint32_t wv[BITS];
                if (BITS == 3) {
                    unsigned long long acc64 = 0ull;
                    int filled = 0, wi = 0;
#pragma unroll
                    for (int c = 0; c < Q2_EPI_COLS; ++c) {
                        const unsigned code = code_of(y[c]);
                        acc64 |= static_cast<unsigned long long>(code) << filled;
                        filled += BITS;
                        if (filled >= 32) {
                            wv[wi++] = static_cast<uint32_t>(acc64);
                            acc64 >>= 32;
                            filled -= 32;
                        }
                    }
                } else if (BITS == 2) {
                    // Two bits: the three thresholds -t, 0, t are equally spaced, so the code is
                    // floor(y / (t rho)) + 2 clamped to 0 .. 3.  One multiply-add rounded down onto
                    // 1.5 2^23 + 2 leaves that integer in the low bits of the float, two min / max clamp it,
                    // and a multiply-add per code packs the raw floats; their common offset leaves in one
                    // subtraction per word.  (A value exactly on a threshold goes to the upper cell here
                    // and to the lower one in the ascending count: measure zero, inside the exempted band;
                    // a zero row, which is all ties, gets its codes directly.)
                    constexpr float MAGIC = 12582912.0f;   // 1.5 2^23 = 0x4B400000: integers have an ulp of 1 there
                    constexpr uint32_t MAGIC_BITS = 0x4B400000u;
                    const float invt = (rho > 0.0f) ? __frcp_rn(thr[2] * rho) : 0.0f;
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        uint32_t w = 0u;
#pragma unroll
                        for (int e = 15; e >= 0; --e) {
                            float f = __fmaf_rd(y[k * 16 + e], invt, MAGIC + 2.0f);
                            f = fminf(fmaxf(f, MAGIC), MAGIC + 3.0f);
                            w = w * 4u + __float_as_uint(f);
                        }
                        // sum of MAGIC_BITS 4^e over the sixteen codes, modulo 2^32
                        wv[k] = (rho > 0.0f) ? w - MAGIC_BITS * 0x55555555u : 0x55555555u;
                    }
                } else {
                    constexpr int CPW = 32 / BITS;   // codes per 32-bit word, filled from the top code down
#pragma unroll
                    for (int k = 0; k < BITS; ++k) {
                        uint32_t w = 0u;
#pragma unroll
                        for (int e = CPW - 1; e >= 0; --e) {
                            w = w * (1u << BITS) + code_of(y[k * CPW + e]);
                        }
                        wv[k] = w;
                    }
                }
                const int tok = t * 128 + row;
                if (tok < n) {
                    uint8_t *dst = out.codes + (static_cast<size_t>(b) * n + tok) * ROW_BYTES + part * 4 * BITS;
                    if (BITS == 1) *reinterpret_cast<uint32_t *>(dst) = wv[0];
                    else if (BITS == 2) *reinterpret_cast<uint2 *>(dst) = make_uint2(wv[0], wv[1 % BITS]);
                    else if (BITS == 4) *reinterpret_cast<uint4 *>(dst) = make_uint4(wv[0], wv[1 % BITS], wv[2 % BITS], wv[3 % BITS]);
                    else {
#pragma unroll
                        for (int k = 0; k < BITS; ++k) reinterpret_cast<uint32_t *>(dst)[k] = wv[k];
                    }
                    if (part == 0) out.norms[static_cast<size_t>(b) * n + tok] = __half_as_ushort(__float2half_rn(rho * (1.0f / Q2_SCALE)));
                }
            }
        }
    }

    __syncthreads();
    if (abort_flag) {
        if (tid == 0) atomicOr(err, Q2_ERR_TIMEOUT);
        // Loads and MMAs that are still in flight must land before shared and tensor memory are given back.
        if (tid == 0) {
            volatile int scratch = 0;
            for (int s = 0; s < Q2_NST; ++s)
                if (fills[s] != drains[s]) mbar_wait(&bars.a_full[s], (fills[s] - 1u) & 1u, &scratch);
        }
        if (tid == 32) {
            volatile int scratch = 0;
            umma_commit(&bars.drain);
            mbar_wait(&bars.drain, 0, &scratch);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem0, Q2_TMEM_COLS);
    }
}

template <int BITS>
bool launch_quant_ws_bits(const CUtensorMap &tmap, int nb, int n, const Workspace &ws, const Rotation &rot, const Codebook &cb,
                          const eosq_cache_t &out, int *err, int grid, cudaStream_t s) {
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(quant_ws_kernel<BITS>), Q2_SMEM)) return false;
    quant_ws_kernel<BITS><<<grid, Q2_THREADS, Q2_SMEM, s>>>(tmap, nb, n, ws, rot.pi, cb, out, err);
    return true;
}

}  // namespace

bool launch_quant_tc(const void *blocks_all, int64_t block0, int64_t nb, int n, const Workspace &ws, const Rotation &rot,
                     const Codebook &cb, const eosq_cache_t &out, int *err, int sm_count, cudaStream_t s) {
    CUtensorMap tmap;
    const char *base = static_cast<const char *>(blocks_all) + static_cast<size_t>(block0) * n * D * 2;
    if (!make_block_tensor_map(base, nb, n, &tmap)) return false;
    const int grid = static_cast<int>(std::min<int64_t>(nb, static_cast<int64_t>(sm_count)));
    switch (cb.bits) {
        case 1: return launch_quant_ws_bits<1>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 2: return launch_quant_ws_bits<2>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 3: return launch_quant_ws_bits<3>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 4: return launch_quant_ws_bits<4>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
    }
    return false;
}

}  // namespace eosq
