// Tensor-core decode for 1- to 4-bit codes (Algorithm 1 DeQuant + the stored low-rank part):
//   x_t = rho_t (z_t Pi) + sum_i P[t][i] zeta_i,     z_t = centroids of the codes of token t.
//
// One persistent CTA of 512 threads per SM holds the rotation once, as the B operand of
//   D1[128 tokens][128] = Z[128][128] (fp16 centroids) x Pi      (Pi scaled by 2^12 and split
//                                                                  into a high and a low fp16 plane),
//   D2[128 tokens][128] = P_tile[128][16] x V[16][128]            (stored fp16 factors: exact products),
// both accumulated in fp32 in tensor memory.  The two halves of the CTA (256 threads each) work
// on different blocks like two CTAs would - each with its own operand buffers, half of the tensor
// memory and its own barriers - so that one half's MMAs overlap the other's expansion and stores.
// Per 128-token tile a half expands the codes into a K-major 128-byte-swizzled A tile (byte
// permutes), writes the factor rows next to it, one thread issues the 17 MMAs, and every thread
// turns 64 columns of one token's accumulators into rho D1 / (kappa 2^12) + D2 and stores them.
#include <algorithm>
#include <cstdint>
#include <cstring>

#include "eosq_common.cuh"
#include "eosq_expand.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

constexpr int TC_ERR_DECODE_TIMEOUT = 16;

constexpr int DT_THREADS = 512, DT_HALF = 256;
constexpr float DT_PSCALE = 4096.0f;                  // keeps the low plane of Pi in fp16's normal range
constexpr uint32_t DT_BOX = 128 * 128;                // 128 rows x 64 fp16 of K
constexpr uint32_t DT_OFF_PI_HI = 0, DT_OFF_PI_LO = 2 * DT_BOX;
constexpr uint32_t DT_OFF_HALF = 4 * DT_BOX;          // per half: A tile (2 boxes), factor tile (1 box), right vectors (1 box)
constexpr uint32_t DT_H_A = 0, DT_H_P = 2 * DT_BOX, DT_H_V = 3 * DT_BOX;
// ... and the raw data of the next tile, copied in while the current one is worked on: packed codes
// (128 tokens x 16 BITS bytes), norms, up to 12 factor rows of 128 fp16
constexpr int DT_PMAX = 12;
constexpr uint32_t DT_H_RAW = 4 * DT_BOX;
constexpr uint32_t DT_RAW_BYTES = 12288;
static_assert(128 * 64 + 256 + DT_PMAX * 256 <= DT_RAW_BYTES && KPILOT < DT_PMAX, "the raw area holds one tile of 4-bit codes");
constexpr uint32_t DT_HALF_BYTES = 4 * DT_BOX + DT_RAW_BYTES;
constexpr size_t DT_SMEM = DT_OFF_HALF + 2 * DT_HALF_BYTES + 1024;   // 217 KB
constexpr uint32_t DT_TMEM_COLS = 512;                // per half: D1 128 columns, D2 128 columns

// Byte offset of the 16-byte chunk `jc` (8 fp16 of K) of row `row` in a K-major, 128-byte-swizzled
// operand of 128 rows: 64-wide K boxes of 16 KB, 8-row groups of 1 KB, chunks XOR-ed with the row.
__device__ __forceinline__ uint32_t dt_offset(int row, int jc) {
    return (jc >> 3) * DT_BOX + (row >> 3) * 1024 + (row & 7) * 128 + (((jc & 7) ^ (row & 7)) << 4);
}

__device__ __forceinline__ void dt_bar_sync(int half) {
    asm volatile("bar.sync %0, %1;" ::"r"(1 + half), "r"(DT_HALF) : "memory");
}
// The same barrier, telling every thread of the half whether any of them brings `failed`.  A bounded
// wait ends per thread, so one thread may give up where its neighbour just succeeds: the outcome is
// made common here, at the next barrier of the half, and the half leaves its loop as a whole (a
// thread that left alone would let this barrier wait for ever).
__device__ __forceinline__ bool dt_bar_any(int half, bool failed) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(failed ? 1u : 0u), "r"(1 + half), "r"(DT_HALF)
        : "memory");
    return r != 0;
}

struct DecodeArgs {
    eosq_cache_t cache;
    int nb, n;
    float inv_scale;            // 1 / (kappa 2^12)
    uint32_t lo_tab[4], hi_tab[4];   // low / high bytes of the fp16 centroids times kappa (level k in byte k)
    const float *pi_t;          // pi_t[j][c] = Pi[c][j]
    void *out;
    int *err;
};

__device__ __forceinline__ void dt_bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :
                 : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

bool make_block_tensor_map(const void *blocks, int64_t nb, int n, CUtensorMap *out);

// `omap` (fp16 output only): the output as [nb][n][128] fp16 with boxes of 128 tokens x 64 coordinates,
// 128-byte swizzled - the layout of the A tile, which doubles as the staging buffer of the stores.
template <typename Tout, int BITS>
__global__ void __launch_bounds__(DT_THREADS, 1) decode_tc_kernel(const DecodeArgs a, const __grid_constant__ CUtensorMap omap) {
    static_assert(BITS >= 1 && BITS <= 4, "code widths of the format");
    extern __shared__ uint8_t dt_smem_raw[];
    __shared__ __align__(8) uint64_t mma_done[2], raw_full[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dt_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5;
    const int half = tid >> 8, ht = tid & (DT_HALF - 1);
    const int r = ht & 127, box = ht >> 7;   // token within the tile (= tensor-memory lane), column half
    const int n = a.n, tiles = (n + 127) / 128;

    if (tid == 0) {
        mbar_init(&mma_done[0], 1);
        mbar_init(&mma_done[1], 1);
        mbar_init(&raw_full[0], 1);
        mbar_init(&raw_full[1], 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, DT_TMEM_COLS);
        tmem_relinquish();
    }
    // B operand of D1, once per CTA: row j (output coordinate), K = c: Pi[c][j] 2^12 as high + low fp16
    for (int chunk = tid; chunk < D * (D / 8); chunk += DT_THREADS) {
        const int j = chunk >> 4, jc = chunk & 15;
        const float4 p0 = __ldg(reinterpret_cast<const float4 *>(a.pi_t + j * D + 8 * jc));
        const float4 p1 = __ldg(reinterpret_cast<const float4 *>(a.pi_t + j * D + 8 * jc + 4));
        const float m[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
        uint32_t h[4], l[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float x0 = m[2 * e] * DT_PSCALE, x1 = m[2 * e + 1] * DT_PSCALE;
            const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
            const __half l0 = __float2half_rn(x0 - __half2float(h0)), l1 = __float2half_rn(x1 - __half2float(h1));
            h[e] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
            l[e] = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
        }
        const uint32_t off = dt_offset(j, jc);
        *reinterpret_cast<uint4 *>(base + DT_OFF_PI_HI + off) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4 *>(base + DT_OFF_PI_LO + off) = make_uint4(l[0], l[1], l[2], l[3]);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    uint8_t *hbase = base + DT_OFF_HALF + half * DT_HALF_BYTES;
    const uint32_t d1 = tmem_base_s + 256u * half, d2 = d1 + 128u;
    const uint32_t lane_off = static_cast<uint32_t>(32 * (warp & 3)) << 16;   // a warp reaches lanes 32 (warp % 4)..
    const uint16_t *Pg = a.cache.P;
    Tout *outp = static_cast<Tout *>(a.out);

    // The second warp of the half asks the copy engine for the raw data of a tile, one copy per lane (a
    // thread needs over 100 cycles per copy it issues, and the first warp's lane 0 is busy issuing MMAs).
    // Ranks are clamped to the rows the raw area holds; the library never stores more than the pilot k = 11.
    constexpr uint32_t ROW = 16 * BITS, DT_RAW_NORMS = 128 * ROW, DT_RAW_P = DT_RAW_NORMS + 256;
    uint8_t *raw = hbase + DT_H_RAW;
    const int cl = ht - 32;   // lane of the copying warp
    auto issue = [&](long long blk, int tile, int rank) {
        const int tok0 = tile * 128;
        const uint32_t rows = static_cast<uint32_t>(min(128, n - tok0));
        const size_t t0 = static_cast<size_t>(blk) * n + tok0;
        if (cl == 0) mbar_arrive_expect_tx(&raw_full[half], rows * (ROW + 2u) + static_cast<uint32_t>(rank) * rows * 2u);
        __syncwarp();   // the byte count is announced before any copy can report completion
        if (cl == 0) {
            dt_bulk_load(raw, a.cache.codes + t0 * ROW, rows * ROW, &raw_full[half]);
        } else if (cl == 1) {
            dt_bulk_load(raw + DT_RAW_NORMS, a.cache.norms + t0, rows * 2u, &raw_full[half]);
        } else if (cl - 2 < rank) {
            const int i = cl - 2;
            dt_bulk_load(raw + DT_RAW_P + i * 256, Pg + (static_cast<size_t>(blk) * RMAX + i) * n + tok0, rows * 2u, &raw_full[half]);
        }
    };

    uint32_t phase = 0, raw_phase = 0;
    bool alive = true, store_pending = false;
    const long long blk0 = 2ll * blockIdx.x + half, bstep = 2ll * gridDim.x;
    int rank_next = (blk0 < a.nb) ? max(0, min(a.cache.rank[blk0], DT_PMAX)) : 0;
    if (ht >= 32 && ht < 64 && blk0 < a.nb) issue(blk0, 0, rank_next);
    for (long long blk = blk0; blk < a.nb && alive; blk += bstep) {
        const int rank = rank_next;
        if (blk + bstep < a.nb) rank_next = max(0, min(a.cache.rank[blk + bstep], DT_PMAX));   // known long before the next block starts
        {   // B operand of D2: row j, K = i: zeta_i[j] (zero beyond the rank); this thread: row r, entries 8 box .. 8 box + 7
            uint32_t vw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int i = 8 * box + e;
                if (i < rank) vw[e >> 1] |= static_cast<uint32_t>(a.cache.V[(static_cast<size_t>(blk) * RMAX + i) * D + r]) << (16 * (e & 1));
            }
            *reinterpret_cast<uint4 *>(hbase + DT_H_V + dt_offset(r, box)) = make_uint4(vw[0], vw[1], vw[2], vw[3]);
        }
        for (int tile = 0; tile < tiles; ++tile) {
            const bool valid = tile * 128 + r < n;
            // the tile's raw data (asked for one tile ago); rows past the end of the block were not copied
            // (a thread whose wait gave up works on with whatever the raw area holds, up to the barrier
            // below the operand stores, where the half learns of it)
            const bool raw_ok = mbar_wait(&raw_full[half], raw_phase, &abort_flag);
            raw_phase ^= 1u;
            uint32_t cw[2 * BITS];
#pragma unroll
            for (int w = 0; w < BITS; ++w) {
                const uint2 v = *reinterpret_cast<const uint2 *>(raw + r * ROW + 8 * BITS * box + 8 * w);
                cw[2 * w] = valid ? v.x : 0u;
                cw[2 * w + 1] = valid ? v.y : 0u;
            }
            const uint32_t rho_raw = valid ? *reinterpret_cast<const unsigned short *>(raw + DT_RAW_NORMS + 2 * r) : 0u;
            uint32_t pw[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) pw[i] = 0u;
            if (box == 0 && valid) {
#pragma unroll
                for (int i = 0; i < DT_PMAX; ++i)
                    if (i < rank) pw[i >> 1] |= static_cast<uint32_t>(*reinterpret_cast<const unsigned short *>(raw + DT_RAW_P + i * 256 + 2 * r)) << (16 * (i & 1));
            }
            {   // A operand of D1: this token's 64 coordinates of column half `box`, as fp16 centroids
                uint32_t o[4][8];
#pragma unroll
                for (int q = 0; q < 4; ++q) expand16_codes<BITS>(cw, q, a.lo_tab, a.hi_tab, o[q]);
                // the tile still holds the previous tile's output until the copy engine has read it: the
                // expansion above ran in the shadow of that read
                if (store_pending) {
                    if (ht == 0) bulk_wait_read_all();
                    dt_bar_sync(half);
                    store_pending = false;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    *reinterpret_cast<uint4 *>(hbase + DT_H_A + dt_offset(r, 8 * box + 2 * q)) = make_uint4(o[q][0], o[q][1], o[q][2], o[q][3]);
                    *reinterpret_cast<uint4 *>(hbase + DT_H_A + dt_offset(r, 8 * box + 2 * q + 1)) = make_uint4(o[q][4], o[q][5], o[q][6], o[q][7]);
                }
                if (box == 0) {   // A operand of D2: the token's factor entries
                    *reinterpret_cast<uint4 *>(hbase + DT_H_P + dt_offset(r, 0)) = make_uint4(pw[0], pw[1], pw[2], pw[3]);
                    *reinterpret_cast<uint4 *>(hbase + DT_H_P + dt_offset(r, 1)) = make_uint4(pw[4], pw[5], pw[6], pw[7]);
                }
            }
            const float f = __half2float(__ushort_as_half(static_cast<unsigned short>(rho_raw))) * a.inv_scale;
            fence_proxy_async_smem();   // the operands were written by ordinary stores and are read by the tensor core
            if (dt_bar_any(half, !raw_ok)) {
                alive = false;
                raw_phase ^= 1u;   // the phase that did not complete is the one the final drain waits for
                break;
            }
            if (ht == 0) {
                tc_fence_after_sync();
                constexpr uint32_t idesc = umma_idesc_f16(128, D, false, false);
                const uint32_t a0 = smem_u32(hbase + DT_H_A), hi0 = smem_u32(base + DT_OFF_PI_HI), lo0 = smem_u32(base + DT_OFF_PI_LO);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t ko = (ks >> 2) * DT_BOX + (ks & 3) * 32;
                    const uint64_t da = umma_desc_sw128(a0 + ko, 16, 1024);
                    umma_f16(d1, da, umma_desc_sw128(hi0 + ko, 16, 1024), idesc, ks ? 1u : 0u);
                    umma_f16(d1, da, umma_desc_sw128(lo0 + ko, 16, 1024), idesc, 1u);
                }
                umma_f16(d2, umma_desc_sw128(smem_u32(hbase + DT_H_P), 16, 1024), umma_desc_sw128(smem_u32(hbase + DT_H_V), 16, 1024), idesc, 0u);
                umma_commit(&mma_done[half]);
            } else if (ht >= 32 && ht < 64) {
                // every thread has taken its part of the raw area (the barrier above): ask for the next tile
                if (tile + 1 < tiles) issue(blk, tile + 1, rank);
                else if (blk + bstep < a.nb) issue(blk + bstep, 0, rank_next);
            }
            // (likewise: a thread that gave up reads accumulators that may not be final, and the barrier
            // behind the epilogue ends the loop for the whole half before anything of the tile is stored)
            const bool mma_ok = mbar_wait(&mma_done[half], phase, &abort_flag);
            phase ^= 1u;
            tc_fence_after_sync();
            const int tok = tile * 128 + r;
            Tout *dst = outp + (static_cast<size_t>(blk) * n + tok) * D + 64 * box;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t v1[32], v2[32];
                tmem_ld32(d1 + lane_off + 64u * box + 32u * c, v1);
                tmem_ld32(d2 + lane_off + 64u * box + 32u * c, v2);
                tmem_ld_wait();
                if (tok < n || sizeof(Tout) == 2) {   // rows past the end are clipped by the tensor store
                    if (sizeof(Tout) == 2) {
                        uint32_t pk[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float x0 = fmaf(f, __uint_as_float(v1[2 * e]), __uint_as_float(v2[2 * e]));
                            const float x1 = fmaf(f, __uint_as_float(v1[2 * e + 1]), __uint_as_float(v2[2 * e + 1]));
                            pk[e] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(x0))) |
                                    (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(x1))) << 16);
                        }
                        // into the A tile (its MMAs are over), in the swizzled layout a tensor store turns back into rows:
                        // a thread's own 16-byte stores to global memory would touch 32 sectors per warp instruction
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            *reinterpret_cast<uint4 *>(hbase + DT_H_A + dt_offset(r, 8 * box + 4 * c + e)) =
                                make_uint4(pk[4 * e], pk[4 * e + 1], pk[4 * e + 2], pk[4 * e + 3]);
                    } else {
                        float4 *d4 = reinterpret_cast<float4 *>(dst + 32 * c);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            d4[e] = make_float4(fmaf(f, __uint_as_float(v1[4 * e]), __uint_as_float(v2[4 * e])),
                                                fmaf(f, __uint_as_float(v1[4 * e + 1]), __uint_as_float(v2[4 * e + 1])),
                                                fmaf(f, __uint_as_float(v1[4 * e + 2]), __uint_as_float(v2[4 * e + 2])),
                                                fmaf(f, __uint_as_float(v1[4 * e + 3]), __uint_as_float(v2[4 * e + 3])));
                    }
                }
            }
            if (sizeof(Tout) == 2) {
                fence_proxy_async_smem();   // the staged tile was written by ordinary stores and is read by the copy engine
                tc_fence_before_sync();
                if (dt_bar_any(half, !mma_ok)) {
                    alive = false;
                    break;
                }
                if (ht == 0) {
                    tma_store_3d(&omap, hbase + DT_H_A, 0, tile * 128, static_cast<int>(blk));
                    tma_store_3d(&omap, hbase + DT_H_A + DT_BOX, 64, tile * 128, static_cast<int>(blk));
                    bulk_commit_group();
                }
                store_pending = true;   // waited for before the tile is overwritten
            } else {
                tc_fence_before_sync();
                if (dt_bar_any(half, !mma_ok)) {   // operands and accumulators are free for the next tile
                    alive = false;
                    break;
                }
            }
        }
    }

    if (!alive && ht == 0) {   // gave up with a copy of raw data possibly in flight: let it land before the CTA goes away
        volatile int unused = 0;
        mbar_wait(&raw_full[half], raw_phase, &unused);
    }
    if (sizeof(Tout) == 2 && ht == 0) bulk_wait_all();
    __syncthreads();
    if (abort_flag && tid == 0) atomicOr(a.err, TC_ERR_DECODE_TIMEOUT);
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base_s, DT_TMEM_COLS);
    }
}

float best_table_scale(const Codebook &cb, uint16_t (&table)[16]);

bool decode_tc_supported(const eosq_cache_t &cache, int bits, const void *out_blocks) {
    auto aligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };   // bulk copies and tensor stores
    return bits >= 1 && bits <= 4 && aligned(cache.codes) && aligned(cache.norms) && aligned(cache.P) && aligned(out_blocks);
}

template <typename Tout, int BITS>
static bool launch_decode_tc_as(const DecodeArgs &a, const CUtensorMap &omap, int grid, cudaStream_t s) {
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(decode_tc_kernel<Tout, BITS>), DT_SMEM)) return false;
    decode_tc_kernel<Tout, BITS><<<grid, DT_THREADS, DT_SMEM, s>>>(a, omap);
    return true;
}

bool launch_decode_tc(const eosq_cache_t &cache, int64_t nb, int n, const Rotation &rot, const Codebook &cb, void *out_blocks,
                      int out_dtype, int *err, int sm_count, cudaStream_t s) {
    // the centroid table depends only on the codebook: search its scale once per code width
    static uint16_t table[5][16];
    static float kappa[5] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    const int bits = cb.bits;
    if (bits < 1 || bits > 4) return false;
    if (kappa[bits] == 0.0f) kappa[bits] = best_table_scale(cb, table[bits]);
    DecodeArgs a;
    a.cache = cache;
    a.nb = static_cast<int>(nb);
    a.n = n;
    a.inv_scale = 1.0f / (kappa[bits] * DT_PSCALE);
    for (int w = 0; w < 4; ++w) a.lo_tab[w] = a.hi_tab[w] = 0u;
    for (int k = 0; k < (1 << bits); ++k) {
        a.lo_tab[k >> 2] |= static_cast<uint32_t>(table[bits][k] & 0xFFu) << (8 * (k & 3));
        a.hi_tab[k >> 2] |= static_cast<uint32_t>(table[bits][k] >> 8) << (8 * (k & 3));
    }
    a.pi_t = rot.pi_t;
    a.out = out_blocks;
    a.err = err;
    const int grid = static_cast<int>(std::min<int64_t>((nb + 1) / 2, sm_count));
    CUtensorMap omap;
    std::memset(&omap, 0, sizeof(omap));
    if (out_dtype == EOSQ_F32) {
        switch (bits) {
            case 1: return launch_decode_tc_as<float, 1>(a, omap, grid, s);
            case 2: return launch_decode_tc_as<float, 2>(a, omap, grid, s);
            case 3: return launch_decode_tc_as<float, 3>(a, omap, grid, s);
            default: return launch_decode_tc_as<float, 4>(a, omap, grid, s);
        }
    }
    if (!make_block_tensor_map(out_blocks, nb, n, &omap)) return false;
    switch (bits) {
        case 1: return launch_decode_tc_as<__half, 1>(a, omap, grid, s);
        case 2: return launch_decode_tc_as<__half, 2>(a, omap, grid, s);
        case 3: return launch_decode_tc_as<__half, 3>(a, omap, grid, s);
        default: return launch_decode_tc_as<__half, 4>(a, omap, grid, s);
    }
}

}  // namespace eosq
