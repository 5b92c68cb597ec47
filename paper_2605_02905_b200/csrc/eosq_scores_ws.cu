// Warp-specialised attention-logit kernel for 1- to 4-bit codes (Remark 6.4): one persistent CTA of 16
// warps per SM in which loading, code expansion, the MMAs and the output run concurrently on
// different tiles.
//
//   warp 0        bulk-copies each 128-token tile (codes, norms, factor rows) and each block's right
//                 vectors from global memory into a ring of shared-memory stages
//   warps 2-3     build the query-side operands: W = Pi q once per head, Aq = q V^T once per block
//   warps 4-11    two groups of four: expand a tile's codes to fp16 centroids (byte permutes) and
//                 store them, the factor entries and the row norm into one of four tensor-memory
//                 buffers, one token per thread
//   warp 1        issues the nine MMAs of a tile (A from tensor memory, B from shared memory)
//   warps 12-15   read the accumulators back, apply norm and scale, write the logits
//
// The high and the low fp16 plane of a query-side operand are stacked along N (columns g and
// 8 + g of one 16-column accumulator), so a pass serves eight query vectors.
#include <algorithm>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"
#include "eosq_expand.cuh"

namespace eosq {

using namespace sm100;

constexpr int TC_ERR_SCORES_WS_TIMEOUT = 8;

constexpr int WS_THREADS = 512;
constexpr int WS_NQ = 8;                   // query vectors per pass
constexpr int WS_STAGES = 5;               // shared-memory stages of WS_TPS tiles each (four with 4-bit codes: their stages are larger)
constexpr int WS_TPS = 4;                  // tiles per stage: few large copies keep the copy engine's queue short
constexpr int WS_BUFS = 4;
constexpr int WS_PMAX = 12;                // factor rows staged per tile (rank <= pilot k = 11)
// a stage holds 512 tokens: codes (16 BITS bytes per token), norms, 2 boxes of 12 x 256 factors
constexpr uint32_t WS_ST_CODES = 0;
constexpr uint32_t WS_ST_PBOX = WS_PMAX * 512;
template <int BITS> struct WsLayout {
    static constexpr uint32_t ROW = 16 * BITS;                              // code bytes per token
    static constexpr int STAGES = (BITS == 4) ? WS_STAGES - 1 : WS_STAGES;
    static constexpr uint32_t ST_NORMS = 512 * ROW, ST_P = ST_NORMS + 1024;
    static constexpr uint32_t STAGE_BYTES = ST_P + 2 * WS_ST_PBOX;         // 29696 (2 bits), 37888 (3 bits)
    static constexpr uint32_t OFF_B1 = STAGES * STAGE_BYTES;            // 2 x 4096: W, hi rows 0-7, lo rows 8-15
    static constexpr uint32_t OFF_B2 = OFF_B1 + 2 * 4096;                  // 2 x 2048: Aq
    static constexpr uint32_t OFF_V = OFF_B2 + 2 * 2048;                   // 2 x 4096: right vectors (fp16)
    static constexpr uint32_t OFF_Q = OFF_V + 2 * 4096;                    // 2 x (8 x 128) fp32 queries, by head parity
    static constexpr uint32_t SMEM_BYTES = OFF_Q + 2 * WS_NQ * D * 4 + 1024;
};
constexpr uint32_t WS_TMEM_COLS = 512;
constexpr uint32_t WS_BUF_COLS = 112;      // per buffer: A 0-63, P 64-71, rho 72, D1 80-95, D2 96-111
constexpr uint32_t WS_COL_P = 64, WS_COL_RHO = 72, WS_COL_D1 = 80, WS_COL_D2 = 96;
constexpr float WS_QSCALE = 256.0f;

struct WsArgs {
    eosq_cache_t cache;
    int bph, head_stride, heads;   // blocks per head, block stride between heads, heads
    int n, G, g0;
    float scale, inv_code;
    uint32_t lo_tab[4], hi_tab[4];   // low / high bytes of the fp16 centroids times kappa (level k in byte k)
    const uint8_t *wimg;   // per head: the 4096-byte image of the operand W = Pi q (made by scores_w_kernel)
    const __half *q;
    float *scores;
    int *err;
};

__device__ __forceinline__ void ws_bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :
                 : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Byte offset of element (row, k) of a K-major, 128-byte-swizzled operand with 16 rows per 64-wide K box.
__device__ __forceinline__ uint32_t ws_b_offset(int row, int k) {
    const int box = k >> 6, kk = k & 63;
    return box * 2048 + row * 128 + ((((kk >> 3) ^ (row & 7)) << 4) | ((kk & 7) << 1));
}

__device__ __forceinline__ void ws_split_store(uint8_t *plane, int g, int k, float v) {
    const __half hi = __float2half_rn(v), lo = __float2half_rn(v - __half2float(hi));
    *reinterpret_cast<__half *>(plane + ws_b_offset(g, k)) = hi;
    *reinterpret_cast<__half *>(plane + ws_b_offset(WS_NQ + g, k)) = lo;
}

// Barrier of the 64 threads of the operand builder that also tells each of them whether any brings
// `failed` (the outcome of a bounded wait, which ends per thread).
__device__ __forceinline__ bool ws_builder_any(bool failed) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 2, 64, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(failed ? 1u : 0u)
        : "memory");
    return r != 0;
}

struct WsBarriers {
    uint64_t st_full[WS_STAGES], st_empty[WS_STAGES];
    uint64_t a_full[WS_BUFS], d_full[WS_BUFS], d_empty[WS_BUFS];
    uint64_t blk_full[2], blk_empty[2], b2_full[2], b2_empty[2], b1_full[2], b1_empty[2];
};

bool make_factor_tensor_map(const void *P, int64_t nb, int n, int rows, CUtensorMap *out);

// W = Pi q for the (at most eight) query vectors g0.. of every head, times 2^8, split into a high and a low
// fp16 plane and laid out as the score kernel's B operand (rows g and 8 + g of a K-major, 128-byte-swizzled
// tile of 16 rows x 128): one 4096-byte image per head, which the score kernel fetches with one bulk copy.
__global__ void __launch_bounds__(D) scores_w_kernel(const float *__restrict__ pi_t, const __half *__restrict__ q, int G, int g0,
                                                     uint8_t *__restrict__ wimg) {
    __shared__ float qs[WS_NQ][D];
    const int c = threadIdx.x, hd = blockIdx.x;
    const int gcount = min(WS_NQ, G - g0);
    for (int g = 0; g < WS_NQ; ++g) qs[g][c] = (g < gcount) ? __half2float(q[(static_cast<long long>(hd) * G + g0 + g) * D + c]) : 0.0f;
    __syncthreads();
    float w[WS_NQ];
#pragma unroll
    for (int g = 0; g < WS_NQ; ++g) w[g] = 0.0f;
#pragma unroll 1
    for (int j0 = 0; j0 < D; j0 += 32) {
        float pv[32];
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) pv[jj] = __ldg(pi_t + (j0 + jj) * D + c);   // 32 loads in flight: the kernel is all L2 latency
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) {
#pragma unroll
            for (int g = 0; g < WS_NQ; ++g) w[g] = fmaf(pv[jj], qs[g][j0 + jj], w[g]);
        }
    }
    uint8_t *img = wimg + static_cast<size_t>(hd) * 4096;
#pragma unroll
    for (int g = 0; g < WS_NQ; ++g) ws_split_store(img, g, c, w[g] * WS_QSCALE);
}

template <int BITS>
__global__ void __launch_bounds__(WS_THREADS, 1) scores_ws_kernel(const WsArgs a, const __grid_constant__ CUtensorMap pmap4,
                                                                  const __grid_constant__ CUtensorMap pmap8,
                                                                  const __grid_constant__ CUtensorMap pmap12) {
    using L = WsLayout<BITS>;
    extern __shared__ uint8_t ws_smem_raw[];
    __shared__ __align__(8) WsBarriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int st_rank[WS_STAGES];
    __shared__ volatile int abort_flag;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(ws_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = a.n, tiles = (n + 127) / 128;
    const int gcount = min(WS_NQ, a.G - a.g0);

    if (tid == 0) {
        for (int s = 0; s < WS_STAGES; ++s) {
            mbar_init(&bars.st_full[s], 1);
            mbar_init(&bars.st_empty[s], 4 * WS_TPS);   // one arrival per expander warp and tile slot
        }
        for (int b = 0; b < WS_BUFS; ++b) {
            mbar_init(&bars.a_full[b], 4);             // one arrival per warp: 128 arrivals on one barrier serialise
            mbar_init(&bars.d_full[b], 1);
            mbar_init(&bars.d_empty[b], 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars.blk_full[b], 1);
            mbar_init(&bars.blk_empty[b], 1);
            mbar_init(&bars.b2_full[b], 1);
            mbar_init(&bars.b2_empty[b], 1);
            mbar_init(&bars.b1_full[b], 1);
            mbar_init(&bars.b1_empty[b], 1);
        }
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_s, WS_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem0 = tmem_base_s;

    // contiguous range of (head, block) items of this CTA; every role walks it in the same order
    const int items = a.heads * a.bph;
    const int ipc = (items + gridDim.x - 1) / gridDim.x;
    const int it0 = min(items, ipc * static_cast<int>(blockIdx.x)), it1 = min(items, it0 + ipc);

    if (warp == 0) {
        // ---------------------------------------------------------------- loader
        // Lane 0 keeps the protocol (waits, expected byte counts) and fetches the factor rows of a tile with
        // one tensor copy (4, 8 or 12 rows, whichever covers the rank); lane 30 copies the codes, lane 31
        // the norms.
        if (it0 < it1) {
            uint32_t sseq = 0;
            int head = it0 / a.bph, jb = it0 - head * a.bph;
            int rank_next = min(__ldg(a.cache.rank + static_cast<long long>(head) * a.head_stride + jb), WS_PMAX);
            bool alive = true;
            for (int item = it0, bi = 0; item < it1 && alive; ++item, ++bi) {
                const long long gb = static_cast<long long>(head) * a.head_stride + jb;
                const int rank = rank_next;
                int nhead = head, njb = jb + 1;
                if (njb == a.bph) {
                    njb = 0;
                    nhead += 1;
                }
                if (item + 1 < it1) rank_next = min(__ldg(a.cache.rank + static_cast<long long>(nhead) * a.head_stride + njb), WS_PMAX);
                const int vb = bi & 1;
                if (lane == 0) {
                    alive = mbar_wait(&bars.blk_empty[vb], ((bi >> 1) & 1u) ^ 1u, &abort_flag);
                    if (alive) {
                        mbar_arrive_expect_tx(&bars.blk_full[vb], 4096);
                        ws_bulk_load(base + L::OFF_V + vb * 4096, a.cache.V + gb * RMAX * D, 4096, &bars.blk_full[vb]);
                    }
                }
                alive = __shfl_sync(0xffffffffu, alive, 0);
                for (int tile = 0; tile < tiles && alive; tile += WS_TPS, ++sseq) {
                    const int stage = sseq % L::STAGES;
                    const int tok0 = tile * 128;
                    const uint32_t rows = static_cast<uint32_t>(min(128 * WS_TPS, n - tok0));
                    const uint32_t boxes = (rows + 255u) >> 8;
                    const int r4 = (rank + 3) >> 2;
                    if (lane == 0) {
                        alive = mbar_wait(&bars.st_empty[stage], ((sseq / L::STAGES) & 1u) ^ 1u, &abort_flag);
                        if (alive) {
                            st_rank[stage] = rank;
                            mbar_arrive_expect_tx(&bars.st_full[stage], rows * (L::ROW + 2u) + boxes * static_cast<uint32_t>(r4) * 2048u);
                        }
                    }
                    alive = __shfl_sync(0xffffffffu, alive, 0);
                    if (!alive) break;
                    uint8_t *st = base + stage * L::STAGE_BYTES;
                    const size_t t0 = static_cast<size_t>(gb) * n + tok0;
                    if (lane < 2) {
                        if (r4 > 0 && static_cast<uint32_t>(lane) < boxes)
                            tma_load_3d(st + L::ST_P + lane * WS_ST_PBOX, r4 == 1 ? &pmap4 : (r4 == 2 ? &pmap8 : &pmap12), &bars.st_full[stage],
                                        tok0 + 256 * lane, 0, static_cast<int>(gb));
                    } else if (lane == 30)
                        ws_bulk_load(st + WS_ST_CODES, a.cache.codes + t0 * L::ROW, rows * L::ROW, &bars.st_full[stage]);
                    else if (lane == 31)
                        ws_bulk_load(st + L::ST_NORMS, a.cache.norms + t0, rows * 2, &bars.st_full[stage]);
                }
                head = nhead;
                jb = njb;
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issue
        if (lane == 0 && it0 < it1) {
            constexpr uint32_t idesc = umma_idesc_f16(128, 16, false, false);
            uint32_t seq = 0;
            int head = it0 / a.bph, jb = it0 - head * a.bph, hidx = -1, prev_head = -1;
            bool alive = true;
            for (int item = it0, bi = 0; item < it1 && alive; ++item, ++bi) {
                if (head != prev_head) {
                    hidx += 1;
                    prev_head = head;
                    if (!mbar_wait(&bars.b1_full[hidx & 1], (hidx >> 1) & 1u, &abort_flag)) break;
                }
                const int vb = bi & 1, hb = hidx & 1;
                if (!mbar_wait(&bars.b2_full[vb], (bi >> 1) & 1u, &abort_flag)) break;
                const uint32_t b1 = smem_u32(base + L::OFF_B1 + hb * 4096), b2 = smem_u32(base + L::OFF_B2 + vb * 2048);
                uint64_t bdesc[D / 16 + 1];
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) bdesc[ks] = umma_desc_sw128(b1 + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024);
                bdesc[D / 16] = umma_desc_sw128(b2, 16, 1024);
                for (int tile = 0; tile < tiles; ++tile, ++seq) {
                    const int buf = seq & (WS_BUFS - 1);
                    const uint32_t u = (seq >> 2) & 1u;
                    // a filled buffer is also a drained one: its expanders waited for the epilogue of its last use
                    if (!mbar_wait(&bars.a_full[buf], u, &abort_flag)) {
                        alive = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t tb = tmem0 + buf * WS_BUF_COLS;
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) umma_f16_ts(tb + WS_COL_D1, tb + 8 * ks, bdesc[ks], idesc, ks ? 1u : 0u);
                    umma_f16_ts(tb + WS_COL_D2, tb + WS_COL_P, bdesc[D / 16], idesc, 0u);
                    umma_commit(&bars.d_full[buf]);   // the one commit of a tile: each costs the issuing thread well over 100 cycles
                }
                if (!alive) break;
                umma_commit(&bars.b2_empty[vb]);
                int nhead = head, njb = jb + 1;
                if (njb == a.bph) {
                    njb = 0;
                    nhead += 1;
                }
                if (nhead != head || item + 1 == it1) umma_commit(&bars.b1_empty[hb]);
                head = nhead;
                jb = njb;
            }
        }
    } else if (warp < 4) {
        // ---------------------------------------------------------------- operand builder (64 threads)
        const int bt = tid - 64;
        float *qs_all = reinterpret_cast<float *>(base + L::OFF_Q);
        // Head `hd`, the `hx`-th head of this CTA: its queries into shared memory (for the Aq products) and the
        // prepared image of W = Pi q, by one bulk copy, into the operand buffer of its parity.
        auto build_w = [&](int hd, int hx) -> bool {
            const int hb = hx & 1;
            float *qs = qs_all + hb * WS_NQ * D;
            // (a bounded wait ends per thread: its outcome is made common at the group's next barrier, so
            // that the 64 threads leave together and never one by one)
            const bool ok = mbar_wait(&bars.b1_empty[hb], ((hx >> 1) & 1u) ^ 1u, &abort_flag);
            if (bt == 0 && ok) {
                mbar_arrive_expect_tx(&bars.b1_full[hb], 4096);
                ws_bulk_load(base + L::OFF_B1 + hb * 4096, a.wimg + static_cast<size_t>(hd) * 4096, 4096, &bars.b1_full[hb]);
            }
            for (int e = bt; e < WS_NQ * D; e += 64) {
                const int g = e / D;
                qs[e] = (g < gcount) ? __half2float(a.q[(static_cast<long long>(hd) * a.G + a.g0 + g) * D + (e % D)]) : 0.0f;
            }
            return !ws_builder_any(!ok);
        };
        int head = (it0 < it1) ? it0 / a.bph : 0, jb = it0 - head * a.bph, hidx = -1, prev_head = -1;
        bool first_of_head = false;
        int rank_next = (it0 < it1) ? min(__ldg(a.cache.rank + static_cast<long long>(head) * a.head_stride + jb), WS_PMAX) : 0;
        for (int item = it0, bi = 0; item < it1; ++item, ++bi) {
            if (head != prev_head) {
                hidx += 1;
                prev_head = head;
                first_of_head = true;
                if (hidx == 0 && !build_w(head, 0)) break;   // later heads were built one head ahead (below)
            }
            const float *qs = qs_all + (hidx & 1) * WS_NQ * D;
            const int vb = bi & 1;
            const int rank = rank_next;
            {   // the next block's rank is asked for now: a load on the critical path of every block costs over 1 000 cycles
                int nh = head, nj = jb + 1;
                if (nj == a.bph) {
                    nj = 0;
                    nh += 1;
                }
                if (item + 1 < it1) rank_next = min(__ldg(a.cache.rank + static_cast<long long>(nh) * a.head_stride + nj), WS_PMAX);
            }
            const bool ok = mbar_wait(&bars.blk_full[vb], (bi >> 1) & 1u, &abort_flag) &&
                            mbar_wait(&bars.b2_empty[vb], ((bi >> 1) & 1u) ^ 1u, &abort_flag);
            const __half *vs = reinterpret_cast<const __half *>(base + L::OFF_V + vb * 4096);
            uint8_t *b2 = base + L::OFF_B2 + vb * 2048;
            // Aq[g][i] = q_g . zeta_i for g < gcount, i < rank, zero elsewhere.  Four lanes share a dot product
            // (16-byte chunks of the row dealt round-robin, rotated by the dot's number so that the lanes of a warp
            // hit different banks), sixteen dot products per round of the 64 threads.
            for (int e = bt; e < WS_NQ * RMAX; e += 64) {
                const int g = e >> 4, i = e & 15;
                if (!(i < rank && g < gcount)) ws_split_store(b2, g, i, 0.0f);
            }
            const int ndots = rank * gcount, part = bt & 3;
            for (int d0i = 0; d0i < ndots; d0i += 16) {
                const int dn = d0i + (bt >> 2);
                const bool act = dn < ndots;
                const int g = act ? dn / rank : 0, i = act ? dn - g * rank : 0;
                const uint4 *vrow = reinterpret_cast<const uint4 *>(vs + i * D);
                const float4 *qrow = reinterpret_cast<const float4 *>(qs + g * D);
                float d0 = 0.0f, d1 = 0.0f;
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int j = (4 * it + part + dn) & 15;
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
                float dot = d0 + d1;
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                if (act && part == 0) ws_split_store(b2, g, i, dot * WS_QSCALE);
            }
            fence_proxy_async_smem();
            if (ws_builder_any(!ok)) break;   // a thread whose wait gave up has built from stale vectors: nothing is handed on
            if (bt == 0) {
                mbar_arrive(&bars.b2_full[vb]);
                mbar_arrive(&bars.blk_empty[vb]);
            }
            if (first_of_head) {
                first_of_head = false;
                if ((head + 1) * a.bph < it1 && !build_w(head + 1, hidx + 1)) break;
            }
            jb += 1;
            if (jb == a.bph) {
                jb = 0;
                head += 1;
            }
        }
    }
    else if (warp < 12) {
        // ---------------------------------------------------------------- expanders (2 groups x 128 threads)
        const int grp = (warp - 4) >> 2;
        const int wt = ((warp - 4) & 3) * 32 + lane;   // token within the tile = tensor-memory lane
        const uint32_t lane_base = static_cast<uint32_t>(32 * (warp & 3)) << 16;
        uint32_t seq = 0, sbase = 0;
        const uint32_t stages_per_block = (tiles + WS_TPS - 1) / WS_TPS;
        bool alive = true;
        for (int item = it0; item < it1 && alive; ++item, sbase += stages_per_block) {
            for (int tile = 0; tile < tiles; ++tile, ++seq) {
                if (static_cast<int>(seq & 1u) != grp) continue;
                const uint32_t sseq = sbase + tile / WS_TPS;
                const int stage = sseq % L::STAGES, buf = seq & (WS_BUFS - 1);
                if (!mbar_wait(&bars.st_full[stage], (sseq / L::STAGES) & 1u, &abort_flag)) {
                    alive = false;
                    break;
                }
                const uint8_t *st = base + stage * L::STAGE_BYTES;
                const int rank = st_rank[stage];
                const bool valid = tile * 128 + wt < n;
                const int st_tok = (tile % WS_TPS) * 128 + wt;   // token within the stage
                uint32_t cw[4 * BITS];   // the token's 128 codes
#pragma unroll
                for (int w = 0; w < BITS; ++w) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(st + WS_ST_CODES + st_tok * L::ROW + 16 * w);
                    cw[4 * w] = v.x;
                    cw[4 * w + 1] = v.y;
                    cw[4 * w + 2] = v.z;
                    cw[4 * w + 3] = v.w;
                }
                unsigned short rho_raw = *reinterpret_cast<const unsigned short *>(st + L::ST_NORMS + st_tok * 2);
                const uint8_t *pcol = st + L::ST_P + (st_tok >> 8) * WS_ST_PBOX + (st_tok & 255) * 2;
                uint32_t pw[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) pw[i] = 0u;
#pragma unroll
                for (int i = 0; i < WS_PMAX; ++i) {
                    if (i < rank) {
                        const uint32_t v = *reinterpret_cast<const unsigned short *>(pcol + i * 512);
                        pw[i >> 1] |= v << (16 * (i & 1));
                    }
                }
                {   // a stage is released by 128 arrivals per tile slot; the last tile of a short stage makes up the rest
                    const int last_in_stage = min(tiles, (tile / WS_TPS + 1) * WS_TPS) - 1;
                    const int arrivals = (tile == last_in_stage) ? 1 + (WS_TPS - 1 - (tile % WS_TPS)) : 1;
                    __syncwarp();   // every lane has its copy of the stage's bytes in registers
                    if (lane == 0)
                        for (int r = 0; r < arrivals; ++r) mbar_arrive(&bars.st_empty[stage]);
                }
                if (!valid) {   // rows past the end of the block were not copied: the stage holds stale bytes there
#pragma unroll
                    for (int w = 0; w < 4 * BITS; ++w) cw[w] = 0u;
                    rho_raw = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) pw[i] = 0u;
                }
                const uint32_t u = (seq >> 2) & 1u;
                // the epilogue has read the last use of this buffer, hence its MMAs are over too
                if (!mbar_wait(&bars.d_empty[buf], u ^ 1u, &abort_flag)) {
                    alive = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t tb = tmem0 + lane_base + buf * WS_BUF_COLS;
                {
                    uint32_t av[32];
#pragma unroll
                    for (int q = 0; q < 4; ++q) expand16_codes<BITS>(cw, q, a.lo_tab, a.hi_tab, &av[8 * q]);
                    tmem_st32(tb, av);
#pragma unroll
                    for (int q = 0; q < 4; ++q) expand16_codes<BITS>(cw + 2 * BITS, q, a.lo_tab, a.hi_tab, &av[8 * q]);
                    tmem_st32(tb + 32, av);
                }
                tmem_st8(tb + WS_COL_P, pw);
                {
                    uint32_t rv[8];
                    rv[0] = __float_as_uint(__half2float(__ushort_as_half(rho_raw)));
#pragma unroll
                    for (int i = 1; i < 8; ++i) rv[i] = 0u;
                    tmem_st8(tb + WS_COL_RHO, rv);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.a_full[buf]);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (128 threads)
        const int wt = (warp & 3) * 32 + lane;
        const uint32_t lane_base = static_cast<uint32_t>(32 * (warp & 3)) << 16;
        const float f2 = a.scale * (1.0f / WS_QSCALE);
        const size_t qstride = static_cast<size_t>(a.bph) * n;
        uint32_t seq = 0;
        bool alive = true;
        int head = (it0 < it1) ? it0 / a.bph : 0, jb = it0 - head * a.bph;
        for (int item = it0; item < it1 && alive; ++item) {
            float *out_row = a.scores + (static_cast<size_t>(head) * a.G + a.g0) * qstride + static_cast<size_t>(jb) * n;
            for (int tile = 0; tile < tiles; ++tile, ++seq) {
                const int buf = seq & (WS_BUFS - 1);
                if (!mbar_wait(&bars.d_full[buf], (seq >> 2) & 1u, &abort_flag)) {
                    alive = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t tb = tmem0 + lane_base + buf * WS_BUF_COLS;
                uint32_t d1[16], d2[16], rv[8];
                tmem_ld16(tb + WS_COL_D1, d1);
                tmem_ld16(tb + WS_COL_D2, d2);
                tmem_ld8(tb + WS_COL_RHO, rv);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.d_empty[buf]);
                const int tok = tile * 128 + wt;
                if (tok < n) {
                    const float f1 = a.scale * __uint_as_float(rv[0]) * a.inv_code;
#pragma unroll
                    for (int g = 0; g < WS_NQ; ++g) {
                        if (g < gcount) {
                            const float code_part = __uint_as_float(d1[g]) + __uint_as_float(d1[WS_NQ + g]);
                            const float low_part = __uint_as_float(d2[g]) + __uint_as_float(d2[WS_NQ + g]);
                            out_row[static_cast<size_t>(g) * qstride + tok] = fmaf(f1, code_part, f2 * low_part);
                        }
                    }
                }
            }
            jb += 1;
            if (jb == a.bph) {
                jb = 0;
                head += 1;
            }
        }
    }

    __syncthreads();
    if (abort_flag && tid == 0) atomicOr(a.err, TC_ERR_SCORES_WS_TIMEOUT);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem0, WS_TMEM_COLS);
    }
}

template <int BITS>
static bool launch_scores_ws_as(WsArgs &a, int G, int grid, const CUtensorMap &m4, const CUtensorMap &m8, const CUtensorMap &m12,
                                const float *pi_t, uint8_t *wimg, int64_t *kernels, cudaStream_t s) {
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(scores_ws_kernel<BITS>), WsLayout<BITS>::SMEM_BYTES)) return false;
    for (int g0 = 0; g0 < G; g0 += WS_NQ) {
        a.g0 = g0;
        scores_w_kernel<<<a.heads, D, 0, s>>>(pi_t, a.q, G, g0, wimg);
        scores_ws_kernel<BITS><<<grid, WS_THREADS, WsLayout<BITS>::SMEM_BYTES, s>>>(a, m4, m8, m12);
        *kernels += 2;
    }
    return true;
}

bool launch_scores_ws(const eosq_cache_t &cache, int bits, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const uint16_t (&table)[16], float kappa, const __half *q, int G, float scale, float *scores, int *err,
                      int sm_count, void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s) {
    if (heads * bph > 0x7fffffff || head_stride > 0x7fffffff || bits < 1 || bits > 4) return false;
    WsArgs a;
    a.cache = cache;
    a.bph = static_cast<int>(bph);
    a.head_stride = static_cast<int>(head_stride);
    a.heads = static_cast<int>(heads);
    a.n = n;
    a.G = G;
    a.scale = scale;
    a.inv_code = 1.0f / (kappa * WS_QSCALE);
    for (int w = 0; w < 4; ++w) a.lo_tab[w] = a.hi_tab[w] = 0u;
    for (int k = 0; k < (1 << bits); ++k) {
        a.lo_tab[k >> 2] |= static_cast<uint32_t>(table[k] & 0xFFu) << (8 * (k & 3));
        a.hi_tab[k >> 2] |= static_cast<uint32_t>(table[k] >> 8) << (8 * (k & 3));
    }
    // one 4096-byte operand image per head, in a buffer the context keeps and grows (earlier work that
    // still reads the old buffer is waited for by cudaFree)
    const size_t need = static_cast<size_t>(heads) * 4096;
    if (*scratch_bytes < need) {
        cudaFree(*scratch);
        *scratch = nullptr;
        *scratch_bytes = 0;
        if (cudaMalloc(scratch, need) != cudaSuccess) return false;
        *scratch_bytes = need;
    }
    a.wimg = static_cast<const uint8_t *>(*scratch);
    a.q = q;
    a.scores = scores;
    a.err = err;
    const int grid = static_cast<int>(std::min<int64_t>(heads * bph, sm_count));
    const int64_t nb_total = (heads - 1) * head_stride + bph;
    CUtensorMap m4, m8, m12;
    if (!make_factor_tensor_map(cache.P, nb_total, n, 4, &m4) || !make_factor_tensor_map(cache.P, nb_total, n, 8, &m8) ||
        !make_factor_tensor_map(cache.P, nb_total, n, 12, &m12))
        return false;
    uint8_t *wimg = static_cast<uint8_t *>(*scratch);
    switch (bits) {
        case 1: return launch_scores_ws_as<1>(a, G, grid, m4, m8, m12, rot.pi_t, wimg, kernels, s);
        case 2: return launch_scores_ws_as<2>(a, G, grid, m4, m8, m12, rot.pi_t, wimg, kernels, s);
        case 3: return launch_scores_ws_as<3>(a, G, grid, m4, m8, m12, rot.pi_t, wimg, kernels, s);
        default: return launch_scores_ws_as<4>(a, G, grid, m4, m8, m12, rot.pi_t, wimg, kernels, s);
    }
}

}  // namespace eosq
