// Tensor-core kernels of the eosq library for fp16 blocks (sm_100a: TMA tile loads, tcgen05.mma
// with the accumulator in tensor memory).
//
//   gram_tc_kernel   G = S^T S of every block.  Products of fp16 values are exact in the fp32
//                    accumulator; only the accumulation rounds.
//   quant_tc_kernel  residual, norm, rotation, Lloyd-Max codes, bit packing and the stored left
//                    factors of every block, as one GEMM  S [M | coef V]  per 128-token tile.
#include <algorithm>
#include <cstdlib>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

// Device-side error word bits (OR-ed into the context's error word when a wait gives up).
constexpr int TC_ERR_GRAM_TIMEOUT = 1;
constexpr int TC_ERR_QUANT_TIMEOUT = 2;

// ------------------------------------------------------------------------------------------
// Tensor map over the blocks: [B][n][128] fp16, boxes of 128 tokens x 64 channels (128 bytes per
// row, 128-byte swizzle).  Tokens past n inside a box are filled with zeros by the hardware.
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

bool make_block_tensor_map(const void *blocks, int64_t nb, int n, CUtensorMap *out) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(n), static_cast<cuuint64_t>(nb)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2, static_cast<cuuint64_t>(n) * D * 2};
    const cuuint32_t box[3] = {64, 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(blocks), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Unswizzled tensor map over the stored left factors P [B][RMAX][n] fp16 with boxes of `rows`
// factor rows x 256 tokens (a box lands in shared memory as `rows` lines of 512 bytes).
bool make_factor_tensor_map(const void *P, int64_t nb, int n, int rows, CUtensorMap *out) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(n), static_cast<cuuint64_t>(RMAX), static_cast<cuuint64_t>(nb)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(n) * 2, static_cast<cuuint64_t>(n) * RMAX * 2};
    const cuuint32_t box[3] = {256, static_cast<cuuint32_t>(rows), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(P), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ------------------------------------------------------------------------------------------
// Gram matrix.  Persistent CTAs, 320 threads: warp 0 loads token tiles by TMA into a ring of
// stages, warp 1 issues the MMAs, warps 2-9 add finished partial sums into fp64 registers.
//
// A stage holds 128 tokens: channels 0-63 in its first 16 KB, channels 64-127 in the second,
// each as 128 rows (tokens) of 128 bytes.  That is the MN-major operand layout: the contraction
// index (token) runs across rows.  Both operands of  G[i][j] = sum_t S[t][i] S[t][j]  are the
// same bytes, so one descriptor serves as A and as B.
//
// The tensor core truncates when it adds into its fp32 accumulator, so the error of a sum grows
// with the number of MMAs chained into one accumulator (measured: 64 chained MMAs move the
// smallest singular values of a block by 2e-4 relative, 8 by 2e-5).  Every 128-token tile
// therefore gets a fresh accumulator (8 chained MMAs) out of a ring of four in tensor memory,
// and the tiles are summed in double precision by the CUDA cores.
// ------------------------------------------------------------------------------------------
constexpr int GRAM_STAGES = 6;
constexpr int GRAM_ACCS = 4;
constexpr int GRAM_THREADS = 320;
constexpr int TILE_T = 128;
constexpr uint32_t HALF_BYTES = TILE_T * 128;       // one 64-channel half of a stage
constexpr uint32_t STAGE_BYTES = 2 * HALF_BYTES;    // 32 KB
constexpr size_t GRAM_SMEM = GRAM_STAGES * STAGE_BYTES + 1024;
constexpr uint32_t GRAM_TMEM_COLS = 128 * GRAM_ACCS;

__global__ void __launch_bounds__(GRAM_THREADS, 1) gram_tc_kernel(const __grid_constant__ CUtensorMap tmap, int nb, int n,
                                                                  double *__restrict__ gram, int *__restrict__ err) {
    extern __shared__ uint8_t gram_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[GRAM_STAGES], empty_bar[GRAM_STAGES], acc_full[GRAM_ACCS], acc_empty[GRAM_ACCS], drain_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t fills[GRAM_STAGES], drains[GRAM_STAGES];
    __shared__ volatile int abort_flag;

    uint8_t *stages = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(gram_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles = (n + TILE_T - 1) / TILE_T;

    if (tid == 0) {
        for (int s = 0; s < GRAM_STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
            fills[s] = 0;
            drains[s] = 0;
        }
        for (int a = 0; a < GRAM_ACCS; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 8);
        }
        mbar_init(&drain_bar, 1);
        abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_s, GRAM_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_acc = tmem_base_s;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            for (int b = blockIdx.x; b < nb && !abort_flag; b += gridDim.x) {
                for (int t = 0; t < tiles; ++t, ++it) {
                    const int s = it % GRAM_STAGES;
                    const uint32_t ph = (it / GRAM_STAGES) & 1u;
                    if (!mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag)) break;
                    mbar_arrive_expect_tx(&full_bar[s], STAGE_BYTES);
                    uint8_t *dst = stages + s * STAGE_BYTES;
                    tma_load_3d(dst, &tmap, &full_bar[s], 0, t * TILE_T, b);
                    tma_load_3d(dst + HALF_BYTES, &tmap, &full_bar[s], 64, t * TILE_T, b);
                    fills[s] += 1;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_f16(128, 128, true, true);
            uint32_t it = 0;
            for (int b = blockIdx.x; b < nb && !abort_flag; b += gridDim.x) {
                bool ok = true;
                for (int t = 0; t < tiles; ++t, ++it) {
                    const int s = it % GRAM_STAGES;
                    const int a = it % GRAM_ACCS;
                    if (!mbar_wait(&acc_empty[a], ((it / GRAM_ACCS) & 1u) ^ 1u, &abort_flag) ||
                        !mbar_wait(&full_bar[s], (it / GRAM_STAGES) & 1u, &abort_flag)) {
                        ok = false;
                        break;
                    }
                    drains[s] += 1;
                    tc_fence_after_sync();
                    const uint32_t base = smem_u32(stages + s * STAGE_BYTES);
#pragma unroll
                    for (int ks = 0; ks < TILE_T / 16; ++ks) {
                        const uint64_t desc = umma_desc_sw128(base + ks * 2048, HALF_BYTES, 1024);
                        umma_f16(tmem_acc + 128u * a, desc, desc, idesc, ks ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[s]);
                    umma_commit(&acc_full[a]);
                }
                if (!ok) break;
            }
        }
    } else {
        const int q = warp & 3;                 // tensor-memory lanes [32q, 32q+32) belong to this warp
        const int half = (warp - 2) >> 2;       // columns [64 half, 64 half + 64)
        const int row = 32 * q + lane;          // G row held by this thread
        uint32_t it = 0;
        for (int b = blockIdx.x; b < nb; b += gridDim.x) {
            double sum[64];
#pragma unroll
            for (int c = 0; c < 64; ++c) sum[c] = 0.0;
            bool ok = true;
            for (int t = 0; t < tiles; ++t, ++it) {
                const int a = it % GRAM_ACCS;
                if (!mbar_wait(&acc_full[a], (it / GRAM_ACCS) & 1u, &abort_flag)) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(32 * q) << 16) + 128u * a + 64u * half;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[32];
                    tmem_ld32(taddr + 32u * h, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 32; ++c) sum[32 * h + c] += static_cast<double>(__uint_as_float(v[c]));
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[a]);
            }
            if (!ok) break;
            // G is symmetric: element (row, c) is stored at [c][row], so a warp writes 256
            // contiguous bytes per column.
            double *G = gram + static_cast<size_t>(b) * D * D;
#pragma unroll
            for (int c = 0; c < 64; ++c) G[(64 * half + c) * D + row] = sum[c];
        }
    }

    __syncthreads();
    if (abort_flag) {
        if (tid == 0) {
            atomicOr(err, TC_ERR_GRAM_TIMEOUT);
            // let loads that are still in flight land before the shared memory is given back
            volatile int scratch = 0;
            for (int s = 0; s < GRAM_STAGES; ++s)
                if (fills[s] != drains[s]) mbar_wait(&full_bar[s], (fills[s] - 1u) & 1u, &scratch);
        }
        if (tid == 32) {
            volatile int scratch = 0;
            umma_commit(&drain_bar);
            mbar_wait(&drain_bar, 0, &scratch);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_acc, GRAM_TMEM_COLS);
    }
}

bool launch_gram_tc(const void *blocks_all, int64_t nb_all, int64_t block0, int64_t nb, int n, double *gram, int *err,
                    int sm_count, cudaStream_t s) {
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(gram_tc_kernel), GRAM_SMEM)) return false;
    (void)nb_all;
    CUtensorMap tmap;
    const char *base = static_cast<const char *>(blocks_all) + static_cast<size_t>(block0) * n * D * 2;
    if (!make_block_tensor_map(base, nb, n, &tmap)) return false;
    const int grid = static_cast<int>(std::min<int64_t>(nb, static_cast<int64_t>(sm_count)));
    gram_tc_kernel<<<grid, GRAM_THREADS, GRAM_SMEM, s>>>(tmap, static_cast<int>(nb), n, gram, err);
    return true;
}

// ------------------------------------------------------------------------------------------
// Residual, norm, rotation, codes, packing and left factors (Algorithm 3; Algorithm 1).
//
// Rows of  Y = R Pi^T  are  S M  with  M = (I - sum_i coef_i zeta_i zeta_i^T) Pi^T  (d x d, built
// per block), and the stored left factors are  S [coef_i zeta_i].  Both come out of one GEMM per
// 128-token tile:  [Y | P] = S [M | coef V]  (N = 128 + 16).  S is fp16, hence exact as the A
// operand.  The B operand is kept to about 2^-22 by splitting it, after a scaling by 2^12 that
// keeps the low part in fp16's normal range, into a high and a low fp16 plane that accumulate
// into the same fp32 tile.
//
// A CTA works through its blocks one at a time: all 256 threads build B in shared memory, then for
// every tile one thread issues the TMA load and the 32 MMAs and all eight warps turn the
// accumulator into norms, codes and factor rows (warp w: tensor-memory lanes 32 (w % 4).., columns
// 64 (w / 4)..).  Two CTAs share an SM so that one's MMAs overlap the other's CUDA-core phases.
// ------------------------------------------------------------------------------------------
constexpr int QT_THREADS = 256;
constexpr int QT_N = D + RMAX;                   // 144 accumulator columns
constexpr uint32_t QT_BBOX = QT_N * 128;         // one 64-wide K half of one plane of B: 144 rows of 128 bytes
constexpr uint32_t QT_BPLANE = 2 * QT_BBOX;
constexpr uint32_t QT_ABOX = 128 * 128;          // 128 tokens x 64 channels
constexpr uint32_t QT_ABYTES = 2 * QT_ABOX;
constexpr size_t QT_SMEM = 2 * QT_BPLANE + QT_ABYTES + 1024;
constexpr uint32_t QT_TMEM_COLS = 256;
constexpr float QT_SCALE = 4096.0f;

// Byte offset of the 16-byte chunk `jc` (8 fp16 along K) of row `row` inside one plane of B.
__device__ __forceinline__ uint32_t qt_b_offset(int row, int jc) {
    return (jc >> 3) * QT_BBOX + (row >> 3) * 1024 + (row & 7) * 128 + (((jc & 7) ^ (row & 7)) << 4);
}

// Splits eight scaled fp32 values into their fp16 high and low parts.
__device__ __forceinline__ void qt_split8(const float (&m)[8], uint4 &hi, uint4 &lo) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float a = m[2 * e] * QT_SCALE, b = m[2 * e + 1] * QT_SCALE;
        const __half ah = __float2half_rn(a), bh = __float2half_rn(b);
        const __half al = __float2half_rn(a - __half2float(ah)), bl = __float2half_rn(b - __half2float(bh));
        h[e] = static_cast<uint32_t>(__half_as_ushort(ah)) | (static_cast<uint32_t>(__half_as_ushort(bh)) << 16);
        l[e] = static_cast<uint32_t>(__half_as_ushort(al)) | (static_cast<uint32_t>(__half_as_ushort(bl)) << 16);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <int BITS>
__global__ void __launch_bounds__(QT_THREADS, 2) quant_tc_kernel(const __grid_constant__ CUtensorMap tmap, int nb, int n, Workspace ws,
                                                                 const float *__restrict__ pi, const float *__restrict__ pi_t,
                                                                 Codebook cb, eosq_cache_t out, int *__restrict__ err) {
    extern __shared__ uint8_t qt_smem_raw[];
    __shared__ __align__(8) uint64_t a_full, mma_done;
    __shared__ uint32_t tmem_base_s;
    __shared__ float ss_part[2][128];
    __shared__ volatile int abort_flag;
    __shared__ int load_pending;

    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(qt_smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t *b_hi = base, *b_lo = base + QT_BPLANE, *a_tile = base + 2 * QT_BPLANE;
    float *Vc = reinterpret_cast<float *>(a_tile);   // the A buffer doubles as scratch while B is built
    float *W = Vc + RMAX * D;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles = (n + 127) / 128;
    constexpr int NTHR = (1 << BITS) - 1;
    constexpr int ROW_BYTES = D * BITS / 8;

    if (tid == 0) {
        mbar_init(&a_full, 1);
        mbar_init(&mma_done, 1);
        abort_flag = 0;
        load_pending = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap);
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, QT_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_acc = tmem_base_s;
    float thr[NTHR];
#pragma unroll
    for (int t = 0; t < NTHR; ++t) thr[t] = cb.threshold[t];

    uint32_t a_cnt = 0, m_cnt = 0;
    for (int b = blockIdx.x; b < nb && !abort_flag; b += gridDim.x) {
        const int rank = ws.rank[b];
        // ---- B = [M | coef V], split and swizzled ---------------------------------------------
        {   // W[i][c] = sum_j Pi[c][j] zeta_i[j]; the rotation comes from L2, a batch of 32 rows ahead of its use
            const int c = tid & (D - 1), half = tid >> 7;
            float pn[32];
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) pn[jj] = __ldg(pi_t + jj * D + c);
            for (int e = tid; e < RMAX * D; e += QT_THREADS) Vc[e] = ws.vr[static_cast<size_t>(b) * RMAX * D + e];
            __syncthreads();
            float w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = 0.0f;
            if (8 * half < rank) {
#pragma unroll 1
                for (int j0 = 0; j0 < D; j0 += 32) {
                    float pv[32];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) pv[jj] = pn[jj];
                    if (j0 + 32 < D) {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) pn[jj] = __ldg(pi_t + (j0 + 32 + jj) * D + c);
                    }
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 4) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {   // one 16-byte broadcast load feeds four multiply-adds
                            const float4 vv = *reinterpret_cast<const float4 *>(Vc + (8 * half + i) * D + j0 + jj);
                            w[i] = fmaf(pv[jj], vv.x, w[i]);
                            w[i] = fmaf(pv[jj + 1], vv.y, w[i]);
                            w[i] = fmaf(pv[jj + 2], vv.z, w[i]);
                            w[i] = fmaf(pv[jj + 3], vv.w, w[i]);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) W[(8 * half + i) * D + c] = w[i];
        }
        __syncthreads();
        for (int e = tid; e < RMAX * D; e += QT_THREADS) Vc[e] *= ws.coef[static_cast<size_t>(b) * RMAX + e / D];
        __syncthreads();
        // chunk = 8 consecutive entries of a row of M; a thread's chunks are QT_THREADS apart, i.e. 16 rows,
        // and the rotation entries of the next chunk are fetched while the current one is worked on
        float4 n0 = __ldg(reinterpret_cast<const float4 *>(pi + tid * 8)), n1 = __ldg(reinterpret_cast<const float4 *>(pi + tid * 8 + 4));
#pragma unroll 1
        for (int it = 0; it < (D * D / 8) / QT_THREADS; ++it) {
            const int chunk = tid + QT_THREADS * it, c = chunk >> 4, jc = chunk & 15;
            const float4 p0 = n0, p1 = n1;
            if (it + 1 < (D * D / 8) / QT_THREADS) {
                n0 = __ldg(reinterpret_cast<const float4 *>(pi + (chunk + QT_THREADS) * 8));
                n1 = __ldg(reinterpret_cast<const float4 *>(pi + (chunk + QT_THREADS) * 8 + 4));
            }
            float m[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
            for (int i = 0; i < rank; ++i) {
                const float w = W[i * D + c];
                const float4 v0 = *reinterpret_cast<const float4 *>(Vc + i * D + 8 * jc);
                const float4 v1 = *reinterpret_cast<const float4 *>(Vc + i * D + 8 * jc + 4);
                m[0] = fmaf(-v0.x, w, m[0]);
                m[1] = fmaf(-v0.y, w, m[1]);
                m[2] = fmaf(-v0.z, w, m[2]);
                m[3] = fmaf(-v0.w, w, m[3]);
                m[4] = fmaf(-v1.x, w, m[4]);
                m[5] = fmaf(-v1.y, w, m[5]);
                m[6] = fmaf(-v1.z, w, m[6]);
                m[7] = fmaf(-v1.w, w, m[7]);
            }
            uint4 hi, lo;
            qt_split8(m, hi, lo);
            const uint32_t off = qt_b_offset(c, jc);
            *reinterpret_cast<uint4 *>(b_hi + off) = hi;
            *reinterpret_cast<uint4 *>(b_lo + off) = lo;
        }
        {   // rows 128..143: coef_i zeta_i (zero beyond the rank)
            const int i = tid >> 4, jc = tid & 15;
            float m[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) m[e] = (i < rank) ? Vc[i * D + 8 * jc + e] : 0.0f;
            uint4 hi, lo;
            qt_split8(m, hi, lo);
            const uint32_t off = qt_b_offset(D + i, jc);
            *reinterpret_cast<uint4 *>(b_hi + off) = hi;
            *reinterpret_cast<uint4 *>(b_lo + off) = lo;
        }
        fence_proxy_async_smem();   // B was written by ordinary stores and is read by the tensor core
        __syncthreads();

        // ---- tiles --------------------------------------------------------------------------
        const long long gb = b;
        bool ok = true;
        for (int t = 0; t < tiles; ++t) {
            if (tid == 0) {
                if (t == 0) {
                    mbar_arrive_expect_tx(&a_full, QT_ABYTES);
                    tma_load_3d(a_tile, &tmap, &a_full, 0, 0, b);
                    tma_load_3d(a_tile + QT_ABOX, &tmap, &a_full, 64, 0, b);
                    load_pending = 1;
                }
                if (mbar_wait(&a_full, a_cnt & 1u, &abort_flag)) {
                    load_pending = 0;
                    tc_fence_after_sync();
                    constexpr uint32_t idesc = umma_idesc_f16(128, QT_N, false, false);
                    const uint32_t a0 = smem_u32(a_tile), h0 = smem_u32(b_hi), l0 = smem_u32(b_lo);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t ka = (ks >> 2) * QT_ABOX + (ks & 3) * 32, kb = (ks >> 2) * QT_BBOX + (ks & 3) * 32;
                        const uint64_t da = umma_desc_sw128(a0 + ka, 16, 1024);
                        umma_f16(tmem_acc, da, umma_desc_sw128(h0 + kb, 16, 1024), idesc, ks ? 1u : 0u);
                        umma_f16(tmem_acc, da, umma_desc_sw128(l0 + kb, 16, 1024), idesc, 1u);
                    }
                    umma_commit(&mma_done);
                }
            }
            a_cnt += 1;
            if (!mbar_wait(&mma_done, m_cnt & 1u, &abort_flag)) {
                ok = false;
                break;
            }
            m_cnt += 1;
            tc_fence_after_sync();
            if (tid == 0 && t + 1 < tiles) {   // the A buffer is free again: fetch the next tile behind the epilogue
                mbar_arrive_expect_tx(&a_full, QT_ABYTES);
                tma_load_3d(a_tile, &tmap, &a_full, 0, (t + 1) * 128, b);
                tma_load_3d(a_tile + QT_ABOX, &tmap, &a_full, 64, (t + 1) * 128, b);
                load_pending = 1;
            }
            // ---- epilogue: this thread owns token `row`, columns [64 h, 64 h + 64) ------------
            const int q = warp & 3, h = warp >> 2;
            const int row = 32 * q + lane;
            const int tok = t * 128 + row;
            const uint32_t lane_addr = tmem_acc + (static_cast<uint32_t>(32 * q) << 16);
            float y[64];
            {
                uint32_t v0[32], v1[32];
                tmem_ld32(lane_addr + 64u * h, v0);
                tmem_ld32(lane_addr + 64u * h + 32u, v1);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    y[c] = __uint_as_float(v0[c]);
                    y[32 + c] = __uint_as_float(v1[c]);
                }
            }
            uint32_t pv[8];
            tmem_ld8(lane_addr + D + 8u * h, pv);
            tmem_ld_wait();
            float ss = 0.0f;
#pragma unroll
            for (int c = 0; c < 64; ++c) ss = fmaf(y[c], y[c], ss);
            ss_part[h][row] = ss;
            tc_fence_before_sync();
            __syncthreads();   // both halves of every row are summed; every warp has read its accumulator part
            const float tot = ss_part[0][row] + ss_part[1][row];
            const float rho = sqrtf(tot);
            // thresholds scaled by the norm: y > thr rho decides as y / rho > thr does (a zero row keeps
            // the plain thresholds, so that it gets the code of z = 0)
            float ts[NTHR];
#pragma unroll
            for (int k = 0; k < NTHR; ++k) ts[k] = (rho > 0.0f) ? thr[k] * rho : thr[k];
            unsigned long long wv[BITS];
            if (BITS == 3) {
#pragma unroll
                for (int k = 0; k < BITS; ++k) wv[k] = 0ull;
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    unsigned code = 0u;
#pragma unroll
                    for (int k = 0; k < NTHR; ++k) code += (ts[k] < y[c]) ? 1u : 0u;
                    const int pos = c * BITS;
                    wv[pos >> 6] |= static_cast<unsigned long long>(code) << (pos & 63);
                    if ((pos & 63) + BITS > 64) wv[(pos >> 6) + 1] |= static_cast<unsigned long long>(code) >> (64 - (pos & 63));
                }
            } else {
                constexpr int CPW = 32 / BITS;   // codes per 32-bit word, filled from the top code down
#pragma unroll
                for (int k = 0; k < BITS; ++k) {
                    uint32_t w2[2];
#pragma unroll
                    for (int hw = 0; hw < 2; ++hw) {
                        uint32_t w = 0u;
#pragma unroll
                        for (int e = CPW - 1; e >= 0; --e) {
                            const float v = y[(2 * k + hw) * CPW + e];
                            uint32_t code = 0u;
#pragma unroll
                            for (int t = 0; t < NTHR; ++t) code += (ts[t] < v) ? 1u : 0u;
                            w = w * (1u << BITS) + code;
                        }
                        w2[hw] = w;
                    }
                    wv[k] = static_cast<unsigned long long>(w2[0]) | (static_cast<unsigned long long>(w2[1]) << 32);
                }
            }
            if (tok < n) {
                unsigned long long *dst = reinterpret_cast<unsigned long long *>(
                    out.codes + (static_cast<size_t>(gb) * n + tok) * ROW_BYTES + h * 8 * BITS);
#pragma unroll
                for (int k = 0; k < BITS; ++k) dst[k] = wv[k];
                if (h == 0) out.norms[static_cast<size_t>(gb) * n + tok] = __half_as_ushort(__float2half_rn(rho * (1.0f / QT_SCALE)));
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int i = 8 * h + e;
                    if (i < rank)
                        out.P[(static_cast<size_t>(gb) * RMAX + i) * n + tok] =
                            __half_as_ushort(__float2half_rn(__uint_as_float(pv[e]) * (1.0f / QT_SCALE)));
                }
            }
            __syncthreads();   // ss_part is reused by the next tile
        }
        if (!ok) break;
    }

    __syncthreads();
    if (abort_flag) {
        if (tid == 0) {
            atomicOr(err, TC_ERR_QUANT_TIMEOUT);
            volatile int scratch = 0;
            if (load_pending) mbar_wait(&a_full, a_cnt & 1u, &scratch);
        }
        __syncthreads();
    }
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_acc, QT_TMEM_COLS);
    }
}

template <int BITS>
static bool launch_quant_tc_bits(const CUtensorMap &tmap, int nb, int n, const Workspace &ws, const Rotation &rot,
                                 const Codebook &cb, const eosq_cache_t &out, int *err, int grid, cudaStream_t s) {
    if (!ensure_dynamic_smem(reinterpret_cast<const void *>(quant_tc_kernel<BITS>), QT_SMEM)) return false;
    quant_tc_kernel<BITS><<<grid, QT_THREADS, QT_SMEM, s>>>(tmap, nb, n, ws, rot.pi, rot.pi_t, cb, out, err);
    return true;
}

bool launch_quant_tc(const void *blocks_all, int64_t block0, int64_t nb, int n, const Workspace &ws, const Rotation &rot,
                     const Codebook &cb, const eosq_cache_t &out, int *err, int sm_count, cudaStream_t s) {
    CUtensorMap tmap;
    const char *base = static_cast<const char *>(blocks_all) + static_cast<size_t>(block0) * n * D * 2;
    if (!make_block_tensor_map(base, nb, n, &tmap)) return false;
    const int grid = static_cast<int>(std::min<int64_t>(nb, 2 * static_cast<int64_t>(sm_count)));
    switch (cb.bits) {
        case 1: return launch_quant_tc_bits<1>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 2: return launch_quant_tc_bits<2>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 3: return launch_quant_tc_bits<3>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
        case 4: return launch_quant_tc_bits<4>(tmap, static_cast<int>(nb), n, ws, rot, cb, out, err, grid, s);
    }
    return false;
}

}  // namespace eosq
