// Tensor-core Gram kernel of the eosq library for fp16 blocks (sm_100a: TMA tile loads, tcgen05.mma
// with the accumulator in tensor memory), and the tensor maps the other kernels share.
//
//   gram_tc_kernel   G = S^T S of every block.  Products of fp16 values are exact in the fp32
//                    accumulator; only the accumulation rounds.
#include <algorithm>
#include <cstdlib>

#include "eosq_common.cuh"
#include "eosq_sm100.cuh"

namespace eosq {

using namespace sm100;

// Device-side error word bits (OR-ed into the context's error word when a wait gives up).
constexpr int TC_ERR_GRAM_TIMEOUT = 1;

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

}  // namespace eosq
