// CUDA-core kernels of the eosq library: Gram matrix and residual + rotation + quantisation +
// packing, as tiled FMA loops in shared memory.  These run for fp32 input blocks and serve as the
// exact-arithmetic path (the Gram matrix also for the second pass over fp16 blocks whose spectrum
// the tensor-core Gram matrix cannot resolve); fp16 blocks take the tensor-core kernels.
#include "eosq_common.cuh"

namespace eosq {

// ------------------------------------------------------------------------------------------
// G = S^T S, one CTA per block.  Products of fp16 or fp32 inputs are exact in double, so the
// only rounding is the double accumulation.  Thread (ty, tx) of a 16 x 16 grid owns rows
// {4ty..4ty+3, 64+4ty..} x columns {4tx..4tx+3, 64+4tx..}.
// ------------------------------------------------------------------------------------------
constexpr int GRAM_ROWS = 32;

template <typename Tin>
__global__ void __launch_bounds__(256) gram_plain_kernel(const Tin *__restrict__ blocks, int n,
                                                         double *__restrict__ gram, const int *__restrict__ list,
                                                         const int *__restrict__ count) {
    __shared__ __align__(16) float tile[GRAM_ROWS][D];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    // without a list: block blockIdx.x; with one: the listed blocks, shared out over the grid
    for (int li = blockIdx.x; !list || li < *count; li += gridDim.x) {
    const int blk = list ? list[li] : li;
    const Tin *S = blocks + static_cast<size_t>(blk) * n * D;
    double acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0;
    for (int r0 = 0; r0 < n; r0 += GRAM_ROWS) {
        __syncthreads();
        for (int e = tid; e < GRAM_ROWS * D; e += 256) {
            const int r = r0 + e / D;
            tile[e / D][e % D] = (r < n) ? load_as_float(S + static_cast<size_t>(r) * D + (e % D)) : 0.0f;
        }
        __syncthreads();
        for (int r = 0; r < GRAM_ROWS; ++r) {
            const float4 a0 = *reinterpret_cast<const float4 *>(&tile[r][4 * ty]);
            const float4 a1 = *reinterpret_cast<const float4 *>(&tile[r][64 + 4 * ty]);
            const float4 b0 = *reinterpret_cast<const float4 *>(&tile[r][4 * tx]);
            const float4 b1 = *reinterpret_cast<const float4 *>(&tile[r][64 + 4 * tx]);
            const double a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const double bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] += a[i] * bb[j];
        }
    }
    double *G = gram + static_cast<size_t>(blk) * D * D;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int row = (i < 4) ? 4 * ty + i : 64 + 4 * ty + (i - 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int col = (j < 4) ? 4 * tx + j : 64 + 4 * tx + (j - 4);
            G[row * D + col] = acc[i][j];
        }
    }
    if (!list) break;
    }
}

void launch_gram_plain(const void *blocks, int in_dtype, int64_t nb, int n, double *gram, const int *list,
                       const int *count, cudaStream_t s) {
    if (in_dtype == EOSQ_F32)
        gram_plain_kernel<float><<<list_grid(nb, list), 256, 0, s>>>(static_cast<const float *>(blocks), n, gram, list, count);
    else
        gram_plain_kernel<__half><<<list_grid(nb, list), 256, 0, s>>>(static_cast<const __half *>(blocks), n, gram, list, count);
}

// ------------------------------------------------------------------------------------------
// Shared 32 x 128 by 128 x 128 tile product used by the quantiser and the decoder:
// warp w owns rows 4w..4w+3 of the tile, lane l owns columns 4l..4l+3.
// ------------------------------------------------------------------------------------------
constexpr int TILE_ROWS = 32;

__device__ __forceinline__ void tile_gemm(const float (*tile)[D], const float *Bm, int warp, int lane,
                                          float acc[4][4]) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0.0f;
#pragma unroll 4
    for (int j = 0; j < D; ++j) {
        const float4 bv = *reinterpret_cast<const float4 *>(Bm + j * D + 4 * lane);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const float a = tile[4 * warp + r][j];
            acc[r][0] = fmaf(a, bv.x, acc[r][0]);
            acc[r][1] = fmaf(a, bv.y, acc[r][1]);
            acc[r][2] = fmaf(a, bv.z, acc[r][2]);
            acc[r][3] = fmaf(a, bv.w, acc[r][3]);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Residual, norm, rotation, code, pack (Algorithm 3 lines 4-9; Algorithm 1).
// The residual is never formed: rows of Y = R Pi^T are computed as S M with
//   M[j][c] = Pi[c][j] - sum_i coef_i zeta_i[j] (Pi zeta_i)[c],
// rho_t = ||y_t|| (Pi is orthogonal), z = y / rho, code = #thresholds below z.
// ------------------------------------------------------------------------------------------
constexpr size_t QUANT_DYN_SMEM = sizeof(float) * (D * D + TILE_ROWS * D + 2 * RMAX * D);

template <typename Tin>
__global__ void __launch_bounds__(256) quant_plain_kernel(const Tin *__restrict__ blocks, int n, Workspace ws,
                                                          const float *__restrict__ pi_t, Codebook cb,
                                                          eosq_cache_t out, long long block0) {
    extern __shared__ __align__(16) float qs[];
    float *M = qs;                                                         // [D][D]   M[j][c]
    float(*tile)[D] = reinterpret_cast<float(*)[D]>(qs + D * D);           // [32][D]
    float *Vc = qs + D * D + TILE_ROWS * D;                                // [RMAX][D] coef_i zeta_i[j]
    float *W = Vc + RMAX * D;                                              // [RMAX][D] (Pi zeta_i)[c]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const long long gb = block0 + b;
    const int rank = ws.rank[b];
    const Tin *S = blocks + static_cast<size_t>(gb) * n * D;

    for (int e = tid; e < RMAX * D; e += 256) Vc[e] = ws.vr[static_cast<size_t>(b) * RMAX * D + e];
    __syncthreads();
    {   // W[i][c] = sum_j Pi[c][j] zeta_i[j]
        const int c = tid & (D - 1), half = tid >> 7;
        float w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = 0.0f;
        if (8 * half < rank) {
            for (int j = 0; j < D; ++j) {
                const float pv = pi_t[j * D + c];
#pragma unroll
                for (int i = 0; i < 8; ++i) w[i] = fmaf(pv, Vc[(8 * half + i) * D + j], w[i]);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) W[(8 * half + i) * D + c] = w[i];
    }
    __syncthreads();
    for (int e = tid; e < RMAX * D; e += 256) Vc[e] *= ws.coef[static_cast<size_t>(b) * RMAX + e / D];
    __syncthreads();
    for (int e = tid; e < D * D; e += 256) {
        const int j = e / D, c = e % D;
        float m = pi_t[e];
        for (int i = 0; i < rank; ++i) m = fmaf(-Vc[i * D + j], W[i * D + c], m);
        M[e] = m;
    }

    const int nthr = (1 << cb.bits) - 1;
    const int chunk_bits = 4 * cb.bits;       // bits contributed by one lane (4 coordinates)
    const int row_words = 4 * cb.bits;        // 128 * bits / 32
    for (int r0 = 0; r0 < n; r0 += TILE_ROWS) {
        __syncthreads();
        for (int e = tid; e < TILE_ROWS * D; e += 256) {
            const int r = r0 + e / D;
            tile[e / D][e % D] = (r < n) ? load_as_float(S + static_cast<size_t>(r) * D + (e % D)) : 0.0f;
        }
        __syncthreads();
        float acc[4][4];
        tile_gemm(tile, M, warp, lane, acc);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = r0 + 4 * warp + r;
            float ss = acc[r][0] * acc[r][0] + acc[r][1] * acc[r][1] + acc[r][2] * acc[r][2] + acc[r][3] * acc[r][3];
            ss = warp_sum(ss);
            const float rho = sqrtf(ss);
            unsigned chunk = 0u;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float z = (rho > 0.0f) ? acc[r][c] / rho : 0.0f;
                unsigned code = 0u;
                for (int t = 0; t < nthr; ++t) code += (cb.threshold[t] < z) ? 1u : 0u;
                chunk |= code << (c * cb.bits);
            }
            // lane l holds bits [l*chunk_bits, (l+1)*chunk_bits) of the row; lane w assembles word w
            unsigned word = 0u;
            const int first = (32 * lane) / chunk_bits;
#pragma unroll
            for (int s = 0; s < 9; ++s) {
                const int src = first + s;
                const unsigned other = __shfl_sync(0xffffffffu, chunk, src & 31);
                const int pos = src * chunk_bits - 32 * lane;
                if (src < 32 && pos < 32) word |= (pos >= 0) ? (other << pos) : (other >> (-pos));
            }
            if (row < n) {
                if (lane < row_words)
                    reinterpret_cast<unsigned *>(out.codes)[(static_cast<size_t>(gb) * n + row) * row_words + lane] = word;
                if (lane == 0) out.norms[static_cast<size_t>(gb) * n + row] = __half_as_ushort(__float2half_rn(rho));
            }
        }
        // left factors P[i][t] = coef_i <s_t, zeta_i>
        for (int e = tid; e < TILE_ROWS * RMAX; e += 256) {
            const int i = e / TILE_ROWS, r = e % TILE_ROWS;
            if (i < rank && r0 + r < n) {
                float p = 0.0f;
                for (int j = 0; j < D; ++j) p = fmaf(tile[r][j], Vc[i * D + j], p);
                out.P[(static_cast<size_t>(gb) * RMAX + i) * n + r0 + r] = __half_as_ushort(__float2half_rn(p));
            }
        }
    }
}

void launch_quant_plain(const void *blocks, int in_dtype, int64_t nb, int n, const Workspace &ws,
                        const Rotation &rot, const Codebook &cb, const eosq_cache_t &out, int64_t block0,
                        cudaStream_t s) {
    ensure_dynamic_smem(reinterpret_cast<const void *>(quant_plain_kernel<float>), QUANT_DYN_SMEM);
    ensure_dynamic_smem(reinterpret_cast<const void *>(quant_plain_kernel<__half>), QUANT_DYN_SMEM);
    if (in_dtype == EOSQ_F32)
        quant_plain_kernel<float><<<static_cast<unsigned>(nb), 256, QUANT_DYN_SMEM, s>>>(
            static_cast<const float *>(blocks), n, ws, rot.pi_t, cb, out, static_cast<long long>(block0));
    else
        quant_plain_kernel<__half><<<static_cast<unsigned>(nb), 256, QUANT_DYN_SMEM, s>>>(
            static_cast<const __half *>(blocks), n, ws, rot.pi_t, cb, out, static_cast<long long>(block0));
}

}  // namespace eosq
