// CUDA-core kernels of the eosq library: Gram matrix, residual + rotation + quantisation +
// packing, reconstruction and attention logits, all as tiled FMA loops in shared memory.
// These run for fp32 input blocks and serve as the exact-arithmetic path; fp16 blocks take the
// tensor-core kernels where those are available.
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
    static bool configured = false;
    if (!configured) {
        cudaFuncSetAttribute(quant_plain_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(QUANT_DYN_SMEM));
        cudaFuncSetAttribute(quant_plain_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(QUANT_DYN_SMEM));
        configured = true;
    }
    if (in_dtype == EOSQ_F32)
        quant_plain_kernel<float><<<static_cast<unsigned>(nb), 256, QUANT_DYN_SMEM, s>>>(
            static_cast<const float *>(blocks), n, ws, rot.pi_t, cb, out, static_cast<long long>(block0));
    else
        quant_plain_kernel<__half><<<static_cast<unsigned>(nb), 256, QUANT_DYN_SMEM, s>>>(
            static_cast<const __half *>(blocks), n, ws, rot.pi_t, cb, out, static_cast<long long>(block0));
}

// ------------------------------------------------------------------------------------------
// Reconstruction x_hat[t] = sum_i P[i][t] V[i][:] + norms[t] * (centroids[codes[t]] Pi).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned extract_code(const uint8_t *row_bytes, int j, int bits) {
    const int pos = j * bits;
    const unsigned lo = row_bytes[pos >> 3];
    const unsigned hi = row_bytes[(pos >> 3) + 1];  // callers keep one readable byte past the row
    return ((lo | (hi << 8)) >> (pos & 7)) & ((1u << bits) - 1u);
}

constexpr size_t DECODE_DYN_SMEM = sizeof(float) * (D * D + TILE_ROWS * D + RMAX * D + RMAX * TILE_ROWS) + TILE_ROWS * 80;

template <typename Tout>
__global__ void __launch_bounds__(256) decode_plain_kernel(eosq_cache_t cache, int n, const float *__restrict__ pi,
                                                           Codebook cb, Tout *__restrict__ outp) {
    extern __shared__ __align__(16) float ds[];
    float *B = ds;                                                    // [c][j] = Pi[c][j]
    float(*tile)[D] = reinterpret_cast<float(*)[D]>(ds + D * D);      // dequantised codes
    float *Vs = ds + D * D + TILE_ROWS * D;                           // [RMAX][D]
    float *Ps = Vs + RMAX * D;                                        // [RMAX][32]
    uint8_t *raw = reinterpret_cast<uint8_t *>(Ps + RMAX * TILE_ROWS); // [32][80] packed rows (+ slack)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long gb = blockIdx.x;
    const int rank = cache.rank[gb];
    const int row_bytes = D * cb.bits / 8;
    for (int e = tid; e < D * D; e += 256) B[e] = pi[e];
    for (int e = tid; e < RMAX * D; e += 256)
        Vs[e] = (e / D < rank) ? __half2float(__ushort_as_half(cache.V[gb * RMAX * D + e])) : 0.0f;
    for (int r0 = 0; r0 < n; r0 += TILE_ROWS) {
        __syncthreads();
        for (int e = tid; e < TILE_ROWS * 80; e += 256) {
            const int r = e / 80, k = e % 80;
            raw[e] = (k < row_bytes && r0 + r < n) ? cache.codes[(static_cast<size_t>(gb) * n + r0 + r) * row_bytes + k] : 0;
        }
        for (int e = tid; e < RMAX * TILE_ROWS; e += 256) {
            const int i = e / TILE_ROWS, r = e % TILE_ROWS;
            Ps[e] = (i < rank && r0 + r < n)
                        ? __half2float(__ushort_as_half(cache.P[(static_cast<size_t>(gb) * RMAX + i) * n + r0 + r]))
                        : 0.0f;
        }
        __syncthreads();
        for (int e = tid; e < TILE_ROWS * D; e += 256)
            tile[e / D][e % D] = cb.centroid[extract_code(raw + (e / D) * 80, e % D, cb.bits)];
        __syncthreads();
        float acc[4][4];
        tile_gemm(tile, B, warp, lane, acc);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int lr = 4 * warp + r, row = r0 + lr;
            if (row >= n) continue;
            const float rho = __half2float(__ushort_as_half(cache.norms[static_cast<size_t>(gb) * n + row]));
            float x[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float low = 0.0f;
                for (int i = 0; i < rank; ++i) low = fmaf(Ps[i * TILE_ROWS + lr], Vs[i * D + 4 * lane + c], low);
                x[c] = fmaf(rho, acc[r][c], low);
            }
            Tout *dst = outp + (static_cast<size_t>(gb) * n + row) * D + 4 * lane;
#pragma unroll
            for (int c = 0; c < 4; ++c) dst[c] = static_cast<Tout>(x[c]);
        }
    }
}

void launch_decode_plain(const eosq_cache_t &cache, int64_t nb, int n, const Rotation &rot, const Codebook &cb,
                         void *out_blocks, int out_dtype, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaFuncSetAttribute(decode_plain_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(DECODE_DYN_SMEM));
        cudaFuncSetAttribute(decode_plain_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(DECODE_DYN_SMEM));
        configured = true;
    }
    if (out_dtype == EOSQ_F32)
        decode_plain_kernel<float><<<static_cast<unsigned>(nb), 256, DECODE_DYN_SMEM, s>>>(
            cache, n, rot.pi, cb, static_cast<float *>(out_blocks));
    else
        decode_plain_kernel<__half><<<static_cast<unsigned>(nb), 256, DECODE_DYN_SMEM, s>>>(
            cache, n, rot.pi, cb, static_cast<__half *>(out_blocks));
}

// ------------------------------------------------------------------------------------------
// Attention logits from the compressed keys (Remark 6.4):
//   s[g][t] = scale ( sum_i (q_g . zeta_i) P[i][t] + rho_t sum_c (Pi q_g)[c] centroid[code[t][c]] ).
// One CTA per (head, block); one thread per token; query heads in groups of at most 8.
// ------------------------------------------------------------------------------------------
constexpr int SCORE_G = 8;

__global__ void __launch_bounds__(256) scores_plain_kernel(eosq_cache_t cache, long long bph, long long head_stride,
                                                           int n, const float *__restrict__ pi_t, Codebook cb,
                                                           const __half *__restrict__ q, int G, float scale,
                                                           float *__restrict__ scores) {
    __shared__ __align__(16) float qs[SCORE_G][D];      // queries of this group
    __shared__ __align__(16) float wq[D][SCORE_G];      // (Pi q_g)[c], g fastest
    __shared__ float aq[SCORE_G][RMAX];                  // q_g . zeta_i
    __shared__ float cen[16];
    const int tid = threadIdx.x;
    const long long head = blockIdx.x / bph, jb = blockIdx.x % bph;
    const long long gb = head * head_stride + jb;
    const int rank = cache.rank[gb];
    const int row_bytes = D * cb.bits / 8;
    const int row_words = row_bytes / 4;
    const unsigned mask = (1u << cb.bits) - 1u;
    if (tid < 16) cen[tid] = cb.centroid[tid];
    for (int g0 = 0; g0 < G; g0 += SCORE_G) {
        const int gcount = min(SCORE_G, G - g0);
        __syncthreads();
        for (int e = tid; e < SCORE_G * D; e += 256) {
            const int g = e / D;
            qs[g][e % D] = (g < gcount) ? __half2float(q[(head * G + g0 + g) * D + (e % D)]) : 0.0f;
        }
        __syncthreads();
        {   // rotate the queries: wq[c][g] = sum_j Pi[c][j] q_g[j]
            const int c = tid & (D - 1), half = tid >> 7;
            float w[SCORE_G / 2];
#pragma unroll
            for (int g = 0; g < SCORE_G / 2; ++g) w[g] = 0.0f;
            for (int j = 0; j < D; ++j) {
                const float pv = pi_t[j * D + c];
#pragma unroll
                for (int g = 0; g < SCORE_G / 2; ++g) w[g] = fmaf(pv, qs[half * (SCORE_G / 2) + g][j], w[g]);
            }
#pragma unroll
            for (int g = 0; g < SCORE_G / 2; ++g) wq[c][half * (SCORE_G / 2) + g] = w[g];
        }
        if (tid < SCORE_G * RMAX) {
            const int g = tid / RMAX, i = tid % RMAX;
            float a = 0.0f;
            if (i < rank)
                for (int j = 0; j < D; ++j)
                    a = fmaf(qs[g][j], __half2float(__ushort_as_half(cache.V[(gb * RMAX + i) * D + j])), a);
            aq[g][i] = a;
        }
        __syncthreads();
        for (int t = tid; t < n; t += 256) {
            const unsigned *row = reinterpret_cast<const unsigned *>(cache.codes) + (static_cast<size_t>(gb) * n + t) * row_words;
            float acc[SCORE_G];
#pragma unroll
            for (int g = 0; g < SCORE_G; ++g) acc[g] = 0.0f;
            unsigned long long window = 0ull;
            int have = 0, next_word = 0;
            for (int c = 0; c < D; ++c) {
                if (have < cb.bits) {
                    window |= static_cast<unsigned long long>(row[next_word++]) << have;
                    have += 32;
                }
                const float zc = cen[static_cast<unsigned>(window) & mask];
                window >>= cb.bits;
                have -= cb.bits;
                const float4 w0 = *reinterpret_cast<const float4 *>(&wq[c][0]);
                const float4 w1 = *reinterpret_cast<const float4 *>(&wq[c][4]);
                acc[0] = fmaf(zc, w0.x, acc[0]);
                acc[1] = fmaf(zc, w0.y, acc[1]);
                acc[2] = fmaf(zc, w0.z, acc[2]);
                acc[3] = fmaf(zc, w0.w, acc[3]);
                acc[4] = fmaf(zc, w1.x, acc[4]);
                acc[5] = fmaf(zc, w1.y, acc[5]);
                acc[6] = fmaf(zc, w1.z, acc[6]);
                acc[7] = fmaf(zc, w1.w, acc[7]);
            }
            const float rho = __half2float(__ushort_as_half(cache.norms[static_cast<size_t>(gb) * n + t]));
            float pt[RMAX];
            for (int i = 0; i < rank; ++i)
                pt[i] = __half2float(__ushort_as_half(cache.P[(static_cast<size_t>(gb) * RMAX + i) * n + t]));
#pragma unroll
            for (int g = 0; g < SCORE_G; ++g) {
                if (g < gcount) {
                    float low = 0.0f;
                    for (int i = 0; i < rank; ++i) low = fmaf(aq[g][i], pt[i], low);
                    scores[(head * G + g0 + g) * (bph * n) + jb * n + t] = scale * fmaf(rho, acc[g], low);
                }
            }
        }
    }
}

void launch_scores_plain(const eosq_cache_t &cache, int64_t heads, int64_t bph, int64_t head_stride, int n,
                         const Rotation &rot, const Codebook &cb, const __half *q, int G, float scale,
                         float *scores, cudaStream_t s) {
    scores_plain_kernel<<<static_cast<unsigned>(heads * bph), 256, 0, s>>>(
        cache, static_cast<long long>(bph), static_cast<long long>(head_stride), n, rot.pi_t, cb, q, G, scale, scores);
}

}  // namespace eosq
