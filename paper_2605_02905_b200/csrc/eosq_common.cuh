// Shared declarations of the eosq CUDA library (sm_100a): constants, the context, the
// workspace view and the kernel launchers implemented in the other translation units.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <string>
#include <vector>

#include "eosq.h"

namespace eosq {

constexpr int D = 128;         // head dimension the kernels are written for
constexpr int RMAX = EOSQ_RMAX;
constexpr int KPILOT = 11;     // floor(128^(1/2.01)), checked against eosq_pilot_k at create time
constexpr int NMAX = 4096;

// Lloyd-Max codebook as kernel parameter (fp32 copies of the host doubles).
struct Codebook {
    float centroid[16];
    float threshold[15];
    int bits;
};

// Device copies of one seeded rotation.
struct Rotation {
    uint64_t seed = 0;
    float *pi = nullptr;     // [c][j]  z_c = sum_j pi[c][j] u_j
    float *pi_t = nullptr;   // [j][c]
};

// Scratch of one chunk of blocks, carved out of the caller's workspace.
struct Workspace {
    double *gram;   // [C][D][D]   Gram matrix, later the Householder vectors (rows, right of the superdiagonal)
    double *diag;   // [C][D]      tridiagonal diagonal
    double *off;    // [C][D]      tridiagonal off-diagonal (D-1 used)
    double *tau;    // [C][D]      Householder scalars (D-2 used)
    double *lam;    // [C][D]      eigenvalues, descending
    float *vr;      // [C][RMAX][D] right vectors as used for the residual
    float *coef;    // [C][RMAX]   phi_i / sigma_i
    int *rank;      // [C]
    int *redo_list; // [C]         blocks whose spectrum the tensor-core Gram matrix cannot resolve
    int *redo_count;// [1]
};

constexpr size_t WS_PER_BLOCK = sizeof(double) * (D * D + 4 * D) + sizeof(float) * (RMAX * D + RMAX) + 64 + 8;
// A block is redone with the exact (double precision) Gram matrix when its smallest eigenvalue is
// below this fraction of its largest: the tensor-core Gram matrix carries an absolute error of
// about 1e-8 of the largest eigenvalue, which would move smaller singular values by more than
// 5e-5 relative.
constexpr double REDO_RATIO = 1e-4;
constexpr int64_t CHUNK_BLOCKS = 18944;  // 128 per SM on 148 SMs.  Every kernel here gives a block to one CTA, team or warp whose
                                        // steps are chains of latencies, so throughput comes from blocks in flight: a 16384-block
                                        // cache went from 18.9 ms in chunks of 1184 to 17.1 ms in one chunk (2.2 GB of scratch).

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Raises a kernel's dynamic shared-memory limit, once per kernel and device (the attribute belongs
// to the device's copy of the function, so a second GPU in the same process needs its own call).
// Implemented in eosq_api.cu.
bool ensure_dynamic_smem(const void *kernel, size_t bytes);

// Carve the scratch arrays of one chunk (capacity `cap` blocks) out of `base`; returns the bytes
// used.  With base = nullptr only the size is computed.
inline size_t carve(void *base, int64_t cap, Workspace *ws) {
    char *p = static_cast<char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void *q = p ? p + off : nullptr;
        off = align_up(off + bytes, 256);
        return q;
    };
    Workspace w;
    w.gram = static_cast<double *>(take(sizeof(double) * cap * D * D));
    w.diag = static_cast<double *>(take(sizeof(double) * cap * D));
    w.off = static_cast<double *>(take(sizeof(double) * cap * D));
    w.tau = static_cast<double *>(take(sizeof(double) * cap * D));
    w.lam = static_cast<double *>(take(sizeof(double) * cap * D));
    w.vr = static_cast<float *>(take(sizeof(float) * cap * RMAX * D));
    w.coef = static_cast<float *>(take(sizeof(float) * cap * RMAX));
    w.rank = static_cast<int *>(take(sizeof(int) * cap));
    w.redo_list = static_cast<int *>(take(sizeof(int) * cap));
    w.redo_count = static_cast<int *>(take(sizeof(int)));
    if (ws) *ws = w;
    return off;
}

}  // namespace eosq

enum Stage { ST_GRAM = 0, ST_TRIDIAG_A, ST_TRIDIAG_B, ST_TRIDIAG_C, ST_EIGVALS, ST_SPECTRAL, ST_QUANT, ST_DECODE, ST_SCORES, ST_REDO, ST_OTHER };

struct eosq_ctx {
    struct Timed {
        int stage;
        cudaEvent_t start, stop;
    };
    int device = 0;
    int sm_count = 148;
    int *dev_err = nullptr;   // device word: bits raised by kernels whose bounded waits gave up
    std::vector<eosq::Rotation> rotations;
    std::string last_error;
    int64_t launches = 0;
    uint32_t profile_mask = 0;   // bit i set: launches of stage i are bracketed by events
    std::vector<Timed> timed;
    std::vector<cudaEvent_t> free_events;
    void *scores_w = nullptr;        // score path: per-head images of the operand W = Pi q (grown on demand)
    size_t scores_w_bytes = 0;
    // host-buffer path: copy streams and hand-over events of its two arena slots (created on first use)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
};

namespace eosq {

// The launch sequence of the encode path for blocks [b0, b0 + nb) of `blocks` (implemented with
// the C entry points; shared by eosq_encode and eosq_encode_static).
int encode_chunk(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t b0, int64_t nb, int n, int bits,
                 const Rotation &rot, const Codebook &cb, const eosq_cache_t &out_all, const Workspace &ws,
                 cudaStream_t s);

// ---- launchers (each enqueues one kernel on `stream`) ---------------------------------------
// Gram matrix G = S^T S of each block, accumulated in double from exact products.
// With `list` given, CTA c works on block list[c] and CTAs c >= *count do nothing (same for the
// two spectral launchers below).
void launch_gram_plain(const void *blocks, int in_dtype, int64_t nb, int n, double *gram, const int *list,
                       const int *count, cudaStream_t s);
// Same result from the tensor cores (fp16 blocks only).  The chunk starts `block0` blocks into
// `blocks_all`.  Returns false if the launch could not be set up (no kernel was enqueued).
bool launch_gram_tc(const void *blocks_all, int64_t nb_all, int64_t block0, int64_t nb, int n, double *gram, int *err,
                    int sm_count, cudaStream_t s);
// Householder tridiagonalisation of each Gram matrix (in place: reflectors overwrite it).
// Grid of a kernel that works through blocks [0, nb), or, with a list, through the few listed
// blocks: those launches are almost always empty, and a small grid keeps them cheap.
constexpr int64_t LIST_GRID = 148;
inline unsigned list_grid(int64_t nb, const int *list) {
    return static_cast<unsigned>(list ? (nb < LIST_GRID ? nb : LIST_GRID) : nb);
}
constexpr int TRIDIAG_PARTS = 3;
void launch_tridiag(int part, int64_t nb, const Workspace &ws, const int *list, const int *count, int sm_count, cudaStream_t s);
// All eigenvalues of each tridiagonal matrix by Sturm bisection.
// With `full` every eigenvalue is resolved, otherwise the 3k + 1 largest and the smallest (what
// Algorithm 2 reads one by one and what the accuracy check of the Gram matrix needs).
void launch_eigvals(int64_t nb, const Workspace &ws, const int *list, const int *count, int *mark_list, bool full, cudaStream_t s);
// Clears the redo list / appends every block whose eigenvalue range exceeds 1 / REDO_RATIO.
// Bulk edge, rank, imputed spectrum, D-transform and shrinkage; kept eigenvectors.
void launch_spectral(int64_t nb, int n, const Workspace &ws, const eosq_cache_t &out, int64_t block0, bool full,
                     cudaStream_t s);
// Residual, norm, rotation, codes, packing and left factors.
void launch_quant_plain(const void *blocks, int in_dtype, int64_t nb, int n, const Workspace &ws,
                        const Rotation &rot, const Codebook &cb, const eosq_cache_t &out, int64_t block0,
                        cudaStream_t s);
// Same outputs from the tensor cores (fp16 blocks only); `out` is already offset to the chunk.
bool launch_quant_tc(const void *blocks_all, int64_t block0, int64_t nb, int n, const Workspace &ws, const Rotation &rot,
                     const Codebook &cb, const eosq_cache_t &out, int *err, int sm_count, cudaStream_t s);
bool decode_tc_supported(const eosq_cache_t &cache, int bits, const void *out_blocks);
bool launch_decode_tc(const eosq_cache_t &cache, int64_t nb, int n, const Rotation &rot, const Codebook &cb, void *out_blocks,
                      int out_dtype, int *err, int sm_count, cudaStream_t s);
// Attention logits on the tensor cores; `supported` checks the 16-byte alignment the kernel's bulk copies
// need, the launcher returns false if nothing was enqueued.
bool scores_tc_supported(const eosq_cache_t &cache, int bits, int n);
bool launch_scores_tc(const eosq_cache_t &cache, int64_t heads, int64_t bph, int64_t head_stride, int n, const Rotation &rot,
                      const Codebook &cb, const __half *q, int G, float scale, float *scores, int *err, int sm_count,
                      void **scratch, size_t *scratch_bytes, int64_t *kernels, cudaStream_t s);

// ---- small device helpers -------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <typename T>
__device__ __forceinline__ float load_as_float(const T *p);
template <>
__device__ __forceinline__ float load_as_float<float>(const float *p) { return *p; }
template <>
__device__ __forceinline__ float load_as_float<__half>(const __half *p) { return __half2float(*p); }

void launch_wait_timeout(int *err, uint32_t polls, cudaStream_t s);

}  // namespace eosq
