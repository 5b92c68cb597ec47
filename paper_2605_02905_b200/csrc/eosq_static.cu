// eosq_encode_static: eosq_encode for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc at the point where they compress
// a block: code running while a stream is being captured, real-time serving loops whose memory
// was carved up at start-up and must not grow, and plug-ins that were handed a fixed arena and no
// allocator.  eosq_encode asks such a caller for a workspace and caches the rotation in memory it
// allocates itself; this variant does neither.  Its scratch (the per-block Gram matrices,
// tridiagonal forms, eigenvalues and kept vectors, plus the two copies of the rotation) lives in
// one file-scope __device__ array that every GPU loading the library holds until exit.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

#include "eosq_common.cuh"

using namespace eosq;

namespace {

constexpr int64_t STATIC_MAX_BLOCKS = EOSQ_STATIC_MAX_BLOCKS;
constexpr size_t ROT_BYTES = sizeof(float) * D * D;  // one copy of Pi
// Upper bound of carve() for STATIC_MAX_BLOCKS blocks: every array rounded up to 256 bytes.
constexpr size_t STATIC_WS_BYTES = STATIC_MAX_BLOCKS * WS_PER_BLOCK + 16 * 256;
constexpr size_t STATIC_BYTES = 2 * ROT_BYTES + STATIC_WS_BYTES;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

constexpr int MAX_DEVICES = 64;
struct PerDevice {
    unsigned char *base = nullptr;  // device address of g_static_scratch on this device
    bool have_rotation = false;
    uint64_t seed = 0;              // seed of the rotation currently stored in the array
};
PerDevice g_dev[MAX_DEVICES];
std::mutex g_mu;

bool fail(eosq_ctx *ctx, cudaError_t err, const char *what) {
    if (err == cudaSuccess) return false;
    ctx->last_error = std::string(what) + ": " + cudaGetErrorString(err);
    return true;
}

}  // namespace

extern "C" int64_t eosq_encode_static_max_blocks(void) { return STATIC_MAX_BLOCKS; }

extern "C" int eosq_encode_static(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t num_blocks, int n, int d,
                                  int bits, uint64_t seed, const eosq_cache_t *out, void *cuda_stream) {
    if (!ctx || num_blocks < 0 || (in_dtype != EOSQ_F16 && in_dtype != EOSQ_F32)) return EOSQ_ERR_INVALID_ARG;
    if (d != D || bits < 1 || bits > 4 || n < d || n > NMAX || (n % 8) != 0) return EOSQ_ERR_UNSUPPORTED;
    if (num_blocks > STATIC_MAX_BLOCKS) {
        ctx->last_error = "eosq_encode_static: num_blocks " + std::to_string(num_blocks) + " exceeds the fixed scratch (" +
                          std::to_string(STATIC_MAX_BLOCKS) + " blocks); split the call or use eosq_encode";
        return EOSQ_ERR_BUFFER_TOO_SMALL;
    }
    if (num_blocks == 0) return EOSQ_OK;
    if (!blocks || !out || !out->codes || !out->norms || !out->rank || !out->sigma || !out->phi || !out->P || !out->V ||
        !out->status)
        return EOSQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blocks) & 15u) || (reinterpret_cast<uintptr_t>(out->codes) & 15u))
        return EOSQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    int dev = -1;
    if (fail(ctx, cudaGetDevice(&dev), "cudaGetDevice")) return EOSQ_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return EOSQ_ERR_UNSUPPORTED;
    if (dev != ctx->device) {   // the context's error word and constants live on its own device
        ctx->last_error = "the current CUDA device is not the one this context was created on";
        return EOSQ_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    PerDevice &pd = g_dev[dev];
    if (!pd.base) {
        // once per device, with that device current: turn the symbol into this device's address
        void *p = nullptr;
        if (fail(ctx, cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)")) return EOSQ_ERR_CUDA;
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255u)) return EOSQ_ERR_CUDA;
        if (carve(nullptr, STATIC_MAX_BLOCKS, nullptr) > STATIC_WS_BYTES) return EOSQ_ERR_BUFFER_TOO_SMALL;
        pd.base = static_cast<unsigned char *>(p);
    }
    Rotation rot;
    rot.seed = seed;
    rot.pi = reinterpret_cast<float *>(pd.base);
    rot.pi_t = reinterpret_cast<float *>(pd.base + ROT_BYTES);
    if (!pd.have_rotation || pd.seed != seed) {
        // stream-ordered upload from ordinary host memory: the runtime stages the bytes before it
        // returns, and earlier calls on this stream that still read the old rotation finish first
        std::vector<double> pi(static_cast<size_t>(D) * D);
        int rc = eosq_rotation(D, seed, pi.data());
        if (rc != EOSQ_OK) return rc;
        std::vector<float> f(2 * pi.size());
        for (int c = 0; c < D; ++c)
            for (int j = 0; j < D; ++j) {
                const float v = static_cast<float>(pi[static_cast<size_t>(c) * D + j]);
                f[static_cast<size_t>(c) * D + j] = v;
                f[pi.size() + static_cast<size_t>(j) * D + c] = v;
            }
        pd.have_rotation = false;
        if (fail(ctx, cudaMemcpyAsync(pd.base, f.data(), 2 * ROT_BYTES, cudaMemcpyHostToDevice, s), "cudaMemcpyAsync(rotation)"))
            return EOSQ_ERR_CUDA;
        pd.have_rotation = true;
        pd.seed = seed;
    }
    Codebook cb;
    {
        double cen[16], thr[15];
        int rc = eosq_codebook(bits, D, cen, thr);
        if (rc != EOSQ_OK) return rc;
        std::memset(&cb, 0, sizeof(cb));
        cb.bits = bits;
        for (int i = 0; i < (1 << bits); ++i) cb.centroid[i] = static_cast<float>(cen[i]);
        for (int i = 0; i + 1 < (1 << bits); ++i) cb.threshold[i] = static_cast<float>(thr[i]);
    }
    // Nothing in the scratch has to start at zero: every array is fully written for the blocks of
    // this call before it is read, so the previous call's contents are simply overwritten.
    Workspace ws;
    carve(pd.base + 2 * ROT_BYTES, num_blocks, &ws);
    int rc = encode_chunk(ctx, blocks, in_dtype, 0, num_blocks, n, bits, rot, cb, *out, ws, s);
    if (rc != EOSQ_OK) return rc;
    if (fail(ctx, cudaGetLastError(), "eosq_encode_static launch")) return EOSQ_ERR_CUDA;
    return EOSQ_OK;
}
