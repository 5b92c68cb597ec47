// C-ABI entry points of the eosq library: argument checks, the context's cached constants,
// workspace carving and the launch sequence of each call.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <utility>

#include "eosq_common.cuh"

using namespace eosq;

bool eosq::ensure_dynamic_smem(const void *kernel, size_t bytes) {
    static std::mutex mu;
    static std::vector<std::pair<const void *, int>> done;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    for (const auto &e : done)
        if (e.first == kernel && e.second == dev) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) != cudaSuccess) return false;
    // every kernel that comes here sizes its CTAs per SM by shared memory: ask for all of it
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) return false;
    done.emplace_back(kernel, dev);
    return true;
}

namespace {

// The context's buffers, constants and error word live on the device it was created on: every
// device entry point refuses to run with another device current.
bool on_ctx_device(eosq_ctx *ctx) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != ctx->device) {
        ctx->last_error = "the current CUDA device is not the one this context was created on";
        return false;
    }
    return true;
}

bool record_cuda(eosq_ctx *ctx, cudaError_t err, const char *what) {
    if (err == cudaSuccess) return false;
    if (ctx) ctx->last_error = std::string(what) + ": " + cudaGetErrorString(err);
    return true;
}

int check_shape(int n, int d, int bits) {
    if (d != D || bits < 1 || bits > 4 || n < d || n > NMAX || (n % 8) != 0) return EOSQ_ERR_UNSUPPORTED;
    return EOSQ_OK;
}

int get_rotation(eosq_ctx *ctx, int d, uint64_t seed, Rotation *out) {
    for (const Rotation &r : ctx->rotations)
        if (r.seed == seed) {
            *out = r;
            return EOSQ_OK;
        }
    std::vector<double> pi(static_cast<size_t>(d) * d);
    int rc = eosq_rotation(d, seed, pi.data());
    if (rc != EOSQ_OK) return rc;
    std::vector<float> f(pi.size()), ft(pi.size());
    for (int c = 0; c < d; ++c)
        for (int j = 0; j < d; ++j) {
            f[static_cast<size_t>(c) * d + j] = static_cast<float>(pi[static_cast<size_t>(c) * d + j]);
            ft[static_cast<size_t>(j) * d + c] = static_cast<float>(pi[static_cast<size_t>(c) * d + j]);
        }
    Rotation r;
    r.seed = seed;
    const size_t bytes = sizeof(float) * f.size();
    if (record_cuda(ctx, cudaMalloc(&r.pi, bytes), "cudaMalloc(rotation)")) return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, cudaMalloc(&r.pi_t, bytes), "cudaMalloc(rotation)")) return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, cudaMemcpy(r.pi, f.data(), bytes, cudaMemcpyHostToDevice), "cudaMemcpy(rotation)")) return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, cudaMemcpy(r.pi_t, ft.data(), bytes, cudaMemcpyHostToDevice), "cudaMemcpy(rotation)")) return EOSQ_ERR_CUDA;
    ctx->rotations.push_back(r);
    *out = r;
    return EOSQ_OK;
}

int get_codebook(int d, int bits, Codebook *cb) {
    double cen[16], thr[15];
    int rc = eosq_codebook(bits, d, cen, thr);
    if (rc != EOSQ_OK) return rc;
    std::memset(cb, 0, sizeof(*cb));
    cb->bits = bits;
    for (int i = 0; i < (1 << bits); ++i) cb->centroid[i] = static_cast<float>(cen[i]);
    for (int i = 0; i + 1 < (1 << bits); ++i) cb->threshold[i] = static_cast<float>(thr[i]);
    return EOSQ_OK;
}

// Offset every array of a cache by `b0` blocks (so kernels can index from 0 within a chunk).
eosq_cache_t shifted(const eosq_cache_t &c, int64_t b0, int n, int bits) {
    eosq_cache_t o = c;
    const int64_t rb = D * bits / 8;
    if (o.codes) o.codes += b0 * n * rb;
    if (o.norms) o.norms += b0 * n;
    if (o.rank) o.rank += b0;
    if (o.sigma) o.sigma += b0 * RMAX;
    if (o.phi) o.phi += b0 * RMAX;
    if (o.P) o.P += b0 * RMAX * n;
    if (o.V) o.V += b0 * RMAX * D;
    if (o.status) o.status += b0;
    if (o.eig) o.eig += b0 * D;
    if (o.lambda_plus) o.lambda_plus += b0;
    if (o.vr32) o.vr32 += b0 * RMAX * D;
    if (o.coef) o.coef += b0 * RMAX;
    return o;
}

cudaEvent_t take_event(eosq_ctx *ctx) {
    if (!ctx->free_events.empty()) {
        cudaEvent_t e = ctx->free_events.back();
        ctx->free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

// Runs `launch` (which enqueues one kernel on `s`; the score path adds its extra ones itself), counting it and, when profiling is
// on, bracketing it with events.
template <typename F>
void run_stage(eosq_ctx *ctx, int stage, cudaStream_t s, F &&launch) {
    if ((ctx->profile_mask >> stage) & 1u) {
        eosq_ctx::Timed t{stage, take_event(ctx), take_event(ctx)};
        cudaEventRecord(t.start, s);
        launch();
        cudaEventRecord(t.stop, s);
        ctx->timed.push_back(t);
    } else {
        launch();
    }
    ctx->launches += 1;
}

bool cache_required_ok(const eosq_cache_t *c) {
    return c && c->codes && c->norms && c->rank && c->sigma && c->phi && c->P && c->V && c->status;
}

}  // namespace

// The launch sequence of eosq_encode for blocks [b0, b0 + nb) of `blocks`, with the scratch of
// one chunk in `ws`.
int eosq::encode_chunk(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t b0, int64_t nb, int n, int bits,
                       const Rotation &rot, const Codebook &cb, const eosq_cache_t &out_all, const Workspace &ws,
                       cudaStream_t s) {
    const size_t esize = (in_dtype == EOSQ_F32) ? 4 : 2;
    const char *chunk_in = static_cast<const char *>(blocks) + static_cast<size_t>(b0) * n * D * esize;
    const eosq_cache_t o = shifted(out_all, b0, n, bits);
    // The queue of blocks for the second pass must be empty when the eigenvalue kernel runs.  Every
    // chunk leaves it empty (the spectral kernel clears it); the first chunk of a call cannot know
    // what the scratch held before.
    if (b0 == 0 && record_cuda(ctx, cudaMemsetAsync(ws.redo_count, 0, sizeof(int), s), "cudaMemsetAsync(redo count)")) return EOSQ_ERR_CUDA;
    if (in_dtype == EOSQ_F16) {
        bool setup_ok = true;
        run_stage(ctx, ST_GRAM, s, [&] { setup_ok = launch_gram_tc(blocks, 0, b0, nb, n, ws.gram, ctx->dev_err, ctx->sm_count, s); });
        if (!setup_ok) {
            ctx->last_error = "tensor-core Gram kernel: tensor map or launch set-up failed";
            return EOSQ_ERR_CUDA;
        }
    } else {
        run_stage(ctx, ST_GRAM, s, [&] { launch_gram_plain(chunk_in, in_dtype, nb, n, ws.gram, nullptr, nullptr, s); });
    }
    const bool full = out_all.eig != nullptr;   // the optional eigenvalue output asks for the whole spectrum
    static_assert(TRIDIAG_PARTS == 3 && ST_TRIDIAG_C == ST_TRIDIAG_A + 2, "one profiling stage per tridiagonalisation kernel");
    for (int part = 0; part < TRIDIAG_PARTS; ++part)
        run_stage(ctx, ST_TRIDIAG_A + part, s, [&] { launch_tridiag(part, nb, ws, nullptr, nullptr, ctx->sm_count, s); });
    // the eigenvalue kernel also queues, in ws.redo_list, the blocks the tensor-core Gram matrix cannot resolve
    run_stage(ctx, ST_EIGVALS, s, [&] { launch_eigvals(nb, ws, nullptr, nullptr, (in_dtype == EOSQ_F16) ? ws.redo_list : nullptr, full, s); });
    if (in_dtype == EOSQ_F16) {
        // second pass, exact Gram matrix, for those blocks (the spectral kernel clears the queue afterwards)
        run_stage(ctx, ST_REDO, s, [&] { launch_gram_plain(chunk_in, in_dtype, nb, n, ws.gram, ws.redo_list, ws.redo_count, s); });
        for (int part = 0; part < TRIDIAG_PARTS; ++part)
            run_stage(ctx, ST_REDO, s, [&] { launch_tridiag(part, nb, ws, ws.redo_list, ws.redo_count, ctx->sm_count, s); });
        run_stage(ctx, ST_REDO, s, [&] { launch_eigvals(nb, ws, ws.redo_list, ws.redo_count, nullptr, full, s); });
    }
    run_stage(ctx, ST_SPECTRAL, s, [&] { launch_spectral(nb, n, ws, o, 0, full, s); });
    if (in_dtype == EOSQ_F16) {
        bool setup_ok = true;
        run_stage(ctx, ST_QUANT, s, [&] { setup_ok = launch_quant_tc(blocks, b0, nb, n, ws, rot, cb, o, ctx->dev_err, ctx->sm_count, s); });
        if (!setup_ok) {
            ctx->last_error = "tensor-core quantisation kernel: tensor map or launch set-up failed";
            return EOSQ_ERR_CUDA;
        }
    } else {
        run_stage(ctx, ST_QUANT, s, [&] { launch_quant_plain(chunk_in, in_dtype, nb, n, ws, rot, cb, o, 0, s); });
    }
    return EOSQ_OK;
}

extern "C" size_t eosq_workspace_bytes(int64_t num_blocks, int n, int d) {
    (void)n;
    if (num_blocks <= 0 || d != D) return 0;
    return carve(nullptr, std::min<int64_t>(num_blocks, CHUNK_BLOCKS), nullptr);
}

extern "C" int eosq_create(eosq_ctx **out) {
    if (!out) return EOSQ_ERR_INVALID_ARG;
    if (eosq_pilot_k(D) != KPILOT) return EOSQ_ERR_UNSUPPORTED;
    eosq_ctx *ctx = new (std::nothrow) eosq_ctx();
    if (!ctx) return EOSQ_ERR_INVALID_ARG;
    if (record_cuda(ctx, cudaGetDevice(&ctx->device), "cudaGetDevice")) {
        delete ctx;
        return EOSQ_ERR_CUDA;
    }
    cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
    if (record_cuda(ctx, cudaMalloc(&ctx->dev_err, 256), "cudaMalloc(error word)") ||
        record_cuda(ctx, cudaMemset(ctx->dev_err, 0, 256), "cudaMemset(error word)")) {
        cudaFree(ctx->dev_err);
        delete ctx;
        return EOSQ_ERR_CUDA;
    }
    *out = ctx;
    return EOSQ_OK;
}

extern "C" int eosq_destroy(eosq_ctx *ctx) {
    if (!ctx) return EOSQ_OK;
    cudaFree(ctx->dev_err);
    for (Rotation &r : ctx->rotations) {
        cudaFree(r.pi);
        cudaFree(r.pi_t);
    }
    for (eosq_ctx::Timed &t : ctx->timed) {
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
    }
    for (cudaEvent_t e : ctx->free_events) cudaEventDestroy(e);
    cudaFree(ctx->scores_w);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    if (ctx->ev_start) cudaEventDestroy(ctx->ev_start);
    for (int i = 0; i < 2; ++i) {
        if (ctx->ev_in[i]) cudaEventDestroy(ctx->ev_in[i]);
        if (ctx->ev_done[i]) cudaEventDestroy(ctx->ev_done[i]);
        if (ctx->ev_out[i]) cudaEventDestroy(ctx->ev_out[i]);
    }
    delete ctx;
    return EOSQ_OK;
}

extern "C" int eosq_profile_enable(eosq_ctx *ctx, int on) {
    if (!ctx) return EOSQ_ERR_INVALID_ARG;
    ctx->profile_mask = on ? ((1u << EOSQ_NUM_STAGES) - 1u) : 0u;
    return EOSQ_OK;
}

extern "C" int eosq_profile_select(eosq_ctx *ctx, uint32_t stage_mask) {
    if (!ctx || (stage_mask >> EOSQ_NUM_STAGES)) return EOSQ_ERR_INVALID_ARG;
    ctx->profile_mask = stage_mask;
    return EOSQ_OK;
}

extern "C" int eosq_profile_read(eosq_ctx *ctx, float *ms, int64_t *launches) {
    if (!ctx || !ms || !launches) return EOSQ_ERR_INVALID_ARG;
    for (int i = 0; i < EOSQ_NUM_STAGES; ++i) {
        ms[i] = 0.0f;
        launches[i] = 0;
    }
    int rc = EOSQ_OK;
    for (eosq_ctx::Timed &t : ctx->timed) {
        float e = 0.0f;
        if (record_cuda(ctx, cudaEventSynchronize(t.stop), "cudaEventSynchronize") ||
            record_cuda(ctx, cudaEventElapsedTime(&e, t.start, t.stop), "cudaEventElapsedTime"))
            rc = EOSQ_ERR_CUDA;
        ms[t.stage] += e;
        launches[t.stage] += 1;
        ctx->free_events.push_back(t.start);
        ctx->free_events.push_back(t.stop);
    }
    ctx->timed.clear();
    return rc;
}

extern "C" const char *eosq_last_cuda_error(const eosq_ctx *ctx) { return ctx ? ctx->last_error.c_str() : ""; }

extern "C" int64_t eosq_launch_count(const eosq_ctx *ctx) { return ctx ? ctx->launches : 0; }

extern "C" int eosq_encode(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t num_blocks, int n, int d,
                           int bits, uint64_t seed, const eosq_cache_t *out, void *workspace,
                           size_t workspace_bytes, void *cuda_stream) {
    if (!ctx || num_blocks < 0 || (in_dtype != EOSQ_F16 && in_dtype != EOSQ_F32)) return EOSQ_ERR_INVALID_ARG;
    int rc = check_shape(n, d, bits);
    if (rc != EOSQ_OK) return rc;
    if (num_blocks == 0) return EOSQ_OK;
    if (!blocks || !cache_required_ok(out) || !workspace || !on_ctx_device(ctx)) return EOSQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blocks) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        (reinterpret_cast<uintptr_t>(out->codes) & 15u))
        return EOSQ_ERR_INVALID_ARG;
    if (workspace_bytes < eosq_workspace_bytes(num_blocks, n, d)) return EOSQ_ERR_BUFFER_TOO_SMALL;
    Rotation rot;
    Codebook cb;
    if ((rc = get_rotation(ctx, d, seed, &rot)) != EOSQ_OK) return rc;
    if ((rc = get_codebook(d, bits, &cb)) != EOSQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int64_t cap = std::min<int64_t>(num_blocks, CHUNK_BLOCKS);
    Workspace ws;
    carve(workspace, cap, &ws);
    for (int64_t b0 = 0; b0 < num_blocks; b0 += cap) {
        const int64_t nb = std::min<int64_t>(cap, num_blocks - b0);
        rc = eosq::encode_chunk(ctx, blocks, in_dtype, b0, nb, n, bits, rot, cb, *out, ws, s);
        if (rc != EOSQ_OK) return rc;
    }
    if (record_cuda(ctx, cudaGetLastError(), "eosq_encode launch")) return EOSQ_ERR_CUDA;
    return EOSQ_OK;
}

extern "C" int eosq_decode(eosq_ctx *ctx, const eosq_cache_t *cache, int64_t num_blocks, int n, int d, int bits,
                           uint64_t seed, void *out_blocks, int out_dtype, void *cuda_stream) {
    if (!ctx || num_blocks < 0 || (out_dtype != EOSQ_F16 && out_dtype != EOSQ_F32)) return EOSQ_ERR_INVALID_ARG;
    int rc = check_shape(n, d, bits);
    if (rc != EOSQ_OK) return rc;
    if (num_blocks == 0) return EOSQ_OK;
    if (!cache || !cache->codes || !cache->norms || !cache->rank || !cache->P || !cache->V || !out_blocks || !on_ctx_device(ctx))
        return EOSQ_ERR_INVALID_ARG;
    Rotation rot;
    Codebook cb;
    if ((rc = get_rotation(ctx, d, seed, &rot)) != EOSQ_OK) return rc;
    if ((rc = get_codebook(d, bits, &cb)) != EOSQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (!decode_tc_supported(*cache, bits, out_blocks)) return EOSQ_ERR_INVALID_ARG;   // 16-byte alignment of codes, norms, P, out_blocks
    {
        bool setup_ok = true;
        run_stage(ctx, ST_DECODE, s, [&] { setup_ok = launch_decode_tc(*cache, num_blocks, n, rot, cb, out_blocks, out_dtype, ctx->dev_err, ctx->sm_count, s); });
        if (!setup_ok) {
            ctx->last_error = "tensor-core decode kernel: launch set-up failed";
            return EOSQ_ERR_CUDA;
        }
    }
    if (record_cuda(ctx, cudaGetLastError(), "eosq_decode launch")) return EOSQ_ERR_CUDA;
    return EOSQ_OK;
}

extern "C" int eosq_scores(eosq_ctx *ctx, const eosq_cache_t *kcache, int64_t num_kv_heads, int64_t blocks_per_head,
                           int64_t head_stride_blocks, int n, int d, int bits, uint64_t seed, const void *q, int G,
                           float scale, float *scores, void *cuda_stream) {
    if (!ctx || num_kv_heads < 0 || blocks_per_head < 0 || head_stride_blocks < blocks_per_head || G < 1)
        return EOSQ_ERR_INVALID_ARG;
    int rc = check_shape(n, d, bits);
    if (rc != EOSQ_OK) return rc;
    if (num_kv_heads == 0 || blocks_per_head == 0) return EOSQ_OK;
    if (!kcache || !kcache->codes || !kcache->norms || !kcache->rank || !kcache->P || !kcache->V || !q || !scores || !on_ctx_device(ctx))
        return EOSQ_ERR_INVALID_ARG;
    if (!scores_tc_supported(*kcache, bits, n)) return EOSQ_ERR_INVALID_ARG;   // 16-byte alignment of codes, norms, P, V
    Rotation rot;
    Codebook cb;
    if ((rc = get_rotation(ctx, d, seed, &rot)) != EOSQ_OK) return rc;
    if ((rc = get_codebook(d, bits, &cb)) != EOSQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    {
        bool setup_ok = true;
        int64_t kernels = 0;
        run_stage(ctx, ST_SCORES, s, [&] {
            setup_ok = launch_scores_tc(*kcache, num_kv_heads, blocks_per_head, head_stride_blocks, n, rot, cb,
                                        static_cast<const __half *>(q), G, scale, scores, ctx->dev_err, ctx->sm_count, &ctx->scores_w,
                                        &ctx->scores_w_bytes, &kernels, s);
        });
        ctx->launches += std::max<int64_t>(kernels, 1) - 1;   // run_stage counted one
        if (!setup_ok) {
            ctx->last_error = "tensor-core score kernel: launch set-up failed";
            return EOSQ_ERR_CUDA;
        }
    }
    if (record_cuda(ctx, cudaGetLastError(), "eosq_scores launch")) return EOSQ_ERR_CUDA;
    return EOSQ_OK;
}

// ---- host-buffer path ----------------------------------------------------------------------
namespace {
constexpr int64_t HOST_CHUNK = 592;   // one encode chunk: a short pipeline fill (the first upload overlaps nothing)

// Two slots (input chunk + its outputs) so that the upload of chunk i + 1 and the download of chunk
// i - 1 run while chunk i is encoded, and one workspace (encodes run one after another).
constexpr int HOST_SLOTS = 2;

struct Arena {
    void *in[HOST_SLOTS];
    eosq_cache_t dev[HOST_SLOTS];
    void *ws;
    size_t ws_bytes;
};

size_t carve_arena(void *base, int64_t cap, int n, int bits, int in_dtype, Arena *a) {
    char *p = static_cast<char *>(base);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        void *q = p ? p + off : nullptr;
        off = align_up(off + bytes, 256);
        return q;
    };
    Arena r;
    std::memset(&r, 0, sizeof(r));
    const size_t esize = (in_dtype == EOSQ_F32) ? 4 : 2;
    for (int slot = 0; slot < HOST_SLOTS; ++slot) {
        eosq_cache_t &c = r.dev[slot];
        r.in[slot] = take(static_cast<size_t>(cap) * n * D * esize);
        c.codes = static_cast<uint8_t *>(take(static_cast<size_t>(cap) * n * D * bits / 8));
        c.norms = static_cast<uint16_t *>(take(static_cast<size_t>(cap) * n * 2));
        c.rank = static_cast<int32_t *>(take(static_cast<size_t>(cap) * 4));
        c.sigma = static_cast<float *>(take(static_cast<size_t>(cap) * RMAX * 4));
        c.phi = static_cast<float *>(take(static_cast<size_t>(cap) * RMAX * 4));
        c.P = static_cast<uint16_t *>(take(static_cast<size_t>(cap) * RMAX * n * 2));
        c.V = static_cast<uint16_t *>(take(static_cast<size_t>(cap) * RMAX * D * 2));
        c.status = static_cast<int32_t *>(take(static_cast<size_t>(cap) * 4));
        c.eig = static_cast<float *>(take(static_cast<size_t>(cap) * D * 4));
        c.lambda_plus = static_cast<float *>(take(static_cast<size_t>(cap) * 4));
    }
    r.ws_bytes = eosq_workspace_bytes(cap, n, D);
    r.ws = take(r.ws_bytes);
    if (a) *a = r;
    return off;
}

// Streams and events of the host-buffer path, made once per context.
bool host_path_ready(eosq_ctx *ctx) {
    if (ctx->copy_in) return true;
    cudaError_t e = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming);
    for (int i = 0; i < HOST_SLOTS && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&ctx->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_out[i], cudaEventDisableTiming);
    }
    return !record_cuda(ctx, e, "host path streams and events");
}
}  // namespace

extern "C" size_t eosq_encode_host_arena_bytes(int64_t num_blocks, int n, int d, int bits, int in_dtype) {
    if (num_blocks <= 0 || check_shape(n, d, bits) != EOSQ_OK) return 0;
    return carve_arena(nullptr, std::min<int64_t>(num_blocks, HOST_CHUNK), n, bits, in_dtype, nullptr);
}

extern "C" int eosq_encode_host(eosq_ctx *ctx, const void *host_blocks, int in_dtype, int64_t num_blocks, int n,
                                int d, int bits, uint64_t seed, const eosq_cache_t *host_out, void *arena,
                                size_t arena_bytes, void *cuda_stream) {
    if (!ctx || num_blocks < 0 || (in_dtype != EOSQ_F16 && in_dtype != EOSQ_F32)) return EOSQ_ERR_INVALID_ARG;
    int rc = check_shape(n, d, bits);
    if (rc != EOSQ_OK) return rc;
    if (num_blocks == 0) return EOSQ_OK;
    if (!host_blocks || !cache_required_ok(host_out) || !arena || (reinterpret_cast<uintptr_t>(arena) & 255u) || !on_ctx_device(ctx))
        return EOSQ_ERR_INVALID_ARG;
    if (arena_bytes < eosq_encode_host_arena_bytes(num_blocks, n, d, bits, in_dtype)) return EOSQ_ERR_BUFFER_TOO_SMALL;
    if (!host_path_ready(ctx)) return EOSQ_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream), s_in = ctx->copy_in, s_out = ctx->copy_out;
    const int64_t cap = std::min<int64_t>(num_blocks, HOST_CHUNK);
    Arena a;
    carve_arena(arena, cap, n, bits, in_dtype, &a);
    const size_t esize = (in_dtype == EOSQ_F32) ? 4 : 2;
    const size_t rb = static_cast<size_t>(D) * bits / 8;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t r) {
        if (e == cudaSuccess) e = r;
        return e == cudaSuccess;
    };
    // Three streams: uploads, the caller's stream for the kernels, downloads.  Slot i % 2 is handed
    // round by events: uploaded -> encoded -> downloaded -> free for the upload of chunk i + 2.
    // Whatever the caller's stream still does with the arena comes first.
    ok(cudaEventRecord(ctx->ev_start, s));
    ok(cudaStreamWaitEvent(s_in, ctx->ev_start, 0));
    ok(cudaStreamWaitEvent(s_out, ctx->ev_start, 0));
    int64_t chunk = 0;
    for (int64_t b0 = 0; b0 < num_blocks && e == cudaSuccess; b0 += cap, ++chunk) {
        const int slot = static_cast<int>(chunk % HOST_SLOTS);
        const int64_t nb = std::min<int64_t>(cap, num_blocks - b0);
        const char *src = static_cast<const char *>(host_blocks) + static_cast<size_t>(b0) * n * D * esize;
        if (chunk >= HOST_SLOTS) ok(cudaStreamWaitEvent(s_in, ctx->ev_done[slot], 0));   // the slot's last encode has read its input
        ok(cudaMemcpyAsync(a.in[slot], src, static_cast<size_t>(nb) * n * D * esize, cudaMemcpyHostToDevice, s_in));
        ok(cudaEventRecord(ctx->ev_in[slot], s_in));
        ok(cudaStreamWaitEvent(s, ctx->ev_in[slot], 0));
        if (chunk >= HOST_SLOTS) ok(cudaStreamWaitEvent(s, ctx->ev_out[slot], 0));       // the slot's last outputs are on the host
        if (e != cudaSuccess) break;
        eosq_cache_t dev = a.dev[slot];
        if (!host_out->eig) dev.eig = nullptr;
        if (!host_out->lambda_plus) dev.lambda_plus = nullptr;
        rc = eosq_encode(ctx, a.in[slot], in_dtype, nb, n, d, bits, seed, &dev, a.ws, a.ws_bytes, s);
        if (rc != EOSQ_OK) break;
        ok(cudaEventRecord(ctx->ev_done[slot], s));
        ok(cudaStreamWaitEvent(s_out, ctx->ev_done[slot], 0));
        const eosq_cache_t h = shifted(*host_out, b0, n, bits);
        auto back = [&](void *dst, const void *srcp, size_t bytes) {
            if (dst) ok(cudaMemcpyAsync(dst, srcp, bytes, cudaMemcpyDeviceToHost, s_out));
        };
        back(h.codes, dev.codes, static_cast<size_t>(nb) * n * rb);
        back(h.norms, dev.norms, static_cast<size_t>(nb) * n * 2);
        back(h.rank, dev.rank, static_cast<size_t>(nb) * 4);
        back(h.sigma, dev.sigma, static_cast<size_t>(nb) * RMAX * 4);
        back(h.phi, dev.phi, static_cast<size_t>(nb) * RMAX * 4);
        back(h.P, dev.P, static_cast<size_t>(nb) * RMAX * n * 2);
        back(h.V, dev.V, static_cast<size_t>(nb) * RMAX * D * 2);
        back(h.status, dev.status, static_cast<size_t>(nb) * 4);
        if (dev.eig) back(h.eig, dev.eig, static_cast<size_t>(nb) * D * 4);
        if (dev.lambda_plus) back(h.lambda_plus, dev.lambda_plus, static_cast<size_t>(nb) * 4);
        ok(cudaEventRecord(ctx->ev_out[slot], s_out));
    }
    // Everything this call enqueued is waited for, also after an error: the caller owns the arena again.
    cudaStreamSynchronize(s_in);
    const cudaError_t e1 = cudaStreamSynchronize(s);
    const cudaError_t e2 = cudaStreamSynchronize(s_out);
    if (rc != EOSQ_OK) return rc;
    if (record_cuda(ctx, e, "host path copy or event")) return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, e1, "cudaStreamSynchronize")) return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, e2, "cudaStreamSynchronize(download stream)")) return EOSQ_ERR_CUDA;
    return EOSQ_OK;
}

extern "C" int eosq_check_status(eosq_ctx *ctx, const int32_t *status, int64_t num_blocks, int64_t *flagged,
                                 void *cuda_stream) {
    if (!ctx || num_blocks < 0 || (num_blocks > 0 && !status) || !on_ctx_device(ctx)) return EOSQ_ERR_INVALID_ARG;
    std::vector<int32_t> h(static_cast<size_t>(num_blocks));
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (num_blocks > 0) {
        if (record_cuda(ctx, cudaMemcpyAsync(h.data(), status, sizeof(int32_t) * h.size(), cudaMemcpyDeviceToHost, s), "status copy"))
            return EOSQ_ERR_CUDA;
    }
    int dev_err = 0;
    if (record_cuda(ctx, cudaMemcpyAsync(&dev_err, ctx->dev_err, sizeof(int), cudaMemcpyDeviceToHost, s), "error word copy"))
        return EOSQ_ERR_CUDA;
    if (record_cuda(ctx, cudaStreamSynchronize(s), "cudaStreamSynchronize")) return EOSQ_ERR_CUDA;
    if (dev_err != 0) {
        ctx->last_error = "a bounded device-side wait gave up (kernel bits " + std::to_string(dev_err) + "); results are incomplete";
        // reported once: the word is cleared so that the context can be used again
        if (record_cuda(ctx, cudaMemsetAsync(ctx->dev_err, 0, sizeof(int), s), "error word reset") ||
            record_cuda(ctx, cudaStreamSynchronize(s), "cudaStreamSynchronize"))
            return EOSQ_ERR_CUDA;
        ctx->last_error = "a bounded device-side wait gave up (kernel bits " + std::to_string(dev_err) + "); results are incomplete";
        return EOSQ_ERR_CUDA;
    }
    int64_t cnt = 0;
    for (int32_t v : h) cnt += (v != 0);
    if (flagged) *flagged = cnt;
    return cnt ? EOSQ_WARN_BLOCK_STATUS : EOSQ_OK;
}

extern "C" int eosq_selftest_wait_timeout(eosq_ctx *ctx, uint32_t polls, void *cuda_stream) {
    if (!ctx || polls == 0 || polls > 4096 || !on_ctx_device(ctx)) return EOSQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    launch_wait_timeout(ctx->dev_err, polls, s);
    ctx->launches += 1;
    return record_cuda(ctx, cudaGetLastError(), "eosq_selftest_wait_timeout launch") ? EOSQ_ERR_CUDA : EOSQ_OK;
}
