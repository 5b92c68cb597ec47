/*
 * eosq -- eOptShrinkQ KV-cache block compression on NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  Every entry point returns an eosq_status code, never throws and never
 * aborts.  "dev" pointers are device memory of the current CUDA device, "host" pointers are
 * ordinary host memory.  The caller owns every buffer it passes in; the library owns only the
 * immutable per-(d, seed, bits) constants it caches inside an eosq_ctx (rotation, codebook).
 * Unless stated otherwise a call only enqueues work on the given stream and does not
 * synchronise it.
 *
 * Notation follows the paper: a block S (n tokens x d channels), eigenvalues lambda_i = sigma_i^2
 * of S^T S in descending order, pilot k = floor(d^c), estimated rank r, shrunk values phi_i,
 * rotation Pi, b bits per residual coordinate.
 */
#ifndef EOSQ_H
#define EOSQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EOSQ_OK = 0,
    EOSQ_ERR_INVALID_ARG = 1,      /* null pointer, negative size, misaligned buffer */
    EOSQ_ERR_UNSUPPORTED = 2,      /* d != 128, bits outside 1..4, n < d, n > 4096, n % 8 != 0 */
    EOSQ_ERR_BUFFER_TOO_SMALL = 3, /* workspace smaller than eosq_workspace_bytes() */
    EOSQ_ERR_CUDA = 4,             /* a CUDA runtime call failed; see eosq_last_cuda_error() */
    EOSQ_WARN_BLOCK_STATUS = 5     /* only from eosq_check_status: some block raised a flag */
} eosq_status;

/* Input / output element types. */
enum { EOSQ_F16 = 0, EOSQ_F32 = 1 };

/* Capacity of the per-block factor arrays.  The rank test of Algorithm 2 cannot return more than
 * the pilot k (= 11 at d = 128) outliers, because its bulk-edge estimate is at least lambda_{k+1}. */
#define EOSQ_RMAX 16

/* Per-block status bits written by eosq_encode into eosq_cache_t.status. */
#define EOSQ_BLOCK_NOT_CONVERGED 1u /* eigenvalue or eigenvector iteration hit its cap */
#define EOSQ_BLOCK_CLAMPED 2u       /* a shrunk value was clamped into [0, sigma_i] */
#define EOSQ_BLOCK_NONFINITE 4u     /* non-finite input or spectrum */
#define EOSQ_BLOCK_CLUSTERED 8u     /* two kept eigenvalues closer than 1e-9 relative */

typedef struct eosq_ctx eosq_ctx;

/*
 * Compressed cache: what Algorithm 3's "Store" line keeps, as structure-of-arrays over B blocks.
 * All pointers are dev.  eig, lambda_plus, vr32 and coef may be null (then they are not written).
 */
typedef struct {
    uint8_t *codes;     /* [B][n][d*bits/8]  row bit string, coordinate j at bits [j*b,(j+1)*b), little endian */
    uint16_t *norms;    /* [B][n]            fp16 row norms rho_t of the residual (Algorithm 1)      */
    int32_t *rank;      /* [B]               estimated rank r (Algorithm 2, Step 1)                   */
    float *sigma;       /* [B][EOSQ_RMAX]    kept singular values sigma_i, entries >= r are 0         */
    float *phi;         /* [B][EOSQ_RMAX]    shrunk values phi_i (Eq. 6, Frobenius), entries >= r are 0 */
    uint16_t *P;        /* [B][EOSQ_RMAX][n] fp16 left factors phi_i xi_i; rows >= r are NOT written  */
    uint16_t *V;        /* [B][EOSQ_RMAX][d] fp16 right vectors zeta_i; rows >= r are zero            */
    int32_t *status;    /* [B]               EOSQ_BLOCK_* bits                                       */
    float *eig;         /* [B][d]            all eigenvalues lambda_i, descending (optional)          */
    float *lambda_plus; /* [B]               bulk-edge estimate (Algorithm 2, Step 1) (optional)      */
    float *vr32;        /* [B][EOSQ_RMAX][d] unrounded right vectors used for the residual (optional) */
    float *coef;        /* [B][EOSQ_RMAX]    phi_i / sigma_i as used for the residual (optional)      */
} eosq_cache_t;

/* Byte sizes per block of each array above, and derived constants. */
typedef struct {
    int32_t k;          /* pilot parameter floor(d^c) */
    int32_t rmax;       /* EOSQ_RMAX */
    int32_t row_bytes;  /* d*bits/8 */
    int32_t reserved;
    int64_t codes_bytes, norms_bytes, P_bytes, V_bytes, sigma_bytes, phi_bytes, eig_bytes;
    int64_t stored_bytes; /* codes + norms + rank*(n+d)*2 at rank = rmax + sigma (upper bound per block) */
} eosq_layout_t;

/* ---- host-side pure functions ------------------------------------------------------------ */

/* Pilot parameter k = floor(d^c), c = min(1/2.01, 1/log log d) (Algorithm 2, REQUIRE line and
 * Step 1).  Returns k, or -1 if d < 3. */
int eosq_pilot_k(int d);

/* Lloyd-Max codebook for the N(0, 1/d) marginal of a rotated unit vector (Algorithm 1, REQUIRE
 * line; Sec. 2.2 item 3).  centroids: host, 2^bits doubles, ascending.  thresholds: host,
 * 2^bits - 1 midpoints (may be null).  Errors: bits outside 1..8 or d < 1 -> INVALID_ARG. */
int eosq_codebook(int bits, int d, double *centroids, double *thresholds);

/* Seeded Haar rotation Pi (Algorithm 1, "shared Haar rotation"): the orthogonal factor, with
 * positive-diagonal R, of the d x d Gaussian matrix whose entry e = i*d + j is Box-Muller
 * sqrt(-2 ln u1) cos(2 pi u2) of u = ((SplitMix64(seed + (c+1)*0x9E3779B97F4A7C15) >> 11) + 0.5) 2^-53
 * at counters c = 2e, 2e+1.  Pi: host, d*d doubles, row-major, z = Pi u. */
int eosq_rotation(int d, uint64_t seed, double *Pi);

/* Sizes of the compressed arrays for one block (Algorithm 3, "Store" and "Bits per entry"). */
int eosq_layout(int n, int d, int bits, eosq_layout_t *out);

/* Bits per entry of Algorithm 3: bits + rank*(n+d)*b_s/(n*d), +1 with the QJL bit. */
double eosq_bits_per_entry(int bits, double rank, int n, int d, double b_s, int prod);

/* Scratch bytes eosq_encode needs for num_blocks blocks (it processes them in chunks, so this
 * saturates; 256-byte aligned dev memory). */
size_t eosq_workspace_bytes(int64_t num_blocks, int n, int d);

/* ---- context ----------------------------------------------------------------------------- */

/* Create / destroy a context on the current device.  The context lazily builds and caches, per
 * (d, seed) and (d, bits), the device copies of Pi and of the codebook; building one performs a
 * synchronous host-to-device copy on first use.  Not thread safe.  Every device entry point below
 * returns EOSQ_ERR_INVALID_ARG when the current CUDA device is not the context's. */
int eosq_create(eosq_ctx **out);
int eosq_destroy(eosq_ctx *ctx);

/* Text of the last CUDA error seen by this context (host pointer owned by the context). */
const char *eosq_last_cuda_error(const eosq_ctx *ctx);

/* ---- device entry points ----------------------------------------------------------------- */

/*
 * Compress num_blocks independent blocks (Algorithm 3): Gram matrix and its eigen-decomposition
 * (the block's singular values and right vectors, Sec. 2.3), bulk edge, rank and shrinkage
 * (Algorithm 2, Eq. 7-9, Eq. 6 Frobenius), residual R = S - sum phi_i xi_i zeta_i^T, then per row
 * norm, rotation, Lloyd-Max code and bit packing (Algorithm 1).
 *   blocks     dev [num_blocks][n][d], in_dtype EOSQ_F16 or EOSQ_F32, row-major, 16-byte aligned
 *   out        arrays as described at eosq_cache_t, sized for num_blocks
 *   workspace  dev scratch of at least eosq_workspace_bytes(num_blocks, n, d)
 * num_blocks = 0 is a no-op.  Errors: see eosq_status.  Block-level trouble never fails the
 * call; it is reported in out->status.
 */
int eosq_encode(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t num_blocks, int n, int d,
                int bits, uint64_t seed, const eosq_cache_t *out, void *workspace,
                size_t workspace_bytes, void *cuda_stream);

/*
 * eosq_encode without any device allocation.  (The paper has no counterpart: this entry point
 * exists for the sake of callers, not of the method.)
 *
 * Who needs it: code that must not call cudaMalloc where it compresses -- a serving loop whose
 * device memory was divided up at start-up, a plug-in that was given buffers but no allocator, a
 * caller that has begun capturing a stream.  eosq_encode makes such callers bring a workspace and
 * allocates the device copy of the rotation on the first use of a seed; this variant does
 * neither.  Its scratch and its copy of the rotation live in one fixed array in the library's
 * device image (about 4.7 MB, held by every GPU that loads the library until the process exits).
 * The call itself performs no cudaMalloc, no cudaFree and no allocating library call.
 *
 * Arguments and results are those of eosq_encode (same kernels, same outputs) minus the
 * workspace.  Limits and rules:
 *   - num_blocks <= EOSQ_STATIC_MAX_BLOCKS; a larger count is rejected with
 *     EOSQ_ERR_BUFFER_TOO_SMALL (text in eosq_last_cuda_error) and nothing is enqueued.
 *   - The first call on a device looks up the array's device address (that device must be
 *     current and must be the context's device, as for every call), the first call with a new seed
 *     uploads that seed's rotation from host memory on the given stream, and the first call with a
 *     new (in_dtype, bits) pair on a device loads those kernels and sets their shared-memory
 *     limits.  Make those calls before any stream capture, and keep per-stage profiling off
 *     (eosq_profile_enable creates events on first use).
 *   - All calls on a device share the one array, and it keeps whatever the last call left.  The
 *     kernels write every scratch value before reading it, so nothing needs clearing, but two
 *     calls that overlap on the GPU (different streams, no ordering between them) race; order
 *     them on one stream or with events.  Calls are serialised on the host by a lock.
 */
#define EOSQ_STATIC_MAX_BLOCKS 32
int64_t eosq_encode_static_max_blocks(void);
int eosq_encode_static(eosq_ctx *ctx, const void *blocks, int in_dtype, int64_t num_blocks, int n, int d,
                       int bits, uint64_t seed, const eosq_cache_t *out, void *cuda_stream);

/*
 * Reconstruct blocks from a compressed cache (Algorithm 1 last TQ_MSE line, Algorithm 2 Return):
 *   x_hat[t] = sum_{i<r} P[i][t] V[i][:] + norms[t] * Pi^T centroids[codes[t]].
 *   out_blocks dev [num_blocks][n][d] of out_dtype (EOSQ_F16 or EOSQ_F32).
 * codes, norms, P and out_blocks must be 16-byte aligned (EOSQ_ERR_INVALID_ARG otherwise: the
 * kernel moves them with bulk copies and tensor stores).  It (and the score kernel) reads at most
 * 12 factor rows per block (eosq_encode stores at most the pilot k = 11), so a cache written
 * elsewhere with a larger rank word is truncated to 12.
 */
int eosq_decode(eosq_ctx *ctx, const eosq_cache_t *cache, int64_t num_blocks, int n, int d, int bits,
                uint64_t seed, void *out_blocks, int out_dtype, void *cuda_stream);

/*
 * Attention logits straight from the compressed keys (Remark 6.4; scores <q,k>/sqrt(d), Sec. 1):
 *   scores[h][g][t] = scale * ( <q V_r^T, P[:, t]> + norms[t] * <Pi q, centroids[codes[t]]> )
 * for every KV head h, each of its G query vectors g and every cached token t = j*n + row of its
 * blocks_per_head blocks.  Block j of head h is block h*head_stride_blocks + j of `kcache`
 * (head_stride_blocks = blocks_per_head for a keys-only cache, 2*blocks_per_head for a cache laid
 * out [head][K|V][block]).
 *   q       dev [num_kv_heads][G][d] fp16
 *   scores  dev [num_kv_heads][G][blocks_per_head*n] fp32
 * codes, norms, P and V of `kcache` must be 16-byte aligned (EOSQ_ERR_INVALID_ARG otherwise).
 * The tensor-core path keeps the rotated queries in a device buffer of 4 KB per KV head that the
 * context owns: the first call (and a later call with more heads) allocates it, which synchronises
 * the device; calls on one context must not overlap in time.
 */
int eosq_scores(eosq_ctx *ctx, const eosq_cache_t *kcache, int64_t num_kv_heads,
                int64_t blocks_per_head, int64_t head_stride_blocks, int n, int d, int bits,
                uint64_t seed, const void *q, int G, float scale, float *scores, void *cuda_stream);

/*
 * Host-buffer convenience for end-to-end use: copies `blocks` (host, pinned preferred) to the
 * device in chunks, encodes, and copies codes, norms, rank, sigma, phi, P, V and status back into
 * the host arrays of `host_out` (optional members may be null).  `arena` is dev scratch of at least
 * eosq_encode_host_arena_bytes(): two slots of one chunk's input and outputs plus one workspace.
 * Uploads and downloads run on two streams the context owns, the kernels on `cuda_stream`, so that
 * with pinned host memory the three overlap; work already queued on `cuda_stream` is waited for
 * first.  Synchronises all three streams before returning.
 */
size_t eosq_encode_host_arena_bytes(int64_t num_blocks, int n, int d, int bits, int in_dtype);
int eosq_encode_host(eosq_ctx *ctx, const void *host_blocks, int in_dtype, int64_t num_blocks, int n,
                     int d, int bits, uint64_t seed, const eosq_cache_t *host_out, void *arena,
                     size_t arena_bytes, void *cuda_stream);

/* Synchronises the stream and returns EOSQ_WARN_BLOCK_STATUS if any of the num_blocks status
 * words (dev) is non-zero, EOSQ_OK otherwise; *flagged (host, may be null) gets the count.
 * If a kernel launched through the context has given up a bounded device-side wait since the last
 * call (its outputs are then incomplete), returns EOSQ_ERR_CUDA instead, with the kernels' bits in
 * eosq_last_cuda_error() (1 Gram, 2 quantise, 8 scores, 16 decode, 32 self-test), and clears that
 * record: it is reported once and the context stays usable. */
int eosq_check_status(eosq_ctx *ctx, const int32_t *status, int64_t num_blocks, int64_t *flagged,
                      void *cuda_stream);

/* Launches a one-CTA kernel that waits on a barrier nothing arrives at, for at most `polls`
 * (1..4096) polls of about 2 us, gives up and records that like any pipeline kernel of the library
 * would: the next eosq_check_status returns EOSQ_ERR_CUDA (bit 32).  No output, no effect on cache
 * data; it exists so that the time-out path can be exercised without a kernel that hangs or faults.
 * EOSQ_ERR_INVALID_ARG for polls outside the range. */
int eosq_selftest_wait_timeout(eosq_ctx *ctx, uint32_t polls, void *cuda_stream);

/* Number of kernels the library has launched through this context so far (for bookkeeping). */
int64_t eosq_launch_count(const eosq_ctx *ctx);

/*
 * Per-stage device timing for benchmarks.  While enabled, every kernel launch is bracketed by
 * CUDA events on the launching stream.  eosq_profile_read synchronises those events, adds their
 * elapsed milliseconds into ms[EOSQ_NUM_STAGES] and their launch counts into
 * launches[EOSQ_NUM_STAGES] (host arrays, overwritten), and clears the record.
 * Stage order: Gram, tridiagonalisation steps 0-63, 64-95 and 96-125 (three kernels), eigenvalues,
 * spectrum + shrinkage + eigenvectors, residual/rotate/quantise/pack, decode, scores, the second
 * pass over blocks whose tensor-core Gram matrix was not accurate enough (all its kernels), other.
 */
#define EOSQ_NUM_STAGES 11
int eosq_profile_enable(eosq_ctx *ctx, int on);
/* Times only the stages whose bit (1 << stage index, in the order above) is set in stage_mask; the
 * two events per launch cost about 2 us of device time each, which adds up over the several hundred
 * launches of a large encode, so a benchmark that wants one kernel's duration inside its timed
 * region selects that stage alone.  EOSQ_ERR_INVALID_ARG for bits beyond EOSQ_NUM_STAGES. */
int eosq_profile_select(eosq_ctx *ctx, uint32_t stage_mask);
int eosq_profile_read(eosq_ctx *ctx, float *ms, int64_t *launches);

#ifdef __cplusplus
}
#endif
#endif /* EOSQ_H */
