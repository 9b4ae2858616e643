/*
 * tng.h -- C ABI of libtng: the data-parallel hot path of Trajectory Normalized
 * Gradients (TNG, arXiv 1901.08227) on one NVIDIA B200 (sm_100a).
 *
 * One round (Algorithm 1 of the paper, with Eq. 2 / Eq. 3 of Section 3):
 *   fuse the ring of past aggregated vectors into a shared reference r
 *   -> normalise every worker's gradient against r (g - r, or g ./ r)
 *   -> compress it (stochastic sign / ternary / s-level quantiser, per-block scale)
 *   -> [the packed codes + scales are the "wire"]
 *   -> decode all M workers, average, add (or multiply) the reference back
 *   -> push the result into the ring.
 * M workers are simulated as a batch: worker m's gradient is row m of `grads`.
 *
 * Conventions
 *   - `*_dev` pointers are CUDA device pointers, `*_host` pointers host memory.
 *     Device vectors must be 16-byte aligned; a row stride `ld` (in floats) must
 *     be a multiple of 4 and >= d.  Violations return TNG_ERR_INVALID_ARG.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     only enqueue work unless stated otherwise.
 *   - The caller owns every buffer it passes.  The library owns the tng_ctx and,
 *     unless a workspace is bound, one device allocation it frees in tng_destroy.
 *   - No call aborts or throws; every failure is a tng_status.  There is no CPU
 *     fallback: without a CUDA device the calls that touch the GPU return TNG_ERR_CUDA.
 *   - A context is not thread-safe; use it from one host thread at a time and with one
 *     stream at a time.
 */
#ifndef TNG_H
#define TNG_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tng_ctx tng_ctx;

typedef enum {
    TNG_OK = 0,
    TNG_ERR_INVALID_ARG = 1, /* bad size, enum, alignment, NULL pointer */
    TNG_ERR_STATE = 2,       /* call not allowed now (options after the first round, ...) */
    TNG_ERR_ALLOC = 3,       /* device or host allocation failed / workspace too small */
    TNG_ERR_CUDA = 4,        /* a CUDA call or launch failed; tng_last_cuda_error() has the code */
    TNG_ERR_NONFINITE = 5,   /* a NaN/Inf block scale was produced in an earlier round */
    TNG_ERR_UNSUPPORTED = 6
} tng_status;

/* value = bits per coordinate symbol */
typedef enum { TNG_CODEC_SIGN1 = 1, TNG_CODEC_TERN2 = 2, TNG_CODEC_QSGD4 = 4 } tng_codec;
/* NONE: v = g.  DIFF: Eq. 2.  QUOT: Eq. 3.  COMB: the combined form of Section 3,
 * r = Q[(g - ref) ./ ref'], v = ref' . r + ref, with ref' = the mean absolute value of the
 * stored aggregates (per coordinate), guarded like the quotient form's denominator.
 * MEAN: the scalar reference of Section 3.1, ref^m = mean(g^m) ones(D): v = g^m - mean(g^m),
 * every worker sends its scalar along with codes and scales (tng_wire_means), decoding adds
 * the average of the M scalars back.  mean(g) is the fp32 adjacent-pairwise tree sum of the
 * d elements divided by d.  No trajectory is used: the fusion stage is skipped (the ring
 * still receives every aggregate). */
typedef enum { TNG_NORM_NONE = 0, TNG_NORM_DIFF = 1, TNG_NORM_QUOT = 2, TNG_NORM_COMB = 3, TNG_NORM_MEAN = 4 } tng_norm_mode;
typedef enum {
    TNG_FUSE_AUTO = 0,     /* K == 1 -> LAST, else LSQ */
    TNG_FUSE_LAST = 1,     /* r = newest aggregate (delayed gradient, Sec. 3.1 / Sec. 4.2 protocol) */
    TNG_FUSE_MEAN = 2,     /* r = window average of the k stored aggregates (Sec. 3.1) */
    TNG_FUSE_LSQ = 3,      /* r = sum_j alpha_j h_j minimising sum_m ||g^m - r||^2 (C_nz of Prop. 2) */
    TNG_FUSE_HINDSIGHT = 4 /* alpha from the history alone: regress h_1 on h_2..h_k, shift by one */
} tng_fuse_mode;

typedef enum {
    TNG_OPT_BLOCK = 0,       /* coordinates per scale; 0 = one scale per vector (the paper's R);
                                otherwise a multiple of 128.  Default 128.  Cost: 128, 256, 512, 1024 and 2048
                                are encoded in one read of the gradient rows; any other value (0 included)
                                needs the scale before the first symbol, i.e. two reads, except for short
                                problems (tiles x workers <= 16384), which are one launch either way. */
    TNG_OPT_QSGD_LEVELS = 1, /* s in 1..7 (TNG_CODEC_QSGD4 only).  Default 7. */
    TNG_OPT_SCALE_KIND = 2,  /* 0 = max|v| (Sec. 3.2), 1 = L2 norm of the block.  Default 0. */
    TNG_OPT_SEED_LO = 3,     /* low / high 32 bits of the Philox key.  Default 0. */
    TNG_OPT_SEED_HI = 4,
    TNG_OPT_FUSE_MODE = 5,   /* a tng_fuse_mode.  Default TNG_FUSE_AUTO. */
    TNG_OPT_RIDGE = 6,       /* relative ridge of the K x K solve.  Default 1e-6. */
    TNG_OPT_QUOT_EPS = 7,    /* floor of |r| relative to its tile maximum, quotient form.  Default 2^-4. */
    TNG_OPT_TIMING = 8,      /* 1 = record CUDA events around every stage of tng_step.  Default 0. */
    TNG_OPT_HOST_STAGING = 9,/* 1 = reserve device staging so tng_step_host can be used.  Default 0. */
    TNG_OPT_REF_EVERY = 10,  /* refresh cadence of the reference (Sec. 3.1, last paragraph; Sec. 4.1 refreshes
                                every 16 iterations): tng_step fuses a new reference in rounds t with
                                t % value == 0 and reuses the previous one in between; the ring still
                                receives every aggregate.  1..65536, default 1. */
    TNG_OPT_COORD_OFFSET = 11 /* the context holds coordinates [offset, offset + d) of a longer vector (one
                                slice per GPU): only the Philox counters see the offset, so that the slices
                                code exactly what one context over the whole vector would.  A multiple of 128
                                and of the scale block; not with one scale per vector nor TNG_NORM_MEAN, which
                                need the whole vector.  Default 0. */
} tng_option;

#define TNG_MAX_WORKERS 64
#define TNG_MAX_HISTORY 16
#define TNG_MAX_COORDS (1ull << 31) /* d; a row stride must stay below 2^32 floats */
#define TNG_TILE 128 /* coordinates per wire tile */

/* Plain-old-data snapshot filled by tng_stats. */
typedef struct {
    uint64_t d;
    uint32_t M, K;
    uint32_t k;              /* history vectors currently stored */
    uint32_t fuse_mode;      /* effective mode (never AUTO) */
    uint64_t rounds;         /* completed rounds (the Philox step counter) */
    double bits_per_coord;   /* b + 32/B + 64 K/d */
    double alpha[TNG_MAX_HISTORY];                     /* coefficients of the last fusion */
    double gram[TNG_MAX_HISTORY * TNG_MAX_HISTORY];    /* G[a][b] at gram[a * TNG_MAX_HISTORY + b], a, b < k: the
                                                          row stride is always 16, whatever k (LSQ / HINDSIGHT) */
    double rhs[TNG_MAX_HISTORY];                       /* <h_i, mean gradient> */
    double grad_sq;          /* (1/M) sum_m ||g^m||^2 of the last fusion */
    double cnz;              /* estimate of C_nz = sum_m||g^m - r||^2 / sum_m||g^m||^2; NaN if unknown */
    uint32_t solver_fallback;   /* 1 = last solve hit a bad pivot and used alpha = e_1 */
    uint32_t pipeline_error;    /* nonzero: a bounded wait inside a staged kernel gave up (results invalid) */
    uint64_t nonfinite_scales;  /* block scales that were NaN/Inf since creation */
    uint64_t kernel_launches;   /* kernels launched by this context since creation */
    /* mean milliseconds per round of each stage over the rounds timed so far
       (TNG_OPT_TIMING = 1), and how many rounds that is */
    uint64_t timed_rounds;
    double ms_dots, ms_solve, ms_combine, ms_encode, ms_decode;
} tng_stats_t;

/* ---- lifetime --------------------------------------------------------------- */
/* 1 <= d <= TNG_MAX_COORDS coordinates, 1 <= M <= 64 workers, ring depth 1 <= K <= 16.  Host only. */
tng_status tng_create(tng_ctx** out, uint64_t d, uint32_t M, uint32_t K, tng_codec codec,
                      tng_norm_mode norm);
/* Waits for the context's last stream, frees what the library allocated.  NULL is allowed. */
void tng_destroy(tng_ctx* ctx);
/* Options can change until the workspace is sized (tng_workspace_bytes, tng_bind_workspace
 * or the first call that touches the device); later: TNG_ERR_STATE. */
tng_status tng_set_option(tng_ctx* ctx, tng_option key, double value);
/* Device bytes the context needs (ring K*d, reference, codes, scales, reduction scratch). */
tng_status tng_workspace_bytes(tng_ctx* ctx, size_t* bytes);
/* Use caller-owned device memory (256-byte aligned, >= tng_workspace_bytes) instead of an
 * internal cudaMalloc.  Must come before the first device call.  Only the small state block
 * (statistics, flags, counters) is cleared, on `stream` of the first device call; the ring, the
 * wire and the scratch areas are left as found and are written before they are read. */
tng_status tng_bind_workspace(tng_ctx* ctx, void* dev_ptr, size_t bytes);

/* ---- the round ------------------------------------------------------------- */
/* Seed the ring with a vector (the start-up of Sec. 4.2, where the first reference is a gradient
 * computed in full rather than zeros). */
tng_status tng_push_reference(tng_ctx* ctx, const float* vec_dev, void* stream);
/* One round of Algorithm 1 on M gradient rows (row m at grads_dev + m*ld, device memory):
 * fusion of the reference from the ring (Sec. 3.1, criterion of Prop. 2), r(w_t) = Q[normalised
 * gradient] (Eq. 2 / Eq. 3 / the combined form, coding of Sec. 3.2), v_t = the average of the
 * decoded codes with the reference put back, ring <- v_t.  Writes v_t (d floats) to agg_out_dev
 * if it is not NULL (device memory, caller-owned); v_t is always stored as the newest ring entry
 * (tng_history(ctx, 0, ...)).  Errors: TNG_ERR_INVALID_ARG (NULL, misaligned, bad ld),
 * TNG_ERR_ALLOC (workspace), TNG_ERR_CUDA (launch failure). */
tng_status tng_step(tng_ctx* ctx, const float* grads_dev, uint64_t ld, float* agg_out_dev,
                    void* stream);
/* Same round for host buffers: copies the M rows to device staging, runs the round, copies the
 * aggregate back, all on `stream`; returns after the stream has finished.  Needs
 * TNG_OPT_HOST_STAGING = 1.  Pinned host memory makes the copies asynchronous and fast. */
tng_status tng_step_host(tng_ctx* ctx, const float* grads_host, uint64_t ld, float* agg_out_host,
                         void* stream);
/* The same without waiting: the copy of the aggregate to agg_out_host runs on a stream of the
 * library's own, so that in a sequence of calls it overlaps the next call's copy of the rows to the
 * device (the link carries both directions at once).  grads_host may be reused once the call has
 * returned and `stream` has passed its copy (tng_host_wait also guarantees that for every earlier
 * call); agg_out_host holds the aggregate only after tng_host_wait.  Pinned host memory is needed
 * for any overlap. */
tng_status tng_step_host_async(tng_ctx* ctx, const float* grads_host, uint64_t ld, float* agg_out_host,
                               void* stream);
/* Blocks until every copy started by tng_step_host_async has finished. */
tng_status tng_host_wait(tng_ctx* ctx);

/* ---- state save / resume ----------------------------------------------------- */
/* The state a context carries between rounds is the ring, the round counter and (with a refresh
 * cadence above 1) the held reference; the codes of round t depend on nothing else, so a context
 * that loads a saved state continues bit for bit.  The blob lives in HOST memory.
 * tng_state_bytes: upper bound of the blob for this context.
 * tng_save_state:  waits for `stream`, writes the blob to host_buf (capacity `bytes`), returns the
 *                  bytes used in *written (may be NULL).  TNG_ERR_ALLOC if the buffer is too small.
 * tng_load_state:  the context must have been created with the same d, M, K, codec, normalisation
 *                  and options (else TNG_ERR_INVALID_ARG); replaces ring, counter and reference;
 *                  returns after the copies have finished. */
tng_status tng_state_bytes(tng_ctx* ctx, size_t* bytes);
tng_status tng_save_state(tng_ctx* ctx, void* host_buf, size_t bytes, size_t* written, void* stream);
tng_status tng_load_state(tng_ctx* ctx, const void* host_buf, size_t bytes, void* stream);

/* ---- stage-level entry points (the kernels tng_step launches; tng_step itself folds the
 * reference combine into the encode pass when there is one scale per 128 coordinates) ---------- */
/* Fusion (Sec. 3.1 pool, criterion C_nz of Prop. 2): statistics G = <h_i,h_j>, c = <h_i, mean g>,
 * solve (G + ridge tr(G)/k I) alpha = c, combine r = sum_j alpha_j h_j (fp32 fma chain, newest
 * first) -> the context's reference (tng_reference); alpha, G, c and C_nz through tng_stats.
 * Ignores the refresh cadence.  grads_dev / ld as in tng_step. */
tng_status tng_fuse(tng_ctx* ctx, const float* grads_dev, uint64_t ld, void* stream);
/* Encode (Eq. 2 / Eq. 3 normalisation; Sec. 3.2: R = max|v|, P(nonzero) = |v|/R; Algorithm 1
 * "compute R, sample z, transmit"): normalise against ref_dev (d floats, device; NULL = the
 * context's reference), one scale per block, stochastic rounding, bit packing -> the wire
 * (tng_wire).  `step` is the Philox step counter (tng_step passes the round number).  With
 * TNG_NORM_COMB the second reference is always the context's own (from the last fusion).  With
 * TNG_NORM_MEAN ref_dev is ignored: the workers' means are computed first (tng_wire_means). */
tng_status tng_encode(tng_ctx* ctx, const float* grads_dev, uint64_t ld, const float* ref_dev,
                      uint32_t step, void* stream);
/* Decode + aggregate (Algorithm 1 "the main server averages", with Eq. 2 / Eq. 3's v = ref + r /
 * ref . r): unpack the M code streams of the wire, v^m = R^m * symbol, a = (sum_m v^m) / M in
 * fp32 (m ascending), de-normalise against ref_dev (NULL = context's; ignored with TNG_NORM_MEAN,
 * which adds the average of the wire's M scalars instead).  Writes out_dev (d floats, device);
 * does not touch the ring. */
tng_status tng_decode_aggregate(tng_ctx* ctx, const float* ref_dev, float* out_dev, void* stream);

/* ---- the same round with the workers on different GPUs ------------------------------- */
/* Algorithm 1 as the paper states it: every server codes its own gradient, the codes are
 * exchanged, every server decodes the same average.  Here each process (one per GPU) holds a
 * context of the SAME (d, M, K, codec, options, seed) and the gradient rows of its own workers
 * m_first .. m_first + m_count - 1; ring, reference and round counter evolve identically on all
 * of them.  The library does the rank-local work; the two exchanges are the caller's (NCCL):
 *   tng_fuse_local      statistics of the local rows: Gram of the ring (the same on every rank)
 *                       and the local SUMS sum_m <h_i, g^m>, sum_m ||g^m||^2
 *   [all-reduce (sum) of the tng_local_stats block: 17 doubles on the device]
 *   tng_fuse_finish     divide by M, solve -> the coefficients of the reference (Sec. 3.1 / Prop. 2); the
 *                       combine itself is done by the pass of the next tng_encode_local, which reads the
 *                       ring anyway (or, should another call need the reference first, by that call)
 *   tng_encode_local    code the local rows as workers m_first.. into THEIR slots of the wire
 *   [all-gather of the wire: every rank's slots of codes and scales (tng_wire)]
 *   tng_decode_commit   decode all M workers, average, put the reference back, push into the
 *                       ring, advance the round counter (the second half of tng_step)
 * With all M rows on one rank this sequence equals tng_step except that the statistics are
 * summed in another order (the reference agrees to rounding of the K coefficients) and that the
 * refresh cadence option is not applied.  The stochastic rounding of worker m depends only on
 * (seed, m, round, coordinate), so the wire does not depend on how workers are spread. */
tng_status tng_fuse_local(tng_ctx* ctx, const float* grads_dev, uint64_t ld, uint32_t m_count, void* stream);
/* Borrowed device pointer to the block to all-reduce (rhs[16], grad_sq) and its length. */
tng_status tng_local_stats(tng_ctx* ctx, double** sums_dev, size_t* count);
/* The other way to spread one round over GPUs: every process holds ALL M workers but only the
 * coordinates [offset, offset + d) of every vector (TNG_OPT_COORD_OFFSET), ring and wire included.
 * Encoding and decoding are local to a slice; the only coupling is the fusion statistics, which
 * are sums over coordinates:
 *   tng_fuse_local      Gram, rhs sums and grad_sq over the local coordinates
 *   [all-reduce (sum) of the tng_local_stats_all block: 273 doubles on the device]
 *   tng_fuse_finish     divide by M, solve, combine -> the slice of the reference
 *   tng_encode_local    (m_first = 0, m_count = M), tng_decode_commit: no exchange of the wire
 * Borrowed device pointer to G (16 x 16, row-major), c (16), grad_sq (1), contiguous. */
tng_status tng_local_stats_all(tng_ctx* ctx, double** sums_dev, size_t* count);
tng_status tng_fuse_finish(tng_ctx* ctx, void* stream);
/* step: the Philox step counter; pass the round number (tng_stats' rounds). */
tng_status tng_encode_local(tng_ctx* ctx, const float* grads_dev, uint64_t ld, uint32_t m_first, uint32_t m_count,
                            uint32_t step, void* stream);
/* agg_out_dev may be NULL (the aggregate is the newest ring entry either way). */
tng_status tng_decode_commit(tng_ctx* ctx, float* agg_out_dev, void* stream);

/* ---- borrowed views (valid until the next call that changes them) ---------- */
/* Wire: codes[m] at codes_dev + m*words_per_worker (uint32), scales[m] at scales_dev +
 * m*scales_per_worker.  Tile T = coordinates [128T,128T+128) owns 4b words; word c*b+p, bit j,
 * is bit p of the symbol of coordinate 128T + 4j + c. */
tng_status tng_wire(tng_ctx* ctx, const uint32_t** codes_dev, size_t* words_per_worker,
                    const float** scales_dev, size_t* scales_per_worker);
/* TNG_NORM_MEAN: the M scalars mean(g^m) of the last encode (device, M floats; part of the
 * wire: with the workers on different GPUs they are gathered like the scales). */
tng_status tng_wire_means(tng_ctx* ctx, const float** means_dev);
tng_status tng_reference(tng_ctx* ctx, const float** ref_dev);
/* h_{j+1}: j = 0 is the newest stored aggregate; j < k. */
tng_status tng_history(tng_ctx* ctx, uint32_t j, const float** vec_dev);

/* ---- self-test of the bounded waits ------------------------------------------------ */
/* The staged kernels wait on shared-memory barriers with a poll limit; when a wait runs out the
 * kernel records it, returns, and tng_stats reports TNG_ERR_CUDA with pipeline_error set.  This
 * call exercises exactly that path without disturbing the context: a one-block kernel waits
 * (same wait routine, limit of 1024 polls) on a barrier that nothing ever completes and writes
 * what happened to a scratch word of the workspace.  *gave_up_host = 1 when the wait ended by
 * its limit, as it must.  Synchronises the stream.  The context stays usable. */
tng_status tng_selftest_bounded_wait(tng_ctx* ctx, uint32_t* gave_up_host, void* stream);

/* ---- fusion statistics without any allocation ------------------------------- */
/* (No counterpart in the paper: this is a packaging of the statistics pass of tng_fuse.)
 * For callers that cannot allocate device memory -- a process whose device memory is
 * owned by its own pool, a steady-state loop that must stay away from cudaMalloc (it
 * synchronises the device and may fail), a plug-in that only receives pointers -- this
 * computes, for k history vectors and M gradient rows,
 *   out[0 .. k*k)      G[a][b] = <h_a, h_b>            (row-major, both triangles)
 *   out[k*k .. k*k+k)  c[a]    = <h_a, mean_m g^m>
 *   out[k*k+k]         (1/M) sum_m ||g^m||^2
 * (doubles) with the same kernel tng_fuse uses.  The per-CTA partial sums and the arrival
 * counter that kernel needs live in a fixed array inside the library image
 * (TNG_STATIC_SCRATCH_BYTES per GPU that loads the library, held until the process
 * exits), so the call performs no cudaMalloc/cudaFree and uses no allocating routine.
 * rows_dev is a HOST array of k device pointers (16-byte aligned vectors of d floats);
 * grads_dev/ld as in tng_step; out_dev: k*k+k+1 doubles, caller-owned device memory.
 * Limits: 1 <= k <= TNG_STATIC_MAX_HISTORY, M <= TNG_MAX_WORKERS; beyond them the call
 * returns TNG_ERR_UNSUPPORTED and launches nothing.
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.  All calls share the one
 * array: it is cleared where it must start at zero, but two calls that overlap on the
 * GPU (different streams, different threads) race and give wrong sums.
 * The call never waits for the GPU, so a failure that only shows there is reported in the
 * output: if a bounded wait of the staged statistics kernel gave up, all k*k+k+1 outputs
 * are NaN (the sums would be incomplete). */
#define TNG_STATIC_MAX_HISTORY 8
#define TNG_STATIC_SCRATCH_BYTES (320 * 1024)
tng_status tng_gram_static(const float* const* rows_dev, uint32_t k, uint64_t d, const float* grads_dev,
                           uint32_t M, uint64_t ld, double* out_dev, void* stream);

/* Synchronises the context's last stream and fills *out.  Returns TNG_ERR_CUDA if a staged
 * kernel reported a pipeline error, TNG_ERR_NONFINITE if new non-finite scales were counted. */
tng_status tng_stats(tng_ctx* ctx, tng_stats_t* out);
const char* tng_status_string(tng_status s);
/* cudaError_t value of the last failing CUDA call seen by this context (0 if none). */
int tng_last_cuda_error(const tng_ctx* ctx);

/* ---- gradient producers of the synthetic workloads (Section 4) -------------- */
/* l2-regularised logistic regression, labels in {-1,+1}:
 *   grad = -(1/n) sum_i b_i a_i sigma(-b_i a_i.w) + lambda2 w.
 * X_dev: n x d row-major (d % 4 == 0 not required; rows are read with scalar tails),
 * scratch_dev: at least tng_logistic_scratch_floats(n, d) floats. */
size_t tng_logistic_scratch_floats(uint64_t n, uint64_t d);
tng_status tng_logistic_grad(const float* X_dev, const float* b_dev, uint64_t n, uint64_t d,
                             const float* w_dev, float lambda2, float* grad_dev, float* scratch_dev,
                             void* stream);
/* loss = (1/n) sum_i log(1+exp(-b_i a_i.w)) + (lambda2/2)||w||^2, written to *loss_dev (double). */
tng_status tng_logistic_loss(const float* X_dev, const float* b_dev, uint64_t n, uint64_t d,
                             const float* w_dev, float lambda2, double* loss_dev, float* scratch_dev,
                             void* stream);
/* Extended, uncoupled Rosenbrock f(x) = sum_i 100 (x_{2i+1} - x_{2i}^2)^2 + (1 - x_{2i})^2 (d even):
 * grads[m][i] = df/dx_i + noise[m][i] (noise_dev may be NULL), rows of stride ld. */
tng_status tng_rosenbrock_grad(const float* x_dev, uint64_t d, const float* noise_dev, uint32_t M,
                               uint64_t ld, float* grads_dev, void* stream);
tng_status tng_rosenbrock_value(const float* x_dev, uint64_t d, double* value_dev, void* stream);
/* w <- w - eta * v (the outer update of Eq. 1). */
tng_status tng_sgd_update(float* w_dev, const float* v_dev, uint64_t d, float eta, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TNG_H */
