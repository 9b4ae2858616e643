/*
 * tng_oracle.h -- CPU oracle for the Trajectory Normalized Gradients (TNG) step.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  This is a plain, slow, step-by-step CPU
 * statement of what one TNG round computes (arXiv 1901.08227, Section 3, Eq. 2,
 * Eq. 3, Section 3.2, Algorithm 1).  It exists so that tests can compare the CUDA
 * library against it and so that a benchmark can time it as a CPU baseline.  It
 * shares no source, table, constant generator or helper with the CUDA path and
 * must never be called from it.
 *
 * Every function below takes plain host pointers.  All "fp32" steps use one IEEE
 * round-to-nearest-even operation each (compiled with -ffp-contract=off, no
 * fast-math); the fusion statistics and the solve are in double.
 *
 * Parity status: every stage function is pinned by CPU tests to facts outside this
 * file (closed forms, library routines, invariants).  The composed multi-step
 * trajectory (tngo_step called repeatedly) has no worked numeric example in the
 * paper: beyond its stage-level pins it is "parity unpinned".
 */
#ifndef TNG_ORACLE_H
#define TNG_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* codec value = bits per symbol */
enum { TNGO_CODEC_SIGN1 = 1, TNGO_CODEC_TERN2 = 2, TNGO_CODEC_QSGD4 = 4 };
/* MEAN: the reference of worker m is the scalar mean(g^m) times ones(D) (Section 3.1); it
 * needs no trajectory, each worker sends its scalar along with the codes. */
enum { TNGO_NORM_NONE = 0, TNGO_NORM_DIFF = 1, TNGO_NORM_QUOT = 2, TNGO_NORM_COMB = 3, TNGO_NORM_MEAN = 4 };
enum { TNGO_SCALE_ABSMAX = 0, TNGO_SCALE_L2 = 1 };
enum { TNGO_FUSE_LAST = 1, TNGO_FUSE_MEAN = 2, TNGO_FUSE_LSQ = 3, TNGO_FUSE_HINDSIGHT = 4 };

#define TNGO_MAX_K 16
#define TNGO_TILE 128

/* ---- counter-based generator (Philox4x32-10, Salmon et al. 2011) ---------- */
void tngo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* u in [0,1): top 24 bits of x times 2^-24 (exact in fp32). */
float tngo_uniform24(uint32_t x);
/* The uniform that belongs to coordinate i of worker m at step t. */
float tngo_coord_uniform(uint32_t seed_lo, uint32_t seed_hi, uint64_t i, uint32_t m, uint32_t t);

/* ---- wire geometry ------------------------------------------------------- */
uint64_t tngo_num_tiles(uint64_t d);                    /* ceil(d/128) */
uint64_t tngo_words_per_worker(uint64_t d, int codec);  /* tiles * 4 * bits */
uint64_t tngo_num_blocks(uint64_t d, uint64_t B);       /* B == 0: one block */

/* ---- trajectory fusion (criterion of Proposition 2 over the pool of Sec. 3.1) */
/* h[j] (j = 0..k-1) points at history vector h_{j+1}; h[0] is the newest.
 * G (k*k, row-major, symmetric) = <h_i,h_j>; c (k) = <h_i, gbar>,
 * gbar = (1/M) sum_m g^m; gg = (1/M) sum_m ||g^m||^2.  All in double. */
void tngo_fuse_stats(const float* const* h, int k, uint64_t d, const float* grads, int M,
                     uint64_t ld, double* G, double* c, double* gg);
/* Solve (G + lambda I) alpha = c, lambda = ridge * trace(G) / k, by Cholesky in
 * double.  Returns 0 on success; 1 if a pivot was <= 0 or not finite, in which
 * case alpha = e_1.  alpha32 = alpha rounded to fp32. */
int tngo_fuse_solve(const double* G, const double* c, int k, double ridge, double* alpha64,
                    float* alpha32);
/* Hindsight-only right-hand side: regress h_1 on h_2..h_k using G alone and apply
 * the coefficients shifted by one position (needs k >= 2).  Returns as above. */
int tngo_fuse_solve_hindsight(const double* G, int k, double ridge, double* alpha64,
                              float* alpha32);
/* ref_d = fma(alpha_k, h_k[d], ... fma(alpha_1, h_1[d], 0)) in fp32, j ascending. */
void tngo_combine(const float* const* h, const float* alpha32, int k, uint64_t d, float* ref);

/* ---- normalisation helpers ---------------------------------------------- */
/* Guarded denominator of the quotient form (Eq. 3), per 128-coordinate tile. */
void tngo_quot_den(const float* ref, uint64_t d, float quot_eps, float* den);

/* ---- encode (Eq. 2 / Eq. 3, Sec. 3.2, Algorithm 1 steps "compute R, sample z,
 * transmit") ---------------------------------------------------------------- */
/* grads: M rows, row stride ld floats.  ref: d floats or NULL (treated as zeros /
 * ones).  codes: M * words_per_worker uint32 (fully overwritten).  scales:
 * M * num_blocks floats.  s: QSGD level count 1..7 (ignored by other codecs). */
void tngo_encode(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref, int norm,
                 float quot_eps, int codec, uint64_t B, int s, int scale_kind, uint32_t seed_lo,
                 uint32_t seed_hi, uint32_t t, uint32_t* codes, float* scales);

/* Same for a window of a longer vector: the d coordinates are i0 .. i0+d-1 of it (i0 a
 * multiple of 128 and of B), which only moves the Philox counters. */
/* ref2: second reference of the combined form r = Q[(g - ref) ./ ref2], v = ref2 . r + ref
 * (Section 3, display after Eq. 3); only read when norm == TNGO_NORM_COMB. */
/* means: the M scalar references mean(g^m) of TNGO_NORM_MEAN (of the WHOLE vectors, when the
 * d coordinates are a window); only read in that mode. */
void tngo_encode_at(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref, const float* ref2,
                    const float* means, int norm, float quot_eps, int codec, uint64_t B, int s, int scale_kind,
                    uint32_t seed_lo, uint32_t seed_hi, uint32_t t, uint64_t i0, uint32_t* codes, float* scales);
/* mean(g): fp32 adjacent-pairwise tree sum over the d elements (zero-padded to a power of
 * two) divided by d (Section 3.1, the scalar reference). */
float tngo_row_mean(const float* g, uint64_t d);
/* (1/M) sum_m means[m], m ascending in fp32: what decoding adds back in TNGO_NORM_MEAN. */
float tngo_mean_of_means(const float* means, int M);
/* r'_d = (1/k) sum_j |h_j,d|: per-coordinate magnitude of the trajectory (fp32 fma chain). */
void tngo_magnitude_reference(const float* const* h, int k, uint64_t d, float* ref2);

/* ---- decode + aggregate + de-normalise (Eq. 2 / Eq. 3, Algorithm 1 "average") */
void tngo_decode_aggregate(const uint32_t* codes, const float* scales, int M, uint64_t d,
                           const float* ref, int norm, float quot_eps, int codec, uint64_t B,
                           int s, float* out);
void tngo_decode_aggregate2(const uint32_t* codes, const float* scales, int M, uint64_t d,
                            const float* ref, const float* ref2, const float* means, int norm, float quot_eps,
                            int codec, uint64_t B, int s, float* out);
/* Decoded value of one symbol (used by tests that unpack the wire themselves). */
float tngo_dequant(int codec, int s, uint32_t symbol, float R);

/* C_nz estimate of Proposition 2 (difference form): sum_m||g^m-ref||^2 / sum_m||g^m||^2. */
double tngo_cnz(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref);
/* bits per coordinate on the wire: b + 32/B_eff + 64K/d. */
double tngo_bits_per_coord(uint64_t d, int K, int codec, uint64_t B);

/* ---- whole-step state machine (Algorithm 1) ------------------------------ */
typedef struct tngo_state tngo_state;
tngo_state* tngo_create(uint64_t d, int M, int K, int codec, int norm);
void tngo_destroy(tngo_state* st);
/* keys: 0 block, 1 qsgd levels, 2 scale kind, 3 seed lo, 4 seed hi, 5 fuse mode
 * (0 auto), 6 ridge, 7 quot eps, 8 reference refresh cadence (tngo_step only).  Returns 0 ok, nonzero on a bad key/value. */
int tngo_set_option(tngo_state* st, int key, double value);
void tngo_push_reference(tngo_state* st, const float* vec);
/* One round: fuse -> normalise -> encode -> decode -> aggregate -> push. */
void tngo_step(tngo_state* st, const float* grads, uint64_t ld, float* out);
/* Stage-level, same order as tngo_step. */
void tngo_stage_fuse(tngo_state* st, const float* grads, uint64_t ld);
void tngo_stage_encode(tngo_state* st, const float* grads, uint64_t ld);
void tngo_stage_decode_push(tngo_state* st, float* out);
/* Borrowed views of the state. */
const float* tngo_ref(const tngo_state* st);
const float* tngo_ref2(const tngo_state* st);
const uint32_t* tngo_codes(const tngo_state* st);
const float* tngo_scales(const tngo_state* st);
const float* tngo_means(const tngo_state* st); /* M scalar references of the last round (TNGO_NORM_MEAN) */
const float* tngo_alpha(const tngo_state* st);
const double* tngo_gram(const tngo_state* st); /* k*k then c (k) then gg (1) */
int tngo_hist_count(const tngo_state* st);
uint32_t tngo_step_count(const tngo_state* st);
int tngo_solver_fallback(const tngo_state* st);
const float* tngo_history(const tngo_state* st, int j); /* h_{j+1}, j=0 newest */

/* ---- gradient producers of the synthetic workloads ----------------------- */
/* l2-regularised logistic regression (Sec. 4.2): labels b in {-1,+1}.
 * loss = (1/n) sum_i log(1+exp(-b_i a_i.w)) + (lambda2/2)||w||^2, in double;
 * grad rounded to fp32.  X is n x d row-major. */
double tngo_logistic_loss(const float* X, const float* b, uint64_t n, uint64_t d, const float* w,
                          double lambda2);
void tngo_logistic_grad(const float* X, const float* b, uint64_t n, uint64_t d, const float* w,
                        double lambda2, float* grad);
/* Extended, uncoupled Rosenbrock (Sec. 4.1 function, textbook pair form):
 * f(x) = sum_{i<d/2} 100 (x_{2i+1} - x_{2i}^2)^2 + (1 - x_{2i})^2, d even.
 * Value in double.  Gradient elementwise in fp32 with a fixed operation order,
 * plus an optional per-worker noise row: grads[m][i] = grad_i + noise[m][i]. */
double tngo_rosenbrock_value(const float* x, uint64_t d);
void tngo_rosenbrock_grad(const float* x, uint64_t d, const float* noise, int M, uint64_t ld,
                          float* grads);
/* w <- w - eta * v, one fp32 multiply and one fp32 subtraction per element. */
void tngo_sgd_update(float* w, const float* v, uint64_t d, float eta);

/* ---- threads of the parallel loops (for timing the oracle; no result depends on them) */
int tngo_max_threads(void);
void tngo_set_threads(int n);

#ifdef __cplusplus
}
#endif
#endif
