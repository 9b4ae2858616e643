/*
 * tng_oracle.c -- CPU oracle for the TNG step.  TEST INFRASTRUCTURE (see header).
 *
 * Written from the paper (arXiv 1901.08227): Section 3 (Eq. 2 difference form,
 * Eq. 3 quotient form), Section 3.1 (pool of reference vectors), Section 3.2
 * (stochastic ternary coding Q[v] = R sign[v] . z(v), R = max|v_d|,
 * P(z_d = 1) = |v_d|/R), Algorithm 1 (the round), Proposition 2 (criterion
 * C_nz for choosing the reference), Section 4 (workloads).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math).
 * The OpenMP pragmas only split independent outer loops; every reduction that
 * defines a value is serial and in the order stated beside it.
 */
#include "tng_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Philox4x32-10: 10 rounds; each round maps (c0,c1,c2,c3) to                 */
/* (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)); the key is bumped */
/* by the Weyl constants between rounds.                                      */
/* ------------------------------------------------------------------------- */
#define PHILOX_M0 0xD2511F53u
#define PHILOX_M1 0xCD9E8D57u
#define PHILOX_W0 0x9E3779B9u
#define PHILOX_W1 0xBB67AE85u

void tngo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += PHILOX_W0;
            k1 += PHILOX_W1;
        }
        uint64_t p0 = (uint64_t)PHILOX_M0 * c0;
        uint64_t p1 = (uint64_t)PHILOX_M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

float tngo_uniform24(uint32_t x) { return (float)(x >> 8) * 0x1p-24f; }

/* counter = (lo32(i/4), hi32(i/4), m, t); word (i mod 4) belongs to coordinate i */
float tngo_coord_uniform(uint32_t seed_lo, uint32_t seed_hi, uint64_t i, uint32_t m, uint32_t t) {
    uint64_t q = i / 4;
    uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), m, t};
    uint32_t key[2] = {seed_lo, seed_hi};
    uint32_t out[4];
    tngo_philox4x32_10(ctr, key, out);
    return tngo_uniform24(out[i % 4]);
}

/* ------------------------------------------------------------------------- */
/* wire geometry                                                              */
/* ------------------------------------------------------------------------- */
uint64_t tngo_num_tiles(uint64_t d) { return (d + TNGO_TILE - 1) / TNGO_TILE; }
uint64_t tngo_words_per_worker(uint64_t d, int codec) { return tngo_num_tiles(d) * 4u * (uint64_t)codec; }
uint64_t tngo_num_blocks(uint64_t d, uint64_t B) { return B == 0 ? 1 : (d + B - 1) / B; }

/* Tile-planar layout: tile T = coordinates [128T, 128T+128) owns 4*b consecutive
 * words; word c*b + p (c = i mod 4, p = bit plane) holds, at bit j = (i mod 128)/4,
 * bit p of coordinate i's symbol. */
static void put_symbol(uint32_t* codes_m, int b, uint64_t i, uint32_t symbol) {
    uint64_t T = i / TNGO_TILE;
    uint32_t within = (uint32_t)(i % TNGO_TILE);
    uint32_t c = within % 4, j = within / 4;
    for (int p = 0; p < b; ++p)
        if ((symbol >> p) & 1u) codes_m[T * 4u * (uint64_t)b + c * (uint32_t)b + (uint32_t)p] |= (1u << j);
}
static uint32_t get_symbol(const uint32_t* codes_m, int b, uint64_t i) {
    uint64_t T = i / TNGO_TILE;
    uint32_t within = (uint32_t)(i % TNGO_TILE);
    uint32_t c = within % 4, j = within / 4, symbol = 0;
    for (int p = 0; p < b; ++p)
        symbol |= ((codes_m[T * 4u * (uint64_t)b + c * (uint32_t)b + (uint32_t)p] >> j) & 1u) << p;
    return symbol;
}

/* ------------------------------------------------------------------------- */
/* trajectory fusion                                                          */
/* ------------------------------------------------------------------------- */
void tngo_fuse_stats(const float* const* h, int k, uint64_t d, const float* grads, int M,
                     uint64_t ld, double* G, double* c, double* gg) {
    /* gbar_d = (1/M) sum_m g^m_d, in double */
    double* gbar = (double*)malloc(sizeof(double) * (d ? d : 1));
    double sumsq = 0.0;
    for (uint64_t i = 0; i < d; ++i) {
        double acc = 0.0;
        for (int m = 0; m < M; ++m) {
            double g = (double)grads[(uint64_t)m * ld + i];
            acc += g;
            sumsq += g * g;
        }
        gbar[i] = acc / (double)M;
    }
    if (gg) *gg = sumsq / (double)M;
    int npair = k * k + k;
#pragma omp parallel for schedule(dynamic)
    for (int idx = 0; idx < npair; ++idx) {
        if (idx < k * k) {
            int a = idx / k, b = idx % k;
            if (b < a) continue; /* filled by symmetry below */
            double acc = 0.0;
            for (uint64_t i = 0; i < d; ++i) acc += (double)h[a][i] * (double)h[b][i];
            G[a * k + b] = acc;
        } else {
            int a = idx - k * k;
            double acc = 0.0;
            for (uint64_t i = 0; i < d; ++i) acc += (double)h[a][i] * gbar[i];
            c[a] = acc;
        }
    }
    for (int a = 0; a < k; ++a)
        for (int b = 0; b < a; ++b) G[a * k + b] = G[b * k + a];
    free(gbar);
}

/* Cholesky A = L L^T then two triangular solves; returns 1 on a bad pivot.  A pivot
 * that is not above 1e-12 times its diagonal entry is rounding noise of a singular
 * matrix and counts as bad. */
static int chol_solve(const double* A, const double* rhs, int n, double* x) {
    double L[TNGO_MAX_K * TNGO_MAX_K];
    double y[TNGO_MAX_K];
    memset(L, 0, sizeof L);
    for (int j = 0; j < n; ++j) {
        double diag = A[j * n + j];
        for (int p = 0; p < j; ++p) diag -= L[j * n + p] * L[j * n + p];
        if (!(diag > 1e-12 * A[j * n + j]) || !(diag > 0.0) || !isfinite(diag)) return 1;
        double ljj = sqrt(diag);
        L[j * n + j] = ljj;
        for (int i = j + 1; i < n; ++i) {
            double v = A[i * n + j];
            for (int p = 0; p < j; ++p) v -= L[i * n + p] * L[j * n + p];
            L[i * n + j] = v / ljj;
        }
    }
    for (int i = 0; i < n; ++i) {
        double v = rhs[i];
        for (int p = 0; p < i; ++p) v -= L[i * n + p] * y[p];
        y[i] = v / L[i * n + i];
    }
    for (int i = n - 1; i >= 0; --i) {
        double v = y[i];
        for (int p = i + 1; p < n; ++p) v -= L[p * n + i] * x[p];
        x[i] = v / L[i * n + i];
    }
    for (int i = 0; i < n; ++i)
        if (!isfinite(x[i])) return 1;
    return 0;
}

static void alpha_fallback(int k, double* alpha64, float* alpha32) {
    for (int j = 0; j < k; ++j) {
        alpha64[j] = (j == 0) ? 1.0 : 0.0;
        alpha32[j] = (float)alpha64[j];
    }
}

int tngo_fuse_solve(const double* G, const double* c, int k, double ridge, double* alpha64,
                    float* alpha32) {
    double A[TNGO_MAX_K * TNGO_MAX_K] = {0};
    if (k < 1) return 1;
    double trace = 0.0;
    for (int j = 0; j < k; ++j) trace += G[j * k + j];
    double lambda = ridge * trace / (double)k;
    for (int a = 0; a < k; ++a)
        for (int b = 0; b < k; ++b) A[a * k + b] = G[a * k + b] + (a == b ? lambda : 0.0);
    if (chol_solve(A, c, k, alpha64)) {
        alpha_fallback(k, alpha64, alpha32);
        return 1;
    }
    for (int j = 0; j < k; ++j) alpha32[j] = (float)alpha64[j];
    return 0;
}

int tngo_fuse_solve_hindsight(const double* G, int k, double ridge, double* alpha64,
                              float* alpha32) {
    if (k < 2) {
        alpha_fallback(k, alpha64, alpha32);
        return k < 1 ? 1 : 0;
    }
    /* beta = argmin || h_1 - sum_{j=2..k} beta_j h_j ||^2 (+ ridge): the sub-Gram
     * of h_2..h_k against the column <h_j, h_1>.  Applied one position later:
     * alpha_j = beta_{j+1} for j = 1..k-1, alpha_k = 0. */
    int n = k - 1;
    double A[TNGO_MAX_K * TNGO_MAX_K], rhs[TNGO_MAX_K], beta[TNGO_MAX_K];
    double trace = 0.0;
    for (int j = 1; j < k; ++j) trace += G[j * k + j];
    double lambda = ridge * trace / (double)n;
    for (int a = 0; a < n; ++a) {
        rhs[a] = G[(a + 1) * k + 0];
        for (int b = 0; b < n; ++b)
            A[a * n + b] = G[(a + 1) * k + (b + 1)] + (a == b ? lambda : 0.0);
    }
    if (chol_solve(A, rhs, n, beta)) {
        alpha_fallback(k, alpha64, alpha32);
        return 1;
    }
    for (int j = 0; j < n; ++j) alpha64[j] = beta[j];
    alpha64[k - 1] = 0.0;
    for (int j = 0; j < k; ++j) alpha32[j] = (float)alpha64[j];
    return 0;
}

void tngo_combine(const float* const* h, const float* alpha32, int k, uint64_t d, float* ref) {
#pragma omp parallel for
    for (uint64_t i = 0; i < d; ++i) {
        float acc = 0.0f;
        for (int j = 0; j < k; ++j) acc = fmaf(alpha32[j], h[j][i], acc);
        ref[i] = acc;
    }
}

/* ------------------------------------------------------------------------- */
/* normalisation                                                              */
/* ------------------------------------------------------------------------- */
/* max of |x| over a range; any NaN makes the result NaN */
static float absmax_nan(const float* x, uint64_t n) {
    float mx = 0.0f;
    for (uint64_t i = 0; i < n; ++i) {
        float a = fabsf(x[i]);
        if (isnan(a)) return NAN;
        if (a > mx) mx = a;
    }
    return mx;
}

/* Quotient form guard.  Per tile: mx = max|ref_d|.  mx not a positive finite
 * number (all zero, NaN, inf) -> den = 1 (plain compression for that tile).
 * Otherwise den_d = sign(ref_d) * max(|ref_d|, quot_eps * mx), zero counting as
 * positive.  A linear elementwise map, so the code stays unbiased. */
void tngo_quot_den(const float* ref, uint64_t d, float quot_eps, float* den) {
    uint64_t ntile = tngo_num_tiles(d);
#pragma omp parallel for
    for (uint64_t T = 0; T < ntile; ++T) {
        uint64_t lo = T * TNGO_TILE, hi = lo + TNGO_TILE < d ? lo + TNGO_TILE : d;
        float mx = ref ? absmax_nan(ref + lo, hi - lo) : 0.0f;
        if (!(mx > 0.0f) || !isfinite(mx)) {
            for (uint64_t i = lo; i < hi; ++i) den[i] = 1.0f;
            continue;
        }
        float floor_ = quot_eps * mx;
        for (uint64_t i = lo; i < hi; ++i) {
            float a = fabsf(ref[i]);
            float g = a > floor_ ? a : floor_;
            den[i] = (ref[i] < 0.0f) ? -g : g;
        }
    }
}

/* v = g - r (Eq. 2), v = g * (1/den) (Eq. 3: the quotient, taken as one IEEE
 * reciprocal per coordinate shared by all workers and one multiply), or v = g. */
static float normalise(float g, int norm, float r_or_rden) {
    if (norm == TNGO_NORM_DIFF) return g - r_or_rden;
    if (norm == TNGO_NORM_QUOT) return g * r_or_rden;
    return g;
}
/* Combined form of Section 3 (the unnumbered display after Eq. 3): v = (g - r) ./ r', taken as
 * one fp32 subtraction and one multiply by the reciprocal of the guarded second reference. */
static float normalise_comb(float g, float r, float rden2) {
    float diff = g - r;
    return diff * rden2;
}

/* Second reference of the combined form: the per-coordinate magnitude of the trajectory,
 * r'_d = (1/k) sum_j |h_j,d| as an fp32 fma chain (j ascending, 1/k one IEEE division). */
void tngo_magnitude_reference(const float* const* h, int k, uint64_t d, float* ref2) {
    float inv = (k > 0) ? 1.0f / (float)k : 0.0f;
#pragma omp parallel for
    for (uint64_t i = 0; i < d; ++i) {
        float acc = 0.0f;
        for (int j = 0; j < k; ++j) acc = fmaf(inv, fabsf(h[j][i]), acc);
        ref2[i] = acc;
    }
}

/* ------------------------------------------------------------------------- */
/* scale of one block                                                         */
/* ------------------------------------------------------------------------- */
static uint64_t pow2_ceil(uint64_t n) {
    uint64_t p = 1;
    while (p < n) p <<= 1;
    return p;
}

/* L2 scale: fp32 adjacent-pairwise tree over v_d^2, block zero-padded to a power
 * of two; R = sqrtf(S). */
static float l2_scale(const float* v, uint64_t n) {
    uint64_t P = pow2_ceil(n);
    float* buf = (float*)calloc(P, sizeof(float));
    for (uint64_t i = 0; i < n; ++i) buf[i] = v[i] * v[i];
    for (uint64_t len = P; len > 1; len /= 2)
        for (uint64_t i = 0; i < len / 2; ++i) buf[i] = buf[2 * i] + buf[2 * i + 1];
    float S = buf[0];
    free(buf);
    return sqrtf(S);
}

static int scale_is_bad(float R) { return !(R > 0.0f) || !isfinite(R); }

/* Scalar reference of Section 3.1 (fourth entry of the list of references): mean(g), the
 * average of all elements of one worker's gradient.  The sum is the fp32 adjacent-pairwise
 * tree over the d coordinates, zero-padded to a power of two; one IEEE division by d. */
float tngo_row_mean(const float* g, uint64_t d) {
    uint64_t P = pow2_ceil(d);
    float* buf = (float*)calloc(P ? P : 1, sizeof(float));
    for (uint64_t i = 0; i < d; ++i) buf[i] = g[i];
    for (uint64_t len = P; len > 1; len /= 2)
        for (uint64_t i = 0; i < len / 2; ++i) buf[i] = buf[2 * i] + buf[2 * i + 1];
    float S = buf[0];
    free(buf);
    return S / (float)d;
}
/* What the server adds back: the average of the workers' means, summed m ascending in fp32. */
float tngo_mean_of_means(const float* means, int M) {
    float acc = 0.0f;
    for (int m = 0; m < M; ++m) acc = (m == 0) ? means[m] : acc + means[m];
    return acc / (float)M;
}

/* ------------------------------------------------------------------------- */
/* quantisers: symbol of one coordinate given v, its block scale R and u       */
/* ------------------------------------------------------------------------- */
/* Ternary (Sec. 3.2): nonzero with probability |v|/R, realised as u*R < |v|
 * (u*R one fp32 product); |v| = R always fires because u < 1, v = 0 never does.
 * symbol bit0 = nonzero, bit1 = negative. */
static uint32_t quant_tern2(float v, float R, float u) {
    uint32_t nz = (u * R < fabsf(v)) ? 1u : 0u;
    uint32_t neg = (nz && v < 0.0f) ? 1u : 0u;
    return nz | (neg << 1);
}
/* Stochastic sign: +R with probability (1 + v/R)/2, else -R, so E = v.
 * Realised as u*R < 0.5 v + 0.5 R.  symbol bit0 = plus. */
static uint32_t quant_sign1(float v, float R, float u) {
    float thr = 0.5f * v + 0.5f * R;
    return (u * R < thr) ? 1u : 0u;
}
/* s-level stochastic uniform quantiser (QSGD, Alistarh et al. 2017):
 * a = (|v|/R) s, level floor(a) or floor(a)+1 with probability frac(a), and never
 * above s: the quantiser has the levels 0..s only.  The bound matters when the L2
 * scale underestimates |v| (v*v subnormal, so sqrtf(fl(v*v)) < |v| and a > s);
 * without it level s+1 would spill into the sign bit of the 4-bit symbol.
 * symbol bits 0..2 = level, bit 3 = negative. */
static uint32_t quant_qsgd4(float v, float R, float u, int s) {
    float q = fabsf(v) / R;
    float a = q * (float)s;
    float l = floorf(a);
    float f = a - l;
    int L = (int)l + ((u < f) ? 1 : 0);
    if (L > s) L = s;
    uint32_t neg = (L > 0 && v < 0.0f) ? 1u : 0u;
    return (uint32_t)L | (neg << 3);
}

float tngo_dequant(int codec, int s, uint32_t symbol, float R) {
    if (scale_is_bad(R)) return 0.0f;
    if (codec == TNGO_CODEC_TERN2) {
        if (!(symbol & 1u)) return 0.0f;
        return (symbol & 2u) ? -R : R;
    }
    if (codec == TNGO_CODEC_SIGN1) return (symbol & 1u) ? R : -R;
    /* QSGD4: level * (R / s) */
    float step = R / (float)s;
    float mag = (float)(symbol & 7u) * step;
    return (symbol & 8u) ? -mag : mag;
}

/* ------------------------------------------------------------------------- */
/* encode                                                                     */
/* ------------------------------------------------------------------------- */
/* The d coordinates handed in are coordinates i0 .. i0+d-1 of a longer vector (i0 a
 * multiple of the block size and of 128): only the Philox counters see i0. */
void tngo_encode_at(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref, const float* ref2,
                    const float* means, int norm, float quot_eps, int codec, uint64_t B, int s, int scale_kind,
                    uint32_t seed_lo, uint32_t seed_hi, uint32_t t, uint64_t i0, uint32_t* codes, float* scales) {
    uint64_t wpw = tngo_words_per_worker(d, codec);
    uint64_t nblk = tngo_num_blocks(d, B);
    uint64_t Beff = (B == 0) ? d : B;
    memset(codes, 0, sizeof(uint32_t) * wpw * (uint64_t)M);

    /* per-coordinate operand of the normalisation, shared by all workers */
    float* opnd = (float*)malloc(sizeof(float) * (d ? d : 1));
    if (norm == TNGO_NORM_QUOT || norm == TNGO_NORM_COMB) {
        tngo_quot_den(norm == TNGO_NORM_QUOT ? ref : ref2, d, quot_eps, opnd);
        for (uint64_t i = 0; i < d; ++i) opnd[i] = 1.0f / opnd[i];
    } else {
        for (uint64_t i = 0; i < d; ++i) opnd[i] = (norm == TNGO_NORM_DIFF && ref) ? ref[i] : 0.0f;
    }

    long long njobs = (long long)M * (long long)nblk;
#pragma omp parallel for schedule(static)
    for (long long job = 0; job < njobs; ++job) {
        int m = (int)(job / (long long)nblk);
        uint64_t blk = (uint64_t)(job % (long long)nblk);
        uint64_t lo = blk * Beff, hi = lo + Beff < d ? lo + Beff : d;
        uint64_t n = hi - lo;
        const float* g = grads + (uint64_t)m * ld;
        float* v = (float*)malloc(sizeof(float) * (n ? n : 1));
        for (uint64_t i = 0; i < n; ++i) {
            if (norm == TNGO_NORM_COMB) v[i] = normalise_comb(g[lo + i], ref ? ref[lo + i] : 0.0f, opnd[lo + i]);
            else if (norm == TNGO_NORM_MEAN) v[i] = g[lo + i] - means[m];   /* reference mean(g^m) ones(D) */
            else v[i] = normalise(g[lo + i], norm, opnd[lo + i]);
        }
        float R = (scale_kind == TNGO_SCALE_L2) ? l2_scale(v, n) : absmax_nan(v, n);
        scales[(uint64_t)m * nblk + blk] = R;
        if (!scale_is_bad(R)) {
            uint32_t* codes_m = codes + (uint64_t)m * wpw;
            for (uint64_t i = 0; i < n; ++i) {
                float u = tngo_coord_uniform(seed_lo, seed_hi, i0 + lo + i, (uint32_t)m, t);
                uint32_t sym;
                if (codec == TNGO_CODEC_TERN2) sym = quant_tern2(v[i], R, u);
                else if (codec == TNGO_CODEC_SIGN1) sym = quant_sign1(v[i], R, u);
                else sym = quant_qsgd4(v[i], R, u, s);
                /* blocks are multiples of 128 coordinates, so two jobs never share a word */
                put_symbol(codes_m, codec, lo + i, sym);
            }
        }
        free(v);
    }
    free(opnd);
}

void tngo_encode(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref, int norm,
                 float quot_eps, int codec, uint64_t B, int s, int scale_kind, uint32_t seed_lo,
                 uint32_t seed_hi, uint32_t t, uint32_t* codes, float* scales) {
    tngo_encode_at(grads, M, ld, d, ref, NULL, NULL, norm, quot_eps, codec, B, s, scale_kind, seed_lo, seed_hi, t, 0, codes,
                   scales);
}

/* ------------------------------------------------------------------------- */
/* decode + aggregate + de-normalise                                          */
/* ------------------------------------------------------------------------- */
void tngo_decode_aggregate2(const uint32_t* codes, const float* scales, int M, uint64_t d,
                            const float* ref, const float* ref2, const float* means, int norm, float quot_eps,
                            int codec, uint64_t B, int s, float* out) {
    uint64_t wpw = tngo_words_per_worker(d, codec);
    uint64_t nblk = tngo_num_blocks(d, B);
    uint64_t Beff = (B == 0) ? d : B;
    float* den = NULL;
    if (norm == TNGO_NORM_QUOT || norm == TNGO_NORM_COMB) {
        den = (float*)malloc(sizeof(float) * (d ? d : 1));
        tngo_quot_den(norm == TNGO_NORM_QUOT ? ref : ref2, d, quot_eps, den);
    }
    float mbar = (norm == TNGO_NORM_MEAN) ? tngo_mean_of_means(means, M) : 0.0f;
#pragma omp parallel for
    for (uint64_t i = 0; i < d; ++i) {
        uint64_t blk = (Beff == 0) ? 0 : i / Beff;
        /* a = (((vhat^0 + vhat^1) + ...) + vhat^{M-1}) / M, workers ascending, fp32 */
        float acc = 0.0f;
        for (int m = 0; m < M; ++m) {
            float R = scales[(uint64_t)m * nblk + blk];
            uint32_t sym = get_symbol(codes + (uint64_t)m * wpw, codec, i);
            float vhat = tngo_dequant(codec, s, sym, R);
            acc = (m == 0) ? vhat : acc + vhat;
        }
        float a = acc / (float)M;
        float r = (ref ? ref[i] : 0.0f);
        if (norm == TNGO_NORM_DIFF) out[i] = r + a;         /* v = ref + r(w_t), Eq. 2 */
        else if (norm == TNGO_NORM_QUOT) out[i] = den[i] * a; /* v = ref . r(w_t), Eq. 3 */
        else if (norm == TNGO_NORM_COMB) {                    /* v = ref' . r(w_t) + ref */
            float scaled = den[i] * a;
            out[i] = scaled + r;
        } else if (norm == TNGO_NORM_MEAN) out[i] = a + mbar; /* (1/M) sum_m (vhat^m + mean^m ones) */
        else out[i] = a;
    }
    free(den);
}

void tngo_decode_aggregate(const uint32_t* codes, const float* scales, int M, uint64_t d,
                           const float* ref, int norm, float quot_eps, int codec, uint64_t B,
                           int s, float* out) {
    tngo_decode_aggregate2(codes, scales, M, d, ref, NULL, NULL, norm, quot_eps, codec, B, s, out);
}

/* ------------------------------------------------------------------------- */
/* statistics                                                                 */
/* ------------------------------------------------------------------------- */
double tngo_cnz(const float* grads, int M, uint64_t ld, uint64_t d, const float* ref) {
    double num = 0.0, den = 0.0;
    for (int m = 0; m < M; ++m)
        for (uint64_t i = 0; i < d; ++i) {
            double g = (double)grads[(uint64_t)m * ld + i];
            double r = ref ? (double)ref[i] : 0.0;
            num += (g - r) * (g - r);
            den += g * g;
        }
    return num / den;
}

double tngo_bits_per_coord(uint64_t d, int K, int codec, uint64_t B) {
    double Beff = (B == 0) ? (double)d : (double)B;
    return (double)codec + 32.0 / Beff + 64.0 * (double)K / (double)d;
}

/* ------------------------------------------------------------------------- */
/* state machine (Algorithm 1)                                                */
/* ------------------------------------------------------------------------- */
struct tngo_state {
    uint64_t d;
    int M, K, codec, norm;
    uint64_t B;
    int s, scale_kind, fuse_mode;
    uint32_t ref_every; /* the reference is re-fused in rounds t with t % ref_every == 0 */
    uint32_t seed_lo, seed_hi;
    double ridge;
    float quot_eps;
    float* H;   /* K slots of d floats */
    int k;      /* valid slots */
    int head;   /* slot of the newest vector */
    uint32_t t; /* rounds done */
    float* ref;
    float* ref2; /* second reference (combined form) */
    uint32_t* codes;
    float* scales;
    float means[64]; /* scalar references of the round (TNGO_NORM_MEAN) */
    double gram[TNGO_MAX_K * TNGO_MAX_K + TNGO_MAX_K + 1];
    double alpha64[TNGO_MAX_K];
    float alpha[TNGO_MAX_K];
    int fallback;
};

tngo_state* tngo_create(uint64_t d, int M, int K, int codec, int norm) {
    if (d == 0 || M < 1 || M > 64 || K < 1 || K > TNGO_MAX_K) return NULL;
    if (codec != 1 && codec != 2 && codec != 4) return NULL;
    if (norm < 0 || norm > 4) return NULL;
    tngo_state* st = (tngo_state*)calloc(1, sizeof *st);
    st->d = d; st->M = M; st->K = K; st->codec = codec; st->norm = norm;
    st->B = 128; st->s = 7; st->scale_kind = TNGO_SCALE_ABSMAX; st->fuse_mode = 0;
    st->seed_lo = 0; st->seed_hi = 0; st->ridge = 1e-6; st->quot_eps = 0x1p-4f; st->ref_every = 1;
    st->H = (float*)calloc((size_t)K * d, sizeof(float));
    st->ref = (float*)calloc(d, sizeof(float));
    st->ref2 = (float*)calloc(d, sizeof(float));
    st->codes = (uint32_t*)calloc((size_t)M * tngo_words_per_worker(d, codec), sizeof(uint32_t));
    st->scales = NULL;
    st->k = 0; st->head = K - 1; st->t = 0;
    return st;
}

void tngo_destroy(tngo_state* st) {
    if (!st) return;
    free(st->H); free(st->ref); free(st->ref2); free(st->codes); free(st->scales);
    free(st);
}

int tngo_set_option(tngo_state* st, int key, double value) {
    switch (key) {
        case 0:
            if (value < 0 || ((uint64_t)value % TNGO_TILE) != 0) return 1;
            st->B = (uint64_t)value; return 0;
        case 1:
            if (value < 1 || value > 7) return 1;
            st->s = (int)value; return 0;
        case 2:
            if (value != 0 && value != 1) return 1;
            st->scale_kind = (int)value; return 0;
        case 3: st->seed_lo = (uint32_t)value; return 0;
        case 4: st->seed_hi = (uint32_t)value; return 0;
        case 5:
            if (value < 0 || value > 4) return 1;
            st->fuse_mode = (int)value; return 0;
        case 6:
            if (!(value >= 0)) return 1;
            st->ridge = value; return 0;
        case 7:
            if (!(value > 0 && value <= 1)) return 1;
            st->quot_eps = (float)value; return 0;
        case 8:
            if (value < 1 || value > 65536) return 1;
            st->ref_every = (uint32_t)value; return 0;
        default: return 1;
    }
}

static int effective_fuse_mode(const tngo_state* st) {
    if (st->fuse_mode != 0) return st->fuse_mode;
    return st->K == 1 ? TNGO_FUSE_LAST : TNGO_FUSE_LSQ;
}

/* h_{j+1}: slot (head - j) mod K */
const float* tngo_history(const tngo_state* st, int j) {
    int slot = ((st->head - j) % st->K + st->K) % st->K;
    return st->H + (size_t)slot * st->d;
}

static void push(tngo_state* st, const float* vec) {
    st->head = (st->head + 1) % st->K;
    memcpy(st->H + (size_t)st->head * st->d, vec, sizeof(float) * st->d);
    if (st->k < st->K) st->k += 1;
}

void tngo_push_reference(tngo_state* st, const float* vec) { push(st, vec); }

void tngo_stage_fuse(tngo_state* st, const float* grads, uint64_t ld) {
    int k = st->k;
    st->fallback = 0;
    memset(st->alpha, 0, sizeof st->alpha);
    memset(st->alpha64, 0, sizeof st->alpha64);
    if (k == 0) { /* empty trajectory: reference = zeros (Algorithm 1 initialisation) */
        memset(st->ref, 0, sizeof(float) * st->d);
        memset(st->ref2, 0, sizeof(float) * st->d);
        return;
    }
    const float* h[TNGO_MAX_K];
    for (int j = 0; j < k; ++j) h[j] = tngo_history(st, j);
    if (st->norm == TNGO_NORM_COMB) tngo_magnitude_reference(h, k, st->d, st->ref2);
    int mode = effective_fuse_mode(st);
    if (mode == TNGO_FUSE_LAST) {
        st->alpha[0] = 1.0f; st->alpha64[0] = 1.0;
    } else if (mode == TNGO_FUSE_MEAN) {
        for (int j = 0; j < k; ++j) { st->alpha[j] = 1.0f / (float)k; st->alpha64[j] = st->alpha[j]; }
    } else {
        double* G = st->gram; double* c = G + k * k; double* gg = c + k;
        tngo_fuse_stats(h, k, st->d, grads, st->M, ld, G, c, gg);
        if (mode == TNGO_FUSE_LSQ) st->fallback = tngo_fuse_solve(G, c, k, st->ridge, st->alpha64, st->alpha);
        else st->fallback = tngo_fuse_solve_hindsight(G, k, st->ridge, st->alpha64, st->alpha);
    }
    tngo_combine(h, st->alpha, k, st->d, st->ref);
}

void tngo_stage_encode(tngo_state* st, const float* grads, uint64_t ld) {
    uint64_t nblk = tngo_num_blocks(st->d, st->B);
    if (!st->scales) st->scales = (float*)calloc((size_t)st->M * nblk, sizeof(float));
    if (st->norm == TNGO_NORM_MEAN)
        for (int m = 0; m < st->M; ++m) st->means[m] = tngo_row_mean(grads + (uint64_t)m * ld, st->d);
    tngo_encode_at(grads, st->M, ld, st->d, st->ref, st->ref2, st->means, st->norm, st->quot_eps, st->codec, st->B,
                   st->s, st->scale_kind, st->seed_lo, st->seed_hi, st->t, 0, st->codes, st->scales);
}

void tngo_stage_decode_push(tngo_state* st, float* out) {
    tngo_decode_aggregate2(st->codes, st->scales, st->M, st->d, st->ref, st->ref2, st->means, st->norm,
                           st->quot_eps, st->codec, st->B, st->s, out);
    push(st, out);
    st->t += 1;
}

/* Reference refresh cadence (Sec. 3.1, last paragraph): a new reference only in rounds t with
 * t % ref_every == 0; in between the previous one is kept.  The ring receives every aggregate. */
void tngo_step(tngo_state* st, const float* grads, uint64_t ld, float* out) {
    /* the scalar reference uses no trajectory */
    if (st->norm != TNGO_NORM_MEAN && st->t % st->ref_every == 0) tngo_stage_fuse(st, grads, ld);
    tngo_stage_encode(st, grads, ld);
    tngo_stage_decode_push(st, out);
}

const float* tngo_ref(const tngo_state* st) { return st->ref; }
const float* tngo_ref2(const tngo_state* st) { return st->ref2; }
const uint32_t* tngo_codes(const tngo_state* st) { return st->codes; }
const float* tngo_scales(const tngo_state* st) { return st->scales; }
const float* tngo_means(const tngo_state* st) { return st->means; }
const float* tngo_alpha(const tngo_state* st) { return st->alpha; }
const double* tngo_gram(const tngo_state* st) { return st->gram; }
int tngo_hist_count(const tngo_state* st) { return st->k; }
uint32_t tngo_step_count(const tngo_state* st) { return st->t; }
int tngo_solver_fallback(const tngo_state* st) { return st->fallback; }

/* ------------------------------------------------------------------------- */
/* producers                                                                  */
/* ------------------------------------------------------------------------- */
/* log(1 + exp(-z)) without overflow */
static double softplus_neg(double z) { return z > 0 ? log1p(exp(-z)) : -z + log1p(exp(z)); }
static double sigmoid(double z) { return z >= 0 ? 1.0 / (1.0 + exp(-z)) : exp(z) / (1.0 + exp(z)); }

double tngo_logistic_loss(const float* X, const float* b, uint64_t n, uint64_t d, const float* w,
                          double lambda2) {
    double loss = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        double z = 0.0;
        for (uint64_t j = 0; j < d; ++j) z += (double)X[i * d + j] * (double)w[j];
        loss += softplus_neg((double)b[i] * z);
    }
    double reg = 0.0;
    for (uint64_t j = 0; j < d; ++j) reg += (double)w[j] * (double)w[j];
    return loss / (double)n + 0.5 * lambda2 * reg;
}

/* grad = -(1/n) sum_i b_i a_i sigma(-b_i a_i.w) + lambda2 w */
void tngo_logistic_grad(const float* X, const float* b, uint64_t n, uint64_t d, const float* w,
                        double lambda2, float* grad) {
    double* acc = (double*)calloc(d ? d : 1, sizeof(double));
    double* coef = (double*)malloc(sizeof(double) * (n ? n : 1));
#pragma omp parallel for
    for (uint64_t i = 0; i < n; ++i) {
        double z = 0.0;
        for (uint64_t j = 0; j < d; ++j) z += (double)X[i * d + j] * (double)w[j];
        coef[i] = -(double)b[i] * sigmoid(-(double)b[i] * z);
    }
#pragma omp parallel for
    for (uint64_t j = 0; j < d; ++j) {
        double a = 0.0;
        for (uint64_t i = 0; i < n; ++i) a += coef[i] * (double)X[i * d + j];
        acc[j] = a;
    }
    for (uint64_t j = 0; j < d; ++j) grad[j] = (float)(acc[j] / (double)n + lambda2 * (double)w[j]);
    free(acc); free(coef);
}

double tngo_rosenbrock_value(const float* x, uint64_t d) {
    double f = 0.0;
    for (uint64_t i = 0; i + 1 < d; i += 2) {
        double a = x[i], b = x[i + 1];
        f += 100.0 * (b - a * a) * (b - a * a) + (1.0 - a) * (1.0 - a);
    }
    return f;
}

/* per pair (a,b) = (x_{2i}, x_{2i+1}), each line one fp32 operation:
 *   q = a*a; t = b - q; d/da = -(400 a) t - 2 (1 - a); d/db = 200 t. */
void tngo_rosenbrock_grad(const float* x, uint64_t d, const float* noise, int M, uint64_t ld,
                          float* grads) {
#pragma omp parallel for
    for (uint64_t i = 0; i < d; i += 2) {
        if (i + 1 >= d) continue;
        float a = x[i], b = x[i + 1];
        float q = a * a;
        float t = b - q;
        float u1 = 400.0f * a;
        float u2 = u1 * t;
        float u3 = 1.0f - a;
        float u4 = 2.0f * u3;
        float ga = -u2 - u4;
        float gb = 200.0f * t;
        for (int m = 0; m < M; ++m) {
            float na = noise ? noise[(uint64_t)m * ld + i] : 0.0f;
            float nb = noise ? noise[(uint64_t)m * ld + i + 1] : 0.0f;
            grads[(uint64_t)m * ld + i] = ga + na;
            grads[(uint64_t)m * ld + i + 1] = gb + nb;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* how many threads the parallel loops use (timing only; results do not depend on it) */
/* ------------------------------------------------------------------------- */
#ifdef _OPENMP
#include <omp.h>
int tngo_max_threads(void) { return omp_get_max_threads(); }
void tngo_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
#else
int tngo_max_threads(void) { return 1; }
void tngo_set_threads(int n) { (void)n; }
#endif

void tngo_sgd_update(float* w, const float* v, uint64_t d, float eta) {
    for (uint64_t i = 0; i < d; ++i) {
        float stepv = eta * v[i];
        w[i] = w[i] - stepv;
    }
}
