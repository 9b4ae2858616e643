// tng_encode / tng_decode_aggregate kernels (sm_100a).
//
// Mapping: one warp owns one wire tile of 128 coordinates at a time; lane j holds
// coordinates 4j..4j+3 (one 128-bit load per vector).  The per-tile scale is a
// warp reduction, the stochastic rounding uses one Philox4x32-10 call per lane
// (its four words belong to the lane's four coordinates), and every code word is
// one __ballot_sync: word c*b+p of a tile collects bit p of the symbols of the
// coordinates 4j+c over the 32 lanes j -- which is exactly the wire layout.
//
// Encode follows Eq. 2 / Eq. 3 and Section 3.2 of the paper (normalise, R, z);
// decode follows Algorithm 1's averaging step with the reference put back.
#include "tng_device.cuh"
#include "tng_internal.h"
#include "tng_pipeline.cuh"

namespace tng {

namespace {

enum { kPhaseFused = 0, kPhaseStat = 1, kPhaseQuant = 2 };
constexpr int kCodecThreads = 256;
constexpr int kWorkerBatch = 4;   // gradient rows whose loads are in flight together

// Row strides are 32-bit element counts (the entry points reject longer rows), so that
// "base + m * stride" is one 32 x 32 -> 64-bit multiply-add per address.
struct EncodeArgs {
    const float* grads;
    const float* ref;
    uint32_t* codes;
    float* scales;
    float* tile_stat;
    unsigned long long* nonfinite;
    uint32_t* pipe_error;
    uint64_t d, ntile, block;
    uint64_t tile_begin;   // first tile this launch handles (the staged kernel takes the ones before it)
    uint64_t tile0;        // tile index of local tile 0 within the whole vector: only the Philox counters see it
    uint32_t ld, nblk, wpw;
    uint32_t M, step;
    uint32_t m_base;   // worker index of row 0 (Philox counter word); the wire pointers are already offset
    uint32_t pow24;    // 1 << 24 as a run-time value: x >> 8 is taken as umulhi(x, 2^24)
    uint32_t rk[20];   // Philox round keys (key + r * Weyl), computed once on the host
    int levels;
    float quot_eps;
    // reference fusion inside the encode pass: r = sum_j alpha[j] hist[j] is computed per tile
    // (fp32 fma chain, j ascending) and written to ref_out, instead of being read from `ref`
    const float* hist[kMaxK];
    const float* alpha;
    float* ref_out;
    int hist_k;
    // combined form (TNG_NORM_COMB): second reference r' = (1/k) sum_j |h_j|, read from ref2 or,
    // when the reference is combined here, formed alongside it (weight inv_k) and written to ref2_out
    const float* ref2;
    float* ref2_out;
    float inv_k;
    // scalar reference (TNG_NORM_MEAN): means[m] = mean(g^m) of the launch's worker m
    const float* means;
};

// max(|a|, |b|) that returns NaN if either is NaN
__device__ __forceinline__ float absmax_nan2(float a, float b) {
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(fabsf(a)), "f"(fabsf(b)));
    return r;
}

// operands of the normalisation for the lane's four coordinates: a = r (difference and combined
// forms) or 1/den (quotient form); b = 1/den' (combined form only)
struct NormOp {
    float4 a, b;
};

// the reference(s) of a tile -> normalisation operands
template <int NORM>
__device__ __forceinline__ NormOp make_norm_op(const float4 r, const float4 r2, const float quot_eps) {
    NormOp op;
    op.a = make_float4(0.f, 0.f, 0.f, 0.f);
    op.b = op.a;
    if (NORM == TNG_NORM_DIFF || NORM == TNG_NORM_COMB) op.a = r;
    if (NORM == TNG_NORM_QUOT || NORM == TNG_NORM_COMB) {
        const float4 den = quot_den4(NORM == TNG_NORM_QUOT ? r : r2, quot_eps);
        const float4 inv = make_float4(__frcp_rn(den.x), __frcp_rn(den.y), __frcp_rn(den.z), __frcp_rn(den.w));
        if (NORM == TNG_NORM_QUOT) op.a = inv; else op.b = inv;
    }
    return op;
}

// r' += inv_k * |h| (the second reference's fma chain)
__device__ __forceinline__ void magnitude_fma(float4& r2, const float inv_k, const float4 h) {
    r2.x = __fmaf_rn(inv_k, fabsf(h.x), r2.x); r2.y = __fmaf_rn(inv_k, fabsf(h.y), r2.y);
    r2.z = __fmaf_rn(inv_k, fabsf(h.z), r2.z); r2.w = __fmaf_rn(inv_k, fabsf(h.w), r2.w);
}

template <int NORM>
__device__ __forceinline__ void encode_normalise(const float4 g, const NormOp& opn, float (&v)[4]) {
    const float4 op = opn.a;
    if (NORM == TNG_NORM_COMB) {   // v = (g - r) * (1/den'), two roundings
        v[0] = __fmul_rn(__fsub_rn(g.x, op.x), opn.b.x); v[1] = __fmul_rn(__fsub_rn(g.y, op.y), opn.b.y);
        v[2] = __fmul_rn(__fsub_rn(g.z, op.z), opn.b.z); v[3] = __fmul_rn(__fsub_rn(g.w, op.w), opn.b.w);
        return;
    }
    if (NORM == TNG_NORM_DIFF || NORM == TNG_NORM_MEAN) {
        v[0] = __fsub_rn(g.x, op.x); v[1] = __fsub_rn(g.y, op.y); v[2] = __fsub_rn(g.z, op.z); v[3] = __fsub_rn(g.w, op.w);
    } else if (NORM == TNG_NORM_QUOT) {
        v[0] = __fmul_rn(g.x, op.x); v[1] = __fmul_rn(g.y, op.y); v[2] = __fmul_rn(g.z, op.z); v[3] = __fmul_rn(g.w, op.w);
    } else {
        v[0] = g.x; v[1] = g.y; v[2] = g.z; v[3] = g.w;
    }
}

// the tile's statistic: max |v| (NaN wins) or the pairwise-tree sum of squares
template <int SCALE>
__device__ __forceinline__ float encode_tile_stat(const float (&v)[4]) {
    if (SCALE == 0) {
        const float mx = absmax_nan2(absmax_nan2(v[0], v[1]), absmax_nan2(v[2], v[3]));
        // non-negative floats and NaNs order like their bit patterns
        return __uint_as_float(__reduce_max_sync(kFullMask, __float_as_uint(mx)));
    }
    return warp_sumsq_tree(v[0], v[1], v[2], v[3]);
}

// Stochastic rounding of the lane's four values with scale R; x = the lane's Philox call,
// word c for coordinate 4j+c.  The ballots leave every code word of the tile in every lane.
// A scale that is NaN or infinite needs no special case, nor does a zero max-scale (the block is
// then all zeros): u*0 < 0, NaN < x and inf < x are all false, and (int)NaN is 0, so every symbol
// of such a block is the zero symbol.  The caller replaces a zero L2 scale by NaN.
//
// The integer/logic pipe is the busy one in the encode kernels (Philox xors, compares,
// ballots), so work that can run on the multiplier pipe is put there: addresses are
// 32 x 32 -> 64 multiply-adds and the uniform's shift is a high multiply.
template <int CODEC, bool FULL>
__device__ __forceinline__ void encode_quantise(const EncodeArgs& a, const float (&v)[4], const float R, const uint4 x,
                                                const uint32_t valid, uint32_t (&w)[4 * CODEC]) {
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        // u = (x >> 8) * 2^-24
        const float u = __fmul_rn(__uint2float_rn(__umulhi(xs[c], a.pow24)), 0x1p-24f);
        const bool live = FULL || ((valid >> c) & 1u);
        if (CODEC == TNG_CODEC_TERN2) {
            // nonzero with probability |v|/R  <=>  u*R < |v|
            const bool nz = live && (__fmul_rn(u, R) < fabsf(v[c]));
            const bool neg = nz && (v[c] < 0.0f);
            w[c * 2 + 0] = __ballot_sync(kFullMask, nz);
            w[c * 2 + 1] = __ballot_sync(kFullMask, neg);
        } else if (CODEC == TNG_CODEC_SIGN1) {
            // +R with probability (1 + v/R)/2  <=>  u*R < v/2 + R/2
            const float thr = __fadd_rn(__fmul_rn(0.5f, v[c]), __fmul_rn(0.5f, R));
            const bool plus = live && (__fmul_rn(u, R) < thr);
            w[c] = __ballot_sync(kFullMask, plus);
        } else {
            // s-level: a = (|v|/R) s; level floor(a) (+1 with probability frac(a)), never above s (an L2
            // scale can fall short of |v| when the squares are subnormal; level s+1 would reach the sign plane)
            const float qv = __fdiv_rn(fabsf(v[c]), R);
            const float av = __fmul_rn(qv, (float)a.levels);
            const float lv = floorf(av);
            const float fv = __fsub_rn(av, lv);
            const int L = live ? min((int)lv + ((u < fv) ? 1 : 0), a.levels) : 0;
            const bool neg = (L > 0) && (v[c] < 0.0f);
            w[c * 4 + 0] = __ballot_sync(kFullMask, L & 1);
            w[c * 4 + 1] = __ballot_sync(kFullMask, L & 2);
            w[c * 4 + 2] = __ballot_sync(kFullMask, L & 4);
            w[c * 4 + 3] = __ballot_sync(kFullMask, neg);
        }
    }
}

// The operands worker m normalises with: the tile's, except for the scalar reference, where every
// worker subtracts its own mean (Section 3.1).  Full tiles only (no element past the end).
template <int NORM>
__device__ __forceinline__ NormOp worker_op(const EncodeArgs& a, const NormOp& op, const uint32_t m) {
    if (NORM != TNG_NORM_MEAN) return op;
    NormOp o = op;
    const float mu = __ldg(a.means + m);
    o.a = make_float4(mu, mu, mu, mu);
    return o;
}

template <int CODEC, int NORM, int SCALE, int PHASE, bool FULL>
__device__ __forceinline__ bool encode_symbols(const EncodeArgs& a, const float4 g, const NormOp& op,
                                               const uint32_t m, const uint64_t T, const uint4 x, const uint64_t blk,
                                               const int lane, const uint32_t valid, uint32_t (&w)[4 * CODEC], float& R) {
    float v[4];
    encode_normalise<NORM>(g, op, v);
    if (PHASE != kPhaseQuant) {
        const float stat = encode_tile_stat<SCALE>(v);
        if (PHASE == kPhaseStat) {
            if (lane == 0) a.tile_stat[(uint64_t)m * a.ntile + T] = stat;
            R = 0.0f;
            return false;
        }
        R = (SCALE == 0) ? stat : __fsqrt_rn(stat);
    } else {
        R = __ldg(a.scales + (uint64_t)m * a.nblk + blk);
    }
    // An L2 scale can be zero although the block is not (all squares underflow): the comparisons below
    // would then fire on u*0 < |v|.  A NaN in R's place makes every one of them false: the zero symbol.
    const float Rq = (SCALE == 1 && !(R > 0.0f)) ? __int_as_float(0x7fc00000) : R;
    encode_quantise<CODEC, FULL>(a, v, Rq, x, valid, w);
    return true;
}

// encode_symbols, then lane 0 writes the words every lane holds (and the scale)
template <int CODEC, int NORM, int SCALE, int PHASE, bool FULL>
__device__ __forceinline__ uint32_t encode_worker(const EncodeArgs& a, const float4 g, const NormOp& op,
                                                  const uint32_t m, const uint64_t T, const uint32_t q_lo,
                                                  const uint32_t q_hi, const uint64_t blk, const int lane,
                                                  const uint32_t valid) {
    constexpr int kWords = 4 * CODEC;
    uint32_t w[kWords];
    float R;
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (PHASE != kPhaseStat) x = philox4x32_10_rk(q_lo, q_hi, a.m_base + m, a.step, a.rk);
    NormOp opm = op;
    if (NORM == TNG_NORM_MEAN) {   // the worker's own scalar, the same for every coordinate (Section 3.1)
        // elements past the end of the vector read as zero and must stay zero after the subtraction
        const float mu = __ldg(a.means + m);
        opm.a = make_float4((valid & 1u) ? mu : 0.0f, (valid & 2u) ? mu : 0.0f, (valid & 4u) ? mu : 0.0f, (valid & 8u) ? mu : 0.0f);
    }
    if (!encode_symbols<CODEC, NORM, SCALE, PHASE, FULL>(a, g, opm, m, T, x, blk, lane, valid, w, R)) return 0u;
    if (lane == 0) {
        uint4* dst = reinterpret_cast<uint4*>(a.codes + ((uint64_t)m * a.wpw + T * (uint64_t)kWords));
#pragma unroll
        for (int q4 = 0; q4 < CODEC; ++q4) __stcs(dst + q4, make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]));
        if (PHASE == kPhaseFused) a.scales[(uint64_t)m * a.nblk + T] = R;
    }
    return __float_as_uint(R);
}

template <int CODEC, int NORM, int SCALE, int PHASE, bool FULL, bool FUSEREF>
__device__ __forceinline__ void encode_tile(const EncodeArgs& a, const float* s_alpha, const uint64_t T, const int lane) {
    const uint64_t i0 = T * kTile + (uint64_t)lane * 4u;
    uint32_t valid = 0xFu;
    if (!FULL) {
        valid = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) valid |= (i0 + c < a.d) ? (1u << c) : 0u;
    }
    const float* gp = a.grads + i0;
    auto load_row = [&](uint32_t m) -> float4 {
        const float* row = gp + (uint64_t)m * a.ld;
        return FULL ? __ldcs(reinterpret_cast<const float4*>(row)) : load4_stream(row - i0, i0, a.d);
    };
    // the first batch of gradient rows is requested before anything is computed
    float4 g[kWorkerBatch];
#pragma unroll
    for (int k = 0; k < kWorkerBatch; ++k)
        if ((uint32_t)k < a.M) g[k] = load_row(k);

    NormOp op = make_norm_op<TNG_NORM_NONE>(make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f), 0.f);
    if (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN) {
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f), r2 = r;
        if (FUSEREF) {
            for (int j0 = 0; j0 < a.hist_k; j0 += 4) {
                float4 h[4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    if (j0 + jj < a.hist_k)
                        h[jj] = FULL ? __ldcs(reinterpret_cast<const float4*>(a.hist[j0 + jj] + i0)) : load4_stream(a.hist[j0 + jj], i0, a.d);
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    if (j0 + jj < a.hist_k) {
                        const float al = s_alpha[j0 + jj];
                        r.x = __fmaf_rn(al, h[jj].x, r.x); r.y = __fmaf_rn(al, h[jj].y, r.y);
                        r.z = __fmaf_rn(al, h[jj].z, r.z); r.w = __fmaf_rn(al, h[jj].w, r.w);
                        if (NORM == TNG_NORM_COMB) magnitude_fma(r2, a.inv_k, h[jj]);
                    }
            }
            if (FULL) *reinterpret_cast<float4*>(a.ref_out + i0) = r;
            else store4(a.ref_out, i0, a.d, r);
            if (NORM == TNG_NORM_COMB) {
                if (FULL) *reinterpret_cast<float4*>(a.ref2_out + i0) = r2;
                else store4(a.ref2_out, i0, a.d, r2);
            }
        } else {
            if (a.ref) r = FULL ? *reinterpret_cast<const float4*>(a.ref + i0) : load4(a.ref, i0, a.d);
            if (NORM == TNG_NORM_COMB && a.ref2) r2 = FULL ? *reinterpret_cast<const float4*>(a.ref2 + i0) : load4(a.ref2, i0, a.d);
        }
        op = make_norm_op<NORM>(r, r2, a.quot_eps);
    }
    const uint64_t blk = (PHASE == kPhaseQuant) ? (T * kTile) / a.block : T;
    const uint64_t q = (T + a.tile0) * 32u + (uint32_t)lane;     // Philox counter of the lane's four coordinates
    const uint32_t q_lo = (uint32_t)q, q_hi = (uint32_t)(q >> 32);
    uint32_t rmax = 0;                                           // largest scale bit pattern of the tile
    // batches of rows; the next batch is in flight while the current one is encoded
    const uint32_t m_batched = a.M - a.M % kWorkerBatch;
    for (uint32_t m0 = 0; m0 < m_batched; m0 += kWorkerBatch) {
        float4 gn[kWorkerBatch];
#pragma unroll
        for (int k = 0; k < kWorkerBatch; ++k)
            if (m0 + kWorkerBatch + k < a.M) gn[k] = load_row(m0 + kWorkerBatch + k);
#pragma unroll
        for (int k = 0; k < kWorkerBatch; ++k)
            rmax = max(rmax, encode_worker<CODEC, NORM, SCALE, PHASE, FULL>(a, g[k], op, m0 + k, T, q_lo, q_hi, blk, lane, valid));
#pragma unroll
        for (int k = 0; k < kWorkerBatch; ++k) g[k] = gn[k];
    }
#pragma unroll
    for (int k = 0; k < kWorkerBatch - 1; ++k)
        if (m_batched + k < a.M)
            rmax = max(rmax, encode_worker<CODEC, NORM, SCALE, PHASE, FULL>(a, g[k], op, m_batched + k, T, q_lo, q_hi, blk, lane, valid));
    // NaN or +inf scales are rare: only then count them, from the scales just written
    if (PHASE == kPhaseFused && rmax >= 0x7f800000u && lane == 0) {
        unsigned long long bad = 0;
        for (uint32_t m = 0; m < a.M; ++m) bad += (__float_as_uint(a.scales[(uint64_t)m * a.nblk + T]) >= 0x7f800000u) ? 1ull : 0ull;
        atomicAdd(a.nonfinite, bad);
    }
}

// Persistent grid: warp w of the grid takes tiles w, w + nwarps, ...; at any moment the
// grid works on one contiguous window of every input row.  Only the last tile can be
// ragged; it runs the bounds-checked instantiation.
template <int CODEC, int NORM, int SCALE, int PHASE, bool FUSEREF>
__global__ void __launch_bounds__(kCodecThreads, 2) encode_kernel(const EncodeArgs a) {
    __shared__ float s_alpha[kMaxK];
    if (FUSEREF) {
        if (threadIdx.x < kMaxK) s_alpha[threadIdx.x] = ((int)threadIdx.x < a.hist_k) ? a.alpha[threadIdx.x] : 0.0f;
        __syncthreads();
    }
    const int lane = threadIdx.x & 31;
    const uint64_t warps_per_cta = kCodecThreads / 32;
    const uint64_t nwarps = (uint64_t)gridDim.x * warps_per_cta;
    const uint64_t gwarp = (uint64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5);
    const uint64_t nfull = a.d / kTile;
    for (uint64_t T = a.tile_begin + gwarp; T < nfull; T += nwarps) encode_tile<CODEC, NORM, SCALE, PHASE, true, FUSEREF>(a, s_alpha, T, lane);
    if (nfull < a.ntile && gwarp == nfull % nwarps) encode_tile<CODEC, NORM, SCALE, PHASE, false, FUSEREF>(a, s_alpha, nfull, lane);
}

// Predicated 16-byte stores of a tile's code words (no branch around them).
template <int CODEC>
__device__ __forceinline__ void store_words_if(const bool pred, uint32_t* dst, const uint32_t (&w)[4 * CODEC]) {
#pragma unroll
    for (int q4 = 0; q4 < CODEC; ++q4)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p st.global.cs.v4.u32 [%1], {%2, %3, %4, %5};\n\t}" ::"r"((uint32_t)pred),
                     "l"(dst + 4 * q4), "r"(w[4 * q4]), "r"(w[4 * q4 + 1]), "r"(w[4 * q4 + 2]), "r"(w[4 * q4 + 3]));
}

// ---------------------------------------------------------------------------
// Encode fed by the bulk-copy pipeline (one scale per tile, full tiles only).
// Row list: the rows that make the reference (the k history rows when the reference is
// combined here, else the reference itself, else nothing), then the M gradient rows.
// A chunk of 2048 coordinates = 16 tiles, one per compute warp; a stage holds up to 8
// rows of one kind.  Per chunk a warp first forms its tile's reference from the
// reference fill(s), then encodes the gradient rows fill by fill, eight workers
// unrolled.  Everything a warp computes is what encode_tile computes; only where the
// operands come from differs.
// ---------------------------------------------------------------------------
using EncGeom = PipeGeom<2048, 8, 3>;
constexpr int kEncPipeWarps = EncGeom::kChunk / kTile;     // 16
constexpr int kEncPipeThreads = kEncPipeWarps * 32 + 32;   // + the producer warp
constexpr uint64_t kEncPipeMinChunks = 8;                  // shorter vectors take the direct kernel
constexpr int kPhiloxBatch = 2;                            // Philox calls whose rounds are interleaved

struct EncodePipeArgs {
    EncodeArgs e;
    PipeRows rows;
};

template <int CODEC, int NORM, int SCALE, bool FUSEREF>
__global__ void __launch_bounds__(kEncPipeThreads, 1) encode_pipe_kernel(const EncodePipeArgs pa) {
    using G = EncGeom;
    extern __shared__ unsigned char dyn_smem[];
    __shared__ float s_alpha[kMaxK];
    const EncodeArgs& a = pa.e;
    if (FUSEREF && threadIdx.x < kMaxK) s_alpha[threadIdx.x] = ((int)threadIdx.x < a.hist_k) ? a.alpha[threadIdx.x] : 0.0f;
    const PipeSmem pipe = pipe_setup<G>(dyn_smem, kEncPipeWarps);   // ends with __syncthreads
    const uint64_t nchunks = a.tile_begin / kEncPipeWarps;          // the chunks ahead of the directly read tiles
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == kEncPipeWarps) {
        if (lane == 0) {
            const uint32_t err = pipe_produce<G>(pipe, pa.rows, blockIdx.x, gridDim.x, nchunks);
            if (err != kPipeOk) atomicMax(a.pipe_error, err);
        }
        return;
    }
    const uint32_t my = (uint32_t)warp * (kTile * 4u) + (uint32_t)lane * 16u;   // byte offset inside a row chunk
    // the stages as ordinary shared memory: plain loads, which the compiler may interleave freely
    // with the arithmetic of neighbouring workers (the barrier waits are memory fences for it)
    const unsigned char* stages = dyn_smem + (pipe.data - smem_u32(dyn_smem));
    const int n_pre = pa.rows.n_pre;
    const uint32_t M = a.M;
    uint32_t it = 0;
    for (uint64_t c = blockIdx.x; c < nchunks; c += gridDim.x) {
        const uint64_t T = c * kEncPipeWarps + (uint32_t)warp;
        const uint64_t q = (T + a.tile0) * 32u + (uint32_t)lane;
        const uint32_t q_lo = (uint32_t)q, q_hi = (uint32_t)(q >> 32);
        // ---- the reference(s) of the tile
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f), r2 = r;
        for (int p0 = 0; p0 < n_pre; p0 += G::kRows) {
            const int n = (n_pre - p0 < G::kRows) ? n_pre - p0 : G::kRows;
            const uint32_t s = it % G::kStages, use = it / G::kStages;
            if (!__all_sync(kFullMask, mbar_wait(pipe.full(s), use & 1u))) {   // warp-uniform outcome
                atomicMax(a.pipe_error, (uint32_t)kPipeFullTimeout);
                return;
            }
            const unsigned char* base = stages + s * G::kStageBytes + my;
            if (FUSEREF) {
                for (int j = 0; j < n; ++j) {
                    const float4 x = *reinterpret_cast<const float4*>(base + (uint32_t)j * G::kRowBytes);
                    const float al = s_alpha[p0 + j];
                    r.x = __fmaf_rn(al, x.x, r.x); r.y = __fmaf_rn(al, x.y, r.y);
                    r.z = __fmaf_rn(al, x.z, r.z); r.w = __fmaf_rn(al, x.w, r.w);
                    if (NORM == TNG_NORM_COMB) magnitude_fma(r2, a.inv_k, x);
                }
            } else {   // the reference itself, then (combined form) the second reference
                r = *reinterpret_cast<const float4*>(base);
                if (NORM == TNG_NORM_COMB && n > 1) r2 = *reinterpret_cast<const float4*>(base + G::kRowBytes);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(pipe.empty(s));
            ++it;
        }
        if (FUSEREF) {
            *reinterpret_cast<float4*>(a.ref_out + (T * kTile + (uint64_t)lane * 4u)) = r;
            if (NORM == TNG_NORM_COMB) *reinterpret_cast<float4*>(a.ref2_out + (T * kTile + (uint64_t)lane * 4u)) = r2;
        }
        const NormOp op = make_norm_op<NORM>(r, r2, a.quot_eps);
        // ---- the gradient rows, one fill of up to 8 workers at a time.  Every lane ends up with
        // all words of every worker; lane k writes worker k of the fill through a pointer it
        // computes once per fill, and the fill's scales go out as one store.
        constexpr int kWords = 4 * CODEC;
        for (uint32_t m0 = 0; m0 < M; m0 += G::kRows) {
            const uint32_t s = it % G::kStages, use = it / G::kStages;
            if (!__all_sync(kFullMask, mbar_wait(pipe.full(s), use & 1u))) {
                atomicMax(a.pipe_error, (uint32_t)kPipeFullTimeout);
                return;
            }
            const unsigned char* base = stages + s * G::kStageBytes + my;
            const uint32_t mine = m0 + (uint32_t)lane;                       // the worker this lane writes
            uint32_t* my_codes = a.codes + ((uint64_t)mine * a.wpw + T * (uint64_t)kWords);
            float my_R = 0.0f;
            if (m0 + G::kRows <= M) {
                // Copy the warp's share of the fill into registers and hand the stage back at once:
                // the copy engine can refill it while the arithmetic below runs, so loads stay in
                // flight all the time instead of in bursts at the end of every fill.
                float4 g[G::kRows];
#pragma unroll
                for (int k = 0; k < G::kRows; ++k) g[k] = *reinterpret_cast<const float4*>(base + (uint32_t)k * G::kRowBytes);
                __syncwarp();
                if (lane == 0) mbar_arrive(pipe.empty(s));
#pragma unroll
                for (int k0 = 0; k0 < G::kRows; k0 += kPhiloxBatch) {
                    uint4 x[kPhiloxBatch];
                    philox4x32_10_rk_batch<kPhiloxBatch>(q_lo, q_hi, a.m_base + m0 + k0, a.step, a.rk, x);
#pragma unroll
                    for (int kk = 0; kk < kPhiloxBatch; ++kk) {
                        const int k = k0 + kk;
                        uint32_t w[kWords];
                        float R;
                        encode_symbols<CODEC, NORM, SCALE, kPhaseFused, true>(a, g[k], worker_op<NORM>(a, op, m0 + k), m0 + k, T, x[kk], T, lane,
                                                                               0xFu, w, R);
                        store_words_if<CODEC>(lane == k, my_codes, w);
                        my_R = (lane == k) ? R : my_R;
                    }
                }
            } else {
                for (uint32_t k = 0; m0 + k < M; ++k) {
                    const float4 g = *reinterpret_cast<const float4*>(base + k * G::kRowBytes);
                    uint32_t w[kWords];
                    float R;
                    const uint4 x = philox4x32_10_rk(q_lo, q_hi, a.m_base + m0 + k, a.step, a.rk);
                    encode_symbols<CODEC, NORM, SCALE, kPhaseFused, true>(a, g, worker_op<NORM>(a, op, m0 + k), m0 + k, T, x, T, lane, 0xFu, w, R);
                    store_words_if<CODEC>((uint32_t)lane == k, my_codes, w);
                    my_R = ((uint32_t)lane == k) ? R : my_R;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(pipe.empty(s));   // this warp has read the stage
            }
            const bool writes = lane < G::kRows && mine < M;
            if (writes) a.scales[(uint64_t)mine * a.nblk + T] = my_R;
            // NaN or +inf scales (rare) are counted from the lanes that hold them
            const uint32_t bad = __ballot_sync(kFullMask, writes && __float_as_uint(my_R) >= 0x7f800000u);
            if (bad != 0u && lane == 0) atomicAdd(a.nonfinite, (unsigned long long)__popc(bad));
            ++it;
        }
    }
}

// ---------------------------------------------------------------------------
// The same pass when one scale spans 2, 4, 8 or 16 tiles (blocks of 256 .. 2048
// coordinates, all inside one chunk): the gradient rows are still read once.  Per fill a
// warp normalises its tile for the (up to) eight workers, keeps the values in registers and
// posts the eight tile statistics in shared memory; after a barrier among the warps of the block
// (each group of 2 .. 16 warps has a hardware barrier of its own, so groups do not wait for one
// another), lane k of every warp combines the statistics of its block for worker k (maximum, or
// the adjacent-pairwise sum that continues the tree inside the tiles; slots beyond the block count
// as zero, the identity of both) and the warp quantises from registers.  Statistics and the
// group's give-up flag are double-buffered, so one barrier per fill is enough: a warp can only run
// one fill ahead of the slowest one of its group.  A warp whose bounded wait runs out raises its
// group's flag and still arrives at the fill's barrier; after it all warps of the group see the flag
// and leave together, so nobody is left waiting at a barrier (the other groups then run out of
// stages, since a stage is only refilled once all sixteen warps have released it, and leave the same way).
// ---------------------------------------------------------------------------
// barrier among the warps of one scale block: hardware barrier 1 + group, `threads` = 32 x warps per block
__device__ __forceinline__ void block_warps_barrier(const int group, const int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "r"(threads) : "memory");
}

template <int CODEC, int NORM, int SCALE, bool FUSEREF>
__global__ void __launch_bounds__(kEncPipeThreads, 1) encode_pipe_blocks_kernel(const EncodePipeArgs pa) {
    using G = EncGeom;
    extern __shared__ unsigned char dyn_smem[];
    __shared__ float s_alpha[kMaxK];
    __shared__ float s_stat[2][G::kRows][kEncPipeWarps + 1];
    __shared__ uint32_t s_gave_up[kEncPipeWarps / 2][2];   // per group of warps that share a block, per buffer
    const EncodeArgs& a = pa.e;
    if (FUSEREF && threadIdx.x < kMaxK) s_alpha[threadIdx.x] = ((int)threadIdx.x < a.hist_k) ? a.alpha[threadIdx.x] : 0.0f;
    if (threadIdx.x < kEncPipeWarps) s_gave_up[threadIdx.x / 2][threadIdx.x % 2] = 0u;
    const PipeSmem pipe = pipe_setup<G>(dyn_smem, kEncPipeWarps);   // ends with __syncthreads
    const uint64_t nchunks = a.tile_begin / kEncPipeWarps;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == kEncPipeWarps) {
        if (lane == 0) {
            const uint32_t err = pipe_produce<G>(pipe, pa.rows, blockIdx.x, gridDim.x, nchunks);
            if (err != kPipeOk) atomicMax(a.pipe_error, err);
        }
        return;
    }
    const uint32_t my = (uint32_t)warp * (kTile * 4u) + (uint32_t)lane * 16u;
    const unsigned char* stages = dyn_smem + (pipe.data - smem_u32(dyn_smem));
    const int n_pre = pa.rows.n_pre;
    const uint32_t M = a.M;
    const int tpb = (int)(a.block / kTile);                // tiles per block: 2, 4, 8 or 16
    const int block_warp0 = warp & ~(tpb - 1);             // first warp (tile) of this warp's block within the chunk
    const int group = warp / tpb;                          // the warps of one block meet on their own barrier
    constexpr int kWords = 4 * CODEC;
    uint32_t it = 0, buf = 0;
    bool alive = true;
    for (uint64_t c = blockIdx.x; c < nchunks; c += gridDim.x) {
        const uint64_t T = c * kEncPipeWarps + (uint32_t)warp;
        const uint64_t blk = T / (uint32_t)tpb;
        const uint64_t q = (T + a.tile0) * 32u + (uint32_t)lane;
        const uint32_t q_lo = (uint32_t)q, q_hi = (uint32_t)(q >> 32);
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f), r2 = r;
        for (int p0 = 0; p0 < n_pre && alive; p0 += G::kRows) {
            const int n = (n_pre - p0 < G::kRows) ? n_pre - p0 : G::kRows;
            const uint32_t s = it % G::kStages, use = it / G::kStages;
            if (!__all_sync(kFullMask, mbar_wait(pipe.full(s), use & 1u))) {
                atomicMax(a.pipe_error, (uint32_t)kPipeFullTimeout);
                s_gave_up[group][buf] = 1u;
                alive = false;
                break;
            }
            const unsigned char* base = stages + s * G::kStageBytes + my;
            if (FUSEREF) {
                for (int j = 0; j < n; ++j) {
                    const float4 x = *reinterpret_cast<const float4*>(base + (uint32_t)j * G::kRowBytes);
                    const float al = s_alpha[p0 + j];
                    r.x = __fmaf_rn(al, x.x, r.x); r.y = __fmaf_rn(al, x.y, r.y);
                    r.z = __fmaf_rn(al, x.z, r.z); r.w = __fmaf_rn(al, x.w, r.w);
                    if (NORM == TNG_NORM_COMB) magnitude_fma(r2, a.inv_k, x);
                }
            } else {
                r = *reinterpret_cast<const float4*>(base);
                if (NORM == TNG_NORM_COMB && n > 1) r2 = *reinterpret_cast<const float4*>(base + G::kRowBytes);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(pipe.empty(s));
            ++it;
        }
        if (FUSEREF && alive) {
            *reinterpret_cast<float4*>(a.ref_out + (T * kTile + (uint64_t)lane * 4u)) = r;
            if (NORM == TNG_NORM_COMB) *reinterpret_cast<float4*>(a.ref2_out + (T * kTile + (uint64_t)lane * 4u)) = r2;
        }
        const NormOp op = make_norm_op<NORM>(r, r2, a.quot_eps);
        for (uint32_t m0 = 0; m0 < M; m0 += G::kRows) {
            float v[G::kRows][4];
            float my_stat = 0.0f;
            if (alive) {
                const uint32_t s = it % G::kStages, use = it / G::kStages;
                if (!__all_sync(kFullMask, mbar_wait(pipe.full(s), use & 1u))) {
                    atomicMax(a.pipe_error, (uint32_t)kPipeFullTimeout);
                    s_gave_up[group][buf] = 1u;
                    alive = false;
                }
                if (alive) {
                    const unsigned char* base = stages + s * G::kStageBytes + my;
#pragma unroll
                    for (int k = 0; k < G::kRows; ++k) {
                        if (m0 + k < M) {   // the same answer in every thread of the grid
                            const float4 g = *reinterpret_cast<const float4*>(base + (uint32_t)k * G::kRowBytes);
                            encode_normalise<NORM>(g, worker_op<NORM>(a, op, m0 + k), v[k]);
                            const float st = encode_tile_stat<SCALE>(v[k]);
                            my_stat = (lane == k) ? st : my_stat;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(pipe.empty(s));
                    ++it;
                    if (lane < G::kRows) s_stat[buf][lane][warp] = my_stat;
                }
            }
            // the first random numbers do not depend on the scale: drawn before the barrier, they fill the wait
            uint4 x[kPhiloxBatch];
            philox4x32_10_rk_batch<kPhiloxBatch>(q_lo, q_hi, a.m_base + m0, a.step, a.rk, x);
            block_warps_barrier(group, tpb * 32);
            if (s_gave_up[group][buf] != 0u) return;       // the same answer in all warps of the block
            // lane k: the block's statistic for worker k of the fill (two tiles per block, the common case, apart)
            const float* mine_stat = &s_stat[buf][lane & (G::kRows - 1)][block_warp0];
            auto join = [](const float p, const float q) {
                return (SCALE == 0) ? __uint_as_float(max(__float_as_uint(p), __float_as_uint(q))) : __fadd_rn(p, q);
            };
            float block_stat;
            if (tpb == 2) {
                block_stat = join(mine_stat[0], mine_stat[1]);
            } else {
                float bs[kEncPipeWarps];
#pragma unroll
                for (int t = 0; t < kEncPipeWarps; ++t) bs[t] = (t < tpb) ? mine_stat[t] : 0.0f;
#pragma unroll
                for (int len = kEncPipeWarps; len > 1; len >>= 1)
#pragma unroll
                    for (int t = 0; t < len / 2; ++t) bs[t] = join(bs[2 * t], bs[2 * t + 1]);
                block_stat = bs[0];
            }
            const float my_R = (SCALE == 0) ? block_stat : __fsqrt_rn(block_stat);
            const uint32_t mine = m0 + (uint32_t)lane;
            uint32_t* my_codes = a.codes + ((uint64_t)mine * a.wpw + T * (uint64_t)kWords);
#pragma unroll
            for (int k0 = 0; k0 < G::kRows; k0 += kPhiloxBatch) {
                if (m0 + k0 < M) {
                    if (k0 > 0) philox4x32_10_rk_batch<kPhiloxBatch>(q_lo, q_hi, a.m_base + m0 + k0, a.step, a.rk, x);
#pragma unroll
                    for (int kk = 0; kk < kPhiloxBatch; ++kk) {
                        const int k = k0 + kk;
                        if (m0 + k < M) {
                            const float R = __shfl_sync(kFullMask, my_R, k);
                            const float Rq = (SCALE == 1 && !(R > 0.0f)) ? __int_as_float(0x7fc00000) : R;
                            uint32_t w[kWords];
                            encode_quantise<CODEC, true>(a, v[k], Rq, x[kk], 0xFu, w);
                            store_words_if<CODEC>(lane == k, my_codes, w);
                        }
                    }
                }
            }
            // the first warp of a block writes its scales
            const bool writes = warp == block_warp0 && lane < G::kRows && mine < M;
            if (writes) a.scales[(uint64_t)mine * a.nblk + blk] = my_R;
            const uint32_t bad = __ballot_sync(kFullMask, writes && __float_as_uint(my_R) >= 0x7f800000u);
            if (bad != 0u && lane == 0) atomicAdd(a.nonfinite, (unsigned long long)__popc(bad));
            buf ^= 1u;
        }
    }
}

// Scalar reference (Section 3.1), first pass: the sum of every tile of every row, as the
// adjacent-pairwise fp32 tree (the lane's four values pairwise, then xor-shuffles pair
// neighbouring lanes); elements past the end count as zero.  The tree over the tiles and
// the division by d follow in block_scale_level_kernel<kTreeSum>.
__global__ void __launch_bounds__(kCodecThreads) row_tile_sum_kernel(const float* __restrict__ grads, uint32_t ld, uint32_t M,
                                                                       uint64_t d, uint64_t ntile, float* __restrict__ tile_sum) {
    const int lane = threadIdx.x & 31;
    const uint64_t nwarps = (uint64_t)gridDim.x * (kCodecThreads / 32);
    for (uint64_t T = (uint64_t)blockIdx.x * (kCodecThreads / 32) + (threadIdx.x >> 5); T < ntile; T += nwarps) {
        const uint64_t i0 = T * kTile + (uint64_t)lane * 4u;
        for (uint32_t m = 0; m < M; ++m) {
            const float4 g = load4_stream(grads + (uint64_t)m * ld, i0, d);
            float s = __fadd_rn(__fadd_rn(g.x, g.y), __fadd_rn(g.z, g.w));
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) s = __fadd_rn(s, __shfl_xor_sync(kFullMask, s, off));
            if (lane == 0) tile_sum[(uint64_t)m * ntile + T] = s;
        }
    }
}

// One level of the per-block scale reduction.  Row m holds n_in entries split
// into segments of `seg` entries (the last one ragged); CTA (segment, chunk)
// reduces entries [chunk*1024, chunk*1024+1024) of its segment, zero-padded, with
// an adjacent-pairwise tree (sum) or a NaN-propagating max, and writes one value.
// At the last level (chunks_per_seg == 1, final = 1) the value becomes the scale.
// SCALE 2 is the plain sum behind the scalar reference: its last level divides by `divisor`
// (the vector length) and the value becomes the worker's mean.
constexpr int kTreeSum = 2;

// The tree over 1024 shared-memory entries (256 threads, all of them call): adjacent pairs level by
// level, a sum (SCALE 1, 2) or the maximum of the bit patterns (SCALE 0: non-negative floats and NaNs
// order like their patterns).  The result is left in buf[0], visible to every thread.
template <int SCALE>
__device__ __forceinline__ void cta_tree_1024(float* buf) {
    for (int len = 1024; len > 1; len >>= 1) {
        float t0 = 0.f, t1 = 0.f;
        const int i0 = threadIdx.x, i1 = threadIdx.x + 256;
        if (i0 < len / 2) {
            t0 = (SCALE == 0) ? __uint_as_float(max(__float_as_uint(buf[2 * i0]), __float_as_uint(buf[2 * i0 + 1])))
                              : __fadd_rn(buf[2 * i0], buf[2 * i0 + 1]);
        }
        if (i1 < len / 2) {
            t1 = (SCALE == 0) ? __uint_as_float(max(__float_as_uint(buf[2 * i1]), __float_as_uint(buf[2 * i1 + 1])))
                              : __fadd_rn(buf[2 * i1], buf[2 * i1 + 1]);
        }
        __syncthreads();
        if (i0 < len / 2) buf[i0] = t0;
        if (i1 < len / 2) buf[i1] = t1;
        __syncthreads();
    }
}

template <int SCALE>
__global__ void __launch_bounds__(256) block_scale_level_kernel(const float* __restrict__ in, uint64_t n_in,
                                                                uint64_t seg, uint64_t chunks_per_seg,
                                                                float* __restrict__ out, uint64_t n_out,
                                                                int final, float divisor, unsigned long long* nonfinite) {
    __shared__ float buf[1024];
    const uint64_t s = blockIdx.x, c = blockIdx.y, m = blockIdx.z;
    const uint64_t seg_lo = s * seg;
    const uint64_t seg_hi = (seg_lo + seg < n_in) ? seg_lo + seg : n_in;
    const uint64_t lo = seg_lo + c * 1024u;
    const float* row = in + m * n_in;
    for (int i = threadIdx.x; i < 1024; i += 256) buf[i] = (lo + i < seg_hi) ? row[lo + i] : 0.0f;
    __syncthreads();
    cta_tree_1024<SCALE>(buf);
    if (threadIdx.x == 0) {
        float r = buf[0];
        if (final) {
            if (SCALE == 1) r = __fsqrt_rn(r);
            if (SCALE == kTreeSum) r = __fdiv_rn(r, divisor);
            if (!(fabsf(r) < __int_as_float(0x7f800000))) atomicAdd(nonfinite, 1ull);
        }
        out[m * n_out + s * chunks_per_seg + c] = r;
    }
}

// The same reduction for blocks of at most 32 tiles (there can be millions of them): one warp per (block,
// worker), a lane per tile, xor-shuffles pair neighbouring lanes.  Zero-padding to 32 entries instead of to the
// next power of two only appends additions of zero (or maxima with zero), so the value is the same.
template <int SCALE>
__global__ void __launch_bounds__(256) block_scale_warp_kernel(const float* __restrict__ in, uint64_t n_in, uint32_t seg,
                                                               float* __restrict__ out, uint64_t n_out, uint64_t nblk,
                                                               uint32_t M, unsigned long long* nonfinite) {
    const int lane = threadIdx.x & 31;
    const uint64_t nwarps = (uint64_t)gridDim.x * 8u;
    for (uint64_t job = (uint64_t)blockIdx.x * 8u + (threadIdx.x >> 5); job < nblk * M; job += nwarps) {
        const uint64_t m = job / nblk, blk = job % nblk;
        const uint64_t t = blk * seg + (uint32_t)lane;
        float x = ((uint32_t)lane < seg && t < n_in) ? in[m * n_in + t] : 0.0f;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float y = __shfl_xor_sync(kFullMask, x, off);
            x = (SCALE == 0) ? __uint_as_float(max(__float_as_uint(x), __float_as_uint(y))) : __fadd_rn(x, y);
        }
        if (lane == 0) {
            const float r = (SCALE == 1) ? __fsqrt_rn(x) : x;
            if (!(fabsf(r) < __int_as_float(0x7f800000))) atomicAdd(nonfinite, 1ull);
            out[m * n_out + blk] = r;
        }
    }
}

// ---------------------------------------------------------------------------
// Short problems (a per-vector scale at small d, odd block sizes of short vectors): the three
// launches statistic -> tree -> quantise are latency, not bandwidth.  Here one CTA owns one
// scale block of one worker (at most 1024 tiles): its warps compute the tile statistics into
// shared memory, the CTA runs the same tree as block_scale_level_kernel, and the warps go over
// the tiles again (now cache-resident) to quantise.  One launch.
// ---------------------------------------------------------------------------
template <int CODEC, int NORM, int SCALE>
__global__ void __launch_bounds__(256) encode_block_cta_kernel(const EncodeArgs a) {
    __shared__ float buf[1024];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t m = blockIdx.y;
    const uint64_t blk = blockIdx.x;
    const uint64_t seg = (a.block + kTile - 1) / kTile;                 // tiles per block, <= 1024
    const uint64_t t0 = blk * seg;
    const uint64_t t1 = (t0 + seg < a.ntile) ? t0 + seg : a.ntile;
    const float* row = a.grads + (uint64_t)m * a.ld;
    const float mu = (NORM == TNG_NORM_MEAN) ? __ldg(a.means + m) : 0.0f;
    constexpr int kWords = 4 * CODEC;

    // the lane's four normalised values of tile T, and which of them exist
    auto tile_values = [&](const uint64_t T, float (&v)[4], uint32_t& valid) {
        const uint64_t i0 = T * kTile + (uint64_t)lane * 4u;
        valid = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) valid |= (i0 + c < a.d) ? (1u << c) : 0u;
        const float4 g = load4(row, i0, a.d);
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f), r2 = r;
        if (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN) {
            if (a.ref) r = load4(a.ref, i0, a.d);
            if (NORM == TNG_NORM_COMB && a.ref2) r2 = load4(a.ref2, i0, a.d);
        }
        NormOp op = make_norm_op<NORM>(r, r2, a.quot_eps);
        if (NORM == TNG_NORM_MEAN)   // elements past the end read as zero and stay zero
            op.a = make_float4((valid & 1u) ? mu : 0.0f, (valid & 2u) ? mu : 0.0f, (valid & 4u) ? mu : 0.0f, (valid & 8u) ? mu : 0.0f);
        encode_normalise<NORM>(g, op, v);
    };

    for (int i = threadIdx.x; i < 1024; i += 256) buf[i] = 0.0f;
    __syncthreads();
    for (uint64_t T = t0 + (uint32_t)warp; T < t1; T += 8) {
        float v[4];
        uint32_t valid;
        tile_values(T, v, valid);
        const float st = encode_tile_stat<SCALE>(v);
        if (lane == 0) buf[T - t0] = st;
    }
    __syncthreads();
    cta_tree_1024<SCALE>(buf);
    const float R = (SCALE == 0) ? buf[0] : __fsqrt_rn(buf[0]);
    if (threadIdx.x == 0) {
        a.scales[(uint64_t)m * a.nblk + blk] = R;
        if (!(fabsf(R) < __int_as_float(0x7f800000))) atomicAdd(a.nonfinite, 1ull);
    }
    const float Rq = (SCALE == 1 && !(R > 0.0f)) ? __int_as_float(0x7fc00000) : R;
    for (uint64_t T = t0 + (uint32_t)warp; T < t1; T += 8) {
        float v[4];
        uint32_t valid;
        tile_values(T, v, valid);
        const uint64_t q = (T + a.tile0) * 32u + (uint32_t)lane;
        const uint4 x = philox4x32_10_rk((uint32_t)q, (uint32_t)(q >> 32), a.m_base + m, a.step, a.rk);
        uint32_t w[kWords];
        encode_quantise<CODEC, false>(a, v, Rq, x, valid, w);
        if (lane == 0) {
            uint4* dst = reinterpret_cast<uint4*>(a.codes + ((uint64_t)m * a.wpw + T * (uint64_t)kWords));
#pragma unroll
            for (int q4 = 0; q4 < CODEC; ++q4) dst[q4] = make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
        }
    }
}

template <int CODEC, int NORM>
cudaError_t encode_block_cta_scale(const EncodeArgs& a, int scale, dim3 grid, cudaStream_t st) {
    if (scale == 0) encode_block_cta_kernel<CODEC, NORM, 0><<<grid, 256, 0, st>>>(a);
    else encode_block_cta_kernel<CODEC, NORM, 1><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}
template <int CODEC>
cudaError_t encode_block_cta_norm(const EncodeArgs& a, int norm, int scale, dim3 grid, cudaStream_t st) {
    switch (norm) {
        case TNG_NORM_DIFF: return encode_block_cta_scale<CODEC, TNG_NORM_DIFF>(a, scale, grid, st);
        case TNG_NORM_QUOT: return encode_block_cta_scale<CODEC, TNG_NORM_QUOT>(a, scale, grid, st);
        case TNG_NORM_COMB: return encode_block_cta_scale<CODEC, TNG_NORM_COMB>(a, scale, grid, st);
        case TNG_NORM_MEAN: return encode_block_cta_scale<CODEC, TNG_NORM_MEAN>(a, scale, grid, st);
        default: return encode_block_cta_scale<CODEC, TNG_NORM_NONE>(a, scale, grid, st);
    }
}
cudaError_t encode_block_cta_dispatch(const EncodeArgs& a, int codec, int norm, int scale, dim3 grid, cudaStream_t st) {
    switch (codec) {
        case TNG_CODEC_SIGN1: return encode_block_cta_norm<TNG_CODEC_SIGN1>(a, norm, scale, grid, st);
        case TNG_CODEC_TERN2: return encode_block_cta_norm<TNG_CODEC_TERN2>(a, norm, scale, grid, st);
        default: return encode_block_cta_norm<TNG_CODEC_QSGD4>(a, norm, scale, grid, st);
    }
}

struct DecodeArgs {
    const uint32_t* codes;
    const float* scales;
    const float* ref;
    const float* ref2;     // second reference (combined form)
    const float* means;    // the M scalar references (TNG_NORM_MEAN)
    float* out_a;
    float* out_b;
    uint32_t* pipe_error;
    uint64_t d, ntile, block;
    uint64_t tile_begin;   // first tile this launch handles (the staged kernel takes the ones before it)
    uint32_t nblk, wpw;
    uint32_t M;
    uint32_t one;  // 1 as a run-time value: "w << s" is taken as w * (one << s), on the multiplier pipe
    int levels;
    float quot_eps;
    float inv_m;   // 1/M when M is a power of two (then x * inv_m == x / M exactly), else 0
};

// Adds worker m's decoded values of the lane's four coordinates to acc.  `w` are the
// tile's code words (the same in every lane); multiplying a word by pw = 2^(31-lane)
// moves the lane's bit to the sign position.  A scale that is zero, NaN or infinite
// decodes to +0 whatever the symbols say.
template <int CODEC>
__device__ __forceinline__ void decode_worker(const uint32_t (&w)[4 * CODEC], const float R, const int levels,
                                              const uint32_t pw, const int lane, float (&acc)[4]) {
    // usable scale: 0 < R < inf, i.e. bit pattern in [1, 0x7f7fffff] (one unsigned compare)
    const bool ok = (__float_as_uint(R) - 1u) < 0x7f7fffffu;
    const uint32_t Re = ok ? __float_as_uint(R) : 0u;
    const uint32_t okm = ok ? 0x80000000u : 0u;
    if (CODEC == TNG_CODEC_TERN2) {
        // Per coordinate: the lane's bit of the non-zero plane decides whether anything is added
        // (acc + 0 == acc, and an unusable scale adds nothing either: the predicate is and-ed with
        // `ok`); the lane's bit of the sign plane, moved to bit 31 by a multiply, flips the sign of R.
        // Written out so that it stays four instructions per coordinate: a logic op that sets the
        // predicate, a multiply, a three-input logic op ((s & 0x80000000) ^ R), a predicated add.
        constexpr int kT = (CODEC == TNG_CODEC_TERN2) ? 2 : 0;   // plane stride (keeps indices in range elsewhere)
        asm("{\n\t.reg .pred p, pk;\n\t.reg .b32 t, s;\n\t"
            "setp.ne.u32 pk, %12, 0;\n\t"
            "lop3.and.b32 t|p, %4, %13, %13, 0xC0, pk;\n\t"
            "mul.lo.u32 s, %5, %14;\n\t"
            "lop3.b32 s, s, 0x80000000, %15, 0x6A;\n\t"
            "@p add.rn.f32 %0, %0, s;\n\t"
            "lop3.and.b32 t|p, %6, %13, %13, 0xC0, pk;\n\t"
            "mul.lo.u32 s, %7, %14;\n\t"
            "lop3.b32 s, s, 0x80000000, %15, 0x6A;\n\t"
            "@p add.rn.f32 %1, %1, s;\n\t"
            "lop3.and.b32 t|p, %8, %13, %13, 0xC0, pk;\n\t"
            "mul.lo.u32 s, %9, %14;\n\t"
            "lop3.b32 s, s, 0x80000000, %15, 0x6A;\n\t"
            "@p add.rn.f32 %2, %2, s;\n\t"
            "lop3.and.b32 t|p, %10, %13, %13, 0xC0, pk;\n\t"
            "mul.lo.u32 s, %11, %14;\n\t"
            "lop3.b32 s, s, 0x80000000, %15, 0x6A;\n\t"
            "@p add.rn.f32 %3, %3, s;\n\t}"
            : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
            : "r"(w[0]), "r"(w[kT ? 1 : 0]), "r"(w[1 * kT]), "r"(w[1 * kT + (kT ? 1 : 0)]), "r"(w[2 * kT]), "r"(w[2 * kT + (kT ? 1 : 0)]),
              "r"(w[3 * kT]), "r"(w[3 * kT + (kT ? 1 : 0)]), "r"((uint32_t)ok), "r"(1u << lane), "r"(pw), "r"(__float_as_uint(R)));
    } else if (CODEC == TNG_CODEC_SIGN1) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            // plus bit clear -> -R: (~s & okm) ^ Re
            asm("{\n\t.reg .b32 s;\n\t"
                "mul.lo.u32 s, %1, %2;\n\t"
                "lop3.b32 s, s, %3, %4, 0xA6;\n\t"
                "add.rn.f32 %0, %0, s;\n\t}"
                : "+f"(acc[c])
                : "r"(w[c]), "r"(pw), "r"(okm), "r"(Re));
        }
    } else {
        // R is what slot_scale left in the slot: the quantiser's step R / s, or NaN for an unusable scale
        const float step = R;
        const uint32_t signmask = (step == step) ? 0x80000000u : 0u;
        const float stepq = (step == step) ? step : 0.0f;
        // the lane's bit of the three level planes, landed at bit 0, 1 and 2 by a shift and two rotations and
        // merged by bit-select operations: six instructions per coordinate
        const uint32_t rot1 = (uint32_t)(lane - 1) & 31u, rot2 = (uint32_t)(lane - 2) & 31u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t x0 = w[c * 4] >> lane;
            const uint32_t x1 = __funnelshift_r(w[c * 4 + 1], w[c * 4 + 1], rot1);
            const uint32_t x2 = __funnelshift_r(w[c * 4 + 2], w[c * 4 + 2], rot2);
            const uint32_t y = (x0 & 1u) | (x1 & ~1u);
            const uint32_t L = ((y & 3u) | (x2 & ~3u)) & 7u;
            const float mag = __fmul_rn((float)L, stepq);
            const float vh = __uint_as_float(__float_as_uint(mag) ^ ((w[c * 4 + 3] * pw) & signmask));
            acc[c] = __fadd_rn(acc[c], vh);
        }
    }
}

// What goes into the decode slot for a worker's scale.  Ternary and sign codes use the scale as it is.  The
// s-level quantiser needs the step R / s (one IEEE division): taken here once per worker and tile by the lane that
// fetched the scale, instead of by every lane for every worker; an unusable scale (zero, NaN, infinite) becomes NaN.
template <int CODEC>
__device__ __forceinline__ float slot_scale(const float R, const int levels) {
    if (CODEC != TNG_CODEC_QSGD4) return R;
    const bool ok = (__float_as_uint(R) - 1u) < 0x7f7fffffu;
    return ok ? __fdiv_rn(R, (float)levels) : __int_as_float(0x7fc00000);
}

// average over the M workers (Algorithm 1), put the reference back (Eq. 2 / Eq. 3), store
template <int NORM>
__device__ __forceinline__ float4 decode_denormalise(const DecodeArgs& a, const float (&acc)[4], const float4 r, const float4 r2) {
    float4 o;
    if (a.inv_m > 0.0f) {
        o.x = __fmul_rn(acc[0], a.inv_m); o.y = __fmul_rn(acc[1], a.inv_m); o.z = __fmul_rn(acc[2], a.inv_m); o.w = __fmul_rn(acc[3], a.inv_m);
    } else {
        const float fm = (float)a.M;
        o.x = __fdiv_rn(acc[0], fm); o.y = __fdiv_rn(acc[1], fm); o.z = __fdiv_rn(acc[2], fm); o.w = __fdiv_rn(acc[3], fm);
    }
    if (NORM == TNG_NORM_DIFF || NORM == TNG_NORM_MEAN) {   // MEAN: r holds the average of the workers' scalars
        o.x = __fadd_rn(r.x, o.x); o.y = __fadd_rn(r.y, o.y); o.z = __fadd_rn(r.z, o.z); o.w = __fadd_rn(r.w, o.w);
    } else if (NORM == TNG_NORM_QUOT) {
        const float4 den = quot_den4(r, a.quot_eps);
        o.x = __fmul_rn(den.x, o.x); o.y = __fmul_rn(den.y, o.y); o.z = __fmul_rn(den.z, o.z); o.w = __fmul_rn(den.w, o.w);
    } else if (NORM == TNG_NORM_COMB) {   // out = den' * a + r, two roundings
        const float4 den = quot_den4(r2, a.quot_eps);
        o.x = __fadd_rn(__fmul_rn(den.x, o.x), r.x); o.y = __fadd_rn(__fmul_rn(den.y, o.y), r.y);
        o.z = __fadd_rn(__fmul_rn(den.z, o.z), r.z); o.w = __fadd_rn(__fmul_rn(den.w, o.w), r.w);
    }
    return o;
}

// ---------------------------------------------------------------------------
// Decode kernel.  One warp per tile.  The code words of a tile are the same for all 32
// lanes, so instead of every lane loading every word, ONE warp-wide load fetches the
// 16-byte pieces of up to 32/b workers (lane = worker * b + piece), a second one their
// scales, a third one the lane's four reference values; the words then go through a
// warp-private shared-memory slot and come back as broadcasts.  The three loads of the
// warp's next tile are issued before the current tile is decoded, so a warp always has
// loads in flight while it computes.
// ---------------------------------------------------------------------------
constexpr int kDecWarps = kCodecThreads / 32;

struct DecodeSlot {          // per warp
    uint4 cw[32];
    float sc[32];
};

template <int CODEC>
__device__ __forceinline__ void decode_fetch(const DecodeArgs& a, const uint64_t T, const uint64_t blk, const uint32_t m0,
                                             const int lane, uint4& cw, float& sc) {
    constexpr int kRound = 32 / CODEC;            // workers per round
    const uint32_t m = m0 + (uint32_t)lane / CODEC, piece = (uint32_t)lane % CODEC;
    cw = make_uint4(0u, 0u, 0u, 0u);
    sc = 0.0f;
    if (m < a.M) cw = __ldcs(reinterpret_cast<const uint4*>(a.codes + ((uint64_t)m * a.wpw + T * (uint64_t)(4 * CODEC))) + piece);
    if (lane < kRound && m0 + (uint32_t)lane < a.M) sc = __ldcs(a.scales + ((uint64_t)(m0 + (uint32_t)lane) * a.nblk + blk));
}

// decode the `n` workers whose words sit in the slot
template <int CODEC>
__device__ __forceinline__ void decode_round(const DecodeSlot* slot, const uint32_t n, const int levels, const uint32_t pw,
                                             const int lane, float (&acc)[4]) {
    constexpr int kWords = 4 * CODEC;
    constexpr int kU = (CODEC == TNG_CODEC_QSGD4) ? 2 : 4;   // workers decoded together
    uint32_t k = 0;
    for (; k + kU <= n; k += kU) {
#pragma unroll
        for (int kk = 0; kk < kU; ++kk) {
            uint32_t w[kWords];
#pragma unroll
            for (int q = 0; q < CODEC; ++q) {
                const uint4 t = slot->cw[(k + kk) * CODEC + q];
                w[4 * q + 0] = t.x; w[4 * q + 1] = t.y; w[4 * q + 2] = t.z; w[4 * q + 3] = t.w;
            }
            decode_worker<CODEC>(w, slot->sc[k + kk], levels, pw, lane, acc);
        }
    }
    for (; k < n; ++k) {
        uint32_t w[kWords];
#pragma unroll
        for (int q = 0; q < CODEC; ++q) {
            const uint4 t = slot->cw[k * CODEC + q];
            w[4 * q + 0] = t.x; w[4 * q + 1] = t.y; w[4 * q + 2] = t.z; w[4 * q + 3] = t.w;
        }
        decode_worker<CODEC>(w, slot->sc[k], levels, pw, lane, acc);
    }
}

// the same with the worker count known at compile time (no loop, constant shared offsets)
template <int CODEC, int N>
__device__ __forceinline__ void decode_round_fixed(const DecodeSlot* slot, const int levels, const uint32_t pw, const int lane,
                                                   float (&acc)[4]) {
    constexpr int kWords = 4 * CODEC;
#pragma unroll
    for (int k = 0; k < N; ++k) {
        uint32_t w[kWords];
#pragma unroll
        for (int q = 0; q < CODEC; ++q) {
            const uint4 t = slot->cw[k * CODEC + q];
            w[4 * q + 0] = t.x; w[4 * q + 1] = t.y; w[4 * q + 2] = t.z; w[4 * q + 3] = t.w;
        }
        decode_worker<CODEC>(w, slot->sc[k], levels, pw, lane, acc);
    }
}

template <int CODEC>
__device__ __forceinline__ void decode_round_any(const DecodeSlot* slot, const uint32_t n, const int levels, const uint32_t pw,
                                                 const int lane, float (&acc)[4]) {
    if (n == 8 && 8 * CODEC <= 32) decode_round_fixed<CODEC, (8 * CODEC <= 32 ? 8 : 1)>(slot, levels, pw, lane, acc);
    else if (n == 4) decode_round_fixed<CODEC, 4>(slot, levels, pw, lane, acc);
    else decode_round<CODEC>(slot, n, levels, pw, lane, acc);
}

template <int CODEC, int NORM>
__global__ void __launch_bounds__(kCodecThreads, 4) decode_kernel(const DecodeArgs a) {
    __shared__ DecodeSlot slots[kDecWarps];
    constexpr uint32_t kRound = 32 / CODEC;
    const int lane = threadIdx.x & 31;
    DecodeSlot* slot = &slots[threadIdx.x >> 5];
    // Tile indices fit 32 bits (d <= 2^31), and so does every per-tile offset below: each address is
    // then ONE 32 x 32 -> 64 multiply-add on a pointer that is either a kernel argument or a per-lane
    // row pointer formed once (the lane's worker is the same for every tile).
    const uint32_t nwarps = gridDim.x * kDecWarps;
    const uint32_t gwarp = blockIdx.x * kDecWarps + (threadIdx.x >> 5);
    const uint32_t nfull = (uint32_t)(a.d / kTile);
    const uint32_t block32 = (uint32_t)a.block;
    const uint32_t pw = a.one << (31 - lane);
    const bool tiled = a.block == (uint64_t)kTile;
    const bool has_ref = (NORM != TNG_NORM_NONE) && (NORM != TNG_NORM_MEAN) && a.ref != nullptr;
    const bool has_ref2 = (NORM == TNG_NORM_COMB) && a.ref2 != nullptr;
    const bool to_a = a.out_a != nullptr, to_b = a.out_b != nullptr;
    const uint32_t n0 = a.M < kRound ? a.M : kRound;                 // workers of the first round
    // first round: lane = worker * b + piece; the lane's own rows of the wire
    const uint32_t my_m = (uint32_t)lane / CODEC, my_piece = (uint32_t)lane % CODEC;
    const bool has_code = my_m < a.M, has_scale = (uint32_t)lane < n0;
    const uint4* code_row = reinterpret_cast<const uint4*>(a.codes + (uint64_t)(has_code ? my_m : 0u) * a.wpw) + my_piece;
    const float* scale_row = a.scales + (uint64_t)(has_scale ? (uint32_t)lane : 0u) * a.nblk;
    const float4* ref4 = reinterpret_cast<const float4*>(a.ref) + lane;
    const float4* ref24 = reinterpret_cast<const float4*>(a.ref2) + lane;
    // the sum starts from -0 so that (-0) + x == x bit for bit; the ternary path starts from +0
    // because it skips zero symbols and +0 is what the sum of skipped terms is
    const float z = (CODEC == TNG_CODEC_TERN2) ? 0.0f : -0.0f;

    float4 r = make_float4(0.f, 0.f, 0.f, 0.f), r2 = r;
    if (NORM == TNG_NORM_MEAN) {
        // what every element gets back: (1/M) sum_m mean(g^m), summed m ascending like the codes
        float sum = a.means[0];
        for (uint32_t m = 1; m < a.M; ++m) sum = __fadd_rn(sum, a.means[m]);
        const float mbar = (a.inv_m > 0.0f) ? __fmul_rn(sum, a.inv_m) : __fdiv_rn(sum, (float)a.M);
        r = make_float4(mbar, mbar, mbar, mbar);
    }
    const float4 r_const = r;
    // the three loads of tile t (first round of workers)
    auto fetch = [&](const uint32_t t, uint4& cw, float& sc, float4& rr, float4& rr2) {
        const uint32_t blk = tiled ? t : (t * (uint32_t)kTile) / block32;
        cw = make_uint4(0u, 0u, 0u, 0u);
        sc = 0.0f;
        if (has_code) cw = __ldcs(code_row + (size_t)t * CODEC);
        if (has_scale) sc = __ldcs(scale_row + blk);
        if (has_ref) rr = ref4[(size_t)t * 32u];
        if (has_ref2) rr2 = ref24[(size_t)t * 32u];
    };

    uint32_t T = (uint32_t)a.tile_begin + gwarp;
    uint4 cw = make_uint4(0u, 0u, 0u, 0u);
    float sc = 0.0f;
    if (T < nfull) fetch(T, cw, sc, r, r2);
    for (; T < nfull; T += nwarps) {
        slot->cw[lane] = cw;
        slot->sc[lane] = slot_scale<CODEC>(sc, a.levels);
        const float4 rcur = r, r2cur = r2;
        __syncwarp();
        const uint32_t Tn = T + nwarps;
        if (Tn < nfull) fetch(Tn, cw, sc, r, r2);                     // next tile's loads go out now
        float acc[4] = {z, z, z, z};
        decode_round_any<CODEC>(slot, n0, a.levels, pw, lane, acc);
        for (uint32_t m0 = kRound; m0 < a.M; m0 += kRound) {         // more workers than one round holds
            uint4 cw2;
            float sc2;
            decode_fetch<CODEC>(a, T, tiled ? T : ((uint64_t)T * kTile) / a.block, m0, lane, cw2, sc2);
            __syncwarp();
            slot->cw[lane] = cw2;
            slot->sc[lane] = slot_scale<CODEC>(sc2, a.levels);
            __syncwarp();
            decode_round<CODEC>(slot, (a.M - m0 < kRound) ? a.M - m0 : kRound, a.levels, pw, lane, acc);
        }
        __syncwarp();                                                // slot is free again
        const float4 o = decode_denormalise<NORM>(a, acc, rcur, r2cur);
        const size_t at = (size_t)T * 32u + (uint32_t)lane;          // float4 index of the lane's coordinates
        if (to_a) reinterpret_cast<float4*>(a.out_a)[at] = o;
        if (to_b) reinterpret_cast<float4*>(a.out_b)[at] = o;
    }
    // the ragged last tile
    if ((uint64_t)nfull < a.ntile && gwarp == nfull % nwarps) {
        const uint64_t Tr = nfull, i0 = Tr * kTile + (uint64_t)lane * 4u;
        const uint64_t blk = tiled ? Tr : (Tr * kTile) / a.block;
        float4 rr = (NORM == TNG_NORM_MEAN) ? r_const : make_float4(0.f, 0.f, 0.f, 0.f), rr2 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (has_ref) rr = load4(a.ref, i0, a.d);
        if (has_ref2) rr2 = load4(a.ref2, i0, a.d);
        float acc[4] = {z, z, z, z};
        for (uint32_t m0 = 0; m0 < a.M; m0 += kRound) {
            uint4 cw2;
            float sc2;
            decode_fetch<CODEC>(a, Tr, blk, m0, lane, cw2, sc2);
            __syncwarp();
            slot->cw[lane] = cw2;
            slot->sc[lane] = slot_scale<CODEC>(sc2, a.levels);
            __syncwarp();
            decode_round<CODEC>(slot, (a.M - m0 < kRound) ? a.M - m0 : kRound, a.levels, pw, lane, acc);
        }
        const float4 o = decode_denormalise<NORM>(a, acc, rr, rr2);
        if (to_a) store4(a.out_a, i0, a.d, o);
        if (to_b) store4(a.out_b, i0, a.d, o);
    }
}

// Persistent launch: as many CTAs as fit on the GPU at once (occupancy of this very
// instantiation times the SM count), fewer when there are not enough tiles.
template <typename Kern>
int persistent_grid(Kern kern, uint64_t ntile, int sm_count) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCodecThreads, 0) != cudaSuccess || per_sm < 1) {
        (void)cudaGetLastError();
        per_sm = 1;
    }
    const uint64_t want = (ntile + 7) / 8;   // 8 warps per CTA, one tile per warp per pass
    const uint64_t cap = (uint64_t)sm_count * (uint64_t)per_sm;
    return (int)(want < cap ? (want ? want : 1) : cap);
}

template <int CODEC, int NORM, int SCALE, int PHASE, bool FUSEREF>
cudaError_t encode_launch_direct(const EncodeArgs& a, int sm_count, cudaStream_t st) {
    static PerDevice<int> cached;   // grid when tiles are plentiful, per device
    auto kern = encode_kernel<CODEC, NORM, SCALE, PHASE, FUSEREF>;
    const int slot = device_slot();
    int per_tiles_grid = slot >= 0 ? cached.v[slot] : 0;
    if (per_tiles_grid == 0) {
        per_tiles_grid = persistent_grid(kern, ~0ull >> 8, sm_count);
        if (slot >= 0) cached.v[slot] = per_tiles_grid;
    }
    const uint64_t want = (a.ntile - a.tile_begin + 7) / 8;
    const int grid = (int)(want < (uint64_t)per_tiles_grid ? (want ? want : 1) : (uint64_t)per_tiles_grid);
    kern<<<grid, kCodecThreads, 0, st>>>(a);
    return cudaGetLastError();
}

// One scale per tile: the whole chunks go through the staged kernel, the remaining tiles
// (fewer than 8 full ones and a ragged one) through the direct kernel.
template <int CODEC, int NORM, int SCALE, bool FUSEREF>
cudaError_t encode_launch_tiles(const EncodeArgs& a0, int sm_count, cudaStream_t st, int* launches) {
    const uint64_t nchunks = a0.d / EncGeom::kChunk;
    EncodeArgs a = a0;
    a.tile_begin = 0;
    if (nchunks >= kEncPipeMinChunks) {
        static PerDevice<bool> configured;   // opt in to the large dynamic shared memory once per instantiation and device
        auto kern = encode_pipe_kernel<CODEC, NORM, SCALE, FUSEREF>;
        const int slot = device_slot();
        if (slot < 0 || !configured.v[slot]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EncGeom::kSmemBytes);
            if (e != cudaSuccess) return e;
            if (slot >= 0) configured.v[slot] = true;
        }
        EncodePipeArgs pa;
        pa.e = a;
        pa.e.tile_begin = nchunks * kEncPipeWarps;
        pa.rows.nrows = 0;
        if (FUSEREF) {
            for (int j = 0; j < a.hist_k; ++j) pa.rows.row[pa.rows.nrows++] = a.hist[j];
        } else if (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN && a.ref) {
            pa.rows.row[pa.rows.nrows++] = a.ref;
            if (NORM == TNG_NORM_COMB && a.ref2) pa.rows.row[pa.rows.nrows++] = a.ref2;
        }
        pa.rows.n_pre = pa.rows.nrows;
        for (uint32_t m = 0; m < a.M; ++m) pa.rows.row[pa.rows.nrows++] = a.grads + (uint64_t)m * a.ld;
        const int grid = (int)(nchunks < (uint64_t)sm_count ? nchunks : (uint64_t)sm_count);
        kern<<<grid, kEncPipeThreads, EncGeom::kSmemBytes, st>>>(pa);
        ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        a.tile_begin = pa.e.tile_begin;
        if (a.tile_begin >= a.ntile) return cudaSuccess;
    }
    ++*launches;
    return encode_launch_direct<CODEC, NORM, SCALE, kPhaseFused, FUSEREF>(a, sm_count, st);
}

// A scale per 256 .. 2048 coordinates: the whole chunks through the staged kernel that shares tile
// statistics between the warps of a block.  The caller handles the coordinates after the last whole chunk.
template <int CODEC, int NORM, int SCALE, bool FUSEREF>
cudaError_t encode_launch_blocks(const EncodeArgs& a, int sm_count, cudaStream_t st, int* launches) {
    const uint64_t nchunks = a.d / EncGeom::kChunk;
    static PerDevice<bool> configured;
    auto kern = encode_pipe_blocks_kernel<CODEC, NORM, SCALE, FUSEREF>;
    const int slot = device_slot();
    if (slot < 0 || !configured.v[slot]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)EncGeom::kSmemBytes);
        if (e != cudaSuccess) return e;
        if (slot >= 0) configured.v[slot] = true;
    }
    EncodePipeArgs pa;
    pa.e = a;
    pa.e.tile_begin = nchunks * kEncPipeWarps;
    pa.rows.nrows = 0;
    if (FUSEREF) {
        for (int j = 0; j < a.hist_k; ++j) pa.rows.row[pa.rows.nrows++] = a.hist[j];
    } else if (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN && a.ref) {
        pa.rows.row[pa.rows.nrows++] = a.ref;
        if (NORM == TNG_NORM_COMB && a.ref2) pa.rows.row[pa.rows.nrows++] = a.ref2;
    }
    pa.rows.n_pre = pa.rows.nrows;
    for (uint32_t m = 0; m < a.M; ++m) pa.rows.row[pa.rows.nrows++] = a.grads + (uint64_t)m * a.ld;
    const int grid = (int)(nchunks < (uint64_t)sm_count ? nchunks : (uint64_t)sm_count);
    kern<<<grid, kEncPipeThreads, EncGeom::kSmemBytes, st>>>(pa);
    ++*launches;
    return cudaGetLastError();
}
template <int CODEC, int NORM, int SCALE>
cudaError_t encode_blocks_fuse(const EncodeArgs& a, int sm_count, cudaStream_t st, int* launches) {
    if constexpr (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN) {
        if (a.hist_k > 0) return encode_launch_blocks<CODEC, NORM, SCALE, true>(a, sm_count, st, launches);
    }
    return encode_launch_blocks<CODEC, NORM, SCALE, false>(a, sm_count, st, launches);
}
template <int CODEC, int NORM>
cudaError_t encode_blocks_scale(const EncodeArgs& a, int scale, int sm_count, cudaStream_t st, int* launches) {
    return scale == 0 ? encode_blocks_fuse<CODEC, NORM, 0>(a, sm_count, st, launches) : encode_blocks_fuse<CODEC, NORM, 1>(a, sm_count, st, launches);
}
template <int CODEC>
cudaError_t encode_blocks_norm(const EncodeArgs& a, int norm, int scale, int sm_count, cudaStream_t st, int* launches) {
    switch (norm) {
        case TNG_NORM_DIFF: return encode_blocks_scale<CODEC, TNG_NORM_DIFF>(a, scale, sm_count, st, launches);
        case TNG_NORM_QUOT: return encode_blocks_scale<CODEC, TNG_NORM_QUOT>(a, scale, sm_count, st, launches);
        case TNG_NORM_COMB: return encode_blocks_scale<CODEC, TNG_NORM_COMB>(a, scale, sm_count, st, launches);
        case TNG_NORM_MEAN: return encode_blocks_scale<CODEC, TNG_NORM_MEAN>(a, scale, sm_count, st, launches);
        default: return encode_blocks_scale<CODEC, TNG_NORM_NONE>(a, scale, sm_count, st, launches);
    }
}
cudaError_t encode_blocks_dispatch(const EncodeArgs& a, int codec, int norm, int scale, int sm_count, cudaStream_t st, int* launches) {
    switch (codec) {
        case TNG_CODEC_SIGN1: return encode_blocks_norm<TNG_CODEC_SIGN1>(a, norm, scale, sm_count, st, launches);
        case TNG_CODEC_TERN2: return encode_blocks_norm<TNG_CODEC_TERN2>(a, norm, scale, sm_count, st, launches);
        default: return encode_blocks_norm<TNG_CODEC_QSGD4>(a, norm, scale, sm_count, st, launches);
    }
}

template <int CODEC, int NORM, int SCALE, int PHASE>
cudaError_t encode_launch(const EncodeArgs& a, int sm_count, cudaStream_t st, int* launches) {
    if constexpr (PHASE == kPhaseFused) {
        if (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN && a.hist_k > 0)
            return encode_launch_tiles<CODEC, NORM, SCALE, (NORM != TNG_NORM_NONE && NORM != TNG_NORM_MEAN)>(a, sm_count, st, launches);
        return encode_launch_tiles<CODEC, NORM, SCALE, false>(a, sm_count, st, launches);
    } else {
        ++*launches;
        return encode_launch_direct<CODEC, NORM, SCALE, PHASE, false>(a, sm_count, st);
    }
}
template <int CODEC, int NORM, int SCALE>
cudaError_t encode_dispatch_phase(const EncodeArgs& a, int phase, int sm_count, cudaStream_t st, int* launches) {
    if (phase == kPhaseFused) return encode_launch<CODEC, NORM, SCALE, kPhaseFused>(a, sm_count, st, launches);
    if (phase == kPhaseStat) return encode_launch<CODEC, NORM, SCALE, kPhaseStat>(a, sm_count, st, launches);
    return encode_launch<CODEC, NORM, SCALE, kPhaseQuant>(a, sm_count, st, launches);
}
template <int CODEC, int NORM>
cudaError_t encode_dispatch_scale(const EncodeArgs& a, int scale, int phase, int sm_count, cudaStream_t st, int* launches) {
    return scale == 0 ? encode_dispatch_phase<CODEC, NORM, 0>(a, phase, sm_count, st, launches)
                      : encode_dispatch_phase<CODEC, NORM, 1>(a, phase, sm_count, st, launches);
}
template <int CODEC>
cudaError_t encode_dispatch_norm(const EncodeArgs& a, int norm, int scale, int phase, int sm_count, cudaStream_t st, int* launches) {
    switch (norm) {
        case TNG_NORM_DIFF: return encode_dispatch_scale<CODEC, TNG_NORM_DIFF>(a, scale, phase, sm_count, st, launches);
        case TNG_NORM_QUOT: return encode_dispatch_scale<CODEC, TNG_NORM_QUOT>(a, scale, phase, sm_count, st, launches);
        case TNG_NORM_COMB: return encode_dispatch_scale<CODEC, TNG_NORM_COMB>(a, scale, phase, sm_count, st, launches);
        case TNG_NORM_MEAN: return encode_dispatch_scale<CODEC, TNG_NORM_MEAN>(a, scale, phase, sm_count, st, launches);
        default: return encode_dispatch_scale<CODEC, TNG_NORM_NONE>(a, scale, phase, sm_count, st, launches);
    }
}
cudaError_t encode_dispatch(const EncodeArgs& a, int codec, int norm, int scale, int phase, int sm_count, cudaStream_t st,
                            int* launches) {
    switch (codec) {
        case TNG_CODEC_SIGN1: return encode_dispatch_norm<TNG_CODEC_SIGN1>(a, norm, scale, phase, sm_count, st, launches);
        case TNG_CODEC_TERN2: return encode_dispatch_norm<TNG_CODEC_TERN2>(a, norm, scale, phase, sm_count, st, launches);
        default: return encode_dispatch_norm<TNG_CODEC_QSGD4>(a, norm, scale, phase, sm_count, st, launches);
    }
}

template <int CODEC, int NORM>
cudaError_t decode_launch(const DecodeArgs& a, int sm_count, cudaStream_t st, int* launches) {
    static PerDevice<int> cached;
    auto kern = decode_kernel<CODEC, NORM>;
    const int slot = device_slot();
    int per_tiles_grid = slot >= 0 ? cached.v[slot] : 0;
    if (per_tiles_grid == 0) {
        per_tiles_grid = persistent_grid(kern, ~0ull >> 8, sm_count);
        if (slot >= 0) cached.v[slot] = per_tiles_grid;
    }
    const uint64_t want = (a.ntile - a.tile_begin + 7) / 8;
    const int grid = (int)(want < (uint64_t)per_tiles_grid ? (want ? want : 1) : (uint64_t)per_tiles_grid);
    kern<<<grid, kCodecThreads, 0, st>>>(a);
    ++*launches;
    return cudaGetLastError();
}
template <int CODEC>
cudaError_t decode_dispatch_norm(const DecodeArgs& a, int norm, int sm_count, cudaStream_t st, int* launches) {
    switch (norm) {
        case TNG_NORM_DIFF: return decode_launch<CODEC, TNG_NORM_DIFF>(a, sm_count, st, launches);
        case TNG_NORM_QUOT: return decode_launch<CODEC, TNG_NORM_QUOT>(a, sm_count, st, launches);
        case TNG_NORM_COMB: return decode_launch<CODEC, TNG_NORM_COMB>(a, sm_count, st, launches);
        case TNG_NORM_MEAN: return decode_launch<CODEC, TNG_NORM_MEAN>(a, sm_count, st, launches);
        default: return decode_launch<CODEC, TNG_NORM_NONE>(a, sm_count, st, launches);
    }
}

}  // namespace

size_t tree_tmp_floats(const CodecGeom& g) {
    // the scalar reference reduces all tiles of a row: two ping-pong levels of M * ceil(ntile / 1024)
    const uint64_t mean_tmp = (g.norm == TNG_NORM_MEAN) ? 2 * (uint64_t)g.M * ((g.ntile + 1023) / 1024) : 0;
    if (g.block == kTile) return (size_t)mean_tmp;
    const uint64_t seg = (g.block + kTile - 1) / kTile;            // tiles per block
    const uint64_t chunks = (seg + 1023) / 1024;
    // two ping-pong levels, each at most M * nblk * chunks entries
    const uint64_t scale_tmp = 2 * (uint64_t)g.M * g.nblk * chunks;
    return (size_t)(scale_tmp > mean_tmp ? scale_tmp : mean_tmp);
}

bool encode_needs_tile_stat(const CodecGeom& g) { return g.block != kTile || g.norm == TNG_NORM_MEAN; }

bool encode_can_fuse_reference(const CodecGeom& g) { return g.norm != TNG_NORM_NONE && g.norm != TNG_NORM_MEAN; }

constexpr uint64_t kShortProblemTiles = 16384;   // tiles x workers up to which the one-launch path is taken

// scale blocks of 2, 4, 8 or 16 tiles lie inside one chunk of the staged pass
static bool block_within_chunk(uint64_t block) { return block == 256 || block == 512 || block == 1024 || block == 2048; }

cudaError_t launch_encode(const CodecGeom& g, uint32_t m_base, const float* grads, uint64_t ld, const float* ref, const float* ref2,
                          const RefFusion* fusion,
                          uint32_t step, uint32_t* codes, float* scales, float* means, float* tile_stat, float* tree_tmp,
                          FuseBlock* fb, int sm_count, cudaStream_t st, int* launches) {
    EncodeArgs a;
    a.means = means;
    a.hist_k = 0; a.alpha = nullptr; a.ref_out = nullptr;
    a.ref2 = ref2; a.ref2_out = nullptr; a.inv_k = 0.0f;
    for (int j = 0; j < kMaxK; ++j) a.hist[j] = nullptr;
    if (fusion && fusion->k > 0 && encode_can_fuse_reference(g)) {
        a.hist_k = fusion->k; a.alpha = fusion->alpha; a.ref_out = fusion->ref_out;
        a.ref2_out = fusion->ref2_out; a.inv_k = 1.0f / (float)fusion->k;
        for (int j = 0; j < fusion->k; ++j) a.hist[j] = fusion->rows[j];
    }
    a.grads = grads; a.ref = ref; a.codes = codes; a.scales = scales; a.tile_stat = tile_stat;
    a.nonfinite = &fb->nonfinite; a.pipe_error = &fb->pipe_error; a.tile_begin = 0; a.tile0 = g.tile0;
    a.ld = (uint32_t)ld; a.d = g.d; a.ntile = g.ntile; a.nblk = (uint32_t)g.nblk; a.block = g.block; a.wpw = (uint32_t)g.wpw;
    a.M = g.M; a.step = step; a.m_base = m_base; a.levels = g.levels; a.pow24 = 1u << 24;
    a.quot_eps = g.quot_eps;
    philox_round_keys(g.seed_lo, g.seed_hi, a.rk);
    cudaError_t e;
    if (g.norm == TNG_NORM_MEAN) {
        // scalar reference: per-tile sums of every row, then the tree over the tiles, divided by d
        const uint64_t want = (g.ntile + 7) / 8, cap = (uint64_t)sm_count * 8u;
        row_tile_sum_kernel<<<(unsigned)(want < cap ? want : cap), kCodecThreads, 0, st>>>(grads, (uint32_t)ld, g.M, g.d, g.ntile, tile_stat);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        const float* in = tile_stat;
        uint64_t n_in = g.ntile;
        float* ping = tree_tmp;
        float* pong = tree_tmp + (uint64_t)g.M * ((g.ntile + 1023) / 1024);
        for (;;) {
            const uint64_t chunks = (n_in + 1023) / 1024;
            const int final = chunks == 1;
            dim3 grid3(1u, (unsigned)chunks, g.M);
            block_scale_level_kernel<kTreeSum><<<grid3, 256, 0, st>>>(in, n_in, n_in, chunks, final ? means : ping, chunks, final,
                                                                      (float)g.d, &fb->nonfinite);
            ++*launches;
            e = cudaGetLastError();
            if (e != cudaSuccess) return e;
            if (final) break;
            in = ping; n_in = chunks;
            float* t = ping; ping = pong; pong = t;
        }
    }
    if (g.block == kTile) return encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseFused, sm_count, st, launches);
    // A scale per 256 .. 2048 coordinates of a long vector: the whole chunks in one pass over the rows.
    uint64_t tile_begin = 0;
    const uint64_t nchunks = g.d / EncGeom::kChunk;
    if (block_within_chunk(g.block) && nchunks >= kEncPipeMinChunks) {
        e = encode_blocks_dispatch(a, g.codec, g.norm, g.scale_kind, sm_count, st, launches);
        if (e != cudaSuccess) return e;
        tile_begin = nchunks * kEncPipeWarps;
        if (tile_begin >= g.ntile) return cudaSuccess;
    }
    // The remaining coordinates (all of them for any other block size), as a problem of its own that starts at
    // coordinate i_begin (a multiple of the block): per-tile statistic -> per-block tree -> quantise.
    const uint64_t i_begin = tile_begin * kTile;
    if (a.hist_k > 0) {   // the reference was left to this pass: combine what the staged kernel did not
        const float* rows[kMaxK];
        for (int j = 0; j < a.hist_k; ++j) rows[j] = a.hist[j] + i_begin;
        e = launch_combine(rows, a.hist_k, g.d - i_begin, fb, a.ref_out + i_begin, a.ref2_out ? a.ref2_out + i_begin : nullptr,
                           sm_count, st, launches);
        if (e != cudaSuccess) return e;
        a.ref = a.ref_out;
        if (a.ref2_out) a.ref2 = a.ref2_out;
        a.hist_k = 0;
    }
    const uint64_t blk_begin = i_begin / g.block;
    const uint64_t nblk_rest = g.nblk - blk_begin;
    a.grads += i_begin;
    if (a.ref) a.ref += i_begin;
    if (a.ref2) a.ref2 += i_begin;
    a.codes += tile_begin * 4u * (uint64_t)g.codec;
    a.scales += blk_begin;
    a.d = g.d - i_begin;
    a.ntile = g.ntile - tile_begin;       // also the row stride of the tile statistics
    a.tile0 = g.tile0 + tile_begin;
    a.tile_begin = 0;
    // Short problem: one launch, a CTA per (scale block, worker), when a block has at most 1024 tiles and
    // there are few enough tiles that launch latency, not bandwidth, is what the three-launch path costs.
    const uint64_t tiles_per_block = (g.block + kTile - 1) / kTile;
    if (tiles_per_block <= 1024 && a.ntile * (uint64_t)g.M <= kShortProblemTiles && nblk_rest <= 65535) {
        dim3 grid((unsigned)nblk_rest, g.M);
        ++*launches;
        return encode_block_cta_dispatch(a, g.codec, g.norm, g.scale_kind, grid, st);
    }
    e = encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseStat, sm_count, st, launches);
    if (e != cudaSuccess) return e;
    const float* in = tile_stat;
    uint64_t n_in = a.ntile;
    uint64_t seg = (g.block + kTile - 1) / kTile;
    float* ping = tree_tmp;
    float* pong = tree_tmp + tree_tmp_floats(g) / 2;
    if (seg <= 32) {   // small blocks: a warp per block instead of a CTA per block
        const uint64_t jobs = nblk_rest * (uint64_t)g.M;
        const uint64_t want = (jobs + 7) / 8, cap = (uint64_t)sm_count * 16u;
        const unsigned grid = (unsigned)(want < cap ? want : cap);
        if (g.scale_kind == 0)
            block_scale_warp_kernel<0><<<grid, 256, 0, st>>>(in, n_in, (uint32_t)seg, a.scales, g.nblk, nblk_rest, g.M, &fb->nonfinite);
        else
            block_scale_warp_kernel<1><<<grid, 256, 0, st>>>(in, n_in, (uint32_t)seg, a.scales, g.nblk, nblk_rest, g.M, &fb->nonfinite);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        return encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseQuant, sm_count, st, launches);
    }
    for (;;) {
        const uint64_t chunks = (seg + 1023) / 1024;
        const int final = chunks == 1;
        float* out = final ? a.scales : ping;
        const uint64_t n_out = final ? g.nblk : nblk_rest * chunks;   // row stride: the wire's for the scales themselves
        dim3 grid3((unsigned)nblk_rest, (unsigned)chunks, g.M);
        if (g.scale_kind == 0)
            block_scale_level_kernel<0><<<grid3, 256, 0, st>>>(in, n_in, seg, chunks, out, n_out, final, 1.0f, &fb->nonfinite);
        else
            block_scale_level_kernel<1><<<grid3, 256, 0, st>>>(in, n_in, seg, chunks, out, n_out, final, 1.0f, &fb->nonfinite);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess || final) break;
        in = out; n_in = n_out; seg = chunks;
        float* t = ping; ping = pong; pong = t;
    }
    if (e != cudaSuccess) return e;
    return encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseQuant, sm_count, st, launches);
}

cudaError_t launch_decode(const CodecGeom& g, const uint32_t* codes, const float* scales, const float* means, const float* ref,
                          const float* ref2, float* out_a, float* out_b, FuseBlock* fb, int sm_count, cudaStream_t st, int* launches) {
    DecodeArgs a;
    a.codes = codes; a.scales = scales; a.means = means; a.ref = ref; a.ref2 = ref2; a.out_a = out_a; a.out_b = out_b;
    a.pipe_error = &fb->pipe_error; a.tile_begin = 0;
    a.d = g.d; a.ntile = g.ntile; a.nblk = (uint32_t)g.nblk; a.block = g.block; a.wpw = (uint32_t)g.wpw; a.M = g.M;
    a.one = 1u; a.levels = g.levels; a.quot_eps = g.quot_eps;
    a.inv_m = ((g.M & (g.M - 1)) == 0) ? 1.0f / (float)g.M : 0.0f;
    cudaError_t e;
    switch (g.codec) {
        case TNG_CODEC_SIGN1: e = decode_dispatch_norm<TNG_CODEC_SIGN1>(a, g.norm, sm_count, st, launches); break;
        case TNG_CODEC_TERN2: e = decode_dispatch_norm<TNG_CODEC_TERN2>(a, g.norm, sm_count, st, launches); break;
        default: e = decode_dispatch_norm<TNG_CODEC_QSGD4>(a, g.norm, sm_count, st, launches); break;
    }
    return e;
}

}  // namespace tng
