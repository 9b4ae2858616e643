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

namespace tng {

namespace {

enum { kPhaseFused = 0, kPhaseStat = 1, kPhaseQuant = 2 };

struct EncodeArgs {
    const float* grads;
    const float* ref;
    uint32_t* codes;
    float* scales;
    float* tile_stat;
    unsigned long long* nonfinite;
    uint64_t ld, d, ntile, nblk, block, wpw;
    uint32_t M, step, seed_lo, seed_hi;
    int levels;
    float quot_eps;
};

template <int CODEC, int NORM, int SCALE, int PHASE>
__device__ __forceinline__ void encode_worker(const EncodeArgs& a, const float4 g, const float4 op,
                                              const uint32_t m, const uint64_t T, const uint64_t blk,
                                              const int lane, const uint32_t valid) {
    // ---- normalise: v = g - r (Eq. 2), v = g * (1/den) (Eq. 3), or v = g
    float v0, v1, v2, v3;
    if (NORM == TNG_NORM_DIFF) {
        v0 = __fsub_rn(g.x, op.x); v1 = __fsub_rn(g.y, op.y); v2 = __fsub_rn(g.z, op.z); v3 = __fsub_rn(g.w, op.w);
    } else if (NORM == TNG_NORM_QUOT) {
        v0 = __fmul_rn(g.x, op.x); v1 = __fmul_rn(g.y, op.y); v2 = __fmul_rn(g.z, op.z); v3 = __fmul_rn(g.w, op.w);
    } else {
        v0 = g.x; v1 = g.y; v2 = g.z; v3 = g.w;
    }
    // ---- scale of the block
    float R;
    if (PHASE != kPhaseQuant) {
        const float stat = (SCALE == 0) ? warp_absmax(v0, v1, v2, v3) : warp_sumsq_tree(v0, v1, v2, v3);
        if (PHASE == kPhaseStat) {
            if (lane == 0) a.tile_stat[(uint64_t)m * a.ntile + T] = stat;
            return;
        }
        R = (SCALE == 0) ? stat : __fsqrt_rn(stat);
        if (lane == 0) {
            a.scales[(uint64_t)m * a.nblk + T] = R;
            if (!(R < __int_as_float(0x7f800000))) atomicAdd(a.nonfinite, 1ull);   // NaN or +inf
        }
    } else {
        R = __ldg(a.scales + (uint64_t)m * a.nblk + blk);
    }
    const bool ok = !scale_is_bad(R);

    // ---- stochastic rounding: one Philox call per lane, word c for coordinate 4j+c
    const uint64_t q = T * 32u + (uint32_t)lane;
    const uint4 x = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), m, a.step, a.seed_lo, a.seed_hi);
    const float u[4] = {uniform24(x.x), uniform24(x.y), uniform24(x.z), uniform24(x.w)};
    const float v[4] = {v0, v1, v2, v3};

    uint32_t mine = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const bool live = ok && ((valid >> c) & 1u);
        if (CODEC == TNG_CODEC_TERN2) {
            // nonzero with probability |v|/R  <=>  u*R < |v|
            const bool nz = live && (__fmul_rn(u[c], R) < fabsf(v[c]));
            const bool neg = nz && (v[c] < 0.0f);
            const uint32_t w0 = __ballot_sync(kFullMask, nz);
            const uint32_t w1 = __ballot_sync(kFullMask, neg);
            if (lane == c * 2 + 0) mine = w0;
            if (lane == c * 2 + 1) mine = w1;
        } else if (CODEC == TNG_CODEC_SIGN1) {
            // +R with probability (1 + v/R)/2  <=>  u*R < v/2 + R/2
            const float thr = __fadd_rn(__fmul_rn(0.5f, v[c]), __fmul_rn(0.5f, R));
            const bool plus = live && (__fmul_rn(u[c], R) < thr);
            const uint32_t w0 = __ballot_sync(kFullMask, plus);
            if (lane == c) mine = w0;
        } else {
            // s-level: a = (|v|/R) s; level floor(a) (+1 with probability frac(a))
            const float qv = __fdiv_rn(fabsf(v[c]), R);
            const float av = __fmul_rn(qv, (float)a.levels);
            const float lv = floorf(av);
            const float fv = __fsub_rn(av, lv);
            int L = live ? ((int)lv + ((u[c] < fv) ? 1 : 0)) : 0;
            const bool neg = (L > 0) && (v[c] < 0.0f);
            const uint32_t w0 = __ballot_sync(kFullMask, L & 1);
            const uint32_t w1 = __ballot_sync(kFullMask, L & 2);
            const uint32_t w2 = __ballot_sync(kFullMask, L & 4);
            const uint32_t w3 = __ballot_sync(kFullMask, neg);
            if (lane == c * 4 + 0) mine = w0;
            if (lane == c * 4 + 1) mine = w1;
            if (lane == c * 4 + 2) mine = w2;
            if (lane == c * 4 + 3) mine = w3;
        }
    }
    if (lane < 4 * CODEC) __stcs(a.codes + (uint64_t)m * a.wpw + T * (4u * CODEC) + lane, mine);
}

template <int CODEC, int NORM, int SCALE, int PHASE>
__global__ void __launch_bounds__(256) encode_kernel(const EncodeArgs a) {
    const int lane = threadIdx.x & 31;
    const uint64_t warps_per_cta = blockDim.x >> 5;
    const uint64_t nwarps = (uint64_t)gridDim.x * warps_per_cta;
    for (uint64_t T = (uint64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5); T < a.ntile; T += nwarps) {
        const uint64_t i0 = T * kTile + (uint64_t)lane * 4u;
        uint32_t valid = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) valid |= (i0 + c < a.d) ? (1u << c) : 0u;
        float4 op = make_float4(0.f, 0.f, 0.f, 0.f);
        if (NORM == TNG_NORM_DIFF) {
            if (a.ref) op = load4(a.ref, i0, a.d);
        } else if (NORM == TNG_NORM_QUOT) {
            float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a.ref) r = load4(a.ref, i0, a.d);
            const float4 den = quot_den4(r, a.quot_eps);
            op = make_float4(__fdiv_rn(1.0f, den.x), __fdiv_rn(1.0f, den.y), __fdiv_rn(1.0f, den.z),
                             __fdiv_rn(1.0f, den.w));
        }
        const uint64_t blk = (PHASE == kPhaseQuant) ? (T * kTile) / a.block : T;
        for (uint32_t m0 = 0; m0 < a.M; m0 += 4) {
            float4 g[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (m0 + k < a.M) g[k] = load4_stream(a.grads + (uint64_t)(m0 + k) * a.ld, i0, a.d);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (m0 + k < a.M) encode_worker<CODEC, NORM, SCALE, PHASE>(a, g[k], op, m0 + k, T, blk, lane, valid);
        }
    }
}

// One level of the per-block scale reduction.  Row m holds n_in entries split
// into segments of `seg` entries (the last one ragged); CTA (segment, chunk)
// reduces entries [chunk*1024, chunk*1024+1024) of its segment, zero-padded, with
// an adjacent-pairwise tree (sum) or a NaN-propagating max, and writes one value.
// At the last level (chunks_per_seg == 1, final = 1) the value becomes the scale.
template <int SCALE>
__global__ void __launch_bounds__(256) block_scale_level_kernel(const float* __restrict__ in, uint64_t n_in,
                                                                uint64_t seg, uint64_t chunks_per_seg,
                                                                float* __restrict__ out, uint64_t n_out,
                                                                int final, unsigned long long* nonfinite) {
    __shared__ float buf[1024];
    const uint64_t s = blockIdx.x, c = blockIdx.y, m = blockIdx.z;
    const uint64_t seg_lo = s * seg;
    const uint64_t seg_hi = (seg_lo + seg < n_in) ? seg_lo + seg : n_in;
    const uint64_t lo = seg_lo + c * 1024u;
    const float* row = in + m * n_in;
    for (int i = threadIdx.x; i < 1024; i += 256) buf[i] = (lo + i < seg_hi) ? row[lo + i] : 0.0f;
    __syncthreads();
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
    if (threadIdx.x == 0) {
        float r = buf[0];
        if (final) {
            if (SCALE == 1) r = __fsqrt_rn(r);
            if (!(r < __int_as_float(0x7f800000))) atomicAdd(nonfinite, 1ull);
        }
        out[m * n_out + s * chunks_per_seg + c] = r;
    }
}

struct DecodeArgs {
    const uint32_t* codes;
    const float* scales;
    const float* ref;
    float* out_a;
    float* out_b;
    uint64_t d, ntile, nblk, block, wpw;
    uint32_t M;
    int levels;
    float quot_eps;
};

template <int CODEC>
__device__ __forceinline__ void decode_worker(const uint32_t (&w)[4 * CODEC], const float R, const int levels,
                                              const int lane, const bool first, float (&acc)[4]) {
    const bool ok = !scale_is_bad(R);
    float step = 0.f;
    if (CODEC == TNG_CODEC_QSGD4) step = __fdiv_rn(R, (float)levels);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float vh;
        if (CODEC == TNG_CODEC_TERN2) {
            const uint32_t nz = (w[c * 2] >> lane) & 1u, neg = (w[c * 2 + 1] >> lane) & 1u;
            vh = nz ? (neg ? -R : R) : 0.0f;
        } else if (CODEC == TNG_CODEC_SIGN1) {
            vh = ((w[c] >> lane) & 1u) ? R : -R;
        } else {
            const uint32_t L = ((w[c * 4] >> lane) & 1u) | (((w[c * 4 + 1] >> lane) & 1u) << 1) |
                               (((w[c * 4 + 2] >> lane) & 1u) << 2);
            const float mag = __fmul_rn((float)L, step);
            vh = ((w[c * 4 + 3] >> lane) & 1u) ? -mag : mag;
        }
        if (!ok) vh = 0.0f;
        acc[c] = first ? vh : __fadd_rn(acc[c], vh);
    }
}

template <int CODEC, int NORM>
__global__ void __launch_bounds__(256) decode_kernel(const DecodeArgs a) {
    const int lane = threadIdx.x & 31;
    const uint64_t warps_per_cta = blockDim.x >> 5;
    const uint64_t nwarps = (uint64_t)gridDim.x * warps_per_cta;
    constexpr int kWords = 4 * CODEC;
    for (uint64_t T = (uint64_t)blockIdx.x * warps_per_cta + (threadIdx.x >> 5); T < a.ntile; T += nwarps) {
        const uint64_t i0 = T * kTile + (uint64_t)lane * 4u;
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
        if (NORM != TNG_NORM_NONE && a.ref) r = load4(a.ref, i0, a.d);
        float4 den = make_float4(1.f, 1.f, 1.f, 1.f);
        if (NORM == TNG_NORM_QUOT) den = quot_den4(r, a.quot_eps);
        const uint64_t blk = (T * kTile) / a.block;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (uint32_t m0 = 0; m0 < a.M; m0 += 2) {
            uint32_t w[2][kWords];
            float R[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (m0 + k < a.M) {
                    const uint4* wp = reinterpret_cast<const uint4*>(a.codes + (uint64_t)(m0 + k) * a.wpw + T * kWords);
#pragma unroll
                    for (int q = 0; q < CODEC; ++q) {
                        const uint4 t = __ldg(wp + q);
                        w[k][4 * q + 0] = t.x; w[k][4 * q + 1] = t.y; w[k][4 * q + 2] = t.z; w[k][4 * q + 3] = t.w;
                    }
                    R[k] = __ldg(a.scales + (uint64_t)(m0 + k) * a.nblk + blk);
                }
            }
#pragma unroll
            for (int k = 0; k < 2; ++k)
                if (m0 + k < a.M) decode_worker<CODEC>(w[k], R[k], a.levels, lane, (m0 + k) == 0, acc);
        }
        // average over the M workers (Algorithm 1), then put the reference back (Eq. 2 / Eq. 3)
        const float fm = (float)a.M;
        float4 o;
        o.x = __fdiv_rn(acc[0], fm); o.y = __fdiv_rn(acc[1], fm); o.z = __fdiv_rn(acc[2], fm); o.w = __fdiv_rn(acc[3], fm);
        if (NORM == TNG_NORM_DIFF) {
            o.x = __fadd_rn(r.x, o.x); o.y = __fadd_rn(r.y, o.y); o.z = __fadd_rn(r.z, o.z); o.w = __fadd_rn(r.w, o.w);
        } else if (NORM == TNG_NORM_QUOT) {
            o.x = __fmul_rn(den.x, o.x); o.y = __fmul_rn(den.y, o.y); o.z = __fmul_rn(den.z, o.z); o.w = __fmul_rn(den.w, o.w);
        }
        if (a.out_a) store4(a.out_a, i0, a.d, o);
        if (a.out_b) store4(a.out_b, i0, a.d, o);
    }
}

int grid_for_tiles(uint64_t ntile, int sm_count, int ctas_per_sm) {
    const uint64_t want = (ntile + 7) / 8;   // 8 warps per CTA, one tile per warp per pass
    const uint64_t cap = (uint64_t)sm_count * ctas_per_sm;
    return (int)(want < cap ? (want ? want : 1) : cap);
}

template <int CODEC, int NORM, int SCALE>
cudaError_t encode_dispatch_phase(const EncodeArgs& a, int phase, int grid, cudaStream_t st) {
    if (phase == kPhaseFused) encode_kernel<CODEC, NORM, SCALE, kPhaseFused><<<grid, 256, 0, st>>>(a);
    else if (phase == kPhaseStat) encode_kernel<CODEC, NORM, SCALE, kPhaseStat><<<grid, 256, 0, st>>>(a);
    else encode_kernel<CODEC, NORM, SCALE, kPhaseQuant><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}
template <int CODEC, int NORM>
cudaError_t encode_dispatch_scale(const EncodeArgs& a, int scale, int phase, int grid, cudaStream_t st) {
    return scale == 0 ? encode_dispatch_phase<CODEC, NORM, 0>(a, phase, grid, st)
                      : encode_dispatch_phase<CODEC, NORM, 1>(a, phase, grid, st);
}
template <int CODEC>
cudaError_t encode_dispatch_norm(const EncodeArgs& a, int norm, int scale, int phase, int grid, cudaStream_t st) {
    switch (norm) {
        case TNG_NORM_DIFF: return encode_dispatch_scale<CODEC, TNG_NORM_DIFF>(a, scale, phase, grid, st);
        case TNG_NORM_QUOT: return encode_dispatch_scale<CODEC, TNG_NORM_QUOT>(a, scale, phase, grid, st);
        default: return encode_dispatch_scale<CODEC, TNG_NORM_NONE>(a, scale, phase, grid, st);
    }
}
cudaError_t encode_dispatch(const EncodeArgs& a, int codec, int norm, int scale, int phase, int grid, cudaStream_t st) {
    switch (codec) {
        case TNG_CODEC_SIGN1: return encode_dispatch_norm<TNG_CODEC_SIGN1>(a, norm, scale, phase, grid, st);
        case TNG_CODEC_TERN2: return encode_dispatch_norm<TNG_CODEC_TERN2>(a, norm, scale, phase, grid, st);
        default: return encode_dispatch_norm<TNG_CODEC_QSGD4>(a, norm, scale, phase, grid, st);
    }
}

template <int CODEC>
cudaError_t decode_dispatch_norm(const DecodeArgs& a, int norm, int grid, cudaStream_t st) {
    switch (norm) {
        case TNG_NORM_DIFF: decode_kernel<CODEC, TNG_NORM_DIFF><<<grid, 256, 0, st>>>(a); break;
        case TNG_NORM_QUOT: decode_kernel<CODEC, TNG_NORM_QUOT><<<grid, 256, 0, st>>>(a); break;
        default: decode_kernel<CODEC, TNG_NORM_NONE><<<grid, 256, 0, st>>>(a); break;
    }
    return cudaGetLastError();
}

}  // namespace

size_t tree_tmp_floats(const CodecGeom& g) {
    if (g.block == kTile) return 0;
    const uint64_t seg = (g.block + kTile - 1) / kTile;            // tiles per block
    const uint64_t chunks = (seg + 1023) / 1024;
    // two ping-pong levels, each at most M * nblk * chunks entries
    return (size_t)(2 * (uint64_t)g.M * g.nblk * chunks);
}

cudaError_t launch_encode(const CodecGeom& g, const float* grads, uint64_t ld, const float* ref, uint32_t step,
                          uint32_t* codes, float* scales, float* tile_stat, float* tree_tmp, FuseBlock* fb,
                          int sm_count, cudaStream_t st, int* launches) {
    EncodeArgs a;
    a.grads = grads; a.ref = ref; a.codes = codes; a.scales = scales; a.tile_stat = tile_stat;
    a.nonfinite = &fb->nonfinite;
    a.ld = ld; a.d = g.d; a.ntile = g.ntile; a.nblk = g.nblk; a.block = g.block; a.wpw = g.wpw;
    a.M = g.M; a.step = step; a.seed_lo = g.seed_lo; a.seed_hi = g.seed_hi; a.levels = g.levels;
    a.quot_eps = g.quot_eps;
    const int grid = grid_for_tiles(g.ntile, sm_count, 8);
    cudaError_t e;
    if (g.block == kTile) {
        e = encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseFused, grid, st);
        ++*launches;
        return e;
    }
    // general block size: per-tile statistic -> per-block tree -> quantise
    e = encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseStat, grid, st);
    ++*launches;
    if (e != cudaSuccess) return e;
    const float* in = tile_stat;
    uint64_t n_in = g.ntile;
    uint64_t seg = (g.block + kTile - 1) / kTile;
    float* ping = tree_tmp;
    float* pong = tree_tmp + tree_tmp_floats(g) / 2;
    for (;;) {
        const uint64_t chunks = (seg + 1023) / 1024;
        const int final = chunks == 1;
        float* out = final ? scales : ping;
        const uint64_t n_out = g.nblk * chunks;
        dim3 grid3((unsigned)g.nblk, (unsigned)chunks, g.M);
        if (g.scale_kind == 0)
            block_scale_level_kernel<0><<<grid3, 256, 0, st>>>(in, n_in, seg, chunks, out, n_out, final, &fb->nonfinite);
        else
            block_scale_level_kernel<1><<<grid3, 256, 0, st>>>(in, n_in, seg, chunks, out, n_out, final, &fb->nonfinite);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess || final) break;
        in = out; n_in = n_out; seg = chunks;
        float* t = ping; ping = pong; pong = t;
    }
    if (e != cudaSuccess) return e;
    e = encode_dispatch(a, g.codec, g.norm, g.scale_kind, kPhaseQuant, grid, st);
    ++*launches;
    return e;
}

cudaError_t launch_decode(const CodecGeom& g, const uint32_t* codes, const float* scales, const float* ref,
                          float* out_a, float* out_b, int sm_count, cudaStream_t st, int* launches) {
    DecodeArgs a;
    a.codes = codes; a.scales = scales; a.ref = ref; a.out_a = out_a; a.out_b = out_b;
    a.d = g.d; a.ntile = g.ntile; a.nblk = g.nblk; a.block = g.block; a.wpw = g.wpw; a.M = g.M;
    a.levels = g.levels; a.quot_eps = g.quot_eps;
    const int grid = grid_for_tiles(g.ntile, sm_count, 8);
    cudaError_t e;
    switch (g.codec) {
        case TNG_CODEC_SIGN1: e = decode_dispatch_norm<TNG_CODEC_SIGN1>(a, g.norm, grid, st); break;
        case TNG_CODEC_TERN2: e = decode_dispatch_norm<TNG_CODEC_TERN2>(a, g.norm, grid, st); break;
        default: e = decode_dispatch_norm<TNG_CODEC_QSGD4>(a, g.norm, grid, st); break;
    }
    ++*launches;
    return e;
}

}  // namespace tng
