// Device-side building blocks shared by the libtng kernels (sm_100a).
//
// Everything that decides a code bit uses explicit round-to-nearest intrinsics
// (__fsub_rn, __fmul_rn, __fadd_rn, __fdiv_rn, __fsqrt_rn), so the compiler can
// neither contract them into FMAs nor replace them by approximations.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace tng {

constexpr int kTile = 128;          // coordinates per wire tile = one warp x float4
constexpr unsigned kFullMask = 0xFFFFFFFFu;

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).  One call yields the four
// uniforms of the four coordinates a lane owns.  The ten round keys (key plus
// multiples of the Weyl constants) are the same for every call of a launch, so
// the host computes them once and the kernel reads them from its arguments.
// ---------------------------------------------------------------------------
constexpr uint32_t kPhiloxMul0 = 0xD2511F53u, kPhiloxMul1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxWeyl0 = 0x9E3779B9u, kPhiloxWeyl1 = 0xBB67AE85u;

inline void philox_round_keys(uint32_t k0, uint32_t k1, uint32_t (&rk)[20]) {
    for (int round = 0; round < 10; ++round) {
        rk[2 * round] = k0;
        rk[2 * round + 1] = k1;
        k0 += kPhiloxWeyl0;
        k1 += kPhiloxWeyl1;
    }
}

__device__ __forceinline__ uint4 philox4x32_10_rk(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                  const uint32_t (&rk)[20]) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = static_cast<uint64_t>(kPhiloxMul0) * c0;
        const uint64_t p1 = static_cast<uint64_t>(kPhiloxMul1) * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ rk[2 * round];
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ rk[2 * round + 1];
        c1 = static_cast<uint32_t>(p1);
        c3 = static_cast<uint32_t>(p0);
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// N independent calls that differ only in counter word c2, with their rounds interleaved in
// program order: the ten rounds of one call form one long dependency chain, N chains side by
// side keep the pipes busy.
template <int N>
__device__ __forceinline__ void philox4x32_10_rk_batch(uint32_t c0, uint32_t c1, uint32_t c2_first, uint32_t c3,
                                                       const uint32_t (&rk)[20], uint4 (&out)[N]) {
    uint32_t a0[N], a1[N], a2[N], a3[N];
#pragma unroll
    for (int i = 0; i < N; ++i) { a0[i] = c0; a1[i] = c1; a2[i] = c2_first + (uint32_t)i; a3[i] = c3; }
#pragma unroll
    for (int round = 0; round < 10; ++round) {
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const uint64_t p0 = static_cast<uint64_t>(kPhiloxMul0) * a0[i];
            const uint64_t p1 = static_cast<uint64_t>(kPhiloxMul1) * a2[i];
            const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ a1[i] ^ rk[2 * round];
            const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ a3[i] ^ rk[2 * round + 1];
            a1[i] = static_cast<uint32_t>(p1);
            a3[i] = static_cast<uint32_t>(p0);
            a0[i] = n0;
            a2[i] = n2;
        }
    }
#pragma unroll
    for (int i = 0; i < N; ++i) out[i] = make_uint4(a0[i], a1[i], a2[i], a3[i]);
}

// u in [0,1) on a 2^-24 grid: the top 24 bits of the word (exact in fp32).
__device__ __forceinline__ float uniform24(uint32_t x) {
    return __uint2float_rn(x >> 8) * 0x1p-24f;
}

// ---------------------------------------------------------------------------
// 128-bit loads/stores with a ragged tail.  `i` is the first of four consecutive
// coordinates, `d` the vector length; elements at or beyond d read as zero and
// are not written.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float4 load4_stream(const float* __restrict__ p, uint64_t i, uint64_t d) {
    if (i + 4 <= d) return __ldcs(reinterpret_cast<const float4*>(p + i));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < d) r.x = __ldcs(p + i);
    if (i + 1 < d) r.y = __ldcs(p + i + 1);
    if (i + 2 < d) r.z = __ldcs(p + i + 2);
    return r;
}
__device__ __forceinline__ float4 load4(const float* __restrict__ p, uint64_t i, uint64_t d) {
    if (i + 4 <= d) return *reinterpret_cast<const float4*>(p + i);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < d) r.x = p[i];
    if (i + 1 < d) r.y = p[i + 1];
    if (i + 2 < d) r.z = p[i + 2];
    return r;
}
__device__ __forceinline__ void store4(float* __restrict__ p, uint64_t i, uint64_t d, float4 v) {
    if (i + 4 <= d) {
        *reinterpret_cast<float4*>(p + i) = v;
        return;
    }
    if (i < d) p[i] = v.x;
    if (i + 1 < d) p[i + 1] = v.y;
    if (i + 2 < d) p[i + 2] = v.z;
}

// ---------------------------------------------------------------------------
// warp reductions
// ---------------------------------------------------------------------------
// max of |x| over the warp's 128 values; any NaN wins (its bit pattern is above
// +inf's), so a block with a NaN gets a NaN scale.
__device__ __forceinline__ float warp_absmax(float a, float b, float c, float d) {
    uint32_t m = __float_as_uint(fabsf(a));
    m = max(m, __float_as_uint(fabsf(b)));
    m = max(m, __float_as_uint(fabsf(c)));
    m = max(m, __float_as_uint(fabsf(d)));
    return __uint_as_float(__reduce_max_sync(kFullMask, m));
}

// fp32 adjacent-pairwise tree sum of the warp's 128 squares: lane j holds the
// squares of coordinates 4j..4j+3, xor-shuffles pair neighbouring lanes.
__device__ __forceinline__ float warp_sumsq_tree(float a, float b, float c, float d) {
    float s = __fadd_rn(__fadd_rn(__fmul_rn(a, a), __fmul_rn(b, b)),
                        __fadd_rn(__fmul_rn(c, c), __fmul_rn(d, d)));
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) s = __fadd_rn(s, __shfl_xor_sync(kFullMask, s, off));
    return s;
}

__device__ __forceinline__ bool scale_is_bad(float R) { return !(R > 0.0f) || !(R < __int_as_float(0x7f800000)); }

// Guarded denominator of the quotient form for one tile: mx = max|r| over the
// tile; not a positive finite number -> 1; else sign(r) max(|r|, eps*mx), zero
// counting as positive.
__device__ __forceinline__ float4 quot_den4(float4 r, float eps) {
    const float mx = warp_absmax(r.x, r.y, r.z, r.w);
    if (scale_is_bad(mx)) return make_float4(1.f, 1.f, 1.f, 1.f);
    const float fl = __fmul_rn(eps, mx);
    float4 den;
    float a;
    a = fabsf(r.x); a = a > fl ? a : fl; den.x = (r.x < 0.f) ? -a : a;
    a = fabsf(r.y); a = a > fl ? a : fl; den.y = (r.y < 0.f) ? -a : a;
    a = fabsf(r.z); a = a > fl ? a : fl; den.z = (r.z < 0.f) ? -a : a;
    a = fabsf(r.w); a = a > fl ? a : fl; den.w = (r.w < 0.f) ? -a : a;
    return den;
}

}  // namespace tng
