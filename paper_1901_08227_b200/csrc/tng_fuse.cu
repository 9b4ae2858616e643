// Trajectory fusion kernels (sm_100a): the sufficient statistics of
//   min_alpha sum_m || g^m - sum_j alpha_j h_j ||^2
// (the C_nz criterion of Proposition 2 over the span of the stored aggregates of
// Section 3.1): Gram G = <h_i,h_j>, rhs c_i = <h_i, mean gradient>; a K x K
// ridge solve; and the reference combine r = sum_j alpha_j h_j.
//
// The statistics pass is one streaming sweep over the ring and the M gradient
// rows.  Each thread owns four coordinates per iteration (128-bit loads of all
// k + M vectors), converts them to double once and accumulates every pair
// product in double, so the result does not depend on how the sum is split.
// Per-CTA partials are combined in CTA order by the CTA that finishes last
// (an arrival counter, nobody waits), which keeps the sums run-to-run identical.
#include "tng_device.cuh"
#include "tng_internal.h"
#include "tng_pipeline.cuh"

namespace tng {

namespace {

constexpr int kDotsThreads = 256;

struct DotsArgs {
    const float* rows_a[8];
    const float* rows_b[8];
    const float* grads;       // nullptr: Gram only
    double* partials;         // gridDim.x * kDotsMaxAcc
    FuseBlock* fb;
    uint64_t d, ld;
    uint32_t M;
    uint32_t divisor;         // rhs and grad_sq are divided by this (M for means, 1 for raw sums)
    short dst[kDotsMaxAcc];   // destination of accumulator i inside fb->gram
};

template <int NA, int NB, bool SAME>
struct DotsShape {
    static constexpr int kPairs = SAME ? NA * (NA + 1) / 2 : NA * NB;
    static constexpr int kAcc = SAME ? kPairs + NA + 1 : kPairs;   // + rhs + grad_sq
};

// CTA reduction (lanes by butterfly, warps in warp order), one partial row per CTA, and
// the CTA that arrives last adds the partial rows in CTA order: run-to-run identical sums,
// nobody waits.  Called by the kDotsThreads threads that hold accumulators (tid in [0, kDotsThreads)) and
// by nobody else: its barriers count exactly those threads.
__device__ __forceinline__ void dots_threads_barrier() {
    asm volatile("bar.sync 2, %0;" ::"n"(kDotsThreads) : "memory");
}
template <int kAcc, int kPairs, bool SAME>
__device__ __forceinline__ void dots_finish(const double (&acc)[kAcc], const DotsArgs& a, const bool with_g, const int tid) {
    __shared__ double warp_part[kDotsThreads / 32][kAcc];
    __shared__ bool is_last;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int i = 0; i < kAcc; ++i) {
        double v = acc[i];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(kFullMask, v, off);
        if (lane == 0) warp_part[warp][i] = v;
    }
    dots_threads_barrier();
    if (tid < kAcc) {
        double v = 0.0;
        for (int w = 0; w < kDotsThreads / 32; ++w) v += warp_part[w][tid];
        a.partials[(uint64_t)blockIdx.x * kDotsMaxAcc + tid] = v;
    }
    __threadfence();
    dots_threads_barrier();
    if (tid == 0) {
        const uint32_t prev = atomicAdd(&a.fb->dots_arrivals, 1u);
        is_last = (prev == gridDim.x - 1);
    }
    dots_threads_barrier();
    if (!is_last) return;
    __threadfence();
    if (tid < kAcc) {
        double v = 0.0;
        for (uint32_t b = 0; b < gridDim.x; ++b) v += __ldcg(a.partials + (uint64_t)b * kDotsMaxAcc + tid);
        if (SAME && tid >= kPairs) v /= (double)a.divisor;   // rhs and grad_sq: mean over the rows, or raw sums
        if (!(SAME && !with_g && tid >= kPairs)) a.fb->gram[a.dst[tid]] = v;
    }
    if (tid == 0) a.fb->dots_arrivals = 0;   // ready for the next launch on this stream
}

// ---------------------------------------------------------------------------
// Statistics pass fed by the bulk-copy pipeline (k <= 8 history rows in one launch).
// Virtual row list: h_1..h_k, then g^0..g^{M-1}.  A chunk of 1024 coordinates of up to 16
// rows is one stage; consumer thread t owns coordinates 4t..4t+3 of the chunk, keeps the
// history values of the chunk in registers while the gradient rows stream through the
// following fills, and accumulates exactly what dots_kernel accumulates.  The ragged end
// of the vectors (d mod 1024) is read directly.
// ---------------------------------------------------------------------------
// 8 consumer warps (two warpgroups) + one warpgroup of which one thread feeds the pipeline.  The kernel starts
// with kDotsLaunchRegs registers per thread; the feeding warpgroup gives all but kDotsFeedRegs of its share back and
// the consumers take it (setmaxnreg), so that the 45 double accumulators of eight history rows, the rows' values
// and the gradient sums fit in registers.  The shares add up exactly:
//   256 x kDotsConsumerRegs + 128 x kDotsFeedRegs = 384 x kDotsLaunchRegs = 64512  (and, per SM partition, which holds
//   two consumer warps and one feeding warp: 32 x (2 x 240 + 24) = 16128 <= 16384).
constexpr int kDotsPipeThreads = kDotsThreads + 128;
constexpr int kDotsLaunchRegs = 168, kDotsConsumerRegs = 240, kDotsFeedRegs = 24;
static_assert(kDotsThreads * kDotsConsumerRegs + 128 * kDotsFeedRegs == kDotsPipeThreads * kDotsLaunchRegs, "register shares must add up to what the launch holds");
using DotsGeom = PipeGeom<1024, 16, 3>;                // 64 KiB stages: a chunk of 1024 coordinates of 16 rows
constexpr uint64_t kDotsPipeMinCoords = 16 * DotsGeom::kChunk;   // shorter vectors take the direct kernel

struct DotsPipeArgs {
    DotsArgs base;      // rows_a = history rows, grads/ld/M, partials, fb, dst
    PipeRows rows;      // history rows then gradient rows
};

// The sum of the M gradients at a coordinate enters the right-hand side, which decides the coefficients down
// to their last fp32 bit: it is kept in double, like everything else the coefficients depend on.  The sum
// of squares only feeds the C_nz estimate: fp32.
struct GradSums {
    double sum[4];
    float4 sq;
};
__device__ __forceinline__ void grad_sums(GradSums& a, const float4 g) {
    a.sum[0] += (double)g.x; a.sum[1] += (double)g.y; a.sum[2] += (double)g.z; a.sum[3] += (double)g.w;
    a.sq.x = fmaf(g.x, g.x, a.sq.x); a.sq.y = fmaf(g.y, g.y, a.sq.y); a.sq.z = fmaf(g.z, g.z, a.sq.z); a.sq.w = fmaf(g.w, g.w, a.sq.w);
}
__device__ __forceinline__ GradSums grad_sums_zero() {
    GradSums a;
    a.sum[0] = a.sum[1] = a.sum[2] = a.sum[3] = 0.0;
    a.sq = make_float4(0.f, 0.f, 0.f, 0.f);
    return a;
}

// acc += products of the four coordinates held in ha[] (history) and gs/gq (sum and sum of
// squares of the gradients at these coordinates, fp32, m ascending)
template <int NA>
__device__ __forceinline__ void dots_accum4(const float4 (&ha)[NA], const GradSums& gsum, const bool with_g,
                                            double (&acc)[NA * (NA + 1) / 2 + NA + 1]) {
    const float4 gq = gsum.sq;
    constexpr int kPairs = NA * (NA + 1) / 2;
#pragma unroll
    for (int comp = 0; comp < 4; ++comp) {
        double da[NA];
#pragma unroll
        for (int j = 0; j < NA; ++j) da[j] = (double)(comp == 0 ? ha[j].x : comp == 1 ? ha[j].y : comp == 2 ? ha[j].z : ha[j].w);
        int p = 0;
#pragma unroll
        for (int i = 0; i < NA; ++i)
#pragma unroll
            for (int j = i; j < NA; ++j) { acc[p] = fma(da[i], da[j], acc[p]); ++p; }
        if (with_g) {
            const double dg = gsum.sum[comp];
#pragma unroll
            for (int i = 0; i < NA; ++i) acc[kPairs + i] = fma(da[i], dg, acc[kPairs + i]);
            acc[kPairs + NA] += (double)(comp == 0 ? gq.x : comp == 1 ? gq.y : comp == 2 ? gq.z : gq.w);
        }
    }
}


template <int NA>
__global__ void __launch_bounds__(kDotsPipeThreads, 1) dots_pipe_kernel(const DotsPipeArgs pa) {
    extern __shared__ unsigned char dyn_smem[];
    constexpr int kPairs = NA * (NA + 1) / 2;
    constexpr int kAcc = kPairs + NA + 1;
    const DotsArgs& a = pa.base;
    using G = DotsGeom;
    const PipeSmem pipe = pipe_setup<G>(dyn_smem, kDotsThreads / 32);
    const bool with_g = a.grads != nullptr;
    const uint64_t nchunks = a.d / G::kChunk;
    const int tid = threadIdx.x;
    if (tid >= kDotsThreads) {
        // ---- the feeding warpgroup: hands its registers over, then one thread feeds the stages
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDotsFeedRegs));
        if (tid == kDotsThreads) {
            const uint32_t err = pipe_produce<G>(pipe, pa.rows, blockIdx.x, gridDim.x, nchunks);
            if (err != kPipeOk) atomicMax(&a.fb->pipe_error, err);
        }
        return;
    }
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kDotsConsumerRegs));
    double acc[kAcc];
#pragma unroll
    for (int i = 0; i < kAcc; ++i) acc[i] = 0.0;
    {
        // ---- consumers: fill 0 of a chunk holds the NA history rows, the others gradient rows
        const int lane = tid & 31;
        const uint32_t my = (uint32_t)tid * 16u;                  // byte offset of the thread's float4 inside a row chunk
        const int ngrad = pa.rows.nrows - pa.rows.n_pre;
        uint32_t it = 0;
        bool alive = true;
        for (uint64_t c = blockIdx.x; c < nchunks && alive; c += gridDim.x) {
            float4 ha[NA];
            GradSums gsum = grad_sums_zero();
            for (int g0 = -G::kRows; g0 < ngrad; g0 += G::kRows) {   // g0 < 0: the history fill
                const uint32_t s = it % G::kStages, use = it / G::kStages;
                if (!__all_sync(kFullMask, mbar_wait(pipe.full(s), use & 1u))) {   // warp-uniform outcome
                    atomicMax(&a.fb->pipe_error, (uint32_t)kPipeFullTimeout);
                    alive = false;
                    break;
                }
                const uint32_t base = pipe.data + s * G::kStageBytes + my;
                if (g0 < 0) {
#pragma unroll
                    for (int j = 0; j < NA; ++j) ha[j] = lds128(base + (uint32_t)j * G::kRowBytes);
                } else {
                    const int n = (ngrad - g0 < G::kRows) ? ngrad - g0 : G::kRows;
                    for (int r = 0; r < n; ++r) grad_sums(gsum, lds128(base + (uint32_t)r * G::kRowBytes));
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(pipe.empty(s));       // this warp has read the stage
                ++it;
            }
            if (alive) dots_accum4<NA>(ha, gsum, with_g, acc);
        }
        // ---- ragged end: coordinates [nchunks*1024, d) straight from global memory
        const uint64_t ngroups = (a.d + 3) / 4;
        for (uint64_t grp = nchunks * (G::kChunk / 4) + (uint64_t)blockIdx.x * kDotsThreads + tid; grp < ngroups;
             grp += (uint64_t)gridDim.x * kDotsThreads) {
            const uint64_t i0 = grp * 4;
            float4 ha[NA];
#pragma unroll
            for (int j = 0; j < NA; ++j) ha[j] = load4_stream(a.rows_a[j], i0, a.d);
            GradSums gsum = grad_sums_zero();
            if (with_g)
                for (uint32_t m = 0; m < a.M; ++m) grad_sums(gsum, load4_stream(a.grads + (uint64_t)m * a.ld, i0, a.d));
            dots_accum4<NA>(ha, gsum, with_g, acc);
        }
    }
    dots_finish<kAcc, kPairs, true>(acc, a, with_g, tid);
}

template <int NA, int NB, bool SAME>
__global__ void __launch_bounds__(kDotsThreads, 1) dots_kernel(const DotsArgs a) {
    using Shape = DotsShape<NA, NB, SAME>;
    constexpr int kAcc = Shape::kAcc;
    double acc[kAcc];
#pragma unroll
    for (int i = 0; i < kAcc; ++i) acc[i] = 0.0;
    const bool with_g = SAME && (a.grads != nullptr);

    const uint64_t ngroups = (a.d + 3) / 4;
    const uint64_t stride = (uint64_t)gridDim.x * kDotsThreads;
    for (uint64_t grp = (uint64_t)blockIdx.x * kDotsThreads + threadIdx.x; grp < ngroups; grp += stride) {
        const uint64_t i0 = grp * 4;
        float4 ha[NA];
        float4 hb[SAME ? 1 : NB];
#pragma unroll
        for (int j = 0; j < NA; ++j) ha[j] = load4_stream(a.rows_a[j], i0, a.d);
        if (!SAME) {
#pragma unroll
            for (int j = 0; j < NB; ++j) hb[j] = load4_stream(a.rows_b[j], i0, a.d);
        }
        // sum (double) and sum of squares (fp32) of the M gradients at these coordinates, m ascending
        GradSums gsum = grad_sums_zero();
        if (with_g) {
            for (uint32_t m0 = 0; m0 < a.M; m0 += 8) {
                float4 g[8];
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (m0 + k < a.M) g[k] = load4_stream(a.grads + (uint64_t)(m0 + k) * a.ld, i0, a.d);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (m0 + k < a.M) grad_sums(gsum, g[k]);
            }
        }
#pragma unroll
        for (int comp = 0; comp < 4; ++comp) {
            double da[NA];
#pragma unroll
            for (int j = 0; j < NA; ++j) da[j] = (double)(comp == 0 ? ha[j].x : comp == 1 ? ha[j].y : comp == 2 ? ha[j].z : ha[j].w);
            if (SAME) {
                int p = 0;
#pragma unroll
                for (int i = 0; i < NA; ++i)
#pragma unroll
                    for (int j = i; j < NA; ++j) { acc[p] = fma(da[i], da[j], acc[p]); ++p; }
                if (with_g) {
                    const double dg = gsum.sum[comp];
#pragma unroll
                    for (int i = 0; i < NA; ++i) acc[Shape::kPairs + i] = fma(da[i], dg, acc[Shape::kPairs + i]);
                    acc[Shape::kPairs + NA] += (double)(comp == 0 ? gsum.sq.x : comp == 1 ? gsum.sq.y : comp == 2 ? gsum.sq.z : gsum.sq.w);
                }
            } else {
                double db[SAME ? 1 : NB];
#pragma unroll
                for (int j = 0; j < NB; ++j) db[j] = (double)(comp == 0 ? hb[j].x : comp == 1 ? hb[j].y : comp == 2 ? hb[j].z : hb[j].w);
#pragma unroll
                for (int i = 0; i < NA; ++i)
#pragma unroll
                    for (int j = 0; j < NB; ++j) acc[i * NB + j] = fma(da[i], db[j], acc[i * NB + j]);
            }
        }
    }

    dots_finish<kAcc, Shape::kPairs, SAME>(acc, a, with_g, threadIdx.x);
}

template <int NA>
cudaError_t dots_same(const DotsArgs& a, int grid, cudaStream_t st) {
    dots_kernel<NA, NA, true><<<grid, kDotsThreads, 0, st>>>(a);
    return cudaGetLastError();
}
template <int NB>
cudaError_t dots_cross(const DotsArgs& a, int grid, cudaStream_t st) {
    dots_kernel<8, NB, false><<<grid, kDotsThreads, 0, st>>>(a);
    return cudaGetLastError();
}

template <int NA>
cudaError_t dots_pipe(const DotsPipeArgs& pa, int grid, cudaStream_t st) {
    static PerDevice<bool> configured;   // opt in to the large dynamic shared memory once per instantiation and device
    const int slot = device_slot();
    if (slot < 0 || !configured.v[slot]) {
        cudaError_t e = cudaFuncSetAttribute(dots_pipe_kernel<NA>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DotsGeom::kSmemBytes);
        if (e != cudaSuccess) return e;
        if (slot >= 0) configured.v[slot] = true;
    }
    // The register hand-over inside the kernel only ends if the launch really holds kDotsLaunchRegs per thread:
    // ask what the kernel was built with instead of trusting it.
    static PerDevice<int> launch_regs;
    int regs = slot >= 0 ? launch_regs.v[slot] : 0;
    if (regs == 0) {
        cudaFuncAttributes attr;
        cudaError_t e = cudaFuncGetAttributes(&attr, dots_pipe_kernel<NA>);
        if (e != cudaSuccess) return e;
        regs = attr.numRegs;
        if (slot >= 0) launch_regs.v[slot] = regs;
    }
    if (regs != kDotsLaunchRegs) return cudaErrorLaunchOutOfResources;
    dots_pipe_kernel<NA><<<grid, kDotsPipeThreads, DotsGeom::kSmemBytes, st>>>(pa);
    return cudaGetLastError();
}
cudaError_t dots_pipe_n(int n, const DotsPipeArgs& pa, int grid, cudaStream_t st) {
    switch (n) {
        case 1: return dots_pipe<1>(pa, grid, st);
        case 2: return dots_pipe<2>(pa, grid, st);
        case 3: return dots_pipe<3>(pa, grid, st);
        case 4: return dots_pipe<4>(pa, grid, st);
        case 5: return dots_pipe<5>(pa, grid, st);
        case 6: return dots_pipe<6>(pa, grid, st);
        case 7: return dots_pipe<7>(pa, grid, st);
        default: return dots_pipe<8>(pa, grid, st);
    }
}

cudaError_t dots_same_n(int n, const DotsArgs& a, int grid, cudaStream_t st) {
    switch (n) {
        case 1: return dots_same<1>(a, grid, st);
        case 2: return dots_same<2>(a, grid, st);
        case 3: return dots_same<3>(a, grid, st);
        case 4: return dots_same<4>(a, grid, st);
        case 5: return dots_same<5>(a, grid, st);
        case 6: return dots_same<6>(a, grid, st);
        case 7: return dots_same<7>(a, grid, st);
        default: return dots_same<8>(a, grid, st);
    }
}
cudaError_t dots_cross_n(int n, const DotsArgs& a, int grid, cudaStream_t st) {
    switch (n) {
        case 1: return dots_cross<1>(a, grid, st);
        case 2: return dots_cross<2>(a, grid, st);
        case 3: return dots_cross<3>(a, grid, st);
        case 4: return dots_cross<4>(a, grid, st);
        case 5: return dots_cross<5>(a, grid, st);
        case 6: return dots_cross<6>(a, grid, st);
        case 7: return dots_cross<7>(a, grid, st);
        default: return dots_cross<8>(a, grid, st);
    }
}

// ---------------------------------------------------------------------------
// K x K ridge solve by one warp (k <= 16), fp64.  mode: TNG_FUSE_LSQ, TNG_FUSE_HINDSIGHT,
// TNG_FUSE_MEAN, TNG_FUSE_LAST.
//
// Lane i owns row i of the augmented system [A | b] in shared memory.  Elimination is
// right-looking: at step j every lane below the pivot scales its entry of column j by the
// reciprocal of the pivot's root, then subtracts the rank-one term from the rest of its row and from its b.
// When the sweep ends column n holds the forward-substituted right-hand side, so only the
// backward sweep (column by column, again one lane per row) remains.  A pivot that is not a
// finite positive number above 1e-12 of the diagonal entry it started from is rounding
// noise of a singular matrix: the solve reports failure and the caller falls back to the
// newest history vector alone.
// ---------------------------------------------------------------------------
constexpr int kSolveLd = kMaxK + 1;   // row stride of the augmented system

// S: n rows of n + 1 entries (stride kSolveLd); all 32 lanes call; returns the same verdict in every lane
// and leaves the solution in x[0..n).
__device__ bool warp_spd_solve(double* S, double* x, const int n, const int lane) {
    const double start_diag = (lane < n) ? S[lane * kSolveLd + lane] : 1.0;
    bool good = true;
    for (int j = 0; j < n; ++j) {
        const double piv = S[j * kSolveLd + j];
        const double ref = __shfl_sync(kFullMask, start_diag, j);
        if (!(piv > 1e-12 * ref) || !(piv > 0.0) || !isfinite(piv)) { good = false; break; }   // the same in all lanes
        // one reciprocal square root per pivot; everything else multiplies by it (the diagonal keeps 1/root,
        // which is what the backward sweep needs)
        const double rinv = rsqrt(piv);
        __syncwarp();
        if (lane >= j && lane < n) S[lane * kSolveLd + j] = (lane == j) ? rinv : S[lane * kSolveLd + j] * rinv;
        if (lane == j) S[j * kSolveLd + n] *= rinv;
        __syncwarp();
        if (lane > j && lane < n) {
            const double mine = S[lane * kSolveLd + j];
            for (int c = j + 1; c <= lane; ++c) S[lane * kSolveLd + c] -= mine * S[c * kSolveLd + j];
            S[lane * kSolveLd + n] -= mine * S[j * kSolveLd + n];
        }
        __syncwarp();
    }
    if (!good) return false;
    // backward sweep on L^T: the newest unknown is final, every lane above it removes its share
    for (int i = n - 1; i >= 0; --i) {
        if (lane == i) S[i * kSolveLd + n] *= S[i * kSolveLd + i];   // the diagonal holds 1/root
        __syncwarp();
        if (lane < i) S[lane * kSolveLd + n] -= S[i * kSolveLd + lane] * S[i * kSolveLd + n];
        __syncwarp();
    }
    const double xi = (lane < n) ? S[lane * kSolveLd + n] : 0.0;
    if (lane < n) x[lane] = xi;
    __syncwarp();
    return __all_sync(kFullMask, isfinite(xi));
}

__global__ void __launch_bounds__(32) solve_kernel(FuseBlock* fb, int k, int mode, double ridge, int have_rhs, double rhs_div) {
    // the whole warp brings the statistics into shared memory (one round trip to global memory
    // instead of one per entry) and writes the mirrored Gram back
    __shared__ double sG[kGramDoubles];
    __shared__ double sS[kMaxK * kSolveLd];
    __shared__ double sx[kMaxK];
    const int lane = threadIdx.x;
    const bool stats = (mode == TNG_FUSE_LSQ) || (mode == TNG_FUSE_HINDSIGHT);
    if (stats) {
        for (int i = lane; i < kGramDoubles; i += 32) {
            double v = fb->gram[i];
            if (rhs_div != 1.0 && i >= kGramRhs) {   // sums over all workers -> means
                v /= rhs_div;
                fb->gram[i] = v;
            }
            sG[i] = v;
        }
        __syncwarp();
        for (int i = lane; i < k * k; i += 32) {   // mirror the upper triangle
            const int a = i / k, b = i % k;
            if (b < a) {
                const double v = sG[b * kGramStride + a];
                sG[a * kGramStride + b] = v;
                fb->gram[a * kGramStride + b] = v;
            }
        }
        __syncwarp();
    }
    double alpha = 0.0;   // lane j holds alpha_j
    uint32_t fallback = 0;
    if (mode == TNG_FUSE_MEAN) {
        if (lane < k) alpha = (double)__fdiv_rn(1.0f, (float)k);
    } else if (mode == TNG_FUSE_LAST) {
        if (lane == 0) alpha = 1.0;
    } else {
        // LSQ: all k vectors against <h_j, mean gradient>.  Hindsight: regress h_1 on h_2..h_k (the
        // sub-Gram without row/column 0 against column 0) and apply the coefficients one position later.
        const int off = (mode == TNG_FUSE_LSQ) ? 0 : 1;
        const int n = k - off;
        if (n >= 1) {
            double tr = (lane < n) ? sG[(lane + off) * kGramStride + lane + off] : 0.0;
            // the trace is summed serially, entry 0 first (the order of a plain loop)
            double trace = 0.0;
            for (int j = 0; j < n; ++j) trace += __shfl_sync(kFullMask, tr, j);
            const double lambda = ridge * trace / (double)n;
            if (lane < n) {
                for (int b = 0; b < n; ++b) sS[lane * kSolveLd + b] = sG[(lane + off) * kGramStride + b + off] + (b == lane ? lambda : 0.0);
                sS[lane * kSolveLd + n] = (mode == TNG_FUSE_LSQ) ? sG[kGramRhs + lane] : sG[(lane + 1) * kGramStride];
            }
            __syncwarp();
            if (warp_spd_solve(sS, sx, n, lane)) {
                if (lane < n) alpha = sx[lane];
            } else {
                fallback = 1;
                alpha = (lane == 0) ? 1.0 : 0.0;
            }
        } else {
            alpha = (lane == 0) ? 1.0 : 0.0;   // a single stored vector has no past to regress on
        }
    }
    const float a32f = (float)alpha;
    if (lane < kMaxK) {
        fb->alpha64[lane] = alpha;
        fb->alpha32[lane] = a32f;
    }
    if (lane == 0) fb->fallback = fallback;
    // C_nz estimate from the statistics: (gg - 2 a.c + a^T G a) / gg with the fp32 coefficients;
    // lane a takes row a, the rows are added in lane order
    double cnz = nan("");
    if (have_rhs && mode != TNG_FUSE_MEAN) {
        const double a32 = (double)a32f;
        double row = 0.0;
        for (int b = 0; b < k; ++b) {
            const double ab = __shfl_sync(kFullMask, a32, b);
            if (lane < k) row += ab * sG[lane * kGramStride + b];
        }
        double quad_l = (lane < k) ? a32 * row : 0.0;
        double lin_l = (lane < k) ? a32 * sG[kGramRhs + lane] : 0.0;
        double quad = 0.0, lin = 0.0;
        for (int a = 0; a < k; ++a) {
            quad += __shfl_sync(kFullMask, quad_l, a);
            lin += __shfl_sync(kFullMask, lin_l, a);
        }
        const double gg = sG[kGramGG];
        cnz = (gg - 2.0 * lin + quad) / gg;
    }
    if (lane == 0) fb->cnz = cnz;
}

// ---------------------------------------------------------------------------
// reference combine: r_d = fma(alpha_k, h_k[d], ... fma(alpha_1, h_1[d], 0)), fp32
// ---------------------------------------------------------------------------
struct CombineArgs {
    const float* rows[kMaxK];
    const float* alpha;
    float* ref;
    float* ref2;     // nullptr, or the second reference r' = (1/k) sum_j |h_j|
    float inv_k;
    uint64_t d;
};

template <int KK>
__global__ void __launch_bounds__(256) combine_kernel(const CombineArgs a) {
    float al[KK];
#pragma unroll
    for (int j = 0; j < KK; ++j) al[j] = __ldg(a.alpha + j);
    const uint64_t ngroups = (a.d + 3) / 4;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += stride) {
        const uint64_t i0 = grp * 4;
        float4 h[KK];
#pragma unroll
        for (int j = 0; j < KK; ++j) h[j] = load4_stream(a.rows[j], i0, a.d);
        float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < KK; ++j) {
            r.x = __fmaf_rn(al[j], h[j].x, r.x); r.y = __fmaf_rn(al[j], h[j].y, r.y);
            r.z = __fmaf_rn(al[j], h[j].z, r.z); r.w = __fmaf_rn(al[j], h[j].w, r.w);
        }
        store4(a.ref, i0, a.d, r);
        if (a.ref2) {
            float4 r2 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < KK; ++j) {
                r2.x = __fmaf_rn(a.inv_k, fabsf(h[j].x), r2.x); r2.y = __fmaf_rn(a.inv_k, fabsf(h[j].y), r2.y);
                r2.z = __fmaf_rn(a.inv_k, fabsf(h[j].z), r2.z); r2.w = __fmaf_rn(a.inv_k, fabsf(h[j].w), r2.w);
            }
            store4(a.ref2, i0, a.d, r2);
        }
    }
}

template <int KK>
cudaError_t combine_k(const CombineArgs& a, int grid, cudaStream_t st) {
    combine_kernel<KK><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_dots(const float* const* rows, int k, uint64_t d, const float* grads, uint32_t M, uint64_t ld,
                        uint32_t divisor, double* partials, FuseBlock* fb, int sm_count, cudaStream_t st, int* launches) {
    const uint64_t ngroups = (d + 3) / 4;
    uint64_t want = (ngroups + kDotsThreads - 1) / kDotsThreads;
    if (want < 1) want = 1;
    // one partial row per CTA: never more CTAs than the partials buffer has rows
    const uint64_t max_ctas = (uint64_t)(sm_count < kDotsMaxCtas ? sm_count : kDotsMaxCtas);
    const int grid = (int)(want < max_ctas ? want : max_ctas);
    DotsArgs a;
    a.grads = grads; a.partials = partials; a.fb = fb; a.d = d; a.ld = ld; a.M = M;
    a.divisor = divisor ? divisor : M;
    cudaError_t e = cudaSuccess;
    // long vectors, at most 8 history rows: the staged kernel
    if (k <= 8 && d >= kDotsPipeMinCoords) {
        DotsPipeArgs pa;
        for (int j = 0; j < 8; ++j) a.rows_a[j] = a.rows_b[j] = rows[j < k ? j : 0];
        int p = 0;
        for (int i = 0; i < k; ++i)
            for (int j = i; j < k; ++j) a.dst[p++] = (short)(i * kGramStride + j);
        for (int i = 0; i < k; ++i) a.dst[p++] = (short)(kGramRhs + i);
        a.dst[p++] = (short)kGramGG;
        pa.base = a;
        pa.rows.nrows = 0;
        for (int j = 0; j < k; ++j) pa.rows.row[pa.rows.nrows++] = rows[j];
        pa.rows.n_pre = k;
        if (grads)
            for (uint32_t m = 0; m < M; ++m) pa.rows.row[pa.rows.nrows++] = grads + (uint64_t)m * ld;
        const uint64_t nchunks = d / DotsGeom::kChunk;
        const int pgrid = (int)(nchunks < max_ctas ? nchunks : max_ctas);
        e = dots_pipe_n(k, pa, pgrid, st);
        ++*launches;
        return e;
    }
    // chunks of at most 8 history vectors: diagonal blocks (with rhs) and, for k > 8, the cross block
    for (int lo = 0; lo < k && e == cudaSuccess; lo += 8) {
        const int n = (k - lo < 8) ? k - lo : 8;
        for (int j = 0; j < 8; ++j) a.rows_a[j] = a.rows_b[j] = rows[lo + (j < n ? j : 0)];
        int p = 0;
        for (int i = 0; i < n; ++i)
            for (int j = i; j < n; ++j) a.dst[p++] = (short)((lo + i) * kGramStride + lo + j);
        for (int i = 0; i < n; ++i) a.dst[p++] = (short)(kGramRhs + lo + i);
        a.dst[p++] = (short)kGramGG;
        e = dots_same_n(n, a, grid, st);
        ++*launches;
    }
    if (k > 8 && e == cudaSuccess) {
        const int nb = k - 8;
        for (int j = 0; j < 8; ++j) {
            a.rows_a[j] = rows[j];
            a.rows_b[j] = rows[8 + (j < nb ? j : 0)];
        }
        for (int i = 0; i < 8; ++i)
            for (int j = 0; j < nb; ++j) a.dst[i * nb + j] = (short)(i * kGramStride + 8 + j);
        e = dots_cross_n(nb, a, grid, st);
        ++*launches;
    }
    return e;
}

cudaError_t launch_solve(FuseBlock* fb, int k, int mode, double ridge, double rhs_div, cudaStream_t st, int* launches) {
    solve_kernel<<<1, 32, 0, st>>>(fb, k, mode, ridge, mode == TNG_FUSE_LSQ ? 1 : 0, rhs_div);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_combine(const float* const* rows, int k, uint64_t d, const FuseBlock* fb, float* ref, float* ref2,
                           int sm_count, cudaStream_t st, int* launches) {
    CombineArgs a;
    a.ref2 = ref2; a.inv_k = 1.0f / (float)k;
    for (int j = 0; j < kMaxK; ++j) a.rows[j] = rows[j < k ? j : 0];
    a.alpha = fb->alpha32; a.ref = ref; a.d = d;
    const uint64_t ngroups = (d + 3) / 4;
    uint64_t want = (ngroups + 255) / 256;
    const uint64_t cap = (uint64_t)sm_count * 8;
    const int grid = (int)(want < cap ? (want ? want : 1) : cap);
    cudaError_t e;
    switch (k) {
        case 1: e = combine_k<1>(a, grid, st); break;
        case 2: e = combine_k<2>(a, grid, st); break;
        case 3: e = combine_k<3>(a, grid, st); break;
        case 4: e = combine_k<4>(a, grid, st); break;
        case 5: e = combine_k<5>(a, grid, st); break;
        case 6: e = combine_k<6>(a, grid, st); break;
        case 7: e = combine_k<7>(a, grid, st); break;
        case 8: e = combine_k<8>(a, grid, st); break;
        case 9: e = combine_k<9>(a, grid, st); break;
        case 10: e = combine_k<10>(a, grid, st); break;
        case 11: e = combine_k<11>(a, grid, st); break;
        case 12: e = combine_k<12>(a, grid, st); break;
        case 13: e = combine_k<13>(a, grid, st); break;
        case 14: e = combine_k<14>(a, grid, st); break;
        case 15: e = combine_k<15>(a, grid, st); break;
        default: e = combine_k<16>(a, grid, st); break;
    }
    ++*launches;
    return e;
}

}  // namespace tng
