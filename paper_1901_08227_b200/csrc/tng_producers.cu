// Local-gradient producers of the synthetic workloads (Section 4 of the paper):
// l2-regularised logistic regression (GEMV for the margins, transposed GEMV for
// the gradient) and the extended, uncoupled Rosenbrock function (elementwise).
// These feed tng_step; they are not part of the timed round.
#include <math.h>

#include "tng_device.cuh"
#include "tng_internal.h"

namespace tng {
namespace {

constexpr int kMaxRowChunks = 64;

// ---- logistic: margins --------------------------------------------------------
// One CTA per sample (grid-stride over samples): the 8 warps split the row, so the many small
// CTAs balance over the SMs whatever n is.  z_i = a_i . w; coef_i = -b_i sigma(-b_i z_i);
// lossrow_i = log(1+exp(-b_i z_i)).
template <bool VEC>
__global__ void __launch_bounds__(256) logistic_margin_kernel(const float* __restrict__ X, const float* __restrict__ b,
                                                              const float* __restrict__ w, uint64_t n, uint64_t d,
                                                              double* __restrict__ coef, float* __restrict__ lossrow) {
    // The pass is bound by reading the features, so the sums can afford double precision: margins,
    // sigmoid and the coefficients the transposed product uses are then good to fp32's last place.
    __shared__ double part[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint64_t i = blockIdx.x; i < n; i += gridDim.x) {
        const float* row = X + i * d;
        double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
        if (VEC) {
            const float4* r4 = reinterpret_cast<const float4*>(row);
            const float4* w4 = reinterpret_cast<const float4*>(w);
#pragma unroll 4
            for (uint64_t j = threadIdx.x; j < d / 4; j += 256) {
                const float4 x = __ldcs(r4 + j);
                const float4 ww = __ldg(w4 + j);
                acc0 = fma((double)x.x, (double)ww.x, acc0); acc1 = fma((double)x.y, (double)ww.y, acc1);
                acc2 = fma((double)x.z, (double)ww.z, acc2); acc3 = fma((double)x.w, (double)ww.w, acc3);
            }
        } else {
            for (uint64_t j = threadIdx.x; j < d; j += 256) acc0 = fma((double)__ldcs(row + j), (double)__ldg(w + j), acc0);
        }
        double z = (acc0 + acc1) + (acc2 + acc3);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(kFullMask, z, off);
        if (lane == 0) part[warp] = z;
        __syncthreads();
        if (threadIdx.x == 0) {
            z = ((part[0] + part[1]) + (part[2] + part[3])) + ((part[4] + part[5]) + (part[6] + part[7]));
            const double bi = (double)b[i];
            const double t = -bi * z;                      // sigma(t), softplus(t), overflow-safe
            double sig, sp;
            if (t >= 0.0) {
                const double e = exp(-t);
                sig = 1.0 / (1.0 + e);
                sp = t + log1p(e);
            } else {
                const double e = exp(t);
                sig = e / (1.0 + e);
                sp = log1p(e);
            }
            coef[i] = -bi * sig;
            lossrow[i] = (float)sp;
        }
        __syncthreads();
    }
}

// ---- logistic: transposed GEMV, rows split into chunks -----------------------------
template <bool VEC>
__global__ void __launch_bounds__(256) logistic_colsum_kernel(const float* __restrict__ X, const double* __restrict__ coef,
                                                              uint64_t n, uint64_t d, uint64_t rows_per_chunk,
                                                              double* __restrict__ partial) {
    const uint64_t col = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) * (VEC ? 4 : 1);
    if (col >= d) return;
    const uint64_t r0 = (uint64_t)blockIdx.y * rows_per_chunk;
    const uint64_t r1 = (r0 + rows_per_chunk < n) ? r0 + rows_per_chunk : n;
    if (VEC) {
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 8
        for (uint64_t i = r0; i < r1; ++i) {
            const double ci = __ldg(coef + i);
            const float4 x = __ldcs(reinterpret_cast<const float4*>(X + i * d + col));
            a0 = fma(ci, (double)x.x, a0); a1 = fma(ci, (double)x.y, a1);
            a2 = fma(ci, (double)x.z, a2); a3 = fma(ci, (double)x.w, a3);
        }
        double* dst = partial + (uint64_t)blockIdx.y * d + col;
        dst[0] = a0; dst[1] = a1; dst[2] = a2; dst[3] = a3;
    } else {
        double acc = 0.0;
        for (uint64_t i = r0; i < r1; ++i) acc = fma(__ldg(coef + i), (double)__ldcs(X + i * d + col), acc);
        partial[(uint64_t)blockIdx.y * d + col] = acc;
    }
}

__global__ void __launch_bounds__(256) logistic_finish_kernel(const double* __restrict__ partial, int chunks, uint64_t n,
                                                              uint64_t d, const float* __restrict__ w, float lambda2,
                                                              float* __restrict__ grad) {
    const uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    double acc = 0.0;
    for (int c = 0; c < chunks; ++c) acc += partial[(uint64_t)c * d + j];
    grad[j] = (float)(acc / (double)n + (double)lambda2 * (double)w[j]);
}

// single CTA: loss = mean(lossrow) + lambda2/2 ||w||^2, accumulated in double
__global__ void __launch_bounds__(1024) logistic_loss_kernel(const float* __restrict__ lossrow, uint64_t n,
                                                             const float* __restrict__ w, uint64_t d, float lambda2,
                                                             double* __restrict__ loss) {
    __shared__ double sh[2][32];
    double a = 0.0, r = 0.0;
    for (uint64_t i = threadIdx.x; i < n; i += blockDim.x) a += (double)lossrow[i];
    for (uint64_t j = threadIdx.x; j < d; j += blockDim.x) r += (double)w[j] * (double)w[j];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        a += __shfl_xor_sync(kFullMask, a, off);
        r += __shfl_xor_sync(kFullMask, r, off);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sh[0][warp] = a; sh[1][warp] = r; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double sa = 0.0, sr = 0.0;
        for (int q = 0; q < (int)(blockDim.x >> 5); ++q) { sa += sh[0][q]; sr += sh[1][q]; }
        *loss = sa / (double)n + 0.5 * (double)lambda2 * sr;
    }
}

// ---- Rosenbrock ----------------------------------------------------------------------
// per pair (a,b) = (x_{2i}, x_{2i+1}), one rounding per line:
//   q = a*a; t = b - q; d/da = -(400 a) t - 2 (1 - a); d/db = 200 t
__global__ void __launch_bounds__(256) rosenbrock_grad_kernel(const float* __restrict__ x, uint64_t npairs,
                                                              const float* __restrict__ noise, uint32_t M, uint64_t ld,
                                                              float* __restrict__ grads) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t p = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; p < npairs; p += stride) {
        const float2 ab = *reinterpret_cast<const float2*>(x + 2 * p);
        const float q = __fmul_rn(ab.x, ab.x);
        const float t = __fsub_rn(ab.y, q);
        const float u2 = __fmul_rn(__fmul_rn(400.0f, ab.x), t);
        const float u4 = __fmul_rn(2.0f, __fsub_rn(1.0f, ab.x));
        const float ga = __fsub_rn(-u2, u4);
        const float gb = __fmul_rn(200.0f, t);
        for (uint32_t m = 0; m < M; ++m) {
            float2 nz = make_float2(0.f, 0.f);
            if (noise) nz = __ldcs(reinterpret_cast<const float2*>(noise + (uint64_t)m * ld + 2 * p));
            __stcs(reinterpret_cast<float2*>(grads + (uint64_t)m * ld + 2 * p),
                   make_float2(__fadd_rn(ga, nz.x), __fadd_rn(gb, nz.y)));
        }
    }
}

__global__ void __launch_bounds__(1024) rosenbrock_value_kernel(const float* __restrict__ x, uint64_t npairs,
                                                                double* __restrict__ value) {
    __shared__ double sh[32];
    double acc = 0.0;
    for (uint64_t p = threadIdx.x; p < npairs; p += blockDim.x) {
        const double a = (double)x[2 * p], b = (double)x[2 * p + 1];
        const double t = b - a * a;
        acc += 100.0 * t * t + (1.0 - a) * (1.0 - a);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(kFullMask, acc, off);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int q = 0; q < (int)(blockDim.x >> 5); ++q) s += sh[q];
        *value = s;
    }
}

__global__ void __launch_bounds__(256) sgd_update_kernel(float* __restrict__ w, const float* __restrict__ v, uint64_t d,
                                                         float eta) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += stride)
        w[i] = __fsub_rn(w[i], __fmul_rn(eta, v[i]));
}

// Row chunks of the transposed product: enough CTAs to fill the GPU (4 per SM), and, when a
// count up to the limit exists, a total that is a multiple of the SM count so that no SM gets
// one CTA more than another.
// SM count of the current device (asked once per device index).
int sm_count_now() {
    static PerDevice<int> cached;
    const int slot = device_slot();
    if (slot >= 0 && cached.v[slot] > 0) return cached.v[slot];
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        (void)cudaGetLastError();
        sms = 1;
    }
    if (slot >= 0) cached.v[slot] = sms;
    return sms;
}

int row_chunks(uint64_t n, uint64_t d, bool vec) {
    const uint64_t colblocks = ((vec ? d / 4 : d) + 255) / 256;
    const uint64_t sms = (uint64_t)sm_count_now();
    uint64_t chunks = (4 * sms + colblocks - 1) / colblocks;
    for (uint64_t c = chunks; c <= (uint64_t)kMaxRowChunks; ++c)
        if ((colblocks * c) % sms == 0) { chunks = c; break; }
    if (chunks > (uint64_t)kMaxRowChunks) chunks = kMaxRowChunks;
    if (chunks > n) chunks = n;
    if (chunks < 1) chunks = 1;
    return (int)chunks;
}

bool vec_ok(const float* X, const float* w, uint64_t d) {
    return d % 4 == 0 && (reinterpret_cast<uintptr_t>(X) & 15u) == 0 && (reinterpret_cast<uintptr_t>(w) & 15u) == 0;
}

cudaError_t launch_margins(const float* X, const float* b, const float* w, uint64_t n, uint64_t d, double* coef,
                           float* lossrow, cudaStream_t st) {
    const uint64_t cap = (uint64_t)sm_count_now() * 64u;
    const int grid = (int)(n < cap ? n : cap);
    if (vec_ok(X, w, d)) logistic_margin_kernel<true><<<grid, 256, 0, st>>>(X, b, w, n, d, coef, lossrow);
    else logistic_margin_kernel<false><<<grid, 256, 0, st>>>(X, b, w, n, d, coef, lossrow);
    return cudaGetLastError();
}

}  // namespace
}  // namespace tng

using namespace tng;

extern "C" {

// scratch layout (in floats): coef as n4 doubles, lossrow as n4 floats, partial as kMaxRowChunks x d doubles
size_t tng_logistic_scratch_floats(uint64_t n, uint64_t d) {
    const uint64_t n4 = (n + 3) / 4 * 4;
    return (size_t)(3 * n4 + 2 * (uint64_t)kMaxRowChunks * d);
}

tng_status tng_logistic_grad(const float* X_dev, const float* b_dev, uint64_t n, uint64_t d, const float* w_dev,
                             float lambda2, float* grad_dev, float* scratch_dev, void* stream) {
    if (!X_dev || !b_dev || !w_dev || !grad_dev || !scratch_dev || n < 1 || d < 1) return TNG_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(scratch_dev) & 15u) != 0) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t n4 = (n + 3) / 4 * 4;
    double* coef = reinterpret_cast<double*>(scratch_dev);
    float* lossrow = scratch_dev + 2 * n4;
    double* partial = reinterpret_cast<double*>(scratch_dev + 3 * n4);   // n4 is a multiple of 4: 16-byte aligned
    if (launch_margins(X_dev, b_dev, w_dev, n, d, coef, lossrow, st) != cudaSuccess) return TNG_ERR_CUDA;
    const bool vec = vec_ok(X_dev, w_dev, d);
    const int chunks = row_chunks(n, d, vec);
    const uint64_t rows_per_chunk = (n + chunks - 1) / chunks;
    dim3 grid((unsigned)(((vec ? d / 4 : d) + 255) / 256), (unsigned)chunks);
    if (vec) logistic_colsum_kernel<true><<<grid, 256, 0, st>>>(X_dev, coef, n, d, rows_per_chunk, partial);
    else logistic_colsum_kernel<false><<<grid, 256, 0, st>>>(X_dev, coef, n, d, rows_per_chunk, partial);
    if (cudaGetLastError() != cudaSuccess) return TNG_ERR_CUDA;
    logistic_finish_kernel<<<(unsigned)((d + 255) / 256), 256, 0, st>>>(partial, chunks, n, d, w_dev, lambda2, grad_dev);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}

tng_status tng_logistic_loss(const float* X_dev, const float* b_dev, uint64_t n, uint64_t d, const float* w_dev,
                             float lambda2, double* loss_dev, float* scratch_dev, void* stream) {
    if (!X_dev || !b_dev || !w_dev || !loss_dev || !scratch_dev || n < 1 || d < 1) return TNG_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(scratch_dev) & 15u) != 0) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t n4 = (n + 3) / 4 * 4;
    double* coef = reinterpret_cast<double*>(scratch_dev);
    float* lossrow = scratch_dev + 2 * n4;
    if (launch_margins(X_dev, b_dev, w_dev, n, d, coef, lossrow, st) != cudaSuccess) return TNG_ERR_CUDA;
    logistic_loss_kernel<<<1, 1024, 0, st>>>(lossrow, n, w_dev, d, lambda2, loss_dev);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}

tng_status tng_rosenbrock_grad(const float* x_dev, uint64_t d, const float* noise_dev, uint32_t M, uint64_t ld,
                               float* grads_dev, void* stream) {
    if (!x_dev || !grads_dev || d < 2 || (d % 2) != 0 || (ld % 2) != 0 || ld < d || M < 1) return TNG_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x_dev) & 7u) || (reinterpret_cast<uintptr_t>(grads_dev) & 7u) ||
        (noise_dev && (reinterpret_cast<uintptr_t>(noise_dev) & 7u)))
        return TNG_ERR_INVALID_ARG;
    const uint64_t npairs = d / 2;
    const uint64_t want = (npairs + 255) / 256;
    const uint64_t cap = (uint64_t)sm_count_now() * 16u;
    const int grid = (int)(want < cap ? want : cap);
    rosenbrock_grad_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(x_dev, npairs, noise_dev, M, ld, grads_dev);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}

tng_status tng_rosenbrock_value(const float* x_dev, uint64_t d, double* value_dev, void* stream) {
    if (!x_dev || !value_dev || d < 2 || (d % 2) != 0) return TNG_ERR_INVALID_ARG;
    rosenbrock_value_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(x_dev, d / 2, value_dev);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}

tng_status tng_sgd_update(float* w_dev, const float* v_dev, uint64_t d, float eta, void* stream) {
    if (!w_dev || !v_dev || d < 1) return TNG_ERR_INVALID_ARG;
    const uint64_t want = (d + 255) / 256;
    const uint64_t cap = (uint64_t)sm_count_now() * 16u;
    const int grid = (int)(want < cap ? want : cap);
    sgd_update_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(w_dev, v_dev, d, eta);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}

}  // extern "C"
