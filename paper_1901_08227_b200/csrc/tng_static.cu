// tng_gram_static: the fusion statistics (Gram matrix, right-hand side, mean squared
// gradient norm) for callers that cannot allocate device memory.
//
// The statistics kernel needs scratch beyond its inputs and outputs: one row of
// partial sums per CTA and an arrival counter.  A tng_ctx keeps that scratch in its
// workspace, which somebody has to allocate.  Some callers cannot: a process that gave
// all device memory to its own pool at start-up, a service whose steady-state loop must
// not touch the allocator (cudaMalloc synchronises the device and can fail late), or a
// plug-in that is simply handed pointers.  For them the scratch lives in the fixed
// array below, which is part of the loaded library image: every GPU that loads libtng
// holds these kTngStaticScratchBytes until the process exits, whether or not the entry
// point is ever called.
#include "tng_device.cuh"
#include "tng_internal.h"

namespace {

using tng::FuseBlock;

constexpr size_t kPartialBytes = sizeof(double) * tng::kDotsMaxCtas * tng::kDotsMaxAcc;
constexpr size_t kBlockOffset = (kPartialBytes + 255) / 256 * 256;
constexpr size_t kTngStaticScratchBytes = kBlockOffset + (sizeof(FuseBlock) + 255) / 256 * 256;
static_assert(kTngStaticScratchBytes <= TNG_STATIC_SCRATCH_BYTES, "header states a smaller scratch than the array needs");

// Host code must never use this name as a pointer: on the host it is only a stand-in
// for the symbol.  The device address comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_static_scratch[TNG_STATIC_SCRATCH_BYTES];

using tng::kMaxDevices;
void* g_scratch_addr[kMaxDevices] = {nullptr};   // per device, filled on first use
int g_sm_count[kMaxDevices] = {0};

// Packs the statistics from the scratch block into the caller's buffer:
// out[0 .. k*k) = G row-major (both triangles), out[k*k .. k*k+k) = rhs, out[k*k+k] = grad_sq.
// If a bounded wait of the staged statistics kernel gave up, the sums are incomplete: every
// output becomes NaN, which is how this entry point (it never synchronises with the host)
// reports that.
__global__ void pack_static_gram_kernel(int k, double* __restrict__ out) {
    const FuseBlock* fb = reinterpret_cast<const FuseBlock*>(g_static_scratch + kBlockOffset);   // device code may name the array
    const int n = k * k + k + 1;
    const bool gave_up = fb->pipe_error != 0u;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        double v;
        if (gave_up) {
            v = nan("");
        } else if (i < k * k) {
            const int a = i / k, b = i % k;
            v = (a <= b) ? fb->gram[a * tng::kGramStride + b] : fb->gram[b * tng::kGramStride + a];
        } else if (i < k * k + k) {
            v = fb->gram[tng::kGramRhs + (i - k * k)];
        } else {
            v = fb->gram[tng::kGramGG];
        }
        out[i] = v;
    }
}

}  // namespace

extern "C" tng_status tng_gram_static(const float* const* rows_dev, uint32_t k, uint64_t d, const float* grads_dev,
                                      uint32_t M, uint64_t ld, double* out_dev, void* stream) {
    if (!rows_dev || !grads_dev || !out_dev || d < 1) return TNG_ERR_INVALID_ARG;
    if (k < 1 || k > TNG_STATIC_MAX_HISTORY || M < 1 || M > TNG_MAX_WORKERS) return TNG_ERR_UNSUPPORTED;   // beyond the fixed scratch
    if (ld < d || (ld % 4) != 0 || (reinterpret_cast<uintptr_t>(grads_dev) & 15u) || (reinterpret_cast<uintptr_t>(out_dev) & 7u))
        return TNG_ERR_INVALID_ARG;
    for (uint32_t j = 0; j < k; ++j)
        if (!rows_dev[j] || (reinterpret_cast<uintptr_t>(rows_dev[j]) & 15u)) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TNG_ERR_CUDA;
    if (!g_scratch_addr[dev]) {
        // set-up, once per device, with that device current
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return TNG_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return TNG_ERR_CUDA;
        g_sm_count[dev] = sms;
        g_scratch_addr[dev] = p;
    }
    unsigned char* base = static_cast<unsigned char*>(g_scratch_addr[dev]);
    double* partials = reinterpret_cast<double*>(base);
    FuseBlock* fb = reinterpret_cast<FuseBlock*>(base + kBlockOffset);
    // the array keeps whatever the last call left: the arrival counter must start at zero
    if (cudaMemsetAsync(fb, 0, sizeof(FuseBlock), st) != cudaSuccess) return TNG_ERR_CUDA;
    int launches = 0;
    if (tng::launch_dots(rows_dev, (int)k, d, grads_dev, M, ld, 0, partials, fb, g_sm_count[dev], st, &launches) != cudaSuccess)
        return TNG_ERR_CUDA;
    pack_static_gram_kernel<<<1, 128, 0, st>>>((int)k, out_dev);
    return cudaGetLastError() == cudaSuccess ? TNG_OK : TNG_ERR_CUDA;
}
