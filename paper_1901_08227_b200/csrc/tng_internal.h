// Host-side declarations shared by the libtng translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "tng.h"

namespace tng {

constexpr int kMaxK = TNG_MAX_HISTORY;
constexpr int kGramStride = kMaxK;                      // G[a*16 + b]
constexpr int kGramRhs = kMaxK * kMaxK;                 // c[a] at 256 + a
constexpr int kGramGG = kGramRhs + kMaxK;               // gg at 272
constexpr int kGramDoubles = kGramGG + 1;
constexpr int kDotsMaxAcc = 64;                         // accumulators of one dots launch
constexpr int kDotsMaxCtas = 592;                       // 4 x 148

// Function attributes (the dynamic shared-memory opt-in) and occupancy belong to a device, not
// to the process: a value cached per kernel instantiation is kept per device index.  Devices
// beyond the table are simply not cached (slot() < 0: the caller sets / asks every time).
constexpr int kMaxDevices = 64;
inline int device_slot() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}
template <typename T>
struct PerDevice {
    T v[kMaxDevices] = {};
};

// Small device-resident block: fusion statistics, coefficients, flags.
struct FuseBlock {
    double gram[kGramDoubles + 7];   // padded to 280 doubles
    double alpha64[kMaxK];
    double cnz;
    float alpha32[kMaxK];
    uint32_t fallback;
    uint32_t dots_arrivals;          // CTAs that finished the current dots launch
    uint32_t pipe_error;             // nonzero: a bounded wait of a staged kernel gave up (PipeError)
    uint32_t pad_;
    unsigned long long nonfinite;    // NaN/Inf block scales seen so far
};

struct CodecGeom {
    uint64_t d;
    uint64_t ntile;      // ceil(d/128)
    uint64_t nblk;       // scales per worker
    uint64_t block;      // coordinates per scale (d for per-vector)
    uint64_t wpw;        // code words per worker
    uint32_t M;
    int codec, norm, scale_kind, levels;
    uint32_t seed_lo, seed_hi;
    float quot_eps;
    uint64_t tile0;      // index of the first tile within the whole vector (a context that holds a slice of it)
};

// ---- fusion (tng_fuse.cu) ---------------------------------------------------
// rows[j] = h_{j+1}.  Accumulates G (and with grads != nullptr the rhs and grad_sq)
// into fb->gram via per-CTA partials in `partials` (kDotsMaxCtas * kDotsMaxAcc doubles).
// divisor: what the gradient sums (rhs, grad_sq) are divided by; 0 = M (the mean over the rows
// given), 1 = raw sums (a caller that adds the sums of several GPUs divides later, in the solve).
cudaError_t launch_dots(const float* const* rows, int k, uint64_t d, const float* grads, uint32_t M,
                        uint64_t ld, uint32_t divisor, double* partials, FuseBlock* fb, int sm_count, cudaStream_t st,
                        int* launches);
// rhs_div: the solve first divides rhs and grad_sq by it (1 = they are means already).
cudaError_t launch_solve(FuseBlock* fb, int k, int mode, double ridge, double rhs_div, cudaStream_t st,
                         int* launches);
// ref2 (may be nullptr): also write r' = (1/k) sum_j |h_j| (second reference of the combined form)
cudaError_t launch_combine(const float* const* rows, int k, uint64_t d, const FuseBlock* fb, float* ref, float* ref2,
                           int sm_count, cudaStream_t st, int* launches);

// ---- codec (tng_codec.cu) -----------------------------------------------------
// tile_stat: M*ntile floats (needed when encode_needs_tile_stat), tree_tmp: scratch of
// tree_tmp_floats(geom) floats; used when geom.block != 128 and by the scalar reference.
size_t tree_tmp_floats(const CodecGeom& g);
bool encode_needs_tile_stat(const CodecGeom& g);
// Optional: let the encode pass build the reference itself, r = sum_j alpha[j] rows[j] (the
// combine step's fp32 fma chain), writing it to ref_out; saves one pass over the ring and
// hides the encode arithmetic behind the ring's memory traffic.  Only for block == 128 with
// a normalisation (encode_can_fuse_reference).
struct RefFusion {
    const float* rows[kMaxK];
    int k;
    const float* alpha;   // device, k floats
    float* ref_out;       // device, d floats
    float* ref2_out;      // device, d floats: second reference (combined form), else nullptr
};
bool encode_can_fuse_reference(const CodecGeom& g);
// The g.M rows at `grads` are workers m_base .. m_base + g.M - 1 (their Philox streams); codes and
// scales (and means, the scalar references written in TNG_NORM_MEAN) point at the wire slot of worker m_base.
cudaError_t launch_encode(const CodecGeom& g, uint32_t m_base, const float* grads, uint64_t ld, const float* ref, const float* ref2,
                          const RefFusion* fusion, uint32_t step, uint32_t* codes, float* scales, float* means, float* tile_stat,
                          float* tree_tmp, FuseBlock* fb, int sm_count, cudaStream_t st, int* launches);
// means: the M scalar references (read in TNG_NORM_MEAN only)
cudaError_t launch_decode(const CodecGeom& g, const uint32_t* codes, const float* scales, const float* means, const float* ref,
                          const float* ref2, float* out_a, float* out_b, FuseBlock* fb, int sm_count, cudaStream_t st, int* launches);

}  // namespace tng
