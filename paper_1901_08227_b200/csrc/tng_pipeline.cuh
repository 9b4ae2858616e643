// Bulk-copy staging for the streaming kernels (sm_100a).
//
// The TNG kernels stream many long rows (history vectors, gradient rows) exactly
// once.  Instead of every thread keeping its own loads in flight, one elected
// thread of a CTA asks the copy engine (TMA, untiled `cp.async.bulk`) to bring the
// same chunk of coordinates of every row into a shared-memory stage; the compute
// warps read the stage with plain shared loads.  Several stages in flight per SM
// keep HBM busy without costing registers, and the compute warps never wait on
// global memory themselves.
//
// Hand-shake per stage: `full` (copy engine -> consumers, transaction-count
// mbarrier) and `empty` (consumers -> producer, one arrival per consumer warp).
// Every wait is bounded: after kSpinLimit failed polls the waiter gives up, the
// caller records an error code in global memory and stops using the pipeline, and
// the host reports TNG_ERR_CUDA.  Nothing ever spins forever.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace tng {

constexpr int kChunk = 1024;                 // coordinates per row per stage (4 KiB)
constexpr int kStageRows = 16;               // rows per stage (64 KiB)
constexpr int kStages = 3;                   // stages per CTA (192 KiB)
constexpr uint32_t kRowBytes = kChunk * 4u;
constexpr uint32_t kStageBytes = kStageRows * kRowBytes;
constexpr uint32_t kPipeSmemBytes = kStages * kStageBytes + 1024;   // + barriers, alignment slack
constexpr int kSpinLimit = 1 << 22;          // polls of try_wait (each may itself block briefly)

enum PipeError : uint32_t { kPipeOk = 0, kPipeFullTimeout = 1, kPipeEmptyTimeout = 2 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// makes the initialised barriers visible to the copy engine
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait; false = gave up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// One row chunk: global -> this CTA's shared memory, completion counted on `bar`.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// Shared-memory footprint of one pipeline: stage data (1 KiB aligned) then the barriers.
struct PipeSmem {
    uint32_t data;                 // shared address of stage 0
    uint32_t full[kStages];
    uint32_t empty[kStages];
};

// Carve the dynamic shared memory and initialise the barriers (thread 0), then sync.
// `consumer_arrivals` = arrivals that free a stage (one per consumer warp).
__device__ __forceinline__ PipeSmem pipe_setup(unsigned char* dyn_smem, uint32_t consumer_arrivals) {
    PipeSmem p;
    const uint32_t base = (smem_u32(dyn_smem) + 127u) & ~127u;
    p.data = base;
    const uint32_t bars = base + kStages * kStageBytes;
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
        p.full[s] = bars + 16u * s;
        p.empty[s] = bars + 16u * s + 8u;
    }
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
            mbar_init(p.full[s], 1);
            mbar_init(p.empty[s], consumer_arrivals);
        }
        mbar_init_fence();
    }
    __syncthreads();
    return p;
}

// Row source list of one launch: pointer of each virtual row (all 16-byte aligned).
// A "fill" is up to kStageRows consecutive rows of the list for one chunk of coordinates.
struct PipeRows {
    const float* row[80];          // up to 16 history rows + 64 gradient rows
    int nrows;
};

// Producer side, run by ONE thread: for chunk indices c = first, first + stride, ... < nchunks
// and for each fill of the row list, wait for a free stage and issue the row copies.
// Returns kPipeOk or the error that stopped it.
__device__ __forceinline__ uint32_t pipe_produce(const PipeSmem& p, const PipeRows& rows, uint64_t first, uint64_t stride,
                                                 uint64_t nchunks) {
    uint32_t it = 0;
    for (uint64_t c = first; c < nchunks; c += stride) {
        for (int r0 = 0; r0 < rows.nrows; r0 += kStageRows) {
            const int n = (rows.nrows - r0 < kStageRows) ? rows.nrows - r0 : kStageRows;
            const uint32_t s = it % kStages, use = it / kStages;
            // a stage is free once its previous use has been consumed (parity of use - 1)
            if (use > 0 && !mbar_wait(p.empty[s], (use - 1) & 1u)) return kPipeEmptyTimeout;
            mbar_expect_tx(p.full[s], (uint32_t)n * kRowBytes);
            const uint32_t dst = p.data + s * kStageBytes;
            for (int r = 0; r < n; ++r) bulk_load(dst + (uint32_t)r * kRowBytes, rows.row[r0 + r] + c * kChunk, kRowBytes, p.full[s]);
            ++it;
        }
    }
    return kPipeOk;
}

}  // namespace tng
