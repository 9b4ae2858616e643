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

// Geometry of one pipeline: CHUNK coordinates of ROWS rows per stage, STAGES stages.
template <int CHUNK, int ROWS, int STAGES>
struct PipeGeom {
    static constexpr int kChunk = CHUNK;
    static constexpr int kRows = ROWS;
    static constexpr int kStages = STAGES;
    static constexpr uint32_t kRowBytes = CHUNK * 4u;
    static constexpr uint32_t kStageBytes = ROWS * kRowBytes;
    static constexpr uint32_t kSmemBytes = STAGES * kStageBytes + 1024;   // + barriers, alignment slack
};
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
// One poll; the hardware may park the thread for up to kConsumerNapNs while the phase is
// incomplete, so a waiting warp costs its scheduler almost no issue slots.
constexpr uint32_t kConsumerNapNs = 50;
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kConsumerNapNs)
        : "memory");
    return ok != 0;
}
// bounded wait; false = gave up
__device__ __forceinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) { return mbar_wait_limited(bar, parity, kSpinLimit); }
// Same for the producer thread, which has nothing else to do: each poll may sleep up to
// `kProducerNapNs` inside the hardware wait, so that its polling does not take issue slots
// from the compute warps of its scheduler.  Still bounded.
constexpr uint32_t kProducerNapNs = 200;
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < kSpinLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kProducerNapNs)
            : "memory");
        if (ok) return true;
    }
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

// Shared-memory footprint of one pipeline: stage data (128-byte aligned) then the barriers.
struct PipeSmem {
    uint32_t data;                 // shared address of stage 0
    uint32_t bars;                 // full[s] at bars + 16 s, empty[s] at bars + 16 s + 8
    __device__ __forceinline__ uint32_t full(uint32_t s) const { return bars + 16u * s; }
    __device__ __forceinline__ uint32_t empty(uint32_t s) const { return bars + 16u * s + 8u; }
};

// Carve the dynamic shared memory and initialise the barriers (thread 0), then sync.
// `consumer_arrivals` = arrivals that free a stage (one per consumer warp).
template <class G>
__device__ __forceinline__ PipeSmem pipe_setup(unsigned char* dyn_smem, uint32_t consumer_arrivals) {
    PipeSmem p;
    p.data = (smem_u32(dyn_smem) + 127u) & ~127u;
    p.bars = p.data + G::kStages * G::kStageBytes;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < G::kStages; ++s) {
            mbar_init(p.full(s), 1);
            mbar_init(p.empty(s), consumer_arrivals);
        }
        mbar_init_fence();
    }
    __syncthreads();
    return p;
}

// Row source list of one launch: pointer of each row (all 16-byte aligned): first n_pre
// rows of one kind (history / reference), then the gradient rows.  A "fill" is up to ROWS
// consecutive rows of ONE kind for one chunk of coordinates: fills never mix the two kinds,
// so a chunk takes ceil(n_pre / ROWS) + ceil((nrows - n_pre) / ROWS) fills, in that order.
struct PipeRows {
    const float* row[80];          // up to 16 history rows + 64 gradient rows
    int nrows;
    int n_pre;
};

// Producer side, run by ONE thread: for chunk indices c = first, first + stride, ... < nchunks
// and for each fill of the row list, wait for a free stage and issue the row copies.
// Returns kPipeOk or the error that stopped it.
template <class G>
__device__ __forceinline__ uint32_t pipe_produce(const PipeSmem& p, const PipeRows& rows, uint64_t first, uint64_t stride,
                                                 uint64_t nchunks) {
    uint32_t it = 0;
    for (uint64_t c = first; c < nchunks; c += stride) {
        int r0 = 0;
        while (r0 < rows.nrows) {
            const int seg_end = (r0 < rows.n_pre) ? rows.n_pre : rows.nrows;
            const int n = (seg_end - r0 < G::kRows) ? seg_end - r0 : G::kRows;
            const uint32_t s = it % G::kStages, use = it / G::kStages;
            // a stage is free once its previous use has been consumed (parity of use - 1)
            if (use > 0 && !mbar_wait_relaxed(p.empty(s), (use - 1) & 1u)) return kPipeEmptyTimeout;
            mbar_expect_tx(p.full(s), (uint32_t)n * G::kRowBytes);
            const uint32_t dst = p.data + s * G::kStageBytes;
            for (int r = 0; r < n; ++r)
                bulk_load(dst + (uint32_t)r * G::kRowBytes, rows.row[r0 + r] + c * G::kChunk, G::kRowBytes, p.full(s));
            ++it;
            r0 += n;
        }
    }
    return kPipeOk;
}

}  // namespace tng
