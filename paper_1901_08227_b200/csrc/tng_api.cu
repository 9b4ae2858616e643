// libtng C ABI: context, workspace, the round of Algorithm 1 as a sequence of
// kernel launches on one stream (no host synchronisation inside a round).
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "tng_internal.h"
#include "tng_pipeline.cuh"

using namespace tng;

namespace {

constexpr size_t kAlign = 256;
constexpr int kTimedRounds = 64;   // event sets kept before they are harvested
constexpr int kStages = 5;         // dots, solve, combine, encode, decode

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

}  // namespace

struct tng_ctx {
    uint64_t d = 0;
    uint32_t M = 0, K = 0;
    int codec = 0, norm = 0;
    // options
    uint64_t block_opt = 128;
    int levels = 7, scale_kind = 0, fuse_mode = TNG_FUSE_AUTO, timing = 0, host_staging = 0;
    uint32_t ref_every = 1;
    uint64_t coord_offset = 0;
    uint32_t seed_lo = 0, seed_hi = 0;
    double ridge = 1e-6;
    float quot_eps = 0.0625f;
    // derived geometry
    bool sized = false;
    uint64_t d_pad = 0;
    CodecGeom geom{};
    // workspace
    void* ws = nullptr;
    size_t ws_bytes = 0;
    bool ws_owned = false, ws_ready = false;
    size_t off_ring = 0, off_ref = 0, off_codes = 0, off_scales = 0, off_tile_stat = 0, off_tree = 0,
           off_partials = 0, off_fb = 0, off_stage_g = 0, off_stage_o = 0, off_ref2 = 0, off_means = 0;
    // state
    uint32_t k = 0;
    int head = 0;
    uint64_t rounds = 0;
    const float* ref_cur = nullptr;   // reference of the last fusion (ref buffer or a ring slot)
    int last_mode = TNG_FUSE_LAST;
    bool last_had_stats = false;
    bool last_solved = false;         // the last fusion ran the solve kernel (alpha lives on the device)
    bool ref2_valid = false;          // combined form: the second-reference buffer has been written
    // rank-local rounds: tng_fuse_finish leaves the combine r = sum alpha_j h_j to the next tng_encode_local (which
    // reads the ring rows anyway); any other reader of the reference has it formed first (materialise_ref)
    bool ref_pending = false;
    RefFusion pending{};
    // bookkeeping
    int device = 0, sm_count = 148;
    cudaStream_t last_stream = nullptr;
    int last_cuda_error = 0;
    uint64_t launches = 0;
    unsigned long long nonfinite_reported = 0;
    // tng_step_host_async: the library's own stream for the copies back to the host
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_round_done = nullptr, ev_copied = nullptr;
    bool copy_pending = false;
    // timing
    cudaEvent_t ev[kTimedRounds][kStages + 1];
    bool ev_created = false;
    int ev_used = 0;
    uint64_t timed_rounds = 0;
    double ms_sum[kStages] = {0, 0, 0, 0, 0};
    bool ev_stage_ran[kTimedRounds][kStages];

    float* ring(int slot) const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_ring) + (size_t)slot * d_pad; }
    float* ref_buf() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_ref); }
    float* ref2_buf() const { return norm == TNG_NORM_COMB ? reinterpret_cast<float*>(static_cast<char*>(ws) + off_ref2) : nullptr; }
    uint32_t* codes() const { return reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + off_codes); }
    float* scales() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_scales); }
    float* means() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_means); }
    // no trajectory reference is involved: plain compression or the scalar reference of Section 3.1
    bool no_ref() const { return norm == TNG_NORM_NONE || norm == TNG_NORM_MEAN; }
    float* tile_stat() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_tile_stat); }
    float* tree() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_tree); }
    double* partials() const { return reinterpret_cast<double*>(static_cast<char*>(ws) + off_partials); }
    FuseBlock* fb() const { return reinterpret_cast<FuseBlock*>(static_cast<char*>(ws) + off_fb); }
    float* stage_g() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_stage_g); }
    float* stage_o() const { return reinterpret_cast<float*>(static_cast<char*>(ws) + off_stage_o); }
    int hist_slot(uint32_t j) const { return (int)(((int64_t)head - (int64_t)j) % (int64_t)K + (int64_t)K) % (int)K; }
    int effective_mode() const {
        if (fuse_mode != TNG_FUSE_AUTO) return fuse_mode;
        return K == 1 ? TNG_FUSE_LAST : TNG_FUSE_LSQ;
    }
};

namespace {

tng_status cuda_fail(tng_ctx* c, cudaError_t e) {
    if (c) c->last_cuda_error = (int)e;
    return TNG_ERR_CUDA;
}
#define TNG_CUDA(ctx, call)                                  \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) return cuda_fail((ctx), e__); \
    } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Freeze the options into the geometry and the workspace layout.
void size_ctx(tng_ctx* c) {
    if (c->sized) return;
    c->d_pad = (c->d + 31) / 32 * 32;
    CodecGeom& g = c->geom;
    g.d = c->d;
    g.ntile = (c->d + TNG_TILE - 1) / TNG_TILE;
    g.block = c->block_opt == 0 ? c->d : c->block_opt;
    g.nblk = c->block_opt == 0 ? 1 : (c->d + c->block_opt - 1) / c->block_opt;
    g.wpw = g.ntile * 4u * (uint64_t)c->codec;
    g.M = c->M; g.codec = c->codec; g.norm = c->norm; g.scale_kind = c->scale_kind; g.levels = c->levels;
    g.seed_lo = c->seed_lo; g.seed_hi = c->seed_hi; g.quot_eps = c->quot_eps;
    g.tile0 = c->coord_offset / TNG_TILE;
    size_t off = 0;
    c->off_ring = off;      off += align_up((size_t)c->K * c->d_pad * sizeof(float));
    c->off_ref = off;       off += align_up((size_t)c->d_pad * sizeof(float));
    c->off_ref2 = off;      off += align_up(c->norm == TNG_NORM_COMB ? (size_t)c->d_pad * sizeof(float) : 0);
    c->off_codes = off;     off += align_up((size_t)c->M * g.wpw * sizeof(uint32_t));
    c->off_scales = off;    off += align_up((size_t)c->M * g.nblk * sizeof(float));
    c->off_means = off;     off += align_up((size_t)TNG_MAX_WORKERS * sizeof(float));
    c->off_tile_stat = off; off += align_up(encode_needs_tile_stat(g) ? (size_t)c->M * g.ntile * sizeof(float) : 0);
    c->off_tree = off;      off += align_up(tree_tmp_floats(g) * sizeof(float));
    c->off_partials = off;  off += align_up((size_t)kDotsMaxCtas * kDotsMaxAcc * sizeof(double));
    c->off_fb = off;        off += align_up(sizeof(FuseBlock));
    c->off_stage_g = off;   off += align_up(c->host_staging ? (size_t)c->M * c->d_pad * sizeof(float) : 0);
    c->off_stage_o = off;   off += align_up(c->host_staging ? (size_t)c->d_pad * sizeof(float) : 0);
    c->ws_bytes = off;
    c->sized = true;
}

// First device use: pick the device, allocate if nothing was bound, clear the small state block.
tng_status ensure_ready(tng_ctx* c, cudaStream_t st) {
    c->last_stream = st;
    if (c->ws_ready) return TNG_OK;
    if (c->coord_offset != 0) {   // a slice of a longer vector: nothing may need the whole of it
        if (c->block_opt == 0 || c->norm == TNG_NORM_MEAN) return TNG_ERR_UNSUPPORTED;
        if (c->coord_offset % c->block_opt != 0) return TNG_ERR_INVALID_ARG;
    }
    size_ctx(c);
    TNG_CUDA(c, cudaGetDevice(&c->device));
    int sms = 0;
    TNG_CUDA(c, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device));
    if (sms > 0) c->sm_count = sms;
    if (!c->ws) {
        cudaError_t e = cudaMalloc(&c->ws, c->ws_bytes);
        if (e != cudaSuccess) {
            c->last_cuda_error = (int)e;
            c->ws = nullptr;
            (void)cudaGetLastError();
            return TNG_ERR_ALLOC;
        }
        c->ws_owned = true;
    }
    TNG_CUDA(c, cudaMemsetAsync(c->fb(), 0, sizeof(FuseBlock), st));
    c->ws_ready = true;
    return TNG_OK;
}

tng_status check_rows(const tng_ctx* c, const float* p, uint64_t ld) {
    if (!p || !aligned16(p) || ld < c->d || (ld % 4) != 0 || ld > 0xFFFFFFFCull) return TNG_ERR_INVALID_ARG;
    return TNG_OK;
}

// ---- timing helpers ---------------------------------------------------------------
void harvest_events(tng_ctx* c) {
    if (!c->ev_created || c->ev_used == 0) return;
    cudaEventSynchronize(c->ev[c->ev_used - 1][kStages]);
    for (int r = 0; r < c->ev_used; ++r) {
        for (int s = 0; s < kStages; ++s) {
            if (!c->ev_stage_ran[r][s]) continue;
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, c->ev[r][s], c->ev[r][s + 1]) == cudaSuccess) c->ms_sum[s] += ms;
        }
        c->timed_rounds += 1;
    }
    c->ev_used = 0;
}

struct StageTimer {
    tng_ctx* c;
    cudaStream_t st;
    int slot = -1;
    StageTimer(tng_ctx* ctx, cudaStream_t s) : c(ctx), st(s) {
        if (!c->timing) return;
        if (!c->ev_created) {
            for (int r = 0; r < kTimedRounds; ++r)
                for (int s2 = 0; s2 <= kStages; ++s2) cudaEventCreate(&c->ev[r][s2]);
            c->ev_created = true;
        }
        if (c->ev_used == kTimedRounds) harvest_events(c);
        slot = c->ev_used++;
        for (int s2 = 0; s2 < kStages; ++s2) c->ev_stage_ran[slot][s2] = false;
        cudaEventRecord(c->ev[slot][0], st);
    }
    // called after stage s has been enqueued; stages must be marked in order 0..4
    void mark(int s, bool ran) {
        if (slot < 0) return;
        c->ev_stage_ran[slot][s] = ran;
        cudaEventRecord(c->ev[slot][s + 1], st);
    }
};

// ---- the stages -----------------------------------------------------------------------
// `defer` (may be nullptr): when the encode pass can build the reference itself, the combine
// launch is skipped and *defer describes the combination for launch_encode.
// `stats_ready`: the statistics are already in the FuseBlock as sums over ALL workers (rank-local
// sums added up by the caller); the statistics pass is skipped and the solve divides them by M.
tng_status do_fuse(tng_ctx* c, const float* grads, uint64_t ld, cudaStream_t st, StageTimer* tm, RefFusion* defer,
                   bool stats_ready = false) {
    if (defer) defer->k = 0;
    const int mode = c->effective_mode();
    c->last_mode = mode;
    c->last_had_stats = false;
    c->last_solved = false;
    int launches = 0;
    if (c->k == 0) {   // empty trajectory: reference = zeros (initial state of Algorithm 1)
        TNG_CUDA(c, cudaMemsetAsync(c->ref_buf(), 0, c->d_pad * sizeof(float), st));
        if (c->ref2_buf()) {
            TNG_CUDA(c, cudaMemsetAsync(c->ref2_buf(), 0, c->d_pad * sizeof(float), st));
            c->ref2_valid = true;
        }
        c->ref_cur = c->ref_buf();
        if (tm) { tm->mark(0, false); tm->mark(1, false); tm->mark(2, false); }
        return TNG_OK;
    }
    const float* rows[kMaxK];
    for (uint32_t j = 0; j < c->k; ++j) rows[j] = c->ring(c->hist_slot(j));
    if (mode == TNG_FUSE_LAST && c->norm != TNG_NORM_COMB) {   // delayed-gradient reference: alias the newest slot, no pass
        c->ref_cur = rows[0];
        if (tm) { tm->mark(0, false); tm->mark(1, false); tm->mark(2, false); }
        return TNG_OK;
    }
    const bool need_dots = (mode == TNG_FUSE_LSQ) || (mode == TNG_FUSE_HINDSIGHT);
    if (need_dots && !stats_ready) {
        const float* g = (mode == TNG_FUSE_LSQ) ? grads : nullptr;
        TNG_CUDA(c, launch_dots(rows, (int)c->k, c->d, g, c->M, ld, 0, c->partials(), c->fb(), c->sm_count, st, &launches));
    }
    c->last_had_stats = need_dots;
    if (tm) tm->mark(0, need_dots && !stats_ready);
    TNG_CUDA(c, launch_solve(c->fb(), (int)c->k, mode, c->ridge, (stats_ready && mode == TNG_FUSE_LSQ) ? (double)c->M : 1.0, st, &launches));
    c->last_solved = true;
    if (tm) tm->mark(1, true);
    if (defer && encode_can_fuse_reference(c->geom)) {
        for (uint32_t j = 0; j < c->k; ++j) defer->rows[j] = rows[j];
        defer->k = (int)c->k;
        defer->alpha = c->fb()->alpha32;
        defer->ref_out = c->ref_buf();
        defer->ref2_out = c->ref2_buf();
        if (tm) tm->mark(2, false);
    } else {
        TNG_CUDA(c, launch_combine(rows, (int)c->k, c->d, c->fb(), c->ref_buf(), c->ref2_buf(), c->sm_count, st, &launches));
        if (tm) tm->mark(2, true);
    }
    c->ref_cur = c->ref_buf();
    if (c->ref2_buf()) c->ref2_valid = true;
    c->launches += (uint64_t)launches;
    return TNG_OK;
}

tng_status do_encode(tng_ctx* c, const float* grads, uint64_t ld, const float* ref, const RefFusion* fusion, uint32_t step,
                     cudaStream_t st) {
    int launches = 0;
    TNG_CUDA(c, launch_encode(c->geom, 0, grads, ld, ref, c->ref2_buf(), fusion, step, c->codes(), c->scales(), c->means(),
                              c->tile_stat(), c->tree(), c->fb(), c->sm_count, st, &launches));
    c->launches += (uint64_t)launches;
    return TNG_OK;
}

tng_status do_decode(tng_ctx* c, const float* ref, float* out_a, float* out_b, cudaStream_t st) {
    int launches = 0;
    TNG_CUDA(c, launch_decode(c->geom, c->codes(), c->scales(), c->means(), ref, c->ref2_buf(), out_a, out_b, c->fb(), c->sm_count, st,
                              &launches));
    c->launches += (uint64_t)launches;
    return TNG_OK;
}

// Form the reference a rank-local fusion left to the encode pass, if it is still owed.
tng_status materialise_ref(tng_ctx* c, cudaStream_t st) {
    if (!c->ref_pending) return TNG_OK;
    int launches = 0;
    TNG_CUDA(c, launch_combine(c->pending.rows, c->pending.k, c->d, c->fb(), c->ref_buf(), c->ref2_buf(), c->sm_count, st, &launches));
    c->launches += (uint64_t)launches;
    c->ref_pending = false;
    return TNG_OK;
}

// The decoded aggregate goes straight into the next ring slot (and to the caller's buffer); the
// round is then complete: ring rotated, round counter advanced.
tng_status decode_commit(tng_ctx* c, float* out, cudaStream_t st) {
    tng_status sm = materialise_ref(c, st);
    if (sm != TNG_OK) return sm;
    const int slot = (c->k == 0) ? c->head : (c->head + 1) % (int)c->K;
    tng_status s = do_decode(c, c->ref_cur, c->ring(slot), out, st);
    if (s != TNG_OK) return s;
    c->head = slot;
    if (c->k < c->K) c->k += 1;
    c->rounds += 1;
    return TNG_OK;
}

tng_status step_impl(tng_ctx* c, const float* grads, uint64_t ld, float* out, cudaStream_t st) {
    {
        tng_status sm = materialise_ref(c, st);   // (a held reference may still be owed by a rank-local fusion)
        if (sm != TNG_OK) return sm;
    }
    StageTimer tm(c, st);
    RefFusion fusion;
    fusion.k = 0;
    tng_status s = TNG_OK;
    if (c->norm == TNG_NORM_MEAN) {   // the scalar reference uses no trajectory
        tm.mark(0, false); tm.mark(1, false); tm.mark(2, false);
    } else if (c->rounds % c->ref_every == 0 || !c->ref_cur) {
        s = do_fuse(c, grads, ld, st, &tm, &fusion);
        if (s != TNG_OK) return s;
        if (c->ref_every > 1 && c->ref_cur != c->ref_buf()) {
            // the reference is held for several rounds: it must not alias a ring slot that will be overwritten
            TNG_CUDA(c, cudaMemcpyAsync(c->ref_buf(), c->ref_cur, c->d * sizeof(float), cudaMemcpyDeviceToDevice, st));
            c->ref_cur = c->ref_buf();
        }
    } else {   // between refreshes: the held reference, no fusion pass
        tm.mark(0, false); tm.mark(1, false); tm.mark(2, false);
    }
    s = do_encode(c, grads, ld, c->ref_cur, &fusion, (uint32_t)c->rounds, st);
    if (s != TNG_OK) return s;
    tm.mark(3, true);
    s = decode_commit(c, out, st);
    if (s != TNG_OK) return s;
    tm.mark(4, true);
    return TNG_OK;
}

// nothing ever arrives on this barrier: the wait has to end by its poll limit
__global__ void bounded_wait_selftest_kernel(uint32_t* outcome) {
    __shared__ uint64_t bar;
    const uint32_t b = tng::smem_u32(&bar);
    if (threadIdx.x == 0) {
        tng::mbar_init(b, 1);
        tng::mbar_init_fence();
    }
    __syncthreads();
    const bool completed = tng::mbar_wait_limited(b, 0u, 1024);
    if (threadIdx.x == 0) *outcome = completed ? 2u : 1u;
}

}  // namespace

// =========================================================================================
extern "C" {

tng_status tng_create(tng_ctx** out, uint64_t d, uint32_t M, uint32_t K, tng_codec codec, tng_norm_mode norm) {
    if (!out) return TNG_ERR_INVALID_ARG;
    *out = nullptr;
    if (d < 1 || d > TNG_MAX_COORDS || M < 1 || M > TNG_MAX_WORKERS || K < 1 || K > TNG_MAX_HISTORY) return TNG_ERR_INVALID_ARG;
    if (codec != TNG_CODEC_SIGN1 && codec != TNG_CODEC_TERN2 && codec != TNG_CODEC_QSGD4) return TNG_ERR_INVALID_ARG;
    if (norm != TNG_NORM_NONE && norm != TNG_NORM_DIFF && norm != TNG_NORM_QUOT && norm != TNG_NORM_COMB && norm != TNG_NORM_MEAN)
        return TNG_ERR_INVALID_ARG;
    tng_ctx* c = new (std::nothrow) tng_ctx();
    if (!c) return TNG_ERR_ALLOC;
    c->d = d; c->M = M; c->K = K; c->codec = (int)codec; c->norm = (int)norm;
    *out = c;
    return TNG_OK;
}

void tng_destroy(tng_ctx* c) {
    if (!c) return;
    if (c->ws_ready) cudaStreamSynchronize(c->last_stream);
    if (c->copy_stream) {
        cudaStreamSynchronize(c->copy_stream);
        cudaEventDestroy(c->ev_round_done);
        cudaEventDestroy(c->ev_copied);
        cudaStreamDestroy(c->copy_stream);
    }
    if (c->ev_created)
        for (int r = 0; r < kTimedRounds; ++r)
            for (int s = 0; s <= kStages; ++s) cudaEventDestroy(c->ev[r][s]);
    if (c->ws_owned && c->ws) cudaFree(c->ws);
    delete c;
}

tng_status tng_set_option(tng_ctx* c, tng_option key, double value) {
    if (!c) return TNG_ERR_INVALID_ARG;
    if (c->sized) return TNG_ERR_STATE;
    if (!(value == value)) return TNG_ERR_INVALID_ARG;
    switch (key) {
        case TNG_OPT_BLOCK:
            if (value < 0 || value > 1e15 || value != floor(value) || ((uint64_t)value % TNG_TILE) != 0) return TNG_ERR_INVALID_ARG;
            c->block_opt = (uint64_t)value; return TNG_OK;
        case TNG_OPT_QSGD_LEVELS:
            if (value < 1 || value > 7 || value != floor(value)) return TNG_ERR_INVALID_ARG;
            c->levels = (int)value; return TNG_OK;
        case TNG_OPT_SCALE_KIND:
            if (value != 0 && value != 1) return TNG_ERR_INVALID_ARG;
            c->scale_kind = (int)value; return TNG_OK;
        case TNG_OPT_SEED_LO:
        case TNG_OPT_SEED_HI:
            if (value < 0 || value > 4294967295.0 || value != floor(value)) return TNG_ERR_INVALID_ARG;
            (key == TNG_OPT_SEED_LO ? c->seed_lo : c->seed_hi) = (uint32_t)value; return TNG_OK;
        case TNG_OPT_FUSE_MODE:
            if (value < 0 || value > 4 || value != floor(value)) return TNG_ERR_INVALID_ARG;
            c->fuse_mode = (int)value; return TNG_OK;
        case TNG_OPT_RIDGE:
            if (!(value >= 0) || !(value < 1e300)) return TNG_ERR_INVALID_ARG;
            c->ridge = value; return TNG_OK;
        case TNG_OPT_QUOT_EPS:
            if (!(value > 0 && value <= 1)) return TNG_ERR_INVALID_ARG;
            c->quot_eps = (float)value; return TNG_OK;
        case TNG_OPT_TIMING:
            if (value != 0 && value != 1) return TNG_ERR_INVALID_ARG;
            c->timing = (int)value; return TNG_OK;
        case TNG_OPT_HOST_STAGING:
            if (value != 0 && value != 1) return TNG_ERR_INVALID_ARG;
            c->host_staging = (int)value; return TNG_OK;
        case TNG_OPT_COORD_OFFSET:
            if (value < 0 || value > 281474976710656.0 || value != floor(value) || fmod(value, (double)TNG_TILE) != 0.0) return TNG_ERR_INVALID_ARG;
            c->coord_offset = (uint64_t)value; return TNG_OK;
        case TNG_OPT_REF_EVERY:
            if (value < 1 || value > 65536 || value != floor(value)) return TNG_ERR_INVALID_ARG;
            c->ref_every = (uint32_t)value; return TNG_OK;
        default: return TNG_ERR_INVALID_ARG;
    }
}

tng_status tng_workspace_bytes(tng_ctx* c, size_t* bytes) {
    if (!c || !bytes) return TNG_ERR_INVALID_ARG;
    size_ctx(c);
    *bytes = c->ws_bytes;
    return TNG_OK;
}

tng_status tng_bind_workspace(tng_ctx* c, void* dev_ptr, size_t bytes) {
    if (!c || !dev_ptr) return TNG_ERR_INVALID_ARG;
    if (c->ws_ready || c->ws) return TNG_ERR_STATE;
    if ((reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0) return TNG_ERR_INVALID_ARG;
    size_ctx(c);
    if (bytes < c->ws_bytes) return TNG_ERR_ALLOC;
    c->ws = dev_ptr;
    c->ws_owned = false;
    return TNG_OK;
}

tng_status tng_push_reference(tng_ctx* c, const float* vec_dev, void* stream) {
    if (!c || !vec_dev || !aligned16(vec_dev)) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    s = materialise_ref(c, st);   // the slot written below may be a row an owed combine still reads
    if (s != TNG_OK) return s;
    const int slot = (c->k == 0) ? c->head : (c->head + 1) % (int)c->K;
    TNG_CUDA(c, cudaMemcpyAsync(c->ring(slot), vec_dev, c->d * sizeof(float), cudaMemcpyDeviceToDevice, st));
    c->head = slot;
    if (c->k < c->K) c->k += 1;
    return TNG_OK;
}

tng_status tng_step(tng_ctx* c, const float* grads_dev, uint64_t ld, float* agg_out_dev, void* stream) {
    if (!c) return TNG_ERR_INVALID_ARG;
    tng_status s = check_rows(c, grads_dev, ld);
    if (s != TNG_OK) return s;
    if (agg_out_dev && !aligned16(agg_out_dev)) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    return step_impl(c, grads_dev, ld, agg_out_dev, st);
}

tng_status tng_step_host(tng_ctx* c, const float* grads_host, uint64_t ld, float* agg_out_host, void* stream) {
    if (!c || !grads_host || !agg_out_host || ld < c->d || ld > 0xFFFFFFFCull) return TNG_ERR_INVALID_ARG;
    if (!c->host_staging) return TNG_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    TNG_CUDA(c, cudaMemcpy2DAsync(c->stage_g(), c->d_pad * sizeof(float), grads_host, ld * sizeof(float),
                                  c->d * sizeof(float), c->M, cudaMemcpyHostToDevice, st));
    if (c->copy_pending) TNG_CUDA(c, cudaStreamWaitEvent(st, c->ev_copied, 0));   // an earlier tng_step_host_async still copying out
    s = step_impl(c, c->stage_g(), c->d_pad, c->stage_o(), st);
    if (s != TNG_OK) return s;
    TNG_CUDA(c, cudaMemcpyAsync(agg_out_host, c->stage_o(), c->d * sizeof(float), cudaMemcpyDeviceToHost, st));
    TNG_CUDA(c, cudaStreamSynchronize(st));
    return TNG_OK;
}

tng_status tng_step_host_async(tng_ctx* c, const float* grads_host, uint64_t ld, float* agg_out_host, void* stream) {
    if (!c || !grads_host || !agg_out_host || ld < c->d || ld > 0xFFFFFFFCull) return TNG_ERR_INVALID_ARG;
    if (!c->host_staging) return TNG_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    if (!c->copy_stream) {
        TNG_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        TNG_CUDA(c, cudaEventCreateWithFlags(&c->ev_round_done, cudaEventDisableTiming));
        TNG_CUDA(c, cudaEventCreateWithFlags(&c->ev_copied, cudaEventDisableTiming));
    }
    TNG_CUDA(c, cudaMemcpy2DAsync(c->stage_g(), c->d_pad * sizeof(float), grads_host, ld * sizeof(float),
                                  c->d * sizeof(float), c->M, cudaMemcpyHostToDevice, st));
    // the previous aggregate must have left the staging buffer before this round's decode rewrites it;
    // the rows above do not wait for that, which is where the two directions overlap
    if (c->copy_pending) TNG_CUDA(c, cudaStreamWaitEvent(st, c->ev_copied, 0));
    s = step_impl(c, c->stage_g(), c->d_pad, c->stage_o(), st);
    if (s != TNG_OK) return s;
    TNG_CUDA(c, cudaEventRecord(c->ev_round_done, st));
    TNG_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_round_done, 0));
    TNG_CUDA(c, cudaMemcpyAsync(agg_out_host, c->stage_o(), c->d * sizeof(float), cudaMemcpyDeviceToHost, c->copy_stream));
    TNG_CUDA(c, cudaEventRecord(c->ev_copied, c->copy_stream));
    c->copy_pending = true;
    return TNG_OK;
}

tng_status tng_host_wait(tng_ctx* c) {
    if (!c) return TNG_ERR_INVALID_ARG;
    if (!c->copy_pending) return TNG_OK;
    TNG_CUDA(c, cudaStreamSynchronize(c->last_stream));   // the rows of the last call have been read
    TNG_CUDA(c, cudaEventSynchronize(c->ev_copied));
    c->copy_pending = false;
    return TNG_OK;
}

namespace {
struct StateHeader {
    uint32_t magic, version;
    uint64_t d;
    uint32_t M, K, codec, norm;
    uint64_t block;
    uint32_t levels, scale_kind, fuse_mode, seed_lo, seed_hi, ref_every;
    double ridge;
    float quot_eps;
    uint32_t k;
    uint64_t rounds;
    uint32_t has_ref, pad;
    uint64_t coord_offset;
};
constexpr uint32_t kStateMagic = 0x53474e54u;   // "TNGS"

void fill_header(const tng_ctx* c, StateHeader* h) {
    memset(h, 0, sizeof *h);
    h->magic = kStateMagic; h->version = 2;
    h->d = c->d; h->M = c->M; h->K = c->K; h->codec = (uint32_t)c->codec; h->norm = (uint32_t)c->norm;
    h->block = c->block_opt; h->levels = (uint32_t)c->levels; h->scale_kind = (uint32_t)c->scale_kind;
    h->fuse_mode = (uint32_t)c->fuse_mode; h->seed_lo = c->seed_lo; h->seed_hi = c->seed_hi; h->ref_every = c->ref_every;
    h->ridge = c->ridge; h->quot_eps = c->quot_eps;
    h->k = c->k; h->rounds = c->rounds; h->has_ref = 0; h->coord_offset = c->coord_offset;
}
}  // namespace

tng_status tng_state_bytes(tng_ctx* c, size_t* bytes) {
    if (!c || !bytes) return TNG_ERR_INVALID_ARG;
    *bytes = sizeof(StateHeader) + ((size_t)c->K + 2) * c->d * sizeof(float);
    return TNG_OK;
}

tng_status tng_save_state(tng_ctx* c, void* host_buf, size_t bytes, size_t* written, void* stream) {
    if (!c || !host_buf) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    s = materialise_ref(c, st);
    if (s != TNG_OK) return s;
    StateHeader h;
    fill_header(c, &h);
    h.has_ref = (c->ref_every > 1 && c->ref_cur) ? 1u : 0u;
    if (h.has_ref && c->norm == TNG_NORM_COMB) h.has_ref = c->ref2_valid ? 2u : 0u;   // both references or none
    const size_t vec = c->d * sizeof(float);
    const size_t need = sizeof h + ((size_t)c->k + h.has_ref) * vec;
    if (bytes < need) return TNG_ERR_ALLOC;
    char* p = static_cast<char*>(host_buf);
    memcpy(p, &h, sizeof h);
    p += sizeof h;
    for (uint32_t j = 0; j < c->k; ++j, p += vec)   // newest first
        TNG_CUDA(c, cudaMemcpyAsync(p, c->ring(c->hist_slot(j)), vec, cudaMemcpyDeviceToHost, st));
    if (h.has_ref) TNG_CUDA(c, cudaMemcpyAsync(p, c->ref_cur, vec, cudaMemcpyDeviceToHost, st));
    if (h.has_ref == 2) TNG_CUDA(c, cudaMemcpyAsync(p + vec, c->ref2_buf(), vec, cudaMemcpyDeviceToHost, st));
    TNG_CUDA(c, cudaStreamSynchronize(st));
    if (written) *written = need;
    return TNG_OK;
}

tng_status tng_load_state(tng_ctx* c, const void* host_buf, size_t bytes, void* stream) {
    if (!c || !host_buf || bytes < sizeof(StateHeader)) return TNG_ERR_INVALID_ARG;
    StateHeader h, mine;
    memcpy(&h, host_buf, sizeof h);
    fill_header(c, &mine);
    if (h.magic != kStateMagic || h.version != 2 || h.coord_offset != mine.coord_offset || h.d != mine.d || h.M != mine.M || h.K != mine.K || h.codec != mine.codec ||
        h.norm != mine.norm || h.block != mine.block || h.levels != mine.levels || h.scale_kind != mine.scale_kind ||
        h.fuse_mode != mine.fuse_mode || h.seed_lo != mine.seed_lo || h.seed_hi != mine.seed_hi || h.ref_every != mine.ref_every ||
        h.ridge != mine.ridge || h.quot_eps != mine.quot_eps || h.k > h.K || h.has_ref > 2 ||
        (h.has_ref == 2) != (h.has_ref != 0 && c->norm == TNG_NORM_COMB))
        return TNG_ERR_INVALID_ARG;
    const size_t vec = c->d * sizeof(float);
    if (bytes < sizeof h + ((size_t)h.k + h.has_ref) * vec) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    const char* p = static_cast<const char*>(host_buf) + sizeof h;
    // h_{j+1} goes to slot k-1-j, the newest entry sitting at head = k-1
    for (uint32_t j = 0; j < h.k; ++j, p += vec)
        TNG_CUDA(c, cudaMemcpyAsync(c->ring((int)(h.k - 1 - j)), p, vec, cudaMemcpyHostToDevice, st));
    if (h.has_ref) TNG_CUDA(c, cudaMemcpyAsync(c->ref_buf(), p, vec, cudaMemcpyHostToDevice, st));
    if (h.has_ref == 2) TNG_CUDA(c, cudaMemcpyAsync(c->ref2_buf(), p + vec, vec, cudaMemcpyHostToDevice, st));
    TNG_CUDA(c, cudaStreamSynchronize(st));
    c->ref2_valid = h.has_ref == 2;
    c->ref_pending = false;
    c->k = h.k;
    c->head = h.k ? (int)h.k - 1 : 0;
    c->rounds = h.rounds;
    c->ref_cur = h.has_ref ? c->ref_buf() : nullptr;
    c->last_mode = c->effective_mode();
    c->last_had_stats = false;
    c->last_solved = false;
    return TNG_OK;
}

// ---- one worker (or a few) per GPU: the rank-local pieces of a round ---------------------
tng_status tng_fuse_local(tng_ctx* c, const float* grads_dev, uint64_t ld, uint32_t m_count, void* stream) {
    if (!c || m_count < 1 || m_count > c->M) return TNG_ERR_INVALID_ARG;
    tng_status s = check_rows(c, grads_dev, ld);
    if (s != TNG_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    // the block the caller adds up over the ranks (rhs[16] and grad_sq, or all of it when the ranks hold
    // slices of the coordinates): zero wherever this round's statistics pass writes nothing
    TNG_CUDA(c, cudaMemsetAsync(c->fb()->gram, 0, kGramDoubles * sizeof(double), st));
    const int mode = c->effective_mode();
    if (c->k == 0 || (mode != TNG_FUSE_LSQ && mode != TNG_FUSE_HINDSIGHT)) return TNG_OK;
    const float* rows[kMaxK];
    for (uint32_t j = 0; j < c->k; ++j) rows[j] = c->ring(c->hist_slot(j));
    int launches = 0;
    TNG_CUDA(c, launch_dots(rows, (int)c->k, c->d, mode == TNG_FUSE_LSQ ? grads_dev : nullptr, m_count, ld, 1, c->partials(), c->fb(),
                            c->sm_count, st, &launches));
    c->launches += (uint64_t)launches;
    return TNG_OK;
}

tng_status tng_local_stats(tng_ctx* c, double** sums_dev, size_t* count) {
    if (!c || !sums_dev || !count) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    *sums_dev = c->fb()->gram + kGramRhs;
    *count = (size_t)kMaxK + 1;
    return TNG_OK;
}

tng_status tng_selftest_bounded_wait(tng_ctx* c, uint32_t* gave_up_host, void* stream) {
    if (!c || !gave_up_host) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    uint32_t* word = reinterpret_cast<uint32_t*>(c->partials());   // scratch between launches of the statistics pass
    TNG_CUDA(c, cudaMemsetAsync(word, 0, sizeof(uint32_t), st));
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(word);
    TNG_CUDA(c, cudaGetLastError());
    uint32_t outcome = 0;
    TNG_CUDA(c, cudaMemcpyAsync(&outcome, word, sizeof outcome, cudaMemcpyDeviceToHost, st));
    TNG_CUDA(c, cudaStreamSynchronize(st));
    *gave_up_host = (outcome == 1u) ? 1u : 0u;
    c->launches += 1;
    return TNG_OK;
}

tng_status tng_local_stats_all(tng_ctx* c, double** sums_dev, size_t* count) {
    if (!c || !sums_dev || !count) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    *sums_dev = c->fb()->gram;
    *count = (size_t)kGramDoubles;
    return TNG_OK;
}

tng_status tng_fuse_finish(tng_ctx* c, void* stream) {
    if (!c) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    c->ref_pending = false;
    s = do_fuse(c, nullptr, 0, st, nullptr, &c->pending, true);
    if (s == TNG_OK && c->pending.k > 0) c->ref_pending = true;
    return s;
}

tng_status tng_encode_local(tng_ctx* c, const float* grads_dev, uint64_t ld, uint32_t m_first, uint32_t m_count, uint32_t step,
                            void* stream) {
    if (!c || m_count < 1 || m_first >= c->M || m_count > c->M - m_first) return TNG_ERR_INVALID_ARG;
    tng_status s = check_rows(c, grads_dev, ld);
    if (s != TNG_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    if (!c->ref_cur && !c->no_ref()) return TNG_ERR_STATE;   // no fusion has produced a reference yet
    if (c->norm == TNG_NORM_COMB && !c->ref2_valid) return TNG_ERR_STATE;
    CodecGeom g = c->geom;
    g.M = m_count;
    int launches = 0;
    const RefFusion* owed = c->ref_pending ? &c->pending : nullptr;   // the first encode after a fusion forms the reference
    c->ref_pending = false;
    TNG_CUDA(c, launch_encode(g, m_first, grads_dev, ld, c->ref_cur, c->ref2_buf(), owed, step, c->codes() + (size_t)m_first * g.wpw,
                              c->scales() + (size_t)m_first * g.nblk, c->means() + m_first, c->tile_stat(), c->tree(), c->fb(),
                              c->sm_count, st, &launches));
    c->launches += (uint64_t)launches;
    return TNG_OK;
}

tng_status tng_decode_commit(tng_ctx* c, float* agg_out_dev, void* stream) {
    if (!c || (agg_out_dev && !aligned16(agg_out_dev))) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    if (!c->ref_cur && !c->no_ref()) return TNG_ERR_STATE;
    return decode_commit(c, agg_out_dev, st);
}

tng_status tng_fuse(tng_ctx* c, const float* grads_dev, uint64_t ld, void* stream) {
    if (!c) return TNG_ERR_INVALID_ARG;
    tng_status s = check_rows(c, grads_dev, ld);
    if (s != TNG_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    c->ref_pending = false;   // a new fusion replaces whatever reference was still owed
    return do_fuse(c, grads_dev, ld, st, nullptr, nullptr);
}

tng_status tng_encode(tng_ctx* c, const float* grads_dev, uint64_t ld, const float* ref_dev, uint32_t step, void* stream) {
    if (!c) return TNG_ERR_INVALID_ARG;
    tng_status s = check_rows(c, grads_dev, ld);
    if (s != TNG_OK) return s;
    if (ref_dev && !aligned16(ref_dev)) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    s = materialise_ref(c, st);
    if (s != TNG_OK) return s;
    const float* ref = ref_dev ? ref_dev : c->ref_cur;
    if (!ref && !c->no_ref()) return TNG_ERR_STATE;   // no fusion has produced a reference yet
    if (c->norm == TNG_NORM_COMB && !c->ref2_valid) return TNG_ERR_STATE;   // the second reference comes from a fusion
    return do_encode(c, grads_dev, ld, ref, nullptr, step, st);
}

tng_status tng_decode_aggregate(tng_ctx* c, const float* ref_dev, float* out_dev, void* stream) {
    if (!c || !out_dev || !aligned16(out_dev)) return TNG_ERR_INVALID_ARG;
    if (ref_dev && !aligned16(ref_dev)) return TNG_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    tng_status s = ensure_ready(c, st);
    if (s != TNG_OK) return s;
    s = materialise_ref(c, st);
    if (s != TNG_OK) return s;
    const float* ref = ref_dev ? ref_dev : c->ref_cur;
    if (!ref && !c->no_ref()) return TNG_ERR_STATE;
    if (c->norm == TNG_NORM_COMB && !c->ref2_valid) return TNG_ERR_STATE;
    return do_decode(c, ref, out_dev, nullptr, st);
}

tng_status tng_wire(tng_ctx* c, const uint32_t** codes_dev, size_t* words_per_worker, const float** scales_dev,
                    size_t* scales_per_worker) {
    if (!c) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    if (codes_dev) *codes_dev = c->codes();
    if (words_per_worker) *words_per_worker = (size_t)c->geom.wpw;
    if (scales_dev) *scales_dev = c->scales();
    if (scales_per_worker) *scales_per_worker = (size_t)c->geom.nblk;
    return TNG_OK;
}

tng_status tng_wire_means(tng_ctx* c, const float** means_dev) {
    if (!c || !means_dev) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready) return TNG_ERR_STATE;
    *means_dev = c->means();
    return TNG_OK;
}

tng_status tng_reference(tng_ctx* c, const float** ref_dev) {
    if (!c || !ref_dev) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready || !c->ref_cur) return TNG_ERR_STATE;
    if (materialise_ref(c, c->last_stream) != TNG_OK) return TNG_ERR_CUDA;   // on the stream of the last call
    *ref_dev = c->ref_cur;
    return TNG_OK;
}

tng_status tng_history(tng_ctx* c, uint32_t j, const float** vec_dev) {
    if (!c || !vec_dev) return TNG_ERR_INVALID_ARG;
    if (!c->ws_ready || j >= c->k) return TNG_ERR_STATE;
    *vec_dev = c->ring(c->hist_slot(j));
    return TNG_OK;
}

tng_status tng_stats(tng_ctx* c, tng_stats_t* out) {
    if (!c || !out) return TNG_ERR_INVALID_ARG;
    memset(out, 0, sizeof *out);
    size_ctx(c);
    out->d = c->d; out->M = c->M; out->K = c->K; out->k = c->k;
    out->fuse_mode = (uint32_t)c->effective_mode();
    out->rounds = c->rounds;
    out->bits_per_coord = (double)c->codec + 32.0 / (double)c->geom.block + 64.0 * (double)c->K / (double)c->d;
    out->cnz = nan("");
    out->kernel_launches = c->launches;
    if (!c->ws_ready) return TNG_OK;
    TNG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    harvest_events(c);
    FuseBlock h;
    TNG_CUDA(c, cudaMemcpy(&h, c->fb(), sizeof h, cudaMemcpyDeviceToHost));
    const int mode = c->last_mode;
    if (!c->last_solved) {
        out->alpha[0] = (mode == TNG_FUSE_LAST && c->ref_cur && c->ref_cur != c->ref_buf()) ? 1.0 : 0.0;
    } else {
        for (int j = 0; j < TNG_MAX_HISTORY; ++j) out->alpha[j] = h.alpha64[j];
        out->solver_fallback = h.fallback;
    }
    if (c->last_had_stats) {
        for (int i = 0; i < TNG_MAX_HISTORY * TNG_MAX_HISTORY; ++i) out->gram[i] = h.gram[i];
        if (mode == TNG_FUSE_LSQ) {
            for (int i = 0; i < TNG_MAX_HISTORY; ++i) out->rhs[i] = h.gram[kGramRhs + i];
            out->grad_sq = h.gram[kGramGG];
            out->cnz = h.cnz;
        }
    }
    out->nonfinite_scales = h.nonfinite;
    out->pipeline_error = h.pipe_error;
    out->timed_rounds = c->timed_rounds;
    if (c->timed_rounds) {
        const double n = (double)c->timed_rounds;
        out->ms_dots = c->ms_sum[0] / n; out->ms_solve = c->ms_sum[1] / n; out->ms_combine = c->ms_sum[2] / n;
        out->ms_encode = c->ms_sum[3] / n; out->ms_decode = c->ms_sum[4] / n;
    }
    if (h.pipe_error != 0) return TNG_ERR_CUDA;
    if (h.nonfinite > c->nonfinite_reported) {
        c->nonfinite_reported = h.nonfinite;
        return TNG_ERR_NONFINITE;
    }
    return TNG_OK;
}

const char* tng_status_string(tng_status s) {
    switch (s) {
        case TNG_OK: return "ok";
        case TNG_ERR_INVALID_ARG: return "invalid argument";
        case TNG_ERR_STATE: return "call not allowed in this state";
        case TNG_ERR_ALLOC: return "allocation failed or workspace too small";
        case TNG_ERR_CUDA: return "CUDA error";
        case TNG_ERR_NONFINITE: return "non-finite block scale";
        case TNG_ERR_UNSUPPORTED: return "unsupported";
        default: return "unknown status";
    }
}

int tng_last_cuda_error(const tng_ctx* c) { return c ? c->last_cuda_error : 0; }

}  // extern "C"
