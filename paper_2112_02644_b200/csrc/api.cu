// C ABI of the SMTM library: argument checking, state ownership and launch planning.
// Every step of the path runs in the kernels of encode.cu, lookup.cu and memory.cu.
#include <string.h>

#include <new>
#include <vector>

#include "internal.h"

using namespace smtm;

struct smtm_cache {
    int n, L, S, k_init, k_min, k_max, W, cl_num, cl_den, max_batch;
    bool forgetting;    // SMTM_FLAG_FORGET_FT
    bool maps_ready;    // SMTM_FLAG_MAPS_READY
    int dims[SMTM_MAX_LAYERS];
    float tau[SMTM_MAX_LAYERS];
    float* d_centers[SMTM_MAX_LAYERS];
    float* d_cnorm[SMTM_MAX_LAYERS];
    uint32_t* d_m[SMTM_MAX_LAYERS];
    int32_t* d_ft;
    int32_t* d_ts;
    int32_t* d_members;
    int32_t* d_k;
    unsigned long long* d_counters;
    int* d_status;
    float* d_warm_sv;   // scratch of smtm_cache_warmup: [max_batch][C_max] semantic vectors (allocated on first use)
    void* d_dense;      // scratch of the tensor-core scorer (fast memories above 64 entries), else NULL
    void* d_cen_split[SMTM_MAX_LAYERS];   // bf16 heads and tails of the centres, per layer (same condition)
    int d_max;          // largest C_l
    int32_t* d_plan;    // scratch of the update: final label and stop layer of every frame, [max_batch]
    unsigned long long* d_tags;  // scratch of the update: stamps of (layer, class), [L][n]
    // pipelined route (SMTM_FLAG_MAPS_READY): the pooling of a step's first layer runs on a stream of the cache's own
    cudaStream_t pool_stream;
    cudaEvent_t ev_fork, ev_pool;       // the caller's stream -> pool stream, and back
    cudaEvent_t ev_mark[2];             // where the caller's stream stood at the last two first lookups (they alternate)
    int split_which;                    // which of the two split buffers the batch under way uses (0 unless pipelined)
    unsigned long long mark_capture[2]; // the stream capture each was recorded in (0 = none)
    bool mark_valid[2];
    int mark_next;                      // which of the two the next first lookup records
    int32_t* d_jobs;             // scratch of the update: [4] counters, [L][n] (layer, class) pairs to fold, [16][L][n] work items
    float* d_norm_part;          // scratch of the update: [L][n][16] squared lengths of the blocks of a centre folded by several CTAs
    int32_t* d_ticket;           // scratch of the update: [L][n] tickets of those CTAs (zero between updates)
    unsigned long long* d_epoch; // [2] device: update calls so far, and the plan kernel's ticket
    // optional timing of the streaming kernel of every lookup (smtm_cache_profile)
    std::vector<cudaEvent_t>* prof_events;  // pairs, in launch order
    std::vector<int>* prof_layer;           // layer of each pair
    size_t prof_used;                       // pairs recorded so far
    unsigned long long* d_prof_clock;       // [steps][SMTM_PROF_KERNELS][2] device-clock stamps of the profiled steps
    size_t prof_steps_cap, prof_steps_used;  // slots of d_prof_clock
    unsigned long long* prof_step;          // the slot of the step under way, nullptr if it is not profiled
    int prof_every;                         // a pair is recorded for every prof_every-th lookup call
    long long prof_seq;                     // lookup calls since profiling was switched on
    int device, sm_count;
    int64_t launches;
    int64_t routes[SMTM_ROUTE_COUNT];  // lookups served by each route (a host-side decision, counted on the host)
    FusedCaps fused_caps;              // cluster capacities of the fused kernel on this cache's device
    // device-side carry and staging used only by smtm_step_host (allocated on first use)
    bool host_ready;
    smtm_batch_t hb;
    int32_t* d_stream_id;
    int32_t* d_fallback;
    uint8_t* h_flags;   // pinned host copy of the exit flags between two layers of smtm_step_host
    void* d_stage[SMTM_MAX_LAYERS];
    size_t stage_bytes[SMTM_MAX_LAYERS];
};

void smtm::cache_shape(const smtm_cache_t* cache, int* n_layers, int* k_max) {
    *n_layers = cache->L;
    *k_max = cache->k_max;
}

namespace {

#define SMTM_CUDA(call)                         \
    do {                                         \
        if ((call) != cudaSuccess) {             \
            (void)cudaGetLastError();            \
            return SMTM_ERR_CUDA;                \
        }                                        \
    } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <class T>
cudaError_t dev_alloc(T** p, size_t count) {
    return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T));
}

void drop_profile(smtm_cache* c) {
    if (c->prof_events) {
        for (cudaEvent_t e : *c->prof_events) cudaEventDestroy(e);
        delete c->prof_events;
        delete c->prof_layer;
        c->prof_events = nullptr;
        c->prof_layer = nullptr;
        cudaFree(c->d_prof_clock);
        c->d_prof_clock = nullptr;
        c->prof_step = nullptr;
        c->prof_steps_used = 0;
    }
    c->prof_used = 0;
}

void free_all(smtm_cache* c) {
    drop_profile(c);
    for (int l = 0; l < SMTM_MAX_LAYERS; ++l) {
        cudaFree(c->d_centers[l]);
        cudaFree(c->d_cnorm[l]);
        cudaFree(c->d_m[l]);
        cudaFree(c->d_stage[l]);
        cudaFree(c->d_cen_split[l]);
        cudaFree(c->hb.d_sv[l]);
    }
    cudaFree(c->d_ft);
    cudaFree(c->d_ts);
    cudaFree(c->d_members);
    cudaFree(c->d_k);
    cudaFree(c->d_counters);
    cudaFree(c->d_status);
    cudaFree(c->d_plan);
    cudaFree(c->d_warm_sv);
    cudaFree(c->d_dense);
    cudaFree(c->d_tags);
    cudaFree(c->d_epoch);
    if (c->pool_stream) cudaStreamDestroy(c->pool_stream);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_pool) cudaEventDestroy(c->ev_pool);
    for (cudaEvent_t e : c->ev_mark)
        if (e) cudaEventDestroy(e);
    cudaFree(c->d_jobs);
    cudaFree(c->d_norm_part);
    cudaFree(c->d_ticket);
    cudaFree(c->hb.d_sa);
    cudaFree(c->hb.d_done);
    cudaFree(c->hb.d_exit_layer);
    cudaFree(c->hb.d_pred);
    cudaFree(c->d_stream_id);
    cudaFree(c->d_fallback);
    cudaFreeHost(c->h_flags);
    delete c;
}

smtm_status_t check_fmap(const smtm_cache* c, int32_t layer, const smtm_fmap_t* f) {
    if (!c || !f) return SMTM_ERR_INVALID_ARG;
    if (layer < 0 || layer >= c->L) return SMTM_ERR_INVALID_ARG;
    if (f->dtype < SMTM_F32 || f->dtype > SMTM_BF16 || f->layout < SMTM_NCHW || f->layout > SMTM_NHWC)
        return SMTM_ERR_DTYPE;
    if (f->B < 1 || f->B > c->max_batch || f->H < 1 || f->W < 1) return SMTM_ERR_SHAPE;
    if (f->C != c->dims[layer]) return SMTM_ERR_SHAPE;
    if ((long long)f->H * f->W > (1 << 24)) return SMTM_ERR_SHAPE;
    return SMTM_OK;
}

smtm_status_t check_batch(const smtm_cache* c, const smtm_batch_t* b) {
    if (!b) return SMTM_ERR_INVALID_ARG;
    if (b->B < 1 || b->B > c->max_batch) return SMTM_ERR_SHAPE;
    if (!b->d_sa || !b->d_done || !b->d_exit_layer || !b->d_pred) return SMTM_ERR_INVALID_ARG;
    return SMTM_OK;
}

// The tensor-core scorer reads the centres as bf16 heads and tails.  That copy is made here whenever the centres of
// a layer are set as a whole (creation, import); Eq. 7's kernel keeps it in step with every centre it moves.
// Layers the scorer does not serve (vectors that are not a multiple of eight long) have none.
bool has_centre_split(const smtm_cache* c, int l) { return c->d_cen_split[l] != nullptr && c->dims[l] % 8 == 0; }

cudaError_t split_centres(smtm_cache* c, int l, cudaStream_t st) {
    if (!has_centre_split(c, l)) return cudaSuccess;
    return launch_centers_split(c->d_centers[l], c->n, c->dims[l], c->d_cen_split[l], st, &c->launches);
}

EncodeArgs encode_args(const smtm_cache* c, const smtm_fmap_t* f, const uint8_t* skip, float* sv) {
    EncodeArgs e{};
    e.x = f->d_data;
    e.dtype = f->dtype;
    e.layout = f->layout;
    e.B = f->B;
    e.C = f->C;
    e.H = f->H;
    e.W = f->W;
    e.skip = skip;
    e.sv = sv;
    e.status = c->d_status;
    return e;
}

// CTA size of the scoring kernel and ring depth of the pooling kernel on the pipelined route: small enough that
// the CTAs of the latency-bound kernels of a step (scoring, sparse pooling, update) fit on an SM beside a CTA of
// the next step's pooling kernel.
constexpr int kPipelinedScoreThreads = 128;
constexpr int kPipelinedRingStages = 5;
constexpr int kPipelinedRingConsumers = 3;
// Copies the pooling kernel keeps outstanding per SM on this route (148 x 2 x 25 KB = 7.4 MB in flight; more did not
// make it faster beside the latency-bound kernels, and every access those make to memory queues behind them).
constexpr int kPipelinedInFlight = 2;
// The same route with the tensor-core scorer: its ring of two stages (129 KB) and a pooling ring of three (77 KB)
// share an SM.
constexpr int kPipelinedDenseRingStages = 3;
constexpr int kPipelinedDenseTcStages = 2;

// The capture the stream is in (0 = none).
cudaError_t capture_of(cudaStream_t st, unsigned long long* id) {
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    unsigned long long cid = 0;
    const cudaError_t e = cudaStreamGetCaptureInfo(st, &status, &cid);
    *id = (e == cudaSuccess && status == cudaStreamCaptureStatusActive) ? cid : 0ull;
    return e;
}

// First lookup of a batch on the pipelined route.  Pooling reads only the maps (complete, by the caller's promise)
// and writes only this batch's SV stash, so it does not have to wait for the step before: it runs on the cache's
// pool stream, ordered after the previous pooling (stream order) and after everything the caller's stream held at
// the first lookup before this one (by then the batch before last, whose stash this batch may share, is done
// with: batches alternate).  Scoring waits for it and for the caller's stream.  Inside a stream capture the pool
// stream joins the capture through these events; a mark recorded outside the capture under way is not waited for
// (the launch of the graph orders the graph after it), and a pool stream that is not part of the capture yet
// is forked from the caller's stream where it stands.
//
// With a large fast memory (dense) the scoring is the tensor-core kernel and the decision kernel after it.  The
// tensor-core kernel gets a ring of two stages and the pooling kernel one of three, so that a CTA of each fits on
// an SM: the next batch's pooling starts as soon as this batch's is done and runs beside all of this batch's
// kernels.  The decision kernel is launched in stream order (see launch_ordered).  The vectors' bf16 split
// alternates between two buffers like the batches do.
smtm_status_t pooled_first_lookup(smtm_cache* c, const EncodeArgs& e, const LookupArgs& a, cudaStream_t st,
                                  const cudaEvent_t* timing, bool profiled_step, bool dense) {
    unsigned long long cap = 0, pool_cap = 0;
    SMTM_CUDA(capture_of(st, &cap));
    SMTM_CUDA(capture_of(c->pool_stream, &pool_cap));
    const int cur = c->mark_next, prev = cur ^ 1;
    const bool wait_prev = c->mark_valid[prev] && c->mark_capture[prev] == cap;
    if (wait_prev) SMTM_CUDA(cudaStreamWaitEvent(c->pool_stream, c->ev_mark[prev], 0));
    if (!wait_prev || (cap != 0 && pool_cap != cap)) {
        // no usable mark (the first call, a capture that has just begun): the pooling follows all of the caller's stream
        SMTM_CUDA(cudaEventRecord(c->ev_fork, st));
        SMTM_CUDA(cudaStreamWaitEvent(c->pool_stream, c->ev_fork, 0));
    }
    SMTM_CUDA(cudaEventRecord(c->ev_mark[cur], st));
    c->mark_capture[cur] = cap;
    c->mark_valid[cur] = true;
    c->mark_next = prev;
    EncodeArgs ep = e;
    ep.skip = nullptr;  // the batch starts here: every frame is in
    ep.ring_stages = dense ? kPipelinedDenseRingStages : kPipelinedRingStages;
    ep.ring_consumers = kPipelinedRingConsumers;
    ep.ring_in_flight = kPipelinedInFlight;
    if (profiled_step && a.layer == 0 && ep.clock)  // the caller's stream clears the step's other stamps at a time of its own
        SMTM_CUDA(cudaMemsetAsync(ep.clock, 0, 2 * sizeof(unsigned long long), c->pool_stream));
    bool sv_split = false;
    if (dense) {
        // this batch's buffer, for its later layers too (the next batch's pooling writes the other one meanwhile)
        c->split_which = cur;
        dense_sv_split(c->d_dense, c->max_batch, c->d_max, cur, &ep.sv_hi, &ep.sv_lo);
    }
    if (timing) SMTM_CUDA(record_timing(timing[0], c->pool_stream));
    SMTM_CUDA(launch_encode(ep, c->sm_count, c->pool_stream, &c->launches, dense ? &sv_split : nullptr));
    if (timing) SMTM_CUDA(record_timing(timing[1], c->pool_stream));
    SMTM_CUDA(cudaEventRecord(c->ev_pool, c->pool_stream));
    if (!dense) {
        SMTM_CUDA(cudaStreamWaitEvent(st, c->ev_pool, 0));
        SMTM_CUDA(launch_score_exit(a, st, &c->launches, kPipelinedScoreThreads));
        return SMTM_OK;
    }
    float *dots = nullptr, *dots2 = nullptr;
    SMTM_CUDA(launch_dense_dots(a.sv, nullptr, a.B, a.centers, a.n, a.D, c->d_dense, c->max_batch, c->d_max, cur, sv_split,
                                c->ev_pool, c->d_cen_split[a.layer], &dots, &dots2, c->d_status,
                                a.clock ? a.clock + 2 * SMTM_PROF_SCORE_TC : nullptr, kPipelinedDenseTcStages, st, &c->launches));
    SMTM_CUDA(launch_finish_dense(a, dots, dots2, true, st, &c->launches));
    return SMTM_OK;
}

smtm_status_t lookup_impl(smtm_cache* c, int32_t layer, const smtm_fmap_t* f, const smtm_batch_t* b,
                          cudaStream_t st, bool begin, bool allow_early = true) {
    LookupArgs a{};
    a.fresh = begin ? 1 : 0;
    a.layer = layer;
    a.L = c->L;
    a.B = f->B;
    a.D = f->C;
    a.n = c->n;
    a.k_max = c->k_max;
    a.tau = c->tau[layer];
    a.sv = b->d_sv[layer];
    a.centers = c->d_centers[layer];
    a.cnorm = c->d_cnorm[layer];
    a.stream_id = b->d_stream_id;
    a.members = c->d_members;
    a.k = c->d_k;
    a.sa = b->d_sa;
    a.done = b->d_done;
    a.exit_layer = b->d_exit_layer;
    a.pred = b->d_pred;
    a.ac = b->d_ac;
    a.sep = b->d_sep;
    a.top = b->d_top;
    a.counters = c->d_counters;
    a.S = c->S;
    a.status = c->d_status;
    EncodeArgs e = encode_args(c, f, b->d_done, b->d_sv[layer]);
    bool fused = false;
    const cudaEvent_t* timing = nullptr;
    bool profiled_step_begins = false;
    // The pipelined route: a cache whose caller keeps the maps resident and alternates its carries
    // (SMTM_FLAG_MAPS_READY), small fast memories, shapes the streaming kernels serve.
    const bool pipelined = c->maps_ready && allow_early && c->k_max <= kFusedMaxK && launch_pool_sparse_supported(e);
    // ... or, for NHWC maps, the first lookup of a batch alone (later layers keep their one kernel per layer)
    const bool pipelined_nhwc = c->maps_ready && allow_early && begin && c->k_max <= kFusedMaxK &&
                                launch_encode_nhwc_vector_supported(e);
    // ... or, for a large fast memory scored on the tensor cores, the first lookup of a batch alone
    const bool dense = c->d_dense && dense_scoring_supported(a.D, a.n);
    const bool pipelined_dense = c->maps_ready && allow_early && begin && dense && launch_encode_ring_supported(e);
    if (c->prof_events && c->prof_seq % c->L == 0) {  // a step begins: does it get a slot for the device-clock stamps?
        c->prof_step = nullptr;
        if ((c->prof_seq / c->L) % c->prof_every == 0 && c->prof_steps_used < c->prof_steps_cap) {
            c->prof_step = c->d_prof_clock + c->prof_steps_used++ * size_t(2 * SMTM_PROF_KERNELS);
            // (the first two words are the stamps of the first layer's streaming kernel: on the pipelined route that
            // kernel runs on the pool stream, which clears them itself)
            const size_t skip = ((pipelined || pipelined_dense || pipelined_nhwc) && begin && layer == 0) ? 2 : 0;
            SMTM_CUDA(cudaMemsetAsync(c->prof_step + skip, 0, (2 * SMTM_PROF_KERNELS - skip) * sizeof(unsigned long long), st));
            profiled_step_begins = true;
        }
    }
    a.clock = c->prof_events ? c->prof_step : nullptr;
    if (c->prof_events && (c->prof_seq++ / c->L) % c->prof_every == 0 &&
        2 * (c->prof_used + 1) <= c->prof_events->size()) {
        timing = c->prof_events->data() + 2 * c->prof_used;
        (*c->prof_layer)[c->prof_used++] = layer;
    }
    if (pipelined) {
        ++c->routes[SMTM_ROUTE_PIPELINED];
        e.clock = a.clock ? a.clock + 2 * layer : nullptr;  // the pooling kernel is this layer's streaming kernel
        if (begin) return pooled_first_lookup(c, e, a, st, timing, profiled_step_begins, false);
        // a later layer: the frames still in are few; clusters of small CTAs look them up whole, or, for shapes
        // those do not serve, small CTAs pool them and small CTAs score them
        if (timing) SMTM_CUDA(record_timing(timing[0], st));
        const bool whole = launch_lookup_sparse_supported(e, a);
        if (whole)
            SMTM_CUDA(launch_lookup_sparse(e, a, c->sm_count, st, &c->launches));
        else
            SMTM_CUDA(launch_pool_sparse(e, c->sm_count, st, &c->launches));
        if (timing) SMTM_CUDA(record_timing(timing[1], st));
        if (!whole) SMTM_CUDA(launch_score_exit(a, st, &c->launches, kPipelinedScoreThreads));
        return SMTM_OK;
    }
    if (pipelined_nhwc) {
        ++c->routes[SMTM_ROUTE_PIPELINED];
        e.clock = a.clock ? a.clock + 2 * layer : nullptr;
        return pooled_first_lookup(c, e, a, st, timing, profiled_step_begins, false);
    }
    if (pipelined_dense) {
        ++c->routes[SMTM_ROUTE_PIPELINED_DENSE];
        e.clock = a.clock ? a.clock + 2 * layer : nullptr;
        return pooled_first_lookup(c, e, a, st, timing, profiled_step_begins, true);
    }
    SMTM_CUDA(launch_lookup_fused(e, a, c->sm_count, &c->fused_caps, st, &c->launches, &fused, timing));
    if (fused) {
        ++c->routes[SMTM_ROUTE_FUSED];
        return SMTM_OK;
    }
    ++c->routes[dense ? SMTM_ROUTE_DENSE : SMTM_ROUTE_PLAIN];
    EncodeArgs e2 = e;
    e2.clock = a.clock ? a.clock + 2 * layer : nullptr;  // the pooling kernel is this layer's streaming kernel
    if (a.fresh) e2.skip = nullptr;  // a batch that starts here: every frame is in, whatever the flags hold
    if (dense) dense_sv_split(c->d_dense, c->max_batch, c->d_max, c->split_which, &e2.sv_hi, &e2.sv_lo);
    bool sv_split = false;
    if (timing) SMTM_CUDA(record_timing(timing[0], st));
    SMTM_CUDA(launch_encode(e2, c->sm_count, st, &c->launches, &sv_split));
    if (timing) SMTM_CUDA(record_timing(timing[1], st));
    if (dense) {
        float *dots = nullptr, *dots2 = nullptr;
        SMTM_CUDA(launch_dense_dots(a.sv, a.fresh ? nullptr : a.done, a.B, a.centers, a.n, a.D, c->d_dense, c->max_batch, c->d_max,
                                    c->split_which, sv_split, nullptr, c->d_cen_split[layer], &dots, &dots2, c->d_status,
                                    a.clock ? a.clock + 2 * SMTM_PROF_SCORE_TC : nullptr, 0, st, &c->launches));
        SMTM_CUDA(launch_finish_dense(a, dots, dots2, false, st, &c->launches));
        return SMTM_OK;
    }
    SMTM_CUDA(launch_score_exit(a, st, &c->launches));
    return SMTM_OK;
}

ResizeArgs resize_args(const smtm_cache* c) {
    ResizeArgs a{};
    a.S = c->S;
    a.n = c->n;
    a.W = c->W;
    a.k_min = c->k_min;
    a.k_max = c->k_max;
    a.cl_num = c->cl_num;
    a.cl_den = c->cl_den;
    a.forgetting = c->forgetting ? 1 : 0;
    a.ft = c->d_ft;
    a.ts = c->d_ts;
    a.members = c->d_members;
    a.k = c->d_k;
    a.clock = c->prof_events ? c->prof_step : nullptr;
    return a;
}

smtm_status_t update_impl(smtm_cache* c, const smtm_batch_t* b, const int32_t* d_fallback, bool with_resize,
                          cudaStream_t st) {
    UpdateArgs a{};
    a.B = b->B;
    a.S = c->S;
    a.n = c->n;
    a.L = c->L;
    a.forget_W = c->forgetting ? c->W : 0;
    a.warm_layer = -1;
    a.plan.frame_code = c->d_plan;
    a.plan.class_tag = c->d_tags;
    a.plan.job_count = c->d_jobs;
    a.plan.jobs = c->d_jobs + 4;
    a.plan.items = c->d_jobs + 4 + size_t(c->L) * c->n;
    a.norm_part = c->d_norm_part;
    a.ticket = c->d_ticket;
    a.plan.epoch = c->d_epoch;
    a.stream_id = b->d_stream_id;
    a.done = b->d_done;
    a.exit_layer = b->d_exit_layer;
    a.pred = b->d_pred;
    a.fallback = d_fallback;
    a.clock = c->prof_events ? c->prof_step : nullptr;
    a.status = c->d_status;
    a.ft = c->d_ft;
    a.ts = c->d_ts;
    for (int l = 0; l < c->L; ++l) {
        a.dims[l] = c->dims[l];
        a.sv[l] = b->d_sv[l];
        a.centers[l] = c->d_centers[l];
        a.cnorm[l] = c->d_cnorm[l];
        a.m[l] = c->d_m[l];
        a.cen_split[l] = has_centre_split(c, l) ? static_cast<__nv_bfloat16*>(c->d_cen_split[l]) : nullptr;
    }
    const ResizeArgs rz = resize_args(c);
    SMTM_CUDA(launch_update(a, with_resize ? &rz : nullptr, c->sm_count, st, &c->launches));
    return SMTM_OK;
}

smtm_status_t resize_impl(smtm_cache* c, cudaStream_t st) {
    SMTM_CUDA(launch_resize(resize_args(c), st, &c->launches));
    return SMTM_OK;
}

smtm_status_t check_lookup(const smtm_cache* c, int32_t layer, const smtm_fmap_t* f, const smtm_batch_t* b) {
    smtm_status_t s = check_fmap(c, layer, f);
    if (s != SMTM_OK) return s;
    if ((s = check_batch(c, b)) != SMTM_OK) return s;
    if (b->B != f->B) return SMTM_ERR_SHAPE;
    if (!f->d_data || !b->d_sv[layer]) return SMTM_ERR_INVALID_ARG;
    if (!aligned16(f->d_data) || !aligned16(b->d_sv[layer])) return SMTM_ERR_ALIGN;
    return SMTM_OK;
}

smtm_status_t check_update(const smtm_cache* c, const smtm_batch_t* b) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    const smtm_status_t s = check_batch(c, b);
    if (s != SMTM_OK) return s;
    for (int l = 0; l < c->L; ++l)
        if (!b->d_sv[l]) return SMTM_ERR_INVALID_ARG;
    return SMTM_OK;
}

}  // namespace

smtm_status_t smtm::lookup_begin_ordered(smtm_cache_t* c, int32_t layer, const smtm_fmap_t* f, const smtm_batch_t* b,
                                         void* stream) {
    const smtm_status_t s = check_lookup(c, layer, f, b);
    if (s != SMTM_OK) return s;
    return lookup_impl(c, layer, f, b, static_cast<cudaStream_t>(stream), true, false);
}

extern "C" {

smtm_status_t smtm_cache_create(const smtm_config_t* cfg, const float* const* h_centers,
                                const uint32_t* const* h_counts, const int32_t* h_init_members,
                                smtm_cache_t** out) {
    if (!cfg || !h_centers || !out || !cfg->dims || !cfg->tau) return SMTM_ERR_INVALID_ARG;
    if (cfg->n_classes < 1 || cfg->n_classes > SMTM_MAX_CLASSES) return SMTM_ERR_INVALID_ARG;
    if (cfg->n_layers < 1 || cfg->n_layers > SMTM_MAX_LAYERS) return SMTM_ERR_INVALID_ARG;
    if (cfg->n_streams < 1 || cfg->max_batch < 1 || (cfg->flags & ~uint32_t(SMTM_FLAG_FORGET_FT | SMTM_FLAG_MAPS_READY)) != 0)
        return SMTM_ERR_INVALID_ARG;
    if (cfg->k_min < 1 || cfg->k_min > cfg->k_init || cfg->k_init > cfg->k_max || cfg->k_max > cfg->n_classes)
        return SMTM_ERR_INVALID_ARG;
    if (cfg->window_W < 1 || cfg->cl_den < 1 || cfg->cl_num < 0 || cfg->cl_num > cfg->cl_den ||
        cfg->cl_den > 1024)
        return SMTM_ERR_INVALID_ARG;
    for (int l = 0; l < cfg->n_layers; ++l) {
        if (cfg->dims[l] < 1 || cfg->dims[l] > (1 << 20) || !h_centers[l]) return SMTM_ERR_INVALID_ARG;
        if (cfg->tau[l] != cfg->tau[l]) return SMTM_ERR_INVALID_ARG;  // NaN
    }
    const int n = cfg->n_classes, S = cfg->n_streams;
    if (h_init_members)
        for (long long i = 0; i < (long long)S * cfg->k_init; ++i)
            if (h_init_members[i] < 0 || h_init_members[i] >= n) return SMTM_ERR_INVALID_ARG;

    smtm_cache* c = new (std::nothrow) smtm_cache();
    if (!c) return SMTM_ERR_ALLOC;
    c->n = n;
    c->L = cfg->n_layers;
    c->S = S;
    c->k_init = cfg->k_init;
    c->k_min = cfg->k_min;
    c->k_max = cfg->k_max;
    c->W = cfg->window_W;
    c->cl_num = cfg->cl_num;
    c->cl_den = cfg->cl_den;
    c->max_batch = cfg->max_batch;
    c->forgetting = (cfg->flags & SMTM_FLAG_FORGET_FT) != 0;
    c->maps_ready = (cfg->flags & SMTM_FLAG_MAPS_READY) != 0;
    for (int l = 0; l < c->L; ++l) {
        c->dims[l] = cfg->dims[l];
        c->tau[l] = cfg->tau[l];
    }
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) {
        (void)cudaGetLastError();
        delete c;
        return SMTM_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    if (prop.major < 10) {  // the kernels are built for sm_100a only
        delete c;
        return SMTM_ERR_CUDA;
    }

    bool ok = encode_setup() == cudaSuccess && lookup_setup() == cudaSuccess && memory_setup() == cudaSuccess;
    if (ok && c->k_max > kFusedMaxK) ok = dense_setup() == cudaSuccess;
    for (int l = 0; ok && l < c->L; ++l) {
        const size_t nd = size_t(n) * c->dims[l];
        ok = ok && dev_alloc(&c->d_centers[l], nd) == cudaSuccess;
        ok = ok && dev_alloc(&c->d_cnorm[l], n) == cudaSuccess;
        ok = ok && dev_alloc(&c->d_m[l], n) == cudaSuccess;
    }
    ok = ok && dev_alloc(&c->d_ft, size_t(S) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_ts, size_t(S) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_members, size_t(S) * c->k_max) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_k, S) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_counters, SMTM_CTR_COUNT) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_status, 1) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_plan, size_t(c->max_batch)) == cudaSuccess;
    for (int l = 0; l < c->L; ++l) c->d_max = c->dims[l] > c->d_max ? c->dims[l] : c->d_max;
    c->d_max = (c->d_max + 7) / 8 * 8;  // keeps the bf16 operand arrays of the tensor-core scorer 16-byte aligned
    if (ok && c->k_max > kFusedMaxK) {
        ok = cudaMalloc(&c->d_dense, dense_scratch_bytes(c->max_batch, n, c->d_max)) == cudaSuccess;
        for (int l = 0; ok && l < c->L; ++l)
            ok = cudaMalloc(&c->d_cen_split[l], dense_centers_split_bytes(n, c->dims[l])) == cudaSuccess;
    }
    ok = ok && dev_alloc(&c->d_tags, size_t(c->L) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_jobs, 4 + 17 * size_t(c->L) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_norm_part, 16 * size_t(c->L) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_ticket, size_t(c->L) * n) == cudaSuccess;
    ok = ok && dev_alloc(&c->d_epoch, 2) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->pool_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_pool, cudaEventDisableTiming) == cudaSuccess;
    for (cudaEvent_t& e : c->ev_mark) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        free_all(c);
        return SMTM_ERR_ALLOC;
    }

    std::vector<int32_t> members(size_t(S) * c->k_max, 0), ks(S, c->k_init);
    std::vector<uint32_t> ones(n, 1u);
    for (int s = 0; s < S; ++s)
        for (int j = 0; j < c->k_max; ++j) {
            int32_t v = j % n;
            if (j < c->k_init && h_init_members) v = h_init_members[size_t(s) * c->k_init + j];
            members[size_t(s) * c->k_max + j] = v;
        }
    cudaError_t e = cudaSuccess;
    for (int l = 0; e == cudaSuccess && l < c->L; ++l) {
        const size_t nd = size_t(n) * c->dims[l];
        e = cudaMemcpy(c->d_centers[l], h_centers[l], nd * sizeof(float), cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(c->d_m[l], (h_counts && h_counts[l]) ? h_counts[l] : ones.data(), n * sizeof(uint32_t),
                           cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = launch_center_norms(c->d_centers[l], n, c->dims[l], c->d_cnorm[l], 0, &c->launches);
        if (e == cudaSuccess) e = split_centres(c, l, 0);
    }
    if (e == cudaSuccess) e = cudaMemset(c->d_ft, 0, size_t(S) * n * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(c->d_ts, 0, size_t(S) * n * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(c->d_counters, 0, SMTM_CTR_COUNT * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->d_tags, 0, size_t(c->L) * n * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(c->d_jobs, 0, (4 + 17 * size_t(c->L) * n) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(c->d_epoch, 0, 2 * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(c->d_ticket, 0, size_t(c->L) * n * sizeof(int32_t));
    if (e == cudaSuccess)
        e = cudaMemcpy(c->d_members, members.data(), members.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(c->d_k, ks.data(), ks.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        free_all(c);
        return SMTM_ERR_CUDA;
    }
    *out = c;
    return SMTM_OK;
}

smtm_status_t smtm_cache_destroy(smtm_cache_t* c) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    (void)cudaDeviceSynchronize();
    free_all(c);
    return SMTM_OK;
}

smtm_status_t smtm_batch_reset(smtm_cache_t* c, const smtm_batch_t* b, void* stream) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    smtm_status_t s = check_batch(c, b);
    if (s != SMTM_OK) return s;
    SMTM_CUDA(launch_batch_reset(b->d_sa, b->d_done, b->d_exit_layer, b->d_pred, b->B, c->k_max,
                                 static_cast<cudaStream_t>(stream), &c->launches));
    return SMTM_OK;
}

smtm_status_t smtm_encode(smtm_cache_t* c, int32_t layer, const smtm_fmap_t* f, const uint8_t* d_skip, float* d_sv,
                          float* d_sv_norm2, void* stream) {
    smtm_status_t s = check_fmap(c, layer, f);
    if (s != SMTM_OK) return s;
    if (!f->d_data || !d_sv) return SMTM_ERR_INVALID_ARG;
    if (!aligned16(f->d_data) || !aligned16(d_sv)) return SMTM_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SMTM_CUDA(launch_encode(encode_args(c, f, d_skip, d_sv), c->sm_count, st, &c->launches));
    if (d_sv_norm2) SMTM_CUDA(launch_row_norm2(d_sv, d_skip, f->B, f->C, d_sv_norm2, st, &c->launches));
    return SMTM_OK;
}

smtm_status_t smtm_lookup_exit(smtm_cache_t* c, int32_t layer, const smtm_fmap_t* f, const smtm_batch_t* b,
                               void* stream) {
    const smtm_status_t s = check_lookup(c, layer, f, b);
    if (s != SMTM_OK) return s;
    return lookup_impl(c, layer, f, b, static_cast<cudaStream_t>(stream), false);
}

smtm_status_t smtm_lookup_exit_begin(smtm_cache_t* c, int32_t layer, const smtm_fmap_t* f, const smtm_batch_t* b,
                                     void* stream) {
    const smtm_status_t s = check_lookup(c, layer, f, b);
    if (s != SMTM_OK) return s;
    return lookup_impl(c, layer, f, b, static_cast<cudaStream_t>(stream), true);
}

smtm_status_t smtm_cache_update(smtm_cache_t* c, const smtm_batch_t* b, const int32_t* d_fallback_label,
                                void* stream) {
    const smtm_status_t s = check_update(c, b);
    if (s != SMTM_OK) return s;
    return update_impl(c, b, d_fallback_label, false, static_cast<cudaStream_t>(stream));
}

smtm_status_t smtm_cache_update_resize(smtm_cache_t* c, const smtm_batch_t* b, const int32_t* d_fallback_label,
                                       void* stream) {
    const smtm_status_t s = check_update(c, b);
    if (s != SMTM_OK) return s;
    return update_impl(c, b, d_fallback_label, true, static_cast<cudaStream_t>(stream));
}

smtm_status_t smtm_cache_warmup(smtm_cache_t* c, int32_t layer, const smtm_fmap_t* f, const int32_t* d_labels,
                                void* stream) {
    smtm_status_t s = check_fmap(c, layer, f);
    if (s != SMTM_OK) return s;
    if (!f->d_data || !d_labels) return SMTM_ERR_INVALID_ARG;
    if (!aligned16(f->d_data)) return SMTM_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!c->d_warm_sv && dev_alloc(&c->d_warm_sv, size_t(c->max_batch) * c->d_max) != cudaSuccess) {
        (void)cudaGetLastError();
        return SMTM_ERR_ALLOC;
    }
    SMTM_CUDA(launch_encode(encode_args(c, f, nullptr, c->d_warm_sv), c->sm_count, st, &c->launches));
    UpdateArgs a{};
    a.B = f->B;
    a.S = c->S;
    a.n = c->n;
    a.L = c->L;
    a.warm_layer = layer;
    a.plan.frame_code = c->d_plan;
    a.plan.class_tag = c->d_tags;
    a.plan.job_count = c->d_jobs;
    a.plan.jobs = c->d_jobs + 4;
    a.plan.items = c->d_jobs + 4 + size_t(c->L) * c->n;
    a.norm_part = c->d_norm_part;
    a.ticket = c->d_ticket;
    a.plan.epoch = c->d_epoch;
    a.fallback = d_labels;
    a.status = c->d_status;
    a.ft = c->d_ft;
    a.ts = c->d_ts;
    for (int l = 0; l < c->L; ++l) {
        a.dims[l] = c->dims[l];
        a.sv[l] = c->d_warm_sv;
        a.centers[l] = c->d_centers[l];
        a.cnorm[l] = c->d_cnorm[l];
        a.m[l] = c->d_m[l];
        a.cen_split[l] = has_centre_split(c, l) ? static_cast<__nv_bfloat16*>(c->d_cen_split[l]) : nullptr;
    }
    SMTM_CUDA(launch_update(a, nullptr, c->sm_count, st, &c->launches));
    return SMTM_OK;
}

smtm_status_t smtm_cache_resize(smtm_cache_t* c, void* stream) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    return resize_impl(c, static_cast<cudaStream_t>(stream));
}

smtm_status_t smtm_step_host(smtm_cache_t* c, const smtm_fmap_t* fmaps, const void* const* h_maps,
                             const int32_t* h_stream_id, const int32_t* h_fallback_label, int32_t do_resize,
                             uint8_t* h_done, int32_t* h_exit_layer, int32_t* h_pred, void* stream) {
    if (!c || !fmaps || !h_maps || !h_done || !h_exit_layer || !h_pred) return SMTM_ERR_INVALID_ARG;
    const int B = fmaps[0].B;
    for (int l = 0; l < c->L; ++l) {
        smtm_status_t s = check_fmap(c, l, &fmaps[l]);
        if (s != SMTM_OK) return s;
        if (fmaps[l].B != B) return SMTM_ERR_SHAPE;
        if (!h_maps[l]) return SMTM_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t mb = size_t(c->max_batch);
    if (!c->host_ready) {  // first use: allocate the device-side carry
        bool ok = dev_alloc(&c->hb.d_sa, mb * c->k_max) == cudaSuccess;
        ok = ok && dev_alloc(&c->hb.d_done, mb) == cudaSuccess;
        ok = ok && dev_alloc(&c->hb.d_exit_layer, mb) == cudaSuccess;
        ok = ok && dev_alloc(&c->hb.d_pred, mb) == cudaSuccess;
        ok = ok && dev_alloc(&c->d_stream_id, mb) == cudaSuccess;
        ok = ok && dev_alloc(&c->d_fallback, mb) == cudaSuccess;
        ok = ok && cudaMallocHost(reinterpret_cast<void**>(&c->h_flags), mb) == cudaSuccess;
        for (int l = 0; ok && l < c->L; ++l) ok = dev_alloc(&c->hb.d_sv[l], mb * c->dims[l]) == cudaSuccess;
        if (!ok) {
            (void)cudaGetLastError();
            return SMTM_ERR_ALLOC;
        }
        c->host_ready = true;
    }
    for (int l = 0; l < c->L; ++l) {
        const size_t need = size_t(B) * fmaps[l].C * fmaps[l].H * fmaps[l].W * (fmaps[l].dtype == SMTM_F32 ? 4 : 2);
        if (need > c->stage_bytes[l]) {
            (void)cudaStreamSynchronize(st);
            cudaFree(c->d_stage[l]);
            c->d_stage[l] = nullptr;
            c->stage_bytes[l] = 0;
            if (cudaMalloc(&c->d_stage[l], need) != cudaSuccess) {
                (void)cudaGetLastError();
                return SMTM_ERR_ALLOC;
            }
            c->stage_bytes[l] = need;
        }
    }
    smtm_batch_t b = c->hb;
    b.B = B;
    b.d_stream_id = nullptr;
    b.d_ac = nullptr;
    b.d_sep = nullptr;
    b.d_top = nullptr;
    if (h_stream_id) {
        SMTM_CUDA(cudaMemcpyAsync(c->d_stream_id, h_stream_id, size_t(B) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        b.d_stream_id = c->d_stream_id;
    }
    if (h_fallback_label)
        SMTM_CUDA(cudaMemcpyAsync(c->d_fallback, h_fallback_label, size_t(B) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    for (int l = 0; l < c->L; ++l) {
        smtm_fmap_t f = fmaps[l];
        const size_t frame_bytes = size_t(f.C) * f.H * f.W * (f.dtype == SMTM_F32 ? 4 : 2);
        if (l == 0) {
            SMTM_CUDA(cudaMemcpyAsync(c->d_stage[l], h_maps[l], size_t(B) * frame_bytes, cudaMemcpyHostToDevice, st));
        } else {
            // A frame that has exited needs nothing of the later layers: only the maps of the frames
            // that are still in cross the bus, one copy per run of consecutive frames.
            SMTM_CUDA(cudaMemcpyAsync(c->h_flags, b.d_done, size_t(B), cudaMemcpyDeviceToHost, st));
            SMTM_CUDA(cudaStreamSynchronize(st));
            for (int b0 = 0; b0 < B;) {
                if (c->h_flags[b0]) {
                    ++b0;
                    continue;
                }
                int b1 = b0 + 1;
                while (b1 < B && !c->h_flags[b1]) ++b1;
                SMTM_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(c->d_stage[l]) + size_t(b0) * frame_bytes,
                                          static_cast<const uint8_t*>(h_maps[l]) + size_t(b0) * frame_bytes,
                                          size_t(b1 - b0) * frame_bytes, cudaMemcpyHostToDevice, st));
                b0 = b1;
            }
        }
        f.d_data = c->d_stage[l];
        smtm_status_t s = lookup_impl(c, l, &f, &b, st, l == 0, false);  // one carry, staged maps: no early start
        if (s != SMTM_OK) return s;
    }
    smtm_status_t s = update_impl(c, &b, h_fallback_label ? c->d_fallback : nullptr, do_resize != 0, st);
    if (s != SMTM_OK) return s;
    SMTM_CUDA(cudaMemcpyAsync(h_done, b.d_done, size_t(B), cudaMemcpyDeviceToHost, st));
    SMTM_CUDA(cudaMemcpyAsync(h_exit_layer, b.d_exit_layer, size_t(B) * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SMTM_CUDA(cudaMemcpyAsync(h_pred, b.d_pred, size_t(B) * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SMTM_CUDA(cudaStreamSynchronize(st));
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_members(smtm_cache_t* c, int32_t* h_members, int32_t* h_k) {
    if (!c || !h_members || !h_k) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemcpy(h_members, c->d_members, size_t(c->S) * c->k_max * sizeof(int32_t), cudaMemcpyDeviceToHost));
    SMTM_CUDA(cudaMemcpy(h_k, c->d_k, size_t(c->S) * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_centers(smtm_cache_t* c, int32_t layer, float* h_centers, uint32_t* h_counts) {
    if (!c || !h_centers || layer < 0 || layer >= c->L) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemcpy(h_centers, c->d_centers[layer], size_t(c->n) * c->dims[layer] * sizeof(float),
                         cudaMemcpyDeviceToHost));
    if (h_counts)
        SMTM_CUDA(cudaMemcpy(h_counts, c->d_m[layer], size_t(c->n) * sizeof(uint32_t), cudaMemcpyDeviceToHost));
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_tables(smtm_cache_t* c, int32_t* h_ft, int32_t* h_ts) {
    if (!c || !h_ft || !h_ts) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemcpy(h_ft, c->d_ft, size_t(c->S) * c->n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    SMTM_CUDA(cudaMemcpy(h_ts, c->d_ts, size_t(c->S) * c->n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_counters(smtm_cache_t* c, int64_t* h_out) {
    if (!c || !h_out) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemcpy(h_out, c->d_counters, SMTM_CTR_COUNT * sizeof(int64_t), cudaMemcpyDeviceToHost));
    return SMTM_OK;
}

smtm_status_t smtm_cache_profile(smtm_cache_t* c, int32_t max_lookups, int32_t every) {
    if (!c || max_lookups < 0 || max_lookups > (1 << 20) || every == 0 || every == INT32_MIN) return SMTM_ERR_INVALID_ARG;
    const bool stamps_only = every < 0;  // no events: the chain of launches stays that of an unprofiled step
    if (stamps_only) every = -every;
    SMTM_CUDA(cudaDeviceSynchronize());
    drop_profile(c);
    c->prof_every = every;
    c->prof_seq = 0;
    if (max_lookups == 0) return SMTM_OK;
    c->prof_events = new (std::nothrow) std::vector<cudaEvent_t>();
    c->prof_layer = new (std::nothrow) std::vector<int>(size_t(max_lookups), 0);
    if (!c->prof_events || !c->prof_layer) return SMTM_ERR_ALLOC;
    c->prof_events->reserve(2 * size_t(max_lookups));
    c->prof_steps_cap = size_t(max_lookups) / size_t(c->L) + 1;
    const size_t clock_bytes = c->prof_steps_cap * 2 * SMTM_PROF_KERNELS * sizeof(unsigned long long);
    if (cudaMalloc(&c->d_prof_clock, clock_bytes) != cudaSuccess || cudaMemset(c->d_prof_clock, 0, clock_bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        drop_profile(c);
        return SMTM_ERR_ALLOC;
    }
    for (int i = 0; !stamps_only && i < 2 * max_lookups; ++i) {
        cudaEvent_t ev;
        if (cudaEventCreate(&ev) != cudaSuccess) {
            (void)cudaGetLastError();
            drop_profile(c);
            return SMTM_ERR_ALLOC;
        }
        c->prof_events->push_back(ev);
    }
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_profile(smtm_cache_t* c, int32_t layer, double* h_total_ms, int64_t* h_count) {
    if (!c || !h_total_ms || !h_count || layer < 0 || layer >= c->L) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    double total = 0.0;
    int64_t count = 0;
    for (size_t i = 0; c->prof_events && i < c->prof_used; ++i) {
        if ((*c->prof_layer)[i] != layer) continue;
        float ms = 0.f;
        SMTM_CUDA(cudaEventElapsedTime(&ms, (*c->prof_events)[2 * i], (*c->prof_events)[2 * i + 1]));
        total += ms;
        ++count;
    }
    *h_total_ms = total;
    *h_count = count;
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_profile_device(smtm_cache_t* c, double* h_total_ms, int64_t* h_count) {
    if (!c || !h_total_ms || !h_count) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    for (int k = 0; k < SMTM_PROF_KERNELS; ++k) {
        h_total_ms[k] = 0.0;
        h_count[k] = 0;
    }
    std::vector<unsigned long long> stamps(2 * SMTM_PROF_KERNELS);
    for (size_t i = 0; c->d_prof_clock && i < c->prof_steps_used; ++i) {
        SMTM_CUDA(cudaMemcpy(stamps.data(), c->d_prof_clock + i * stamps.size(), stamps.size() * sizeof(unsigned long long),
                             cudaMemcpyDeviceToHost));
        for (int k = 0; k < SMTM_PROF_KERNELS; ++k) {
            const unsigned long long begin = ~stamps[2 * k], end = stamps[2 * k + 1];
            if (end == 0 || end < begin) continue;  // the kernel did not run in this step
            h_total_ms[k] += double(end - begin) * 1e-6;
            ++h_count[k];
        }
    }
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_profile_timeline(smtm_cache_t* c, int64_t step, uint64_t* h_begin_ns, uint64_t* h_end_ns) {
    if (!c || !h_begin_ns || !h_end_ns) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    if (!c->d_prof_clock || step < 0 || size_t(step) >= c->prof_steps_used) return SMTM_ERR_INVALID_ARG;
    std::vector<unsigned long long> stamps(2 * SMTM_PROF_KERNELS);
    SMTM_CUDA(cudaMemcpy(stamps.data(), c->d_prof_clock + size_t(step) * stamps.size(),
                         stamps.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
    for (int k = 0; k < SMTM_PROF_KERNELS; ++k) {
        const unsigned long long begin = ~stamps[2 * k], end = stamps[2 * k + 1];  // the begin is kept as its complement
        const bool ran = end != 0 && end >= begin;
        h_begin_ns[k] = ran ? begin : 0;
        h_end_ns[k] = ran ? end : 0;
    }
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_routes(smtm_cache_t* c, int64_t* h_out) {
    if (!c || !h_out) return SMTM_ERR_INVALID_ARG;
    for (int r = 0; r < SMTM_ROUTE_COUNT; ++r) h_out[r] = c->routes[r];
    return SMTM_OK;
}

// ---- snapshot of the memory (export / import) ----------------------------------------------------------------

namespace {

struct BlobHeader {
    uint64_t magic;
    uint32_t version, n, L, S, k_max, forgetting;
    uint32_t dims[SMTM_MAX_LAYERS];
    uint64_t bytes;  // of the whole blob
};
constexpr uint64_t kBlobMagic = 0x4d454d2d4d544d53ull;  // "SMTM-MEM"

size_t blob_bytes(const smtm_cache* c) {
    size_t b = sizeof(BlobHeader);
    for (int l = 0; l < c->L; ++l)  // centres, their lengths, their counts
        b += size_t(c->n) * c->dims[l] * sizeof(float) + size_t(c->n) * sizeof(float) + size_t(c->n) * sizeof(uint32_t);
    b += 2 * size_t(c->S) * c->n * sizeof(int32_t);                        // FT, TS
    b += size_t(c->S) * c->k_max * sizeof(int32_t) + size_t(c->S) * sizeof(int32_t);  // members, k
    b += SMTM_CTR_COUNT * sizeof(uint64_t);
    return b;
}

// Walks the sections of a blob in their fixed order, copying each to (to_host) or from the device.
cudaError_t blob_copy(smtm_cache* c, unsigned char* p, bool to_host) {
    cudaError_t e = cudaSuccess;
    const auto section = [&](void* dev, size_t bytes) {
        if (e == cudaSuccess)
            e = to_host ? cudaMemcpy(p, dev, bytes, cudaMemcpyDeviceToHost) : cudaMemcpy(dev, p, bytes, cudaMemcpyHostToDevice);
        p += bytes;
    };
    for (int l = 0; l < c->L; ++l) {
        section(c->d_centers[l], size_t(c->n) * c->dims[l] * sizeof(float));
        section(c->d_cnorm[l], size_t(c->n) * sizeof(float));  // as the kernels left them: recomputing would round differently
        section(c->d_m[l], size_t(c->n) * sizeof(uint32_t));
    }
    section(c->d_ft, size_t(c->S) * c->n * sizeof(int32_t));
    section(c->d_ts, size_t(c->S) * c->n * sizeof(int32_t));
    section(c->d_members, size_t(c->S) * c->k_max * sizeof(int32_t));
    section(c->d_k, size_t(c->S) * sizeof(int32_t));
    section(c->d_counters, SMTM_CTR_COUNT * sizeof(uint64_t));
    return e;
}

}  // namespace

smtm_status_t smtm_cache_export_size(smtm_cache_t* c, uint64_t* h_bytes) {
    if (!c || !h_bytes) return SMTM_ERR_INVALID_ARG;
    *h_bytes = blob_bytes(c);
    return SMTM_OK;
}

smtm_status_t smtm_cache_export(smtm_cache_t* c, void* h_blob, uint64_t bytes) {
    if (!c || !h_blob) return SMTM_ERR_INVALID_ARG;
    if (bytes < blob_bytes(c)) return SMTM_ERR_SHAPE;
    SMTM_CUDA(cudaDeviceSynchronize());
    BlobHeader h{};
    h.magic = kBlobMagic;
    h.version = 1;
    h.n = uint32_t(c->n);
    h.L = uint32_t(c->L);
    h.S = uint32_t(c->S);
    h.k_max = uint32_t(c->k_max);
    h.forgetting = c->forgetting ? 1u : 0u;
    for (int l = 0; l < c->L; ++l) h.dims[l] = uint32_t(c->dims[l]);
    h.bytes = blob_bytes(c);
    unsigned char* p = static_cast<unsigned char*>(h_blob);
    memcpy(p, &h, sizeof(h));
    SMTM_CUDA(blob_copy(c, p + sizeof(h), true));
    return SMTM_OK;
}

smtm_status_t smtm_cache_import(smtm_cache_t* c, const void* h_blob, uint64_t bytes) {
    if (!c || !h_blob) return SMTM_ERR_INVALID_ARG;
    if (bytes < sizeof(BlobHeader)) return SMTM_ERR_SHAPE;
    BlobHeader h;
    memcpy(&h, h_blob, sizeof(h));
    if (h.magic != kBlobMagic || h.version != 1) return SMTM_ERR_INVALID_ARG;
    bool same = h.n == uint32_t(c->n) && h.L == uint32_t(c->L) && h.S == uint32_t(c->S) && h.k_max == uint32_t(c->k_max) &&
                h.forgetting == (c->forgetting ? 1u : 0u) && h.bytes == blob_bytes(c) && bytes >= h.bytes;
    for (int l = 0; same && l < c->L; ++l) same = h.dims[l] == uint32_t(c->dims[l]);
    if (!same) return SMTM_ERR_SHAPE;  // a snapshot of a memory of another shape
    // the sections are checked before anything is overwritten: sizes in range, members inside the memory
    const unsigned char* p = static_cast<const unsigned char*>(h_blob) + sizeof(h);
    for (int l = 0; l < c->L; ++l)
        p += size_t(c->n) * c->dims[l] * sizeof(float) + size_t(c->n) * sizeof(float) + size_t(c->n) * sizeof(uint32_t);
    p += 2 * size_t(c->S) * c->n * sizeof(int32_t);
    const int32_t* members = reinterpret_cast<const int32_t*>(p);
    const int32_t* ks = members + size_t(c->S) * c->k_max;
    for (size_t i = 0; i < size_t(c->S) * c->k_max; ++i)
        if (members[i] < 0 || members[i] >= c->n) return SMTM_ERR_INVALID_ARG;
    for (int s = 0; s < c->S; ++s)
        if (ks[s] < 1 || ks[s] > c->k_max) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(blob_copy(c, const_cast<unsigned char*>(static_cast<const unsigned char*>(h_blob)) + sizeof(h), false));
    for (int l = 0; l < c->L; ++l) SMTM_CUDA(split_centres(c, l, 0));  // the tensor-core scorer's bf16 copy of the centres
    SMTM_CUDA(cudaDeviceSynchronize());
    return SMTM_OK;
}

smtm_status_t smtm_cache_get_launches(smtm_cache_t* c, int64_t* h_out) {
    if (!c || !h_out) return SMTM_ERR_INVALID_ARG;
    *h_out = c->launches;
    return SMTM_OK;
}

smtm_status_t smtm_cache_status(smtm_cache_t* c) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    int v = 0;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemcpy(&v, c->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    return static_cast<smtm_status_t>(v);
}

smtm_status_t smtm_cache_clear_status(smtm_cache_t* c) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(cudaDeviceSynchronize());
    SMTM_CUDA(cudaMemset(c->d_status, 0, sizeof(int)));
    return SMTM_OK;
}

smtm_status_t smtm_cache_selftest_wait(smtm_cache_t* c, void* stream) {
    if (!c) return SMTM_ERR_INVALID_ARG;
    SMTM_CUDA(launch_wait_selftest(c->d_status, static_cast<cudaStream_t>(stream), &c->launches));
    return SMTM_OK;
}

const char* smtm_status_string(smtm_status_t s) {
    switch (s) {
        case SMTM_OK: return "ok";
        case SMTM_ERR_INVALID_ARG: return "invalid argument";
        case SMTM_ERR_SHAPE: return "shape mismatch";
        case SMTM_ERR_DTYPE: return "unknown dtype or layout";
        case SMTM_ERR_ALIGN: return "misaligned device buffer";
        case SMTM_ERR_ALLOC: return "allocation failed";
        case SMTM_ERR_CUDA: return "CUDA runtime error";
        case SMTM_ERR_STATE: return "invalid state";
        case SMTM_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
