// Host-side declarations shared by the translation units of the SMTM library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/smtm.h"

namespace smtm {

// Records a timing event on `st`; inside a stream capture it becomes an event-record node that
// is re-recorded at every replay of the graph.
inline cudaError_t record_timing(cudaEvent_t ev, cudaStream_t st) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return cudaGetLastError();
    return cudaEventRecordWithFlags(ev, st, cap == cudaStreamCaptureStatusActive ? cudaEventRecordExternal
                                                                                : cudaEventRecordDefault);
}

// Launches `kernel` so that it may start while the previous kernel of the stream is finishing
// (programmatic stream serialisation); the kernel itself waits with chain_wait() before it
// touches global memory.
template <bool kEarly = true, class... Params, class... Args>
cudaError_t launch_chained_cluster(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, int cluster_x,
                                   cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = kEarly ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;  // thread-block clusters of cluster_x consecutive CTAs
    attr[1].val.clusterDim.x = unsigned(cluster_x);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster_x > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <class... Params, class... Args>
cudaError_t launch_chained(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                           Args&&... args) {
    return launch_chained_cluster(kernel, grid, block, smem, 1, st, static_cast<Args&&>(args)...);
}

// The same launch without the early start.  A kernel launched with launch_chained becomes resident as soon as
// every CTA of the kernel before it has called chain_release(), and its CTAs then sit in chain_wait() holding
// their registers and shared memory.  On the pipelined route that is harmful for a kernel of many CTAs that
// follows a long one: while they wait they keep the CTAs of the next step's pooling kernel, which comes from the
// other stream at about the same time, off the SMs.  Such a kernel is launched in stream order instead; it costs
// it a microsecond.
template <class... Params, class... Args>
cudaError_t launch_ordered_cluster(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, int cluster_x,
                                   cudaStream_t st, Args&&... args) {
    return launch_chained_cluster<false>(kernel, grid, block, smem, cluster_x, st, static_cast<Args&&>(args)...);
}

template <class... Params, class... Args>
cudaError_t launch_ordered(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                           Args&&... args) {
    return launch_chained_cluster<false>(kernel, grid, block, smem, 1, st, static_cast<Args&&>(args)...);
}

// Number of exit layers and the fast-memory capacity of a cache.
void cache_shape(const smtm_cache_t* cache, int* n_layers, int* k_max);
// smtm_lookup_exit_begin without the early start that SMTM_FLAG_MAPS_READY allows: nothing is read or
// written before the stream's previous kernel is complete.  For callers whose carry is not private to
// the batch (the entry point that works in the library's fixed array).
smtm_status_t lookup_begin_ordered(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                                   const smtm_batch_t* batch, void* stream);

// Sets `kernel`'s limit on dynamic shared memory to everything the current device offers beside the
// kernel's static arrays.  The attribute belongs to the (kernel, device) pair and setting it again is
// harmless, so every cache sets it for its own device when it is created and no process-wide record of
// what has been set is kept.
template <class K>
cudaError_t allow_max_dynamic_smem(K kernel) {
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    cudaFuncAttributes fa{};
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, kernel);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - int(fa.sharedSizeBytes));
}

// ---- encode (Sec. 4.1) ------------------------------------------------------------------
struct EncodeArgs {
    const void* x;        // device, 16-byte aligned
    int dtype, layout;
    int B, C, H, W;
    const uint8_t* skip;  // device [B] or nullptr
    float* sv;            // device [B][C]
    void* sv_hi;          // optional: bf16 head and tail of sv for the tensor-core scorer (same indexing)
    void* sv_lo;
    int* status;          // device sticky status word
    unsigned long long* clock;  // nullptr, or two words for the kernel's device-clock stamps (see ClockScope)
    int ring_stages;      // 0 = the default depth of the streaming kernel's ring; fewer stages leave shared memory to
                          // the kernels that run beside it
    int ring_consumers;   // 0 = the default number of reducer warps; fewer leave registers to those kernels
    int ring_in_flight;   // 0 = the default number of copies kept outstanding per CTA
};
// Enqueues the pooling of every non-skipped frame.  *launches is incremented per kernel launched.
// *wrote_split (may be null) tells whether sv_hi / sv_lo were filled by the kernel that ran.
cudaError_t launch_encode(const EncodeArgs& a, int sm_count, cudaStream_t st, int64_t* launches,
                          bool* wrote_split = nullptr);
// Whether launch_encode serves the NHWC shape with the kernel that reads whole 16-byte pieces of a pixel's row.
bool launch_encode_nhwc_vector_supported(const EncodeArgs& a);
// Whether launch_encode serves the shape with the streaming ring, whose depth the ring_* fields set.
bool launch_encode_ring_supported(const EncodeArgs& a);
// Asks that SMs running `kernel` be configured with as much shared memory as they can have.  Kernels that
// are meant to share an SM with a streaming kernel (whose CTAs need most of it) must not leave the SM in a
// configuration with less: a CTA of the streaming kernel would wait until the SM has drained.
template <class K>
cudaError_t prefer_max_smem_carveout(K kernel) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, int(cudaSharedmemCarveoutMaxShared));
}

// Opt-in to large dynamic shared memory for the kernels that need it, on the current device (every
// cache does this for its own device at creation).
cudaError_t encode_setup();
// Pooling of the frames that are still in (skip[b] == 0) by small CTAs that fit beside a streaming kernel; NCHW
// shapes the streaming pipeline serves whose channels are at most 12.5 KB.  Same bits as launch_encode.
bool launch_pool_sparse_supported(const EncodeArgs& a);
cudaError_t launch_pool_sparse(const EncodeArgs& a, int sm_count, cudaStream_t st, int64_t* launches);
cudaError_t lookup_setup();
cudaError_t memory_setup();
cudaError_t dense_setup();
cudaError_t launch_row_norm2(const float* sv, const uint8_t* skip, int B, int D, float* out, cudaStream_t st,
                             int64_t* launches);

// ---- lookup (Sec. 4.2, Sec. 5) -------------------------------------------------------------
struct LookupArgs {
    int layer, L, B, D, n, k_max;
    int S;                    // streams of the cache: a frame whose stream id lies outside [0, S) is not looked up
    int* status;              // device sticky status word
    int fresh;                // the batch starts here: the carry is taken as SA = 0, nobody done, and is overwritten
    float tau;
    const float* sv;          // [B][D]
    const float* centers;     // [n][D]
    const float* cnorm;       // [n] lengths of the centres
    const int32_t* stream_id; // [B] or nullptr
    const int32_t* members;   // [S][k_max]
    const int32_t* k;         // [S]
    float* sa;                // [B][k_max]
    uint8_t* done;
    int32_t* exit_layer;
    int32_t* pred;
    float* ac;                // [B][L] or nullptr
    float* sep;               // [B][L] or nullptr
    int32_t* top;             // [B][2] or nullptr
    unsigned long long* counters;
    unsigned long long* clock;  // nullptr, or the profiled step's stamps [SMTM_PROF_KERNELS][2] (see ClockScope)
};
// threads: CTA size (a multiple of 32, at most 256; 0 = 256).  Smaller CTAs fit beside a streaming kernel.
cudaError_t launch_score_exit(const LookupArgs& a, cudaStream_t st, int64_t* launches, int threads = 0);
// Encode + score + exit in one kernel (NCHW shapes the streaming pipeline serves, fast
// memories of at most 64 entries).  *handled is false when the shape is not served, in which
// case nothing was launched.
constexpr int kFusedMaxK = 64;  // fast-memory capacity the fused path supports (two slots per lane)
// Lookup (pooling, scoring, decision) of the frames still in at a later layer by clusters of small CTAs that fit
// beside a streaming kernel: NCHW shapes the streaming pipeline cuts into at most 8 chunks per frame.
bool launch_lookup_sparse_supported(const EncodeArgs& e, const LookupArgs& a);
cudaError_t launch_lookup_sparse(const EncodeArgs& e, const LookupArgs& a, int sm_count, cudaStream_t st, int64_t* launches);
// What the device answered when asked how many clusters of 2, 4, 8 CTAs of each variant of the fused
// kernel it runs at once (0 = not asked yet, -1 = refused); kept per cache, i.e. per device.
struct FusedCaps {
    int clusters[16][9];
};
// timing: nullptr, or two events recorded on `st` right before and after the kernel.
cudaError_t launch_lookup_fused(const EncodeArgs& e, const LookupArgs& a, int sm_count, FusedCaps* caps, cudaStream_t st,
                                int64_t* launches, bool* handled, const cudaEvent_t* timing);
// ---- large fast memories: dot products against every class on the tensor cores ---------------
bool dense_scoring_supported(int D, int n);
size_t dense_scratch_bytes(int max_batch, int n, int d_max);
// DOT[b][c] = <sv[b], centers[c]> for b < B, c < n into scratch; *dots_out = the [B][n] result.
// The bf16 heads and tails of the semantic vectors sit at the start of scratch, in two sets (see
// dense_sv_split; `which` picks one); sv_split_done says whether they are already current; sv_ready: nullptr, or
// an event `st` has to wait for before it reads the vectors or their split (the pooling of the pipelined route).
// centers_split holds the same split of the centres ([n][D] heads, then [n][D] tails, D a multiple of 4): made by
// launch_centers_split whenever the centres are set as a whole, and kept in step by Eq. 7's kernel afterwards.
// ring_stages: 0 = the default depth of the operand ring; fewer stages leave shared memory to a kernel beside it.
void dense_sv_split(void* scratch, int max_batch, int d_max, int which, void** hi, void** lo);
cudaError_t launch_centers_split(const float* centers, int n, int D, void* centers_split, cudaStream_t st,
                                 int64_t* launches);
cudaError_t launch_dense_dots(const float* sv, const uint8_t* skip, int B, const float* centers, int n, int D,
                              void* scratch, int max_batch, int d_max, int which, bool sv_split_done,
                              cudaEvent_t sv_ready, void* centers_split, float** dots_out, float** dots2_out,
                              int* status, unsigned long long* clock, int ring_stages, cudaStream_t st,
                              int64_t* launches);
size_t dense_centers_split_bytes(int n, int D);
// Eq. 1 from the dot products, Eq. 3, top-2, Eq. 4 / Eq. 2 and the exit rule; dots: [B][n], and dots2
// (nullptr, or [B][n]: the second half of the vector length, added to the first).
// beside_pooling: the next batch's pooling kernel runs meanwhile (launched in stream order, see launch_ordered).
cudaError_t launch_finish_dense(const LookupArgs& a, const float* dots, const float* dots2, bool beside_pooling,
                                cudaStream_t st, int64_t* launches);
// One warp that waits, bounded, on a barrier nobody arrives on (the self-test of the time-out path).
cudaError_t launch_wait_selftest(int* status, cudaStream_t st, int64_t* launches);
cudaError_t launch_batch_reset(float* sa, uint8_t* done, int32_t* exit_layer, int32_t* pred, int B, int k_max,
                               cudaStream_t st, int64_t* launches);

// ---- memory maintenance (Sec. 6) -------------------------------------------------------------
cudaError_t launch_center_norms(const float* centers, int n, int D, float* cnorm, cudaStream_t st,
                                int64_t* launches);

// Scratch of an update (all device).
struct UpdatePlan {
    int32_t* frame_code;             // [max_batch] per frame: final label | stop layer (the paper's l) << 16, or -1 without a label
    unsigned long long* class_tag;   // [L][n] number of the last update call that touched (layer, class)
    int32_t* job_count;              // [0], [1]: (layer, class) pairs listed by this call ([number & 1]) and, zeroed, for the
                                     // next; [2]: this call's count, published by the plan kernel's last CTA; [3]: its items
    int32_t* jobs;                   // [L][n] the (layer << 16 | class) pairs Eq. 7 touches in this call, in no particular order
    int32_t* items;                  // [16][L][n] work items of the apply kernel: a pair, or one of the column blocks a heavy pair is cut into
    unsigned long long* epoch;       // [2] device: [0] number of update calls completed so far, [1] CTAs of the plan
                                     // kernel that are through (zero between calls).  The number lives on the
                                     // device so that a replayed CUDA graph counts on like eager calls do.
};

struct UpdateArgs {
    int B, S, n, L;
    unsigned long long* clock;  // nullptr, or the profiled step's stamps [SMTM_PROF_KERNELS][2] (see ClockScope)
    __nv_bfloat16* cen_split[SMTM_MAX_LAYERS];  // nullptr, or that split ([n][D] heads, then [n][D] tails): Eq. 7 keeps it in step with the centre it moves
    int forget_W;              // 0, or W when the frequency table itself forgets (SMTM_FLAG_FORGET_FT)
    int warm_layer;            // -1, or the one layer a warm-up batch folds into (no tables; done == nullptr)
    UpdatePlan plan;
    const int32_t* stream_id;  // [B] or nullptr
    const uint8_t* done;
    const int32_t* exit_layer;
    const int32_t* pred;
    const int32_t* fallback;   // [B] or nullptr
    int32_t* ft;               // [S][n]
    int32_t* ts;               // [S][n]
    int* status;               // device sticky status word
    int dims[SMTM_MAX_LAYERS];
    const float* sv[SMTM_MAX_LAYERS];
    float* centers[SMTM_MAX_LAYERS];
    float* cnorm[SMTM_MAX_LAYERS];
    uint32_t* m[SMTM_MAX_LAYERS];
    float* norm_part;          // [L][n][16] scratch: squared lengths of the column blocks of a centre that several CTAs fold
    int32_t* ticket;           // [L][n] scratch, zero between updates: how many of those CTAs are through
};


struct ResizeArgs {
    int S, n, W, k_min, k_max, cl_num, cl_den;
    int forgetting;    // the tables are the forgetting variant: the score is FT itself
    const int32_t* ft;
    const int32_t* ts;
    int32_t* members;  // [S][k_max]
    int32_t* k;        // [S]
    unsigned long long* clock;  // nullptr, or the profiled step's stamps [SMTM_PROF_KERNELS][2] (see ClockScope)
};
cudaError_t launch_resize(const ResizeArgs& a, cudaStream_t st, int64_t* launches);
// Tables and centres; with rz != nullptr also the Eq. 5 / Eq. 6 refresh of every stream that
// had a frame in the batch.  Two launches on `st`.
cudaError_t launch_update(const UpdateArgs& a, const ResizeArgs* rz, int sm_count, cudaStream_t st, int64_t* launches);

}  // namespace smtm
