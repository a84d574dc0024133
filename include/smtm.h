/*
 * smtm.h — C ABI of the SMTM semantic-memory hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the per-exit-layer procedure of
 * "Boosting Mobile CNN Inference through Semantic Memory" (arxiv 2112.02644):
 *
 *   Sec. 4.1        semantic vector = global average pooling of a feature map
 *   Sec. 4.2 Eq. 1  cosine similarity against the semantic centres in fast memory
 *   Sec. 4.2 Eq. 2  single-layer separability
 *   Sec. 5   Eq. 3  cross-layer cumulative similarity, weights 2^(l-1)
 *   Sec. 5   Eq. 4  accumulated confidence; exit when it exceeds the threshold
 *   Sec. 6.1        frequency table and time-stamp table
 *   Sec. 6.1 Eq. 5  replacement score, top-k members of the fast memory
 *   Sec. 6.2 Eq. 6  adaptive fast-memory size at a confidence level
 *   Sec. 6.3 Eq. 7  running-mean update of the semantic centres
 *
 * Conventions
 *   d_*  device pointer on the current CUDA device, owned by the caller.
 *   h_*  host pointer; read or written during the call, never retained.
 *   stream  a cudaStream_t passed as void* (NULL = the default stream).
 *   Calls that take a stream only enqueue work on it and return without
 *   synchronising; their results are valid once the caller has synchronised
 *   that stream.  Calls without a stream argument synchronise the device.
 *   `layer` is 0-based in this interface; the paper's l is layer + 1, so the
 *   weight of Eq. 3 is 2^layer.
 *   Every function returns an smtm_status_t.  Arguments are checked on the host
 *   before anything is launched; on an error nothing has been enqueued and no
 *   output argument has been written.  The library never aborts, throws, or
 *   traps on the device; a device-side bounded wait that gives up records
 *   SMTM_ERR_TIMEOUT in a sticky status word read by smtm_cache_status.
 *   A cache object is not thread-safe; distinct caches are independent.
 */
#ifndef SMTM_H
#define SMTM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct smtm_cache smtm_cache_t; /* opaque; owns centres, tables, fast memories, scratch */

typedef enum {
    SMTM_OK = 0,
    SMTM_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, value out of range */
    SMTM_ERR_SHAPE = 2,       /* feature-map shape does not match the cache's layer */
    SMTM_ERR_DTYPE = 3,       /* unknown dtype or layout code */
    SMTM_ERR_ALIGN = 4,       /* a device buffer is not aligned as documented */
    SMTM_ERR_ALLOC = 5,       /* device or host allocation failed */
    SMTM_ERR_CUDA = 6,        /* a CUDA runtime call failed */
    SMTM_ERR_STATE = 7,       /* call not valid in the cache's current state */
    SMTM_ERR_TIMEOUT = 8      /* a bounded device-side wait gave up */
} smtm_status_t;

enum { SMTM_F32 = 0, SMTM_F16 = 1, SMTM_BF16 = 2 }; /* feature-map element types */
enum { SMTM_NCHW = 0, SMTM_NHWC = 1 };              /* feature-map layouts */
enum { SMTM_MAX_LAYERS = 16 };
enum { SMTM_MAX_CLASSES = 8192 };

/* Counter slots returned by smtm_cache_get_counters. */
enum {
    SMTM_CTR_EXITS = 0,                           /* [0, MAX_LAYERS): exits taken at each layer */
    SMTM_CTR_NEAR = SMTM_MAX_LAYERS,              /* lookups with |AC - tau| <= 1e-4 */
    SMTM_CTR_LOOKUPS = SMTM_MAX_LAYERS + 1,       /* frames scored (not yet exited) over all layers */
    SMTM_CTR_COUNT = SMTM_MAX_LAYERS + 2
};

/* Config flag.  SMTM_FLAG_FORGET_FT: the variant the paper uses for rapidly changing scenes
 * (Sec. 7.1: the forgetting of Sec. 6.1 applied to the frequency table itself): the
 * 0.25-per-window decay of Eq. 5 is applied to the stored counts.
 * FT is then fixed point with 10 fractional bits (smtm_cache_get_tables returns it raw): an
 * appearance adds 1024, each further W consecutive unseen frames multiply it by 0.25 rounding
 * down, and Eq. 5's score is FT itself. */
enum { SMTM_FLAG_FORGET_FT = 1, SMTM_FLAG_MAPS_READY = 2 };
/* SMTM_FLAG_MAPS_READY is a promise of the caller that lets the library pipeline consecutive steps:
 * (1) the maps given to smtm_lookup_exit_begin are complete in memory when the call is enqueued, i.e.
 * they are not written by earlier work on the same stream; (2) consecutive batches use different
 * smtm_batch_t carries (two that alternate are enough).  Pooling (Sec. 4.1) reads only the maps and
 * does not depend on the memory, so the library then runs the pooling of a step's first layer on a
 * stream of its own, beside the later layers and the update of the step before (which are bound by
 * latency, not by bandwidth), and everything that depends on the memory (Eq. 1 onwards) after them on
 * the caller's stream.  The first lookup writes its batch's d_sv[layer] while the previous batch's
 * update may still read its own; it is ordered after all work the caller's stream held when the first
 * lookup before it was enqueued.  To the caller every result is ordered on its stream as usual, and
 * inside a stream capture the library's stream joins the capture (fork and join become part of the
 * graph).  Without the flag nothing is touched before the stream's previous work is complete. */

typedef struct {
    int32_t n_classes;      /* n: classes in global memory (Sec. 6), 1..SMTM_MAX_CLASSES */
    int32_t n_layers;       /* L: candidate exit layers (Sec. 4.2), 1..SMTM_MAX_LAYERS */
    const int32_t* dims;    /* h_ [L] C_l = length of the semantic vector at layer l (Sec. 4.1) */
    const float* tau;       /* h_ [L] exit thresholds; the paper's single tau = all equal (Sec. 5) */
    int32_t n_streams;      /* S: independent fast memories (1 = the paper's single video stream) */
    int32_t k_init;         /* initial fast-memory size, k_min <= k_init <= k_max */
    int32_t k_min, k_max;   /* bounds of the adaptive size, 1 <= k_min <= k_max <= n (Sec. 6.2) */
    int32_t window_W;       /* W of Eq. 5, >= 1 */
    int32_t cl_num, cl_den; /* confidence level of Eq. 6 as a fraction, e.g. 19/20 */
    int32_t max_batch;      /* largest B any call will pass; sizes the library's scratch */
    uint32_t flags;         /* 0 or an OR of SMTM_FLAG_FORGET_FT, SMTM_FLAG_MAPS_READY */
} smtm_config_t;

/* A batch of feature maps at one exit layer: dense, frame stride C*H*W elements,
 * d_data aligned to 16 bytes.  NCHW: [B][C][H][W];  NHWC: [B][H][W][C]. */
typedef struct {
    const void* d_data;
    int32_t dtype;  /* SMTM_F32 / SMTM_F16 / SMTM_BF16 */
    int32_t layout; /* SMTM_NCHW / SMTM_NHWC */
    int32_t B, C, H, W;
} smtm_fmap_t;

/* Per-batch carry across the exit layers of one inference; every array is a
 * caller-owned device array.  Before the first layer of a batch the caller
 * zeroes d_sa, d_done and d_exit_layer and sets d_pred to -1 (smtm_batch_reset, or
 * smtm_lookup_exit_begin for the first lookup).  The library keeps
 * d_done[b] == (d_exit_layer[b] != 0); a caller that edits one edits the other.
 * A layer is looked up at most once per batch. */
typedef struct {
    int32_t B;
    const int32_t* d_stream_id; /* [B] fast memory each frame looks up, in [0, S); NULL = all stream 0.  A frame
                                   whose id lies outside that range is scored against nothing (AC = 0, it stays
                                   in), takes no part in the update of tables or centres, and
                                   SMTM_ERR_INVALID_ARG is recorded in the sticky status word */
    float* d_sa;                /* [B][k_max] cumulative similarity per fast-memory slot (Eq. 3) */
    uint8_t* d_done;            /* [B] 1 once a frame has exited; later lookups skip it, reading none of its map */
    int32_t* d_exit_layer;      /* [B] 0 = not exited, else the paper's l in 1..L */
    int32_t* d_pred;            /* [B] class of SA_H at the exit layer */
    float* d_ac;                /* [B][L] accumulated confidence (Eq. 4) per evaluated layer; may be NULL */
    float* d_sep;               /* [B][L] separability (Eq. 2) per evaluated layer; may be NULL */
    int32_t* d_top;             /* [B][2] classes of SA_H, SA_SH at the last evaluated layer (-1 = none); may be NULL */
    float* d_sv[SMTM_MAX_LAYERS]; /* [l] -> [B][C_l] semantic vectors, kept for Eq. 7; 16-byte aligned */
} smtm_batch_t;

/* Creates a cache on the current device.  h_centers[l] -> [n][C_l] fp32 initial
 * semantic centres (the paper warms them up on training data, Sec. 5);
 * h_counts[l] -> [n] their update counts m (Eq. 7), NULL = all 1;
 * h_init_members -> [S][k_init] class ids initially in each fast memory,
 * NULL = 0..k_init-1 for every stream.  Frequency and time-stamp tables start
 * at zero (Sec. 6.1).  On success *out receives the cache. */
smtm_status_t smtm_cache_create(const smtm_config_t* cfg, const float* const* h_centers,
                                const uint32_t* const* h_counts, const int32_t* h_init_members,
                                smtm_cache_t** out);

/* Frees the cache and everything it owns (synchronises the device). */
smtm_status_t smtm_cache_destroy(smtm_cache_t* cache);

/* Prepares the carry for a new batch of frames: d_sa = 0, d_done = 0,
 * d_exit_layer = 0, d_pred = -1 (one kernel; d_ac/d_sep/d_top/d_sv untouched). */
smtm_status_t smtm_batch_reset(smtm_cache_t* cache, const smtm_batch_t* batch, void* stream);

/* Sec. 4.1.  d_sv[b][c] = mean over H x W of frame b, channel c, accumulated in
 * fp32, for every frame with d_skip[b] == 0 (d_skip NULL = all frames); rows of
 * skipped frames are not written and none of their map is read.
 * d_sv_norm2 (may be NULL) receives the squared length of each written row.
 * fmap->C must equal dims[layer]. */
smtm_status_t smtm_encode(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                          const uint8_t* d_skip, float* d_sv, float* d_sv_norm2, void* stream);

/* Sec. 5, one candidate exit layer, for every frame with d_done[b] == 0:
 * encode (as smtm_encode, into batch->d_sv[layer]); Eq. 1 against the k members
 * of the frame's fast memory; Eq. 3 into d_sa; top-1/top-2 (ties: lower class
 * id first; NaN ranks last); Eq. 4 and Eq. 2 into d_ac/d_sep[b][layer]; exit
 * when  SA_H > 0  and  SA_H - SA_SH > tau * max(SA_SH, 0)  (Eq. 4's AC > tau,
 * division-free, evaluated in fp32), which sets d_done, d_exit_layer = layer+1
 * and d_pred.  Fewer than two members never exit.  A zero-length vector has
 * similarity 0 to everything.  The fused route decides inside the streaming
 * kernel and tells the frames that are still in from d_exit_layer (0, or this
 * very layer when another CTA of the same launch has just decided the frame). */
smtm_status_t smtm_lookup_exit(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                               const smtm_batch_t* batch, void* stream);

/* Sec. 5: the first lookup of a batch, where every frame starts with SA = 0 and
 * nothing has exited.  Same result as smtm_batch_reset followed by
 * smtm_lookup_exit, without the pass over the carry: whatever d_sa, d_done,
 * d_exit_layer and d_pred held is ignored and overwritten for all B frames (all
 * k_max slots of d_sa).  `layer` is normally 0 but may be any layer at which the
 * caller starts looking up.  Same arguments and errors as smtm_lookup_exit. */
smtm_status_t smtm_lookup_exit_begin(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                                     const smtm_batch_t* batch, void* stream);

/* (No counterpart in the paper: a packaging of smtm_lookup_exit for callers that
 * must not allocate.)  Some callers cannot call cudaMalloc or anything that may:
 * a plug-in running inside another engine's enqueue step that is handed only its
 * inputs and outputs, a real-time thread that must not take the allocator's
 * locks, a process whose memory budget is frozen after start-up.  This entry
 * point does one self-contained lookup at `layer` (the cumulative similarity
 * starts from zero, so the decision is that layer's alone) and keeps its working
 * memory (semantic vectors [B][C], similarities [B][k_max], exit layers [B]) in a
 * fixed array of SMTM_STATIC_SCRATCH_BYTES compiled into the library; every GPU
 * that loads the library holds that array until the process exits.  It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *   fmap, d_stream_id   as in smtm_lookup_exit.
 *   d_exit [B]          1 where the frame exits at this layer, else 0.
 *   d_pred [B]          class of the best match where it exits, else -1.
 *   d_ac   [B][L]       column `layer` receives Eq. 4's value; may be NULL.
 * A batch whose working memory would exceed the array (roughly
 * 4 B (C + k_max + 1) bytes > SMTM_STATIC_SCRATCH_BYTES) is refused with
 * SMTM_ERR_SHAPE before anything is launched.  The first call on a device looks
 * up the array's device address; make that first call outside any stream
 * capture.  All calls on a device share the one array, which keeps the previous
 * call's contents (the call clears what it accumulates into): two calls whose
 * GPU work overlaps, e.g. on different streams, race on it.  Calls on one stream
 * are ordered: the entry never uses the early start of SMTM_FLAG_MAPS_READY, so
 * nothing of the array is touched before the stream's previous kernel is done. */
enum { SMTM_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024 };
smtm_status_t smtm_lookup_exit_static(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                                      const int32_t* d_stream_id, uint8_t* d_exit, int32_t* d_pred,
                                      float* d_ac, void* stream);

/* Sec. 6.1 tables and Eq. 7 centres for a finished batch.  The label of frame b
 * is d_pred[b] if it exited, else d_fallback_label[b] (the full network's
 * answer; -1 or a NULL array = no label); its stop layer is d_exit_layer[b] if it
 * exited, else L.  Per stream, frames are applied in ascending b: FT[label] + 1
 * (saturating at 2^20), TS[label] = 0, TS of every other class + 1.  For every
 * class j and layer l0 the frames with label j and stop layer >= l0 are folded
 * into the centre in ascending b:  SC = (SC m + sum SV) / (m + q), m += q
 * (summed as four interleaved partial sums added in a fixed order).
 * Tables and centres are kept by different CTAs of one kernel, after a small
 * kernel that plans the work; everything is enqueued on `stream`.  The call's
 * bookkeeping lives on the device: a captured update may be replayed any number
 * of times. */
smtm_status_t smtm_cache_update(smtm_cache_t* cache, const smtm_batch_t* batch,
                                const int32_t* d_fallback_label, void* stream);

/* smtm_cache_update followed by smtm_cache_resize restricted to the streams that
 * had at least one frame in the batch, in one pass (the tables of the other
 * streams did not change, so neither would their fast memories if they were
 * refreshed after their own last update). */
smtm_status_t smtm_cache_update_resize(smtm_cache_t* cache, const smtm_batch_t* batch,
                                       const int32_t* d_fallback_label, void* stream);

/* Centre warm-up (Sec. 5 / Sec. 6.3: a centre starts as the mean semantic vector of
 * its class over training frames): encodes a batch
 * of labelled frames at `layer` and folds each into the centre of its class
 * d_labels[b] (-1 = skip) by Eq. 7 in ascending frame order; a centre created with
 * count 0 thereby becomes the class mean.  Tables and fast memories are not touched.
 * The first call allocates [max_batch][max C_l] floats of scratch. */
smtm_status_t smtm_cache_warmup(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                                const int32_t* d_labels, void* stream);

/* Eq. 5 and Eq. 6 for every stream: Score_i = FT_i 0.25^floor(TS_i / W) (exact,
 * floor clamped at 12); classes ranked by (score descending, id ascending); the
 * new size is the smallest k in [k_min, k_max] whose k best scores sum to more
 * than cl_num/cl_den of all scores (k_max if none); the fast memory becomes the
 * first k of the ranking.  A stream whose scores are all zero is left as is. */
smtm_status_t smtm_cache_resize(smtm_cache_t* cache, void* stream);

/* One whole step from host memory: copies the L feature maps (h_maps[l], host,
 * dtype/layout/shape as in fmaps[l] whose d_data is ignored) to the device,
 * runs smtm_lookup_exit for layers 0..L-1, then smtm_cache_update_resize if
 * do_resize else smtm_cache_update, then copies the decisions back.  Synchronises
 * `stream` before returning.  h_stream_id / h_fallback_label may be NULL as in
 * the device calls; h_done [B], h_exit_layer [B], h_pred [B] receive the results.
 * B <= max_batch.  Pinned host buffers make the copies asynchronous.  After the
 * first layer only the maps of the frames that have not exited are copied (the
 * call reads the exit flags back between layers), so the bytes moved follow the
 * exits: sum over layers l of the frames still in at l times the frame's size. */
smtm_status_t smtm_step_host(smtm_cache_t* cache, const smtm_fmap_t* fmaps, const void* const* h_maps,
                             const int32_t* h_stream_id, const int32_t* h_fallback_label,
                             int32_t do_resize, uint8_t* h_done, int32_t* h_exit_layer,
                             int32_t* h_pred, void* stream);

/* State read-back (each synchronises the device). */
smtm_status_t smtm_cache_get_members(smtm_cache_t* cache, int32_t* h_members /*[S][k_max]*/,
                                     int32_t* h_k /*[S]*/);
smtm_status_t smtm_cache_get_centers(smtm_cache_t* cache, int32_t layer, float* h_centers /*[n][C_l]*/,
                                     uint32_t* h_counts /*[n], may be NULL*/);
smtm_status_t smtm_cache_get_tables(smtm_cache_t* cache, int32_t* h_ft /*[S][n]*/,
                                    int32_t* h_ts /*[S][n]*/);
smtm_status_t smtm_cache_get_counters(smtm_cache_t* cache, int64_t* h_out /*[SMTM_CTR_COUNT]*/);

/* Timing of the streaming kernel (the one that reads the feature maps) of
 * lookups: with max_lookups > 0, every `every`-th step's calls of
 * smtm_lookup_exit (a step = L consecutive calls) record a pair of CUDA events on
 * the caller's stream right around that kernel, up to max_lookups pairs; 0
 * switches it off and frees the events.  Inside a stream capture the events
 * become graph nodes that are re-recorded at every replay.  A negative `every`
 * profiles every |every|-th step with the device-clock stamps alone (below): no
 * event is recorded, so the step's launches follow one another as in an
 * unprofiled step, but for the memset that clears the stamps at its start.
 * smtm_cache_get_profile adds up the elapsed times of the recorded lookups of
 * one layer.  smtm_cache_get_profile_device reports, for the same steps, how long
 * each kernel of the step ran by the device's own clock, from the moment its
 * first CTA began (after its wait for the previous kernel) to the moment its
 * last CTA ended: h_total_ms[i] and h_count[i], i < SMTM_PROF_KERNELS, are the
 * sum over the profiled steps and their number, for the streaming kernel of
 * layer i (i < SMTM_MAX_LAYERS: the fused lookup kernel, or the pooling kernel
 * of the other routes), for the scoring kernel of layer i where pooling and
 * scoring are separate kernels (SMTM_PROF_SCORE + i), for the update (the plan
 * kernel SMTM_PROF_PLAN; the CTAs of the apply kernel that fold centres,
 * _CENTERS, and those that keep the tables, _TABLES; the refresh of the fast
 * memories where it is a kernel of its own, _REFRESH) and for the dense route
 * (the tensor-core scorer SMTM_PROF_SCORE_TC and the decision kernel after it,
 * _FINISH_DENSE; with several dense layers in a step, from the first one's
 * begin to the last one's end).  This
 * leaves out what the event nodes add around a kernel.  Only the most recent
 * run of each profiled step is kept.  smtm_cache_get_profile_timeline gives the
 * two stamps themselves for the step-th profiled step (counted from 0;
 * SMTM_ERR_INVALID_ARG beyond the steps recorded): h_begin_ns[i] and
 * h_end_ns[i], i < SMTM_PROF_KERNELS, in nanoseconds of the device's global
 * timer, both 0 for a kernel that did not run in that step, so that the gaps
 * between the kernels of a step can be read off.  All four synchronise the
 * device. */
enum {
    SMTM_PROF_SCORE = SMTM_MAX_LAYERS,  /* + layer: the scoring kernel of a layer whose pooling is a kernel of its own */
    SMTM_PROF_PLAN = 2 * SMTM_MAX_LAYERS, SMTM_PROF_CENTERS, SMTM_PROF_TABLES, SMTM_PROF_SCORE_TC,
    SMTM_PROF_FINISH_DENSE, SMTM_PROF_REFRESH,
    SMTM_PROF_KERNELS
};
smtm_status_t smtm_cache_profile(smtm_cache_t* cache, int32_t max_lookups, int32_t every);
smtm_status_t smtm_cache_get_profile(smtm_cache_t* cache, int32_t layer, double* h_total_ms, int64_t* h_count);
smtm_status_t smtm_cache_get_profile_device(smtm_cache_t* cache, double* h_total_ms /*[SMTM_PROF_KERNELS]*/,
                                            int64_t* h_count /*[SMTM_PROF_KERNELS]*/);
smtm_status_t smtm_cache_get_profile_timeline(smtm_cache_t* cache, int64_t step,
                                              uint64_t* h_begin_ns /*[SMTM_PROF_KERNELS]*/,
                                              uint64_t* h_end_ns /*[SMTM_PROF_KERNELS]*/);

/* Number of kernels the library has launched on behalf of this cache so far. */
smtm_status_t smtm_cache_get_launches(smtm_cache_t* cache, int64_t* h_out);

/* How many lookups (smtm_lookup_exit, _begin, _static and the lookups inside smtm_step_host) each
 * route has served so far.  The route is chosen from the shape and the cache's flags:
 *   SMTM_ROUTE_FUSED  pooling, Eq. 1, Eq. 3, Eq. 4 and the exit rule in one streaming kernel
 *                     (fast memories of at most 64 entries; NCHW shapes and NHWC shapes whose
 *                     pixel rows are multiples of 16 bytes);
 *   SMTM_ROUTE_DENSE  fast memories above 64 entries: pooling, then Eq. 1's dot products against
 *                     every class on the tensor cores, then a finishing kernel;
 *   SMTM_ROUTE_PLAIN  everything else: pooling, then a CUDA-core scoring kernel;
 *   SMTM_ROUTE_PIPELINED  on a cache created with SMTM_FLAG_MAPS_READY (small fast memories, NCHW shapes
 *                     the streaming kernels serve): the pooling of a step's first layer runs on a stream of
 *                     the cache's own, under the previous step's later layers and update; scoring follows
 *                     on the caller's stream; later layers are pooled and scored by small CTAs.  With
 *                     NHWC maps whose pixel rows are multiples of 16 bytes only the first lookup of a
 *                     batch takes this route (later layers: SMTM_ROUTE_FUSED);
 *   SMTM_ROUTE_PIPELINED_DENSE  the same for fast memories above 64 entries, first lookup of a batch only:
 *                     the pooling runs on the cache's stream beside the previous step's decision kernel and
 *                     update, the tensor-core kernel and the decision kernel follow on the caller's stream. */
enum {
    SMTM_ROUTE_FUSED = 0, SMTM_ROUTE_DENSE = 1, SMTM_ROUTE_PLAIN = 2, SMTM_ROUTE_PIPELINED = 3,
    SMTM_ROUTE_PIPELINED_DENSE = 4, SMTM_ROUTE_COUNT = 5
};
smtm_status_t smtm_cache_get_routes(smtm_cache_t* cache, int64_t* h_out /*[SMTM_ROUTE_COUNT]*/);

/* Snapshot of the memory of Sec. 6 (the paper keeps it for the life of the application; a host copy
 * lets a caller put a cache back into a known state, or carry it to another process): semantic centres
 * (with their lengths) and their update counts m (Eq. 7) of every layer, frequency and time-stamp tables (Sec. 6.1), the
 * fast memories and their sizes (Eq. 5, Eq. 6), and the counters.  smtm_cache_export_size gives the
 * size of the blob; smtm_cache_export writes it to h_blob (`bytes` = the room there, SMTM_ERR_SHAPE if
 * too small); smtm_cache_import reads one back into a cache of the same shape (n, L, C_l, S, k_max and
 * the forgetting flag must match: SMTM_ERR_SHAPE otherwise; a blob that is not a snapshot, or whose
 * fast memories name classes outside [0, n), SMTM_ERR_INVALID_ARG); the steps that follow give bit for
 * bit what they gave after the export.  Nothing is changed when an error is returned.  The blob's layout is
 * private to one build of the library.  All three synchronise the device; profiling records and the
 * sticky status word are not part of the snapshot. */
smtm_status_t smtm_cache_export_size(smtm_cache_t* cache, uint64_t* h_bytes);
smtm_status_t smtm_cache_export(smtm_cache_t* cache, void* h_blob, uint64_t bytes);
smtm_status_t smtm_cache_import(smtm_cache_t* cache, const void* h_blob, uint64_t bytes);

/* Reads the sticky device status word (synchronises the device): SMTM_OK or
 * the first device-side error recorded since creation (or since it was cleared). */
smtm_status_t smtm_cache_status(smtm_cache_t* cache);

/* Puts the status word back to SMTM_OK (synchronises the device). */
smtm_status_t smtm_cache_clear_status(smtm_cache_t* cache);

/* Self-test of the bounded waits: enqueues one small kernel that waits on a shared-memory barrier
 * nobody will ever arrive on, exactly as the streaming kernels wait for their copies.  The wait
 * gives up after its limit (about 2^31 clock cycles: a second or so), records SMTM_ERR_TIMEOUT in
 * the status word and the kernel returns normally: nothing traps, the context stays usable, and
 * smtm_cache_status reports the timeout.  Costs a second of device time; meant for tests. */
smtm_status_t smtm_cache_selftest_wait(smtm_cache_t* cache, void* stream);

const char* smtm_status_string(smtm_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* SMTM_H */
