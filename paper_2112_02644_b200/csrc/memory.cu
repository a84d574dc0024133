// Adaptive priming memory (Sec. 6): frequency / time-stamp tables, running-mean centres
// (Eq. 7), replacement score and top-k (Eq. 5), adaptive fast-memory size (Eq. 6).
//
// All floating-point reductions are segmented and atomics-free: one owner walks the batch in
// ascending frame index, so the result is the one a frame-by-frame replay would give and does
// not depend on scheduling.
//
// An update is two launches on the caller's stream.  The plan kernel writes every frame's final
// label and stop layer and lists the (layer, class) pairs Eq. 7 has to touch: up to 4096 frames and
// 65 536 pairs a single CTA elects the pairs in a shared-memory bitmap (k_update_plan_one); past
// that k_update_plan does it with many CTAs (the first frame to stamp a pair with the call's
// sequence number appends it; the number is kept on the device and moved on by the kernel
// itself, so that a replayed CUDA graph counts on exactly like eager calls).  The apply kernel is
// a grid of small CTAs (128 threads, a few KB of shared memory) with two kinds of work: the
// first B CTAs look after the tables, one per frame (the CTA of a stream's first frame in the
// batch applies all of the stream's frames to its tables and, when asked, refreshes its fast
// memory by Eq. 5 / Eq. 6; the others leave at once); the remaining CTAs take the listed pairs,
// one each, and fold the pair's frames into the centre (Eq. 7; a pair with many frames is several items, each
// a block of the vector's columns).  Small CTAs on purpose: there
// are hundreds of independent pieces of work, each a short chain of dependent trips to L2, so
// the kernel is as fast as the number of pieces in flight, and its CTAs fit beside the CTAs of a
// streaming kernel that holds most of an SM's shared memory.  Classes and streams the batch does
// not touch cost nothing.
#include <algorithm>

#include "common.cuh"
#include <cuda_bf16.h>

#include "internal.h"

namespace smtm {

namespace {

constexpr int kFtMax = 1 << 20;  // frequency counts saturate here so that Eq. 6's sums fit 64 bits
constexpr int kEMax = 12;        // floor(TS / W) is clamped here: 0.25^12 of a count is below one
constexpr int kFtFrac = 10;      // fractional bits of FT when the table itself forgets (SMTM_FLAG_FORGET_FT)

// One frame of a stream applied to one class's table entry (Sec. 6.1).  forget_W > 0 is the
// variant of Sec. 7.1: FT is fixed point, an appearance adds one unit, and every W-th
// consecutive unseen frame multiplies it by 0.25 (rounding down).
__device__ __forceinline__ void table_step(int& ft, int& ts, bool appears, int forget_W) {
    if (appears) {
        ft = forget_W ? int(min((long long)ft + (1 << kFtFrac), (long long)kFtMax << kFtFrac)) : min(ft + 1, kFtMax);
        ts = 0;
    } else if (ts < INT32_MAX) {
        ++ts;
        if (forget_W && ts % forget_W == 0) ft >>= 2;
    }
}

constexpr int kUpdThreads = 256;   // plan kernel (many-CTA form) and the stand-alone refresh
constexpr int kApplyThreads = 128; // CTAs of the apply kernel
constexpr int kTabPer = 8;         // consecutive frames a thread of a tables CTA looks at per trip to memory

// The label a finished frame ends up with: the prediction if it exited, else the fallback label
// (the full network's answer, -1 = none); a label outside the memory counts as no label.
__device__ __forceinline__ int final_label_of(const UpdateArgs& a, int b) {
    const int lab = (a.done && a.done[b] != 0) ? a.pred[b] : (a.fallback ? a.fallback[b] : -1);
    return lab >= a.n ? -1 : lab;
}

// ---- plan -----------------------------------------------------------------------------------
//
// What the plan leaves for the kernels that follow: per frame its final label and stop layer packed into one
// word (label | stop layer << 16, or -1 for a frame without a label); the list of
// pairs (layer, class) Eq. 7 touches (`jobs`, job_count[2] of them); and the list of work items of the apply
// kernel (`items`, job_count[3] of them): a pair whose frames are many is cut into several items, each a
// block of the vector's columns, so that no CTA folds more than a few rows per thread.
//   item = layer << 16 | class | block << 20 | log2(blocks) << 24      (class < 2^13, layer < 2^4, blocks <= 16)

constexpr int kItemBlocksMax = 16;

// Column blocks for a pair with `rows` frames at a layer whose vector has D entries: a CTA of the apply kernel
// should not load more than about eight 16-byte pieces per thread.  A power of two, at most 16, and no block
// narrower than 32 columns; vectors that are not a whole number of 16-byte pieces are never cut.
__device__ __forceinline__ int item_blocks(int rows, int D) {
    if (D & 3) return 1;
    const int D4 = D >> 2;
    const long long want = ((long long)rows * D4 + 8 * kApplyThreads - 1) / (8 * kApplyThreads);
    int nb = 1;
    while (nb < want && nb < kItemBlocksMax && (D4 / (2 * nb)) >= 8) nb *= 2;
    return nb;
}
__device__ __forceinline__ int ilog2_pow2(int v) { return 31 - __clz(v); }

// Label and stop layer of a finished frame: the prediction and exit layer if it exited,
// else the fallback label (the full network's answer, -1 = none) and L.
__global__ void __launch_bounds__(kUpdThreads) k_update_plan(const UpdateArgs a) {
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_PLAN : nullptr);
    const int b = blockIdx.x * kUpdThreads + threadIdx.x;
    const unsigned long long epoch = *a.plan.epoch + 1;  // this call's number; every CTA reads it before any is through
    if (b < a.B) {
        // every load unconditional, so that they make one trip to memory (no carry at all: a warm-up batch
        // of labelled frames)
        const int dn = a.done ? a.done[b] : 0, pr = a.done ? a.pred[b] : -1, el = a.done ? a.exit_layer[b] : 0;
        const int fb = a.fallback ? a.fallback[b] : -1;
        const int sid = a.stream_id ? a.stream_id[b] : 0;
        const bool ex = dn != 0;
        int lab = ex ? pr : fb;
        if (lab >= a.n) lab = -1;  // a label outside the memory counts as no label
        if (sid < 0 || sid >= a.S) {  // a stream outside the cache: the frame takes no part in the update
            lab = -1;
            set_status(a.status, kDevInvalidArg);
        }
        a.plan.frame_code[b] = lab < 0 ? -1 : (lab | ((ex ? el : a.L) << 16));
        if (lab >= 0) {
            // Eq. 7 touches the layers up to the stop layer: the first frame to stamp (layer, class)
            // with the call's number lists the pair as a job, and as a single item (this form of the plan
            // does not count the frames of a pair)
            const int l_lo = a.warm_layer >= 0 ? a.warm_layer : 0;
            const int l_hi = a.warm_layer >= 0 ? a.warm_layer + 1 : (ex ? el : a.L);
            for (int l = l_lo; l < l_hi; ++l)
                if (atomicExch(a.plan.class_tag + (size_t)l * a.n + lab, epoch) != epoch) {
                    const int at = atomicAdd(a.plan.job_count + (epoch & 1), 1);
                    a.plan.jobs[at] = (l << 16) | lab;
                    a.plan.items[at] = (l << 16) | lab;
                }
        }
    }
    if (b == 0) a.plan.job_count[(epoch + 1) & 1] = 0;  // the next call's counter (the call before this one is over)
    // the last CTA through makes the number current for the kernels that follow and publishes the
    // number of jobs (every CTA's appends are complete and visible before its ticket)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && atomicAdd(a.plan.epoch + 1, 1ull) == gridDim.x - 1) {
        __threadfence();
        const int jobs = *reinterpret_cast<volatile int32_t*>(a.plan.job_count + (epoch & 1));
        a.plan.job_count[2] = jobs;
        a.plan.job_count[3] = jobs;
        a.plan.epoch[1] = 0;
        a.plan.epoch[0] = epoch;
    }
}

// The same plan by a single CTA, for batches and memories small enough that one CTA's trip to
// memory is all it takes.  Up to kPlanCountMax pairs the frames of every pair are counted in shared memory
// (integer atomics: a sum), and a pair is listed with as many items as its count asks for; beyond, the pairs
// are only elected, in a bitmap, and listed with one item each.  Nothing waits on a ticket or a fence.
constexpr int kPlanOneThreads = 512;   // (a CTA that fits on an SM beside a streaming kernel's)
constexpr int kPlanOneMaxB = 8 * kPlanOneThreads;
constexpr int kPlanOneWords = 2048;   // 65 536 (layer, class) pairs as a bitmap
constexpr int kPlanCountMax = 8192;   // pairs that get a counter each

__global__ void __launch_bounds__(kPlanOneThreads) k_update_plan_one(const UpdateArgs a) {
    extern __shared__ int s_plan[];  // counters [pairs] or bitmap words
    __shared__ int s_jobs, s_items;
    const int tid = threadIdx.x;
    const int pairs = a.L * a.n;
    const bool counted = pairs <= kPlanCountMax;
    const int words = counted ? pairs : (pairs + 31) / 32;
    for (int i = tid; i < words; i += kPlanOneThreads) s_plan[i] = 0;
    if (tid == 0) s_jobs = s_items = 0;
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_PLAN : nullptr);
    __syncthreads();
    for (int b = tid; b < a.B; b += kPlanOneThreads) {
        const int dn = a.done ? a.done[b] : 0, pr = a.done ? a.pred[b] : -1, el = a.done ? a.exit_layer[b] : 0;
        const int fb = a.fallback ? a.fallback[b] : -1;
        const int sid = a.stream_id ? a.stream_id[b] : 0;
        const bool ex = dn != 0;
        int lab = ex ? pr : fb;
        if (lab >= a.n) lab = -1;
        if (sid < 0 || sid >= a.S) {  // a stream outside the cache: the frame takes no part in the update
            lab = -1;
            set_status(a.status, kDevInvalidArg);
        }
        a.plan.frame_code[b] = lab < 0 ? -1 : (lab | ((ex ? el : a.L) << 16));
        if (lab >= 0) {
            const int l_lo = a.warm_layer >= 0 ? a.warm_layer : 0;
            const int l_hi = a.warm_layer >= 0 ? a.warm_layer + 1 : (ex ? el : a.L);
            for (int l = l_lo; l < l_hi; ++l) {
                const int pair = l * a.n + lab;
                if (counted) {
                    atomicAdd(&s_plan[pair], 1);
                } else {
                    const unsigned int bit = 1u << (pair & 31);
                    if (!(atomicOr(reinterpret_cast<unsigned int*>(&s_plan[pair >> 5]), bit) & bit)) {
                        const int at = atomicAdd(&s_jobs, 1);
                        a.plan.jobs[at] = (l << 16) | lab;
                        a.plan.items[at] = (l << 16) | lab;
                    }
                }
            }
        }
    }
    __syncthreads();
    if (counted) {
        for (int pair = tid; pair < pairs; pair += kPlanOneThreads) {
            const int rows = s_plan[pair];
            if (rows == 0) continue;
            const int l = pair / a.n, code = (l << 16) | (pair - l * a.n);
            a.plan.jobs[atomicAdd(&s_jobs, 1)] = code;
            const int nb = item_blocks(rows, a.dims[l]), lg = ilog2_pow2(nb);
            const int at = atomicAdd(&s_items, nb);
            for (int k = 0; k < nb; ++k) a.plan.items[at + k] = code | (k << 20) | (lg << 24);
        }
        __syncthreads();
    }
    if (tid == 0) {
        a.plan.job_count[2] = s_jobs;
        a.plan.job_count[3] = counted ? s_items : s_jobs;
    }
}

// ---- Eq. 5 / Eq. 6 ------------------------------------------------------------------------

__device__ __forceinline__ unsigned long long score_of(int ft, int ts, int W, int forgetting = 0) {
    if (forgetting) return (unsigned long long)max(ft, 0);  // the decay already sits in the table
    int e = ts / W;
    if (e > kEMax) e = kEMax;
    const unsigned long long f = (unsigned long long)min(max(ft, 0), kFtMax);
    return f << (2 * (kEMax - e));  // FT * 4^(12 - e) = 4^12 * FT * 0.25^e
}

__host__ __device__ constexpr int pow2_at_least(int v) {
    int p = 2;
    while (p < v) p *= 2;
    return p;
}
// Ranking key of a class with a non-zero score: the score above the complement of the class id, so that a
// larger key means (score descending, id ascending).  Scores stay below 2^44 (FT <= 2^20 times 4^12, or a
// fixed-point FT below 2^31) and ids below 2^13.
static_assert(SMTM_MAX_CLASSES <= (1 << 13), "the ranking key keeps 13 bits for the class id");
__device__ __forceinline__ unsigned long long refresh_key(unsigned long long score, int id) {
    return (score << 13) | (unsigned long long)(8191 - id);
}
__device__ __forceinline__ int key_class(unsigned long long key) { return 8191 - int(key & 8191ull); }
__device__ __forceinline__ unsigned long long key_score(unsigned long long key) { return key >> 13; }

// Shared memory of a refresh: the keys of the non-zero scores (padded to a power of two for the sort) and the
// k_max best scores.
__host__ __device__ constexpr size_t refresh_smem(int n, int k_max) { return size_t(pow2_at_least(n)) * 8 + size_t(k_max) * 8; }

constexpr int kCountRankMax = 256;  // up to this many non-zero scores are ranked by counting, more by sorting
constexpr int kResizeThreadsMax = 1024;  // CTA of the stand-alone refresh when the memory has many classes

// Sum over the block of a 64-bit value; every thread gets the total.  s_part holds >= 32 words.
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* s_part) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long t = 0;
    for (int w = 0; w < int(blockDim.x + 31) >> 5; ++w) t += s_part[w];
    return t;
}

// Eq. 6 by one warp: the smallest k in [k_min, k_max] with cl_den * (sum of the k best scores) > cl_num * total;
// s_top holds the k_max best scores in rank order.  Every lane looks after a run of consecutive ranks (of odd
// length, which spreads the lanes over the banks): it adds its run up, a scan over the lanes gives the sum of
// the ranks before it, and a second walk finds the first rank of the run that satisfies the test.
__device__ __forceinline__ void adaptive_size(const ResizeArgs& a, int s, const unsigned long long* s_top,
                                              unsigned long long total, int lane) {
    int chosen = a.k_max;
    if (a.k_min < a.k_max) {  // (otherwise there is nothing to choose)
        const int per = ((a.k_max + kWarp - 1) / kWarp) | 1;
        const int lo = min(lane * per, a.k_max), hi = min(lo + per, a.k_max);
        unsigned long long run = 0;
        for (int r = lo; r < hi; ++r) run += s_top[r];
        unsigned long long inc = run;
#pragma unroll
        for (int o = 1; o < kWarp; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += t;
        }
        unsigned long long prefix = inc - run;
        const unsigned long long need = (unsigned long long)a.cl_num * total;
        for (int r = lo; r < hi; ++r) {
            prefix += s_top[r];
            if (r + 1 >= a.k_min && (unsigned long long)a.cl_den * prefix > need) {
                chosen = r + 1;
                break;
            }
        }
        chosen = __reduce_min_sync(kFull, chosen);
    }
    if (lane == 0) a.k[s] = chosen;
}

// Descending bitonic sort of nz keys in s_key by the whole CTA (padded to a power of two with zeros: no key is zero).
__device__ void sort_keys(unsigned long long* s_key, int nz) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int P = pow2_at_least(nz), half = P >> 1;
    for (int i = nz + tid; i < P; i += nt) s_key[i] = 0ull;
    __syncthreads();
    // Pair t of a round with stride j is (i, i + j), i = t with a zero bit put in at j's position.  Thread t keeps
    // pair t in every round, so with strides up to 32 the pairs of a warp stay inside the 64 keys that warp alone
    // touches: such a round needs the whole CTA only when the round before or after it has a longer stride.
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < half; t += nt) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1)), l = i + j;
                const unsigned long long ki = s_key[i], kl = s_key[l];
                if (((i & k) == 0) ? kl > ki : kl < ki) {
                    s_key[i] = kl;
                    s_key[l] = ki;
                }
            }
            const int next = j > 1 ? j >> 1 : k;  // (the next phase opens with stride k)
            if (j > kWarp || next > kWarp) __syncthreads();
            else __syncwarp();
        }
    }
    __syncthreads();
}

// Descending bitonic sort with one key per thread (thread i holds element i; a CTA of P threads, P a power of two
// and a multiple of 32; every thread of the CTA calls): partners up to 16 apart trade keys by warp shuffle, those
// further apart through shared memory, one barrier per round over two alternating buffers of P words each.
__device__ __forceinline__ unsigned long long sort_one_key_per_thread(unsigned long long key, int P,
                                                                      unsigned long long* s_x) {
    const int i = threadIdx.x;
    int flip = 0;
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            unsigned long long other;
            if (j < kWarp) {
                other = __shfl_xor_sync(kFull, key, j);
            } else {
                unsigned long long* buf = s_x + (flip ? P : 0);
                flip ^= 1;
                buf[i] = key;
                __syncthreads();
                other = buf[i ^ j];
            }
            // the lower index of a pair keeps the larger key where the run is descending, the smaller one elsewhere
            const bool larger = ((i & j) == 0) == ((i & k) == 0);
            key = larger ? max(key, other) : min(key, other);
        }
    }
    return key;
}

// Descending bitonic sort of PER keys per thread (thread t holds elements t * PER ... in key[]; blockDim.x * PER a
// power of two; every thread of the CTA calls).  A compare-exchange whose partner sits in the same thread is done
// in registers, one up to 31 threads away by warp shuffle, the few beyond through shared memory (s_x: a word per
// element, laid out [register][thread]).
template <int PER>
__device__ __forceinline__ void sort_keys_in_registers(unsigned long long (&key)[PER], unsigned long long* s_x) {
    const int tid = threadIdx.x, nt = blockDim.x, P = nt * PER;
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j >= PER; j >>= 1) {
            const int tj = j / PER;
            // the lower element of a pair keeps the larger key where the run is descending, the smaller one elsewhere
            const bool larger = ((tid & tj) == 0) == (((tid * PER) & k) == 0);
            if (tj < kWarp) {
#pragma unroll
                for (int i = 0; i < PER; ++i) {
                    const unsigned long long other = __shfl_xor_sync(kFull, key[i], tj);
                    key[i] = larger ? max(key[i], other) : min(key[i], other);
                }
            } else {
                __syncthreads();  // the previous round's readers are done
#pragma unroll
                for (int i = 0; i < PER; ++i) s_x[i * nt + tid] = key[i];
                __syncthreads();
#pragma unroll
                for (int i = 0; i < PER; ++i) {
                    const unsigned long long other = s_x[i * nt + (tid ^ tj)];
                    key[i] = larger ? max(key[i], other) : min(key[i], other);
                }
            }
        }
#pragma unroll
        for (int j = PER >> 1; j > 0; j >>= 1) {
            if (j < k) {
#pragma unroll
                for (int i = 0; i < PER; ++i)
                    if ((i & j) == 0) {
                        const bool desc = ((tid * PER + i) & k) == 0;
                        const unsigned long long hi = max(key[i], key[i | j]), lo = min(key[i], key[i | j]);
                        key[i] = desc ? hi : lo;
                        key[i | j] = desc ? lo : hi;
                    }
            }
        }
    }
}

// Eq. 5 / Eq. 6 for stream s from the scores of PER consecutive classes per thread (c_lo ...), by a sort in
// registers: for memories of so many classes that most scores are non-zero and ranking by counting would cost
// a pass over all keys per key.  The key of a class is one more than its ranking key, so that classes with a zero
// score sort behind the others in ascending id (as the refresh wants them) and before the padding.
// `dyn`: blockDim.x * PER words for the sort, then the k_max best scores.
template <int PER>
__device__ void refresh_sorted_in_registers(const ResizeArgs& a, int s, const unsigned long long (&sc)[PER], int c_lo,
                                            unsigned char* dyn, unsigned long long* s_part) {
    const int tid = threadIdx.x, P = blockDim.x * PER;
    unsigned long long* s_x = reinterpret_cast<unsigned long long*>(dyn);  // [P]
    unsigned long long* s_top = s_x + P;                                    // [k_max]
    unsigned long long key[PER], local = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = c_lo + i;
        key[i] = c < a.n ? refresh_key(sc[i], c) + 1ull : 0ull;
        local += c < a.n ? sc[i] : 0ull;
    }
    const unsigned long long total = block_sum_u64(local, s_part);
    if (total == 0) return;  // nothing seen yet: keep size and members (the same for every thread)
    sort_keys_in_registers<PER>(key, s_x);
    int32_t* mem = a.members + (size_t)s * a.k_max;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int r = tid * PER + i;
        if (r < a.k_max && r < a.n) {
            mem[r] = key_class(key[i] - 1ull);
            s_top[r] = key_score(key[i] - 1ull);
        }
    }
    __syncthreads();
    if (tid < kWarp) adaptive_size(a, s, s_top, total, tid);
}

// Eq. 5 / Eq. 6 for stream s when every thread of the CTA holds the scores of its PER consecutive classes
// (c_lo ...) in registers.  The keys of the non-zero scores are appended to a list in shared memory in whatever
// order the threads come (a key carries its class, and ranking by key does not care about the list's order);
// the rest is one warp's work: ranks by counting (a sort by the whole CTA when the keys are many), zero-score
// classes in ascending id for the slots that remain (they are among the first k_max ids), Eq. 6.
// `dyn`: keys [pow2 >= n] | best scores [k_max] | zero flags [k_max] bytes.  *s_nz and *s_total are zero on entry.
template <int PER>
__device__ void refresh_from_registers(const ResizeArgs& a, int s, const unsigned long long (&sc)[PER], int c_lo,
                                       unsigned char* dyn, int* s_nz, unsigned long long* s_total) {
    const int cap = pow2_at_least(a.n);
    unsigned long long* s_key = reinterpret_cast<unsigned long long*>(dyn);  // [cap]
    unsigned long long* s_top = s_key + cap;                                 // [k_max]
    unsigned char* s_zero = reinterpret_cast<unsigned char*>(s_top + a.k_max);  // [k_max]
    const int tid = threadIdx.x, lane = tid & 31;
    unsigned long long local = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int c = c_lo + i;
        if (c < a.n) {
            if (sc[i] != 0) {
                s_key[atomicAdd(s_nz, 1)] = refresh_key(sc[i], c);
                local += sc[i];
            }
            if (c < a.k_max) s_zero[c] = sc[i] == 0 ? 1 : 0;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(kFull, local, o);
    if (lane == 0 && local != 0) atomicAdd(s_total, local);
    __syncthreads();
    const int nz = *s_nz;
    const unsigned long long total = *s_total;
    if (total == 0) return;  // nothing seen yet: keep size and members (the same for every thread)
    const bool sorted = nz > kCountRankMax;
    if (sorted) sort_keys(s_key, nz);
    if (tid >= kWarp) return;
    int32_t* mem = a.members + (size_t)s * a.k_max;
    if (sorted) {
        for (int r = lane; r < nz && r < a.k_max; r += kWarp) {
            mem[r] = key_class(s_key[r]);
            s_top[r] = key_score(s_key[r]);
        }
    } else {
        for (int i = lane; i < nz; i += kWarp) {  // rank = keys larger than this one (keys are distinct)
            const unsigned long long key = s_key[i];
            int r0 = 0, r1 = 0;
            int j = 0;
            for (; j + 1 < nz; j += 2) {
                r0 += s_key[j] > key ? 1 : 0;
                r1 += s_key[j + 1] > key ? 1 : 0;
            }
            if (j < nz) r0 += s_key[j] > key ? 1 : 0;
            const int r = r0 + r1;
            if (r < a.k_max) {
                mem[r] = key_class(key);
                s_top[r] = key_score(key);
            }
        }
    }
    const unsigned lt = (1u << lane) - 1u;
    int filled = nz;
    for (int c0 = 0; c0 < a.k_max && filled < a.k_max; c0 += kWarp) {
        const int c = c0 + lane;
        const bool z = c < a.k_max && s_zero[c] != 0;
        const unsigned m = __ballot_sync(kFull, z);
        const int pos = filled + __popc(m & lt);
        if (z && pos < a.k_max) {
            mem[pos] = c;
            s_top[pos] = 0;
        }
        filled += __popc(m);
    }
    __syncwarp();
    adaptive_size(a, s, s_top, total, lane);
}

// Eq. 5 / Eq. 6 for stream s by the whole CTA (any number of threads), from the stream's tables in global memory
// as this CTA left them.  Every thread looks after a run of consecutive classes; the keys of the
// non-zero scores are compacted by one scan over the threads and ranked, largest first: by counting when they
// are few, by a bitonic sort otherwise; zero-score classes follow in ascending id.  Then the smallest k in
// [k_min, k_max] whose k best scores exceed cl_num / cl_den of all.  `dyn` holds refresh_smem(n, k_max) bytes.
__device__ void refresh_stream(const ResizeArgs& a, int s, unsigned char* dyn, int* s_scan, unsigned long long* s_part) {
    const int cap = pow2_at_least(a.n);
    unsigned long long* s_key = reinterpret_cast<unsigned long long*>(dyn);  // [cap]
    unsigned long long* s_top = s_key + cap;                                 // [k_max]
    const int tid = threadIdx.x, nt = blockDim.x;
    const int32_t* ft = a.ft + (size_t)s * a.n;
    const int32_t* ts = a.ts + (size_t)s * a.n;
    int32_t* mem = a.members + (size_t)s * a.k_max;
    if (nt == cap) {
        // A thread per class: the key of class tid (one more than the ranking key, so that the classes with a zero
        // score sort behind the others in ascending id, as the refresh wants them, and before the padding),
        // sorted in registers; thread r ends up with the class of rank r.
        const bool real = tid < a.n;
        const unsigned long long sc = real ? score_of(ft[tid], ts[tid], a.W, a.forgetting) : 0ull;
        const unsigned long long total = block_sum_u64(sc, s_part);
        if (total == 0) return;  // nothing seen yet: keep size and members (the same for every thread)
        const unsigned long long key = sort_one_key_per_thread(real ? refresh_key(sc, tid) + 1ull : 0ull, cap, s_key);
        unsigned long long* s_best = s_key + 2 * cap;
        if (tid < a.k_max && tid < a.n) {
            mem[tid] = key_class(key - 1ull);
            s_best[tid] = key_score(key - 1ull);
        }
        __syncthreads();
        if (tid < kWarp) adaptive_size(a, s, s_best, total, tid);
        return;
    }
    const int per = (a.n + nt - 1) / nt;
    const int c_lo = min(a.n, tid * per), c_hi = min(a.n, c_lo + per);
    const auto score_at = [&](int c) { return score_of(ft[c], ts[c], a.W, a.forgetting); };

    int nzl = 0;
    unsigned long long local = 0;
    for (int c = c_lo; c < c_hi; ++c) {
        const unsigned long long sc = score_at(c);
        nzl += sc != 0 ? 1 : 0;
        local += sc;
    }
    int nz;
    int pos = block_exclusive_scan(nzl, s_scan, &nz);
    const unsigned long long total = block_sum_u64(local, s_part);
    if (total == 0) return;  // nothing seen yet: keep size and members (the same for every thread)
    for (int c = c_lo; c < c_hi && nzl; ++c) {
        const unsigned long long sc = score_at(c);
        if (sc != 0) s_key[pos++] = refresh_key(sc, c);
    }
    __syncthreads();
    if (nz <= kCountRankMax) {
        // rank = keys larger than this one (keys are distinct); rank r < k_max goes to slot r
        for (int i = tid; i < nz; i += nt) {
            const unsigned long long key = s_key[i];
            int r0 = 0, r1 = 0;
            int j = 0;
            for (; j + 1 < nz; j += 2) {
                r0 += s_key[j] > key ? 1 : 0;
                r1 += s_key[j + 1] > key ? 1 : 0;
            }
            if (j < nz) r0 += s_key[j] > key ? 1 : 0;
            const int r = r0 + r1;
            if (r < a.k_max) {
                mem[r] = key_class(key);
                s_top[r] = key_score(key);
            }
        }
    } else {
        sort_keys(s_key, nz);
        for (int r = tid; r < nz && r < a.k_max; r += nt) {
            mem[r] = key_class(s_key[r]);
            s_top[r] = key_score(s_key[r]);
        }
    }
    // zero-score classes fill the remaining slots in ascending id
    if (nz < a.k_max) {
        int zl = 0;
        for (int c = c_lo; c < c_hi; ++c) zl += score_at(c) == 0 ? 1 : 0;
        int zt;
        int zp = nz + block_exclusive_scan(zl, s_scan, &zt);
        for (int c = c_lo; c < c_hi && zl && zp < a.k_max; ++c)
            if (score_at(c) == 0) {
                mem[zp] = c;
                s_top[zp] = 0;
                ++zp;
            }
    }
    __syncthreads();
    if (tid < kWarp) adaptive_size(a, s, s_top, total, tid);
}

__global__ void __launch_bounds__(kResizeThreadsMax) k_resize(const ResizeArgs a) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[32];
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_REFRESH : nullptr);
    refresh_stream(a, blockIdx.x, reinterpret_cast<unsigned char*>(s_dyn), s_scan, s_part);
}

// ---- apply: tables ----------------------------------------------------------------------------

// Compacts, in ascending frame index, the frames of a tile of blockDim.x for which `hit`
// is set into list[0..cnt); returns cnt (the same in every thread).
__device__ __forceinline__ int compact_tile(int hit, int value, int* list, int* s_scan) {
    int cnt;
    const int pos = block_exclusive_scan(hit, s_scan, &cnt);
    if (cnt) {
        __syncthreads();  // the previous tile's readers are done with list
        if (hit) list[pos] = value;
        __syncthreads();
    }
    return cnt;
}

// Shared memory of a tables CTA: the refresh buffers, which also serve as the two integer arrays [n] of the
// closed form before the refresh begins.
__host__ __device__ constexpr size_t tables_smem(int n, int k_max, bool with_refresh) {
    const size_t closed = size_t(n) * 2 * sizeof(int);
    const size_t refresh = with_refresh ? refresh_smem(n, k_max) + size_t(k_max) : 0;  // ... and a flag per slot
    return closed > refresh ? closed : refresh;
}

// Sec. 6.1 for the stream of frame g by one CTA, if g is the stream's first frame in the batch (else the
// CTA of that frame does it; g < 0: the only stream of a cache that has one, whichever frame of it comes
// first): all of the stream's frames, in ascending index, applied to its tables; then,
// if asked, the stream's Eq. 5 / Eq. 6 refresh.  Every thread looks after a run of PER consecutive classes
// and keeps their entries in registers from the one trip to memory that fetches them to the refresh
// (PER == 0: any number of classes, the entries stay in global memory).
template <int PER>
__device__ void tables_of_frame(const UpdateArgs& a, const ResizeArgs& rz, int g, int do_resize, unsigned char* dyn,
                                int* s_list, int* s_scan, unsigned long long* s_part) {
    const int tid = threadIdx.x, nt = blockDim.x;
    if (tid == 0) {  // the refresh's counters (read after the barriers below)
        s_scan[32] = 0;
        s_part[31] = 0ull;
    }
    const bool lone = g < 0;
    if (lone) g = 0;
    const int s = (a.stream_id && !lone) ? a.stream_id[g] : 0;
    if (s < 0 || s >= a.S) return;  // no such stream (the same for every thread; the plan kernel records the error)
    const int per = PER ? PER : (a.n + nt - 1) / nt;
    const int c_lo = min(a.n, tid * per), c_hi = min(a.n, c_lo + per);
    int32_t* ft = a.ft + (size_t)s * a.n;
    int32_t* ts = a.ts + (size_t)s * a.n;
    // the label frame g ends up with, every load issued at once (final_label_of would wait for the exit flag first)
    const int dn_g = a.done ? a.done[g] : 0, pr_g = a.done ? a.pred[g] : -1, fb_g = a.fallback ? a.fallback[g] : -1;
    int f[PER ? PER : 1], t[PER ? PER : 1];
#pragma unroll
    for (int i = 0; i < PER; ++i) {  // in flight with the stream ids below
        f[i] = c_lo + i < a.n ? ft[c_lo + i] : 0;
        t[i] = c_lo + i < a.n ? ts[c_lo + i] : 0;
    }
    // an earlier frame of the same stream: its CTA does the work.  Also: is g the stream's only frame?
    int earlier = (!a.stream_id && g > 0) ? 1 : 0, later = ((!a.stream_id && g + 1 < a.B) || lone) ? 1 : 0;
    for (int b0 = 0; a.stream_id && !lone && b0 < a.B; b0 += 4 * nt) {
        int sidv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) sidv[u] = a.stream_id[min(b0 + u * nt + tid, a.B - 1)];  // one trip to memory
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int b = b0 + u * nt + tid;
            const int same = (b < a.B && sidv[u] == s) ? 1 : 0;
            earlier |= (b < g) ? same : 0;
            later |= (b > g) ? same : 0;
        }
    }
    if (__syncthreads_or(earlier)) return;
    const bool single = !__syncthreads_or(later);
    int label_g = dn_g != 0 ? pr_g : fb_g;
    if (label_g >= a.n) label_g = -1;
    if (single) {
        // one frame (a video stream that delivers a frame per step): Sec. 6.1 as printed, one pass over the classes
        if (PER) {
#pragma unroll
            for (int i = 0; i < PER; ++i) table_step(f[i], t[i], c_lo + i == label_g, a.forget_W);
        } else {
            for (int c = c_lo; c < c_hi; ++c) {
                int fc = ft[c], tc = ts[c];
                table_step(fc, tc, c == label_g, a.forget_W);
                ft[c] = fc;
                ts[c] = tc;
            }
        }
    } else if (a.forget_W == 0) {
        // Plain counts: what a frame-by-frame replay leaves behind has a closed form per class.  With
        // m frames of the stream in the batch, a class that appears q times, last at position p, ends
        // with FT + q and TS = m - 1 - p; one that does not appear ends with TS + m.  q and p are
        // gathered by shared-memory atomics on integers (a sum and a maximum: order does not matter).
        int* s_cnt = reinterpret_cast<int*>(dyn);  // [n]; the refresh below reuses the space
        int* s_last = s_cnt + a.n;                 // [n]
        for (int c = tid; c < a.n; c += nt) {
            s_cnt[c] = 0;
            s_last[c] = -1;
        }
        __syncthreads();
        // Every thread looks at a run of eight consecutive frames (their stream ids and the plan's codes in one
        // trip to memory); a scan over the threads gives each of the stream's frames its position in the stream.
        int m = 0;
        for (int p0 = g; p0 < a.B; p0 += kTabPer * nt) {
            const int b0 = p0 + tid * kTabPer;
            int sidv[kTabPer], code[kTabPer];
#pragma unroll
            for (int i = 0; i < kTabPer; ++i) {
                const int b = min(b0 + i, a.B - 1);
                sidv[i] = a.stream_id ? a.stream_id[b] : s;
                code[i] = a.plan.frame_code[b];
            }
            int hits = 0;
#pragma unroll
            for (int i = 0; i < kTabPer; ++i) {
                sidv[i] = (b0 + i < a.B && sidv[i] == s) ? 1 : 0;
                hits += sidv[i];
            }
            int cnt;
            int pos = m + block_exclusive_scan(hits, s_scan, &cnt);
#pragma unroll
            for (int i = 0; i < kTabPer; ++i)
                if (sidv[i]) {
                    if (code[i] >= 0) {  // (a frame without a label only ages the classes)
                        atomicAdd(&s_cnt[code[i] & 0xffff], 1);
                        atomicMax(&s_last[code[i] & 0xffff], pos);
                    }
                    ++pos;
                }
            m += cnt;
        }
        __syncthreads();
        const auto closed = [&](int c, int& fc, int& tc) {
            const int q = s_cnt[c];
            if (q > 0) {
                fc = int(min((long long)fc + q, (long long)kFtMax));
                tc = m - 1 - s_last[c];
            } else {
                tc = int(min((long long)tc + m, (long long)INT32_MAX));
            }
        };
        if (PER) {
#pragma unroll
            for (int i = 0; i < PER; ++i)
                if (c_lo + i < a.n) closed(c_lo + i, f[i], t[i]);
        } else {
            for (int c = c_lo; c < c_hi; ++c) {
                int fc = ft[c], tc = ts[c];
                closed(c, fc, tc);
                ft[c] = fc;
                ts[c] = tc;
            }
        }
    } else {
        // the forgetting table has no closed form: the stream's frames, a tile at a time, replayed per class
        for (int t0 = g - g % nt; t0 < a.B; t0 += nt) {
            const int b = t0 + tid;
            const int hit = (b >= g && b < a.B && (a.stream_id ? a.stream_id[b] : 0) == s) ? 1 : 0;
            const int cnt = compact_tile(hit, hit ? final_label_of(a, b) : -1, s_list, s_scan);
            if (cnt == 0) continue;
            if (PER) {
#pragma unroll
                for (int i = 0; i < PER; ++i)
                    for (int j = 0; j < cnt; ++j) table_step(f[i], t[i], s_list[j] == c_lo + i, a.forget_W);
            } else {
                for (int c = c_lo; c < c_hi; ++c) {
                    int fc = ft[c], tc = ts[c];
                    for (int j = 0; j < cnt; ++j) table_step(fc, tc, s_list[j] == c, a.forget_W);
                    ft[c] = fc;
                    ts[c] = tc;
                }
            }
        }
    }
    unsigned long long sc[PER ? PER : 1];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        if (c_lo + i < a.n) {
            ft[c_lo + i] = f[i];
            ts[c_lo + i] = t[i];
        }
        sc[i] = c_lo + i < a.n ? score_of(f[i], t[i], rz.W, rz.forgetting) : 0ull;
    }
    if (do_resize) {
        __syncthreads();  // every thread is done with the closed form's arrays (and sees its own table entries)
        if (PER == 8)
            refresh_sorted_in_registers<(PER ? PER : 1)>(rz, s, sc, c_lo, dyn, s_part);
        else if (PER)
            refresh_from_registers<(PER ? PER : 1)>(rz, s, sc, c_lo, dyn, &s_scan[32], &s_part[31]);
        else
            refresh_stream(rz, s, dyn, s_scan, s_part);
    }
}

// ---- apply: Eq. 7 -----------------------------------------------------------------------------

constexpr int kCenPer = 8;                         // consecutive frames a thread looks at
constexpr int kCenTile = kCenPer * kApplyThreads;  // frames listed at a time
constexpr int kRowGroupsMax = 8;
constexpr int kWideSweeps = 4;                     // an item up to this many times as wide as the CTA is folded in one go

// Lists, in ascending index, the frames base .. base + kCenTile - 1 whose label is cls and that stopped at
// layer l0 + 1 or deeper; returns how many (the same in every thread).  Every thread fetches the codes of its
// run of consecutive frames in one trip to memory (first_tile: those of frames 0 .. kCenTile - 1, which do not
// depend on the pair and are fetched before the pair is known); one scan over the threads places them.
__device__ __forceinline__ int list_pair_frames(const UpdateArgs& a, int base, int cls, int l0, int* s_list, int* s_scan,
                                                const int (&first_tile)[kCenPer]) {
    const int f0 = base + threadIdx.x * kCenPer;
    int code[kCenPer];
#pragma unroll
    for (int i = 0; i < kCenPer; ++i)  // (the first tile's codes were fetched when the CTA began)
        code[i] = base == 0 ? first_tile[i] : a.plan.frame_code[min(f0 + i, a.B - 1)];
    int mine = 0;
#pragma unroll
    for (int i = 0; i < kCenPer; ++i) {
        const bool hit = f0 + i < a.B && code[i] >= 0 && (code[i] & 0xffff) == cls && (code[i] >> 16) >= l0 + 1;
        code[i] = hit ? 1 : 0;
        mine += code[i];
    }
    int cnt;
    int pos = block_exclusive_scan(mine, s_scan, &cnt);
    if (cnt == 0) return 0;
    __syncthreads();  // the previous tile's readers are done with the list
#pragma unroll
    for (int i = 0; i < kCenPer; ++i)
        if (code[i]) s_list[pos++] = f0 + i;
    __syncthreads();
    return cnt;
}

// Eq. 7 for one 16-byte group of columns of a centre: SC = (SC m + sum SV) / (m + q), in double (the count is
// exact at any size and SC m + sum SV is rounded once; inv = 1 / (m + q)); the tensor-core scorer's bf16 copy of
// the centre, where there is one, follows it (x = hi + lo).  Returns the group's part of the squared length.
__device__ __forceinline__ float fold_centre(const UpdateArgs& a, int l0, int cls, int D, int c4, const float4& old,
                                             const float (&acc)[4], double dm, double inv, float* cen) {
    float4 v;
    v.x = float((double(old.x) * dm + double(acc[0])) * inv);
    v.y = float((double(old.y) * dm + double(acc[1])) * inv);
    v.z = float((double(old.z) * dm + double(acc[2])) * inv);
    v.w = float((double(old.w) * dm + double(acc[3])) * inv);
    *reinterpret_cast<float4*>(cen + 4 * c4) = v;
    if (a.cen_split[l0]) {
        __nv_bfloat16* hi = a.cen_split[l0] + (size_t)cls * D + 4 * c4;
        __nv_bfloat16* lo = hi + (size_t)a.n * D;
        const float x[4] = {v.x, v.y, v.z, v.w};
        __nv_bfloat16 h[4], t[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            h[j] = __float2bfloat16_rn(x[j]);
            t[j] = __float2bfloat16_rn(x[j] - __bfloat162float(h[j]));
        }
        *reinterpret_cast<uint2*>(hi) = *reinterpret_cast<const uint2*>(h);
        *reinterpret_cast<uint2*>(lo) = *reinterpret_cast<const uint2*>(t);
    }
    float nrm = 0.f;
    nrm = fmaf(v.x, v.x, nrm); nrm = fmaf(v.y, v.y, nrm); nrm = fmaf(v.z, v.z, nrm); nrm = fmaf(v.w, v.w, nrm);
    return nrm;
}

// Eq. 7 for one item: the columns [block's share] of the centre of (layer l0, class cls).  The frames whose
// label is cls and that stopped at layer l0 + 1 or deeper are listed in ascending index, a tile of frames at a
// time (every thread looks at a run of consecutive frames, one scan over the threads).  A thread is (a 16-byte
// group of columns, a row group): row group r adds the listed rows r, r + R, ... in that order (eight rows in
// flight), the groups' sums are added in a fixed order, then SC = (SC m + sum SV) / (m + q).  A pair that is a
// single item then renews the centre's length and count itself.  The items of a cut pair leave the squared
// length of their blocks in norm_part and take a ticket; the last one through adds the blocks in order and
// renews length and count (every item has read the count by then), and puts the ticket back to zero.
__device__ void centre_item(const UpdateArgs& a, int item, const int (&first_tile)[kCenPer], int* s_list, int* s_scan,
                            float4* s_acc) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int cls = item & 0x1fff, l0 = (item >> 16) & 15, blk = (item >> 20) & 15, nblk = 1 << ((item >> 24) & 7);
    const int D = a.dims[l0];
    const float* sv = a.sv[l0];
    float* cen = a.centers[l0] + (size_t)cls * D;
    const uint32_t m = a.m[l0][cls];
    float nrm = 0.f;
    int q = 0;
    if ((D & 3) == 0) {
        const int D4 = D >> 2, per_blk = (D4 + nblk - 1) / nblk;
        const int lo4 = min(D4, blk * per_blk), hi4 = min(D4, lo4 + per_blk);  // this item's 16-byte column groups
        int R = 1;                                                             // row groups
        while (R < kRowGroupsMax && 2 * R * (hi4 - lo4) <= nt) R *= 2;
        const int cpp = nt / R;                                                // column groups per sweep
        const int rg = tid / cpp, c = tid - rg * cpp;
        const int sweeps = (hi4 - lo4 + cpp - 1) / cpp;
        const bool wide = sweeps > 1 && sweeps <= kWideSweeps && a.B <= kCenTile;  // (more than one sweep: R == 1)
        if (wide) {
            // An item a few times as wide as the CTA whose frames fit one listing (the usual pair: a row or two of
            // a long vector): the frames are listed once, and a thread has its column groups of two sweeps in
            // flight together, a row at a time.  Same order of additions as below.
            const int cnt = list_pair_frames(a, 0, cls, l0, s_list, s_scan, first_tile);
            q = cnt;
            const double dm = double(m), inv = 1.0 / (dm + double(q));
            for (int w0 = 0; w0 < sweeps && q > 0; w0 += 2) {
                const int ca = lo4 + w0 * nt + tid, cb = ca + nt;
                const int la = min(ca, hi4 - 1), lb = min(cb, hi4 - 1);  // unconditional loads (past the item's end: its last group)
                float acc_a[4] = {0.f, 0.f, 0.f, 0.f}, acc_b[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
                for (int i = 0; i < cnt; ++i) {
                    const float4* rp = reinterpret_cast<const float4*>(sv + (size_t)s_list[i] * D);
                    const float4 ra = __ldg(rp + la), rb = __ldg(rp + lb);
                    acc_a[0] += ra.x; acc_a[1] += ra.y; acc_a[2] += ra.z; acc_a[3] += ra.w;
                    acc_b[0] += rb.x; acc_b[1] += rb.y; acc_b[2] += rb.z; acc_b[3] += rb.w;
                }
                const float4 old_a = *reinterpret_cast<const float4*>(cen + 4 * la);
                const float4 old_b = *reinterpret_cast<const float4*>(cen + 4 * lb);
                if (ca < hi4) nrm += fold_centre(a, l0, cls, D, ca, old_a, acc_a, dm, inv, cen);
                if (cb < hi4) nrm += fold_centre(a, l0, cls, D, cb, old_b, acc_b, dm, inv, cen);
            }
        }
        for (int s4 = lo4; s4 < hi4 && !wide; s4 += cpp) {  // (one sweep unless the item is wider than the CTA)
            const int c4 = s4 + c;
            const bool mine_col = c4 < hi4;
            float4 old = make_float4(0.f, 0.f, 0.f, 0.f);
            if (mine_col && rg == 0) old = *reinterpret_cast<const float4*>(cen + 4 * c4);  // in flight with the listing
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            q = 0;
            for (int base = 0; base < a.B; base += kCenTile) {
                const int cnt = list_pair_frames(a, base, cls, l0, s_list, s_scan, first_tile);
                if (cnt == 0) continue;  // (the same for every thread)
                q += cnt;
                if (!mine_col) continue;
                for (int i0 = rg; i0 < cnt; i0 += 8 * R) {
                    float4 r[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)  // unconditional loads (past the end: the last row again, unused)
                        r[u] = __ldg(reinterpret_cast<const float4*>(sv + (size_t)s_list[min(i0 + u * R, cnt - 1)] * D) + c4);
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (i0 + u * R < cnt) {
                            acc[0] += r[u].x; acc[1] += r[u].y; acc[2] += r[u].z; acc[3] += r[u].w;
                        }
                }
            }
            // the row groups' sums in a fixed order: ((g0 + g1) + g2) + ...
            __syncthreads();
            if (rg > 0 && mine_col) s_acc[(rg - 1) * cpp + c] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            __syncthreads();
            if (rg == 0 && mine_col && q > 0) {
                for (int g2 = 1; g2 < R; ++g2) {
                    const float4 o = s_acc[(g2 - 1) * cpp + c];
                    acc[0] += o.x; acc[1] += o.y; acc[2] += o.z; acc[3] += o.w;
                }
                const double dm = double(m), inv = 1.0 / (dm + double(q));
                nrm += fold_centre(a, l0, cls, D, c4, old, acc, dm, inv, cen);
            }
        }
    } else {
        // a vector that is not a whole number of 16-byte pieces (never cut into blocks): a column per thread
        for (int d = tid; d < D || d - tid < D; d += nt) {  // every thread makes every trip (the listing is the CTA's)
            float acc = 0.f;
            q = 0;
            for (int base = 0; base < a.B; base += kCenTile) {
                const int cnt = list_pair_frames(a, base, cls, l0, s_list, s_scan, first_tile);
                if (cnt == 0) continue;
                q += cnt;
                if (d < D)
                    for (int i = 0; i < cnt; ++i) acc += sv[(size_t)s_list[i] * D + d];
            }
            if (d < D && q > 0) {
                const float v = float((double(cen[d]) * double(m) + double(acc)) / (double(m) + double(q)));
                cen[d] = v;
                nrm = fmaf(v, v, nrm);
            }
        }
    }
    if (q == 0) return;  // cannot happen for a listed pair (the same for every thread)
    __syncthreads();     // s_acc is free: it serves the sum below
    nrm = block_sum(nrm, reinterpret_cast<float*>(s_acc));
    if (tid != 0) return;
    if (nblk > 1) {
        const size_t pair = (size_t)l0 * a.n + cls;
        a.norm_part[pair * kItemBlocksMax + blk] = nrm;
        __threadfence();  // this item's part of the centre and of its length, before the ticket
        if (atomicAdd(a.ticket + pair, 1) != nblk - 1) return;
        __threadfence();
        nrm = 0.f;
        for (int k = 0; k < nblk; ++k) nrm += *reinterpret_cast<volatile float*>(a.norm_part + pair * kItemBlocksMax + k);
        a.ticket[pair] = 0;
    }
    a.cnorm[l0][cls] = __fsqrt_rn(nrm);
    a.m[l0][cls] = m + uint32_t(q);
}

// The apply kernel: CTAs [0, table_ctas) are tables CTAs, one per frame (a single one for a cache with one stream);
// the others take the listed items.
__global__ void __launch_bounds__(kApplyThreads, 8) k_update_apply(const UpdateArgs a, const ResizeArgs rz, int do_resize,
                                                                    int table_ctas) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_list[kCenTile];
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[32];
    __shared__ float4 s_acc[kApplyThreads];  // (row groups - 1) x column groups of a sweep
    chain_wait();
    chain_release();
    if (int(blockIdx.x) < table_ctas) {
        const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_TABLES : nullptr);
        unsigned char* dyn = reinterpret_cast<unsigned char*>(s_dyn);
        if (a.n <= 4 * kApplyThreads)
            tables_of_frame<4>(a, rz, a.S == 1 ? -1 : int(blockIdx.x), do_resize, dyn, s_list, s_scan, s_part);
        else if (a.n <= 8 * kApplyThreads)
            tables_of_frame<8>(a, rz, a.S == 1 ? -1 : int(blockIdx.x), do_resize, dyn, s_list, s_scan, s_part);
        else
            tables_of_frame<0>(a, rz, a.S == 1 ? -1 : int(blockIdx.x), do_resize, dyn, s_list, s_scan, s_part);
        return;
    }
    const int first = int(blockIdx.x) - table_ctas, stride = int(gridDim.x) - table_ctas;
    int first_tile[kCenPer];  // the codes of the first frames, the item and the count: one trip to memory
#pragma unroll
    for (int i = 0; i < kCenPer; ++i) first_tile[i] = a.plan.frame_code[min(int(threadIdx.x) * kCenPer + i, a.B - 1)];
    int item = a.plan.items[first];  // (the list has room for every CTA)
    const int n_items = a.plan.job_count[3];
    if (first >= n_items) return;
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_CENTERS : nullptr);
    for (int it = first; it < n_items; it += stride) {
        if (it != first) {
            __syncthreads();  // the previous item's readers are done with the list
            item = a.plan.items[it];
        }
        centre_item(a, item, first_tile, s_list, s_scan, s_acc);
    }
}

__global__ void k_center_norms(const float* __restrict__ centers, int n, int D, float* __restrict__ cnorm) {
    __shared__ float s_red[32];
    chain_wait();
    chain_release();
    const int c = blockIdx.x;
    float nrm = 0.f;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const float v = centers[(size_t)c * D + d];
        nrm = fmaf(v, v, nrm);
    }
    nrm = block_sum(nrm, s_red);
    if (threadIdx.x == 0) cnorm[c] = __fsqrt_rn(nrm);
}

}  // namespace

cudaError_t memory_setup() {
    cudaError_t e = allow_max_dynamic_smem(k_update_apply);
    if (e == cudaSuccess) e = allow_max_dynamic_smem(k_resize);
    // the update's kernels share SMs with the next step's pooling kernel on the pipelined route
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_update_apply);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_update_plan_one);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_update_plan);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_resize);

    return e;   // (the single-CTA plan needs at most 32 KB + its statics: below the default limit)
}

cudaError_t launch_center_norms(const float* centers, int n, int D, float* cnorm, cudaStream_t st,
                                int64_t* launches) {
    ++*launches;
    return launch_chained(k_center_norms, n, 256, 0, st, centers, n, D, cnorm);
}

cudaError_t launch_update(const UpdateArgs& a, const ResizeArgs* rz, int sm_count, cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    ++*launches;
    const long long pairs = (long long)a.L * a.n;
    if (a.B <= kPlanOneMaxB && pairs <= 32LL * kPlanOneWords) {
        const size_t words = pairs <= kPlanCountMax ? size_t(pairs) : size_t((pairs + 31) / 32);
        e = launch_chained(k_update_plan_one, 1, kPlanOneThreads, words * sizeof(int), st, a);
    } else {
        e = launch_chained(k_update_plan, (a.B + kUpdThreads - 1) / kUpdThreads, kUpdThreads, 0, st, a);
    }
    if (e != cudaSuccess) return e;
    const bool tables = a.warm_layer < 0;  // a warm-up batch has no streams
    const int table_ctas = tables ? (a.S == 1 ? 1 : a.B) : 0;  // a CTA per frame finds out whether its frame is its stream's first
    // Eq. 7: at most min(B, n) classes appear per layer; a CTA per item, and a heavy pair is several items (never
    // more than twice the rows' worth); beyond a few waves of CTAs they stride
    const int pairs_max = std::min(a.B, a.n) * (a.warm_layer >= 0 ? 1 : a.L);
    const int centre_ctas = std::min(pairs_max + pairs_max / 2 + kItemBlocksMax, 16 * sm_count);
    // A memory of many classes is refreshed by a kernel of its own with CTAs of 1024 threads (sorting a thousand
    // keys is 55 rounds of compare-exchange: a round per barrier with 1024 threads, eight times that with the 128
    // threads of a tables CTA); it refreshes every stream, which gives the streams without a frame in the batch
    // the fast memory they already have.
    const bool refresh_apart = tables && rz && a.n > 8 * kApplyThreads;
    const bool refresh_here = tables && rz && !refresh_apart;
    const size_t smem = tables ? tables_smem(a.n, rz ? rz->k_max : 0, refresh_here) : 0;
    ++*launches;
    e = launch_chained(k_update_apply, table_ctas + centre_ctas, kApplyThreads, smem, st, a, rz ? *rz : ResizeArgs{},
                       refresh_here ? 1 : 0, table_ctas);
    if (e != cudaSuccess || !refresh_apart) return e;
    return launch_resize(*rz, st, launches);
}

cudaError_t launch_resize(const ResizeArgs& a, cudaStream_t st, int64_t* launches) {
    ++*launches;
    // a memory of more than 512 and up to 1024 classes gets a thread per class (padded to a power of two): the
    // sort then runs in registers and needs two buffers for the trades; larger ones 1024 threads
    const int cap = pow2_at_least(a.n);
    const int threads = a.n > 4 * kApplyThreads ? std::min(cap, kResizeThreadsMax) : kUpdThreads;
    const size_t smem = refresh_smem(a.n, a.k_max) + (threads == cap ? size_t(cap) * 8 : 0);
    return launch_chained(k_resize, a.S, threads, smem, st, a);
}

}  // namespace smtm
