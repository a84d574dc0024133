// Adaptive priming memory (Sec. 6): frequency / time-stamp tables, running-mean centres
// (Eq. 7), replacement score and top-k (Eq. 5), adaptive fast-memory size (Eq. 6).
//
// All floating-point reductions are segmented and atomics-free: one owner walks the batch in
// ascending frame index, so the result is the one a frame-by-frame replay would give and does
// not depend on scheduling.
//
// An update is three launches on two streams.  The plan kernel writes every frame's final label
// and stop layer and lists the (layer, class) pairs Eq. 7 has to touch: up to 4096 frames and
// 65 536 pairs a single CTA elects the pairs in a shared-memory bitmap (k_update_plan_one); past
// that k_update_plan does it with many CTAs (the first frame to stamp a pair with the call's
// sequence number appends it; the number is kept on the device and moved on by the kernel
// itself, so that a replayed CUDA graph counts on exactly like eager calls).  The CTAs of
// k_update_centers then walk that list.  k_update_tables depends on neither:
// a warp per frame checks whether an earlier frame of the batch belongs to the same stream and
// leaves if so, else it applies the stream's frames to the stream's tables (staged in shared memory)
// and, when asked, refreshes the stream's fast memory (Eq. 5 / Eq. 6).  It runs on a side
// stream, forked before the plan and joined after the centres, so the two halves of the update
// overlap.  Classes and streams the batch does not touch cost nothing.
#include <algorithm>

#include "common.cuh"
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

constexpr int kUpdThreads = 256;
constexpr int kUpdWarps = kUpdThreads / kWarp;
constexpr int kTblWarps = 16;  // warps (streams) to a CTA of k_update_tables in its warp-per-stream form
constexpr int kTblGroups = 16;  // groups of 32 frames a warp looks up per trip to memory

// The label a finished frame ends up with: the prediction if it exited, else the fallback label
// (the full network's answer, -1 = none); a label outside the memory counts as no label.
__device__ __forceinline__ int final_label_of(const UpdateArgs& a, int b) {
    const int lab = (a.done && a.done[b] != 0) ? a.pred[b] : (a.fallback ? a.fallback[b] : -1);
    return lab >= a.n ? -1 : lab;
}

// ---- plan -----------------------------------------------------------------------------------

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
        a.plan.final_label[b] = lab;
        a.plan.stop_layer[b] = ex ? el : a.L;
        if (lab >= 0) {
            // Eq. 7 touches the layers up to the stop layer: the first frame to stamp (layer, class)
            // with the call's number lists the pair as a job
            const int l_lo = a.warm_layer >= 0 ? a.warm_layer : 0;
            const int l_hi = a.warm_layer >= 0 ? a.warm_layer + 1 : (ex ? el : a.L);
            for (int l = l_lo; l < l_hi; ++l)
                if (atomicExch(a.plan.class_tag + (size_t)l * a.n + lab, epoch) != epoch)
                    a.plan.jobs[atomicAdd(a.plan.job_count + (epoch & 1), 1)] = (l << 16) | lab;
        }
    }
    if (b == 0) a.plan.job_count[(epoch + 1) & 1] = 0;  // the next call's counter (the call before this one is over)
    // the last CTA through makes the number current for the kernels that follow and publishes the
    // number of jobs (every CTA's appends are complete and visible before its ticket)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && atomicAdd(a.plan.epoch + 1, 1ull) == gridDim.x - 1) {
        __threadfence();
        a.plan.job_count[2] = *reinterpret_cast<volatile int32_t*>(a.plan.job_count + (epoch & 1));
        a.plan.epoch[1] = 0;
        a.plan.epoch[0] = epoch;
    }
}

// The same plan by a single CTA, for batches and memories small enough that one CTA's trip to
// memory is all it takes: the pairs are elected in a bitmap in shared memory and counted there, so
// nothing waits on a ticket or a fence.
constexpr int kPlanOneThreads = 1024;
constexpr int kPlanOneMaxB = 4 * kPlanOneThreads;
constexpr int kPlanOneWords = 2048;  // 65 536 (layer, class) pairs

__global__ void __launch_bounds__(kPlanOneThreads) k_update_plan_one(const UpdateArgs a) {
    __shared__ unsigned int s_seen[kPlanOneWords];
    __shared__ int s_jobs;
    const int tid = threadIdx.x;
    for (int i = tid; i < (a.L * a.n + 31) / 32; i += kPlanOneThreads) s_seen[i] = 0u;
    if (tid == 0) s_jobs = 0;
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
        a.plan.final_label[b] = lab;
        a.plan.stop_layer[b] = ex ? el : a.L;
        if (lab >= 0) {
            const int l_lo = a.warm_layer >= 0 ? a.warm_layer : 0;
            const int l_hi = a.warm_layer >= 0 ? a.warm_layer + 1 : (ex ? el : a.L);
            for (int l = l_lo; l < l_hi; ++l) {
                const int pair = l * a.n + lab;
                const unsigned int bit = 1u << (pair & 31);
                if (!(atomicOr(&s_seen[pair >> 5], bit) & bit)) a.plan.jobs[atomicAdd(&s_jobs, 1)] = (l << 16) | lab;
            }
        }
    }
    __syncthreads();
    if (tid == 0) a.plan.job_count[2] = s_jobs;
}

// ---- Eq. 5 / Eq. 6 ------------------------------------------------------------------------

__device__ __forceinline__ unsigned long long score_of(int ft, int ts, int W, int forgetting = 0) {
    if (forgetting) return (unsigned long long)max(ft, 0);  // the decay already sits in the table
    int e = ts / W;
    if (e > kEMax) e = kEMax;
    const unsigned long long f = (unsigned long long)min(max(ft, 0), kFtMax);
    return f << (2 * (kEMax - e));  // FT * 4^(12 - e) = 4^12 * FT * 0.25^e
}

__host__ __device__ constexpr size_t resize_smem(int n, int k_max) { return size_t(n) * 8 + size_t(n + (n & 1)) * 4 + size_t(k_max) * 8; }
// The one-CTA-per-stream refresh sorts: its score and id arrays are padded to a power of two.
__host__ __device__ constexpr int pow2_at_least(int v) {
    int p = 2;
    while (p < v) p *= 2;
    return p;
}
__host__ __device__ constexpr size_t resize_cta_smem(int n, int k_max) {
    return size_t(pow2_at_least(n)) * 12 + size_t(k_max) * 8;
}

// Refresh of one stream's fast memory by a CTA of kUpdThreads threads.  Classes with a
// non-zero score are compacted in ascending id and ranked among themselves by counting;
// zero-score classes follow in ascending id.  `smem` holds resize_cta_smem(n, k_max) bytes.
__device__ void resize_stream(const ResizeArgs& a, int s, unsigned char* smem, int* s_scan,
                              unsigned long long* s_part) {
    unsigned long long* s_score = reinterpret_cast<unsigned long long*>(smem);  // [n] compacted non-zero scores
    const int cap = pow2_at_least(a.n);                                         // both arrays hold `cap` entries
    int* s_id = reinterpret_cast<int*>(s_score + cap);                          // their class ids
    unsigned long long* s_top = reinterpret_cast<unsigned long long*>(s_id + cap);  // [k_max]
    const int tid = threadIdx.x;
    const int32_t* ft = a.ft + (size_t)s * a.n;
    const int32_t* ts = a.ts + (size_t)s * a.n;
    int32_t* mem = a.members + (size_t)s * a.k_max;

    // pass 1: compact the non-zero scores (ascending id) and add everything up
    int nz = 0;
    unsigned long long local = 0;
    for (int c0 = 0; c0 < a.n; c0 += kUpdThreads) {
        const int c = c0 + tid;
        const unsigned long long sc = c < a.n ? score_of(ft[c], ts[c], a.W, a.forgetting) : 0ull;
        int cnt;
        const int pos = block_exclusive_scan(sc != 0 ? 1 : 0, s_scan, &cnt);
        if (sc != 0) {
            s_score[nz + pos] = sc;
            s_id[nz + pos] = c;
        }
        nz += cnt;
        local += sc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(kFull, local, o);
    __syncthreads();
    if ((tid & 31) == 0) s_part[tid >> 5] = local;
    __syncthreads();
    unsigned long long total = 0;
    for (int w = 0; w < kUpdThreads / 32; ++w) total += s_part[w];
    if (total == 0) return;  // nothing seen yet: keep size and members

    // pass 2: order the non-zero classes by (score descending, id ascending): a bitonic sort of the
    // pairs, padded to a power of two with entries that rank last; rank r < k_max goes to slot r
    const int P = pow2_at_least(nz);
    for (int i = nz + tid; i < P; i += kUpdThreads) {
        s_score[i] = 0ull;
        s_id[i] = INT32_MAX;
    }
    __syncthreads();
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < P / 2; t += kUpdThreads) {
                const int i = 2 * j * (t / j) + (t % j), l = i + j;
                const unsigned long long si = s_score[i], sl = s_score[l];
                const int ii = s_id[i], il = s_id[l];
                const bool l_first = sl > si || (sl == si && il < ii);  // the entry at l ranks before the one at i
                if (((i & k) == 0) ? l_first : !l_first) {             // (ids are distinct: never equal)
                    s_score[i] = sl; s_score[l] = si;
                    s_id[i] = il; s_id[l] = ii;
                }
            }
            __syncthreads();
        }
    }
    for (int r = tid; r < nz && r < a.k_max; r += kUpdThreads) {
        mem[r] = s_id[r];
        s_top[r] = s_score[r];
    }
    // pass 3: zero-score classes fill the remaining slots in ascending id
    if (nz < a.k_max) {
        int filled = nz;
        for (int c0 = 0; c0 < a.n && filled < a.k_max; c0 += kUpdThreads) {
            const int c = c0 + tid;
            const int z = (c < a.n && score_of(ft[c], ts[c], a.W, a.forgetting) == 0) ? 1 : 0;
            int cnt;
            const int pos = block_exclusive_scan(z, s_scan, &cnt);
            if (z && filled + pos < a.k_max) {
                mem[filled + pos] = c;
                s_top[filled + pos] = 0;
            }
            filled += cnt;
        }
    }
    __syncthreads();
    // pass 4: smallest k in [k_min, k_max] with cl_den * prefix(k) > cl_num * total
    if (tid < kWarp) {  // warp 0: a scan of 32 entries per step
        const int lane = tid;
        unsigned long long carry = 0;
        int chosen = a.k_max;
        for (int base = 0; base < a.k_max; base += kWarp) {
            const int idx = base + lane;
            unsigned long long v = idx < a.k_max ? s_top[idx] : 0ull;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(kFull, v, o);
                if (lane >= o) v += t;
            }
            const unsigned long long prefix = carry + v;
            const bool ok = idx < a.k_max && idx + 1 >= a.k_min &&
                            (unsigned long long)a.cl_den * prefix > (unsigned long long)a.cl_num * total;
            const unsigned m = __ballot_sync(kFull, ok);
            if (m) {
                chosen = base + __ffs(m);
                break;
            }
            carry += __shfl_sync(kFull, v, 31);
        }
        if (lane == 0) a.k[s] = chosen;
    }
}

__global__ void __launch_bounds__(kUpdThreads) k_resize(const ResizeArgs a) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[kUpdThreads / 32];
    chain_wait();
    chain_release();
    resize_stream(a, blockIdx.x, reinterpret_cast<unsigned char*>(s_dyn), s_scan, s_part);
}

// ---- apply ------------------------------------------------------------------------------------

// Compacts, in ascending frame index, the frames of a tile of kUpdThreads for which `hit`
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

// Sec. 6.1 for the stream whose first frame in the batch is g, by one warp with the stream's
// tables in registers (class c lives in lane c % 32, register c / 32), then, if asked, that
// stream's Eq. 5 / Eq. 6 refresh.  `smem` is this warp's resize_smem(n, k_max) bytes.
// 16 bytes from global to shared memory without passing through registers (both addresses 16-byte
// aligned); the thread goes on and collects all of its copies with copy_async_wait_all().
__device__ __forceinline__ void copy_async_16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void copy_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// The stream's tables are staged in shared memory (class c belongs to lane c % 32) and every pass
// over the classes is a rolled loop: the kernel runs once per warp, so its time is the time to
// fetch its instructions, and unrolled loops over registers were several times slower.
__host__ __device__ constexpr size_t tables_smem(int n, int k_max) { return resize_smem(n, k_max) + size_t(n + (n & 1)) * 8; }

__device__ void tables_by_warp(const UpdateArgs& a, const ResizeArgs& rz, int g, int s, int do_resize,
                               unsigned char* smem, int* s_hits) {
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
    int32_t* ftp = a.ft + (size_t)s * a.n;
    int32_t* tsp = a.ts + (size_t)s * a.n;
    int* s_ft = reinterpret_cast<int*>(smem + resize_smem(a.n, rz.k_max));  // [n]
    int* s_ts = s_ft + a.n + (a.n & 1);                                     // [n]
    // Staged by 16-byte asynchronous copies where the rows allow it: every copy is in flight at once and
    // lands while the stream's frames are being looked up below.
    const bool staged_async = (a.n & 3) == 0 && ((reinterpret_cast<uintptr_t>(ftp) | reinterpret_cast<uintptr_t>(tsp) |
                                                   smem_u32(s_ft) | smem_u32(s_ts)) & 15) == 0;
    if (staged_async) {
        for (int v = lane; v < a.n / 4; v += kWarp) {
            copy_async_16(s_ft + 4 * v, ftp + 4 * v);
            copy_async_16(s_ts + 4 * v, tsp + 4 * v);
        }
    } else {
#pragma unroll 4
        for (int c = lane; c < a.n; c += kWarp) {
            s_ft[c] = ftp[c];
            s_ts[c] = tsp[c];
        }
    }
    // Plain counts have a closed form (see the one-CTA-per-stream variant in k_update_tables): per class
    // the number of appearances and the position of the last one, gathered in the space the refresh
    // uses afterwards.  The forgetting table is replayed frame by frame.
    const bool plain = a.forget_W == 0;
    int* s_cnt = reinterpret_cast<int*>(smem);  // [n]
    int* s_last = s_cnt + a.n;                  // [n]
    if (plain)
        for (int c = lane; c < a.n; c += kWarp) {
            s_cnt[c] = 0;
            s_last[c] = -1;
        }
    __syncwarp();
    int m = 0;  // frames of the stream so far
    // The stream's frames in ascending index (none precedes g), kTblGroups groups of 32 frames per trip
    // to memory: their labels are listed in order (s_hits, this warp's), then applied.
    for (int b0 = g - g % kWarp; b0 < a.B; b0 += kTblGroups * kWarp) {
        int sidv[kTblGroups], labv[kTblGroups];
#pragma unroll
        for (int u = 0; u < kTblGroups; ++u) {  // unconditional loads (a clamped index), all in flight at once
            const int bb = min(b0 + u * kWarp + lane, a.B - 1);
            sidv[u] = a.stream_id ? a.stream_id[bb] : 0;
            const int dn = a.done ? a.done[bb] : 0, pr = a.done ? a.pred[bb] : -1, fb = a.fallback ? a.fallback[bb] : -1;
            const int lab = dn != 0 ? pr : fb;  // final_label_of with every load issued up front
            labv[u] = lab >= a.n ? -1 : lab;
        }
        int n_hits = 0;
#pragma unroll
        for (int u = 0; u < kTblGroups; ++u) {
            const int b = b0 + u * kWarp + lane;
            const bool hit = b >= g && b < a.B && sidv[u] == s;
            const unsigned mask = __ballot_sync(kFull, hit);
            if (hit) s_hits[n_hits + __popc(mask & lt)] = labv[u];
            n_hits += __popc(mask);
        }
        __syncwarp();
        if (!plain && staged_async) {  // the replay works on the staged tables
            copy_async_wait_all();
            __syncwarp();
        }
        if (plain) {
            for (int h = lane; h < n_hits; h += kWarp) {
                const int l = s_hits[h];
                if (l >= 0) {
                    atomicAdd(&s_cnt[l], 1);
                    atomicMax(&s_last[l], m + h);
                }
            }
        } else {
#pragma unroll 1
            for (int h = 0; h < n_hits; ++h) {
                const int l = s_hits[h];
#pragma unroll 2
                for (int c = lane; c < a.n; c += kWarp) table_step(s_ft[c], s_ts[c], c == l, a.forget_W);
            }
        }
        m += n_hits;
        __syncwarp();
    }
    if (staged_async) {
        copy_async_wait_all();
        __syncwarp();
    }
    if (plain)
        for (int c = lane; c < a.n; c += kWarp) {
            const int q = s_cnt[c];
            if (q > 0) {
                s_ft[c] = int(min((long long)s_ft[c] + q, (long long)kFtMax));
                s_ts[c] = m - 1 - s_last[c];
            } else {
                s_ts[c] = int(min((long long)s_ts[c] + m, (long long)INT32_MAX));
            }
        }
    __syncwarp();
#pragma unroll 4
    for (int c = lane; c < a.n; c += kWarp) {
        ftp[c] = s_ft[c];
        tsp[c] = s_ts[c];
    }
    if (!do_resize) return;

    // Eq. 5 scores; non-zero ones compacted in ascending class id
    unsigned long long* s_score = reinterpret_cast<unsigned long long*>(smem);  // [n]
    int* s_id = reinterpret_cast<int*>(s_score + a.n);                          // [n]
    unsigned long long* s_top = reinterpret_cast<unsigned long long*>(s_id + a.n + (a.n & 1));  // [k_max]
    int32_t* mem = rz.members + (size_t)s * rz.k_max;
    unsigned long long total = 0;
    int nz = 0;
#pragma unroll 1
    for (int c0 = 0; c0 < a.n; c0 += kWarp) {
        const int c = c0 + lane;
        const unsigned long long sc = c < a.n ? score_of(s_ft[c], s_ts[c], rz.W, rz.forgetting) : 0ull;
        const unsigned m = __ballot_sync(kFull, sc != 0);
        if (sc != 0) {
            const int pos = nz + __popc(m & lt);
            s_score[pos] = sc;
            s_id[pos] = c;
        }
        nz += __popc(m);
        total += sc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(kFull, total, o);
    if (total == 0) return;  // nothing seen yet: keep size and members
    __syncwarp();
    // rank the non-zero classes by counting; rank r < k_max goes to slot r
    for (int i = lane; i < nz; i += kWarp) {
        const unsigned long long sc = s_score[i];
        int r0 = 0, r1 = 0, r2 = 0, r3 = 0;  // four counters: the loop is a chain of additions otherwise
        int j = 0;
        for (; j + 3 < nz; j += 4) {
            const unsigned long long o0 = s_score[j], o1 = s_score[j + 1], o2 = s_score[j + 2], o3 = s_score[j + 3];
            r0 += (o0 > sc || (o0 == sc && j < i)) ? 1 : 0;  // compacted order is ascending id
            r1 += (o1 > sc || (o1 == sc && j + 1 < i)) ? 1 : 0;
            r2 += (o2 > sc || (o2 == sc && j + 2 < i)) ? 1 : 0;
            r3 += (o3 > sc || (o3 == sc && j + 3 < i)) ? 1 : 0;
        }
        for (; j < nz; ++j) {
            const unsigned long long o = s_score[j];
            r0 += (o > sc || (o == sc && j < i)) ? 1 : 0;
        }
        const int r = (r0 + r1) + (r2 + r3);
        if (r < rz.k_max) {
            mem[r] = s_id[i];
            s_top[r] = sc;
        }
    }
    // zero-score classes fill the remaining slots in ascending id
    int filled = nz;
#pragma unroll 1
    for (int c0 = 0; c0 < a.n && filled < rz.k_max; c0 += kWarp) {
        const int c = c0 + lane;
        const bool z = c < a.n && score_of(s_ft[c], s_ts[c], rz.W, rz.forgetting) == 0;
        const unsigned m = __ballot_sync(kFull, z);
        if (z) {
            const int pos = filled + __popc(m & lt);
            if (pos < rz.k_max) {
                mem[pos] = c;
                s_top[pos] = 0;
            }
        }
        filled += __popc(m);
    }
    __syncwarp();
    // Eq. 6: smallest k in [k_min, k_max] with cl_den * prefix(k) > cl_num * total
    unsigned long long carry = 0;
    int chosen = rz.k_max;
    for (int base = 0; base < rz.k_max; base += kWarp) {
        const int idx = base + lane;
        unsigned long long v = idx < rz.k_max ? s_top[idx] : 0ull;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(kFull, v, o);
            if (lane >= o) v += t;
        }
        const unsigned long long prefix = carry + v;
        const bool ok = idx < rz.k_max && idx + 1 >= rz.k_min &&
                        (unsigned long long)rz.cl_den * prefix > (unsigned long long)rz.cl_num * total;
        const unsigned m = __ballot_sync(kFull, ok);
        if (m) {
            chosen = base + __ffs(m);
            break;
        }
        carry += __shfl_sync(kFull, v, 31);
    }
    if (lane == 0) rz.k[s] = chosen;
}

// Tables (and, if asked, the refresh) of the streams whose first frames are among this CTA's
// frames: a warp per frame, or, when the classes do not fit a warp's registers, the whole CTA
// for one frame.
__global__ void __launch_bounds__(kTblWarps * kWarp) k_update_tables(const UpdateArgs a, const ResizeArgs rz, int do_resize,
                                                               int warp_tables) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_list[kUpdThreads];
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[kUpdWarps];
    __shared__ int s_hits[kTblWarps][kTblGroups * kWarp];  // labels of a stream's frames among 512 consecutive ones, per warp
    const int tid = threadIdx.x;
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_TABLES : nullptr, true);
    {
        if (warp_tables) {
            const int g = blockIdx.x * (blockDim.x >> 5) + (tid >> 5);  // the launch decides how many warps share a CTA
            if (g >= a.B) return;
            const int s = a.stream_id ? a.stream_id[g] : 0;
            if (s < 0 || s >= a.S) return;  // no such stream: nothing to update (the plan kernel records the error)
            // not the stream's first frame in the batch: the warp of that frame does the work
            bool earlier = !a.stream_id && g > 0;
            for (int b0 = 0; a.stream_id && b0 < g && !earlier; b0 += kTblGroups * kWarp) {
                bool same = false;
#pragma unroll
                for (int u = 0; u < kTblGroups; ++u) {  // unconditional loads (a clamped index), all in flight at once
                    const int bb = b0 + u * kWarp + (tid & 31);
                    same |= a.stream_id[min(bb, g)] == s && bb < g;
                }
                earlier = __any_sync(kFull, same);
            }
            if (earlier) return;
            tables_by_warp(a, rz, g, s, do_resize,
                           reinterpret_cast<unsigned char*>(s_dyn) + size_t(tid >> 5) * tables_smem(a.n, rz.k_max),
                           s_hits[tid >> 5]);
            return;
        }
        // ---- Sec. 6.1 by a whole CTA: the stream's frames, ascending, replayed per class -------
        const int g = blockIdx.x;
        const int s = a.stream_id ? a.stream_id[g] : 0;
        if (s < 0 || s >= a.S) return;  // no such stream (the same for every thread of the CTA)
        int earlier = (!a.stream_id && g > 0) ? 1 : 0;  // an earlier frame of the same stream: its CTA does the work
        for (int b = tid; a.stream_id && b < g; b += kUpdThreads) earlier |= a.stream_id[b] == s ? 1 : 0;
        if (__syncthreads_or(earlier)) return;
        if (a.forget_W == 0) {
            // Plain counts: what a frame-by-frame replay leaves behind has a closed form per class.  With
            // m frames of the stream in the batch, a class that appears q times, last at position p, ends
            // with FT + q and TS = m - 1 - p; one that does not appear ends with TS + m.  q and p are
            // gathered by shared-memory atomics on integers (a sum and a maximum: order does not matter).
            int* s_cnt = reinterpret_cast<int*>(s_dyn);  // [n]; the refresh below reuses the space
            int* s_last = s_cnt + a.n;                   // [n]
            for (int c = tid; c < a.n; c += kUpdThreads) {
                s_cnt[c] = 0;
                s_last[c] = -1;
            }
            __syncthreads();
            int m = 0;
            for (int t0 = g - g % kUpdThreads; t0 < a.B; t0 += kUpdThreads) {
                const int b = t0 + tid;
                const int hit = (b < a.B && (a.stream_id ? a.stream_id[b] : 0) == s) ? 1 : 0;
                const int cnt = compact_tile(hit, hit ? final_label_of(a, b) : -1, s_list, s_scan);
                if (tid < cnt && s_list[tid] >= 0) {
                    atomicAdd(&s_cnt[s_list[tid]], 1);
                    atomicMax(&s_last[s_list[tid]], m + tid);
                }
                m += cnt;
            }
            __syncthreads();
            for (int c = tid; c < a.n; c += kUpdThreads) {
                const size_t at = (size_t)s * a.n + c;
                const int q = s_cnt[c];
                if (q > 0) {
                    a.ft[at] = int(min((long long)a.ft[at] + q, (long long)kFtMax));
                    a.ts[at] = m - 1 - s_last[c];
                } else {
                    a.ts[at] = int(min((long long)a.ts[at] + m, (long long)INT32_MAX));
                }
            }
        } else {
            for (int t0 = g - g % kUpdThreads; t0 < a.B; t0 += kUpdThreads) {
                const int b = t0 + tid;
                const int hit = (b < a.B && (a.stream_id ? a.stream_id[b] : 0) == s) ? 1 : 0;
                const int cnt = compact_tile(hit, hit ? final_label_of(a, b) : -1, s_list, s_scan);
                if (cnt == 0) continue;
                for (int c = tid; c < a.n; c += kUpdThreads) {
                    int f = a.ft[(size_t)s * a.n + c], t = a.ts[(size_t)s * a.n + c];
                    for (int i = 0; i < cnt; ++i) table_step(f, t, s_list[i] == c, a.forget_W);
                    a.ft[(size_t)s * a.n + c] = f;
                    a.ts[(size_t)s * a.n + c] = t;
                }
            }
        }
        if (do_resize) {
            __syncthreads();  // this CTA's table writes are visible to all of its threads
            resize_stream(rz, s, reinterpret_cast<unsigned char*>(s_dyn), s_scan, s_part);
        }
    }
}

// Eq. 7 over the jobs (layer, class) listed by the plan kernel, taken round-robin by CTAs of
// 1024 threads.  The frames' labels and stop layers are staged in shared memory once; per job the
// matching frames are listed in ascending index (every thread looks at a run of consecutive
// frames, one block scan), then thread = (four columns, group): group r folds the listed frames
// r, r + 4, ... with eight rows in flight, the four groups are added in a fixed order, and the
// centre, its length and its count are rewritten.  Nothing here waits on another CTA.
constexpr int kCenThreads = 1024;
constexpr int kCenCols = kCenThreads;        // columns per sweep: 256 threads x 4 columns, four groups
constexpr int kCenTile = 2 * kCenThreads;    // frames staged and listed at a time

// Lists, in ascending index, the frames of the staged tile whose label is cls and that stopped at
// layer l0 + 1 or deeper; returns how many.  s_code[i] = label | stop layer << 16, or -1.
__device__ __forceinline__ int list_frames(const int* s_code, int tile_frames, int cls, int l0, int* s_list, int* s_scan) {
    const int per = (tile_frames + kCenThreads - 1) / kCenThreads;  // consecutive frames per thread (1 or 2)
    const int f0 = threadIdx.x * per;
    int mine = 0;
    for (int i = 0; i < per; ++i) {
        const int code = f0 + i < tile_frames ? s_code[f0 + i] : -1;
        mine += (code >= 0 && (code & 0xffff) == cls && (code >> 16) >= l0 + 1) ? 1 : 0;
    }
    int cnt;
    int pos = block_exclusive_scan(mine, s_scan, &cnt);
    for (int i = 0; i < per && mine; ++i) {
        const int code = f0 + i < tile_frames ? s_code[f0 + i] : -1;
        if (code >= 0 && (code & 0xffff) == cls && (code >> 16) >= l0 + 1) s_list[pos++] = f0 + i;
    }
    __syncthreads();
    return cnt;
}

__global__ void __launch_bounds__(kCenThreads, 1) k_update_centers(const UpdateArgs a) {
    __shared__ int s_code[kCenTile];
    __shared__ int s_list[kCenTile];
    __shared__ float4 s_acc[3][kCenCols / 4];
    __shared__ int s_scan[33];
    __shared__ float s_red[32];
    const int tid = threadIdx.x;
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_CENTERS : nullptr);
    const bool single = a.B <= kCenTile;  // the whole batch fits one tile: staged once, listed once per job
    const auto stage = [&](int base) {
        for (int i = tid; i < kCenTile && base + i < a.B; i += kCenThreads) {
            const int lab = a.plan.final_label[base + i], stop = a.plan.stop_layer[base + i];
            s_code[i] = lab < 0 ? -1 : (lab | (stop << 16));
        }
        __syncthreads();
    };
    const int n_jobs = a.plan.job_count[2];
    int next_code = a.plan.jobs[blockIdx.x];  // (the list has room for every pair) in flight with the count and the labels
    if (single) stage(0);
    const int cg = tid & (kCenCols / 4 - 1), grp = tid / (kCenCols / 4);
    for (int job = blockIdx.x; job < n_jobs; job += gridDim.x) {
        const int cls = next_code & 0xffff, l0 = next_code >> 16;  // l0 is 0-based; the paper's is l0 + 1
        if (job + int(gridDim.x) < n_jobs) next_code = a.plan.jobs[job + gridDim.x];
        const int D = a.dims[l0];
        const bool vec = (D & 3) == 0;  // rows are 16-byte aligned
        const float* sv = a.sv[l0];
        float* cen = a.centers[l0] + (size_t)cls * D;
        int cnt = single ? list_frames(s_code, a.B, cls, l0, s_list, s_scan) : 0;
        float nrm = 0.f;
        int q = 0;
        for (int d0 = 0; d0 < D; d0 += kCenCols) {  // a sweep of columns, four per thread
            const int d = d0 + cg * 4;
            float old[4] = {0.f, 0.f, 0.f, 0.f};  // the centre and its count as they are, fetched along with the rows
            uint32_t m = 0;
            if (grp == 0) {
                m = a.m[l0][cls];
                for (int j = 0; j < 4; ++j)
                    if (d + j < D) old[j] = cen[d + j];
            }
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            q = 0;
            for (int base = 0; base < a.B; base += kCenTile) {
                if (!single) {
                    __syncthreads();  // the previous tile's readers are done with the staged codes and the list
                    stage(base);
                    cnt = list_frames(s_code, min(kCenTile, a.B - base), cls, l0, s_list, s_scan);
                }
                q += cnt;
                if (d >= D) continue;
                if (vec) {
                    // eight rows in flight per thread; each group adds its rows in ascending frame order
                    for (int i0 = grp; i0 < cnt; i0 += 32) {
                        float4 r[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)  // unconditional loads (past the end: the last row again, unused)
                            r[u] = __ldg(reinterpret_cast<const float4*>(
                                sv + (size_t)(base + s_list[min(i0 + 4 * u, cnt - 1)]) * D + d));
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            if (i0 + 4 * u < cnt) {
                                acc[0] += r[u].x; acc[1] += r[u].y; acc[2] += r[u].z; acc[3] += r[u].w;
                            }
                        }
                    }
                } else {
                    for (int i = grp; i < cnt; i += 4)
                        for (int j = 0; j < 4; ++j)
                            if (d + j < D) acc[j] += sv[(size_t)(base + s_list[i]) * D + d + j];
                }
            }
            if (q == 0) break;  // cannot happen for a listed job; kept so that nothing divides by the old count alone
            // the groups' sums in a fixed order: ((g0 + g1) + g2) + g3
            __syncthreads();
            if (grp > 0) s_acc[grp - 1][cg] = make_float4(acc[0], acc[1], acc[2], acc[3]);
            __syncthreads();
            if (grp == 0 && d < D) {
#pragma unroll
                for (int g = 0; g < 3; ++g) {
                    const float4 o = s_acc[g][cg];
                    acc[0] += o.x; acc[1] += o.y; acc[2] += o.z; acc[3] += o.w;
                }
                for (int j = 0; j < 4; ++j)
                    if (d + j < D) {
                        // Eq. 7 in double: the count is exact at any size and SC m + sum SV is rounded once
                        const float v = float((double(old[j]) * double(m) + double(acc[j])) / (double(m) + double(q)));
                        cen[d + j] = v;
                        nrm = fmaf(v, v, nrm);
                    }
            }
        }
        if (q == 0) continue;
        nrm = block_sum(nrm, s_red);  // also separates the reads of the count above from its update below
        if (tid == 0) {
            a.cnorm[l0][cls] = __fsqrt_rn(nrm);
            a.m[l0][cls] += (uint32_t)q;
            if (a.split_current) a.split_current[l0] = 0;  // the tensor-core scorer's copy of this layer's centres is stale
        }
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
    const cudaError_t e = allow_max_dynamic_smem(k_update_tables);
    return e != cudaSuccess ? e : allow_max_dynamic_smem(k_resize);
}

cudaError_t launch_center_norms(const float* centers, int n, int D, float* cnorm, cudaStream_t st,
                                int64_t* launches) {
    ++*launches;
    return launch_chained(k_center_norms, n, 256, 0, st, centers, n, D, cnorm);
}

cudaError_t launch_update(const UpdateArgs& a, const ResizeArgs* rz, int sm_count, cudaStream_t st, cudaStream_t side,
                          cudaEvent_t fork, cudaEvent_t join, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    // a warp per frame when eight streams' tables and refresh buffers fit a CTA's shared memory
    const size_t per_warp = tables_smem(a.n, rz ? rz->k_max : 0);
    const bool warp_tables = per_warp * kUpdWarps <= 100 * 1024;
    // one CTA per stream: the refresh buffers, and at least the two integer arrays [n] of the closed-form tables
    // Sixteen warps to a CTA when their buffers fit: the CTAs of k_update_centers fill an SM's registers, so
    // every SM a tables CTA sits on is one that Eq. 7 cannot use until the tables are done (512 streams: 32
    // SMs for the tables, 116 for the centres; with eight warps to a CTA it was 64 and 84)
    const int warps = !warp_tables ? kUpdWarps : (per_warp * kTblWarps <= 180 * 1024 ? kTblWarps : kUpdWarps);
    const size_t smem = warp_tables ? per_warp * warps
                                    : std::max<size_t>(rz ? resize_cta_smem(a.n, rz->k_max) : 0, size_t(a.n) * 2 * sizeof(int));
    cudaError_t e = cudaSuccess;
    const bool tables = a.warm_layer < 0;  // a warm-up batch has no streams
    const int table_ctas = warp_tables ? (a.B + warps - 1) / warps : a.B;
    if (tables) {
        // the tables need nothing of the plan: they run beside plan + centres on the side stream
        // (inside a stream capture the side stream joins the capture through the events)
        if ((e = cudaEventRecord(fork, st)) != cudaSuccess) return e;
        if ((e = cudaStreamWaitEvent(side, fork, 0)) != cudaSuccess) return e;
        ++*launches;
        e = launch_chained(k_update_tables, table_ctas, warps * kWarp, smem, side, a,
                           rz ? *rz : ResizeArgs{}, rz ? 1 : 0, warp_tables ? 1 : 0);
        if (e != cudaSuccess) return e;
        if ((e = cudaEventRecord(join, side)) != cudaSuccess) return e;
    }
    ++*launches;
    if (a.B <= kPlanOneMaxB && (long long)a.L * a.n <= 32LL * kPlanOneWords)
        e = launch_chained(k_update_plan_one, 1, kPlanOneThreads, 0, st, a);
    else
        e = launch_chained(k_update_plan, (a.B + kUpdThreads - 1) / kUpdThreads, kUpdThreads, 0, st, a);
    if (e != cudaSuccess) return e;
    // Eq. 7: at most min(B, n) classes appear per layer; a CTA of 1024 threads per (layer, class) job, one per SM
    // A centres CTA fills an SM's registers, and plan + centres start before the side stream's tables do:
    // with a centres CTA on every SM the tables wait until some have left.  Up to a quarter of the SMs are
    // left to the tables' CTAs.
    const int table_sms = tables && warp_tables ? std::min(table_ctas, sm_count / 4) : 0;
    const int centre_ctas = std::min(std::min(a.B, a.n) * (a.warm_layer >= 0 ? 1 : a.L), sm_count - table_sms);
    ++*launches;
    e = launch_chained(k_update_centers, centre_ctas, kCenThreads, 0, st, a);
    if (e != cudaSuccess) return e;
    return tables ? cudaStreamWaitEvent(st, join, 0) : cudaSuccess;
}

cudaError_t launch_resize(const ResizeArgs& a, cudaStream_t st, int64_t* launches) {
    const size_t smem = resize_cta_smem(a.n, a.k_max);
    ++*launches;
    return launch_chained(k_resize, a.S, kUpdThreads, smem, st, a);
}

}  // namespace smtm
