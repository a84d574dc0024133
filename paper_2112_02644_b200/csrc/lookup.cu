// Memory lookup at one exit layer (Sec. 4.2 Eq. 1-2, Sec. 5 Eq. 3-4): cosine similarity of
// each frame's semantic vector against the members of its fast memory, cumulative
// similarity, top-1 / top-2, accumulated confidence and the exit decision.
//
// One CTA per frame.  The semantic vector is staged in shared memory, each warp takes
// fast-memory slots round-robin and reads the member's centre (L2-resident) with 128-bit
// loads; lanes keep four independent fp32 accumulators and combine with xor-shuffles, so
// every dot product has a fixed evaluation order.  Warp 0 then selects the two best slots.
#include <math.h>

#include <algorithm>

#include "lookup_common.cuh"

namespace smtm {

namespace {

constexpr int kThreads = 256;
constexpr int kFinishThreads = 128;  // decision kernel of the dense route: eight CTAs fit an SM, a frame each

// Any whole number of warps up to kThreads per CTA.
__global__ void __launch_bounds__(kThreads) k_score_exit(const LookupArgs a) {
    extern __shared__ float smem[];
    float* sv = smem;                 // [D]
    float* s_cur = sv + a.D;          // [k_max] similarities of this layer
    float* s_acc = s_cur + a.k_max;   // [k_max] cumulative similarities, then [k_max] the slots' classes
    __shared__ float scratch[32];

    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * (SMTM_PROF_SCORE + a.layer) : nullptr);
    const int b = blockIdx.x;
    const int sid_raw = a.stream_id ? a.stream_id[b] : 0;  // in flight with the exit flag
    if (!a.fresh && a.done[b]) return;  // (a batch that starts here: every frame is in, whatever the flags hold)
    const int tid = threadIdx.x, nthreads = blockDim.x;
    const SlotPrefetch pf = prefetch_slots(a, sid_raw);  // in flight with the semantic vector
    const float* row = a.sv + (size_t)b * a.D;
    float nrm = 0.f;
    for (int d = tid; d < a.D; d += nthreads) {
        const float v = row[d];
        sv[d] = v;
        nrm = fmaf(v, v, nrm);
    }
    nrm = block_sum(nrm, scratch);  // also orders the shared writes above
    score_frame(a, b, pf, sv, nrm, s_cur, s_acc);
}

// The best two keys of the CTA, valid in thread 0.  (b1, b2): this thread's best two; s_keys: [2 * warps].
__device__ __forceinline__ Top2 block_top2_keys(unsigned long long b1, unsigned long long b2, unsigned long long* s_keys) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long k1 = warp_max_u64(b1);
    const unsigned long long k2 = warp_max_u64(b1 == k1 ? b2 : b1);  // keys are unique: the runner-up sits below the winner or elsewhere
    if (lane == 0) {
        s_keys[2 * warp] = k1;
        s_keys[2 * warp + 1] = k2;
    }
    __syncthreads();
    Top2 t{0.f, 0.f, -1, -1};
    if (threadIdx.x == 0) {
        unsigned long long c1 = 0ull, c2 = 0ull;
        for (int i = 0; i < 2 * int(blockDim.x >> 5); ++i) keep_two(s_keys[i], c1, c2);
        rank_key_decode(c1, &t.v1, &t.id1);
        rank_key_decode(c2, &t.v2, &t.id2);
    }
    __syncthreads();
    return t;
}

// Finishing kernel of the tensor-core path: one CTA per frame turns the frame's row of dot products into
// similarities of its fast-memory slots and decides.  The row (both halves of the vector length added) and the
// centres' lengths come in with coalesced 16-byte loads and are parked in shared memory, from where the slots
// pick their class's entry: a gather straight from global memory costs a sector per slot, and a thousand slots
// for each of a thousand frames are then bound by that.  Everything a frame needs after its stream id is fetched
// in one trip: the size and the members of its fast memory, the carries, the row, the lengths and the semantic
// vector (for its length).  Every thread keeps the two best of its own slots as 64-bit ranking keys; warps merge
// by two warp-wide maxima, the CTA through shared memory.  With a.fresh the carry is taken as SA = 0, nobody done.
constexpr int kFinishSlots = 4;  // slots a thread fetches per trip

__global__ void __launch_bounds__(kFinishThreads, 10) k_finish_dense(const LookupArgs a, const float* __restrict__ dots,
                                                                    const float* __restrict__ dots2) {
    extern __shared__ float s_row[];  // [n] dot products, then [n] lengths of the centres
    __shared__ float scratch[32];
    __shared__ unsigned long long s_keys[2 * (kFinishThreads / kWarp)];
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * SMTM_PROF_FINISH_DENSE : nullptr);
    const int b = blockIdx.x, tid = threadIdx.x;
    const int gone = a.fresh ? 0 : a.done[b];
    const int sid = stream_of(a, b);  // (in flight with the flag)
    if (gone) return;
    float* s_len = s_row + a.n;
    const int32_t* mem = a.members + (size_t)max(sid, 0) * a.k_max;
    float* sa_row = a.sa + (size_t)b * a.k_max;
    const float weight = float(1u << a.layer);
    // this trip: the fast memory's size, the first slots' classes and carries (unconditional: up to k_max) ...
    const int k = sid < 0 ? 0 : a.k[sid];  // a stream id outside the cache: nothing to score against
    int cls[kFinishSlots];
    float old[kFinishSlots];
#pragma unroll
    for (int u = 0; u < kFinishSlots; ++u) {
        const int j = min(u * kFinishThreads + tid, a.k_max - 1);
        cls[u] = mem[j];
        old[u] = a.fresh ? 0.f : sa_row[j];
    }
    // ... the row of dot products and the lengths (n is a multiple of 4 on this route) ...
    const float4* drow = reinterpret_cast<const float4*>(dots + (size_t)b * a.n);
    const float4* drow2 = dots2 ? reinterpret_cast<const float4*>(dots2 + (size_t)b * a.n) : nullptr;
    const float4* clen = reinterpret_cast<const float4*>(a.cnorm);
    for (int c4 = tid; c4 < a.n / 4; c4 += kFinishThreads) {
        float4 d = drow[c4];
        if (drow2) {  // second half of the vector length
            const float4 e = drow2[c4];
            d.x += e.x; d.y += e.y; d.z += e.z; d.w += e.w;
        }
        reinterpret_cast<float4*>(s_row)[c4] = d;
        reinterpret_cast<float4*>(s_len)[c4] = clen[c4];
    }
    // ... and the squared length of the semantic vector (D is a multiple of 8 on this route)
    const float4* row4 = reinterpret_cast<const float4*>(a.sv + (size_t)b * a.D);
    float q[4] = {0.f, 0.f, 0.f, 0.f};
    for (int d = tid; d < a.D / 4; d += kFinishThreads) {
        const float4 v = row4[d];
        q[0] = fmaf(v.x, v.x, q[0]);
        q[1] = fmaf(v.y, v.y, q[1]);
        q[2] = fmaf(v.z, v.z, q[2]);
        q[3] = fmaf(v.w, v.w, q[3]);
    }
    const float nrm = block_sum((q[0] + q[1]) + (q[2] + q[3]), scratch);  // (also orders the shared writes above)
    const float sv_len = __fsqrt_rn(nrm);
    unsigned long long a1 = 0ull, a2 = 0ull, c1 = 0ull, c2 = 0ull;  // best two cumulative / single-layer keys
    for (int j0 = 0; j0 < k; j0 += kFinishSlots * kFinishThreads) {
        if (j0 > 0) {  // a fast memory of more than 512 slots: one more trip per 512
#pragma unroll
            for (int u = 0; u < kFinishSlots; ++u) {
                const int j = min(j0 + u * kFinishThreads + tid, a.k_max - 1);
                cls[u] = mem[j];
                old[u] = a.fresh ? 0.f : sa_row[j];
            }
        }
#pragma unroll
        for (int u = 0; u < kFinishSlots; ++u) {
            const int j = j0 + u * kFinishThreads + tid;
            if (j < k) {
                const float dot = s_row[cls[u]], cl = s_len[cls[u]];
                const float sim = (nrm == 0.f || cl == 0.f) ? 0.f : __fdiv_rn(dot, __fmul_rn(sv_len, cl));  // Eq. 1
                const float acc = __fmaf_rn(sim, weight, old[u]);                                              // Eq. 3
                sa_row[j] = acc;
                keep_two(rank_key(acc, cls[u]), a1, a2);
                if (a.sep) keep_two(rank_key(sim, cls[u]), c1, c2);  // only Eq. 2 (a diagnostic) needs it
            }
        }
    }
    if (a.fresh)
        for (int j = k + tid; j < a.k_max; j += kFinishThreads) sa_row[j] = 0.f;  // unused slots start from zero too
    const Top2 ta = block_top2_keys(a1, a2, s_keys);
    Top2 ts{0.f, 0.f, -1, -1};
    if (a.sep) ts = block_top2_keys(c1, c2, s_keys);
    if (tid == 0) decide_from_top2(a, b, ta, ts);
}

__global__ void k_batch_reset(float* __restrict__ sa, uint8_t* __restrict__ done, int32_t* __restrict__ exit_layer,
                              int32_t* __restrict__ pred, int B, long long n_sa) {
    chain_wait();
    chain_release();
    const long long i0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long step = (long long)gridDim.x * blockDim.x;
    for (long long i = i0; i < n_sa; i += step) sa[i] = 0.f;
    for (long long i = i0; i < B; i += step) {
        done[i] = 0;
        exit_layer[i] = 0;
        pred[i] = -1;
    }
}

// The wait of the streaming kernels (mbar_wait_bounded), on a barrier that never completes its phase.
__global__ void k_wait_selftest(int* status) {
    __shared__ uint64_t bar;
    chain_wait();
    chain_release();
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_init_fence();
        mbar_wait_bounded(&bar, 0, status);  // gives up after its limit and records the time-out
    }
}

}  // namespace

cudaError_t launch_wait_selftest(int* status, cudaStream_t st, int64_t* launches) {
    ++*launches;
    return launch_chained(k_wait_selftest, 1, kWarp, 0, st, status);
}

cudaError_t lookup_setup() {
    cudaError_t e = allow_max_dynamic_smem(k_score_exit);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_score_exit);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_finish_dense);
    if (e == cudaSuccess) e = allow_max_dynamic_smem(k_finish_dense);  // (two words per class: 64 KB at 8192 classes)
    return e;
}

cudaError_t launch_batch_reset(float* sa, uint8_t* done, int32_t* exit_layer, int32_t* pred, int B, int k_max,
                               cudaStream_t st, int64_t* launches) {
    if (B <= 0) return cudaSuccess;
    const long long n_sa = (long long)B * k_max;
    const int grid = int(std::min<long long>((n_sa + 255) / 256, 1184));
    ++*launches;
    return launch_chained(k_batch_reset, grid, 256, 0, st, sa, done, exit_layer, pred, B, n_sa);
}

cudaError_t launch_finish_dense(const LookupArgs& a, const float* dots, const float* dots2, bool beside_pooling,
                                cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    ++*launches;
    const size_t smem = 2 * size_t(a.n) * sizeof(float);
    if (beside_pooling) return launch_ordered(k_finish_dense, a.B, kFinishThreads, smem, st, a, dots, dots2);
    return launch_chained(k_finish_dense, a.B, kFinishThreads, smem, st, a, dots, dots2);
}

cudaError_t launch_score_exit(const LookupArgs& a, cudaStream_t st, int64_t* launches, int threads) {
    if (a.B <= 0) return cudaSuccess;
    const size_t smem = (size_t(a.D) + 3 * size_t(a.k_max)) * sizeof(float);
    ++*launches;
    return launch_chained(k_score_exit, a.B, threads > 0 ? threads : kThreads, smem, st, a);
}

}  // namespace smtm
