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

#include "common.cuh"
#include "internal.h"

namespace smtm {

namespace {

constexpr int kThreads = 256;

// Ranking used for top-1 / top-2: NaN ranks last, larger value first, ties -> lower class id.
__device__ __forceinline__ bool ranks_before(float va, int ida, float vb, int idb) {
    const bool na = isnan(va), nb = isnan(vb);
    if (na != nb) return nb;
    if (!na && va != vb) return va > vb;
    return ida < idb;
}

struct Top2 {
    float v1, v2;
    int id1, id2;  // class ids, -1 = absent
};

__device__ __forceinline__ void top2_push(Top2& t, float v, int id) {
    if (t.id1 < 0 || ranks_before(v, id, t.v1, t.id1)) {
        t.v2 = t.v1; t.id2 = t.id1;
        t.v1 = v; t.id1 = id;
    } else if (t.id2 < 0 || ranks_before(v, id, t.v2, t.id2)) {
        t.v2 = v; t.id2 = id;
    }
}

// Best two of the values v[0..k) with class ids ids[0..k); executed by one full warp.
__device__ __forceinline__ Top2 warp_top2(const float* v, const int32_t* ids, int k, int lane) {
    Top2 t{0.f, 0.f, -1, -1};
    for (int j = lane; j < k; j += kWarp) top2_push(t, v[j], ids[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov1 = __shfl_xor_sync(kFull, t.v1, o), ov2 = __shfl_xor_sync(kFull, t.v2, o);
        const int oi1 = __shfl_xor_sync(kFull, t.id1, o), oi2 = __shfl_xor_sync(kFull, t.id2, o);
        if (oi1 >= 0) top2_push(t, ov1, oi1);
        if (oi2 >= 0) top2_push(t, ov2, oi2);
    }
    return t;
}

// (top - second) / second with the sign cases: top <= 0 -> 0; second <= 0 < top -> +inf.
__device__ __forceinline__ float ratio_margin(float top, float second) {
    if (!(top > 0.f)) return 0.f;
    if (!(second > 0.f)) return INFINITY;
    return __fdiv_rn(__fsub_rn(top, second), second);
}

__global__ void __launch_bounds__(kThreads) k_score_exit(const LookupArgs a) {
    extern __shared__ float smem[];
    float* sv = smem;                 // [D]
    float* s_cur = sv + a.D;          // [k_max] similarities of this layer
    float* s_acc = s_cur + a.k_max;   // [k_max] cumulative similarities
    __shared__ float scratch[32];

    const int b = blockIdx.x;
    if (a.done[b]) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sid = a.stream_id ? a.stream_id[b] : 0;
    const int k = a.k[sid];
    const int32_t* mem = a.members + (size_t)sid * a.k_max;
    const float* row = a.sv + (size_t)b * a.D;

    float nrm = 0.f;
    for (int d = tid; d < a.D; d += kThreads) {
        const float v = row[d];
        sv[d] = v;
        nrm = fmaf(v, v, nrm);
    }
    nrm = block_sum(nrm, scratch);  // also orders the shared writes above
    const float sv_len = __fsqrt_rn(nrm);

    const float weight = float(1u << a.layer);  // 2^(l-1) with l = layer + 1
    const int D4 = (a.D & 3) ? 0 : a.D >> 2;  // 128-bit loads need rows that are multiples of 16 bytes
    for (int j = warp; j < k; j += kThreads / kWarp) {
        const int cls = mem[j];
        const float4* c4 = reinterpret_cast<const float4*>(a.centers + (size_t)cls * a.D);
        const float4* v4 = reinterpret_cast<const float4*>(sv);
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
        for (int i = lane; i < D4; i += kWarp) {
            const float4 c = __ldg(c4 + i);
            const float4 v = v4[i];
            d0 = fmaf(c.x, v.x, d0); d1 = fmaf(c.y, v.y, d1); d2 = fmaf(c.z, v.z, d2); d3 = fmaf(c.w, v.w, d3);
        }
        for (int i = (D4 << 2) + lane; i < a.D; i += kWarp) d0 = fmaf(a.centers[(size_t)cls * a.D + i], sv[i], d0);
        float dot = (d0 + d1) + (d2 + d3);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(kFull, dot, o);
        if (lane == 0) {
            const float cl = a.cnorm[cls];
            const float s = (nrm == 0.f || cl == 0.f) ? 0.f : __fdiv_rn(dot, __fmul_rn(sv_len, cl));  // Eq. 1
            const float acc = __fmaf_rn(s, weight, a.sa[(size_t)b * a.k_max + j]);                     // Eq. 3
            a.sa[(size_t)b * a.k_max + j] = acc;
            s_cur[j] = s;
            s_acc[j] = acc;
        }
    }
    __syncthreads();
    if (warp != 0) return;

    const Top2 ta = warp_top2(s_acc, mem, k, lane);
    const Top2 ts = warp_top2(s_cur, mem, k, lane);
    if (lane != 0) return;
    float ac = 0.f, sep = 0.f;
    bool leave = false;
    if (ta.id2 >= 0) {
        ac = ratio_margin(ta.v1, ta.v2);   // Eq. 4
        sep = ratio_margin(ts.v1, ts.v2);  // Eq. 2
        leave = (ta.v1 > 0.f) && (__fsub_rn(ta.v1, ta.v2) > __fmul_rn(a.tau, fmaxf(ta.v2, 0.f)));
    }
    if (a.ac) a.ac[(size_t)b * a.L + a.layer] = ac;
    if (a.sep) a.sep[(size_t)b * a.L + a.layer] = sep;
    if (a.top) {
        a.top[2 * b] = ta.id1;
        a.top[2 * b + 1] = ta.id2;
    }
    atomicAdd(&a.counters[SMTM_CTR_LOOKUPS], 1ull);
    if (isfinite(ac) && fabsf(ac - a.tau) <= 1e-4f) atomicAdd(&a.counters[SMTM_CTR_NEAR], 1ull);
    if (leave) {
        a.done[b] = 1;
        a.exit_layer[b] = a.layer + 1;
        a.pred[b] = ta.id1;
        atomicAdd(&a.counters[SMTM_CTR_EXITS + a.layer], 1ull);
    }
}

__global__ void k_batch_reset(float* __restrict__ sa, uint8_t* __restrict__ done, int32_t* __restrict__ exit_layer,
                              int32_t* __restrict__ pred, int B, long long n_sa) {
    const long long i0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const long long step = (long long)gridDim.x * blockDim.x;
    for (long long i = i0; i < n_sa; i += step) sa[i] = 0.f;
    for (long long i = i0; i < B; i += step) {
        done[i] = 0;
        exit_layer[i] = 0;
        pred[i] = -1;
    }
}

}  // namespace

cudaError_t launch_batch_reset(float* sa, uint8_t* done, int32_t* exit_layer, int32_t* pred, int B, int k_max,
                               cudaStream_t st, int64_t* launches) {
    if (B <= 0) return cudaSuccess;
    const long long n_sa = (long long)B * k_max;
    const int grid = int(std::min<long long>((n_sa + 255) / 256, 1184));
    ++*launches;
    k_batch_reset<<<grid, 256, 0, st>>>(sa, done, exit_layer, pred, B, n_sa);
    return cudaGetLastError();
}

cudaError_t launch_score_exit(const LookupArgs& a, cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    const size_t smem = (size_t(a.D) + 2 * size_t(a.k_max)) * sizeof(float);
    static size_t opted = 48 * 1024;
    if (smem > opted) {
        cudaError_t e = cudaFuncSetAttribute(k_score_exit, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        opted = smem;
    }
    ++*launches;
    k_score_exit<<<a.B, kThreads, smem, st>>>(a);
    return cudaGetLastError();
}

}  // namespace smtm
