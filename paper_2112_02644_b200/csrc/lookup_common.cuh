// Decision logic shared by the lookup kernels: ranking, top-1 / top-2, the margin ratio of
// Eq. 2 / Eq. 4 and the exit rule (Sec. 4.2, Sec. 5).
#pragma once

#include <math.h>

#include "common.cuh"
#include "internal.h"

namespace smtm {

// Ranking used for top-1 / top-2: NaN ranks last, larger value first, ties -> lower class id.
__device__ __forceinline__ bool ranks_before(float va, int ida, float vb, int idb) {
    const bool na = isnan(va), nb = isnan(vb);
    if (na != nb) return nb;
    if (!na && va != vb) return va > vb;
    return ida < idb;
}

// The fast memory frame b looks up: its stream id, or -1 (and an invalid-argument code in the status word)
// when the id lies outside [0, S).  Such a frame is scored against nothing, stays in, and is left out of
// the update.
__device__ __forceinline__ int stream_checked(const LookupArgs& a, int sid) {
    if (sid >= 0 && sid < a.S) return sid;
    set_status(a.status, kDevInvalidArg);
    return -1;
}
__device__ __forceinline__ int stream_of(const LookupArgs& a, int b) {
    return stream_checked(a, a.stream_id ? a.stream_id[b] : 0);
}

struct Top2 {
    float v1, v2;
    int id1, id2;  // class ids, -1 = absent
};

// (top - second) / second with the sign cases: top <= 0 -> 0; second NaN -> NaN; second <= 0 < top -> +inf.
__device__ __forceinline__ float ratio_margin(float top, float second) {
    if (!(top > 0.f)) return 0.f;
    if (isnan(second)) return __int_as_float(0x7fc00000);
    if (!(second > 0.f)) return INFINITY;
    return __fdiv_rn(__fsub_rn(top, second), second);
}

__device__ __forceinline__ void decide_from_top2(const LookupArgs& a, int b, const Top2& ta, const Top2& ts);
__device__ __forceinline__ float cosine_from(float dot, float sv_norm2, float center_len);

// ---- top-2 through one 64-bit key per entry ------------------------------------------------------
//
// The ranking (NaN last, larger value first, ties -> lower class id) as an unsigned comparison:
// the value's bits made monotone in the upper half (-0 counts as +0, NaN as the smallest), the
// complement of the class id in the lower half.  Key 0 = no entry.
__device__ __forceinline__ unsigned long long rank_key(float v, int id) {
    uint32_t hi = 0u;
    if (!isnan(v)) {
        const uint32_t u = __float_as_uint(v + 0.f);
        hi = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    return ((unsigned long long)hi << 32) | (unsigned long long)(0xffffffffu - uint32_t(id));
}

__device__ __forceinline__ void rank_key_decode(unsigned long long key, float* v, int* id) {
    if (key == 0ull) {
        *v = 0.f;
        *id = -1;
        return;
    }
    const uint32_t hi = uint32_t(key >> 32);
    *v = __uint_as_float((hi & 0x80000000u) ? (hi & 0x7fffffffu) : ~hi);
    *id = int(0xffffffffu - uint32_t(key));
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long t = __shfl_xor_sync(kFull, v, o);
        v = t > v ? t : v;
    }
    return v;
}

// Keeps the two largest keys seen so far.
__device__ __forceinline__ void keep_two(unsigned long long e, unsigned long long& b1, unsigned long long& b2) {
    if (e > b1) {
        b2 = b1;
        b1 = e;
    } else if (e > b2) {
        b2 = e;
    }
}

// Best two of v[0..k) with classes ids[0..k) (any k), executed by one full warp: every lane keeps the best two keys of
// its own slots, then two warp-wide maxima (keys are distinct: the runner-up sits below the winner in the
// winner's lane or is some lane's best).
__device__ __forceinline__ Top2 warp_top2_by_keys(const float* v, const int32_t* ids, int k, int lane) {
    unsigned long long b1 = 0ull, b2 = 0ull;
    for (int j = lane; j < k; j += kWarp) keep_two(rank_key(v[j], ids[j]), b1, b2);
    const unsigned long long k1 = warp_max_u64(b1);
    const unsigned long long k2 = warp_max_u64(b1 == k1 ? b2 : b1);
    Top2 t;
    rank_key_decode(k1, &t.v1, &t.id1);
    rank_key_decode(k2, &t.v2, &t.id2);
    return t;
}

// Best two of values held in registers (lane l holds slots l and l + 32 of k), by two warp-wide
// maxima over the keys: the same result as pushing every entry through top2_push and merging by
// shuffles, in a fraction of the instructions.
__device__ __forceinline__ Top2 warp_top2_keys(const float (&v)[2], const int (&ids)[2], int k, int lane) {
    const unsigned long long e0 = lane < k ? rank_key(v[0], ids[0]) : 0ull;
    const unsigned long long e1 = lane + kWarp < k ? rank_key(v[1], ids[1]) : 0ull;
    const unsigned long long k1 = warp_max_u64(e0 > e1 ? e0 : e1);
    const unsigned long long c0 = e0 == k1 ? 0ull : e0, c1 = e1 == k1 ? 0ull : e1;  // keys are unique: ids differ
    const unsigned long long k2 = warp_max_u64(c0 > c1 ? c0 : c1);
    Top2 t;
    rank_key_decode(k1, &t.v1, &t.id1);
    rank_key_decode(k2, &t.v2, &t.id2);
    return t;
}

// Executed by one full warp once the similarities of frame b are known: s_cur[j] (this
// layer, Eq. 1) and s_acc[j] (cumulative, Eq. 3) for the k slots whose classes are mem[j].
// Selects the two best of each, evaluates Eq. 4 / Eq. 2 and the exit rule in fp32, and
// writes the frame's outputs and the counters.
__device__ __forceinline__ void decide_frame(const LookupArgs& a, int b, const float* s_cur, const float* s_acc,
                                             const int32_t* mem, int k, int lane) {
    const Top2 ta = warp_top2_by_keys(s_acc, mem, k, lane);
    Top2 ts{0.f, 0.f, -1, -1};
    if (a.sep) ts = warp_top2_by_keys(s_cur, mem, k, lane);  // only Eq. 2 (a diagnostic) needs it
    if (lane != 0) return;
    decide_from_top2(a, b, ta, ts);
}

// Lane-0 part of the decision without the global counters: Eq. 4 / Eq. 2 from the two best
// cumulative (ta) and single-layer (ts) similarities, the exit rule in fp32 and the frame's
// outputs.  Returns bit 0 = the frame exits, bit 1 = its AC lies within 1e-4 of the threshold.
__device__ __forceinline__ int decide_core(const LookupArgs& a, int b, const Top2& ta, const Top2& ts) {
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
    if (leave) {
        a.done[b] = 1;
        a.exit_layer[b] = a.layer + 1;
        a.pred[b] = ta.id1;
    } else if (a.fresh) {  // the reset state of a frame that stays in
        a.done[b] = 0;
        a.exit_layer[b] = 0;
        a.pred[b] = -1;
    }
    const int near = (isfinite(ac) && fabsf(ac - a.tau) <= 1e-4f) ? 2 : 0;
    return (leave ? 1 : 0) | near;
}

// The same with the counters added straight to global memory.
__device__ __forceinline__ void decide_from_top2(const LookupArgs& a, int b, const Top2& ta, const Top2& ts) {
    const int r = decide_core(a, b, ta, ts);
    atomicAdd(&a.counters[SMTM_CTR_LOOKUPS], 1ull);
    if (r & 2) atomicAdd(&a.counters[SMTM_CTR_NEAR], 1ull);
    if (r & 1) atomicAdd(&a.counters[SMTM_CTR_EXITS + a.layer], 1ull);
}

// Scores frame b against the members of its fast memory and decides, by a whole CTA (any whole number of
// warps): pf is what prefetch_slots returned for the frame's stream id, sv the frame's semantic vector in shared memory (already visible to every thread), nrm its squared
// length; s_cur and s_acc hold k_max floats each and s_acc is followed by k_max more words (the slots' classes).  Each warp takes fast-memory slots round-robin and reads the
// member's centre (L2-resident) with 128-bit loads; lanes keep four independent fp32 accumulators and combine
// with xor-shuffles, so every dot product has a fixed evaluation order.  Warp 0 then selects the two best.
// The kernel's time is the number of dependent trips to memory: the size of the fast memory and the warp's
// first class come in one trip, and a slot's centre, its length, its carry and the next slot's class in one more.
// What score_frame needs of the frame's fast memory before it can fetch a centre: its size and this warp's
// first class.  Fetched early (the loads only need the stream id), so that they are in flight with the
// caller's own loads (the semantic vector, or the map that is being pooled).
struct SlotPrefetch {
    int sid, k, cls;
};
__device__ __forceinline__ SlotPrefetch prefetch_slots(const LookupArgs& a, int sid_raw) {
    SlotPrefetch pf;
    pf.sid = stream_checked(a, sid_raw);
    const int32_t* mem = a.members + (size_t)max(pf.sid, 0) * a.k_max;
    pf.cls = mem[min(int(threadIdx.x >> 5), a.k_max - 1)];  // unconditional: in flight with the size
    pf.k = pf.sid < 0 ? 0 : a.k[pf.sid];                     // a stream id outside the cache: nothing to score against
    return pf;
}

__device__ __forceinline__ void score_frame(const LookupArgs& a, int b, const SlotPrefetch& pf, const float* sv, float nrm,
                                            float* s_cur, float* s_acc) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nw = nthreads / kWarp;
    int32_t* s_ids = reinterpret_cast<int32_t*>(s_acc + a.k_max);  // the slots' classes, for the decision
    const int32_t* mem = a.members + (size_t)max(pf.sid, 0) * a.k_max;
    int cls_next = pf.cls;
    const int k = pf.k;
    const float weight = float(1u << a.layer);   // 2^(l-1) with l = layer + 1
    const int D4 = (a.D & 3) ? 0 : a.D >> 2;     // 128-bit loads need rows that are multiples of 16 bytes
    const float4* v4 = reinterpret_cast<const float4*>(sv);
    for (int j = warp; j < k; j += nw) {
        const int cls = cls_next;
        const float4* c4 = reinterpret_cast<const float4*>(a.centers + (size_t)cls * a.D);
        float cl = 0.f, old = 0.f;
        if (lane == 0) {  // issued with the centre's loads
            cl = a.cnorm[cls];
            old = a.fresh ? 0.f : a.sa[(size_t)b * a.k_max + j];
        }
        if (j + nw < k) cls_next = mem[j + nw];
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
        for (int i0 = 0; i0 < D4; i0 += 8 * kWarp) {  // eight pieces per lane in flight
            float4 c[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) c[u] = __ldg(c4 + min(i0 + u * kWarp + lane, D4 - 1));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * kWarp + lane;
                if (i < D4) {
                    const float4 v = v4[i];
                    d0 = fmaf(c[u].x, v.x, d0); d1 = fmaf(c[u].y, v.y, d1); d2 = fmaf(c[u].z, v.z, d2); d3 = fmaf(c[u].w, v.w, d3);
                }
            }
        }
        for (int i = (D4 << 2) + lane; i < a.D; i += kWarp) d0 = fmaf(a.centers[(size_t)cls * a.D + i], sv[i], d0);
        float dot = (d0 + d1) + (d2 + d3);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(kFull, dot, o);
        if (lane == 0) {
            const float s = cosine_from(dot, nrm, cl);    // Eq. 1
            const float acc = __fmaf_rn(s, weight, old);  // Eq. 3
            a.sa[(size_t)b * a.k_max + j] = acc;
            s_cur[j] = s;
            s_acc[j] = acc;
            s_ids[j] = cls;
        }
    }
    if (a.fresh)
        for (int j = k + tid; j < a.k_max; j += nthreads) a.sa[(size_t)b * a.k_max + j] = 0.f;  // unused slots start from zero too
    __syncthreads();
    if (warp != 0) return;
    decide_frame(a, b, s_cur, s_acc, s_ids, k, lane);
}

// Eq. 1 from a dot product and the two lengths; a zero-length vector is similar to nothing.
__device__ __forceinline__ float cosine_from(float dot, float sv_norm2, float center_len) {
    return (sv_norm2 == 0.f || center_len == 0.f) ? 0.f
                                                  : __fdiv_rn(dot, __fmul_rn(__fsqrt_rn(sv_norm2), center_len));
}

}  // namespace smtm
