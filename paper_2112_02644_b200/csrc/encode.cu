// Semantic-vector encoding (Sec. 4.1): SV[b][c] = mean over H x W of the feature map.
//
// The feature maps are read exactly once from HBM; this is the only step of the hot path
// whose traffic grows with C*H*W, so everything here is organised around streaming.
//
// NCHW.  A frame is a flat run of C channels of H*W elements.  Channels are grouped into
// "units": the smallest number G of consecutive channels whose bytes are a multiple of 16
// (7x7 bf16: 8 channels = 784 B).  A persistent CTA per SM runs a ring of shared-memory
// stages; one producer thread fills stages with 1-D bulk asynchronous copies of whole
// chunks (a run of units, <= 25 KB) completing on an mbarrier, and eight consumer warps each
// reduce the chunks of their own stages and write the channel means straight to SV.
// Chunks partition channels, so no two warps ever touch the same output: no atomics, and
// the summation order of every channel is fixed.
//   * unit-per-lane reducer (H*W small and odd-sized): lane i owns unit i of the chunk and
//     walks its 16-byte vectors; the stride between lanes is an odd number of vectors, so the
//     128-bit shared loads are conflict-free; the element -> channel map is resolved at compile time.
//   * team-per-channel reducer (channel bytes a multiple of 16): T lanes share a channel,
//     stride over its vectors and combine with xor-shuffles.
// NHWC.  Consecutive 16-byte vectors of a frame are consecutive channel groups of a pixel;
// each thread owns one channel group and a pixel phase, loads coalesced 128-bit vectors
// directly and the phases are combined through shared memory in ascending order.
// Any other shape falls back to a plain thread-per-(frame, channel) loop.
#include <algorithm>
#include <cmath>

#include "lookup_common.cuh"

namespace smtm {

namespace {

constexpr int kStages = 8;             // ring depth
constexpr int kConsumers = 8;          // consumer warps; stage s belongs to warp s % kConsumers
constexpr int kStageCap = 25600;       // bytes per stage
constexpr int kThreadsTma = (kConsumers + 1) * kWarp;
constexpr size_t kSmemTma = size_t(kStages) * kStageCap + 2 * kStages * sizeof(uint64_t) + 128;

struct NchwParams {
    const uint8_t* x;
    const uint8_t* skip;
    float* sv;
    __nv_bfloat16* sv_hi;    // optional bf16 head and tail of sv (sv = hi + lo), same indexing; may be null
    __nv_bfloat16* sv_lo;
    int* status;
    long long total_chunks;  // B * chunks per frame
    int C;
    int chunks_per_frame;
    int chunk_channels;      // channels in a full chunk
    int ch_bytes;            // bytes of one channel
    long long frame_bytes;
    float inv_hw;
    int team;                // team-per-channel: lanes per channel (power of two)
    int vec_per_channel;     // team-per-channel: 16-byte vectors per channel
    int max_in_flight;       // copies the producer keeps outstanding (<= kStages)
};

// Writes the bf16 head and tail of n consecutive values (n a multiple of 2, dst 4-byte aligned).
template <int N>
__device__ __forceinline__ void store_split(const float (&v)[N], __nv_bfloat16* hi, __nv_bfloat16* lo) {
#pragma unroll
    for (int g = 0; g < N; g += 2) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(v[g]), h1 = __float2bfloat16_rn(v[g + 1]);
        const __nv_bfloat16 l0 = __float2bfloat16_rn(v[g] - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16_rn(v[g + 1] - __bfloat162float(h1));
        *reinterpret_cast<__nv_bfloat162*>(hi + g) = __nv_bfloat162(h0, h1);
        *reinterpret_cast<__nv_bfloat162*>(lo + g) = __nv_bfloat162(l0, l1);
    }
}

// ---- reducers --------------------------------------------------------------------------

// Lane i reduces unit i: G channels of HW elements stored as UW consecutive 16-byte vectors.
template <class E, int HW>
struct UnitPerLane {
    static constexpr int kUnitBytesRaw = HW * E::kSize;
    static constexpr int gcd16(int a) { return (a % 16 == 0) ? 16 : (a % 8 == 0) ? 8 : (a % 4 == 0) ? 4 : (a % 2 == 0) ? 2 : 1; }
    static constexpr int G = 16 / gcd16(kUnitBytesRaw);
    static constexpr int UW = G * kUnitBytesRaw / 16;

    static __device__ __forceinline__ void run(const uint8_t* stage, int nch, int lane, float* out, float* out_s,
                                               float inv_hw, const NchwParams& p) {
        const int units = nch / G;
        if (lane >= units) return;
        const uint4* u = reinterpret_cast<const uint4*>(stage) + lane * UW;
        float acc[G];
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] = 0.f;
#pragma unroll
        for (int i = 0; i < UW; ++i) {
            const uint4 v = u[i];
#pragma unroll
            for (int j = 0; j < E::kPerVec; ++j) acc[(i * E::kPerVec + j) / HW] += E::at(v, j);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] *= inv_hw;
        float* o = out + lane * G;  // G floats, aligned to G * 4 bytes
        if (G == 2) {
            *reinterpret_cast<float2*>(o) = make_float2(acc[0], acc[1]);
        } else {
#pragma unroll
            for (int g = 0; g + 3 < G; g += 4)
                *reinterpret_cast<float4*>(o + g) = make_float4(acc[g], acc[g + 1], acc[g + 2], acc[g + 3]);
        }
        if (p.sv_hi) {
            const ptrdiff_t at = (o - p.sv);
            store_split<G>(acc, p.sv_hi + at, p.sv_lo + at);
        }
        if (out_s) {
            float* os = out_s + lane * G;
            if (G == 2) {
                *reinterpret_cast<float2*>(os) = make_float2(acc[0], acc[1]);
            } else {
#pragma unroll
                for (int g = 0; g + 3 < G; g += 4)
                    *reinterpret_cast<float4*>(os + g) = make_float4(acc[g], acc[g + 1], acc[g + 2], acc[g + 3]);
            }
        }
    }
};

// T lanes per channel; channel bytes are a multiple of 16.
template <class E>
struct TeamPerChannel {
    static __device__ __forceinline__ void run(const uint8_t* stage, int nch, int lane, float* out, float* out_s,
                                               float inv_hw, const NchwParams& p) {
        const int T = p.team, uw = p.vec_per_channel;
        const int per_pass = kWarp / T;
        const int team = lane / T, r = lane - team * T;
        const int passes = (nch + per_pass - 1) / per_pass;
        for (int ps = 0; ps < passes; ++ps) {
            const int c = ps * per_pass + team;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            if (c < nch) {
                const uint4* u = reinterpret_cast<const uint4*>(stage) + size_t(c) * uw;
                for (int i = r; i < uw; i += T) {
                    const uint4 v = u[i];
                    if (E::kPerVec == 4) {
                        a0 += E::at(v, 0); a1 += E::at(v, 1); a2 += E::at(v, 2); a3 += E::at(v, 3);
                    } else {
                        a0 += E::at(v, 0); a1 += E::at(v, 1); a2 += E::at(v, 2); a3 += E::at(v, 3);
                        a0 += E::at(v, 4); a1 += E::at(v, 5); a2 += E::at(v, 6); a3 += E::at(v, 7);
                    }
                }
            }
            float s = (a0 + a1) + (a2 + a3);
            for (int o = T >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(kFull, s, o);
            if (c < nch && r == 0) {
                const float v = s * inv_hw;
                out[c] = v;
                if (out_s) out_s[c] = v;
                if (p.sv_hi) {
                    const ptrdiff_t at = (out + c) - p.sv;
                    const __nv_bfloat16 h = __float2bfloat16_rn(v);
                    p.sv_hi[at] = h;
                    p.sv_lo[at] = __float2bfloat16_rn(v - __bfloat162float(h));
                }
            }
        }
    }
};

// ---- persistent bulk-copy pipeline -------------------------------------------------------

template <class R>
__global__ void __launch_bounds__(kThreadsTma, 1) k_encode_nchw(const NchwParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint8_t* stages = base;
    uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(kStages) * kStageCap);
    uint64_t* empty = full + kStages;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init_fence();
    }
    chain_release();
    __syncthreads();
    chain_wait();  // the barriers are set up while the previous kernel finishes

    const bool producer = warp == kConsumers;  // last warp; lane 0 issues the copies
    int it = 0;                                // chunks of this CTA that are not skipped, so far
    bool failed = false;
    if (!producer || lane == 0) {
        for (long long g = blockIdx.x; g < p.total_chunks; g += gridDim.x) {
            const int b = int(g / p.chunks_per_frame);
            if (p.skip && p.skip[b]) continue;
            const int ci = int(g - (long long)b * p.chunks_per_frame);
            const int stage = it % kStages;
            const uint32_t use = uint32_t(it / kStages);
            const int c0 = ci * p.chunk_channels;
            const int nch = min(p.chunk_channels, p.C - c0);
            if (producer) {
                if (use > 0 && !mbar_wait_bounded(&empty[stage], (use - 1) & 1, p.status)) {
                    failed = true;
                    break;
                }
                if (it >= p.max_in_flight) {  // bound the bytes in flight: wait for an older copy to land
                    const int old = it - p.max_in_flight;
                    if (!mbar_wait_bounded(&full[old % kStages], (old / kStages) & 1, p.status)) {
                        failed = true;
                        break;
                    }
                }
                const uint32_t bytes = uint32_t(nch) * uint32_t(p.ch_bytes);
                mbar_expect_tx(&full[stage], bytes);
                bulk_load(stages + size_t(stage) * kStageCap,
                          p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes, bytes, &full[stage]);
            } else if (stage % kConsumers == warp) {
                if (!mbar_wait_bounded(&full[stage], use & 1, p.status)) {
                    failed = true;
                    break;
                }
                R::run(stages + size_t(stage) * kStageCap, nch, lane, p.sv + (long long)b * p.C + c0, nullptr, p.inv_hw, p);
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[stage]);
            }
            ++it;
        }
    }
    // No thread leaves before every copy that was issued has landed: shared memory must
    // stay allocated until the copy engine is done with it.
    const int any_failed = __syncthreads_or(failed ? 1 : 0);
    if (any_failed && producer && lane == 0) {
        for (int s = 0; s < kStages && s < it; ++s) {
            const uint32_t last_use = uint32_t((it - 1 - s) / kStages);
            mbar_wait_bounded(&full[s], last_use & 1, p.status);
        }
    }
}

// ---- fused lookup: encode + similarity scoring in one persistent kernel -----------------------
//
// Work is cut into units: (frame, part), a part being a run of chunks_per_unit chunks, i.e. a
// slice of the frame's channels.  Every CTA first compacts the frames that are still active
// and takes the units u = blockIdx.x, blockIdx.x + gridDim.x, ... of that list, so exited
// frames cost nothing and the load is even.  Per unit the reducer warps leave the slice of
// the semantic vector in shared memory (four buffers) as well as in the SV stash; eight dot
// warps then share the unit's dot products, slot j on warp j % 8: each lane has every load of
// its slot's centre slice in flight at once, so a unit costs one trip to L2.  The partial dot
// products and the partial squared length go to global scratch [frame][part][slot]; the small
// finishing kernel in lookup.cu adds the parts up in part order and decides.  No atomics:
// the evaluation order of every sum is fixed.
constexpr int kReducersF = 4;       // reducer warps of the fused kernel; stage s belongs to warp s % kReducersF
constexpr int kDotWarps = 8;        // warps that share the dot products of a unit
constexpr int kSvBufs = 4;          // shared-memory slices; unit u passes through buffer u % kSvBufs
constexpr int kThreadsFused = (kReducersF + 1 + kDotWarps) * kWarp;
constexpr int kMaxUnits = 1024;     // units per CTA
constexpr int kMaxSlice = 1024;     // floats of a semantic-vector slice (eight 16-byte vectors per lane)
static_assert(kStages % kReducersF == 0, "stage ownership must be periodic");

struct FusedParams {
    NchwParams e;
    LookupArgs a;
    int parts;            // P: parts per frame (divides chunks_per_frame)
    int chunks_per_unit;  // chunks_per_frame / P
    int slice_cap;        // channels of a full slice = chunks_per_unit * chunk_channels (multiple of 4)
    float* partials;      // [B][P][k_max + 1]: partial dot products per slot, then the partial squared length
};

constexpr size_t fused_smem(int slice_cap) {
    return size_t(kStages) * kStageCap + size_t(kSvBufs) * size_t(slice_cap) * 4 + kMaxUnits * 4 +
           (2 * kStages + 2 * kSvBufs) * 8 + 40 * 4 + 192;
}

template <class R>
__global__ void __launch_bounds__(kThreadsFused, 1) k_lookup_nchw(const FusedParams f) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint8_t* stages = base;
    float* sv_s = reinterpret_cast<float*>(base + size_t(kStages) * kStageCap);  // [kSvBufs][slice_cap]
    int* my_units = reinterpret_cast<int*>(sv_s + kSvBufs * f.slice_cap);        // [kMaxUnits]
    int* s_scan = my_units + kMaxUnits;                                          // [40]
    uint64_t* full = reinterpret_cast<uint64_t*>(
        (reinterpret_cast<uintptr_t>(s_scan + 40) + 7) & ~uintptr_t(7));         // [kStages]
    uint64_t* empty = full + kStages;                                            // [kStages]
    uint64_t* sv_full = empty + kStages;                                         // [kSvBufs]  slice written
    uint64_t* sv_empty = sv_full + kSvBufs;                                      // [kSvBufs]  slice read by all dot warps

    const NchwParams& p = f.e;
    const LookupArgs& a = f.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int P = f.parts, cpu = f.chunks_per_unit;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int s = 0; s < kSvBufs; ++s) {
            mbar_init(&sv_full[s], cpu);
            mbar_init(&sv_empty[s], kDotWarps);
        }
        mbar_init_fence();
    }
    chain_release();

    // ---- the active frames and this CTA's share of their units -----------------------------
    int n_active = a.fresh ? a.B : 0;  // a batch that starts here has every frame active: no flags to read
    for (int idx = threadIdx.x; a.fresh && idx < kMaxUnits; idx += kThreadsFused) {
        const long long u = (long long)blockIdx.x + (long long)idx * gridDim.x;
        if (u < (long long)a.B * P) my_units[idx] = int(u / P) * kMaxParts + int(u % P);
    }
    chain_wait();  // everything above touched shared memory only and overlaps the previous kernel's tail
    for (int t0 = 0; !a.fresh && t0 < a.B; t0 += kThreadsFused) {
        const int b = t0 + threadIdx.x;
        const int act = (b < a.B && !a.done[b]) ? 1 : 0;
        int cnt;
        const int pos = block_exclusive_scan(act, s_scan, &cnt);
        if (act) {
            for (int part = 0; part < P; ++part) {
                const int u = (n_active + pos) * P + part;
                if (u % int(gridDim.x) == int(blockIdx.x)) {
                    const int idx = u / int(gridDim.x);
                    if (idx < kMaxUnits) my_units[idx] = b * kMaxParts + part;
                }
            }
        }
        n_active += cnt;
    }
    const int total_units = n_active * P;
    int nu = total_units > int(blockIdx.x) ? (total_units - int(blockIdx.x) + int(gridDim.x) - 1) / int(gridDim.x) : 0;
    nu = min(nu, kMaxUnits);
    __syncthreads();

    const int n_chunks = nu * cpu;
    bool failed = false;
    int issued = 0;
    if (warp < kReducersF) {
        // ---- reducers: warp w owns the stages w, w + kReducersF, ... -----------------------------
        for (int it = warp; it < n_chunks; it += kReducersF) {
            const int i = it / cpu, c = it - i * cpu;
            const int unit = my_units[i], b = unit / kMaxParts, part = unit % kMaxParts;
            const int c0 = (part * cpu + c) * p.chunk_channels;
            const int nch = min(p.chunk_channels, p.C - c0);
            const int stage = it % kStages;
            const int buf = i % kSvBufs, round = i / kSvBufs;
            if (round > 0 && !mbar_wait_bounded(&sv_empty[buf], (round - 1) & 1, p.status)) { failed = true; break; }
            if (!mbar_wait_bounded(&full[stage], (it / kStages) & 1, p.status)) { failed = true; break; }
            R::run(stages + size_t(stage) * kStageCap, nch, lane, p.sv + (long long)b * p.C + c0,
                   sv_s + buf * f.slice_cap + c * p.chunk_channels, p.inv_hw, p);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&empty[stage]);
                mbar_arrive(&sv_full[buf]);
            }
        }
    } else if (warp == kReducersF) {
        // ---- producer -------------------------------------------------------------------------
        if (lane == 0) {
            for (int it = 0; it < n_chunks; ++it) {
                const int i = it / cpu, c = it - i * cpu;
                const int unit = my_units[i], b = unit / kMaxParts, part = unit % kMaxParts;
                const int c0 = (part * cpu + c) * p.chunk_channels;
                const int nch = min(p.chunk_channels, p.C - c0);
                const int stage = it % kStages;
                const uint32_t use = uint32_t(it / kStages);
                if (use > 0 && !mbar_wait_bounded(&empty[stage], (use - 1) & 1, p.status)) { failed = true; break; }
                if (it >= p.max_in_flight) {  // bound the bytes in flight: wait for an older copy to land
                    const int old = it - p.max_in_flight;
                    if (!mbar_wait_bounded(&full[old % kStages], (old / kStages) & 1, p.status)) { failed = true; break; }
                }
                const uint32_t bytes = uint32_t(nch) * uint32_t(p.ch_bytes);
                mbar_expect_tx(&full[stage], bytes);
                bulk_load(stages + size_t(stage) * kStageCap,
                          p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes, bytes, &full[stage]);
                issued = it + 1;
            }
        }
    } else {
        // ---- dot warps: all of them work on unit u together, slot j on warp j % kDotWarps --------
        const int dw = warp - kReducersF - 1;
        // fast memory of the unit in hand, fetched one unit ahead
        int nx_k = 0, nx_ids[2] = {0, 0};
        if (nu > 0) {
            const int b = my_units[0] / kMaxParts;
            const int sid = a.stream_id ? a.stream_id[b] : 0;
            nx_k = min(a.k[sid], kFusedMaxK);
            const int32_t* mem = a.members + (size_t)sid * a.k_max;
            nx_ids[0] = lane < nx_k ? mem[lane] : 0;
            nx_ids[1] = lane + kWarp < nx_k ? mem[lane + kWarp] : 0;
        }
        for (int u = 0; u < nu; ++u) {
            const int unit = my_units[u], b = unit / kMaxParts, part = unit % kMaxParts;
            const int sb = part * f.slice_cap;          // first channel of the slice
            const int Dp = min(f.slice_cap, p.C - sb);  // channels in it (a multiple of 4)
            const int n4 = Dp >> 2;
            const int k = nx_k;
            const int ids[2] = {nx_ids[0], nx_ids[1]};  // lane l knows the classes of slots l and l + 32
            const int buf = u % kSvBufs;
            int nb_sid = 0;
            if (u + 1 < nu) {
                const int nb = my_units[u + 1] / kMaxParts;
                nb_sid = a.stream_id ? a.stream_id[nb] : 0;  // in flight while this unit is scored
            }
            float* out = f.partials + ((size_t)b * P + part) * (a.k_max + 1);
            if (!mbar_wait_bounded(&sv_full[buf], (u / kSvBufs) & 1, p.status)) { failed = true; break; }
            const float4* v4 = reinterpret_cast<const float4*>(sv_s + buf * f.slice_cap);
            if (dw == kDotWarps - 1) {  // partial squared length of the semantic vector
                float nn = 0.f;
                for (int q = lane; q < n4; q += kWarp) {
                    const float4 x = v4[q];
                    nn = fmaf(x.x, x.x, nn); nn = fmaf(x.y, x.y, nn); nn = fmaf(x.z, x.z, nn); nn = fmaf(x.w, x.w, nn);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(kFull, nn, o);
                if (lane == 0) out[a.k_max] = nn;
            }
            for (int j = dw; j < k; j += kDotWarps) {  // partial dot product of slot j (Eq. 1's numerator)
                const int cls = __shfl_sync(kFull, (j & 32) ? ids[1] : ids[0], j & 31);
                const float4* crow = reinterpret_cast<const float4*>(a.centers + (size_t)cls * p.C + sb);
                float4 cc[kMaxSlice / 4 / kWarp];  // every load of the slot in flight at once
#pragma unroll
                for (int r = 0; r < kMaxSlice / 4 / kWarp; ++r) {
                    const int q = lane + r * kWarp;
                    cc[r] = q < n4 ? __ldg(crow + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float d = 0.f;
#pragma unroll
                for (int r = 0; r < kMaxSlice / 4 / kWarp; ++r) {
                    const int q = lane + r * kWarp;
                    if (q < n4) {
                        const float4 x = v4[q];
                        d = fmaf(cc[r].x, x.x, d); d = fmaf(cc[r].y, x.y, d);
                        d = fmaf(cc[r].z, x.z, d); d = fmaf(cc[r].w, x.w, d);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(kFull, d, o);
                if (lane == 0) out[j] = d;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sv_empty[buf]);
            if (u + 1 < nu) {  // fast memory of the next unit (its stream id has arrived by now)
                nx_k = min(a.k[nb_sid], kFusedMaxK);
                const int32_t* mem = a.members + (size_t)nb_sid * a.k_max;
                nx_ids[0] = lane < nx_k ? mem[lane] : 0;
                nx_ids[1] = lane + kWarp < nx_k ? mem[lane + kWarp] : 0;
            }
        }
    }
    // No thread leaves before every copy that was issued has landed.
    const int any_failed = __syncthreads_or(failed ? 1 : 0);
    if (any_failed && warp == kReducersF && lane == 0) {
        for (int s = 0; s < kStages && s < issued; ++s) {
            const uint32_t last_use = uint32_t((issued - 1 - s) / kStages);
            mbar_wait_bounded(&full[s], last_use & 1, p.status);
        }
    }
}

// ---- NHWC: direct coalesced loads ----------------------------------------------------------

constexpr int kThreadsNhwc = 256;

template <class E>
__global__ void __launch_bounds__(kThreadsNhwc) k_encode_nhwc(const uint8_t* __restrict__ x,
                                                              const uint8_t* __restrict__ skip,
                                                              float* __restrict__ sv, int B, int C, int HW,
                                                              float inv_hw) {
    extern __shared__ float part[];  // [phases][min(C, 256 * kPerVec)]
    chain_release();
    chain_wait();
    constexpr int V = E::kPerVec;
    const int CG = C / V;            // 16-byte vectors per pixel
    for (int b = blockIdx.x; b < B; b += gridDim.x) {
        if (skip && skip[b]) continue;
        const uint4* f = reinterpret_cast<const uint4*>(x + (long long)b * HW * C * E::kSize);
        for (int cg0 = 0; cg0 < CG; cg0 += kThreadsNhwc) {
            const int cgs = min(CG - cg0, kThreadsNhwc);  // channel groups handled in this sweep
            const int phases = kThreadsNhwc / cgs;
            const int ph = threadIdx.x / cgs, cg = threadIdx.x - ph * cgs;
            float acc[V];
#pragma unroll
            for (int j = 0; j < V; ++j) acc[j] = 0.f;
            if (ph < phases) {
                const uint4* col = f + cg0 + cg;
                int px = ph;
                for (; px + 3 * phases < HW; px += 4 * phases) {
                    const uint4 v0 = __ldg(col + (long long)px * CG);
                    const uint4 v1 = __ldg(col + (long long)(px + phases) * CG);
                    const uint4 v2 = __ldg(col + (long long)(px + 2 * phases) * CG);
                    const uint4 v3 = __ldg(col + (long long)(px + 3 * phases) * CG);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[j] += E::at(v0, j);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[j] += E::at(v1, j);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[j] += E::at(v2, j);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[j] += E::at(v3, j);
                }
                for (; px < HW; px += phases) {
                    const uint4 v = __ldg(col + (long long)px * CG);
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[j] += E::at(v, j);
                }
                float* dst = part + (size_t(ph) * cgs + cg) * V;
#pragma unroll
                for (int j = 0; j < V; ++j) dst[j] = acc[j];
            }
            __syncthreads();
            for (int c = threadIdx.x; c < cgs * V; c += kThreadsNhwc) {
                float s = 0.f;
                for (int q = 0; q < phases; ++q) s += part[size_t(q) * cgs * V + c];
                sv[(long long)b * C + cg0 * V + c] = s * inv_hw;
            }
            __syncthreads();
        }
    }
}

// ---- any shape: one thread per (frame, channel) ---------------------------------------------

template <class E>
__global__ void k_encode_generic(const void* __restrict__ x, const uint8_t* __restrict__ skip,
                                 float* __restrict__ sv, int B, int C, int HW, int nhwc, float inv_hw) {
    chain_release();
    chain_wait();
    const long long total = (long long)B * C;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int b = int(i / C), c = int(i - (long long)b * C);
        if (skip && skip[b]) continue;
        const size_t f0 = size_t(b) * C * HW;
        float s = 0.f;
        if (nhwc)
            for (int px = 0; px < HW; ++px) s += E::scalar(x, f0 + size_t(px) * C + c);
        else
            for (int px = 0; px < HW; ++px) s += E::scalar(x, f0 + size_t(c) * HW + px);
        sv[i] = s * inv_hw;
    }
}

__global__ void k_row_norm2(const float* __restrict__ sv, const uint8_t* __restrict__ skip, int B, int D,
                            float* __restrict__ out) {
    __shared__ float scratch[32];
    chain_release();
    chain_wait();
    const int b = blockIdx.x;
    if (skip && skip[b]) return;
    float s = 0.f;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const float v = sv[(size_t)b * D + d];
        s = fmaf(v, v, s);
    }
    s = block_sum(s, scratch);
    if (threadIdx.x == 0) out[b] = s;
}

template <class R>
cudaError_t launch_nchw(const NchwParams& p, int grid, cudaStream_t st) {
    return launch_chained(k_encode_nchw<R>, grid, kThreadsTma, kSmemTma, st, p);
}

template <class R>
cudaError_t opt_in() {
    return cudaFuncSetAttribute(k_encode_nchw<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemTma));
}

template <class E>
cudaError_t launch_generic(const EncodeArgs& a, cudaStream_t st) {
    const long long total = (long long)a.B * a.C;
    const int grid = int(std::min<long long>((total + 255) / 256, 148 * 16));
    return launch_chained(k_encode_generic<E>, grid, 256, 0, st, a.x, a.skip, a.sv, a.B, a.C, a.H * a.W,
                          int(a.layout == SMTM_NHWC), 1.0f / float(a.H * a.W));
}

template <class E>
cudaError_t launch_nhwc(const EncodeArgs& a, cudaStream_t st) {
    const int CG = a.C / E::kPerVec;
    const int cgs = std::min(CG, kThreadsNhwc);
    const size_t smem = size_t(kThreadsNhwc / cgs) * cgs * E::kPerVec * sizeof(float);
    return launch_chained(k_encode_nhwc<E>, a.B, kThreadsNhwc, smem, st, static_cast<const uint8_t*>(a.x), a.skip, a.sv,
                          a.B, a.C, a.H * a.W, 1.0f / float(a.H * a.W));
}

int pow2_floor(int v) {
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}



// Copies the producer keeps outstanding.  Four 25 KB copies per SM (15 MB over the chip) cover
// the bandwidth-delay product of HBM with margin; more only lengthens the queues that the
// centre loads of the dot warps wait in.
constexpr int kMaxInFlight = 4;

// Which reducer a shape is served by, and the chunking that goes with it.
enum Reducer { kNone, kUnitBf16x49, kUnitBf16x196, kUnitF16x49, kUnitF16x196, kUnitF32x49, kTeamF32, kTeamF16, kTeamBf16 };

Reducer plan_nchw(const EncodeArgs& a, NchwParams* p) {
    const int HW = a.H * a.W;
    const int es = a.dtype == SMTM_F32 ? 4 : 2;
    *p = NchwParams{};
    p->x = static_cast<const uint8_t*>(a.x);
    p->skip = a.skip;
    p->sv = a.sv;
    p->sv_hi = static_cast<__nv_bfloat16*>(a.sv_hi);
    p->sv_lo = static_cast<__nv_bfloat16*>(a.sv_lo);
    p->status = a.status;
    p->C = a.C;
    p->ch_bytes = HW * es;
    p->frame_bytes = (long long)a.C * p->ch_bytes;
    p->inv_hw = 1.0f / float(HW);
    p->max_in_flight = kMaxInFlight;
    // unit-per-lane shapes (compile-time H*W)
    int G = 0;
    if ((HW == 49 || HW == 196) && es == 2) G = HW == 49 ? 8 : 2;
    if (HW == 49 && es == 4) G = 4;
    if (G && a.C % G == 0) {
        p->chunk_channels = 32 * G;
        p->chunks_per_frame = (a.C + p->chunk_channels - 1) / p->chunk_channels;
        p->total_chunks = (long long)a.B * p->chunks_per_frame;
        if (es == 4) return kUnitF32x49;
        if (a.dtype == SMTM_BF16) return HW == 49 ? kUnitBf16x49 : kUnitBf16x196;
        return HW == 49 ? kUnitF16x49 : kUnitF16x196;
    }
    // team-per-channel: channel bytes a multiple of 16 and at most one stage
    if (p->ch_bytes % 16 == 0 && p->ch_bytes <= kStageCap) {
        p->vec_per_channel = p->ch_bytes / 16;
        p->team = std::min(32, pow2_floor(std::max(1, p->vec_per_channel / 4)));
        const int per_pass = 32 / p->team;
        int cc = kStageCap / p->ch_bytes;
        if (cc > per_pass) cc -= cc % per_pass;
        p->chunk_channels = std::min(cc, a.C);
        p->chunks_per_frame = (a.C + p->chunk_channels - 1) / p->chunk_channels;
        p->total_chunks = (long long)a.B * p->chunks_per_frame;
        return a.dtype == SMTM_F32 ? kTeamF32 : a.dtype == SMTM_F16 ? kTeamF16 : kTeamBf16;
    }
    return kNone;
}

#define SMTM_FOR_REDUCER(r, CALL)                                   \
    switch (r) {                                                    \
        case kUnitBf16x49: CALL(UnitPerLane<BF16, 49>); break;      \
        case kUnitBf16x196: CALL(UnitPerLane<BF16, 196>); break;    \
        case kUnitF16x49: CALL(UnitPerLane<F16, 49>); break;        \
        case kUnitF16x196: CALL(UnitPerLane<F16, 196>); break;      \
        case kUnitF32x49: CALL(UnitPerLane<F32, 49>); break;        \
        case kTeamF32: CALL(TeamPerChannel<F32>); break;            \
        case kTeamF16: CALL(TeamPerChannel<F16>); break;            \
        case kTeamBf16: CALL(TeamPerChannel<BF16>); break;          \
        default: break;                                             \
    }

template <class R>
cudaError_t opt_in_fused() {
    return cudaFuncSetAttribute(k_lookup_nchw<R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                int(fused_smem(kMaxSlice)));
}

}  // namespace

cudaError_t encode_setup() {
    cudaError_t e = cudaSuccess;
#define SMTM_OPT_IN(...)                                        \
    if (e == cudaSuccess) e = opt_in<__VA_ARGS__>();            \
    if (e == cudaSuccess) e = opt_in_fused<__VA_ARGS__>();
    for (int r = kUnitBf16x49; r <= kTeamBf16; ++r) SMTM_FOR_REDUCER(r, SMTM_OPT_IN)
#undef SMTM_OPT_IN
    return e;
}

cudaError_t launch_encode(const EncodeArgs& a, int sm_count, cudaStream_t st, int64_t* launches, bool* wrote_split) {
    if (wrote_split) *wrote_split = false;
    if (a.B <= 0) return cudaSuccess;
    ++*launches;
    if (a.layout == SMTM_NHWC) {
        const int V = a.dtype == SMTM_F32 ? 4 : 8;
        if (a.C % V == 0) {
            if (a.dtype == SMTM_F32) return launch_nhwc<F32>(a, st);
            if (a.dtype == SMTM_F16) return launch_nhwc<F16>(a, st);
            return launch_nhwc<BF16>(a, st);
        }
    } else {
        NchwParams p;
        const Reducer r = plan_nchw(a, &p);
        if (r != kNone) {
            cudaError_t e = cudaSuccess;
            if (wrote_split) *wrote_split = p.sv_hi != nullptr;
#define SMTM_LAUNCH(...) e = launch_nchw<__VA_ARGS__>(p, sm_count, st)
            SMTM_FOR_REDUCER(r, SMTM_LAUNCH)
#undef SMTM_LAUNCH
            return e;
        }
    }
    if (a.dtype == SMTM_F32) return launch_generic<F32>(a, st);
    if (a.dtype == SMTM_F16) return launch_generic<F16>(a, st);
    return launch_generic<BF16>(a, st);
}

size_t fused_partials_floats(int max_batch, int k_max) {
    return size_t(max_batch) * kMaxParts * (size_t(std::min(k_max, kFusedMaxK)) + 1);
}

cudaError_t launch_lookup_fused(const EncodeArgs& e, const LookupArgs& a, float* partials, int sm_count,
                                cudaStream_t st, int64_t* launches, bool* handled, const cudaEvent_t* timing) {
    *handled = false;
    if (e.B <= 0 || e.layout != SMTM_NCHW || a.k_max > kFusedMaxK || !partials) return cudaSuccess;
    FusedParams f{};
    const Reducer r = plan_nchw(e, &f.e);
    if (r == kNone) return cudaSuccess;
    // Parts per frame.  A unit must fit the scorers' registers (slice <= kMaxSlice channels, a
    // multiple of 4); among the divisors of the chunk count take the smallest that fills the
    // last round of units to 95 % (else the best filled), preferring units of >= 4 chunks.
    const int cpf = f.e.chunks_per_frame;
    if ((e.C & 3) || (f.e.chunk_channels & 3)) return cudaSuccess;
    const auto pick = [&](int min_chunks) {
        int best_d = 0;
        double best_eff = -1.0;
        for (int d = 1; d <= std::min(cpf, kMaxParts); ++d) {
            if (cpf % d || cpf / d < min_chunks || (cpf / d) * f.e.chunk_channels > kMaxSlice) continue;
            if (((long long)e.B * d + sm_count - 1) / sm_count > kMaxUnits) continue;
            const double rounds = double(e.B) * d / sm_count;
            const double eff = rounds / std::ceil(rounds);
            if (eff >= 0.95) return d;
            if (eff > best_eff + 1e-9) {
                best_eff = eff;
                best_d = d;
            }
        }
        return (best_eff >= 0.8 || min_chunks <= 1) ? best_d : 0;
    };
    int P = pick(4);
    if (P == 0) P = pick(1);
    if (P <= 0) return cudaSuccess;
    f.a = a;
    f.parts = P;
    f.chunks_per_unit = cpf / P;
    f.slice_cap = f.chunks_per_unit * f.e.chunk_channels;
    f.partials = partials;
    const size_t smem = fused_smem(f.slice_cap);
    cudaError_t err = cudaSuccess;
    if (timing) record_timing(timing[0], st);
#define SMTM_LAUNCH(...) err = launch_chained(k_lookup_nchw<__VA_ARGS__>, sm_count, kThreadsFused, smem, st, f)
    SMTM_FOR_REDUCER(r, SMTM_LAUNCH)
#undef SMTM_LAUNCH
    if (timing) record_timing(timing[1], st);
    ++*launches;
    *handled = true;
    if (err != cudaSuccess) return err;
    return launch_finish_partials(a, partials, P, st, launches);
}

cudaError_t launch_row_norm2(const float* sv, const uint8_t* skip, int B, int D, float* out, cudaStream_t st,
                             int64_t* launches) {
    if (B <= 0) return cudaSuccess;
    ++*launches;
    return launch_chained(k_row_norm2, B, 256, 0, st, sv, skip, B, D, out);
}

}  // namespace smtm
