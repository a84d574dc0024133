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
    int max_in_flight;       // copies the producer keeps outstanding (<= stages)
    int stages;              // k_encode_nchw: ring depth, 2 .. kStages (the fused kernel always uses kStages)
    int consumers;           // k_encode_nchw: consumer warps, 1 .. kConsumers; the CTA has one more warp, the producer's
    unsigned long long* clock;  // nullptr, or two words for the device-clock stamps of the pooling kernel
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

// T lanes per channel; channel bytes are a multiple of 16.  Two passes (channels per team) are
// folded at a time, one accumulator per element of a vector and two vectors of each in
// flight: a single warp has to keep up with the copies, so the loop must not be one chain of
// dependent additions.
template <class E>
struct TeamPerChannel {
    static __device__ __forceinline__ void run(const uint8_t* stage, int nch, int lane, float* out, float* out_s,
                                               float inv_hw, const NchwParams& p) {
        const int T = p.team, uw = p.vec_per_channel;
        const int per_pass = kWarp / T;
        const int team = lane / T, r = lane - team * T;
        const int passes = (nch + per_pass - 1) / per_pass;
        for (int ps = 0; ps < passes; ps += 2) {
            const int c0 = ps * per_pass + team, c1 = c0 + per_pass;  // this team's channels of the two passes
            // a channel past the end is read as the chunk's last one and dropped afterwards
            const uint4* u0 = reinterpret_cast<const uint4*>(stage) + size_t(min(c0, nch - 1)) * uw;
            const uint4* u1 = reinterpret_cast<const uint4*>(stage) + size_t(min(c1, nch - 1)) * uw;
            float a[2][E::kPerVec];
#pragma unroll
            for (int j = 0; j < E::kPerVec; ++j) a[0][j] = a[1][j] = 0.f;
            int i = r;
            for (; i + T < uw; i += 2 * T) {
                const uint4 v00 = u0[i], v01 = u0[i + T], v10 = u1[i], v11 = u1[i + T];
#pragma unroll
                for (int j = 0; j < E::kPerVec; ++j) {
                    a[0][j] += E::at(v00, j);
                    a[1][j] += E::at(v10, j);
                }
#pragma unroll
                for (int j = 0; j < E::kPerVec; ++j) {
                    a[0][j] += E::at(v01, j);
                    a[1][j] += E::at(v11, j);
                }
            }
            for (; i < uw; i += T) {
                const uint4 v0 = u0[i], v1 = u1[i];
#pragma unroll
                for (int j = 0; j < E::kPerVec; ++j) {
                    a[0][j] += E::at(v0, j);
                    a[1][j] += E::at(v1, j);
                }
            }
            float s[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                s[h] = (a[h][0] + a[h][1]) + (a[h][2] + a[h][3]);
                if (E::kPerVec == 8)
                    s[h] += (a[h][4 % E::kPerVec] + a[h][5 % E::kPerVec]) + (a[h][6 % E::kPerVec] + a[h][7 % E::kPerVec]);
            }
            for (int o = T >> 1; o > 0; o >>= 1) {
                s[0] += __shfl_xor_sync(kFull, s[0], o);
                s[1] += __shfl_xor_sync(kFull, s[1], o);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c = h ? c1 : c0;
                if (c < nch && r == 0) {
                    const float v = s[h] * inv_hw;
                    out[c] = v;
                    if (out_s) out_s[c] = v;
                    if (p.sv_hi) {
                        const ptrdiff_t at = (out + c) - p.sv;
                        const __nv_bfloat16 hh = __float2bfloat16_rn(v);
                        p.sv_hi[at] = hh;
                        p.sv_lo[at] = __float2bfloat16_rn(v - __bfloat162float(hh));
                    }
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
    const int n_stages = p.stages;
    uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(n_stages) * kStageCap);
    uint64_t* empty = full + n_stages;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init_fence();
    }
    __syncthreads();
    chain_wait();  // the barriers are set up while the previous kernel finishes
    chain_release();
    const ClockScope stamps(p.clock);

    const int n_consumers = p.consumers;
    const bool producer = warp == n_consumers;  // last warp; lane 0 issues the copies
    const uint64_t stream_once = l2_evict_first_policy();
    int it = 0;                                // chunks of this CTA that are not skipped, so far
    bool failed = false;
    if (!producer || lane == 0) {
        for (long long g = blockIdx.x; g < p.total_chunks; g += gridDim.x) {
            const int b = int(g / p.chunks_per_frame);
            if (p.skip && p.skip[b]) continue;
            const int ci = int(g - (long long)b * p.chunks_per_frame);
            const int stage = it % n_stages;
            const uint32_t use = uint32_t(it / n_stages);
            const int c0 = ci * p.chunk_channels;
            const int nch = min(p.chunk_channels, p.C - c0);
            if (producer) {
                if (use > 0 && !mbar_wait_bounded(&empty[stage], (use - 1) & 1, p.status)) {
                    failed = true;
                    break;
                }
                if (it >= p.max_in_flight) {  // bound the bytes in flight: wait for an older copy to land
                    const int old = it - p.max_in_flight;
                    if (!mbar_wait_bounded(&full[old % n_stages], (old / n_stages) & 1, p.status)) {
                        failed = true;
                        break;
                    }
                }
                const uint32_t bytes = uint32_t(nch) * uint32_t(p.ch_bytes);
                mbar_expect_tx(&full[stage], bytes);
                bulk_load_hint(stages + size_t(stage) * kStageCap,
                               p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes, bytes, &full[stage], stream_once);
            } else if (stage % n_consumers == warp) {
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
        for (int s = 0; s < n_stages && s < it; ++s) {
            const uint32_t last_use = uint32_t((it - 1 - s) / n_stages);
            mbar_wait_bounded(&full[s], last_use & 1, p.status);
        }
    }
}

// ---- fused lookup: encode + similarity scoring + decision in one persistent kernel ------------
//
// A frame is cut into P parts (runs of chunks_per_unit chunks, i.e. slices of its channels) and
// a thread-block cluster of P CTAs takes whole frames: CTA `rank` of the cluster streams and
// scores part `rank`.  Every CTA first compacts the frames that are still active; cluster c
// takes the frames c, c + clusters, ... of that list, so exited frames cost nothing and the
// load is even.  Per frame the reducer warps leave the slice of the semantic vector in shared
// memory (four buffers) as well as in the SV stash; eight dot warps then share the slice's dot
// products, slot j on warp j % 8: each lane has every load of its slot's centre slice in
// flight at once, so a frame costs one trip to L2.  The partial dot products and the partial
// squared length go, through distributed shared memory, to a receive buffer in the cluster's
// first CTA, whose finisher warp adds the parts up in rank order and decides: Eq. 1, Eq. 3,
// top-2, Eq. 4 / Eq. 2 and the exit rule.  No atomics on floating point and no global scratch:
// the evaluation order of every sum is fixed.
constexpr int kReducersF = 4;       // reducer warps of the fused kernel; stage s belongs to warp s % kReducersF
constexpr int kDotWarps = 8;        // warps that share the dot products of a slice
constexpr int kSvBufs = 4;          // shared-memory slices; frame u passes through buffer u % kSvBufs
constexpr int kRx = 4;              // receive buffers between the dot warps and the finisher
constexpr int kRxRow = kFusedMaxK + 4;  // words per row of a receive buffer
// A receive buffer holds P + 2 rows: one per part (the partial dots, then the partial squared length at
// [kFusedMaxK]) and, from the first CTA's own dot warps, the slots' classes (then k at [kFusedMaxK]) and the
// lengths of their centres, so that the finisher has nothing to fetch once the parts are in.
constexpr int kMaxCluster = 8;      // CTAs per cluster = parts per frame
constexpr int kThreadsFused = (kReducersF + 1 + kDotWarps + 1) * kWarp;  // reducers, producer, dot warps, finisher
constexpr int kMaxUnits = 1024;     // frames per cluster
constexpr int kMaxSlice = 1024;     // floats of a semantic-vector slice (eight 16-byte vectors per lane)
constexpr size_t kSmemLimit = 227 * 1024;
static_assert(kStages % kReducersF == 0, "stage ownership must be periodic");

struct FusedParams {
    NchwParams e;
    LookupArgs a;
    int parts;            // P: CTAs per cluster, one part of every frame each (divides chunks_per_frame)
    int chunks_per_unit;  // chunks_per_frame / P
    int slice_cap;        // channels of a full slice = chunks_per_unit * chunk_channels (multiple of 4)
};

constexpr size_t fused_smem(int slice_cap, int parts) {
    return size_t(kStages) * kStageCap + size_t(kSvBufs) * size_t(slice_cap) * 4 +
           size_t(kRx) * size_t(parts + 2) * kRxRow * 4 + kMaxUnits * 4 + 40 * 4 +
           (2 * kStages + 2 * kSvBufs + 2 * kRx) * 8 + 192;
}

// ---- cluster primitives ------------------------------------------------------------------------

// Address of the same shared-memory location in CTA `rank` of this cluster.
__device__ __forceinline__ uint32_t peer_smem(const void* p, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(smem_u32(p)), "r"(rank));
    return out;
}

__device__ __forceinline__ void peer_store(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// Arrival on a barrier of any CTA of the cluster; orders this thread's earlier writes before it.
__device__ __forceinline__ void peer_arrive(uint32_t bar_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// As mbar_wait_bounded, for a barrier that CTAs of the whole cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint64_t* bar, uint32_t parity, int* status) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (clock64() - t0 > (1ll << 31)) {
            set_status(status, kDevTimeout);
            return false;
        }
    }
}

// All threads of all CTAs of the cluster.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <class R>
__global__ void __launch_bounds__(kThreadsFused, 1) k_lookup_nchw(const FusedParams f) {
    extern __shared__ uint8_t smem_raw[];
    const NchwParams& p = f.e;
    const LookupArgs& a = f.a;
    const int P = f.parts, cpu = f.chunks_per_unit;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    uint8_t* stages = base;
    float* sv_s = reinterpret_cast<float*>(base + size_t(kStages) * kStageCap);  // [kSvBufs][slice_cap]
    float* rx = sv_s + kSvBufs * f.slice_cap;                                    // [kRx][P + 2][kRxRow]
    int* my_units = reinterpret_cast<int*>(rx + kRx * (P + 2) * kRxRow);               // [kMaxUnits] frames of this cluster
    int* s_scan = my_units + kMaxUnits;                                          // [36]
    unsigned int* s_ctr = reinterpret_cast<unsigned int*>(s_scan + 36);          // [4] lookups, near, exits
    uint64_t* full = reinterpret_cast<uint64_t*>(
        (reinterpret_cast<uintptr_t>(s_scan + 40) + 7) & ~uintptr_t(7));         // [kStages]
    uint64_t* empty = full + kStages;                                            // [kStages]
    uint64_t* sv_full = empty + kStages;                                         // [kSvBufs]  slice written
    uint64_t* sv_empty = sv_full + kSvBufs;                                      // [kSvBufs]  slice read by all dot warps
    uint64_t* rx_full = sv_empty + kSvBufs;                                      // [kRx]  every part has arrived here
    uint64_t* rx_empty = rx_full + kRx;                                          // [kRx]  every rank: the finisher is done with it

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = int(blockIdx.x) % P;       // clusters are runs of P consecutive CTAs
    const int cluster = int(blockIdx.x) / P, n_clusters = int(gridDim.x) / P;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int s = 0; s < kSvBufs; ++s) {
            mbar_init(&sv_full[s], cpu);
            mbar_init(&sv_empty[s], kDotWarps);
        }
        for (int s = 0; s < kRx; ++s) {
            mbar_init(&rx_full[s], P * kDotWarps);
            mbar_init(&rx_empty[s], 1);
        }
        mbar_init_fence();
        s_ctr[0] = s_ctr[1] = s_ctr[2] = 0u;
    }

    // ---- the active frames and this cluster's share of them ---------------------------------
    int n_active = a.fresh ? a.B : 0;  // a batch that starts here has every frame active: no flags to read
    for (int idx = threadIdx.x; a.fresh && idx < kMaxUnits; idx += kThreadsFused) {
        const long long u = (long long)cluster + (long long)idx * n_clusters;
        if (u < a.B) my_units[idx] = int(u);
    }
    // Everything above touched shared memory only and overlaps the previous kernel's tail.
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * a.layer : nullptr);  // profiling
    for (int t0 = 0; !a.fresh && t0 < a.B; t0 += kThreadsFused) {
        const int b = t0 + threadIdx.x;
        // Active = not exited at an earlier layer.  A finisher of this launch may already have
        // decided the frame: an exit at this very layer leaves it active, so every CTA gets
        // the same list whenever it looks.
        int act = 0;
        if (b < a.B) {
            const int el = *reinterpret_cast<const volatile int32_t*>(a.exit_layer + b);
            act = (el == 0 || el == a.layer + 1) ? 1 : 0;
        }
        int cnt;
        const int pos = block_exclusive_scan(act, s_scan, &cnt);
        if (act) {
            const int u = n_active + pos;
            if (u % n_clusters == cluster && u / n_clusters < kMaxUnits) my_units[u / n_clusters] = b;
        }
        n_active += cnt;
    }
    int nu = n_active > cluster ? (n_active - cluster + n_clusters - 1) / n_clusters : 0;
    nu = min(nu, kMaxUnits);
    __syncthreads();
    if (P > 1) cluster_sync_all();  // every CTA's barriers exist before anyone arrives on them

    const int n_chunks = nu * cpu;
    bool failed = false;
    int issued = 0;
    if (warp < kReducersF) {
        // ---- reducers: warp w owns the stages w, w + kReducersF, ... -----------------------------
        for (int it = warp; it < n_chunks; it += kReducersF) {
            const int i = it / cpu, c = it - i * cpu;
            const int b = my_units[i];
            const int c0 = (rank * cpu + c) * p.chunk_channels;
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
            const uint64_t stream_once = l2_evict_first_policy();
            for (int it = 0; it < n_chunks; ++it) {
                const int i = it / cpu, c = it - i * cpu;
                const int b = my_units[i];
                const int c0 = (rank * cpu + c) * p.chunk_channels;
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
                bulk_load_hint(stages + size_t(stage) * kStageCap,
                               p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes, bytes, &full[stage], stream_once);
                issued = it + 1;
            }
        }
    } else if (warp <= kReducersF + kDotWarps) {
        // ---- dot warps: all of them work on frame u together, slot j on warp j % kDotWarps -------
        const int dw = warp - kReducersF - 1;
        const int sb = rank * f.slice_cap;          // first channel of this CTA's slice
        const int Dp = max(0, min(f.slice_cap, p.C - sb));  // channels in it (a multiple of 4)
        const int n4 = Dp >> 2;
        // fast memory of the frame in hand, fetched one frame ahead
        int nx_k = 0, nx_ids[2] = {0, 0};
        if (nu > 0) {
            const int b = my_units[0];
            const int sid = stream_of(a, b);
            nx_k = sid < 0 ? 0 : min(a.k[sid], kFusedMaxK);  // a stream id outside the cache: nothing to score against
            const int32_t* mem = a.members + (size_t)max(sid, 0) * a.k_max;
            nx_ids[0] = lane < nx_k ? mem[lane] : 0;
            nx_ids[1] = lane + kWarp < nx_k ? mem[lane + kWarp] : 0;
        }
        for (int u = 0; u < nu; ++u) {
            const int k = nx_k;
            const int ids[2] = {nx_ids[0], nx_ids[1]};  // lane l knows the classes of slots l and l + 32
            const int buf = u % kSvBufs, x = u % kRx;
            int nb_sid = 0;
            if (u + 1 < nu) {
                const int nb = my_units[u + 1];
                nb_sid = a.stream_id ? a.stream_id[nb] : 0;  // in flight while this frame is scored
            }
            // The CTAs of a cluster take turns at finishing: frame u goes to CTA u % P.  This part's
            // row of receive buffer x over there:
            const int fin = u % P;
            const uint32_t out = peer_smem(rx + (x * (P + 2) + rank) * kRxRow, fin);
            // the centre slice of this warp's first slot is fetched while the slice of the
            // semantic vector is still being pooled
            float4 cc[kMaxSlice / 4 / kWarp];  // every load of a slot in flight at once
            float clen = 0.f;
            if (dw < k) {
                const int cls = __shfl_sync(kFull, ids[0], dw);
                const float4* crow = reinterpret_cast<const float4*>(a.centers + (size_t)cls * p.C + sb);
                if (rank == fin && lane == 0) clen = __ldg(a.cnorm + cls);
#pragma unroll
                for (int r = 0; r < kMaxSlice / 4 / kWarp; ++r) {
                    const int q = lane + r * kWarp;
                    cc[r] = q < n4 ? __ldg(crow + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            if (!mbar_wait_bounded(&sv_full[buf], (u / kSvBufs) & 1, p.status)) { failed = true; break; }
            if (u >= kRx && !mbar_wait_cluster_bounded(&rx_empty[x], (u / kRx - 1) & 1, p.status)) { failed = true; break; }
            const float4* v4 = reinterpret_cast<const float4*>(sv_s + buf * f.slice_cap);
            int* meta_ids = reinterpret_cast<int*>(rx + (x * (P + 2) + P) * kRxRow);  // in the finishing CTA only
            float* meta_len = rx + (x * (P + 2) + P + 1) * kRxRow;
            if (rank == fin && dw == 0) {  // the slots' classes and k, in the layout the finisher's lanes want
                meta_ids[lane] = ids[0];
                meta_ids[lane + kWarp] = ids[1];
                if (lane == 0) meta_ids[kFusedMaxK] = k;
            }
            if (dw == kDotWarps - 1) {  // partial squared length of the semantic vector
                float nn = 0.f;
                for (int q = lane; q < n4; q += kWarp) {
                    const float4 xv = v4[q];
                    nn = fmaf(xv.x, xv.x, nn); nn = fmaf(xv.y, xv.y, nn); nn = fmaf(xv.z, xv.z, nn); nn = fmaf(xv.w, xv.w, nn);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(kFull, nn, o);
                if (lane == 0) peer_store(out + kFusedMaxK * 4, nn);
            }
            for (int j = dw; j < k; j += kDotWarps) {  // partial dot product of slot j (Eq. 1's numerator)
                if (j != dw) {  // the first slot's loads are already under way
                    const int cls = __shfl_sync(kFull, (j & 32) ? ids[1] : ids[0], j & 31);
                    const float4* crow = reinterpret_cast<const float4*>(a.centers + (size_t)cls * p.C + sb);
                    if (rank == fin && lane == 0) clen = __ldg(a.cnorm + cls);  // in flight with the centre
#pragma unroll
                    for (int r = 0; r < kMaxSlice / 4 / kWarp; ++r) {
                        const int q = lane + r * kWarp;
                        cc[r] = q < n4 ? __ldg(crow + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                float d = 0.f;
#pragma unroll
                for (int r = 0; r < kMaxSlice / 4 / kWarp; ++r) {
                    const int q = lane + r * kWarp;
                    if (q < n4) {
                        const float4 xv = v4[q];
                        d = fmaf(cc[r].x, xv.x, d); d = fmaf(cc[r].y, xv.y, d);
                        d = fmaf(cc[r].z, xv.z, d); d = fmaf(cc[r].w, xv.w, d);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(kFull, d, o);
                if (lane == 0) {
                    peer_store(out + j * 4, d);
                    if (rank == fin) meta_len[j] = clen;
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&sv_empty[buf]);
                peer_arrive(peer_smem(&rx_full[x], fin));  // this warp's share of the part has been delivered
            }
            if (u + 1 < nu) {  // fast memory of the next frame (its stream id has arrived by now)
                nb_sid = stream_checked(a, nb_sid);
                nx_k = nb_sid < 0 ? 0 : min(a.k[nb_sid], kFusedMaxK);
                const int32_t* mem = a.members + (size_t)max(nb_sid, 0) * a.k_max;
                nx_ids[0] = lane < nx_k ? mem[lane] : 0;
                nx_ids[1] = lane + kWarp < nx_k ? mem[lane + kWarp] : 0;
            }
        }
    } else {
        // ---- finisher warp: every P-th frame of the cluster; lane l looks after slots l and l + 32 ----
        const float weight = float(1u << a.layer);  // 2^(l-1) with l = layer + 1
        const int reuse = max(P, kRx);              // frames between two uses of a receive buffer in this CTA
        for (int u = rank; u < nu; u += P) {
            const int b = my_units[u], x = u % kRx;
            float sa_old[2];  // the carry, fetched while the frame is being scored
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = lane + h * kWarp;
                sa_old[h] = (j < a.k_max && !a.fresh) ? a.sa[(size_t)b * a.k_max + j] : 0.f;
            }
            if (!mbar_wait_cluster_bounded(&rx_full[x], (u / reuse) & 1, p.status)) { failed = true; break; }
            const int* meta_ids = reinterpret_cast<const int*>(rx + (x * (P + 2) + P) * kRxRow);
            const float* meta_len = rx + (x * (P + 2) + P + 1) * kRxRow;
            const int k = meta_ids[kFusedMaxK];
            const int ids[2] = {meta_ids[lane], meta_ids[lane + kWarp]};
            const float clen[2] = {lane < k ? meta_len[lane] : 0.f, lane + kWarp < k ? meta_len[lane + kWarp] : 0.f};
            float nn = 0.f, dots[2] = {0.f, 0.f};
            for (int r = 0; r < P; ++r) {  // the parts in rank order
                const float* row = rx + (x * (P + 2) + r) * kRxRow;
                nn += row[kFusedMaxK];
                if (lane < k) dots[0] += row[lane];
                if (lane + kWarp < k) dots[1] += row[lane + kWarp];
            }
            __syncwarp();
            // every rank may fill buffer x again; nobody waits for that after the last kRx frames
            if (lane < P && u + kRx < nu) peer_arrive(peer_smem(&rx_empty[x], lane));
            float s_cur[2] = {0.f, 0.f}, s_acc[2] = {0.f, 0.f};
            const float sv_len = __fsqrt_rn(nn);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = lane + h * kWarp;
                if (j < k) {
                    s_cur[h] = (nn == 0.f || clen[h] == 0.f) ? 0.f : __fdiv_rn(dots[h], __fmul_rn(sv_len, clen[h]));  // Eq. 1
                    s_acc[h] = __fmaf_rn(s_cur[h], weight, sa_old[h]);   // Eq. 3
                    a.sa[(size_t)b * a.k_max + j] = s_acc[h];
                } else if (a.fresh && j < a.k_max) {
                    a.sa[(size_t)b * a.k_max + j] = 0.f;                 // unused slots start from zero too
                }
            }
            const Top2 ta = warp_top2_keys(s_acc, ids, k, lane);
            Top2 ts{0.f, 0.f, -1, -1};
            if (a.sep) ts = warp_top2_keys(s_cur, ids, k, lane);  // only Eq. 2 (a diagnostic) needs it
            if (lane == 0) {
                const int r = decide_core(a, b, ta, ts);
                s_ctr[0] += 1u;  // only this lane touches the tallies until the CTA is done
                if (r & 2) s_ctr[1] += 1u;
                if (r & 1) s_ctr[2] += 1u;
            }
        }
    }
    // No thread leaves before every copy that was issued has landed, and no CTA before its
    // peers are done with its shared memory.
    const int any_failed = __syncthreads_or(failed ? 1 : 0);
    if (threadIdx.x < 3 && s_ctr[threadIdx.x]) {  // this CTA's tallies: lookups, near-threshold, exits
        const int slot = threadIdx.x == 0 ? SMTM_CTR_LOOKUPS : threadIdx.x == 1 ? SMTM_CTR_NEAR : SMTM_CTR_EXITS + a.layer;
        atomicAdd(&a.counters[slot], (unsigned long long)s_ctr[threadIdx.x]);
    }
    if (any_failed && warp == kReducersF && lane == 0) {
        for (int s = 0; s < kStages && s < issued; ++s) {
            const uint32_t last_use = uint32_t((issued - 1 - s) / kStages);
            mbar_wait_bounded(&full[s], last_use & 1, p.status);
        }
    }
    __syncthreads();
    if (P > 1) cluster_sync_all();
}

// ---- pooling of the few frames still in at a later layer, by small CTAs ------------------------
//
// When most frames have left at an earlier layer, the streaming kernel above is the wrong tool: it
// wants a whole SM per CTA, and on a device whose SMs are held by another streaming kernel (the
// pooling of the next step's first layer, see the pipelined route in api.cu) it would wait for one.
// This kernel pools the active frames with CTAs of 128 threads and a single 12.5 KB stage, so that
// several fit beside such a kernel.  The grid is cpf x G CTAs: CTA c looks after chunk c % cpf of the
// active frames number c / cpf, c / cpf + G, ... (every CTA compacts the list of active frames for
// itself, as the fused kernel does).  A chunk is fetched with plain coalesced 16-byte loads, all in
// flight at once, and reduced by the reducers of the streaming kernel, the warps sharing its
// channels: every channel is summed in the same order as there, so both kernels give the same bits.
constexpr int kLightThreads = 128;
constexpr int kLightStageCap = 12800;   // bytes of a chunk here (half a stage of the streaming kernel)
constexpr int kLightFrames = 256;       // frames a CTA can be given

struct LightParams {
    NchwParams e;   // chunking as for the streaming kernel, with chunks of at most kLightStageCap bytes
    int groups;     // G
    int gran;       // channels that must stay in one warp's share (the reducer's unit)
};

template <class R>
__global__ void __launch_bounds__(kLightThreads) k_pool_sparse(const LightParams f) {
    __shared__ __align__(16) uint8_t stage[kLightStageCap];
    __shared__ int my_frames[kLightFrames];
    __shared__ int s_scan[33];
    const NchwParams& p = f.e;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int B = int(p.total_chunks / p.chunks_per_frame);
    const int ci = int(blockIdx.x) % p.chunks_per_frame, group = int(blockIdx.x) / p.chunks_per_frame;
    chain_wait();  // the exit flags are the previous kernel's
    chain_release();
    const ClockScope stamps(p.clock);
    uint8_t flags[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int n_active = 0;
    for (int t0 = 0; t0 < B; t0 += kLightThreads) {
        const int b = t0 + tid;
        int act = b < B ? 1 : 0;
        if (p.skip) {  // the flags of eight tiles in one trip to memory
            if ((t0 / kLightThreads) % 8 == 0) {
#pragma unroll
                for (int u = 0; u < 8; ++u) flags[u] = p.skip[min(b + u * kLightThreads, B - 1)];
            }
            uint8_t mine = 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) mine = ((t0 / kLightThreads) % 8 == u) ? flags[u] : mine;
            act = (b < B && !mine) ? 1 : 0;
        }
        int cnt;
        const int pos = block_exclusive_scan(act, s_scan, &cnt);
        if (act) {
            const int u = n_active + pos;
            if (u % f.groups == group && u / f.groups < kLightFrames) my_frames[u / f.groups] = b;
        }
        n_active += cnt;
    }
    const int nu = n_active > group ? min((n_active - group + f.groups - 1) / f.groups, kLightFrames) : 0;
    __syncthreads();
    const int c0 = ci * p.chunk_channels;
    const int nch = min(p.chunk_channels, p.C - c0);
    const int vectors = nch * p.ch_bytes / 16;
    // this warp's share of the chunk's channels (whole reducer units)
    const int units = (nch + f.gran - 1) / f.gran;
    const int u_lo = min(units, warp * ((units + 3) / 4)), u_hi = min(units, u_lo + (units + 3) / 4);
    const int w_c0 = u_lo * f.gran, w_nch = min(nch, u_hi * f.gran) - w_c0;
    for (int k = 0; k < nu; ++k) {
        const int b = my_frames[k];
        const uint4* src = reinterpret_cast<const uint4*>(p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes);
        uint4* dst = reinterpret_cast<uint4*>(stage);
        for (int v0 = 0; v0 < vectors; v0 += 8 * kLightThreads) {  // eight loads per thread in flight
            uint4 r[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) r[u] = load_once(src + min(v0 + u * kLightThreads + tid, vectors - 1));
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (v0 + u * kLightThreads + tid < vectors) dst[v0 + u * kLightThreads + tid] = r[u];
        }
        __syncthreads();
        if (w_nch > 0)
            R::run(stage + size_t(w_c0) * p.ch_bytes, w_nch, lane, p.sv + (long long)b * p.C + c0 + w_c0, nullptr, p.inv_hw, p);
        __syncthreads();  // the stage is free for the next frame
    }
}

// ---- the same frames looked up whole: pooling, scoring and the decision by a cluster of small CTAs ----
//
// A thread-block cluster of P CTAs takes active frames one at a time; CTA `rank` fetches chunk `rank` of the
// frame (one trip to memory for the whole frame), pools it, and scores its slice of the semantic vector
// against the frame's fast-memory centres; the partial dot products and the partial squared length go
// through distributed shared memory to the cluster's first CTA, whose first warp adds the parts in rank
// order and decides (Eq. 1, Eq. 3, top-2, Eq. 4, the exit rule), as the fused streaming kernel does.  One
// cluster-wide barrier per frame; two receive buffers take turns.  P = chunks per frame <= 8, and a chunk
// here is a chunk of the streaming kernel (<= 25 KB): a whole frame is in flight at once.
constexpr int kSparseStageCap = kStageCap;
constexpr int kSparseFrames = 64;    // frames a cluster can be given
constexpr int kSparseSlice = 1024;   // channels of a chunk at most (as the fused kernel's slices)

struct SparseParams {
    NchwParams e;
    LookupArgs a;
    int groups;  // clusters
    int gran;    // channels that must stay in one warp's share (the reducer's unit)
};

constexpr size_t sparse_smem(int slice) {
    return size_t(kSparseStageCap) + size_t(slice) * 4 + 2 * size_t(kMaxCluster) * kRxRow * 4 + 2 * kSparseFrames * 4 + 64 * 4 + 64;
}

template <class R>
__global__ void __launch_bounds__(kLightThreads) k_lookup_sparse(const SparseParams f) {
    extern __shared__ uint8_t smem_raw[];
    const NchwParams& p = f.e;
    const LookupArgs& a = f.a;
    uint8_t* stage = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 15) & ~uintptr_t(15));
    float* sv_s = reinterpret_cast<float*>(stage + kSparseStageCap);       // [chunk_channels] this CTA's slice
    float* rx = sv_s + p.chunk_channels;                                   // [2][P][kRxRow] (used in the first CTA)
    int* my_frames = reinterpret_cast<int*>(rx + 2 * kMaxCluster * kRxRow);  // [kSparseFrames]
    int* my_sids = my_frames + kSparseFrames;                              // [kSparseFrames] their stream ids
    int* s_scan = my_sids + kSparseFrames;                                 // [33]
    const int P = p.chunks_per_frame;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int B = a.B;
    const int rank = int(blockIdx.x) % P, group = int(blockIdx.x) / P;
    chain_wait();  // the exit flags are the previous kernel's
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * a.layer : nullptr);
    // The active frames of this cluster and their streams.  Exit flags and stream ids of eight tiles of frames
    // come in one trip to memory.
    uint8_t flags[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int sids[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int n_active = 0;
    for (int t0 = 0; t0 < B; t0 += kLightThreads) {
        const int b = t0 + tid;
        if ((t0 / kLightThreads) % 8 == 0) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                flags[u] = a.done[min(b + u * kLightThreads, B - 1)];
                sids[u] = a.stream_id ? a.stream_id[min(b + u * kLightThreads, B - 1)] : 0;
            }
        }
        uint8_t mine = 0;
        int sid_b = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            mine = ((t0 / kLightThreads) % 8 == u) ? flags[u] : mine;
            sid_b = ((t0 / kLightThreads) % 8 == u) ? sids[u] : sid_b;
        }
        const int act = (b < B && !mine) ? 1 : 0;
        int cnt;
        const int pos = block_exclusive_scan(act, s_scan, &cnt);
        if (act) {
            const int u = n_active + pos;
            if (u % f.groups == group && u / f.groups < kSparseFrames) {
                my_frames[u / f.groups] = b;
                my_sids[u / f.groups] = sid_b;
            }
        }
        n_active += cnt;
    }
    const int nu = n_active > group ? min((n_active - group + f.groups - 1) / f.groups, kSparseFrames) : 0;
    __syncthreads();
    const int c0 = rank * p.chunk_channels;
    const int nch = min(p.chunk_channels, p.C - c0);   // channels of this CTA's slice (a multiple of 4)
    const int vectors = nch * p.ch_bytes / 16;
    const int units = (nch + f.gran - 1) / f.gran;
    const int u_lo = min(units, warp * ((units + 3) / 4)), u_hi = min(units, u_lo + (units + 3) / 4);
    const int w_c0 = u_lo * f.gran, w_nch = min(nch, u_hi * f.gran) - w_c0;
    const int n4 = nch >> 2;
    const int pp = (n4 + kWarp - 1) / kWarp;       // 16-byte pieces of a centre's slice per lane (at most 8)
    const int spr = max(1, 8 / max(pp, 1));        // slots a warp scores per trip to memory
    const float weight = float(1u << a.layer);     // 2^(l-1) with l = layer + 1
    constexpr int kLoads = (kSparseStageCap / 16 + kLightThreads - 1) / kLightThreads;  // 13: a whole chunk in flight
    for (int k_it = 0; k_it < nu; ++k_it) {
        const int b = my_frames[k_it];
        const int sid = stream_checked(a, my_sids[k_it]);
        const uint4* src = reinterpret_cast<const uint4*>(p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes);
        uint4* dst = reinterpret_cast<uint4*>(stage);
        uint4 r[kLoads];
#pragma unroll
        for (int u = 0; u < kLoads; ++u) r[u] = load_once(src + min(u * kLightThreads + tid, vectors - 1));
        // the frame's fast memory: its size and this warp's classes (slot j = warp + 4 i), in flight with the chunk
        const int32_t* mem = a.members + (size_t)max(sid, 0) * a.k_max;
        const int k = sid < 0 ? 0 : min(a.k[sid], kFusedMaxK);
        int cls_w = 0;  // lane i < 16 holds the class of slot warp + 4 i
        if (lane < kFusedMaxK / 4 && warp + 4 * lane < a.k_max) cls_w = mem[warp + 4 * lane];
        // the finisher's own loads: the slots' classes (lane l: slots l and l + 32)
        int ids[2] = {0, 0};
        if (rank == 0 && warp == 0) {
            ids[0] = lane < a.k_max ? mem[lane] : 0;
            ids[1] = lane + kWarp < a.k_max ? mem[lane + kWarp] : 0;
        }
#pragma unroll
        for (int u = 0; u < kLoads; ++u)
            if (u * kLightThreads + tid < vectors) dst[u * kLightThreads + tid] = r[u];
        __syncthreads();
        if (w_nch > 0)
            R::run(stage + size_t(w_c0) * p.ch_bytes, w_nch, lane, p.sv + (long long)b * p.C + c0 + w_c0, sv_s + w_c0, p.inv_hw, p);
        __syncthreads();  // the slice is complete; the stage is free
        const uint32_t out = peer_smem(rx + ((k_it & 1) * kMaxCluster + rank) * kRxRow, 0);
        const float4* v4 = reinterpret_cast<const float4*>(sv_s);
        // the centres' lengths and the carry, for the finisher: in flight with the centre slices below
        float clen[2] = {0.f, 0.f}, sa_old[2] = {0.f, 0.f};
        if (rank == 0 && warp == 0) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = lane + h * kWarp;
                if (j < k) {
                    clen[h] = a.cnorm[ids[h]];
                    sa_old[h] = a.fresh ? 0.f : a.sa[(size_t)b * a.k_max + j];
                }
            }
        }
        if (warp == 3) {  // partial squared length of the semantic vector
            float nn = 0.f;
            for (int q = lane; q < n4; q += kWarp) {
                const float4 xv = v4[q];
                nn = fmaf(xv.x, xv.x, nn); nn = fmaf(xv.y, xv.y, nn); nn = fmaf(xv.z, xv.z, nn); nn = fmaf(xv.w, xv.w, nn);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) nn += __shfl_xor_sync(kFull, nn, o);
            if (lane == 0) peer_store(out + kFusedMaxK * 4, nn);
        }
        // this warp's slots, `spr` of them per trip to memory: eight pieces of centre slices per lane in flight
        for (int i0 = 0; warp + 4 * i0 < k; i0 += spr) {
            float4 c[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int si = e / pp, piece = e - si * pp;       // slot within the round, piece of its slice
                const int j = warp + 4 * (i0 + si), q = lane + piece * kWarp;
                const int cls = __shfl_sync(kFull, cls_w, min(i0 + si, kFusedMaxK / 4 - 1));
                c[e] = (si < spr && j < k && q < n4)
                           ? __ldg(reinterpret_cast<const float4*>(a.centers + (size_t)cls * p.C + c0) + q)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (int si = 0; si < spr; ++si) {
                const int j = warp + 4 * (i0 + si);
                if (j >= k) break;
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int q = lane + (e - si * pp) * kWarp;
                    if (e / pp == si && q < n4) {
                        const float4 xv = v4[q];
                        d = fmaf(c[e].x, xv.x, d); d = fmaf(c[e].y, xv.y, d); d = fmaf(c[e].z, xv.z, d); d = fmaf(c[e].w, xv.w, d);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(kFull, d, o);
                if (lane == 0) peer_store(out + j * 4, d);
            }
        }
        // every part of this frame has been delivered (and the previous frame's decision is made)
        if (P > 1) cluster_sync_all(); else __syncthreads();
        if (rank == 0 && warp == 0) {
            const float* rxb = rx + (k_it & 1) * kMaxCluster * kRxRow;
            float nn = 0.f, dots[2] = {0.f, 0.f};
            for (int rr = 0; rr < P; ++rr) {  // the parts in rank order
                const float* row = rxb + rr * kRxRow;
                nn += row[kFusedMaxK];
                if (lane < k) dots[0] += row[lane];
                if (lane + kWarp < k) dots[1] += row[lane + kWarp];
            }
            float s_cur[2] = {0.f, 0.f}, s_acc[2] = {0.f, 0.f};
            const float sv_len = __fsqrt_rn(nn);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int j = lane + h * kWarp;
                if (j < k) {
                    s_cur[h] = (nn == 0.f || clen[h] == 0.f) ? 0.f : __fdiv_rn(dots[h], __fmul_rn(sv_len, clen[h]));  // Eq. 1
                    s_acc[h] = __fmaf_rn(s_cur[h], weight, sa_old[h]);   // Eq. 3
                    a.sa[(size_t)b * a.k_max + j] = s_acc[h];
                } else if (a.fresh && j < a.k_max) {
                    a.sa[(size_t)b * a.k_max + j] = 0.f;                 // unused slots start from zero too
                }
            }
            const Top2 ta = warp_top2_keys(s_acc, ids, k, lane);
            Top2 ts{0.f, 0.f, -1, -1};
            if (a.sep) ts = warp_top2_keys(s_cur, ids, k, lane);  // only Eq. 2 (a diagnostic) needs it
            if (lane == 0) decide_from_top2(a, b, ta, ts);
        }
    }
    if (P > 1) cluster_sync_all();  // no CTA leaves while a peer may still write to its shared memory
}

// ---- NHWC: direct coalesced loads ----------------------------------------------------------

constexpr int kThreadsNhwc = 256;

template <class E>
__global__ void __launch_bounds__(kThreadsNhwc) k_encode_nhwc(const uint8_t* __restrict__ x,
                                                              const uint8_t* __restrict__ skip,
                                                              float* __restrict__ sv, int B, int C, int HW,
                                                              float inv_hw, unsigned long long* clock) {
    extern __shared__ float part[];  // [phases][min(C, 256 * kPerVec)]
    chain_wait();
    chain_release();
    const ClockScope stamps(clock);
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
                    const uint4 v0 = load_once(col + (long long)px * CG);
                    const uint4 v1 = load_once(col + (long long)(px + phases) * CG);
                    const uint4 v2 = load_once(col + (long long)(px + 2 * phases) * CG);
                    const uint4 v3 = load_once(col + (long long)(px + 3 * phases) * CG);
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
                    const uint4 v = load_once(col + (long long)px * CG);
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

// ---- NHWC, small fast memory: pooling, scoring and the decision by one CTA per frame ---------------
//
// A frame of an NHWC map is H*W rows of C channels: pooling is a column sum, and one CTA holds all of a
// frame's column sums at the end, so the same CTA goes on to Eq. 1, Eq. 3, Eq. 4 and the exit rule (one
// launch per layer).  Thread = (16-byte column group, pixel phase); every thread keeps eight loads in
// flight (a frame is a few dozen KB: the CTA's time is the number of trips to memory it makes); the
// phases are added in ascending order through shared memory.  Frames that have exited cost a CTA that
// leaves at once.
constexpr int kThreadsNhwcLookup = 512;  // more threads, fewer trips to memory per thread: a frame is one CTA's

template <class E>
__global__ void __launch_bounds__(kThreadsNhwcLookup) k_lookup_nhwc(const uint8_t* __restrict__ x, int C, int HW, float inv_hw,
                                                                    float* __restrict__ sv_out, const LookupArgs a) {
    extern __shared__ float nhwc_smem[];  // sv [C] | s_cur [k_max] | s_acc [k_max] | classes [k_max] | part [phases][cgs * V]
    __shared__ float scratch[32];
    float* sv_s = nhwc_smem;
    float* s_cur = sv_s + C;
    float* s_acc = s_cur + a.k_max;
    float* part = s_acc + 2 * a.k_max;
    chain_wait();
    chain_release();
    const ClockScope stamps(a.clock ? a.clock + 2 * a.layer : nullptr);
    const int b = blockIdx.x;
    const int sid_raw = a.stream_id ? a.stream_id[b] : 0;  // in flight with the exit flag
    if (!a.fresh && a.done[b]) return;
    const SlotPrefetch pf = prefetch_slots(a, sid_raw);    // in flight with the map
    constexpr int V = E::kPerVec;
    constexpr int T = kThreadsNhwcLookup;
    const int CG = C / V;  // 16-byte vectors per pixel
    const uint4* f = reinterpret_cast<const uint4*>(x + (long long)b * HW * C * E::kSize);
    float nrm = 0.f;
    for (int cg0 = 0; cg0 < CG; cg0 += T) {
        const int cgs = min(CG - cg0, T);  // column groups handled in this sweep
        const int phases = T / cgs;
        const int ph = threadIdx.x / cgs, cg = threadIdx.x - ph * cgs;
        float acc[V];
#pragma unroll
        for (int j = 0; j < V; ++j) acc[j] = 0.f;
        if (ph < phases) {
            const uint4* col = f + cg0 + cg;
            for (int px = ph; px < HW; px += 8 * phases) {
                uint4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = load_once(col + (long long)min(px + u * phases, HW - 1) * CG);
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (px + u * phases < HW) {
#pragma unroll
                        for (int j = 0; j < V; ++j) acc[j] += E::at(v[u], j);
                    }
            }
            float* dst = part + (size_t(ph) * cgs + cg) * V;
#pragma unroll
            for (int j = 0; j < V; ++j) dst[j] = acc[j];
        }
        __syncthreads();
        for (int c = threadIdx.x; c < cgs * V; c += T) {
            float s = 0.f;
            for (int q = 0; q < phases; ++q) s += part[size_t(q) * cgs * V + c];
            s *= inv_hw;
            sv_s[cg0 * V + c] = s;
            sv_out[(long long)b * C + cg0 * V + c] = s;
            nrm = fmaf(s, s, nrm);
        }
        __syncthreads();
    }
    nrm = block_sum(nrm, scratch);  // also orders the shared writes above
    score_frame(a, b, pf, sv_s, nrm, s_cur, s_acc);
}

// ---- any shape: one thread per (frame, channel) ---------------------------------------------

template <class E>
__global__ void k_encode_generic(const void* __restrict__ x, const uint8_t* __restrict__ skip,
                                 float* __restrict__ sv, int B, int C, int HW, int nhwc, float inv_hw,
                                 unsigned long long* clock) {
    chain_wait();
    chain_release();
    const ClockScope stamps(clock);
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
    chain_wait();
    chain_release();
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

constexpr size_t nchw_smem(int stages) { return size_t(stages) * kStageCap + 2 * size_t(stages) * sizeof(uint64_t) + 128; }

template <class R>
cudaError_t launch_nchw(const NchwParams& p, int grid, cudaStream_t st) {
    return launch_chained(k_encode_nchw<R>, grid, (p.consumers + 1) * kWarp, nchw_smem(p.stages), st, p);
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
                          int(a.layout == SMTM_NHWC), 1.0f / float(a.H * a.W), a.clock);
}

template <class E>
cudaError_t launch_nhwc(const EncodeArgs& a, cudaStream_t st) {
    const int CG = a.C / E::kPerVec;
    const int cgs = std::min(CG, kThreadsNhwc);
    const size_t smem = size_t(kThreadsNhwc / cgs) * cgs * E::kPerVec * sizeof(float);
    return launch_chained(k_encode_nhwc<E>, a.B, kThreadsNhwc, smem, st, static_cast<const uint8_t*>(a.x), a.skip, a.sv,
                          a.B, a.C, a.H * a.W, 1.0f / float(a.H * a.W), a.clock);
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
    p->clock = a.clock;
    p->C = a.C;
    p->ch_bytes = HW * es;
    p->frame_bytes = (long long)a.C * p->ch_bytes;
    p->inv_hw = 1.0f / float(HW);
    p->max_in_flight = a.ring_in_flight > 0 ? std::min(a.ring_in_flight, kMaxInFlight) : kMaxInFlight;
    p->stages = (a.ring_stages >= 2 && a.ring_stages <= kStages) ? a.ring_stages : kStages;
    if (p->max_in_flight > p->stages - 1) p->max_in_flight = p->stages - 1;
    p->consumers = (a.ring_consumers >= 1 && a.ring_consumers <= kConsumers) ? a.ring_consumers : kConsumers;
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
    return cudaFuncSetAttribute(k_lookup_nchw<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemLimit));
}

// Clusters of `parts` CTAs of the fused kernel that the device runs at once (each CTA fills an SM).
template <class R>
cudaError_t max_clusters(int parts, size_t smem, int* out) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(parts));
    cfg.blockDim = dim3(kThreadsFused);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = unsigned(parts);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaOccupancyMaxActiveClusters(out, k_lookup_nchw<R>, &cfg);
}

}  // namespace

template <class R>
cudaError_t carveout_pipelined() {
    cudaError_t e = prefer_max_smem_carveout(k_encode_nchw<R>);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_pool_sparse<R>);
    if (e == cudaSuccess) e = prefer_max_smem_carveout(k_lookup_sparse<R>);
    if (e == cudaSuccess) e = allow_max_dynamic_smem(k_lookup_sparse<R>);
    return e;
}

cudaError_t encode_setup() {
    cudaError_t e = allow_max_dynamic_smem(k_lookup_nhwc<F32>);
    if (e == cudaSuccess) e = allow_max_dynamic_smem(k_lookup_nhwc<F16>);
    if (e == cudaSuccess) e = allow_max_dynamic_smem(k_lookup_nhwc<BF16>);
#define SMTM_OPT_IN(...)                                        \
    if (e == cudaSuccess) e = opt_in<__VA_ARGS__>();            \
    if (e == cudaSuccess) e = carveout_pipelined<__VA_ARGS__>();  \
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

bool launch_encode_nhwc_vector_supported(const EncodeArgs& a) {
    if (a.layout != SMTM_NHWC || a.B <= 0) return false;
    return a.C % (a.dtype == SMTM_F32 ? 4 : 8) == 0;
}

bool launch_encode_ring_supported(const EncodeArgs& a) {
    if (a.layout != SMTM_NCHW || a.B <= 0) return false;
    NchwParams p;
    return plan_nchw(a, &p) != kNone;
}

bool launch_pool_sparse_supported(const EncodeArgs& a) {
    if (a.layout != SMTM_NCHW || a.B <= 0) return false;
    NchwParams p;
    const Reducer r = plan_nchw(a, &p);
    return r != kNone && p.ch_bytes <= kLightStageCap;
}

cudaError_t launch_pool_sparse(const EncodeArgs& a, int sm_count, cudaStream_t st, int64_t* launches) {
    LightParams f{};
    const Reducer r = plan_nchw(a, &f.e);
    if (r == kNone || f.e.ch_bytes > kLightStageCap) return cudaErrorInvalidValue;
    // chunks of at most kLightStageCap bytes: half the units of a unit-per-lane chunk, or as many whole channels as fit
    const bool unit = r <= kUnitF32x49;
    f.gran = unit ? f.e.chunk_channels / 32 : std::max(1, 32 / std::max(1, f.e.team));
    if (unit) {
        f.e.chunk_channels /= 2;
    } else {
        int cc = kLightStageCap / f.e.ch_bytes;
        if (cc > f.gran) cc -= cc % f.gran;
        f.e.chunk_channels = std::min(cc, a.C);
    }
    f.e.chunks_per_frame = (a.C + f.e.chunk_channels - 1) / f.e.chunk_channels;
    f.e.total_chunks = (long long)a.B * f.e.chunks_per_frame;
    // about four CTAs to an SM; enough groups that no CTA is given more frames than it can list
    const int cpf = f.e.chunks_per_frame;
    int groups = std::max(1, std::min(a.B, 8 * sm_count / cpf));
    groups = std::max(groups, (a.B + kLightFrames - 1) / kLightFrames);
    f.groups = groups;
    cudaError_t e = cudaSuccess;
    ++*launches;
#define SMTM_LAUNCH(...) e = launch_chained(k_pool_sparse<__VA_ARGS__>, cpf * groups, kLightThreads, 0, st, f)
    SMTM_FOR_REDUCER(r, SMTM_LAUNCH)
#undef SMTM_LAUNCH
    return e;
}

// The layout of a sparse lookup, or kNone when the shape is not served: chunks as the streaming kernel cuts
// them, at most 8 to a frame, slices that are whole 16-byte pieces and fit the scorers' registers.
Reducer plan_sparse(const EncodeArgs& e, const LookupArgs& a, SparseParams* f) {
    if (e.layout != SMTM_NCHW || e.B <= 0 || a.k_max > kFusedMaxK || (e.C & 3)) return kNone;
    const Reducer r = plan_nchw(e, &f->e);
    if (r == kNone) return kNone;
    if (f->e.chunks_per_frame > kMaxCluster || (f->e.chunk_channels & 3) || f->e.chunk_channels > kSparseSlice) return kNone;
    f->gran = r <= kUnitF32x49 ? f->e.chunk_channels / 32 : std::max(1, 32 / std::max(1, f->e.team));
    return r;
}

bool launch_lookup_sparse_supported(const EncodeArgs& e, const LookupArgs& a) {
    SparseParams f{};
    return plan_sparse(e, a, &f) != kNone;
}

cudaError_t launch_lookup_sparse(const EncodeArgs& e, const LookupArgs& a, int sm_count, cudaStream_t st, int64_t* launches) {
    SparseParams f{};
    const Reducer r = plan_sparse(e, a, &f);
    if (r == kNone) return cudaErrorInvalidValue;
    f.a = a;
    const int P = f.e.chunks_per_frame;
    // about three CTAs to an SM (they sit beside a streaming kernel); enough clusters that none is given more
    // frames than it can list
    int groups = std::max(1, std::min(e.B, 3 * sm_count / P));
    groups = std::max(groups, (e.B + kSparseFrames - 1) / kSparseFrames);
    f.groups = groups;
    const size_t smem = sparse_smem(f.e.chunk_channels);
    cudaError_t err = cudaSuccess;
    ++*launches;
    // (in stream order, without the early start: the clusters would wait on the SMs for the scoring kernel before
    // them and keep the next step's pooling CTAs out meanwhile)
#define SMTM_LAUNCH(...) err = launch_ordered_cluster(k_lookup_sparse<__VA_ARGS__>, P * groups, kLightThreads, smem, P, st, f)
    SMTM_FOR_REDUCER(r, SMTM_LAUNCH)
#undef SMTM_LAUNCH
    return err;
}

cudaError_t launch_lookup_fused(const EncodeArgs& e, const LookupArgs& a, int sm_count, FusedCaps* caps, cudaStream_t st,
                                int64_t* launches, bool* handled, const cudaEvent_t* timing) {
    *handled = false;
    if (e.B <= 0 || a.k_max > kFusedMaxK) return cudaSuccess;
    if (e.layout == SMTM_NHWC) {
        const int V = e.dtype == SMTM_F32 ? 4 : 8;
        if (e.C % V || e.C > 8192) return cudaSuccess;
        const int cgs = std::min(e.C / V, kThreadsNhwcLookup);
        const size_t smem = (size_t(e.C) + 3 * size_t(a.k_max) + size_t(kThreadsNhwcLookup / cgs) * cgs * V) * sizeof(float);
        const float inv_hw = 1.0f / float(e.H * e.W);
        const uint8_t* x = static_cast<const uint8_t*>(e.x);
        cudaError_t err = cudaSuccess;
        if (timing) record_timing(timing[0], st);
        if (e.dtype == SMTM_F32) err = launch_chained(k_lookup_nhwc<F32>, e.B, kThreadsNhwcLookup, smem, st, x, e.C, e.H * e.W, inv_hw, e.sv, a);
        else if (e.dtype == SMTM_F16) err = launch_chained(k_lookup_nhwc<F16>, e.B, kThreadsNhwcLookup, smem, st, x, e.C, e.H * e.W, inv_hw, e.sv, a);
        else err = launch_chained(k_lookup_nhwc<BF16>, e.B, kThreadsNhwcLookup, smem, st, x, e.C, e.H * e.W, inv_hw, e.sv, a);
        if (timing) record_timing(timing[1], st);
        ++*launches;
        *handled = true;
        return err;
    }
    FusedParams f{};
    const Reducer r = plan_nchw(e, &f.e);
    if (r == kNone) return cudaSuccess;
    const int cpf = f.e.chunks_per_frame;
    if (e.C & 3) return cudaSuccess;
    // Parts per frame = CTAs per cluster.  A part must fit the scorers' registers (slice <= kMaxSlice
    // channels, a multiple of 4) and the CTA's shared memory; among 1, 2, 4, 8 take the smallest
    // that keeps the SMs 95 % busy over the rounds of frames (else the busiest).
    static_assert(kTeamBf16 < 16 && kMaxCluster < 9, "FusedCaps holds an entry per (reducer, cluster size)");
    int best_P = 0, best_grid = 0;
    double best_eff = -1.0;
    for (int P = 1; P <= kMaxCluster; P *= 2) {
        if (cpf % P || (cpf / P) * f.e.chunk_channels > kMaxSlice) continue;
        if (((cpf / P) * f.e.chunk_channels) & 3) continue;  // the scorers read a part's slice as 16-byte vectors
        const size_t smem = fused_smem((cpf / P) * f.e.chunk_channels, P);
        if (smem > kSmemLimit) continue;
        int clusters = sm_count;
        if (P > 1) {
            int& cap = caps->clusters[r][P];  // clusters the device runs at once, 0 = not asked yet
            if (cap == 0) {
                cudaError_t err = cudaSuccess;
#define SMTM_ASK(...) err = max_clusters<__VA_ARGS__>(P, smem, &cap)
                SMTM_FOR_REDUCER(r, SMTM_ASK)
#undef SMTM_ASK
                if (err != cudaSuccess) {
                    (void)cudaGetLastError();
                    cap = -1;
                }
            }
            if (cap <= 0) continue;
            clusters = std::min(cap, sm_count / P);
        }
        if (clusters < 1 || ((long long)e.B + clusters - 1) / clusters > kMaxUnits) continue;
        const double rounds = double(e.B) / clusters;
        const double eff = rounds / std::ceil(rounds) * double(clusters * P) / sm_count;
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best_P = P;
            best_grid = clusters * P;
        }
        if (eff >= 0.95) break;
    }
    if (best_P == 0) return cudaSuccess;
    const int P = best_P;
    f.a = a;
    f.parts = P;
    f.chunks_per_unit = cpf / P;
    f.slice_cap = f.chunks_per_unit * f.e.chunk_channels;
    const size_t smem = fused_smem(f.slice_cap, P);
    cudaError_t err = cudaSuccess;
    if (timing) record_timing(timing[0], st);
#define SMTM_LAUNCH(...) err = launch_chained_cluster(k_lookup_nchw<__VA_ARGS__>, best_grid, kThreadsFused, smem, P, st, f)
    SMTM_FOR_REDUCER(r, SMTM_LAUNCH)
#undef SMTM_LAUNCH
    if (timing) record_timing(timing[1], st);
    ++*launches;
    *handled = true;
    return err;
}

cudaError_t launch_row_norm2(const float* sv, const uint8_t* skip, int B, int D, float* out, cudaStream_t st,
                             int64_t* launches) {
    if (B <= 0) return cudaSuccess;
    ++*launches;
    return launch_chained(k_row_norm2, B, 256, 0, st, sv, skip, B, D, out);
}

}  // namespace smtm
