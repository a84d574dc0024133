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

#include "common.cuh"
#include "internal.h"

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
};

// ---- reducers --------------------------------------------------------------------------

// Lane i reduces unit i: G channels of HW elements stored as UW consecutive 16-byte vectors.
template <class E, int HW>
struct UnitPerLane {
    static constexpr int kUnitBytesRaw = HW * E::kSize;
    static constexpr int gcd16(int a) { return (a % 16 == 0) ? 16 : (a % 8 == 0) ? 8 : (a % 4 == 0) ? 4 : (a % 2 == 0) ? 2 : 1; }
    static constexpr int G = 16 / gcd16(kUnitBytesRaw);
    static constexpr int UW = G * kUnitBytesRaw / 16;

    static __device__ __forceinline__ void run(const uint8_t* stage, int nch, int lane, float* out, float inv_hw,
                                               const NchwParams&) {
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
    }
};

// T lanes per channel; channel bytes are a multiple of 16.
template <class E>
struct TeamPerChannel {
    static __device__ __forceinline__ void run(const uint8_t* stage, int nch, int lane, float* out, float inv_hw,
                                               const NchwParams& p) {
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
            if (c < nch && r == 0) out[c] = s * inv_hw;
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
    __syncthreads();

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
                const uint32_t bytes = uint32_t(nch) * uint32_t(p.ch_bytes);
                mbar_expect_tx(&full[stage], bytes);
                bulk_load(stages + size_t(stage) * kStageCap,
                          p.x + (long long)b * p.frame_bytes + (long long)c0 * p.ch_bytes, bytes, &full[stage]);
            } else if (stage % kConsumers == warp) {
                if (!mbar_wait_bounded(&full[stage], use & 1, p.status)) {
                    failed = true;
                    break;
                }
                R::run(stages + size_t(stage) * kStageCap, nch, lane, p.sv + (long long)b * p.C + c0, p.inv_hw, p);
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

// ---- NHWC: direct coalesced loads ----------------------------------------------------------

constexpr int kThreadsNhwc = 256;

template <class E>
__global__ void __launch_bounds__(kThreadsNhwc) k_encode_nhwc(const uint8_t* __restrict__ x,
                                                              const uint8_t* __restrict__ skip,
                                                              float* __restrict__ sv, int B, int C, int HW,
                                                              float inv_hw) {
    extern __shared__ float part[];  // [phases][min(C, 256 * kPerVec)]
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
    k_encode_nchw<R><<<grid, kThreadsTma, kSmemTma, st>>>(p);
    return cudaGetLastError();
}

template <class R>
cudaError_t opt_in() {
    return cudaFuncSetAttribute(k_encode_nchw<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmemTma));
}

template <class E>
cudaError_t launch_generic(const EncodeArgs& a, cudaStream_t st) {
    const long long total = (long long)a.B * a.C;
    const int grid = int(std::min<long long>((total + 255) / 256, 148 * 16));
    k_encode_generic<E><<<grid, 256, 0, st>>>(a.x, a.skip, a.sv, a.B, a.C, a.H * a.W, a.layout == SMTM_NHWC,
                                               1.0f / float(a.H * a.W));
    return cudaGetLastError();
}

template <class E>
cudaError_t launch_nhwc(const EncodeArgs& a, cudaStream_t st) {
    const int CG = a.C / E::kPerVec;
    const int cgs = std::min(CG, kThreadsNhwc);
    const size_t smem = size_t(kThreadsNhwc / cgs) * cgs * E::kPerVec * sizeof(float);
    k_encode_nhwc<E><<<a.B, kThreadsNhwc, smem, st>>>(static_cast<const uint8_t*>(a.x), a.skip, a.sv, a.B, a.C,
                                                      a.H * a.W, 1.0f / float(a.H * a.W));
    return cudaGetLastError();
}

int pow2_floor(int v) {
    int p = 1;
    while (p * 2 <= v) p *= 2;
    return p;
}

}  // namespace

cudaError_t encode_setup() {
    cudaError_t e;
    if ((e = opt_in<UnitPerLane<BF16, 49>>()) != cudaSuccess) return e;
    if ((e = opt_in<UnitPerLane<BF16, 196>>()) != cudaSuccess) return e;
    if ((e = opt_in<UnitPerLane<F16, 49>>()) != cudaSuccess) return e;
    if ((e = opt_in<UnitPerLane<F16, 196>>()) != cudaSuccess) return e;
    if ((e = opt_in<UnitPerLane<F32, 49>>()) != cudaSuccess) return e;
    if ((e = opt_in<TeamPerChannel<BF16>>()) != cudaSuccess) return e;
    if ((e = opt_in<TeamPerChannel<F16>>()) != cudaSuccess) return e;
    if ((e = opt_in<TeamPerChannel<F32>>()) != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_encode(const EncodeArgs& a, int sm_count, cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    const int HW = a.H * a.W;
    const int es = a.dtype == SMTM_F32 ? 4 : 2;
    const float inv_hw = 1.0f / float(HW);
    ++*launches;

    if (a.layout == SMTM_NHWC) {
        const int V = 16 / es;
        if (a.C % V == 0) {
            if (a.dtype == SMTM_F32) return launch_nhwc<F32>(a, st);
            if (a.dtype == SMTM_F16) return launch_nhwc<F16>(a, st);
            return launch_nhwc<BF16>(a, st);
        }
    } else {
        NchwParams p{};
        p.x = static_cast<const uint8_t*>(a.x);
        p.skip = a.skip;
        p.sv = a.sv;
        p.status = a.status;
        p.C = a.C;
        p.ch_bytes = HW * es;
        p.frame_bytes = (long long)a.C * p.ch_bytes;
        p.inv_hw = inv_hw;
        const int grid = sm_count;
        // unit-per-lane shapes (compile-time H*W)
        int G = 0;
        if ((HW == 49 || HW == 196) && es == 2) G = HW == 49 ? 8 : 2;
        if (HW == 49 && es == 4) G = 4;
        if (G && a.C % G == 0) {
            p.chunk_channels = 32 * G;
            p.chunks_per_frame = (a.C + p.chunk_channels - 1) / p.chunk_channels;
            p.total_chunks = (long long)a.B * p.chunks_per_frame;
            if (es == 4) return launch_nchw<UnitPerLane<F32, 49>>(p, grid, st);
            if (a.dtype == SMTM_BF16)
                return HW == 49 ? launch_nchw<UnitPerLane<BF16, 49>>(p, grid, st)
                                : launch_nchw<UnitPerLane<BF16, 196>>(p, grid, st);
            return HW == 49 ? launch_nchw<UnitPerLane<F16, 49>>(p, grid, st)
                            : launch_nchw<UnitPerLane<F16, 196>>(p, grid, st);
        }
        // team-per-channel: channel bytes a multiple of 16 and at most one stage
        if (p.ch_bytes % 16 == 0 && p.ch_bytes <= kStageCap) {
            p.vec_per_channel = p.ch_bytes / 16;
            p.team = std::min(32, pow2_floor(std::max(1, p.vec_per_channel / 4)));
            const int per_pass = 32 / p.team;
            int cc = kStageCap / p.ch_bytes;
            if (cc > per_pass) cc -= cc % per_pass;
            p.chunk_channels = std::min(cc, a.C);
            p.chunks_per_frame = (a.C + p.chunk_channels - 1) / p.chunk_channels;
            p.total_chunks = (long long)a.B * p.chunks_per_frame;
            if (a.dtype == SMTM_F32) return launch_nchw<TeamPerChannel<F32>>(p, grid, st);
            if (a.dtype == SMTM_F16) return launch_nchw<TeamPerChannel<F16>>(p, grid, st);
            return launch_nchw<TeamPerChannel<BF16>>(p, grid, st);
        }
    }
    if (a.dtype == SMTM_F32) return launch_generic<F32>(a, st);
    if (a.dtype == SMTM_F16) return launch_generic<F16>(a, st);
    return launch_generic<BF16>(a, st);
}

cudaError_t launch_row_norm2(const float* sv, const uint8_t* skip, int B, int D, float* out, cudaStream_t st,
                             int64_t* launches) {
    if (B <= 0) return cudaSuccess;
    ++*launches;
    k_row_norm2<<<B, 256, 0, st>>>(sv, skip, B, D, out);
    return cudaGetLastError();
}

}  // namespace smtm
