// Adaptive priming memory (Sec. 6): frequency / time-stamp tables, running-mean centres
// (Eq. 7), replacement score and top-k (Eq. 5), adaptive fast-memory size (Eq. 6).
//
// All reductions are segmented and atomics-free: a CTA owns a stream's tables, or one
// (class, layer) centre, and walks the batch in ascending frame index, so the result is
// the one a frame-by-frame replay would give and does not depend on scheduling.
#include "common.cuh"
#include "internal.h"

namespace smtm {

namespace {

constexpr int kFtMax = 1 << 20;  // frequency counts saturate here so that Eq. 6's sums fit 64 bits
constexpr int kEMax = 12;        // floor(TS / W) is clamped here: 0.25^12 of a count is below one

// Label and stop layer of a finished frame: the prediction and exit layer if it exited,
// else the fallback label (the full network's answer, -1 = none) and L.
__device__ __forceinline__ int final_label(const UpdateArgs& a, int b) {
    return a.done[b] ? a.pred[b] : (a.fallback ? a.fallback[b] : -1);
}
__device__ __forceinline__ int stop_layer(const UpdateArgs& a, int b) { return a.done[b] ? a.exit_layer[b] : a.L; }

constexpr int kUpdThreads = 256;
constexpr int kSliceCols = kUpdThreads * 4;  // columns of a centre handled by one CTA (one float4 per thread)

// Compacts, in ascending frame index, the frames of [t0, t0 + kUpdThreads) for which `hit`
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

// blockIdx.x <  S : frequency / time-stamp tables of stream blockIdx.x
// blockIdx.x >= S : centre of (class, layer) = divmod(blockIdx.x - S, L)
__global__ void __launch_bounds__(kUpdThreads) k_update(const UpdateArgs a) {
    __shared__ int s_list[kUpdThreads];
    __shared__ int s_scan[33];
    __shared__ float s_red[32];
    const int tid = threadIdx.x;

    if (int(blockIdx.x) < a.S) {
        // ---- Sec. 6.1: the stream's frames, in ascending index, replayed per class ----------
        const int s = blockIdx.x;
        for (int t0 = 0; t0 < a.B; t0 += kUpdThreads) {
            const int b = t0 + tid;
            const int hit = (b < a.B && (a.stream_id ? a.stream_id[b] : 0) == s) ? 1 : 0;
            const int cnt = compact_tile(hit, hit ? final_label(a, b) : -1, s_list, s_scan);
            if (cnt == 0) continue;
            for (int c = tid; c < a.n; c += kUpdThreads) {
                int f = a.ft[(size_t)s * a.n + c], t = a.ts[(size_t)s * a.n + c];
                for (int i = 0; i < cnt; ++i) {
                    if (s_list[i] == c) {
                        f = min(f + 1, kFtMax);
                        t = 0;
                    } else if (t < INT32_MAX) {
                        ++t;
                    }
                }
                a.ft[(size_t)s * a.n + c] = f;
                a.ts[(size_t)s * a.n + c] = t;
            }
        }
        return;
    }

    // ---- Eq. 7 for one (class, layer): fold the matching frames in ascending index --------
    const int job = blockIdx.x - a.S;
    const int cls = job / a.L, l0 = job - cls * a.L;  // l0 is 0-based here; the paper's l0 is l0 + 1
    const int D = a.dims[l0];
    const bool vec = (D & 3) == 0;  // rows are 16-byte aligned
    const float* sv = a.sv[l0];
    float* cen = a.centers[l0] + (size_t)cls * D;
    const float m = float(a.m[l0][cls]);
    float nrm = 0.f;
    int q = 0;
    for (int d0 = 0; d0 < D; d0 += kSliceCols) {  // a slice of columns per sweep, four per thread
        const int d = d0 + tid * 4;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        q = 0;
        for (int t0 = 0; t0 < a.B; t0 += kUpdThreads) {
            const int b = t0 + tid;
            const int hit = (b < a.B && final_label(a, b) == cls && stop_layer(a, b) >= l0 + 1) ? 1 : 0;
            const int cnt = compact_tile(hit, b, s_list, s_scan);
            if (cnt == 0) continue;
            q += cnt;
            if (d >= D) continue;
            if (vec) {
#pragma unroll 4
                for (int i = 0; i < cnt; ++i) {
                    const float4 r = __ldg(reinterpret_cast<const float4*>(sv + (size_t)s_list[i] * D + d));
                    acc[0] += r.x; acc[1] += r.y; acc[2] += r.z; acc[3] += r.w;
                }
            } else {
                for (int i = 0; i < cnt; ++i)
                    for (int j = 0; j < 4; ++j)
                        if (d + j < D) acc[j] += sv[(size_t)s_list[i] * D + d + j];
            }
        }
        if (q == 0) return;  // class not seen at this layer in this batch: nothing changes
        for (int j = 0; j < 4; ++j)
            if (d + j < D) {
                const float v = __fdiv_rn(__fmaf_rn(cen[d + j], m, acc[j]), m + float(q));
                cen[d + j] = v;
                nrm = fmaf(v, v, nrm);
            }
    }
    nrm = block_sum(nrm, s_red);
    if (tid == 0) {
        a.cnorm[l0][cls] = __fsqrt_rn(nrm);
        a.m[l0][cls] += (uint32_t)q;
    }
}

__global__ void k_center_norms(const float* __restrict__ centers, int n, int D, float* __restrict__ cnorm) {
    __shared__ float s_red[32];
    const int c = blockIdx.x;
    float nrm = 0.f;
    for (int d = threadIdx.x; d < D; d += blockDim.x) {
        const float v = centers[(size_t)c * D + d];
        nrm = fmaf(v, v, nrm);
    }
    nrm = block_sum(nrm, s_red);
    if (threadIdx.x == 0) cnorm[c] = __fsqrt_rn(nrm);
}

// ---- Eq. 5 / Eq. 6 ------------------------------------------------------------------------

constexpr int kRszThreads = 256;

__device__ __forceinline__ unsigned long long score_of(int ft, int ts, int W) {
    int e = ts / W;
    if (e > kEMax) e = kEMax;
    const unsigned long long f = (unsigned long long)min(max(ft, 0), kFtMax);
    return f << (2 * (kEMax - e));  // FT * 4^(12 - e) = 4^12 * FT * 0.25^e
}

// One CTA per stream.  Classes with a non-zero score are compacted in ascending id and
// ranked among themselves by counting; zero-score classes follow in ascending id.
__global__ void __launch_bounds__(kRszThreads) k_resize(const ResizeArgs a) {
    extern __shared__ unsigned long long s_score[];                  // [n] compacted non-zero scores
    int* s_id = reinterpret_cast<int*>(s_score + a.n);               // [n] their class ids
    unsigned long long* s_top = reinterpret_cast<unsigned long long*>(s_id + a.n + (a.n & 1));  // [k_max]
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[kRszThreads / 32];
    const int s = blockIdx.x, tid = threadIdx.x;
    const int32_t* ft = a.ft + (size_t)s * a.n;
    const int32_t* ts = a.ts + (size_t)s * a.n;
    int32_t* mem = a.members + (size_t)s * a.k_max;

    // pass 1: compact the non-zero scores (ascending id) and add everything up
    int nz = 0;
    unsigned long long local = 0;
    for (int c0 = 0; c0 < a.n; c0 += kRszThreads) {
        const int c = c0 + tid;
        const unsigned long long sc = c < a.n ? score_of(ft[c], ts[c], a.W) : 0ull;
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
    if ((tid & 31) == 0) s_part[tid >> 5] = local;
    __syncthreads();
    unsigned long long total = 0;
    for (int w = 0; w < kRszThreads / 32; ++w) total += s_part[w];
    if (total == 0) return;  // nothing seen yet: keep size and members

    // pass 2: rank the non-zero classes; rank r < k_max goes to slot r
    for (int i = tid; i < nz; i += kRszThreads) {
        const unsigned long long sc = s_score[i];
        int r = 0;
        for (int j = 0; j < nz; ++j) {
            const unsigned long long o = s_score[j];
            r += (o > sc || (o == sc && j < i)) ? 1 : 0;  // compacted order is ascending id
        }
        if (r < a.k_max) {
            mem[r] = s_id[i];
            s_top[r] = sc;
        }
    }
    // pass 3: zero-score classes fill the remaining slots in ascending id
    if (nz < a.k_max) {
        int filled = nz;
        for (int c0 = 0; c0 < a.n && filled < a.k_max; c0 += kRszThreads) {
            const int c = c0 + tid;
            const int z = (c < a.n && score_of(ft[c], ts[c], a.W) == 0) ? 1 : 0;
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
    if (tid == 0) {
        unsigned long long prefix = 0;
        int chosen = a.k_max;
        for (int i = 0; i < a.k_max; ++i) {
            prefix += s_top[i];
            if (i + 1 >= a.k_min && (unsigned long long)a.cl_den * prefix > (unsigned long long)a.cl_num * total) {
                chosen = i + 1;
                break;
            }
        }
        a.k[s] = chosen;
    }
}

}  // namespace

cudaError_t launch_center_norms(const float* centers, int n, int D, float* cnorm, cudaStream_t st,
                                int64_t* launches) {
    ++*launches;
    k_center_norms<<<n, 256, 0, st>>>(centers, n, D, cnorm);
    return cudaGetLastError();
}

cudaError_t launch_update(const UpdateArgs& a, cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    ++*launches;
    k_update<<<a.S + a.n * a.L, kUpdThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_resize(const ResizeArgs& a, cudaStream_t st, int64_t* launches) {
    const size_t smem = size_t(a.n) * 8 + size_t(a.n + (a.n & 1)) * 4 + size_t(a.k_max) * 8;
    static size_t opted = 48 * 1024;
    if (smem > opted) {
        cudaError_t e = cudaFuncSetAttribute(k_resize, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
        if (e != cudaSuccess) return e;
        opted = smem;
    }
    ++*launches;
    k_resize<<<a.S, kRszThreads, smem, st>>>(a);
    return cudaGetLastError();
}

}  // namespace smtm
