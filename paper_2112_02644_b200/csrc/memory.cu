// Adaptive priming memory (Sec. 6): frequency / time-stamp tables, running-mean centres
// (Eq. 7), replacement score and top-k (Eq. 5), adaptive fast-memory size (Eq. 6).
//
// All reductions are segmented and atomics-free: a CTA owns a stream's tables, or one
// (class, layer) centre, and walks the batch in ascending frame index, so the result is
// the one a frame-by-frame replay would give and does not depend on scheduling.
//
// An update is two launches.  k_update_plan (one CTA) writes every frame's final label and
// stop layer and lists the first frame of every class and of every stream present in the
// batch.  k_update_apply then starts one CTA per listed stream (tables, optionally followed
// by that stream's Eq. 5 / Eq. 6 refresh) and one per (listed class, layer) (Eq. 7); classes
// and streams the batch does not touch cost nothing.
#include <algorithm>

#include "common.cuh"
#include "internal.h"

namespace smtm {

namespace {

constexpr int kFtMax = 1 << 20;  // frequency counts saturate here so that Eq. 6's sums fit 64 bits
constexpr int kEMax = 12;        // floor(TS / W) is clamped here: 0.25^12 of a count is below one

constexpr int kPlanThreads = 1024;
constexpr int kUpdThreads = 256;
constexpr int kSliceCols = kUpdThreads * 4;  // columns of a centre handled per sweep (one float4 per thread)

// ---- plan -----------------------------------------------------------------------------------

// Label and stop layer of a finished frame: the prediction and exit layer if it exited,
// else the fallback label (the full network's answer, -1 = none) and L.
__global__ void __launch_bounds__(kPlanThreads) k_update_plan(const UpdateArgs a) {
    extern __shared__ int s_keys[];  // [B] labels, [B] stream ids
    int* s_lab = s_keys;
    int* s_sid = s_keys + a.B;
    __shared__ int s_scan[33];
    const int tid = threadIdx.x;
    for (int b = tid; b < a.B; b += kPlanThreads) {
        const bool ex = a.done[b] != 0;
        const int lab = ex ? a.pred[b] : (a.fallback ? a.fallback[b] : -1);
        s_lab[b] = lab;
        s_sid[b] = a.stream_id ? a.stream_id[b] : 0;
        a.plan.final_label[b] = lab;
        a.plan.stop_layer[b] = ex ? a.exit_layer[b] : a.L;
    }
    __syncthreads();
    int n_cls = 0, n_str = 0;
    for (int b0 = 0; b0 < a.B; b0 += kPlanThreads) {
        const int b = b0 + tid;
        int first_c = 0, first_s = 0;
        if (b < a.B) {
            const int lab = s_lab[b], sid = s_sid[b];
            first_c = lab >= 0;
            first_s = 1;
            for (int j = b - 1; j >= 0 && (first_c | first_s); --j) {
                if (s_lab[j] == lab) first_c = 0;
                if (s_sid[j] == sid) first_s = 0;
            }
        }
        int cnt;
        int pos = block_exclusive_scan(first_c, s_scan, &cnt);
        if (first_c) a.plan.first_of_class[n_cls + pos] = b;
        n_cls += cnt;
        pos = block_exclusive_scan(first_s, s_scan, &cnt);
        if (first_s) a.plan.first_of_stream[n_str + pos] = b;
        n_str += cnt;
    }
    if (tid == 0) {
        a.plan.counts[0] = n_cls;
        a.plan.counts[1] = n_str;
    }
}

// ---- Eq. 5 / Eq. 6 ------------------------------------------------------------------------

__device__ __forceinline__ unsigned long long score_of(int ft, int ts, int W) {
    int e = ts / W;
    if (e > kEMax) e = kEMax;
    const unsigned long long f = (unsigned long long)min(max(ft, 0), kFtMax);
    return f << (2 * (kEMax - e));  // FT * 4^(12 - e) = 4^12 * FT * 0.25^e
}

constexpr size_t resize_smem(int n, int k_max) { return size_t(n) * 8 + size_t(n + (n & 1)) * 4 + size_t(k_max) * 8; }

// Refresh of one stream's fast memory by a CTA of kUpdThreads threads.  Classes with a
// non-zero score are compacted in ascending id and ranked among themselves by counting;
// zero-score classes follow in ascending id.  `smem` holds resize_smem(n, k_max) bytes.
__device__ void resize_stream(const ResizeArgs& a, int s, unsigned char* smem, int* s_scan,
                              unsigned long long* s_part) {
    unsigned long long* s_score = reinterpret_cast<unsigned long long*>(smem);  // [n] compacted non-zero scores
    int* s_id = reinterpret_cast<int*>(s_score + a.n);                          // [n] their class ids
    unsigned long long* s_top = reinterpret_cast<unsigned long long*>(s_id + a.n + (a.n & 1));  // [k_max]
    const int tid = threadIdx.x;
    const int32_t* ft = a.ft + (size_t)s * a.n;
    const int32_t* ts = a.ts + (size_t)s * a.n;
    int32_t* mem = a.members + (size_t)s * a.k_max;

    // pass 1: compact the non-zero scores (ascending id) and add everything up
    int nz = 0;
    unsigned long long local = 0;
    for (int c0 = 0; c0 < a.n; c0 += kUpdThreads) {
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
    __syncthreads();
    if ((tid & 31) == 0) s_part[tid >> 5] = local;
    __syncthreads();
    unsigned long long total = 0;
    for (int w = 0; w < kUpdThreads / 32; ++w) total += s_part[w];
    if (total == 0) return;  // nothing seen yet: keep size and members

    // pass 2: rank the non-zero classes; rank r < k_max goes to slot r
    for (int i = tid; i < nz; i += kUpdThreads) {
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
        for (int c0 = 0; c0 < a.n && filled < a.k_max; c0 += kUpdThreads) {
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

__global__ void __launch_bounds__(kUpdThreads) k_resize(const ResizeArgs a) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_scan[33];
    __shared__ unsigned long long s_part[kUpdThreads / 32];
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

// blockIdx.x <  table_ctas : tables (and, if asked, the refresh) of the stream of the
//                            blockIdx.x-th listed frame
// blockIdx.x >= table_ctas : centre of (class of the g-th listed frame, layer), g, layer =
//                            divmod(blockIdx.x - table_ctas, L)
__global__ void __launch_bounds__(kUpdThreads) k_update_apply(const UpdateArgs a, const ResizeArgs rz, int table_ctas,
                                                              int do_resize) {
    extern __shared__ unsigned long long s_dyn[];
    __shared__ int s_list[kUpdThreads];
    __shared__ int s_scan[33];
    __shared__ float s_red[32];
    __shared__ unsigned long long s_part[kUpdThreads / 32];
    const int tid = threadIdx.x;

    if (int(blockIdx.x) < table_ctas) {
        // ---- Sec. 6.1: the stream's frames, in ascending index, replayed per class ----------
        if (int(blockIdx.x) >= a.plan.counts[1]) return;
        const int bf = a.plan.first_of_stream[blockIdx.x];
        const int s = a.stream_id ? a.stream_id[bf] : 0;
        for (int t0 = bf - bf % kUpdThreads; t0 < a.B; t0 += kUpdThreads) {
            const int b = t0 + tid;
            const int hit = (b < a.B && (a.stream_id ? a.stream_id[b] : 0) == s) ? 1 : 0;
            const int cnt = compact_tile(hit, hit ? a.plan.final_label[b] : -1, s_list, s_scan);
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
        if (do_resize) {
            __syncthreads();  // this CTA's table writes are visible to all of its threads
            resize_stream(rz, s, reinterpret_cast<unsigned char*>(s_dyn), s_scan, s_part);
        }
        return;
    }

    // ---- Eq. 7 for one (class, layer): fold the matching frames in ascending index --------
    const int job = blockIdx.x - table_ctas;
    const int g = job / a.L, l0 = job - g * a.L;  // l0 is 0-based here; the paper's l0 is l0 + 1
    if (g >= a.plan.counts[0]) return;
    const int bf = a.plan.first_of_class[g];
    const int cls = a.plan.final_label[bf];
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
        for (int t0 = bf - bf % kUpdThreads; t0 < a.B; t0 += kUpdThreads) {
            const int b = t0 + tid;
            const int hit = (b < a.B && a.plan.final_label[b] == cls && a.plan.stop_layer[b] >= l0 + 1) ? 1 : 0;
            const int cnt = compact_tile(hit, b, s_list, s_scan);
            if (cnt == 0) continue;
            q += cnt;
            if (d >= D) continue;
            if (vec) {
                // eight rows in flight per thread; the additions stay in ascending frame order
                for (int i0 = 0; i0 < cnt; i0 += 8) {
                    float4 r[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        r[u] = i0 + u < cnt
                                   ? __ldg(reinterpret_cast<const float4*>(sv + (size_t)s_list[i0 + u] * D + d))
                                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (i0 + u < cnt) {
                            acc[0] += r[u].x; acc[1] += r[u].y; acc[2] += r[u].z; acc[3] += r[u].w;
                        }
                    }
                }
            } else {
                for (int i = 0; i < cnt; ++i)
                    for (int j = 0; j < 4; ++j)
                        if (d + j < D) acc[j] += sv[(size_t)s_list[i] * D + d + j];
            }
        }
        if (q == 0) return;  // no frame of this class stopped this deep: nothing changes
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

cudaError_t opt_in_smem(const void* fn, size_t smem, size_t* opted) {
    if (smem <= *opted) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    if (e == cudaSuccess) *opted = smem;
    return e;
}

}  // namespace

cudaError_t launch_center_norms(const float* centers, int n, int D, float* cnorm, cudaStream_t st,
                                int64_t* launches) {
    ++*launches;
    k_center_norms<<<n, 256, 0, st>>>(centers, n, D, cnorm);
    return cudaGetLastError();
}

cudaError_t launch_update(const UpdateArgs& a, const ResizeArgs* rz, cudaStream_t st, int64_t* launches) {
    if (a.B <= 0) return cudaSuccess;
    static size_t opted_plan = 48 * 1024, opted_apply = 48 * 1024;
    const size_t plan_smem = size_t(a.B) * 2 * sizeof(int);
    cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_update_plan), plan_smem, &opted_plan);
    if (e != cudaSuccess) return e;
    const size_t apply_smem = rz ? resize_smem(a.n, rz->k_max) : 0;
    e = opt_in_smem(reinterpret_cast<const void*>(k_update_apply), apply_smem, &opted_apply);
    if (e != cudaSuccess) return e;
    *launches += 2;
    k_update_plan<<<1, kPlanThreads, plan_smem, st>>>(a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int table_ctas = std::min(a.B, a.S);
    const int centre_ctas = std::min(a.B, a.n) * a.L;
    k_update_apply<<<table_ctas + centre_ctas, kUpdThreads, apply_smem, st>>>(a, rz ? *rz : ResizeArgs{}, table_ctas,
                                                                              rz ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_resize(const ResizeArgs& a, cudaStream_t st, int64_t* launches) {
    static size_t opted = 48 * 1024;
    const size_t smem = resize_smem(a.n, a.k_max);
    const cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_resize), smem, &opted);
    if (e != cudaSuccess) return e;
    ++*launches;
    k_resize<<<a.S, kUpdThreads, smem, st>>>(a);
    return cudaGetLastError();
}

}  // namespace smtm
