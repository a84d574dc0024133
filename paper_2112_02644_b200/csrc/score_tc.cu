// Similarity scoring against a large fast memory (Sec. 4.2 Eq. 1's numerators for every class
// at once): DOT[b][c] = <SV_b, SC_c>, a dense B x D x n contraction on the tensor cores.
//
// Precision.  Exit decisions are compared in fp32, so bf16 operands alone (2^-9 relative) would
// not do.  Each fp32 operand is split into a bf16 head and a bf16 tail (x = hi + lo, |lo| <=
// 2^-9 |hi|) and the product is taken as hi*hi + hi*lo + lo*hi with fp32 accumulation in tensor
// memory; the dropped lo*lo term is 2^-18 relative.  One k-block therefore loads four tiles
// (A_hi, A_lo, B_hi, B_lo) and issues three groups of MMAs on them.  The tensor core truncates
// when it adds into its fp32 accumulator, an error that grows with the number of additions, so
// the long hi*hi sum is cut into three runs of k-blocks with an accumulator each and the two
// small cross terms share a fourth; the epilogue adds the four in fp32 with rounding.
//
// Kernel.  One CTA per 128 x 128 tile of DOT (frames x classes) and half of the vector length:
// with N = 128 an MMA reads as many bytes of shared memory per cycle as it can use (with N = 64
// the 128 x 16 slice of A was re-read for half the work and the instruction was operand-bound),
// and cutting the length in two keeps 128 CTAs busy on the 1024 x 1000 problem.  The two halves
// go to two result arrays that the finishing kernel adds in a fixed order.  Warp 0 is the TMA
// producer (cp.async.bulk.tensor, 128-byte swizzle, three stages of 64 KB), warp 1 allocates
// tensor memory (4 x 128 fp32 columns) and issues tcgen05.mma (M = 128, N = 128, K = 16,
// kind::f16 with bf16 inputs), warps 2..5 read the accumulators back with tcgen05.ld and store
// them.  Rows and classes beyond the problem are zero-filled by TMA and dropped by the
// epilogue.  Every mbarrier wait is bounded.
#include <cuda.h>

#include <algorithm>

#include "common.cuh"
#include "internal.h"

namespace smtm {

namespace {

constexpr int kTileM = 128;   // frames per tile = MMA M
constexpr int kTileN = 128;   // classes per tile = MMA N
constexpr int kTileK = 64;    // bf16 elements per k-block = one 128-byte swizzled row
constexpr int kMmaK = 16;     // K of one tcgen05.mma with 16-bit inputs
constexpr int kTcStages = 3;
constexpr int kBytesA = kTileM * kTileK * 2;                   // 16 KB
constexpr int kBytesB = kTileN * kTileK * 2;                   // 16 KB
constexpr int kStageBytes = 2 * kBytesA + 2 * kBytesB;         // hi and lo of both operands
constexpr int kTcThreads = 6 * kWarp;
constexpr int kHeadRuns = 3;                                   // accumulators the hi*hi sum is spread over
constexpr int kSplitK = 2;                                     // CTAs that share the vector length of a tile
constexpr int kAccs = kHeadRuns + 1;                           // ... plus one for the cross terms
constexpr int kTmemCols = 512;                                 // power of two >= kAccs * kTileN fp32 columns
constexpr size_t kTcSmem = size_t(kTcStages) * kStageBytes + 1024 + 256;

// ---- operand split ---------------------------------------------------------------------------

// x = hi + lo with hi = bf16(x) and lo = bf16(x - hi); rows of skipped frames are left alone.
__global__ void k_split_bf16(const float* __restrict__ src, const uint8_t* __restrict__ skip, int rows, int D,
                             __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
    chain_wait();
    chain_release();
    const long long total = (long long)rows * D;
    for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * 4; i < total;
         i += (long long)gridDim.x * blockDim.x * 4) {
        if (skip && skip[i / D]) continue;
        const float4 v = *reinterpret_cast<const float4*>(src + i);  // D is a multiple of 8
        const float x[4] = {v.x, v.y, v.z, v.w};
        __nv_bfloat16 h[4], l[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            h[j] = __float2bfloat16_rn(x[j]);
            l[j] = __float2bfloat16_rn(x[j] - __bfloat162float(h[j]));
        }
        *reinterpret_cast<uint2*>(hi + i) = *reinterpret_cast<const uint2*>(h);
        *reinterpret_cast<uint2*>(lo + i) = *reinterpret_cast<const uint2*>(l);
    }
}

// ---- tcgen05 / TMA wrappers --------------------------------------------------------------------

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory operand descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle, groups of
// eight rows 1024 bytes apart; the tile base is 1024-byte aligned.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= uint64_t((addr & 0x3ffff) >> 4);   // start address, 16-byte units
    d |= uint64_t(1024 >> 4) << 32;         // stride between 8-row groups
    d |= uint64_t(1) << 46;                 // descriptor version of this architecture
    d |= uint64_t(2) << 61;                 // 128-byte swizzle
    return d;
}

// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M x N as given.
__device__ __forceinline__ uint32_t idesc_bf16_f32(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(N >> 3) << 17) | (uint32_t(M >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

struct TcParams {
    int M, N, D;       // frames, classes, vector length
    int ld_out;        // floats between rows of `out`
    float* out;        // [splits][M][ld_out] dot products over each part of the vector length
    size_t split_stride;  // floats between the result arrays of two parts
    int* status;
    unsigned long long* clock;  // nullptr, or two words for the device-clock stamps
    int stages;                 // depth of the operand ring, 2 .. kTcStages
};

__global__ void __launch_bounds__(kTcThreads, 1)
k_score_tc(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
           const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
           const TcParams p) {
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
    const int stages = p.stages;
    uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(stages) * kStageBytes);  // [stages]
    uint64_t* empty = full + stages;                                                    // [stages]
    uint64_t* acc_full = empty + stages;                                                // [1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.y * kTileM, n0 = blockIdx.x * kTileN;
    // this CTA's share of the k-blocks
    const int n_kb_all = (p.D + kTileK - 1) / kTileK;
    const int kb0 = int(blockIdx.z) * n_kb_all / int(gridDim.z);
    const int n_kb = (int(blockIdx.z) + 1) * n_kb_all / int(gridDim.z) - kb0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(acc_full, 1);
        mbar_init_fence();
    }
    if (warp == 1) {  // the allocating warp also frees the columns at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;
    chain_wait();  // barriers and tensor memory are set up while the previous kernel finishes
    chain_release();
    const ClockScope stamps(p.clock);

    bool failed = false;
    int issued = 0;
    if (warp == 0) {
        // ---- producer: four tiles per k-block ---------------------------------------------------
        if (lane == 0) {
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % stages;
                const uint32_t use = uint32_t(kb / stages);
                if (use > 0 && !mbar_wait_bounded(&empty[s], (use - 1) & 1, p.status)) { failed = true; break; }
                uint8_t* st = base + size_t(s) * kStageBytes;
                mbar_expect_tx(&full[s], kStageBytes);
                const int x = (kb0 + kb) * kTileK;  // a multiple of 64 elements = 128 bytes
                tma_load_2d(st, &map_a_hi, x, m0, &full[s]);
                tma_load_2d(st + kBytesA, &map_a_lo, x, m0, &full[s]);
                tma_load_2d(st + 2 * kBytesA, &map_b_hi, x, n0, &full[s]);
                tma_load_2d(st + 2 * kBytesA + kBytesB, &map_b_lo, x, n0, &full[s]);
                issued = kb + 1;
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer -------------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16_f32(kTileM, kTileN);
            uint32_t started = 0;  // bit i: accumulator i holds something
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % stages;
                if (!mbar_wait_bounded(&full[s], (kb / stages) & 1, p.status)) { failed = true; break; }
                tc_fence_after();
                const uint32_t a_hi = smem_u32(base + size_t(s) * kStageBytes);
                const uint32_t a_lo = a_hi + kBytesA, b_hi = a_hi + 2 * kBytesA, b_lo = b_hi + kBytesB;
                const int run = kb * kHeadRuns / n_kb;  // consecutive k-blocks share an accumulator
                // lo*hi and hi*lo into the cross-term accumulator, hi*hi into its run's
                const uint32_t a_of[3] = {a_lo, a_hi, a_hi};
                const uint32_t b_of[3] = {b_hi, b_lo, b_hi};
                const int acc_of[3] = {kHeadRuns, kHeadRuns, run};
#pragma unroll
                for (int t = 0; t < 3; ++t) {
#pragma unroll
                    for (int ks = 0; ks < kTileK / kMmaK; ++ks) {
                        const uint64_t da = smem_desc_sw128(a_of[t] + ks * kMmaK * 2);
                        const uint64_t db = smem_desc_sw128(b_of[t] + ks * kMmaK * 2);
                        umma_bf16(tmem_acc + uint32_t(acc_of[t] * kTileN), da, db, idesc, (started >> acc_of[t]) & 1u);
                        started |= 1u << acc_of[t];
                    }
                }
                umma_commit(&empty[s]);  // the stage may be refilled once these MMAs have read it
            }
            if (!failed && started != (1u << kAccs) - 1u) failed = true;  // fewer k-blocks than runs: not launched
            umma_commit(acc_full);  // accumulator complete
        }
    } else {
        // ---- epilogue: warp w may touch the tensor-memory lanes 32 * (w % 4) .. + 31 --------------
        const int q = warp & 3;
        if (!mbar_wait_bounded(acc_full, 0, p.status)) {
            failed = true;
        } else {
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < kTileN; c0 += 16) {
                uint32_t r[kAccs][16];
#pragma unroll
                for (int acc = 0; acc < kAccs; ++acc) {
                    const uint32_t taddr = tmem_acc + (uint32_t(q * 32) << 16) + uint32_t(acc * kTileN + c0);
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                        : "=r"(r[acc][0]), "=r"(r[acc][1]), "=r"(r[acc][2]), "=r"(r[acc][3]), "=r"(r[acc][4]),
                          "=r"(r[acc][5]), "=r"(r[acc][6]), "=r"(r[acc][7]), "=r"(r[acc][8]), "=r"(r[acc][9]),
                          "=r"(r[acc][10]), "=r"(r[acc][11]), "=r"(r[acc][12]), "=r"(r[acc][13]), "=r"(r[acc][14]),
                          "=r"(r[acc][15])
                        : "r"(taddr)
                        : "memory");
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row < p.M) {
                    float* dst = p.out + size_t(blockIdx.z) * p.split_stride + (size_t)row * p.ld_out + n0 + c0;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        if (n0 + c0 + j < p.N) {  // N and ld_out are multiples of 4
                            float o[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float h = __uint_as_float(r[0][j + e]);
#pragma unroll
                                for (int run = 1; run < kHeadRuns; ++run) h += __uint_as_float(r[run][j + e]);
                                o[e] = h + __uint_as_float(r[kHeadRuns][j + e]);
                            }
                            *reinterpret_cast<float4*>(dst + j) = make_float4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    const int any_failed = __syncthreads_or(failed ? 1 : 0);
    if (any_failed && warp == 0 && lane == 0) {  // let every copy that was issued land before leaving
        for (int s = 0; s < stages && s < issued; ++s)
            mbar_wait_bounded(&full[s], uint32_t((issued - 1 - s) / stages) & 1, p.status);
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(kTmemCols) : "memory");
    }
}

// ---- host ---------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Map of a row-major bf16 matrix [rows][D] loaded in boxes of box_rows x 64 elements, 128-byte swizzle.
bool make_map(CUtensorMap* map, const __nv_bfloat16* ptr, int rows, int D, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cuuint64_t(D), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(D) * 2};
    const cuuint32_t box[2] = {cuuint32_t(kTileK), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t dense_setup() {
    const cudaError_t e = cudaFuncSetAttribute(k_score_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kTcSmem));
    // (with a short ring the kernel shares SMs with the pooling kernel of the pipelined route)
    return e != cudaSuccess ? e : prefer_max_smem_carveout(k_score_tc);
}

bool dense_scoring_supported(int D, int n) {
    return D % 8 == 0 && D >= 4 * kTileK && n % 4 == 0 && encode_tiled_fn() != nullptr;
}

size_t dense_scratch_bytes(int max_batch, int n, int d_max) {
    // bf16 heads and tails of the semantic vectors (two sets: the pipelined route pools a batch while the one
    // before it is still being scored), then the dot products
    return 2 * size_t(max_batch) * d_max * 2 * 2 + size_t(kSplitK) * max_batch * n * sizeof(float) + 1024;
}

size_t dense_centers_split_bytes(int n, int D) { return size_t(n) * D * 2 * 2; }

void dense_sv_split(void* scratch, int max_batch, int d_max, int which, void** hi, void** lo) {
    __nv_bfloat16* a_hi = reinterpret_cast<__nv_bfloat16*>(scratch) + size_t(which & 1) * 2 * size_t(max_batch) * d_max;
    *hi = a_hi;
    *lo = a_hi + size_t(max_batch) * d_max;
}

cudaError_t launch_centers_split(const float* centers, int n, int D, void* centers_split, cudaStream_t st,
                                 int64_t* launches) {
    __nv_bfloat16* b_hi = reinterpret_cast<__nv_bfloat16*>(centers_split);
    ++*launches;
    const int grid = int(std::min<long long>(((long long)n * D / 4 + 255) / 256, 148 * 8));
    return launch_chained(k_split_bf16, grid, 256, 0, st, centers, static_cast<const uint8_t*>(nullptr), n, D, b_hi,
                          b_hi + size_t(n) * D);
}

cudaError_t launch_dense_dots(const float* sv, const uint8_t* skip, int B, const float* centers, int n, int D,
                              void* scratch, int max_batch, int d_max, int which, bool sv_split_done,
                              cudaEvent_t sv_ready, void* centers_split, float** dots_out, float** dots2_out,
                              int* status, unsigned long long* clock, int ring_stages, cudaStream_t st,
                              int64_t* launches) {
    void *hi = nullptr, *lo = nullptr;
    dense_sv_split(scratch, max_batch, d_max, which, &hi, &lo);
    __nv_bfloat16* a_hi = static_cast<__nv_bfloat16*>(hi);
    __nv_bfloat16* a_lo = static_cast<__nv_bfloat16*>(lo);
    __nv_bfloat16* b_hi = reinterpret_cast<__nv_bfloat16*>(centers_split);
    __nv_bfloat16* b_lo = b_hi + size_t(n) * D;
    float* dots = reinterpret_cast<float*>(
        (reinterpret_cast<uintptr_t>(reinterpret_cast<__nv_bfloat16*>(scratch) + 4 * size_t(max_batch) * d_max) + 255) &
        ~uintptr_t(255));
    // the vector length is cut in two when each part still has a k-block for every accumulator
    const int splits = (D + kTileK - 1) / kTileK >= kSplitK * kHeadRuns ? kSplitK : 1;
    *dots_out = dots;
    *dots2_out = splits > 1 ? dots + size_t(max_batch) * n : nullptr;

    CUtensorMap ma_hi, ma_lo, mb_hi, mb_lo;
    if (!make_map(&ma_hi, a_hi, B, D, kTileM) || !make_map(&ma_lo, a_lo, B, D, kTileM) ||
        !make_map(&mb_hi, b_hi, n, D, kTileN) || !make_map(&mb_lo, b_lo, n, D, kTileN))
        return cudaErrorInvalidValue;
    if (sv_ready) {
        const cudaError_t e = cudaStreamWaitEvent(st, sv_ready, 0);
        if (e != cudaSuccess) return e;
    }
    if (!sv_split_done) {
        ++*launches;
        const int grid_a = int(std::min<long long>(((long long)B * D / 4 + 255) / 256, 148 * 8));
        const cudaError_t e = launch_chained(k_split_bf16, grid_a, 256, 0, st, sv, skip, B, D, a_hi, a_lo);
        if (e != cudaSuccess) return e;
    }
    ++*launches;
    TcParams p{};
    p.M = B;
    p.N = n;
    p.D = D;
    p.ld_out = n;
    p.out = dots;
    p.split_stride = size_t(max_batch) * n;
    p.status = status;
    p.clock = clock;
    p.stages = ring_stages >= 2 && ring_stages <= kTcStages ? ring_stages : kTcStages;
    const dim3 grid((n + kTileN - 1) / kTileN, (B + kTileM - 1) / kTileM, splits);
    const size_t smem = size_t(p.stages) * kStageBytes + 1024 + 256;
    return launch_chained(k_score_tc, grid, kTcThreads, smem, st, ma_hi, ma_lo, mb_hi, mb_lo, p);
}

}  // namespace smtm
