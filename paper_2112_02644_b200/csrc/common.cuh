// Device-side building blocks shared by the SMTM kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace smtm {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// Error codes written to the sticky device status word (same values as smtm_status_t).
constexpr int kDevInvalidArg = 1;
constexpr int kDevTimeout = 8;

__device__ __forceinline__ void set_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

// ---- chained launches -----------------------------------------------------------------
//
// Every kernel of the library is launched with programmatic stream serialisation: its CTAs may
// become resident, and run their prologue, while the kernel before it in the stream is still
// running.  chain_wait() returns once the previous kernel has completed and its writes are
// visible; nothing that reads or writes global memory comes before it.  chain_release() lets
// the next kernel's CTAs in as soon as all of this kernel's have called it.  Kernels call it
// right after chain_wait(): a kernel then only ever shares the device with its direct
// neighbours (released before the wait, a chain of small kernels would let a much later
// kernel in, whose CTAs take registers and shared memory away from the ones still running).

__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- profiling by the device's clock ------------------------------------------------------------

__device__ __forceinline__ unsigned long long device_clock_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Notes when the first CTA of a kernel began and the last one ended.  slot: two words that are
// zero before the kernel runs; [0] ends up as the complement of the earliest begin, [1] as the
// latest end (two maxima: one memset prepares both).  Thread 0 of every CTA stamps, so the
// object has to live in a scope that thread 0 leaves last (or see every_warp).  slot == nullptr:
// nothing happens.
struct ClockScope {
    unsigned long long* slot;
    // every_warp: lane 0 of every warp stamps (kernels whose warps work on their own and leave at different times)
    __device__ __forceinline__ explicit ClockScope(unsigned long long* s, bool every_warp = false)
        : slot((every_warp ? (threadIdx.x & 31) == 0 : threadIdx.x == 0) ? s : nullptr) {
        if (slot) atomicMax(slot, ~device_clock_ns());
    }
    __device__ __forceinline__ ~ClockScope() {
        if (slot) atomicMax(slot + 1, device_clock_ns());
    }
};

// ---- shared-memory barriers and bulk asynchronous copies -------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the asynchronous copy engine.
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Waits for the phase with the given parity to complete, for at most ~2^31 clock
// cycles (about a second).  Returns false on giving up, after recording a timeout.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > (1ll << 31)) {
            set_status(status, kDevTimeout);
            return false;
        }
    }
}

// 1-D bulk copy global -> shared, completion counted in bytes on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// The same with an L2 eviction hint: a stream that is read once should not push the data other kernels keep
// coming back to (centres, tables, semantic vectors) out of L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void bulk_load_hint(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// 16 bytes of a feature map by a plain load: read once, so marked for early eviction from L2 (the data the
// kernels keep coming back to should stay there).
__device__ __forceinline__ uint4 load_once(const uint4* p) { return __ldcs(p); }

// ---- element widening -----------------------------------------------------------------

struct F32 {
    static constexpr int kSize = 4;
    static constexpr int kPerVec = 4;  // elements in a 16-byte vector
    static __device__ __forceinline__ float at(const uint4& v, int j) {
        const uint32_t w = j == 0 ? v.x : j == 1 ? v.y : j == 2 ? v.z : v.w;
        return __uint_as_float(w);
    }
    static __device__ __forceinline__ float scalar(const void* p, size_t i) {
        return reinterpret_cast<const float*>(p)[i];
    }
};

struct BF16 {
    static constexpr int kSize = 2;
    static constexpr int kPerVec = 8;
    // bfloat16 is the upper half of a binary32: widen by placing it there.
    static __device__ __forceinline__ float at(const uint4& v, int j) {
        const int wi = j >> 1;
        const uint32_t w = wi == 0 ? v.x : wi == 1 ? v.y : wi == 2 ? v.z : v.w;
        return __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    static __device__ __forceinline__ float scalar(const void* p, size_t i) {
        return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(p)[i]) << 16);
    }
};

struct F16 {
    static constexpr int kSize = 2;
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ float at(const uint4& v, int j) {
        const int wi = j >> 1;
        const uint32_t w = wi == 0 ? v.x : wi == 1 ? v.y : wi == 2 ? v.z : v.w;
        const __half2 h = *reinterpret_cast<const __half2*>(&w);
        return (j & 1) ? __high2float(h) : __low2float(h);
    }
    static __device__ __forceinline__ float scalar(const void* p, size_t i) {
        return __half2float(reinterpret_cast<const __half*>(p)[i]);
    }
};

// ---- block-level helpers (fixed evaluation order: results do not depend on timing) -----

// Sum over the block; every thread gets the total.  `scratch` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += scratch[w];
    return t;
}

// Exclusive prefix sum of `v` over the block in thread order; *total receives the block sum.
// `scratch` holds >= 33 ints.
__device__ __forceinline__ int block_exclusive_scan(int v, int* scratch, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    int base = 0, sum = 0;
    for (int w = 0; w < nw; ++w) {
        if (w < warp) base += scratch[w];
        sum += scratch[w];
    }
    *total = sum;
    return base + inc - v;
}

}  // namespace smtm
