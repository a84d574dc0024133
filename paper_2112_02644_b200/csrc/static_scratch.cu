// smtm_lookup_exit_static: a single-layer lookup for callers that must not allocate.
//
// Some callers cannot call cudaMalloc (or anything that might): a plug-in that runs inside
// another engine's enqueue step and is handed only its inputs and outputs, a real-time
// thread that must not take the allocator's locks, code that runs after the process has
// pinned down its memory budget.  The regular lookup needs working memory per batch (the
// semantic vectors, the cumulative similarities, the exit layers), which such a caller has
// nowhere to put.  Here it lives in a fixed array compiled into the library image, so the
// call touches no allocator at all: not cudaMalloc / cudaFree, not torch, not the host heap.
#include <atomic>

#include "internal.h"

using namespace smtm;

// Working memory shared by every call on a device.  Each GPU that loads the library holds
// these bytes until the process exits.
__device__ __align__(256) static unsigned char g_static_scratch[SMTM_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch, per device; null until the first call on that device.  Published
// through an atomic so that the calls after the first one take no lock (two first calls that race both
// ask the runtime and store the same address).
std::atomic<unsigned char*> g_scratch_addr[kMaxDevices];

// In host code the name g_static_scratch is only a handle for the runtime, not an address a
// kernel can use; the device address is obtained, once per device and with that device
// current, from cudaGetSymbolAddress.
cudaError_t scratch_address(unsigned char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    unsigned char* p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!p) {
        e = cudaGetSymbolAddress((void**)&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return cudaSuccess;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

extern "C" smtm_status_t smtm_lookup_exit_static(smtm_cache_t* cache, int32_t layer, const smtm_fmap_t* fmap,
                                                 const int32_t* d_stream_id, uint8_t* d_exit, int32_t* d_pred,
                                                 float* d_ac, void* stream) {
    int L = 0, k_max = 0;
    if (!cache || !fmap || !d_exit || !d_pred) return SMTM_ERR_INVALID_ARG;
    cache_shape(cache, &L, &k_max);
    if (layer < 0 || layer >= L) return SMTM_ERR_INVALID_ARG;
    if (fmap->B < 1 || fmap->C < 1) return SMTM_ERR_SHAPE;
    // layout of the working memory: [B][C] semantic vectors | [B][k_max] similarities | [B] exit layers
    const size_t B = size_t(fmap->B);
    const size_t off_sa = round_up(B * size_t(fmap->C) * sizeof(float), 256);
    const size_t off_el = off_sa + round_up(B * size_t(k_max) * sizeof(float), 256);
    const size_t need = off_el + round_up(B * sizeof(int32_t), 256);
    if (need > SMTM_STATIC_SCRATCH_BYTES) return SMTM_ERR_SHAPE;  // batch too large for the fixed working memory

    unsigned char* base = nullptr;
    if (scratch_address(&base) != cudaSuccess) {
        (void)cudaGetLastError();
        return SMTM_ERR_CUDA;
    }
    smtm_batch_t b{};
    b.B = fmap->B;
    b.d_stream_id = d_stream_id;
    b.d_sa = reinterpret_cast<float*>(base + off_sa);
    b.d_done = d_exit;
    b.d_exit_layer = reinterpret_cast<int32_t*>(base + off_el);
    b.d_pred = d_pred;
    b.d_ac = d_ac;
    b.d_sv[layer] = reinterpret_cast<float*>(base);
    // The array keeps whatever the previous call left: the lookup starts the carry afresh.  It never starts
    // early (SMTM_FLAG_MAPS_READY is for carries that alternate; every call here shares the one array, which
    // the stream's previous kernel may be a static call still reading).
    return lookup_begin_ordered(cache, layer, fmap, &b, stream);
}
