// Prompt compression for callers that cannot allocate device memory: the pass's scratch
// lives in a fixed array that is part of the loaded library image.
#include "../../include/zsm.h"

#include <cuda_runtime.h>

#include "zsm_noalloc.cuh"

#include <mutex>

namespace {

// Scratch of zsm_prefill_compress_static.  Every GPU that loads the library holds these
// bytes until the process exits.  In host code this name is only a handle for the runtime's
// symbol lookup, never an address a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[ZSM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices];  // device address of the array on each device, once looked up

// Device address of the array on the current device; looked up once per device.  The first
// look-up on a device is also the first use of this file's module there: under lazy module
// loading that is when the device reserves the array's bytes, so it belongs to set-up time
// (zsm_cache_create calls it through zsm::static_scratch_setup), not to the no-allocation call.
zsm_status_t static_scratch(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZSM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ZSM_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return ZSM_OK;
}

}  // namespace

namespace zsm {
int static_scratch_setup() {
    void *p = nullptr;
    return static_scratch(&p) == ZSM_OK ? 0 : 1;
}
}  // namespace zsm

extern "C" zsm_status_t zsm_prefill_compress_static(zsm_cache_t *c, int32_t layer, const void *K,
                                                    const void *V, const void *Qw,
                                                    const float *scores, int32_t T, int32_t W,
                                                    float *dbg_scores, uint8_t *dbg_evicted,
                                                    int32_t *dbg_targets, zsm_stream_t stream) {
    size_t need = 0;
    const zsm_status_t st = zsm_prefill_workspace_bytes(c, T, Qw ? W : 0, &need);
    if (st != ZSM_OK) return st;
    if (need > static_cast<size_t>(ZSM_STATIC_SCRATCH_BYTES)) return ZSM_ERR_BUFFER_TOO_SMALL;
    void *scratch = nullptr;
    const zsm_status_t sa = static_scratch(&scratch);
    if (sa != ZSM_OK) return sa;
    return zsm_prefill_compress(c, layer, K, V, Qw, scores, T, W, scratch,
                                static_cast<size_t>(ZSM_STATIC_SCRATCH_BYTES), dbg_scores,
                                dbg_evicted, dbg_targets, stream);
}
