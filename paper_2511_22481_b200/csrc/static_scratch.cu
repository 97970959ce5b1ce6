// omni_sparse_mla_decode_static: the decode call for callers that cannot hand the library a
// workspace.  The split-KV partial results live in a fixed array that is part of the library
// image, so the call needs no allocation by anyone.
#include <cuda_runtime.h>

#include <mutex>

#include "omni_mla.h"

namespace {

// Split-KV scratch (fp32 partial outputs + partial log-sum-exps).  Every GPU that loads the
// library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[OMNI_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mu;

// Device address of the scratch array on the current device.  In host code the array's name
// is only a handle for the runtime, not an address a kernel could use, so the address is
// looked up once per device (with that device current) and cached.
cudaError_t scratch_address(void **ptr)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void *p = nullptr;
        err = cudaGetSymbolAddress(&p, g_static_scratch);
        if (err != cudaSuccess) return err;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = p;
    }
    *ptr = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" omni_status_t omni_sparse_mla_decode_static(const omni_mla_desc_t *desc, const void *q,
                                                       const void *kv_cache, const int32_t *page_table,
                                                       const int32_t *sel_idx, const int32_t *sel_len,
                                                       void *out, float *lse, int32_t *device_status,
                                                       void *stream)
{
    if (!desc) return OMNI_ERR_NULL;
    const size_t need = omni_sparse_mla_workspace_bytes(desc);
    if (need == 0) return OMNI_ERR_SHAPE;
    if (need > (size_t)OMNI_STATIC_SCRATCH_BYTES) return OMNI_ERR_WORKSPACE;
    void *scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return OMNI_ERR_CUDA;
    // The caller has nothing to clear: the decode kernel writes the partial result of every
    // (request, split, head) it later merges, empty splits included, and the arrival counters
    // of the fused merge (OMNI_FLAG_FUSED_MERGE), the only words that must start at zero, are
    // cleared on the stream by omni_sparse_mla_decode itself.
    return omni_sparse_mla_decode(desc, q, kv_cache, page_table, sel_idx, sel_len, out, lse, scratch,
                                  (size_t)OMNI_STATIC_SCRATCH_BYTES, device_status, stream);
}
