// dsla_prefill_static_ws: prefill for callers that cannot supply (or allocate) a scratch buffer.
// The scratch lives in a fixed device array that is part of the library image, so the call path
// contains no allocation at all.
#include <atomic>

#include "dsla_internal.cuh"

namespace {

// One copy per GPU that loads the library, resident until the process exits.  In HOST code this name
// is only a handle for the runtime, not a device address: the address kernels may use is obtained
// once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[DSLA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// device address of the array on each device, filled on first use; two host threads that race on the first call both
// look the address up and store the same value
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Device address of the scratch array on the current device (looked up once per device).
dsla_status static_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DSLA_ERR_CUDA;
    void* ptr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return DSLA_ERR_CUDA;
        }
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return DSLA_OK;
}

}  // namespace

extern "C" dsla_status dsla_prefill_static_ws(const dsla_prefill_args* a, dsla_state* st, void* cuda_stream) {
    if (!a) return DSLA_ERR_INVALID_ARG;
    dsla_prefill_args b = *a;
    b.workspace = nullptr;
    b.workspace_bytes = 0;
    const size_t need = dsla_prefill_workspace_bytes(&b);   // 0 for invalid sizes; those are rejected below
    if (need > (size_t)DSLA_STATIC_SCRATCH_BYTES) return DSLA_ERR_SCRATCH_LIMIT;
    if (need > 0) {
        void* ptr = nullptr;
        const dsla_status rc = static_scratch(&ptr);
        if (rc != DSLA_OK) return rc;
        b.workspace = ptr;
        b.workspace_bytes = DSLA_STATIC_SCRATCH_BYTES;
    }
    // Same checks, same kernels as dsla_prefill.  Every summary entry the main kernel reads is
    // written earlier in this same call, so stale contents from a previous call are never used.
    return dsla::prefill_checked(&b, st, static_cast<cudaStream_t>(cuda_stream));
}
