// cadd_build_tree_static_scratch: tree construction for callers that have no way to hand the library
// a scratch buffer.  The scratch lives in a fixed-size array inside the library image.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "cadd.h"

namespace {

// The scratch itself: part of the module, so every device that loads the library carries these
// bytes from the first use until the process exits.  In host code this name is only a handle for
// the runtime (it is not a device address); the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[CADD_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_lock;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device; looked up on the first call per device.
int static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return CADD_ERR_LAUNCH;
    }
    std::lock_guard<std::mutex> guard(g_lock);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return CADD_ERR_LAUNCH;
        }
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return CADD_OK;
}

}  // namespace

extern "C" int cadd_build_tree_static_scratch(const cadd_build_args* a, void* cuda_stream) {
    size_t need = 0;
    int rc = cadd_build_workspace_bytes(a, &need);          // also validates struct size and shapes
    if (rc != CADD_OK) return rc;
    if (need > (size_t)CADD_STATIC_SCRATCH_BYTES) return CADD_ERR_STATIC_SCRATCH;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != CADD_OK) return rc;
    cadd_build_args with_scratch = *a;                       // the caller's struct is left untouched
    with_scratch.workspace = scratch;
    with_scratch.workspace_bytes = (size_t)CADD_STATIC_SCRATCH_BYTES;
    return cadd_build_tree(&with_scratch, cuda_stream);
}
