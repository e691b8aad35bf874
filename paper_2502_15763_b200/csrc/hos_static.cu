// hos_lower_bound_static: the lower-bound call for callers that cannot allocate device memory.
//
// The scratch that hos_lower_bound takes from its caller (sorted estimates, order, per-instance
// facts) lives here in a fixed array inside the library's device image.  Host code must not
// hand the array's name to a kernel: on the host that name is only a stand-in for the symbol.
// The device address comes from cudaGetSymbolAddress, looked up once per device with that
// device current, and that pointer is what the kernels receive.
#include <cuda_runtime.h>

#include <mutex>

#include "hos.h"

namespace {

// Held by every GPU that loads the library, from module load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HOS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device, or nullptr with *rc set.
void* scratch_on_current_device(int* rc) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        *rc = HOS_E_CUDA;
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            *rc = HOS_E_CUDA;
            return nullptr;
        }
        g_scratch_ptr[dev] = ptr;
    }
    *rc = HOS_OK;
    return g_scratch_ptr[dev];
}

}  // namespace

extern "C" int hos_lower_bound_static(const hos_batch* batch, const hos_cost_model* cm, hos_lb* out,
                                      int32_t* status, void* stream) {
    if (!batch || batch->n_inst < 1 || batch->n_req < 1) return HOS_E_INVALID;
    const size_t need = hos_lower_bound_workspace_bytes(batch);
    if (need == 0) return HOS_E_INVALID;
    if (need > (size_t)HOS_STATIC_SCRATCH_BYTES) return HOS_E_TOO_LARGE;
    int rc = HOS_OK;
    void* ptr = scratch_on_current_device(&rc);
    if (!ptr) return rc;
    // Nothing in the scratch has to start at zero: every word the kernels read is written
    // earlier in the same call, so the previous call's contents are simply overwritten.
    return hos_lower_bound(batch, cm, out, status, ptr, (size_t)HOS_STATIC_SCRATCH_BYTES, stream);
}
