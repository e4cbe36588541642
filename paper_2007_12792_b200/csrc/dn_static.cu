// dn_energy_grad_static: the fused energy+residual call for callers that cannot allocate
// device memory.  Its scratch (energy partials and KL tables) lives in a fixed array that is
// part of the library image, so no workspace is passed in and nothing is allocated.
#include <atomic>

#include "dn_internal.cuh"

namespace {

// Scratch shared by every dn_energy_grad_static call on a device.  Each GPU that loads the
// library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[DN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch, per device ordinal.  The only state the library keeps: written once per
// device (two threads racing on the first call store the same value), never freed.
std::atomic<void*> g_scratch_ptr[kMaxDevices];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// the address a kernel can use has to be asked for, once per device, with that device current.
dn_status scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DN_ERR_CUDA;
    void* ptr = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DN_ERR_CUDA;
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return DN_OK;
}

}  // namespace

extern "C" dn_status dn_energy_grad_static(const dn_problem* problem, const float* u, const float* gJ, float* J,
                                           float* r, void* stream) {
    // A bad argument, or a problem whose scratch does not fit (DN_ERR_WORKSPACE), is refused on the host before
    // the device is touched.
    dn_status st = dn::check_tight(problem, u, r, DN_STATIC_SCRATCH_BYTES);
    if (st != DN_OK) return st;
    void* scratch = nullptr;
    st = scratch_address(&scratch);
    if (st != DN_OK) return st;
    return dn::run_tight(problem, u, gJ, J, r, scratch, DN_STATIC_SCRATCH_BYTES, stream);
}
