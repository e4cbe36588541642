// dn_energy_grad_static: the fused energy+residual call for callers that cannot allocate
// device memory.  Its scratch (energy partials and KL tables) lives in a fixed array that is
// part of the library image, so no workspace is passed in and nothing is allocated.
#include "dn_internal.cuh"

namespace {

// Scratch shared by every dn_energy_grad_static call on a device.  Each GPU that loads the
// library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[DN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// the address a kernel can use has to be asked for, once per device, with that device current.
dn_status scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DN_ERR_CUDA;
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DN_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return DN_OK;
}

}  // namespace

extern "C" dn_status dn_energy_grad_static(const dn_problem* problem, const float* u, const float* gJ, float* J,
                                           float* r, void* stream) {
    void* scratch = nullptr;
    const dn_status st = scratch_address(&scratch);
    if (st != DN_OK) return st;
    // A problem whose scratch does not fit is refused with DN_ERR_WORKSPACE before anything is enqueued.
    return dn::run_tight(problem, u, gJ, J, r, scratch, DN_STATIC_SCRATCH_BYTES, stream);
}
