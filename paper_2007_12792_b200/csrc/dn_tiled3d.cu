// Tiled 3D kernel (placeholder: not yet applicable to any problem).
#include "dn_internal.cuh"
namespace dn {
bool tiled3d_applicable(const dn_problem&) { return false; }
Launch tiled3d_geometry(const dn_problem&) { return Launch{}; }
cudaError_t launch_tiled3d(const Params&, const Launch&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace dn
