// Tensor-core (tcgen05 / TMEM / TMA) path.  Placeholder until the kernels land: reports "not supported".
#include "laser_common.cuh"
namespace laser {
bool tensor_supported(const Plan&) { return false; }
void tensor_geometry(const Plan&, TensorGeom* g) { g->IT = 16; g->NT = 1; g->n_tiles = 0; g->cand_tiles_max = 0; }
int tensor_sta(const Plan&, const void*, const int32_t*, const void*, const int32_t*, const void*, const void*,
               const void*, void*, char*, cudaStream_t) { return LASER_ERR_UNSUPPORTED; }
int tensor_gsta(const Plan&, const void*, const int32_t*, const int32_t*, const void*, const void*, void*, char*,
                cudaStream_t) { return LASER_ERR_UNSUPPORTED; }
}  // namespace laser
