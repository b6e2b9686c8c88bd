// One-candidate-per-user HBM-streaming path.  Placeholder until the kernel lands: reports "not supported".
#include "laser_common.cuh"
namespace laser {
bool stream_supported(const Plan&) { return false; }
int stream_forward(const Plan&, const void*, const int32_t*, const void*, const int32_t*, const void*, const void*,
                   const void*, const void*, void*, void*, char*, cudaStream_t) { return LASER_ERR_UNSUPPORTED; }
}  // namespace laser
