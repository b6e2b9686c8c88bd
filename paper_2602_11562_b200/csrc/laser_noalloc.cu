// laser_sta_forward_static: STA for callers that cannot provide (or obtain) a device workspace.
//
// Some callers of this library have no way to allocate device memory: a plug-in running inside a serving
// process whose GPU memory is owned, down to the last byte, by the host framework's pool; a request thread
// with a hard latency bound, where cudaMalloc's implicit device-wide synchronisation is not acceptable; a
// client that was handed a fixed set of input and output buffers and nothing else.  For them the scratch
// that the FP32-ALU STA kernels need (fp32 Q, K, V and the status word) lives in a fixed array that is part
// of the library image itself: every GPU that loads the library holds kStaticScratchBytes of it until the
// process exits.
#include <mutex>

#include "laser_common.cuh"

namespace laser {
namespace {

constexpr size_t kStaticScratchBytes = LASER_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a host-side stand-in for the symbol, NOT a device
// address: host code must go through cudaGetSymbolAddress (below) and hand the result to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
char* g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch on each device, once resolved

// Resolves, once per device and with that device current, where g_static_scratch lives on the current device.
int static_scratch_for_current_device(char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LASER_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return LASER_ERR_CUDA;
    g_scratch_ptr[dev] = static_cast<char*>(ptr);
  }
  *out = g_scratch_ptr[dev];
  return LASER_OK;
}

}  // namespace
}  // namespace laser

using namespace laser;

extern "C" int laser_sta_forward_static(const laser_config* cfg, const void* items, const int32_t* lengths,
                                        const void* cands, const int32_t* cand_offsets, const void* Wq,
                                        const void* Wk, const void* Wv, void* Hprime, int32_t* status_out,
                                        void* cuda_stream) {
  reset_launch_count();
  if (!cfg) return LASER_ERR_INVALID_ARG;
  laser_config c = *cfg;
  c.path = LASER_PATH_SIMT;     // the kernels whose scratch the static array replaces
  Plan p;
  int rc = make_plan(&c, &p);
  if (rc != LASER_OK) return rc;
  // Re-carve the scratch without the internal H' region (the caller supplies H'): status, Q, K, V.
  size_t off = 0;
  p.off_status = off; off = align_up(off + kStatusWords * sizeof(int));
  p.off_hp = 0;
  p.off_q = off; off = align_up(off + (size_t)p.N * p.dqk * sizeof(float));
  p.off_k = off; off = align_up(off + (size_t)p.U * p.L * p.dqk * sizeof(float));
  p.off_v = off; off = align_up(off + (size_t)p.U * p.L * p.d * sizeof(float));
  p.total = off;
  if (p.total > kStaticScratchBytes) return LASER_ERR_WORKSPACE;   // problem too large for the built-in scratch
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0) {
    const void* ptrs[] = {items, cands, Wq, Wk, Wv, Hprime};
    for (const void* q : ptrs)
      if (!q || (reinterpret_cast<uintptr_t>(q) & 15u)) return LASER_ERR_INVALID_ARG;
  }
  char* scratch = nullptr;
  if ((rc = static_scratch_for_current_device(&scratch)) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // The array keeps whatever the previous call left in it.  Only the status word must start at zero: Q, K and
  // V are fully rewritten for every row that is read afterwards.
  LASER_CUDA_OK(cudaMemsetAsync(scratch + p.off_status, 0, kStatusWords * sizeof(int), st));
  if (p.N > 0) {
    rc = simt_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, scratch, st);
    if (rc != LASER_OK) return rc;
  }
  if (status_out)
    LASER_CUDA_OK(cudaMemcpyAsync(status_out, scratch + p.off_status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return LASER_OK;
}
