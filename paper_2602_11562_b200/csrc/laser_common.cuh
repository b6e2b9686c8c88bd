// Shared host-side plan (validated configuration + workspace carve-up) and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "laser.h"

namespace laser {

constexpr int kStatusWords = 64;          // int32 words reserved at the start of every workspace
constexpr size_t kAlign = 256;
constexpr size_t kGuardBytes = 256;       // left unused after every workspace region (overruns show up there)
constexpr int kMaxRegions = 24;

// Tile geometry of the tensor-core path (defined by laser_tensor.cu, used by the plan for sizing).
struct TensorGeom {
  int IT;        // items per tile (multiple of 16, <= 128)
  int NT;        // tiles per segment
  int n_tiles;   // tiles per user = L' * NT
  int cand_tiles_max;  // upper bound on 128-candidate tiles over all users
};

struct Plan {
  int U, L, d, dqk, H, S, M, dtype, N, maxC, path;
  int Lp, dqh, dvh;
  float inv_gamma, inv_tau;
  size_t esize;
  const int32_t* item_offsets;     // packed item layout: first row of every user ([U + 1]); null = padded [U, L, d]
  // workspace byte offsets
  size_t off_status;
  size_t off_q, off_k, off_v;      // SIMT: fp32 Q [N,dqk], K [U,L,dqk], V [U,L,d]
  size_t off_hp;                   // internal H' [N,Lp,d] in the I/O dtype
  // tensor path
  TensorGeom tg;
  size_t off_tq, off_tk, off_tv, off_twork, off_tcount, off_tctile, off_timg;
  size_t off_gimg;                 // GSTA weight images in MMA fragment order (bf16 paths)
  // stream path
  size_t off_su;
  size_t total;
  // every region of the carve-up (byte offset, bytes in use), in order: what a call may write inside the workspace
  int n_regions;
  size_t reg_off[kMaxRegions], reg_size[kMaxRegions];
};

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Validates cfg and fills the plan. Returns LASER_OK or a negative status.
int make_plan(const laser_config* cfg, Plan* p);

// Launch accounting (thread-local).  Every kernel launch sits inside a LaunchScope: it counts the launch and, when
// profiling is enabled through laser_profile_enable, brackets it with CUDA events on the launching stream.
void reset_launch_count();
class LaunchScope {
 public:
  LaunchScope(const char* name, cudaStream_t st);
  ~LaunchScope();
 private:
  cudaStream_t st_;
  int slot_;
};

// --- per-path launchers (each returns LASER_OK / LASER_ERR_*) -------------------------------------------------------
int simt_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
             const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st);
// Softmax-aggregation variant of STA (the paper's ablation of the sigmoid gate); FP32-ALU kernels, same scratch as simt_sta.
int simt_sta_softmax(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                     const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws,
                     cudaStream_t st);
int simt_gsta(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets, const void* cands,
              const void* Wg, void* z, char* ws, cudaStream_t st);
// Eq. 8-9 on the FP32 ALUs: leaves fp32 Q / gamma, K, V at off_q, off_k, off_v.
int simt_project(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const void* Wq,
                 const void* Wk, const void* Wv, char* ws, cudaStream_t st);
// STA on the FP32 ALUs with an fp32 H' whatever the I/O dtype; leaves fp32 Q / gamma, K, V at off_q, off_k, off_v.
int simt_sta_f32(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
                 const void* Wq, const void* Wk, const void* Wv, float* Hprime32, char* ws, cudaStream_t st);

// Backward pass (laser_backward.cu): p is a plan of the FP32-ALU path; the workspace holds p.total bytes of the forward
// plan followed by backward_scratch_bytes(p).  Gradients are fp32.  tensor: bf16 batches take the tensor-core kernels
// where backward_tensor_supported(p) says they exist.
size_t backward_scratch_bytes(const Plan& p);
bool backward_tensor_supported(const Plan& p);
int backward(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
             const void* Wq, const void* Wk, const void* Wv, const void* Wg, const float* dz, float* d_items,
             float* d_cands, float* dWq, float* dWk, float* dWv, float* dWg, char* ws, cudaStream_t st, bool tensor);
// Tensor-core kernels of the backward pass (laser_backward_mma.cu), all on bf16 copies kept in `scratch`
// (sta_bwd_mma_scratch_bytes): sta_mma_operands makes the copies of Qf (Q / gamma), Kf and Vf; sta_fwd_mma recomputes H'
// in fp32 from them (rows of empty segments are left as they are); sta_bwd_mma copies dHp (null: the bf16 copy is there
// already), writes the dK / dV rows of valid items (the rest must hold zeros) and adds to dQf.
bool sta_bwd_mma_supported(const Plan& p);
bool sta_fwd_mma_supported(const Plan& p);
size_t sta_bwd_mma_scratch_bytes(const Plan& p);
int sta_mma_operands(const Plan& p, const float* Qf, const float* Kf, const float* Vf, char* scratch, cudaStream_t st);
// The bf16 K [U L, d_qk] and V [U L, d] arrays inside `scratch`, for a producer that writes them directly (it then passes
// Kf = Vf = null to sta_mma_operands).
void sta_mma_operand_arrays(const Plan& p, char* scratch, __nv_bfloat16** Kb, __nv_bfloat16** Vb);
int sta_fwd_mma(const Plan& p, const int32_t* lengths, const int32_t* cand_offsets, float* Hp, bool bf16_copy, char* scratch,
                cudaStream_t st);
// The attention of a recomputed GSTA layer on the bf16 copy of H' that sta_fwd_mma keeps (bf16_copy): writes the weights
// Aw [N, H, Lp] and the weighted sums Mh [N, H, d] (fp32) from Qt [N, H, d].
bool gsta_attn_mma_supported(const Plan& p);
int gsta_attn_fwd_mma(const Plan& p, const float* Qt, const int32_t* lengths, const int32_t* cand_offsets, float* Aw,
                      float* Mh, char* scratch, cudaStream_t st);
// Its backward: dQt [N, H, d] from Qt, Aw and dM [N, H, d]; dHp [N, Lp, d] written (overwrite) or added to; for the
// layer processed last the sum leaves as the bf16 array sta_bwd_mma reads (which then takes dHp = null) and dHp stays
// as it was.
int gsta_attn_bwd_mma(const Plan& p, const float* Qt, const float* Aw, const float* dM, const int32_t* lengths,
                      const int32_t* cand_offsets, float* dQt, float* dHp, bool overwrite, bool last, char* scratch,
                      cudaStream_t st);
int sta_bwd_mma(const Plan& p, const float* dHp, const int32_t* lengths, const int32_t* cand_offsets, float* dQf,
                float* dK, float* dV, char* scratch, cudaStream_t st);

bool tensor_supported(const Plan& p);
void tensor_geometry(const Plan& p, TensorGeom* g);
// Wg_images: when non-null (and the fused GSTA kernel will follow), the set-up kernel also builds the GSTA weight images.
// softmax: the softmax-aggregation variant (the paper's ablation of the sigmoid gate); needs tensor_softmax_supported(p).
bool tensor_softmax_supported(const Plan& p);
int tensor_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
               const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st,
               const void* Wg_images, bool softmax = false);
// Launches the bounded-wait self-test block (laser_tensor.cu); the status word is the first word of ws.
int tensor_wait_selftest(char* ws, int poll_limit, cudaStream_t st);
int tensor_gsta(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets,
                const void* cands, const void* Wg, void* z, char* ws, cudaStream_t st, bool images_ready);

// Fused warp-MMA GSTA kernel for bf16 (laser_gsta.cu); needs gsta_mma_image_bytes(p) of scratch at off_gimg.
bool gsta_mma_supported(const Plan& p);
size_t gsta_mma_image_bytes(const Plan& p);   // weight images, then the per-candidate segment counts
size_t gsta_nseg_offset(const Plan& p);       // byte offset of the segment counts inside that scratch
size_t gsta_order_offset(const Plan& p);      // byte offset of the block launch order (n ints) and its sort keys (n ints), n = ceil(N / 8)
int gsta_candidates_per_block(const Plan& p);
bool gsta_wants_order(const Plan& p);         // the kernel runs its blocks longest first (a set-up kernel must build the order)
// images_ready: the weight images at off_gimg were already built for these weights earlier on the same stream.
int gsta_mma(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets, const void* cands,
             const void* Wg, void* z, char* ws, cudaStream_t st, bool images_ready);

// One-candidate-per-user STA (laser_stream.cu); needs stream_scratch_bytes(p) of scratch at off_su.  Its GSTA is gsta_mma.
bool stream_supported(const Plan& p);
size_t stream_scratch_bytes(const Plan& p);
int stream_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
               const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st,
               const void* Wg_images);

// Multi-resolution feature fusion (laser_fusion.cu); uses only the status word of the workspace.
int fusion_forward(const Plan& p, const void* Hprime, const void* z, const int32_t* lengths, const int32_t* cand_offsets,
                   int num_recent, void* fused, char* ws, cudaStream_t st);

// Feed-forward refinement of H' (laser_ffn.cu); needs ffn_scratch_bytes(p, d_hidden) of scratch of its own.
bool ffn_supported(const Plan& p, int hid);
size_t ffn_scratch_bytes(const Plan& p, int hid);
int ffn_forward(const Plan& p, const laser_ffn_params* f, void* H, const int32_t* lengths, const int32_t* cand_offsets,
                char* ws, char* scratch, cudaStream_t st);

// --- device helpers ---------------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void report_status(int* status, int code) { atomicCAS(status, 0, code); }

// Programmatic dependent launch.  Kernels launched with launch_chained may start (block scheduling, shared-memory and
// barrier set-up) while the previous kernel of the stream is still running; chain_wait() blocks until that kernel
// has completed and its writes are visible, and must precede every access to global memory.  chain_release() lets the
// next chained kernel of the stream start launching once every block of this grid has called it (or exited).
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args... args) {
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#define LASER_CUDA_OK(expr)                          \
  do {                                               \
    cudaError_t _e = (expr);                         \
    if (_e != cudaSuccess) return LASER_ERR_CUDA;    \
  } while (0)

}  // namespace laser
