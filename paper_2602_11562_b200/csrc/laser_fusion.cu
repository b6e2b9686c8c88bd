// Multi-resolution feature fusion: fused = [ z | max-pool of the non-empty segment vectors | the r most recent ones ].
// One warp per candidate; every row of H' is read once with 128-bit loads (HBM bound: 2 L'_valid d bytes in,
// (2 + r) d elements out per candidate).
#include "laser_common.cuh"

namespace laser {
namespace {

constexpr int kFThreads = 128;

template <typename T> struct Vec16;     // 16 bytes of T as floats
template <> struct Vec16<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ void load(const float* p, float (&v)[8]) {
    const float4 x = *reinterpret_cast<const float4*>(p);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&v)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 x = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {   // values are exact bf16
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = (__float_as_uint(v[2 * i]) >> 16) | (__float_as_uint(v[2 * i + 1]) & 0xFFFF0000u);
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

template <typename T>
__global__ void __launch_bounds__(kFThreads)
fusion_kernel(const T* __restrict__ Hp, const T* __restrict__ z, const int* __restrict__ lengths,
              const int* __restrict__ cand_offsets, T* __restrict__ fused, int U, int L, int S, int Lp, int d, int N,
              int r, int* __restrict__ status) {
  constexpr int E = Vec16<T>::kElems;
  const int lane = threadIdx.x & 31;
  const int c = blockIdx.x * (kFThreads / 32) + (threadIdx.x >> 5);
  if (c >= N) return;
  int nseg = 0;
  if (cand_offsets[0] > c || cand_offsets[U] <= c) {
    if (lane == 0) report_status(status, LASER_ERR_BAD_INPUT);
  } else {
    // the warp searches together, 32 probes per round trip: cand_offsets[lo] <= c < cand_offsets[hi]
    int lo = 0, hi = U;
    while (hi - lo > 1) {
      const int step = (hi - lo + 31) / 32;
      const int idx = min(lo + lane * step, hi);
      const unsigned le = __ballot_sync(0xffffffffu, idx < hi && cand_offsets[idx] <= c);   // a prefix of the lanes
      const int k = __popc(le);                         // >= 1: lane 0 probes lo itself
      lo = lo + (k - 1) * step;
      hi = min(lo + step, hi);
    }
    const int len = lengths[lo];
    if (len < 0 || len > L) { if (lane == 0) report_status(status, LASER_ERR_BAD_INPUT); }
    else nseg = min((len + S - 1) / S, Lp);
  }
  const int ppr = d / E;                    // 16-byte pieces per row
  const T* hc = Hp + (size_t)c * Lp * d;
  T* out = fused + (size_t)c * (2 + r) * d;
  for (int p = lane; p < ppr; p += 32) {
    float v[8];
    Vec16<T>::load(z + (size_t)c * d + p * E, v);
    Vec16<T>::store(out + p * E, v);
  }
  // max pool: the warp walks the valid rows piece by piece; lane l owns piece l % ppr of rows l / ppr, + 32 / ppr, ...
  // (when a row has more than 32 pieces, every lane owns several pieces of every row)
  if (ppr <= 32) {
    const int rows_per_step = 32 / ppr, my_p = lane % ppr, my_r = lane / ppr;
    float best[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) best[i] = -INFINITY;
    if (my_r < rows_per_step) {
      int j = my_r;
      for (; j + 3 * rows_per_step < nseg; j += 4 * rows_per_step) {      // four independent loads in flight
        float v[4][8];
#pragma unroll
        for (int k = 0; k < 4; ++k) Vec16<T>::load(hc + (size_t)(j + k * rows_per_step) * d + my_p * E, v[k]);
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
          for (int i = 0; i < E; ++i) best[i] = fmaxf(best[i], v[k][i]);
      }
      for (; j < nseg; j += rows_per_step) {
        float v[8];
        Vec16<T>::load(hc + (size_t)j * d + my_p * E, v);
#pragma unroll
        for (int i = 0; i < E; ++i) best[i] = fmaxf(best[i], v[i]);
      }
    }
    // combine the row groups: lanes p, p + ppr, p + 2 ppr, ... hold the same piece
    for (int off = ppr; off < 32; off <<= 1) {
#pragma unroll
      for (int i = 0; i < E; ++i) {
        const float o = __shfl_down_sync(0xffffffffu, best[i], off);
        if (lane + off < rows_per_step * ppr) best[i] = fmaxf(best[i], o);
      }
    }
    if (lane < ppr) {
      if (nseg == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) best[i] = 0.f;
      }
      Vec16<T>::store(out + d + lane * E, best);
    }
  } else {
    for (int p = lane; p < ppr; p += 32) {
      float best[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) best[i] = nseg > 0 ? -INFINITY : 0.f;
      for (int j = 0; j < nseg; ++j) {
        float v[8];
        Vec16<T>::load(hc + (size_t)j * d + p * E, v);
#pragma unroll
        for (int i = 0; i < E; ++i) best[i] = fmaxf(best[i], v[i]);
      }
      Vec16<T>::store(out + d + p * E, best);
    }
  }
  // the r most recent segment vectors (zero vectors past the user's segments)
  for (int q = lane; q < r * ppr; q += 32) {
    const int j = q / ppr, p = q - j * ppr;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    if (j < nseg) Vec16<T>::load(hc + (size_t)j * d + p * E, v);
    Vec16<T>::store(out + (size_t)(2 + j) * d + p * E, v);
  }
}

}  // namespace

int fusion_forward(const Plan& p, const void* Hprime, const void* z, const int32_t* lengths, const int32_t* cand_offsets,
                   int num_recent, void* fused, char* ws, cudaStream_t st) {
  if (p.N == 0) return LASER_OK;
  if ((p.d * p.esize) % 16) return LASER_ERR_UNSUPPORTED;
  int* status = reinterpret_cast<int*>(ws + p.off_status);
  const int blocks = (p.N + kFThreads / 32 - 1) / (kFThreads / 32);
  LaunchScope ls("fusion", st);
  if (p.dtype == LASER_F32)
    fusion_kernel<float><<<blocks, kFThreads, 0, st>>>((const float*)Hprime, (const float*)z, lengths, cand_offsets,
                                                        (float*)fused, p.U, p.L, p.S, p.Lp, p.d, p.N, num_recent, status);
  else
    fusion_kernel<__nv_bfloat16><<<blocks, kFThreads, 0, st>>>((const __nv_bfloat16*)Hprime, (const __nv_bfloat16*)z,
                                                                lengths, cand_offsets, (__nv_bfloat16*)fused, p.U, p.L,
                                                                p.S, p.Lp, p.d, p.N, num_recent, status);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace laser
