// Fragment-ordered images of the GSTA weights, shared by the kernels that can build them on the side (the GSTA
// kernel's own set-up launch, or spare blocks of the STA paths' set-up kernels when STA and GSTA run back to back).
//
// Entry (layer, matrix, kt, p, lane) holds the mma.sync B fragments of k-tile kt for the two 8-column tiles 2p and
// 2p+1: {b0, b1 of tile 2p, b0, b1 of tile 2p+1}.  For W_q and W_v the MMA's B is W itself (B[k][n] = W[k][n]); for
// W_k it is the transpose (B[k][n] = W_k[n][k]).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

#include "laser.h"

namespace laser {

// Called by `n_workers` threads with ranks worker = 0 .. n_workers - 1; img has M * 3 * (d/16)^2 * 32 entries.
__device__ __forceinline__ void gsta_build_images(const __nv_bfloat16* Wg, uint4* img, int d, int M, int worker,
                                                  int n_workers) {
  const int D16 = d >> 4;
  const int total = M * 3 * D16 * D16 * 32;
  for (int i = worker; i < total; i += n_workers) {
    const int lane = i & 31;
    int r = i >> 5;
    const int p = r % D16; r /= D16;
    const int kt = r % D16; r /= D16;
    const int m = r % 3;
    const int l = r / 3;
    const uint16_t* W = reinterpret_cast<const uint16_t*>(Wg) + (size_t)(l * 3 + m) * d * d;
    const int g = lane >> 2, t = lane & 3;
    uint32_t v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int n = (2 * p + (q >> 1)) * 8 + g;
      const int k = kt * 16 + 2 * t + (q & 1) * 8;
      uint32_t lo, hi;
      if (m == 1) { lo = W[(size_t)n * d + k]; hi = W[(size_t)n * d + k + 1]; }
      else { lo = W[(size_t)k * d + n]; hi = W[(size_t)(k + 1) * d + n]; }
      v[q] = lo | (hi << 16);
    }
    img[i] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

// Per candidate: the number of non-empty segments of its user (what the GSTA kernel's softmax runs over), so that the
// kernel's blocks need no search through the candidate offsets.  Filled user by user: warp `warp_id` of `n_warps` takes
// users warp_id, warp_id + n_warps, ... and its lanes write that user's candidates.  A user with an invalid length or
// offsets is reported through `status` and skipped (its candidates keep whatever the scratch held; the GSTA kernel
// clamps what it reads to [0, L']); so are offsets that do not cover candidates 0 .. N - 1.
__device__ __forceinline__ void gsta_build_nseg(const int* lengths, const int* cand_offsets, int U, int N, int L, int S,
                                                int Lp, int* status, int* nseg, int warp_id, int n_warps, int lane) {
  if (warp_id == 0 && lane == 0 && N > 0 && (cand_offsets[0] != 0 || cand_offsets[U] < N))
    atomicCAS(status, 0, LASER_ERR_BAD_INPUT);
  for (int u = warp_id; u < U; u += n_warps) {
    const int len = lengths[u], c0 = cand_offsets[u], c1 = cand_offsets[u + 1];
    if (len < 0 || len > L || c0 < 0 || c1 < c0 || c1 > N) {
      if (lane == 0) atomicCAS(status, 0, LASER_ERR_BAD_INPUT);
      continue;
    }
    const int nv = min((len + S - 1) / S, Lp);
    for (int c = c0 + lane; c < c1; c += 32) nseg[c] = nv;
  }
}

// Counting sort, largest key first: order[0 .. n - 1] = the indices 0 .. n - 1 by descending key(i) (keys in
// 0 .. kGstaOrderBins - 1; equal keys land in arbitrary order).  Run by ONE thread block (all of its threads call this, at
// least one warp); keys: n ints of scratch.
constexpr int kGstaOrderBins = 1024;
template <class KeyFn>
__device__ __forceinline__ void sort_desc_by_key(int n, KeyFn key_of, int* order, int* keys) {
  __shared__ int bins[kGstaOrderBins + kGstaOrderBins / 32];      // bin k at k + k / 32: lane-strided walks stay conflict-free
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int i = tid; i < kGstaOrderBins + kGstaOrderBins / 32; i += nt) bins[i] = 0;
  __syncthreads();
  constexpr int kBatch = 8;                      // independent loads first, then the atomics: the passes are latency-bound
  for (int b0 = tid; b0 < n; b0 += kBatch * nt) {
    int key[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int b = b0 + j * nt;
      key[j] = b < n ? min(max(key_of(b), 0), kGstaOrderBins - 1) : -1;
    }
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      if (key[j] >= 0) {
        keys[b0 + j * nt] = key[j];
        atomicAdd(&bins[key[j] + (key[j] >> 5)], 1);
      }
    }
  }
  __syncthreads();
  if (tid < 32) {                                // bins[k] <- number of items with a larger key (lane `tid` owns 32 bins)
    int mine = 0;
    for (int j = 0; j < 32; ++j) mine += bins[tid * 33 + j];
    int incl = mine;                             // items in this lane's bins and in those of the lanes above
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_down_sync(0xffffffffu, incl, off);
      if (tid + off < 32) incl += v;
    }
    int run = incl - mine;
    for (int j = 31; j >= 0; --j) {
      const int cnt = bins[tid * 33 + j];
      bins[tid * 33 + j] = run;
      run += cnt;
    }
  }
  __syncthreads();
  for (int b0 = tid; b0 < n; b0 += kBatch * nt) {
    int key[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) key[j] = b0 + j * nt < n ? keys[b0 + j * nt] : -1;
#pragma unroll
    for (int j = 0; j < kBatch; ++j)
      if (key[j] >= 0) order[atomicAdd(&bins[key[j] + (key[j] >> 5)], 1)] = b0 + j * nt;
  }
}

// Launch order of the GSTA kernel's blocks, longest first: block b of the kernel takes candidates
// order[b] * cpb .. order[b] * cpb + cpb - 1.  A block's time grows with the number of segments of its candidates, and a
// grid of several waves that ends on long blocks leaves most SMs idle during the last of them; started longest first,
// the tail is made of the shortest blocks.  Sorted by the segment count of each block's first candidate (counts
// above kGstaOrderBins - 1 share the last bin), by ONE thread block.  keys: n_blocks ints of scratch.  Invalid lengths
// or offsets are reported elsewhere; here they are clamped, so `order` is a permutation of 0 .. n_blocks - 1 whatever
// the inputs hold.
__device__ __forceinline__ void gsta_build_order(const int* lengths, const int* cand_offsets, int U, int N, int L, int S,
                                                 int Lp, int cpb, int* order, int* keys) {
  const int n_blocks = (N + cpb - 1) / cpb;
  sort_desc_by_key(n_blocks, [&](int b) {
    const int c = b * cpb;
    int lo = 0, hi = U - 1;                      // the last user whose first candidate is <= c
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (cand_offsets[mid] <= c) lo = mid; else hi = mid - 1;
    }
    const int len = min(max(lengths[lo], 0), L);
    return min((len + S - 1) / S, Lp);
  }, order, keys);
}

}  // namespace laser
