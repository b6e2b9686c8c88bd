// Feed-forward refinement of the segment vectors (Eq. 6):  s <- LN(max(s W_1 + b_1, 0) W_2 + b_2 + s), applied in place
// to the rows of H' that belong to non-empty segments.
//
//   ffn_prep_kernel   prefix of the valid rows per user (the "compact" row numbering the main kernel tiles over), the
//                     weights re-laid as MMA operand images (one 128-hidden-unit chunk after the other) and fp32 copies
//                     of b_2 and of the layer norm's gain and shift.
//   ffn_map_kernel    compact row -> row of H' for every valid row, so that the main kernel finds its rows with one
//                     coalesced load.
//   ffn_tc_kernel     bf16, tcgen05: a persistent block (one per SM) owns pairs of 128-row tiles.  Per pair and per chunk
//                     j of 128 hidden units:  acc1 = X W_1[:, j] (shared-memory operands, TMEM accumulator)  ->  + b_1,
//                     ReLU, bf16 in registers, written back over acc1  ->  acc2 += hidden_j W_2[j, :] with the hidden
//                     activations read straight from TMEM.  Nothing of the hidden layer ever leaves the SM; the weights
//                     stream through a three-slot ring of bulk copies (they stay in L2) and both tiles of the pair share
//                     every chunk.  At the end of a pair the layer-norm warps add b_2 and the residual, normalise each row
//                     (one thread owns one row of the accumulator) and write bf16 rows back, while the other warps are
//                     already busy with the next pair.
//   ffn_simt_kernel   FP32-ALU version for fp32 data and for shapes outside the tensor kernel's envelope.
//
// Roofline: 4 d d_hidden flops per valid row on the tensor cores (the H' rows themselves are read and written once,
// 4 d bytes per row, far below the HBM bound at d_hidden = 4 d).
#include "laser_common.cuh"
#include "laser_ptx.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
using namespace ptx;

constexpr int kRows = 128;            // rows per tile = MMA M = TMEM lanes
constexpr int kChunk = 128;           // hidden units per step
constexpr int kPairRows = 2 * kRows;  // two tiles share every weight chunk
constexpr int kFfnThreads = 576;      // warp 0 weight producer + TMEM, warp 1 MMA issuer, warps 2-5 / 6-9 hidden-
                                      // activation warpgroups of tile 0 / 1, warps 10-13 / 14-17 layer-norm warpgroups
constexpr int kWStages = 3;
constexpr int kFfnTmemCols = 512;     // acc2[t] at 128 t; acc1[t], then the hidden activations, at 256 + 128 t
constexpr int kSimtRows = 8;

struct FfnParams {
  int U, N, L, Lp, S, d, hid, NJ, maxC;
  float eps;
  bf16* H;                                    // [N, Lp, d] in / out
  const bf16 *W1, *b1, *W2, *b2, *g, *beta;
  const int *lengths, *cand_offsets;
  int* prefix;                                // [U + 1] valid rows before each user
  int* counters;                              // [0] total valid rows
  bf16 *img1, *img2;                          // chunk j of W_1^T / W_2^T at + j * 128 * d
  float* lnv;                                 // [3][d] fp32 copies of b_2, the layer norm's gain and its shift
  int* rowmap;                                // [N * Lp] compact row -> row of H' (first counters[0] entries valid)
  int* status;
};

struct RowUser {
  int c0, nc, nseg;
};
// Sanitised view of one user (an invalid length / offset pair behaves like an empty user).
template <typename PT>
__device__ __forceinline__ RowUser row_user(const PT& P, int u) {
  const int len = P.lengths[u], c0 = P.cand_offsets[u], c1 = P.cand_offsets[u + 1];
  const bool bad = len < 0 || len > P.L || c0 < 0 || c1 < c0 || c1 > P.N || c1 - c0 > P.maxC;
  RowUser s;
  s.c0 = bad ? 0 : c0;
  s.nc = bad ? 0 : c1 - c0;
  s.nseg = bad ? 0 : (len + P.S - 1) / P.S;
  return s;
}
// Compact row -> row of H' (candidate * Lp + segment); compact rows enumerate, user by user and candidate by candidate,
// the segments that hold items.  -1 past the end.
template <typename PT>
__device__ __forceinline__ int global_row(const PT& P, int crow, int total) {
  if (crow >= total) return -1;
  int lo = 0, hi = P.U - 1;                   // largest u with prefix[u] <= crow
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (P.prefix[mid] <= crow) lo = mid; else hi = mid - 1;
  }
  const RowUser s = row_user(P, lo);
  const int local = crow - P.prefix[lo];
  if (s.nseg <= 0 || local >= s.nc * s.nseg) return -1;
  const int c = local / s.nseg;
  return (s.c0 + c) * P.Lp + (local - c * s.nseg);
}

__device__ __forceinline__ int canon_off(int row, int k, int kdim) {   // K-major 8x8 core matrices, no swizzle
  return ((row >> 3) * (kdim >> 3) + (k >> 3)) * 64 + (row & 7) * 8 + (k & 7);
}

// ------------------------------------------------------------------------------------------------------- set-up
template <typename PT>
__device__ void scan_rows(const PT& P, int* status) {
  __shared__ int sa[1024];
  const int tid = threadIdx.x;
  const int per = (P.U + 1023) / 1024;
  const int n_act = max(1, (P.U + per - 1) / per);        // threads that own users: the scan runs over these only
  const int u0 = min(tid * per, P.U), u1 = min(u0 + per, P.U);
  int a = 0;
  bool bad = false;
  for (int u = u0; u < u1; ++u) {
    const int len = P.lengths[u], c0 = P.cand_offsets[u], c1 = P.cand_offsets[u + 1];
    bad |= len < 0 || len > P.L || c0 < 0 || c1 < c0 || c1 > P.N || c1 - c0 > P.maxC;
    const RowUser s = row_user(P, u);
    a += s.nc * s.nseg;
  }
  if (bad) report_status(status, LASER_ERR_BAD_INPUT);
  sa[tid] = a;
  __syncthreads();
  for (int off = 1; off < n_act; off <<= 1) {
    const int v = tid >= off ? sa[tid - off] : 0;
    __syncthreads();
    sa[tid] += v;
    __syncthreads();
  }
  int pa = sa[tid] - a;
  for (int u = u0; u < u1; ++u) {
    const RowUser s = row_user(P, u);
    P.prefix[u] = pa;
    pa += s.nc * s.nseg;
  }
  if (tid == n_act - 1) {
    P.prefix[P.U] = sa[n_act - 1];
    P.counters[0] = sa[n_act - 1];
  }
}

__global__ void __launch_bounds__(1024) ffn_prep_kernel(FfnParams P, int build_images) {
  chain_wait();
  chain_release();
  if (blockIdx.x == 0) {
    scan_rows(P, P.status);
    return;
  }
  if (!build_images) return;
  const int nthreads = (gridDim.x - 1) * blockDim.x;
  const int g = (blockIdx.x - 1) * blockDim.x + threadIdx.x;
  for (int i = g; i < P.d; i += nthreads) {
    P.lnv[i] = __bfloat162float(P.b2[i]);
    P.lnv[P.d + i] = __bfloat162float(P.g[i]);
    P.lnv[2 * P.d + i] = __bfloat162float(P.beta[i]);
  }
  const int n = P.d * P.hid;
  const int chunk_elems = kChunk * P.d;
  for (int i = g; i < n; i += nthreads) {          // W_1[k][h]: B operand of step j = h / 128, row h % 128, K index k
    const int k = i / P.hid, h = i - k * P.hid;
    P.img1[(h / kChunk) * chunk_elems + canon_off(h % kChunk, k, P.d)] = P.W1[i];
  }
  for (int i = g; i < n; i += nthreads) {          // W_2[h][e]: B operand of step j = h / 128, row e, K index h % 128
    const int h = i / P.d, e = i - h * P.d;
    P.img2[(h / kChunk) * chunk_elems + canon_off(e, h % kChunk, kChunk)] = P.W2[i];
  }
}

// Compact row -> row of H', for every valid row (the main kernel reads it with coalesced loads).
__global__ void __launch_bounds__(256) ffn_map_kernel(FfnParams P) {
  chain_wait();
  chain_release();
  const int total = P.counters[0];
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x)
    P.rowmap[i] = global_row(P, i, total);
}

// ------------------------------------------------------------------------------------------------------- tensor kernel
struct FfnBars {
  uint64_t w_full[kWStages], w_empty[kWStages];
  uint64_t x_full[2];                   // X[t] staged (4 hidden-activation warps)
  uint64_t x_free[2];                   // X[t] of a finished pair written back (4 layer-norm warps)
  uint64_t a1_full[2];                  // first-layer product of tile t complete
  uint64_t hid_full[2];                 // hidden activations of tile t written to TMEM (4 epilogue warps)
  uint64_t a2_full[2], a2_free[2];      // second-layer accumulator of tile t complete / drained (4 epilogue warps)
  uint64_t done;
};

__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
// max(a + b, 0) on two packed bf16 values (one fused multiply-add by 1 with the ReLU modifier)
__device__ __forceinline__ uint32_t relu_add_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("fma.rn.relu.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(0x3F803F80u), "r"(b));
  return r;
}

// Roles: warp 0 streams the weight chunks (W_1 chunk 0, W_2 chunk 0, W_1 chunk 1, ...), warp 1 issues the MMAs, warps
// 2-5 / 6-9 are the epilogue warpgroups of tile 0 / tile 1.  Per chunk j the issue order is
//     acc1[0] = X[0] W_1j,  acc1[1] = X[1] W_1j,  acc2[0] += hid[0] W_2j,  acc2[1] += hid[1] W_2j
// so tile 1's first-layer product runs while tile 0's epilogue warps turn acc1[0] into hidden activations, and so on.
// The hidden activations (bf16) are written back into the first 64 columns of the accumulator they came from and feed
// the second-layer product straight from TMEM: the first layer's operand reads already take the whole shared-memory
// bandwidth, the second layer then leaves it to the weight copies, the row staging and the output staging.
// The tensor pipe executes a block's MMAs in issue order, so the next first-layer product cannot overwrite hidden
// activations that the second-layer product before it still reads.
// An epilogue warp owns 32 rows of its tile (TMEM lanes 32 (warp mod 4) .. + 31): it stages them (K-major) for the
// first layer, produces their hidden activations, normalises them at the end and writes them back; the shared memory
// it touches for all of this is its own rows' slice of X and of the output staging, so the warps never meet at a barrier.
__global__ void __launch_bounds__(kFfnThreads, 1) ffn_tc_kernel(FfnParams P) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ FfnBars bars;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = P.d, NJ = P.NJ;
  const uint32_t x_bytes = kRows * d * 2, w_bytes = kChunk * d * 2;
  uint8_t* Xs = smem_raw;                              // [2 pairs][2 tiles][128 x d]  K-major, K = d; pair p in buffer p & 1
  uint8_t* Ws = Xs + 4 * x_bytes;                      // [kWStages][128 d]  one weight chunk each
  float* s_lnv = reinterpret_cast<float*>(Ws + kWStages * w_bytes);        // [3][d] b_2, gain, shift
  bf16* s_b1 = reinterpret_cast<bf16*>(s_lnv + 3 * d);                      // [hid]

  if (tid == 0) {
    for (int i = 0; i < kWStages; ++i) { mbar_init(&bars.w_full[i], 1); mbar_init(&bars.w_empty[i], 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.x_full[i], 4);
      mbar_init(&bars.x_free[i], 4);
      mbar_init(&bars.a1_full[i], 1);
      mbar_init(&bars.hid_full[i], 4);
      mbar_init(&bars.a2_full[i], 1);
      mbar_init(&bars.a2_free[i], 4);
    }
    mbar_init(&bars.done, 1);
    s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s_tmem, kFfnTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;
  chain_wait();                         // H' rows, the row map and the weight images are complete
  chain_release();

  for (int i = tid; i < 3 * d; i += kFfnThreads) s_lnv[i] = P.lnv[i];
  for (int i = tid; i < P.hid; i += kFfnThreads) s_b1[i] = P.b1[i];
  __syncthreads();
  const int total = P.counters[0];
  const int n_pairs = (total + kPairRows - 1) / kPairRows;
  const int G = gridDim.x, bidx = blockIdx.x;
  const int my_pairs = bidx < n_pairs ? (n_pairs - bidx + G - 1) / G : 0;
  auto wait_all = [&](uint64_t* bar, uint32_t parity) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abortp)) != 0;
  };
  // Two barriers polled together (their round trips to shared memory overlap); bounded like mbar_wait.
  auto wait_both = [&](uint64_t* b0, uint32_t p0, uint64_t* b1, uint32_t p1) {
    bool done = false;
    for (uint32_t i = 0; i < kSpinLimit && !done; ++i) {
      const bool r0 = mbar_try_wait(b0, p0), r1 = mbar_try_wait(b1, p1);
      done = r0 && r1;
      if (!done && (i & 63u) == 63u) {
        if (*abortp) break;
        __nanosleep(64);
      }
    }
    if (!done) *abortp = 1;
    return __all_sync(0xffffffffu, done) != 0;
  };

  if (my_pairs > 0) {
    if (warp == 0) {
      // ------------------------------------------------------------------ weight chunks: L2 -> ring
      if (lane == 0) {
        uint32_t use = 0;
        bool ok = true;
        for (int it = 0; it < my_pairs && ok; ++it) {
          for (int s = 0; s < 2 * NJ && ok; ++s, ++use) {
            const uint32_t slot = use % kWStages;
            ok = mbar_wait(&bars.w_empty[slot], ((use / kWStages) & 1) ^ 1, abortp);
            if (!ok) break;
            mbar_arrive_expect_tx(&bars.w_full[slot], w_bytes);
            bulk_g2s(Ws + slot * w_bytes, ((s & 1) ? P.img2 : P.img1) + (size_t)(s >> 1) * kChunk * d, w_bytes,
                     &bars.w_full[slot]);
          }
        }
        if (!ok) {                                       // let the copies in flight land before the block goes away
          const uint32_t first = use > kWStages ? use - kWStages : 0;
          for (uint32_t k = first; k < use; ++k) {
            const uint32_t slot = k % kWStages, par = (k / kWStages) & 1;
            for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(&bars.w_full[slot], par); ++i) __nanosleep(64);
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------------ MMA issuer (warp-uniform loop, one lane issues)
      const bool leader = elect_one();
      const uint32_t x_sbo = (d >> 3) * 128, h_sbo = (kChunk >> 3) * 128;
      const uint32_t id1 = idesc_bf16(128, kChunk), id2 = idesc_bf16(128, d);
      const int ks1 = d >> 4;
      const uint64_t xd0 = smem_desc(smem_u32(Xs), 128, x_sbo);
      const uint64_t w1d0 = smem_desc(smem_u32(Ws), 128, x_sbo), w2d0 = smem_desc(smem_u32(Ws), 128, h_sbo);
      uint32_t slot = 0, w_par = 0;
      bool ok = true;
      for (int it = 0; it < my_pairs && ok; ++it) {
        for (int j = 0; j < NJ && ok; ++j) {
          const uint32_t k = (uint32_t)it * NJ + j;
          // ---- first layer of chunk j, both tiles
          if (j == 0) ok = wait_both(&bars.x_full[0], it & 1, &bars.x_full[1], it & 1);
          ok = ok && wait_all(&bars.w_full[slot], w_par);
          if (!ok) break;
          tc_fence_after();
          {
            const uint64_t bd = w1d0 + (uint64_t)(slot * (w_bytes >> 4));
            if (leader) {
              for (int t = 0; t < 2; ++t) {
                const uint64_t ad = xd0 + (uint64_t)((2 * (it & 1) + t) * (x_bytes >> 4));
                for (int ks = 0; ks < ks1; ++ks) mma_ss(tmem + 256 + t * kChunk, ad + ks * 16, bd + ks * 16, id1, ks > 0);
                tc_commit(&bars.a1_full[t]);
              }
              tc_commit(&bars.w_empty[slot]);
            }
            __syncwarp();
            if (++slot == kWStages) { slot = 0; w_par ^= 1; }
          }
          // ---- second layer of chunk j: acc2[t] += hid[t] (TMEM) W_2j
          ok = wait_both(&bars.w_full[slot], w_par, &bars.hid_full[0], k & 1);
          if (ok && j == 0) ok = wait_both(&bars.a2_free[0], (it & 1) ^ 1, &bars.a2_free[1], (it & 1) ^ 1);
          if (!ok) break;
          tc_fence_after();
          const uint64_t bd = w2d0 + (uint64_t)(slot * (w_bytes >> 4));
          for (int t = 0; t < 2; ++t) {
            if (t == 1) {
              ok = wait_all(&bars.hid_full[1], k & 1);
              if (!ok) break;
              tc_fence_after();
            }
            if (leader) {
#pragma unroll
              for (int ks = 0; ks < kChunk / 16; ++ks)
                mma_ts(tmem + t * 128, tmem + 256 + t * kChunk + ks * 8, bd + ks * 16, id2, (j | ks) != 0);
              if (j == NJ - 1) tc_commit(&bars.a2_full[t]);
            }
            __syncwarp();
          }
          if (ok && leader) tc_commit(&bars.w_empty[slot]);
          __syncwarp();
          if (++slot == kWStages) { slot = 0; w_par ^= 1; }
        }
      }
      if (leader) tc_commit(&bars.done);
      __syncwarp();
      wait_all(&bars.done, 0);
    } else if (warp < 10) {
      // ------------------------------------------------------------------ hidden-activation warp: rows 32 quad .. + 31 of tile t
      const int t = (warp - 2) >> 2, quad = warp & 3;
      const int r = quad * 32 + lane;                      // my row of the tile = my TMEM lane
      const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
      const int cpr = d >> 3;                              // 16-byte chunks per row
      // this warp's four 8-row groups of X[t] in buffer b (32 rows, K-major)
      auto x_slice = [&](int b) { return Xs + (size_t)(2 * b + t) * x_bytes + (size_t)(quad * 4) * cpr * 128; };
      // pieces [i0, i1) of the cpr this lane copies for one pair: piece i is (group, chunk) number (lane >> 3) + 4 i of
      // row-in-group lane & 7
      auto stage = [&](int grow_mine, uint8_t* xw, int i0, int i1) {
        int idx = (lane >> 3) + 4 * i0;
        int gq = idx / cpr, c = idx - gq * cpr;
        for (int i = i0; i < i1; ++i, idx += 4, c += 4) {
          while (c >= cpr) { c -= cpr; ++gq; }
          const int grow = __shfl_sync(0xffffffffu, grow_mine, gq * 8 + (lane & 7));
          const bf16* src = grow >= 0 ? P.H + (size_t)grow * d + c * 8 : P.H;
          cp_async16(xw + (size_t)idx * 128 + (lane & 7) * 16, src, grow >= 0 ? 16u : 0u);
        }
      };
      auto publish_x = [&]() {                             // my copies have landed: tell the issuer
        cp_async_wait_all();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.x_full[t]);
      };
      auto row_of = [&](int pair) {
        const int crow = pair * kPairRows + t * kRows + r;
        return crow < total ? P.rowmap[crow] : -1;
      };
      stage(row_of(bidx), x_slice(0), 0, cpr);
      publish_x();
      const int j_stage0 = NJ / 2;
      bool ok = true;
      for (int it = 0; it < my_pairs && ok; ++it) {
        const int grow_next = it + 1 < my_pairs ? row_of(bidx + (it + 1) * G) : -1;
        const uint32_t tA = tmem + lane_base + 256 + t * kChunk;
        uint8_t* x_next = x_slice((it + 1) & 1);
        // ---- first layer: acc1 -> + b_1, ReLU, bf16 -> back into the first 64 columns of acc1 (A operand of the
        // second layer)
        for (int j = 0; j < NJ && ok; ++j) {
          const uint32_t kh = (uint32_t)it * NJ + j;
          // in the later chunks a share of the next pair's rows goes on its way while the first-layer product runs
          if (it + 1 < my_pairs && j >= j_stage0) {
            // (the other buffer: the layer-norm warps must have written its pair back)
            if (j == j_stage0 && it > 0) ok = wait_all(&bars.x_free[t], (it - 1) & 1);
            if (!ok) break;
            stage(grow_next, x_next, ((j - j_stage0) * cpr) / (NJ - j_stage0), ((j - j_stage0 + 1) * cpr) / (NJ - j_stage0));
          }
          ok = wait_all(&bars.a1_full[t], kh & 1);
          if (!ok) break;
          tc_fence_after();
          const uint4* bias = reinterpret_cast<const uint4*>(s_b1 + (size_t)j * kChunk);
          // 32 accumulator columns at a time; their 16 packed columns land on accumulator columns that are already in
          // registers (packed columns 16 c .. 16 c + 15 lie inside the 32-column batch c / 2)
#pragma unroll
          for (int c = 0; c < kChunk / 32; ++c) {
            uint32_t v[32], w16[16];
            tmem_ld32(tA + c * 32, v);
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 bb = bias[c * 4 + q];
              const uint32_t bw[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
              for (int e = 0; e < 4; ++e)                  // round the pair to bf16, then max(h + b_1, 0) on both halves at once
                w16[q * 4 + e] = relu_add_bf16x2(
                    pack_bf16x2(__uint_as_float(v[q * 8 + 2 * e]), __uint_as_float(v[q * 8 + 2 * e + 1])), bw[e]);
            }
            tmem_st16(tA + c * 16, w16);
          }
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars.hid_full[t]);
        }
        if (!ok) break;
        if (it + 1 < my_pairs) publish_x();                // the next pair's rows are staged
      }
      cp_async_wait_all();
    } else {
      // ------------------------------------------------------------------ layer-norm warp: rows 32 quad .. + 31 of tile t
      const int t = (warp - 10) >> 2, quad = warp & 3;
      const int r = quad * 32 + lane;                      // my row of the tile = my TMEM lane
      const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
      const int cpr = d >> 3;                              // 16-byte chunks per row
      const float inv_d = 1.f / (float)d;
      const bool swz = (cpr & (cpr - 1)) == 0;             // XOR-swizzled staging rows when cpr is a power of two
      const int rows_per = 32 / cpr;                       // rows covered by one coalesced store instruction
      bool ok = true;
      for (int it = 0; it < my_pairs && ok; ++it) {
        const int crow = (bidx + it * G) * kPairRows + t * kRows + r;
        const int grow = crow < total ? P.rowmap[crow] : -1;
        // this warp's 32 rows of X[t]: K-major as staged (read for the residual), then row-major output staging
        uint8_t* x_warp = Xs + (size_t)(2 * (it & 1) + t) * x_bytes + (size_t)(quad * 4) * cpr * 128;
        uint8_t* o_row = x_warp + (size_t)lane * (d * 2);   // my row of the output staging; chunk c sits at slot(c)
        auto slot_of = [&](int c) { return (swz ? c ^ (lane & (cpr - 1)) : c) << 4; };
        const uint8_t* x_row = x_warp + (size_t)(lane >> 3) * cpr * 128 + (lane & 7) * 16;   // my staged row: chunk c at + 128 c
        // ---- second layer: y = acc2 + b_2 + s, layer norm over the row
        ok = wait_all(&bars.a2_full[t], it & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tO = tmem + lane_base + t * 128;
        const float4* vb2 = reinterpret_cast<const float4*>(s_lnv);
        const float4* vg = reinterpret_cast<const float4*>(s_lnv + d);
        const float4* vbeta = reinterpret_cast<const float4*>(s_lnv + 2 * d);
        // pass 1: y = acc2 + b_2 + s (two features at a time with the packed fp32 instructions), written back over the
        // accumulator; row sums of y and y^2
        float2 sum2 = make_float2(0.f, 0.f), sq2 = make_float2(0.f, 0.f);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          if (h * 32 < d) {
            uint32_t v[2][16];
#pragma unroll
            for (int k = 0; k < 2; ++k)
              if (h * 32 + k * 16 < d) tmem_ld16(tO + h * 32 + k * 16, v[k]);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              if (h * 32 + k * 16 < d) {
                const int c16 = h * 2 + k;
#pragma unroll
                for (int q = 0; q < 2; ++q) {                // 8 features: one 16-byte chunk of the residual
                  const uint4 xx = *reinterpret_cast<const uint4*>(x_row + (c16 * 2 + q) * 128);
                  const float4 b0 = vb2[c16 * 4 + q * 2], b1 = vb2[c16 * 4 + q * 2 + 1];
                  const uint32_t xw[4] = {xx.x, xx.y, xx.z, xx.w};
                  const float2 bb[4] = {make_float2(b0.x, b0.y), make_float2(b0.z, b0.w), make_float2(b1.x, b1.y),
                                        make_float2(b1.z, b1.w)};
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    const float2 acc = make_float2(__uint_as_float(v[k][q * 8 + 2 * e]), __uint_as_float(v[k][q * 8 + 2 * e + 1]));
                    const float2 y = __fadd2_rn(__fadd2_rn(acc, bb[e]), make_float2(bf_lo(xw[e]), bf_hi(xw[e])));
                    sum2 = __fadd2_rn(sum2, y);
                    sq2 = __ffma2_rn(y, y, sq2);
                    v[k][q * 8 + 2 * e] = __float_as_uint(y.x);
                    v[k][q * 8 + 2 * e + 1] = __float_as_uint(y.y);
                  }
                }
                tmem_st16(tO + c16 * 16, v[k]);
              }
            }
          }
        }
        tc_wait_st();
        __syncwarp();                                      // every lane has read its residual: the slice becomes output staging
        const float mean = (sum2.x + sum2.y) * inv_d;
        const float rstd = rsqrtf(fmaxf((sq2.x + sq2.y) * inv_d - mean * mean, 0.f) + P.eps);
        const float2 rstd2 = make_float2(rstd, rstd), shift2 = make_float2(-mean * rstd, -mean * rstd);
        // pass 2: ((y - mean) rstd) gain + shift -> bf16 -> my row of the output staging
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          if (h * 32 < d) {
            uint32_t v[2][16];
#pragma unroll
            for (int k = 0; k < 2; ++k)
              if (h * 32 + k * 16 < d) tmem_ld16(tO + h * 32 + k * 16, v[k]);
            tc_wait_ld();
            if ((h + 1) * 32 >= d) {                       // last read of the accumulator: hand it back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(&bars.a2_free[t]);
            }
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              if (h * 32 + k * 16 < d) {
                const int c16 = h * 2 + k;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                  const float4 g0 = vg[c16 * 4 + q * 2], g1 = vg[c16 * 4 + q * 2 + 1];
                  const float4 e0 = vbeta[c16 * 4 + q * 2], e1 = vbeta[c16 * 4 + q * 2 + 1];
                  const float2 gg[4] = {make_float2(g0.x, g0.y), make_float2(g0.z, g0.w), make_float2(g1.x, g1.y),
                                        make_float2(g1.z, g1.w)};
                  const float2 be[4] = {make_float2(e0.x, e0.y), make_float2(e0.z, e0.w), make_float2(e1.x, e1.y),
                                        make_float2(e1.z, e1.w)};
                  uint32_t o[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    const float2 y = make_float2(__uint_as_float(v[k][q * 8 + 2 * e]), __uint_as_float(v[k][q * 8 + 2 * e + 1]));
                    const float2 r2 = __ffma2_rn(__ffma2_rn(y, rstd2, shift2), gg[e], be[e]);
                    o[e] = pack_bf16x2(r2.x, r2.y);
                  }
                  *reinterpret_cast<uint4*>(o_row + slot_of(c16 * 2 + q)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
              }
            }
          }
        }
        __syncwarp();
        // coalesced write-back: cpr consecutive lanes write one row, 32 / cpr rows per instruction
        {
          const int rr0 = lane / cpr, cc = lane - rr0 * cpr;
#pragma unroll 4
          for (int base = 0; base < 32; base += rows_per) {
            const int rr = base + rr0;
            const int g_row = __shfl_sync(0xffffffffu, grow, rr & 31);
            if (rr0 < rows_per && rr < 32 && g_row >= 0) {
              const uint4 val = *reinterpret_cast<const uint4*>(
                  x_warp + (size_t)rr * (d * 2) + ((swz ? cc ^ (rr & (cpr - 1)) : cc) << 4));
              *reinterpret_cast<uint4*>(P.H + (size_t)g_row * d + cc * 8) = val;
            }
          }
        }
        __syncwarp();                                      // the slice is read: the pair after the next may be staged into it
        if (lane == 0) mbar_arrive(&bars.x_free[t]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kFfnTmemCols);
  if (tid == 0 && s_abort) report_status(P.status, LASER_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------- FP32-ALU kernel
template <typename T>
struct FfnSimtParams {
  int U, N, L, Lp, S, d, hid, maxC;
  float eps;
  T* H;
  const T *W1, *b1, *W2, *b2, *g, *beta;
  const int *lengths, *cand_offsets;
  int* prefix;
  int* counters;
  int* status;
};

template <typename T>
__global__ void __launch_bounds__(1024) ffn_simt_prep_kernel(FfnSimtParams<T> P) {
  chain_wait();
  chain_release();
  scan_rows(P, P.status);
}

template <typename T>
__global__ void __launch_bounds__(256) ffn_simt_kernel(FfnSimtParams<T> P) {
  extern __shared__ __align__(16) float sm[];
  const int d = P.d, hid = P.hid, tid = threadIdx.x;
  float* xs = sm;                      // [8][d]
  float* ys = xs + kSimtRows * d;      // [8][d]
  float* hs = ys + kSimtRows * d;      // [8][hid]
  __shared__ int s_row[kSimtRows];
  chain_wait();
  chain_release();
  const int total = P.counters[0];
  for (int base = blockIdx.x * kSimtRows; base < total; base += gridDim.x * kSimtRows) {
    __syncthreads();
    if (tid < kSimtRows) s_row[tid] = global_row(P, base + tid, total);
    __syncthreads();
    for (int i = tid; i < kSimtRows * d; i += blockDim.x) {
      const int r = i / d, k = i - r * d;
      xs[i] = s_row[r] >= 0 ? to_f32<T>(P.H[(size_t)s_row[r] * d + k]) : 0.f;
    }
    __syncthreads();
    for (int h = tid; h < hid; h += blockDim.x) {
      float acc[kSimtRows];
#pragma unroll
      for (int r = 0; r < kSimtRows; ++r) acc[r] = 0.f;
      for (int k = 0; k < d; ++k) {
        const float w = to_f32<T>(P.W1[(size_t)k * hid + h]);
#pragma unroll
        for (int r = 0; r < kSimtRows; ++r) acc[r] = fmaf(xs[r * d + k], w, acc[r]);
      }
      const float bb = to_f32<T>(P.b1[h]);
#pragma unroll
      for (int r = 0; r < kSimtRows; ++r) hs[r * hid + h] = fmaxf(acc[r] + bb, 0.f);
    }
    __syncthreads();
    for (int e = tid; e < d; e += blockDim.x) {
      float acc[kSimtRows];
#pragma unroll
      for (int r = 0; r < kSimtRows; ++r) acc[r] = 0.f;
      for (int j = 0; j < hid; ++j) {
        const float w = to_f32<T>(P.W2[(size_t)j * d + e]);
#pragma unroll
        for (int r = 0; r < kSimtRows; ++r) acc[r] = fmaf(hs[r * hid + j], w, acc[r]);
      }
      const float bb = to_f32<T>(P.b2[e]);
#pragma unroll
      for (int r = 0; r < kSimtRows; ++r) ys[r * d + e] = acc[r] + bb + xs[r * d + e];
    }
    __syncthreads();
    const int w = tid >> 5, lane = tid & 31;            // warp w normalises row w
    if (w < kSimtRows && s_row[w] >= 0) {
      float sum = 0.f;
      for (int e = lane; e < d; e += 32) sum += ys[w * d + e];
      for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float mean = sum / (float)d;
      float sq = 0.f;
      for (int e = lane; e < d; e += 32) sq += (ys[w * d + e] - mean) * (ys[w * d + e] - mean);
      for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      const float rstd = rsqrtf(sq / (float)d + P.eps);
      for (int e = lane; e < d; e += 32)
        P.H[(size_t)s_row[w] * d + e] =
            from_f32<T>((ys[w * d + e] - mean) * rstd * to_f32<T>(P.g[e]) + to_f32<T>(P.beta[e]));
    }
  }
}

int ffn_sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

size_t ffn_tc_smem(int d, int hid) {
  return (size_t)4 * kRows * d * 2 + (size_t)kWStages * kChunk * d * 2 + (size_t)3 * d * sizeof(float) + (size_t)hid * 2;
}

bool ffn_tc_supported(const Plan& p, int hid) {
  if (p.dtype != LASER_BF16) return false;
  if (p.d % 16 || p.d < 16 || p.d > 128) return false;
  if (hid % kChunk || hid < kChunk) return false;
  return ffn_tc_smem(p.d, hid) + 512 <= 227 * 1024;   // dynamic + static shared memory of one block
}

template <typename T>
int ffn_simt(const Plan& p, const laser_ffn_params* f, void* H, const int32_t* lengths, const int32_t* cand_offsets,
             char* ws, char* scratch, cudaStream_t st) {
  FfnSimtParams<T> P;
  P.U = p.U; P.N = p.N; P.L = p.L; P.Lp = p.Lp; P.S = p.S; P.d = p.d; P.hid = f->d_hidden; P.maxC = p.maxC;
  P.eps = f->ln_eps > 0.f ? f->ln_eps : 1e-5f;
  P.H = (T*)H;
  P.W1 = (const T*)f->W1; P.b1 = (const T*)f->b1; P.W2 = (const T*)f->W2; P.b2 = (const T*)f->b2;
  P.g = (const T*)f->ln_gain; P.beta = (const T*)f->ln_shift;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.counters = (int*)scratch;
  P.prefix = (int*)(scratch + kAlign);
  P.status = (int*)(ws + p.off_status);
  const size_t smem = ((size_t)2 * kSimtRows * p.d + (size_t)kSimtRows * f->d_hidden) * sizeof(float);
  if (smem > 200 * 1024) return LASER_ERR_UNSUPPORTED;
  {
    LaunchScope ls("ffn_prep", st);
    LASER_CUDA_OK(launch_chained(ffn_simt_prep_kernel<T>, dim3(1), dim3(1024), 0, st, P));
  }
  {
    LASER_CUDA_OK(cudaFuncSetAttribute(ffn_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const long long blocks_needed = ((long long)p.N * p.Lp + kSimtRows - 1) / kSimtRows;
    const int grid = (int)(blocks_needed < 8LL * ffn_sm_count() ? (blocks_needed > 0 ? blocks_needed : 1) : 8LL * ffn_sm_count());
    LaunchScope ls("ffn_simt", st);
    LASER_CUDA_OK(launch_chained(ffn_simt_kernel<T>, dim3(grid), dim3(256), smem, st, P));
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace

size_t ffn_scratch_bytes(const Plan& p, int hid) {
  return kAlign + align_up(((size_t)p.U + 1) * sizeof(int)) + 2 * align_up((size_t)p.d * hid * 2) +
         align_up((size_t)3 * p.d * sizeof(float)) + align_up((size_t)p.N * p.Lp * sizeof(int));
}

bool ffn_supported(const Plan& p, int hid) {
  if (hid < 1) return false;
  if ((long long)p.N * p.Lp >= (1ll << 31) - kPairRows) return false;
  if (ffn_tc_supported(p, hid) && p.path != LASER_PATH_SIMT) return true;
  if ((p.d * p.esize) % 16) return false;
  return ((size_t)2 * kSimtRows * p.d + (size_t)kSimtRows * hid) * sizeof(float) <= 200 * 1024;
}

int ffn_forward(const Plan& p, const laser_ffn_params* f, void* H, const int32_t* lengths, const int32_t* cand_offsets,
                char* ws, char* scratch, cudaStream_t st) {
  if (p.N == 0 || p.U == 0) return LASER_OK;
  const int hid = f->d_hidden;
  if (!ffn_supported(p, hid)) return LASER_ERR_UNSUPPORTED;
  if (!(ffn_tc_supported(p, hid) && p.path != LASER_PATH_SIMT)) {
    if (p.dtype == LASER_F32) return ffn_simt<float>(p, f, H, lengths, cand_offsets, ws, scratch, st);
    return ffn_simt<bf16>(p, f, H, lengths, cand_offsets, ws, scratch, st);
  }
  FfnParams P;
  P.U = p.U; P.N = p.N; P.L = p.L; P.Lp = p.Lp; P.S = p.S; P.d = p.d; P.hid = hid; P.NJ = hid / kChunk; P.maxC = p.maxC;
  P.eps = f->ln_eps > 0.f ? f->ln_eps : 1e-5f;
  P.H = (bf16*)H;
  P.W1 = (const bf16*)f->W1; P.b1 = (const bf16*)f->b1; P.W2 = (const bf16*)f->W2; P.b2 = (const bf16*)f->b2;
  P.g = (const bf16*)f->ln_gain; P.beta = (const bf16*)f->ln_shift;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.counters = (int*)scratch;
  P.prefix = (int*)(scratch + kAlign);
  P.img1 = (bf16*)(scratch + kAlign + align_up(((size_t)p.U + 1) * sizeof(int)));
  P.img2 = (bf16*)((char*)P.img1 + align_up((size_t)p.d * hid * 2));
  P.lnv = (float*)((char*)P.img2 + align_up((size_t)p.d * hid * 2));
  P.rowmap = (int*)((char*)P.lnv + align_up((size_t)3 * p.d * sizeof(float)));
  P.status = (int*)(ws + p.off_status);
  {
    LaunchScope ls("ffn_prep", st);
    LASER_CUDA_OK(launch_chained(ffn_prep_kernel, dim3(1 + 16), dim3(1024), 0, st, P, 1));
  }
  {
    const long long rows_max = (long long)p.N * p.Lp;
    const int grid = (int)(rows_max < 256LL * 4 * ffn_sm_count() ? (rows_max + 255) / 256 : 4 * ffn_sm_count());
    LaunchScope ls("ffn_map", st);
    LASER_CUDA_OK(launch_chained(ffn_map_kernel, dim3(grid > 0 ? grid : 1), dim3(256), 0, st, P));
  }
  {
    const size_t smem = ffn_tc_smem(p.d, hid);
    LASER_CUDA_OK(cudaFuncSetAttribute(ffn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const long long pairs_max = ((long long)p.N * p.Lp + kPairRows - 1) / kPairRows;
    const int sms = ffn_sm_count();
    const int grid = (int)(pairs_max < sms ? (pairs_max > 0 ? pairs_max : 1) : sms);
    LaunchScope ls("ffn_tc", st);
    LASER_CUDA_OK(launch_chained(ffn_tc_kernel, dim3(grid), dim3(kFfnThreads), smem, st, P));
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace laser
