// One-candidate-per-user path (bf16): a single pass over each user's raw item rows, bound by HBM bandwidth.
//
// With one target per user, materialising K = X W_k and V = X W_v (Eq. 9) would cost 2 d (d_qk + d) flops per
// 2 d-byte item row and make the pass compute bound.  Both projections are therefore folded out of the item loop
// (exact in real arithmetic):
//
//   gate      q_h . k_{n,h} / gamma = x_n . u_h          with  u_h = W_k[:, head h] (t W_q)_h / gamma   in R^d
//   segment   s_i[head h] = sum_n g_{n,h} (x_n W_v)[head h] = r_{i,h} W_v[:, head h]   with  r_{i,h} = sum_n g_{n,h} x_n
//
// so the item loop only needs the 2 H dot products x_n . u_h and the 2 H d multiply-adds of r += g x per row
// (Eq. 10-12), and W_v is applied once per segment afterwards.
//
//   stream_pre_kernel    u [U, H, d] (fp32) for every user (one warp per 16 users, two small warp-level MMA products
//                        with the intermediate query split into bf16 high and low parts), and the fragment-ordered
//                        image of W_v (spare warps)
//   stream_sta_kernel    one block per user; every warp owns whole segments, streams their rows through a private
//                        cp.async ring (16 rows per stage, 128-bit copies, padded rows) and feeds them twice to
//                        warp-level MMAs: scores = U X^T (rows = heads), then R += G X.  u, the gates and r are
//                        split into bf16 high and low parts that occupy MMA rows h and h + 8, so the fp32 values
//                        survive the bf16 operands to about 16 bits.  After the item loop the block multiplies all
//                        its segment sums by W_v (MMA, rows = segments) and writes H'.
//   GSTA                 the shared fused GSTA kernel (laser_gsta.cu) on that H'.
#include "laser_common.cuh"
#include "laser_gsta_img.cuh"
#include "laser_mma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
using namespace mma;

constexpr int kSW = 4;            // warps per block
constexpr int kSThreads = kSW * 32;
constexpr int kSRows = 16;        // item rows per stage (one MMA k / n step)
constexpr int kSStages = 4;       // ring depth per warp
constexpr int kPreWarps = 4;      // warps per block of the pre kernel; a warp folds 16 users

struct StreamParams {
  int U, L, d, dqk, H, S, Lp, N;
  float inv_gamma;
  const bf16 *items, *cands, *Wq, *Wk, *Wv;
  const int *lengths, *cand_offsets;
  const int* item_off;            // packed item layout: first row of every user ([U + 1]); null = padded [U, L, d]
  float* u;                       // [U, H, d]
  uint4* imgv;                    // W_v as MMA B fragments: [d/16 k-tiles][d/16 column pairs][32 lanes]
  bf16* Hp;                       // [N, Lp, d]
  int zero_empty;                 // write zero rows for segments without valid items
  const bf16* Wg;                 // GSTA weights whose images the pre kernel also builds (null: none)
  uint4* gimg;
  int* gnseg;                     // per-candidate segment counts for the GSTA kernel (built with the images)
  int M;
  int* order;                     // [U] users by descending length (null: blocks take the users in index order)
  int* order_keys;                // [U] scratch of the sort
  int* status;
};

// Candidate of user u, or -1 when it has none (or its offsets / length are invalid).
__device__ __forceinline__ int user_candidate(const StreamParams& P, int u, int* len_out) {
  const int c0 = P.cand_offsets[u], c1 = P.cand_offsets[u + 1], len = P.lengths[u];
  bool bad = c0 < 0 || c1 < c0 || c1 > P.N || c1 - c0 > 1 || len < 0 || len > P.L;
  if (!bad && P.item_off) bad = P.item_off[u] < 0 || P.item_off[u] > P.item_off[P.U] - len;
  if (bad) {
    report_status(P.status, LASER_ERR_BAD_INPUT);
    return -1;
  }
  *len_out = len;
  return c1 > c0 ? c0 : -1;
}

template <int D16>
__global__ void __launch_bounds__(kPreWarps * 32) stream_pre_kernel(StreamParams P, int user_warps) {
  constexpr int d = D16 * 16;
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wg = blockIdx.x * kPreWarps + (threadIdx.x >> 5);
  const int dqk = P.dqk, H = P.H, dqh = dqk / H;
  chain_wait();
  chain_release();
  if (P.order && blockIdx.x == gridDim.x - 1) {
    // the last block sorts the users by length, longest first: the attention kernel's grid runs in several waves of
    // blocks whose time is proportional to the user's length, and its last wave should be made of the shortest
    const float per_row = (float)(kGstaOrderBins - 1) / (float)P.L;
    sort_desc_by_key(P.U, [&](int u) { return (int)((float)min(max(P.lengths[u], 0), P.L) * per_row); }, P.order,
                     P.order_keys);
    return;
  }
  if (wg >= user_warps) {
    // spare warps: W_v image, entry (kt, p, lane) = {b0, b1 of column tile 2p, b0, b1 of column tile 2p+1},
    // B[k][n] = W_v[k][n]; and the GSTA weight images when GSTA follows
    const int worker = (wg - user_warps) * 32 + lane;
    const int n_workers = (((int)gridDim.x - (P.order ? 1 : 0)) * kPreWarps - user_warps) * 32;
    const int total = D16 * D16 * 32;
    const uint16_t* W = reinterpret_cast<const uint16_t*>(P.Wv);
    for (int i = worker; i < total; i += n_workers) {
      const int ln = i & 31, p = (i >> 5) % D16, kt = (i >> 5) / D16;
      const int gg = ln >> 2, tt = ln & 3;
      uint32_t v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int n = (2 * p + (q >> 1)) * 8 + gg, k = kt * 16 + 2 * tt + (q & 1) * 8;
        v[q] = (uint32_t)W[(size_t)k * d + n] | ((uint32_t)W[(size_t)(k + 1) * d + n] << 16);
      }
      P.imgv[i] = make_uint4(v[0], v[1], v[2], v[3]);
    }
    if (P.Wg) gsta_build_images(P.Wg, P.gimg, d, P.M, worker, n_workers);
    return;
  }
  // users 16 wg + g (MMA rows g) and 16 wg + g + 8 (rows g + 8); a user without a candidate is a zero row
  const int uA = wg * 16 + g, uB = uA + 8;
  int lenA = 0, lenB = 0;
  const int cA = uA < P.U ? user_candidate(P, uA, &lenA) : -1;
  const int cB = uB < P.U ? user_candidate(P, uB, &lenB) : -1;
  if (P.Wg && t == 0) {                                  // segment counts of these users' candidates for the GSTA kernel
    if (cA >= 0) P.gnseg[cA] = min((lenA + P.S - 1) / P.S, P.Lp);
    if (cB >= 0) P.gnseg[cB] = min((lenB + P.S - 1) / P.S, P.Lp);
  }
  uint32_t ta[D16][4];                                   // A fragments of T (bf16, exact)
#pragma unroll
  for (int kt = 0; kt < D16; ++kt) {
    const int k = kt * 16 + 2 * t;
    ta[kt][0] = cA >= 0 ? *reinterpret_cast<const uint32_t*>(P.cands + (size_t)cA * d + k) : 0u;
    ta[kt][1] = cB >= 0 ? *reinterpret_cast<const uint32_t*>(P.cands + (size_t)cB * d + k) : 0u;
    ta[kt][2] = cA >= 0 ? *reinterpret_cast<const uint32_t*>(P.cands + (size_t)cA * d + k + 8) : 0u;
    ta[kt][3] = cB >= 0 ? *reinterpret_cast<const uint32_t*>(P.cands + (size_t)cB * d + k + 8) : 0u;
  }
  const uint16_t* Wq = reinterpret_cast<const uint16_t*>(P.Wq);
  for (int h = 0; h < H; ++h) {
    float uacc[2 * D16][4];                              // u_h of the 16 users: (user g | g + 8, features 8 nt + 2t..)
#pragma unroll
    for (int nt = 0; nt < 2 * D16; ++nt) uacc[nt][0] = uacc[nt][1] = uacc[nt][2] = uacc[nt][3] = 0.f;
    for (int a0 = h * dqh; a0 < (h + 1) * dqh; a0 += 16) {
      // 16 columns of q = t W_q / gamma   (Eq. 4 / Eq. 8)
      float qc[2][4] = {};
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const uint16_t* w = Wq + (size_t)(kt * 16 + 2 * t) * dqk + a0 + nt * 8 + g;
          const uint32_t b0 = (uint32_t)w[0] | ((uint32_t)w[dqk] << 16);
          const uint32_t b1 = (uint32_t)w[8 * dqk] | ((uint32_t)w[9 * dqk] << 16);
          mma16816(qc[nt], ta[kt][0], ta[kt][1], ta[kt][2], ta[kt][3], b0, b1);
        }
      }
      // the accumulator layout of two 8-column tiles is the A layout of one 16-wide k-tile; high and low bf16 parts
      uint32_t qh[4], ql[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float x0 = qc[r >> 1][(r & 1) * 2] * P.inv_gamma, x1 = qc[r >> 1][(r & 1) * 2 + 1] * P.inv_gamma;
        qh[r] = pack2(x0, x1);
        ql[r] = pack2(x0 - bf16_lo(qh[r]), x1 - bf16_hi(qh[r]));
      }
      // u_h[i] += sum_{a in this chunk} W_k[i][a] q[a]: B[k = a][n = i] = W_k[i][a0 + k]
#pragma unroll
      for (int nt = 0; nt < 2 * D16; ++nt) {
        const bf16* w = P.Wk + (size_t)(nt * 8 + g) * dqk + a0 + 2 * t;
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(w), b1 = *reinterpret_cast<const uint32_t*>(w + 8);
        mma16816(uacc[nt], qh[0], qh[1], qh[2], qh[3], b0, b1);
        mma16816(uacc[nt], ql[0], ql[1], ql[2], ql[3], b0, b1);
      }
    }
#pragma unroll
    for (int nt = 0; nt < 2 * D16; ++nt) {
      if (uA < P.U) *reinterpret_cast<float2*>(P.u + ((size_t)uA * H + h) * d + nt * 8 + 2 * t) = make_float2(uacc[nt][0], uacc[nt][1]);
      if (uB < P.U) *reinterpret_cast<float2*>(P.u + ((size_t)uB * H + h) * d + nt * 8 + 2 * t) = make_float2(uacc[nt][2], uacc[nt][3]);
    }
  }
}

__device__ __forceinline__ float sigmoid_fast(float x) {
  // 1 / (1 + 2^(-x log2 e)) with the approximate ex2 and rcp units (relative error ~1e-7 each);
  // the exponential overflowing to +inf gives exactly 0
  float e, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.f + e));
  return r;
}

template <int D16>
__global__ void __launch_bounds__(kSThreads) stream_sta_kernel(StreamParams P) {
  constexpr int d = D16 * 16;
  constexpr int RS = 2 * d + 16;                 // bytes per staged row (the padding keeps ldmatrix conflict-free)
  extern __shared__ __align__(128) uint8_t smem[];
  const int H = P.H, dvh = d / H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  chain_wait();
  chain_release();
  const int u = P.order ? min(max(P.order[blockIdx.x], 0), P.U - 1) : (int)blockIdx.x;
  int len = 0;
  const int cand = user_candidate(P, u, &len);
  if (cand < 0) return;
  const int nv = (len + P.S - 1) / P.S;          // non-empty segments
  const int Lp16 = (P.Lp + 15) & ~15;
  uint8_t* Rhi = smem;                           // [Lp16][H] rows: bf16 high part of r_{i,h}
  uint8_t* Rlo = Rhi + (size_t)Lp16 * H * RS;    // same shape: bf16 low part
  uint8_t* ring = Rlo + (size_t)Lp16 * H * RS + (size_t)warp * kSStages * kSRows * RS;

  if (nv > 0) {
    // A fragments of U: row h = high part of u_h, row h + 8 = low part
    uint32_t ua[D16][4];
    {
      const float* up = P.u + ((size_t)u * H + g) * d;
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
        ua[kt][0] = ua[kt][1] = ua[kt][2] = ua[kt][3] = 0u;
        if (g < H) {
          const float2 x0 = *reinterpret_cast<const float2*>(up + kt * 16 + 2 * t);
          const float2 x1 = *reinterpret_cast<const float2*>(up + kt * 16 + 2 * t + 8);
          ua[kt][0] = pack2(x0.x, x0.y);
          ua[kt][1] = pack2(x0.x - bf16_lo(ua[kt][0]), x0.y - bf16_hi(ua[kt][0]));
          ua[kt][2] = pack2(x1.x, x1.y);
          ua[kt][3] = pack2(x1.x - bf16_lo(ua[kt][2]), x1.y - bf16_hi(ua[kt][2]));
        }
      }
    }
    const bf16* xu = P.items + (P.item_off ? (size_t)P.item_off[u] : (size_t)u * P.L) * d;

    // fetch cursor over this warp's (segment, 16-row group) sequence.  A stage is kSRows rows of 2 D16 16-byte
    // pieces; lane l copies pieces l, l + 32, ...: their row, source offset and destination offset never change.
    int f_seg = warp, f_grp = 0;
    bool f_valid = warp < nv;
    int p_row[D16], p_src[D16];
    uint32_t p_dst[D16];
#pragma unroll
    for (int i = 0; i < D16; ++i) {
      const int piece = i * 32 + lane;
      p_row[i] = piece / (2 * D16);
      const int q = piece - p_row[i] * (2 * D16);
      p_src[i] = p_row[i] * d + q * 8;
      p_dst[i] = p_row[i] * RS + q * 16;
    }
    const uint32_t ring_addr = smem_addr(ring);
    auto groups_of = [&](int seg) { return (min(P.S, len - seg * P.S) + kSRows - 1) / kSRows; };
    auto issue = [&](int stage) {
      const int n0 = f_seg * P.S + f_grp * kSRows;
      const int rows = min((f_seg + 1) * P.S, len) - n0;   // rows past the segment (or the valid prefix) become zeros
      const bf16* src = xu + (size_t)n0 * d;
      const uint32_t dst = ring_addr + stage * (kSRows * RS);
#pragma unroll
      for (int i = 0; i < D16; ++i) {
        const bool ok = p_row[i] < rows;
        cp16(dst + p_dst[i], ok ? (const void*)(src + p_src[i]) : (const void*)P.items, ok ? 16u : 0u);
      }
      if (++f_grp >= groups_of(f_seg)) {
        f_grp = 0;
        f_seg += kSW;
        if (f_seg >= nv) f_valid = false;
      }
    };
#pragma unroll
    for (int s = 0; s < kSStages - 1; ++s) {
      if (f_valid) issue(s);
      cp_commit();
    }

    int stage = 0;
    const uint32_t off1 = ((lane & 7) + ((lane >> 4) & 1) * 8) * RS + ((lane >> 3) & 1) * 16;   // [item][k] operand
    const uint32_t off2 = ((lane & 7) + ((lane >> 3) & 1) * 8) * RS + (lane >> 4) * 16;         // [item][col], transposed
    for (int seg = warp; seg < nv; seg += kSW) {
      float racc[2 * D16][4];
#pragma unroll
      for (int j = 0; j < 2 * D16; ++j) racc[j][0] = racc[j][1] = racc[j][2] = racc[j][3] = 0.f;
      const int ngrp = groups_of(seg);
      for (int grp = 0; grp < ngrp; ++grp) {
        cp_wait<kSStages - 2>();
        __syncwarp();
        if (f_valid) issue((stage + kSStages - 1) % kSStages);
        cp_commit();
        const uint32_t sb = ring_addr + stage * (kSRows * RS);
        // scores (Eq. 10 before the sigmoid): rows = heads (high / low parts), columns = the 16 items
        float sc[2][4] = {};
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) {
          uint32_t b[4];
          ldsm_x4(b, sb + off1 + kt * 32);
          mma16816(sc[0], ua[kt][0], ua[kt][1], ua[kt][2], ua[kt][3], b[0], b[1]);
          mma16816(sc[1], ua[kt][0], ua[kt][1], ua[kt][2], ua[kt][3], b[2], b[3]);
        }
        // gates; a zero row has score 0, gate 1/2 and contributes 1/2 * 0 = 0, so no mask is needed here
        uint32_t ga[4] = {0u, 0u, 0u, 0u};
        if (g < H) {
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const float g0 = sigmoid_fast(sc[nt][0] + sc[nt][2]), g1 = sigmoid_fast(sc[nt][1] + sc[nt][3]);
            ga[2 * nt] = pack2(g0, g1);
            ga[2 * nt + 1] = pack2(g0 - bf16_lo(ga[2 * nt]), g1 - bf16_hi(ga[2 * nt]));
          }
        }
        // r += G X  (Eq. 11-12 with the value projection postponed): rows = heads, k = items, columns = d
#pragma unroll
        for (int jp = 0; jp < D16; ++jp) {
          uint32_t b[4];
          ldsm_x4_t(b, sb + off2 + jp * 32);
          mma16816(racc[2 * jp], ga[0], ga[1], ga[2], ga[3], b[0], b[1]);
          mma16816(racc[2 * jp + 1], ga[0], ga[1], ga[2], ga[3], b[2], b[3]);
        }
        stage = (stage + 1) % kSStages;
      }
      if (g < H) {
#pragma unroll
        for (int j = 0; j < 2 * D16; ++j) {
          const float r0 = racc[j][0] + racc[j][2], r1 = racc[j][1] + racc[j][3];
          const uint32_t hi = pack2(r0, r1);
          const uint32_t lo = pack2(r0 - bf16_lo(hi), r1 - bf16_hi(hi));
          const size_t o = (size_t)(seg * H + g) * RS + (j * 8 + 2 * t) * 2;
          *reinterpret_cast<uint32_t*>(Rhi + o) = hi;
          *reinterpret_cast<uint32_t*>(Rlo + o) = lo;
        }
      }
    }
    cp_wait<0>();
  }
  __syncthreads();

  // s_i[head h] = r_{i,h} W_v[:, head h]: one unit = (16 segments, head)
  {
    const int NP = dvh >> 4;                      // 16-column pairs per head
    const int units = ((nv + 15) >> 4) * H;
    const uint32_t arow = (lane & 7) + ((lane >> 3) & 1) * 8, akc = lane >> 4;
    for (int unit = warp; unit < units; unit += kSW) {
      const int mt = unit / H, h = unit - mt * H;
      float acc[2 * D16][4];
#pragma unroll
      for (int j = 0; j < 2 * D16; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
        uint32_t ah[4], al[4];
        const size_t o = (size_t)((mt * 16 + arow) * H + h) * RS + (kt * 2 + akc) * 16;
        ldsm_x4(ah, smem_addr(Rhi + o));
        ldsm_x4(al, smem_addr(Rlo + o));
#pragma unroll
        for (int p = 0; p < D16; ++p) {
          if (p < NP) {
            const uint4 b = __ldg(P.imgv + (kt * D16 + h * NP + p) * 32 + lane);
            mma16816(acc[2 * p], ah[0], ah[1], ah[2], ah[3], b.x, b.y);
            mma16816(acc[2 * p], al[0], al[1], al[2], al[3], b.x, b.y);
            mma16816(acc[2 * p + 1], ah[0], ah[1], ah[2], ah[3], b.z, b.w);
            mma16816(acc[2 * p + 1], al[0], al[1], al[2], al[3], b.z, b.w);
          }
        }
      }
      const int s0 = mt * 16 + g, s1 = s0 + 8;
#pragma unroll
      for (int j = 0; j < 2 * D16; ++j) {
        if (j < 2 * NP) {
          const int col = h * dvh + j * 8 + 2 * t;
          if (s0 < nv) *reinterpret_cast<uint32_t*>(P.Hp + ((size_t)cand * P.Lp + s0) * d + col) = pack2(acc[j][0], acc[j][1]);
          if (s1 < nv) *reinterpret_cast<uint32_t*>(P.Hp + ((size_t)cand * P.Lp + s1) * d + col) = pack2(acc[j][2], acc[j][3]);
        }
      }
    }
  }
  if (P.zero_empty) {
    const int vec = d / 8;
    for (int i = tid; i < (P.Lp - nv) * vec; i += kSThreads) {
      const int seg = nv + i / vec, q = i % vec;
      *reinterpret_cast<uint4*>(P.Hp + ((size_t)cand * P.Lp + seg) * d + q * 8) = make_uint4(0, 0, 0, 0);
    }
  }
}

size_t stream_smem_bytes(int d, int H, int Lp) {
  const size_t RS = 2 * (size_t)d + 16;
  const size_t Lp16 = ((size_t)Lp + 15) & ~(size_t)15;
  return 2 * Lp16 * H * RS + (size_t)kSW * kSStages * kSRows * RS;
}

template <int D16>
int launch_stream(const StreamParams& P, cudaStream_t st) {
  const size_t smem = stream_smem_bytes(P.d, P.H, P.Lp);
  LASER_CUDA_OK(cudaFuncSetAttribute(stream_sta_kernel<D16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("stream_sta", st);
  LASER_CUDA_OK(launch_chained(stream_sta_kernel<D16>, dim3(P.U), dim3(kSThreads), smem, st, P));
  return LASER_OK;
}

}  // namespace

bool stream_supported(const Plan& p) {
  if (p.dtype != LASER_BF16 || p.maxC > 1) return false;
  if (p.d % 16 || p.d < 16 || p.d > 128) return false;
  if (p.H > 8 || p.dvh % 16) return false;
  if (p.dqh % 16) return false;                    // the query fold works on 16-column chunks of a head
  if (!gsta_mma_supported(p)) return false;
  return stream_smem_bytes(p.d, p.H, p.Lp) <= 200 * 1024;
}

size_t stream_scratch_bytes(const Plan& p) {   // u, the W_v image, the launch order of the users and its sort keys
  return align_up((size_t)p.U * p.H * p.d * sizeof(float)) + align_up((size_t)p.d * p.d * 2) +
         align_up(2 * (size_t)p.U * sizeof(int));
}

// Sorting the users pays only when the attention grid runs in more than one wave (four blocks per SM).
static bool stream_wants_order(const Plan& p) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return p.U > 4 * sms;
}

int stream_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
               const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st,
               const void* Wg_images) {
  if (p.N == 0 || p.U == 0) return LASER_OK;
  StreamParams P;
  P.Wg = (const bf16*)Wg_images;
  P.gimg = reinterpret_cast<uint4*>(ws + p.off_gimg);
  P.gnseg = reinterpret_cast<int*>(ws + p.off_gimg + gsta_nseg_offset(p));
  P.M = p.M;
  P.U = p.U; P.L = p.L; P.d = p.d; P.dqk = p.dqk; P.H = p.H; P.S = p.S; P.Lp = p.Lp; P.N = p.N;
  P.inv_gamma = p.inv_gamma;
  P.items = (const bf16*)items; P.cands = (const bf16*)cands;
  P.Wq = (const bf16*)Wq; P.Wk = (const bf16*)Wk; P.Wv = (const bf16*)Wv;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.item_off = p.item_offsets;
  P.u = reinterpret_cast<float*>(ws + p.off_su);
  P.imgv = reinterpret_cast<uint4*>(ws + p.off_su + align_up((size_t)p.U * p.H * p.d * sizeof(float)));
  P.Hp = (bf16*)Hprime;
  P.zero_empty = Hprime != (void*)(ws + p.off_hp);
  P.status = reinterpret_cast<int*>(ws + p.off_status);
  P.order = nullptr;
  P.order_keys = nullptr;
  if (stream_wants_order(p)) {
    P.order = reinterpret_cast<int*>(ws + p.off_su + align_up((size_t)p.U * p.H * p.d * sizeof(float)) +
                                     align_up((size_t)p.d * p.d * 2));
    P.order_keys = P.order + p.U;
  }
  {
    const int user_warps = (p.U + 15) / 16;
    const dim3 grid((user_warps + kPreWarps - 1) / kPreWarps + 2 + (P.order ? 1 : 0)), block(kPreWarps * 32);
    LaunchScope ls("stream_pre", st);
    cudaError_t e;
    switch (p.d / 16) {
      case 1: e = launch_chained(stream_pre_kernel<1>, grid, block, 0, st, P, user_warps); break;
      case 2: e = launch_chained(stream_pre_kernel<2>, grid, block, 0, st, P, user_warps); break;
      case 3: e = launch_chained(stream_pre_kernel<3>, grid, block, 0, st, P, user_warps); break;
      case 4: e = launch_chained(stream_pre_kernel<4>, grid, block, 0, st, P, user_warps); break;
      case 5: e = launch_chained(stream_pre_kernel<5>, grid, block, 0, st, P, user_warps); break;
      case 6: e = launch_chained(stream_pre_kernel<6>, grid, block, 0, st, P, user_warps); break;
      case 7: e = launch_chained(stream_pre_kernel<7>, grid, block, 0, st, P, user_warps); break;
      case 8: e = launch_chained(stream_pre_kernel<8>, grid, block, 0, st, P, user_warps); break;
      default: return LASER_ERR_UNSUPPORTED;
    }
    LASER_CUDA_OK(e);
  }
  int rc;
  switch (p.d / 16) {
    case 1: rc = launch_stream<1>(P, st); break;
    case 2: rc = launch_stream<2>(P, st); break;
    case 3: rc = launch_stream<3>(P, st); break;
    case 4: rc = launch_stream<4>(P, st); break;
    case 5: rc = launch_stream<5>(P, st); break;
    case 6: rc = launch_stream<6>(P, st); break;
    case 7: rc = launch_stream<7>(P, st); break;
    case 8: rc = launch_stream<8>(P, st); break;
    default: return LASER_ERR_UNSUPPORTED;
  }
  if (rc != LASER_OK) return rc;
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace laser
