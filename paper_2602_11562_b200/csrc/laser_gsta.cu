// Fused GSTA kernel (Eq. 7 and the residual update t_l = t_{l-1} + o_l) for bf16 inputs.
//
// One block owns 16 consecutive candidates (the 16 rows of every warp-level MMA) and runs all M layers for them:
//
//   A   Q   = T W_q^l                              [16 x d]    batched over the 16 candidates
//   B   Qt_h = Q[:, head h] W_k^l[:, head h]^T / tau  [16 x d] per head: (s_j W_k)_h . q_h = s_j . Qt_h
//   C   per candidate: scores e_{j,h} = s_j . Qt_h over its non-empty segments j, softmax over j, m_h = sum_j a_{j,h} s_j.
//       A candidate's segment vectors are staged in shared memory 16 at a time (cp.async, two buffers per warp, padded
//       rows); every vector is read from global memory once per layer and feeds both contractions as the 16-row MMA
//       operand: scores = S Qt^T (rows = segments, columns =
//       heads) and m^T = S^T P (rows = features), with an online softmax across chunks.
//   D   o[:, head h] = m_h W_v^l[:, head h];  T += o
//
// This is Eq. 7 re-associated (exact in real arithmetic): the key / value projections are applied to the query and to
// the attention-weighted sum instead of to every segment vector, which cuts the cost per candidate and layer from
// 4 L' d^2 to 6 d^2 + 4 H L' d flops.  Operands of every MMA are bf16, accumulators and the running target T are fp32.
// The weights reach the MMAs as B fragments straight from a fragment-ordered image in global memory (built once per
// call by gsta_prep_kernel), so they need no shared memory.
#include "laser_common.cuh"
#include "laser_gsta_img.cuh"
#include "laser_mma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
using namespace mma;

constexpr int kGT = 16;        // candidates per block
constexpr int kGW = 8;         // warps per block: two candidates per warp
constexpr int kGThreads = kGW * 32;
constexpr int kChunk = 16;     // segment vectors per staged chunk (one MMA k-step)

struct GstaParams {
  int N, U, L, S, Lp, H, M, d;
  float inv_tau;
  const bf16 *Hp, *cands, *Wg;
  const int *lengths, *cand_offsets;
  uint4* img;                  // [M][3][d/16 k-tiles][d/16 column pairs][32 lanes]
  int* nseg;                   // [N] non-empty segments per candidate (built with the images)
  int cpb;                     // candidates per block: 16, or 8 (one per warp) when that still fits one wave of blocks
  int* order;                  // [blocks] launch order, longest first (null: blocks run in candidate order)
  int* order_keys;             // [blocks] scratch of the sort that builds `order`
  int build_order;             // the set-up kernel's last block builds `order`
  int early_setup;             // images, counts and order come from a kernel at least two launches back (see the kernel)
  bf16* z;
  int* status;
};

__global__ void __launch_bounds__(256) gsta_prep_kernel(GstaParams P) {
  chain_wait();
  chain_release();
  const int n_blocks = gridDim.x - (P.build_order ? 1 : 0);          // blocks that build images and segment counts
  if ((int)blockIdx.x == n_blocks) {
    gsta_build_order(P.lengths, P.cand_offsets, P.U, P.N, P.L, P.S, P.Lp, P.cpb, P.order, P.order_keys);
    return;
  }
  gsta_build_images(P.Wg, P.img, P.d, P.M, blockIdx.x * blockDim.x + threadIdx.x, n_blocks * blockDim.x);
  gsta_build_nseg(P.lengths, P.cand_offsets, P.U, P.N, P.L, P.S, P.Lp, P.status, P.nseg,
                  (blockIdx.x * blockDim.x + threadIdx.x) >> 5, (n_blocks * blockDim.x) >> 5, threadIdx.x & 31);
}

// BPS = blocks per SM the registers are budgeted for: two (127 registers), or three at d <= 64 (80 registers, ~57 KB of
// shared memory per block) for grids of several waves, where the kernel is latency-bound and a third block's warps fill
// issue slots (cfg4 49.5 -> 47.6 us); a grid of one wave keeps the two-block budget, whose code has the shorter
// dependency chains.
template <int D16, int BPS>
__global__ void __launch_bounds__(kGThreads, BPS) gsta_mma_kernel(GstaParams P) {
  constexpr int d = D16 * 16;
  constexpr int RS = 2 * d + 16;            // bytes per staged bf16 row (16 bytes of padding: conflict-free ldmatrix)
  constexpr int TS = d + 8;                 // floats per row of the running target
  extern __shared__ __align__(128) uint8_t smem[];
  const int H = P.H, dvh = d / H, KH = dvh >> 4;
  float* Ts = reinterpret_cast<float*>(smem);                       // [16][TS]
  uint8_t* Qs = smem + kGT * TS * 4;                                // [16] rows: Q (bf16)
  uint8_t* Qt = Qs + kGT * RS;                                      // [16][H] rows: Qt, later m
  uint8_t* zrow = Qt + kGT * H * RS;                                // one row of zeros
  int* nv_s = reinterpret_cast<int*>(zrow + RS);                    // [16] non-empty segments per candidate
  uint8_t* stage = reinterpret_cast<uint8_t*>(nv_s + kGT);          // [kGW][2][kChunk] rows

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  // The block's set-up reads the candidates (an input) and what the set-up kernel built.  After a full forward call that
  // kernel lies at least two launches back: every kernel of the chain waits for its predecessor before it lets its
  // successor start, so those results are complete whenever this block runs, and the set-up can overlap the tail of the
  // attention kernel in front of this one; only H' has to wait for it.  Called on its own, the set-up kernel is the direct
  // predecessor and the wait comes first.
  if (!P.early_setup) {
    chain_wait();
    chain_release();
  }
  // which 16 (or 8) candidates: in launch order when the set-up kernel sorted the blocks, else in candidate order
  const int blk = P.order ? min(max(P.order[blockIdx.x], 0), (int)gridDim.x - 1) : (int)blockIdx.x;
  const int c_base = blk * P.cpb;
  const int c_end = min(c_base + P.cpb, P.N);          // rows of the 16-row tile past this are empty

  // Dense phases (A, B, D): warp p < d / 16 owns the 16 output columns 16 p .. 16 p + 15.  Its weight fragments come
  // straight from L2; those of the next dense phase are requested before the block-wide barrier that precedes it, so the
  // round trip overlaps the barrier and the stores around it.
  static_assert(D16 <= kGW, "one column pair per warp");
  const bool dense = warp < D16;
  uint4 wpre[D16];
  if (dense && P.M > 0) {
#pragma unroll
    for (int kt = 0; kt < D16; ++kt) wpre[kt] = __ldg(P.img + (kt * D16 + warp) * 32 + lane);
  }

  // ---- set-up: number of non-empty segments per candidate (from the set-up kernel's map); T = candidates; zero row
  if (tid < kGT) nv_s[tid] = (P.M > 0 && c_base + tid < c_end) ? min(max(P.nseg[c_base + tid], 0), P.Lp) : 0;
  for (int i = tid; i < kGT * (d / 8); i += kGThreads) {     // 8 features (16 bytes) at a time
    const int r = i / (d / 8), c8 = (i - r * (d / 8)) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (c_base + r < c_end) v = *reinterpret_cast<const uint4*>(P.cands + (size_t)(c_base + r) * d + c8);
    float* dst = Ts + r * TS + c8;
    dst[0] = bf16_lo(v.x); dst[1] = bf16_hi(v.x); dst[2] = bf16_lo(v.y); dst[3] = bf16_hi(v.y);
    dst[4] = bf16_lo(v.z); dst[5] = bf16_hi(v.z); dst[6] = bf16_lo(v.w); dst[7] = bf16_hi(v.w);
  }
  for (int i = tid; i < RS / 4; i += kGThreads) reinterpret_cast<uint32_t*>(zrow)[i] = 0u;
  __syncthreads();

  // ---- this warp's two candidates (slots): candidate warp + kGW s; two staging buffers of kChunk rows.
  // A chunk is kChunk rows of 2 D16 16-byte pieces; lane l copies pieces l, l + 32, ...
  static_assert(kGT == 2 * kGW, "two candidates per warp");
  static_assert((kChunk * 2 * D16) % 32 == 0, "a chunk is a whole number of 16-byte pieces per lane");
  constexpr int kPieces = kChunk * 2 * D16 / 32;
  uint8_t* my_stage = stage + (size_t)warp * 2 * kChunk * RS;
  const uint32_t stage_addr = smem_addr(my_stage);
  int p_row[kPieces], p_src[kPieces];
  uint32_t p_dst[kPieces];
#pragma unroll
  for (int i = 0; i < kPieces; ++i) {
    const int piece = i * 32 + lane;
    p_row[i] = piece / (2 * D16);
    const int q = piece - p_row[i] * (2 * D16);
    p_src[i] = p_row[i] * d + q * 8;
    p_dst[i] = p_row[i] * RS + q * 16;
  }
  // fetch cursor over (layer, slot, chunk) in processing order; the two buffers alternate
  int nv2[2];
#pragma unroll
  for (int sl = 0; sl < 2; ++sl) nv2[sl] = nv_s[warp + kGW * sl];
  const int first_sl = nv2[0] > 0 ? 0 : (nv2[1] > 0 ? 1 : -1);
  int f_layer = 0, f_sl = first_sl, f_ch = 0;
  bool f_valid = first_sl >= 0 && P.M > 0;
  auto issue = [&](int buf) {   // stage chunk (f_sl, f_ch) into buffer `buf`, then step the cursor
    const int nv = f_sl ? nv2[1] : nv2[0];
    const bf16* src = P.Hp + ((size_t)(c_base + warp + kGW * f_sl) * P.Lp + f_ch * kChunk) * d;
    const uint32_t dst = stage_addr + buf * (kChunk * RS);
    const int rows = nv - f_ch * kChunk;               // rows past the candidate's segments become zeros
#pragma unroll
    for (int i = 0; i < kPieces; ++i) {
      const bool ok = p_row[i] < rows;
      cp16(dst + p_dst[i], ok ? (const void*)(src + p_src[i]) : (const void*)P.Hp, ok ? 16u : 0u);
    }
    if (++f_ch * kChunk >= nv) {
      f_ch = 0;
      if (f_sl == 0 && nv2[1] > 0) f_sl = 1;
      else {
        f_sl = first_sl;
        if (++f_layer >= P.M) f_valid = false;
      }
    }
  };
  int buf = 0;
  if (P.early_setup) {
    chain_wait();
    chain_release();
  }
  if (f_valid) issue(0);
  cp_commit();

  const uint32_t ldsm_row = (lane & 7) + ((lane >> 3) & 1) * 8;   // row supplied by this lane (A-operand order)
  const uint32_t ldsm_kc = lane >> 4;                             // 16-byte k-chunk supplied by this lane

  for (int l = 0; l < P.M; ++l) {
    const uint4* imgk = P.img + (size_t)(l * 3 + 1) * D16 * D16 * 32;
    const uint4* imgv = P.img + (size_t)(l * 3 + 2) * D16 * D16 * 32;

    // ---------------------------------------------------------------- A: Q = T W_q
    {
      uint32_t ta[D16][4];
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
        const float2 x0 = *reinterpret_cast<const float2*>(Ts + g * TS + kt * 16 + 2 * t);
        const float2 x1 = *reinterpret_cast<const float2*>(Ts + (g + 8) * TS + kt * 16 + 2 * t);
        const float2 x2 = *reinterpret_cast<const float2*>(Ts + g * TS + kt * 16 + 2 * t + 8);
        const float2 x3 = *reinterpret_cast<const float2*>(Ts + (g + 8) * TS + kt * 16 + 2 * t + 8);
        ta[kt][0] = pack2(x0.x, x0.y);
        ta[kt][1] = pack2(x1.x, x1.y);
        ta[kt][2] = pack2(x2.x, x2.y);
        ta[kt][3] = pack2(x3.x, x3.y);
      }
      if (dense) {
        const int p = warp;
        float acc[2][4] = {};
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) {
          mma16816(acc[0], ta[kt][0], ta[kt][1], ta[kt][2], ta[kt][3], wpre[kt].x, wpre[kt].y);
          mma16816(acc[1], ta[kt][0], ta[kt][1], ta[kt][2], ta[kt][3], wpre[kt].z, wpre[kt].w);
        }
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) wpre[kt] = __ldg(imgk + (kt * D16 + p) * 32 + lane);   // for phase B
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int col = p * 16 + nt * 8 + 2 * t;
          *reinterpret_cast<uint32_t*>(Qs + g * RS + col * 2) = pack2(acc[nt][0], acc[nt][1]);
          *reinterpret_cast<uint32_t*>(Qs + (g + 8) * RS + col * 2) = pack2(acc[nt][2], acc[nt][3]);
        }
      }
    }
    __syncthreads();

    // ---------------------------------------------------------------- B: Qt_h = Q[:, head h] W_k[:, head h]^T / tau
    {
      uint32_t qa[D16][4];
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) ldsm_x4(qa[kt], smem_addr(Qs + ldsm_row * RS + (kt * 2 + ldsm_kc) * 16));
      if (dense) {
        const int p = warp;
        float acc[2][4] = {};
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) {
          const uint4 b = wpre[kt];
          mma16816(acc[0], qa[kt][0], qa[kt][1], qa[kt][2], qa[kt][3], b.x, b.y);
          mma16816(acc[1], qa[kt][0], qa[kt][1], qa[kt][2], qa[kt][3], b.z, b.w);
          if ((kt + 1) % KH == 0) {   // last k-tile of head h: store its Qt columns and start the next head
            const int h = kt / KH;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              const int col = p * 16 + nt * 8 + 2 * t;
              *reinterpret_cast<uint32_t*>(Qt + (g * H + h) * RS + col * 2) =
                  pack2(acc[nt][0] * P.inv_tau, acc[nt][1] * P.inv_tau);
              *reinterpret_cast<uint32_t*>(Qt + ((g + 8) * H + h) * RS + col * 2) =
                  pack2(acc[nt][2] * P.inv_tau, acc[nt][3] * P.inv_tau);
              acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
            }
          }
        }
      }
    }
    __syncthreads();

    // ---------------------------------------------------------------- C: per candidate, online softmax over chunks
    {
      const uint32_t a_off = ((lane & 7) + ((lane >> 3) & 1) * 8) * RS + (lane >> 4) * 16;     // S as [segment][k]
      const uint32_t t_off = ((lane & 7) + (lane >> 4) * 8) * RS + ((lane >> 3) & 1) * 16;     // S^T: [feature][segment]
#pragma unroll 1
      for (int sl = 0; sl < 2; ++sl) {
        const int c = warp + kGW * sl;
        const int nv = sl ? nv2[1] : nv2[0];
        float macc[D16][4];           // m^T tiles: (feature 16 jt + g | + 8, heads 2t, 2t+1)
#pragma unroll
        for (int jt = 0; jt < D16; ++jt) macc[jt][0] = macc[jt][1] = macc[jt][2] = macc[jt][3] = 0.f;
        float rm0 = -INFINITY, rm1 = -INFINITY, rs0 = 0.f, rs1 = 0.f;
        // B fragments of Qt^T: rows = heads of the candidate's Qt block (rows >= H read the zero row)
        uint32_t qb[D16][2];
        {
          const int h = lane & 7;
          const uint8_t* qrow = (h < H ? Qt + (c * H + h) * RS : zrow) + ((lane >> 3) & 1) * 16;
#pragma unroll
          for (int kt = 0; kt < D16; ++kt) ldsm_x2(qb[kt], smem_addr(qrow + kt * 32));
        }
        const int nch = (nv + kChunk - 1) / kChunk;
        for (int ch = 0; ch < nch; ++ch) {
          if (f_valid) issue(buf ^ 1);
          cp_commit();
          cp_wait<1>();
          __syncwarp();
          const uint32_t sb = stage_addr + buf * (kChunk * RS);
          const int rows = nv - ch * kChunk;
          float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f};   // even / odd k-tiles: two MMA chains
#pragma unroll
          for (int kt = 0; kt < D16; ++kt) {
            uint32_t a[4];
            ldsm_x4(a, sb + a_off + kt * 32);
            if (kt & 1) mma16816(e1, a[0], a[1], a[2], a[3], qb[kt][0], qb[kt][1]);
            else mma16816(e0, a[0], a[1], a[2], a[3], qb[kt][0], qb[kt][1]);
          }
          float c0 = e0[0] + e1[0], c1 = e0[1] + e1[1], c2 = e0[2] + e1[2], c3 = e0[3] + e1[3];
          if (g >= rows) c0 = c1 = -INFINITY;
          if (g + 8 >= rows) c2 = c3 = -INFINITY;
          // the chunk holds at least one valid segment, so both maxima are finite
          const float nm0 = fmaxf(rm0, group_max(fmaxf(c0, c2))), nm1 = fmaxf(rm1, group_max(fmaxf(c1, c3)));
          const float sc0 = __expf(rm0 - nm0), sc1 = __expf(rm1 - nm1);
          rm0 = nm0;
          rm1 = nm1;
          const uint32_t plo = pack2(__expf(c0 - nm0), __expf(c1 - nm1));
          const uint32_t phi = pack2(__expf(c2 - nm0), __expf(c3 - nm1));
          // normalise by exactly the weights the MMA uses (this lane's share; summed over the lane groups at the end)
          rs0 = rs0 * sc0 + bf16_lo(plo) + bf16_lo(phi);
          rs1 = rs1 * sc1 + bf16_hi(plo) + bf16_hi(phi);
          const uint32_t pb0 = movmatrix_t(plo), pb1 = movmatrix_t(phi);   // (segments 2t, 2t+1 | + 8, head g)
#pragma unroll
          for (int jt = 0; jt < D16; ++jt) {
            uint32_t a[4];
            ldsm_x4_t(a, sb + t_off + jt * 32);
            if (ch > 0) {                       // (the first chunk starts from zero)
              macc[jt][0] *= sc0; macc[jt][1] *= sc1;
              macc[jt][2] *= sc0; macc[jt][3] *= sc1;
            }
            mma16816(macc[jt], a[0], a[1], a[2], a[3], pb0, pb1);
          }
          __syncwarp();               // every lane is done with this buffer before the next iteration refills it
          buf ^= 1;
        }
        // m_h = (sum_j p_j s_j) / (sum_j p_j), stored as rows [head][feature] of the candidate's block
        const float s0 = group_sum(rs0), s1 = group_sum(rs1);
        const float i0 = s0 > 0.f ? 1.f / s0 : 0.f, i1 = s1 > 0.f ? 1.f / s1 : 0.f;   // no segment: m = 0 (o_l = 0)
        uint8_t* dst = Qt + (c * H + g) * RS + 4 * t;
#pragma unroll
        for (int jt = 0; jt < D16; ++jt) {
          const uint32_t lo = movmatrix_t(pack2(macc[jt][0] * i0, macc[jt][1] * i1));   // (head g, features 16 jt + 2t..)
          const uint32_t hi = movmatrix_t(pack2(macc[jt][2] * i0, macc[jt][3] * i1));   // (head g, features 16 jt + 8 + 2t..)
          if (g < H) {
            *reinterpret_cast<uint32_t*>(dst + jt * 32) = lo;
            *reinterpret_cast<uint32_t*>(dst + jt * 32 + 16) = hi;
          }
        }
      }
    }
    __syncthreads();

    // ---------------------------------------------------------------- D: o[:, head h] = m_h W_v[:, head h];  T += o
    if (dense) {
      const int p = warp;
      const int h = (p * 16) / dvh;
      float acc[2][4] = {};
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) wpre[kt] = __ldg(imgv + (kt * D16 + p) * 32 + lane);
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
        uint32_t a[4];
        ldsm_x4(a, smem_addr(Qt + ((int)ldsm_row * H + h) * RS + (kt * 2 + ldsm_kc) * 16));
        mma16816(acc[0], a[0], a[1], a[2], a[3], wpre[kt].x, wpre[kt].y);
        mma16816(acc[1], a[0], a[1], a[2], a[3], wpre[kt].z, wpre[kt].w);
      }
      if (l + 1 < P.M) {                                   // next layer's W_q fragments for its phase A
        const uint4* nq = P.img + (size_t)((l + 1) * 3) * D16 * D16 * 32;
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) wpre[kt] = __ldg(nq + (kt * D16 + p) * 32 + lane);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int col = p * 16 + nt * 8 + 2 * t;
        float2* r0 = reinterpret_cast<float2*>(Ts + g * TS + col);
        float2* r1 = reinterpret_cast<float2*>(Ts + (g + 8) * TS + col);
        float2 v0 = *r0, v1 = *r1;
        v0.x += acc[nt][0]; v0.y += acc[nt][1];
        v1.x += acc[nt][2]; v1.y += acc[nt][3];
        *r0 = v0;
        *r1 = v1;
      }
    }
    __syncthreads();
  }
  cp_wait<0>();

  for (int i = tid; i < kGT * (d / 2); i += kGThreads) {
    const int r = i / (d / 2), q = i - r * (d / 2);
    if (c_base + r < c_end) {
      const float2 v = *reinterpret_cast<const float2*>(Ts + r * TS + 2 * q);
      *reinterpret_cast<uint32_t*>(P.z + (size_t)(c_base + r) * d + 2 * q) = pack2(v.x, v.y);
    }
  }
}

template <int D16>
int launch_gsta(const GstaParams& P, cudaStream_t st) {
  constexpr int d = D16 * 16, RS = 2 * d + 16, TS = d + 8;
  const size_t smem = (size_t)kGT * TS * 4 + (size_t)kGT * RS + (size_t)kGT * P.H * RS + RS + kGT * sizeof(int) +
                      (size_t)kGW * 2 * kChunk * RS;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int blocks = (P.N + P.cpb - 1) / P.cpb;
  auto kernel = (D16 <= 4 && blocks > 2 * sms) ? gsta_mma_kernel<D16, (D16 <= 4 ? 3 : 2)> : gsta_mma_kernel<D16, 2>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("gsta_mma", st);
  LASER_CUDA_OK(launch_chained(kernel, dim3(blocks), dim3(kGThreads), smem, st, P));
  return LASER_OK;
}

}  // namespace

bool gsta_mma_supported(const Plan& p) {
  if (p.dtype != LASER_BF16) return false;
  if (p.d % 16 || p.d < 16 || p.d > 128) return false;
  if (p.H > 8 || p.dvh % 16) return false;
  return true;
}

size_t gsta_nseg_offset(const Plan& p) { return align_up((size_t)p.M * 3 * p.d * p.d * 2); }
size_t gsta_order_offset(const Plan& p) { return align_up(gsta_nseg_offset(p) + (size_t)p.N * sizeof(int)); }
size_t gsta_mma_image_bytes(const Plan& p) {       // the order table and its sort keys: one int each per block of >= 8
  return gsta_order_offset(p) + 2 * (size_t)((p.N + 7) / 8) * sizeof(int);
}

// Small batches: 8 candidates per block (every warp then has one candidate instead of two, which halves the
// per-candidate part of a block's latency) as long as all blocks still run at once.
int gsta_candidates_per_block(const Plan& p) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return (p.N + 7) / 8 <= 2 * sms ? 8 : kGT;
}

// Sorting the blocks pays only when the grid runs in more than one wave.
bool gsta_wants_order(const Plan& p) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int cpb = gsta_candidates_per_block(p);
  return p.M > 0 && (p.N + cpb - 1) / cpb > 2 * sms;
}

int gsta_mma(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets, const void* cands,
             const void* Wg, void* z, char* ws, cudaStream_t st, bool images_ready) {
  if (p.N == 0) return LASER_OK;
  GstaParams P;
  P.N = p.N; P.U = p.U; P.L = p.L; P.S = p.S; P.Lp = p.Lp; P.H = p.H; P.M = p.M; P.d = p.d;
  P.inv_tau = p.inv_tau;
  P.Hp = (const bf16*)Hprime; P.cands = (const bf16*)cands; P.Wg = (const bf16*)Wg;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.img = reinterpret_cast<uint4*>(ws + p.off_gimg);
  P.nseg = reinterpret_cast<int*>(ws + p.off_gimg + gsta_nseg_offset(p));
  P.z = (bf16*)z;
  P.status = reinterpret_cast<int*>(ws + p.off_status);
  P.cpb = gsta_candidates_per_block(p);
  // The block order exists when this call's own set-up kernel builds it, or when the tensor-core STA path's set-up
  // kernel built it beside the images; the one-candidate path builds none (its batches are one wave of blocks).
  const bool ordered = gsta_wants_order(p) && (!images_ready || p.path == LASER_PATH_TENSOR);
  int* order = reinterpret_cast<int*>(ws + p.off_gimg + gsta_order_offset(p));
  P.order = ordered ? order : nullptr;
  P.order_keys = order + (p.N + 7) / 8;
  P.build_order = ordered && !images_ready;
  P.early_setup = images_ready ? 1 : 0;
  if (p.M > 0 && !images_ready) {
    const int total = p.M * 3 * (p.d / 16) * (p.d / 16) * 32;
    LaunchScope ls("gsta_prep", st);
    LASER_CUDA_OK(launch_chained(gsta_prep_kernel, dim3((total + 255) / 256 + P.build_order), dim3(256), 0, st, P));
  }
  int rc;
  switch (p.d / 16) {
    case 1: rc = launch_gsta<1>(P, st); break;
    case 2: rc = launch_gsta<2>(P, st); break;
    case 3: rc = launch_gsta<3>(P, st); break;
    case 4: rc = launch_gsta<4>(P, st); break;
    case 5: rc = launch_gsta<5>(P, st); break;
    case 6: rc = launch_gsta<6>(P, st); break;
    case 7: rc = launch_gsta<7>(P, st); break;
    case 8: rc = launch_gsta<8>(P, st); break;
    default: return LASER_ERR_UNSUPPORTED;
  }
  if (rc != LASER_OK) return rc;
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace laser
