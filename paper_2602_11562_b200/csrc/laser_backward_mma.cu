// Tensor-core version of the backward pass through the segment aggregation and the sigmoid gates (Eq. 10-12), for bf16
// batches: the five contractions per (user, head, item tile, candidate tile) run as warp-level mma.sync m16n8k16 with bf16
// operands and fp32 accumulation.  Operands are bf16 copies of the fp32 intermediates of the recomputed forward (Q / gamma,
// K, V) and of the upstream gradient dH'; results (dK, dV, the query-side sums dQf) are fp32.
//
// With x = q_h . k_n / gamma, g = Sigmoid(x) = (1 + tanh(x / 2)) / 2 and g (1 - g) = (1 - tanh^2(x / 2)) / 4.  The bf16
// query copy holds Q / (2 gamma), so the score product gives x / 2 directly, and with th = tanh(x / 2), w = 1 - th^2:
//   dG^T[n, c]  = v_n . ds_i[c, h]                           (i = the segment of item n)
//   dV[n]      += sum_c g[n, c] ds_i[c, h]
//   dK[n]       = 1/2 sum_c (dG w)[n, c] Qb[c]               (Qb = Q / (2 gamma), de = dG w / 4, dK = sum de Q / gamma)
//   dQf[c]     += 1/4 sum_n (dG w)[n, c] k_n
//
// One warp = one job (segment i, item tile of 16 MT rows inside it, head h) of one user; it keeps the job's K_h / V_h tiles
// as A fragments and the dK / dV accumulators in registers and walks the user's candidates 16 at a time.  Everything is
// formed transposed (items on the MMA rows), so that the gates and the score gradients leave their MMA in the register
// layout the next one wants as its A operand; only the query-side product contracts over the items and takes its B operand
// through movmatrix.  The candidate rows of Qb and ds_i (bf16) are staged per warp in shared memory (cp.async, two
// buffers) and read with ldmatrix, plain for the products that contract over the head width, transposed for those that
// contract over the candidates.  Rows of the tile past the segment's end or the user's length are zero rows of K and V:
// they contribute nothing and are not written.  Candidate rows past the user's last are zero-filled: their score
// gradients vanish with ds.  dK and dV rows are written once, by their job; dQf is summed over the jobs with atomics
// (eight lanes per 32-byte sector).
#include "laser_common.cuh"
#include "laser_mma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
using namespace mma;

constexpr int kBwdWarps = 8;

// dst = bf16(scale * src), four elements per thread and step (n4 = number of groups of four; n is a multiple of 4:
// every array converted here has a row width that is a multiple of 16).
__global__ void __launch_bounds__(256) cast_bf16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, size_t n4,
                                                        float scale) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 v = src[i];
    dst[i] = make_uint2(pack2(v.x * scale, v.y * scale), pack2(v.z * scale, v.w * scale));
  }
}

__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct BwdMmaParams {
  const bf16 *Qb, *Kb, *Vb, *dSb;
  const int32_t *lengths, *cand_offsets;
  float *dQf, *dK, *dV;
  int L, d, dqk, H, S, Lp, N, R, jobs;           // R item tiles per segment, jobs = Lp R H per user
};

// (Budgeted for two blocks per SM: at 32-row tiles the kernel would take 165 registers and run one block of eight warps
// per SM; capped at 128 it spills a few words and runs 16 warps, which is faster: 211 against 268 us at U = 64, C = 256,
// L = 4096, d = 128.)
template <int MT, int DQ16, int DV16>
__global__ void __launch_bounds__(kBwdWarps * 32, 2) sta_bwd_mma_kernel(const BwdMmaParams P) {
  constexpr int DQH = 16 * DQ16, DVH = 16 * DV16;
  constexpr int QS = 2 * DQH + 16, DS = 2 * DVH + 16;          // bytes per staged row (padding: conflict-free ldmatrix)
  constexpr int kBuf = 16 * (QS + DS);                         // one staging buffer: 16 candidate rows of Qb_h and ds_i,h
  extern __shared__ __align__(16) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int u = blockIdx.y, job = blockIdx.x * kBwdWarps + warp;
  if (job >= P.jobs) return;
  const int h = job % P.H, r = (job / P.H) % P.R, seg = job / (P.H * P.R);
  const int len = P.lengths[u], off0 = P.cand_offsets[u], off1 = P.cand_offsets[u + 1];
  if (len <= 0 || len > P.L || off0 < 0 || off1 <= off0 || off1 > P.N) return;
  const int C = off1 - off0;
  const int n0 = seg * P.S + r * 16 * MT, n_end = min(min((seg + 1) * P.S, P.L), len);
  if (n0 >= n_end) return;
  const int cnt = min(16 * MT, n_end - n0);
  const int d = P.d, dqk = P.dqk;

  // ---- the job's K_h and V_h tiles as A fragments (rows = items), zero rows past cnt
  uint32_t Ka[MT][DQ16][4], Va[MT][DV16][4];
  {
    const bf16* Kr = P.Kb + ((size_t)u * P.L + n0) * dqk + h * DQH;
    const bf16* Vr = P.Vb + ((size_t)u * P.L + n0) * d + h * DVH;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int r0 = mt * 16 + g, r1 = r0 + 8;
#pragma unroll
      for (int k = 0; k < DQ16; ++k) {
        const int c = k * 16 + 2 * t;
        Ka[mt][k][0] = r0 < cnt ? *reinterpret_cast<const uint32_t*>(Kr + (size_t)r0 * dqk + c) : 0u;
        Ka[mt][k][1] = r1 < cnt ? *reinterpret_cast<const uint32_t*>(Kr + (size_t)r1 * dqk + c) : 0u;
        Ka[mt][k][2] = r0 < cnt ? *reinterpret_cast<const uint32_t*>(Kr + (size_t)r0 * dqk + c + 8) : 0u;
        Ka[mt][k][3] = r1 < cnt ? *reinterpret_cast<const uint32_t*>(Kr + (size_t)r1 * dqk + c + 8) : 0u;
      }
#pragma unroll
      for (int k = 0; k < DV16; ++k) {
        const int c = k * 16 + 2 * t;
        Va[mt][k][0] = r0 < cnt ? *reinterpret_cast<const uint32_t*>(Vr + (size_t)r0 * d + c) : 0u;
        Va[mt][k][1] = r1 < cnt ? *reinterpret_cast<const uint32_t*>(Vr + (size_t)r1 * d + c) : 0u;
        Va[mt][k][2] = r0 < cnt ? *reinterpret_cast<const uint32_t*>(Vr + (size_t)r0 * d + c + 8) : 0u;
        Va[mt][k][3] = r1 < cnt ? *reinterpret_cast<const uint32_t*>(Vr + (size_t)r1 * d + c + 8) : 0u;
      }
    }
  }
  // K_h^T as A fragments (rows = key components, k = items), from the fragments above: the transposed 8 x 8 blocks
  uint32_t Kt[DQ16][MT][4];
#pragma unroll
  for (int q = 0; q < DQ16; ++q)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      Kt[q][mt][0] = movmatrix_t(Ka[mt][q][0]);
      Kt[q][mt][1] = movmatrix_t(Ka[mt][q][2]);
      Kt[q][mt][2] = movmatrix_t(Ka[mt][q][1]);
      Kt[q][mt][3] = movmatrix_t(Ka[mt][q][3]);
    }

  float dKacc[MT][2 * DQ16][4], dVacc[MT][2 * DV16][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
    for (int j = 0; j < 2 * DQ16; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) dKacc[mt][j][e] = 0.f;
#pragma unroll
    for (int j = 0; j < 2 * DV16; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) dVacc[mt][j][e] = 0.f;
  }

  // ---- staging of 16 candidate rows: Qb[c, h] (DQH values) and ds_seg[c, h] (DVH values)
  const uint32_t stage0 = smem_addr(smem) + warp * 2 * kBuf;
  const bf16* Qg = P.Qb + (size_t)off0 * dqk + h * DQH;
  const bf16* Sg = P.dSb + ((size_t)off0 * P.Lp + seg) * d + h * DVH;
  const size_t s_row = (size_t)P.Lp * d;
  auto stage = [&](int c0, int buf) {
    const uint32_t base = stage0 + buf * kBuf;
#pragma unroll
    for (int k = 0; k < DQ16; ++k) {
      const int x = lane + 32 * k, row = x / (2 * DQ16), ch = x % (2 * DQ16);
      const int c = c0 + row;
      cp16(base + row * QS + ch * 16, Qg + (size_t)min(c, C - 1) * dqk + ch * 8, c < C ? 16u : 0u);
    }
#pragma unroll
    for (int k = 0; k < DV16; ++k) {
      const int x = lane + 32 * k, row = x / (2 * DV16), ch = x % (2 * DV16);
      const int c = c0 + row;
      cp16(base + 16 * QS + row * DS + ch * 16, Sg + (size_t)min(c, C - 1) * s_row + ch * 8, c < C ? 16u : 0u);
    }
    cp_commit();
  };
  // ldmatrix lane addresses inside a buffer.  Plain (B operand with k = head component, n = candidate): matrices
  // (cands 0-7, k 0-7), (cands 0-7, k 8-15), (cands 8-15, k 0-7), (cands 8-15, k 8-15) of a 16-component step.
  // Transposed (k = candidate, n = component): (cands 0-7, n 0-7), (cands 8-15, n 0-7), (cands 0-7, n 8-15), (cands 8-15, n 8-15).
  const int mi = lane >> 3, lr = lane & 7;
  const uint32_t q_plain = ((mi >> 1) * 8 + lr) * QS + (mi & 1) * 16;
  const uint32_t q_trans = ((mi & 1) * 8 + lr) * QS + (mi >> 1) * 16;
  const uint32_t s_plain = 16 * QS + ((mi >> 1) * 8 + lr) * DS + (mi & 1) * 16;
  const uint32_t s_trans = 16 * QS + ((mi & 1) * 8 + lr) * DS + (mi >> 1) * 16;

  float* dQg = P.dQf + (size_t)off0 * dqk + h * DQH;
  const int slabs = (C + 15) >> 4;
  stage(0, 0);
  for (int s = 0; s < slabs; ++s) {
    const int c0 = s * 16;
    if (s + 1 < slabs) {
      stage(c0 + 16, (s + 1) & 1);
      cp_wait<1>();
    } else {
      cp_wait<0>();
    }
    __syncwarp();
    const uint32_t base = stage0 + (s & 1) * kBuf;

    // scores^T / 2 and dG^T ([items] x [16 candidates]), one 16-item row tile at a time, then its gates and score
    // gradients packed as the A operands of the products that contract over the candidates
    uint32_t qb[DQ16][4], sb[DV16][4];
#pragma unroll
    for (int k = 0; k < DQ16; ++k) ldsm_x4(qb[k], base + q_plain + k * 32);
#pragma unroll
    for (int k = 0; k < DV16; ++k) ldsm_x4(sb[k], base + s_plain + k * 32);
    uint32_t gA[MT][4], eA[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float E[2][4], G[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) E[nt][e] = G[nt][e] = 0.f;
#pragma unroll
      for (int k = 0; k < DQ16; ++k) {
        mma16816(E[0], Ka[mt][k][0], Ka[mt][k][1], Ka[mt][k][2], Ka[mt][k][3], qb[k][0], qb[k][1]);
        mma16816(E[1], Ka[mt][k][0], Ka[mt][k][1], Ka[mt][k][2], Ka[mt][k][3], qb[k][2], qb[k][3]);
      }
#pragma unroll
      for (int k = 0; k < DV16; ++k) {
        mma16816(G[0], Va[mt][k][0], Va[mt][k][1], Va[mt][k][2], Va[mt][k][3], sb[k][0], sb[k][1]);
        mma16816(G[1], Va[mt][k][0], Va[mt][k][1], Va[mt][k][2], Va[mt][k][3], sb[k][2], sb[k][3]);
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float gg[4], ee[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float th = tanh_fast(E[nt][e]);
          gg[e] = fmaf(th, 0.5f, 0.5f);
          ee[e] = G[nt][e] * fmaf(-th, th, 1.f);
        }
        gA[mt][2 * nt] = pack2(gg[0], gg[1]);
        gA[mt][2 * nt + 1] = pack2(gg[2], gg[3]);
        eA[mt][2 * nt] = pack2(ee[0], ee[1]);
        eA[mt][2 * nt + 1] = pack2(ee[2], ee[3]);
      }
    }
    // dV += g^T ds,  dK += (dG w)^T Qb
#pragma unroll
    for (int k = 0; k < DV16; ++k) {
      uint32_t b[4];
      ldsm_x4_t(b, base + s_trans + k * 32);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        mma16816(dVacc[mt][2 * k], gA[mt][0], gA[mt][1], gA[mt][2], gA[mt][3], b[0], b[1]);
        mma16816(dVacc[mt][2 * k + 1], gA[mt][0], gA[mt][1], gA[mt][2], gA[mt][3], b[2], b[3]);
      }
    }
#pragma unroll
    for (int k = 0; k < DQ16; ++k) {
      uint32_t b[4];
      ldsm_x4_t(b, base + q_trans + k * 32);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        mma16816(dKacc[mt][2 * k], eA[mt][0], eA[mt][1], eA[mt][2], eA[mt][3], b[0], b[1]);
        mma16816(dKacc[mt][2 * k + 1], eA[mt][0], eA[mt][1], eA[mt][2], eA[mt][3], b[2], b[3]);
      }
    }
    // dQf^T [key components] x [candidates] = K_h^T (dG w)^T: the B operand is the transposed 8 x 8 blocks of eA
    float dQ[DQ16][2][4];
#pragma unroll
    for (int q = 0; q < DQ16; ++q)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) dQ[q][nt][e] = 0.f;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const uint32_t b0 = movmatrix_t(eA[mt][2 * nt]), b1 = movmatrix_t(eA[mt][2 * nt + 1]);
#pragma unroll
        for (int q = 0; q < DQ16; ++q) mma16816(dQ[q][nt], Kt[q][mt][0], Kt[q][mt][1], Kt[q][mt][2], Kt[q][mt][3], b0, b1);
      }
#pragma unroll
    for (int q = 0; q < DQ16; ++q)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int c = c0 + nt * 8 + 2 * t, kq = q * 16 + g;
        if (c < C) {
          atomicAdd(dQg + (size_t)c * dqk + kq, 0.25f * dQ[q][nt][0]);
          atomicAdd(dQg + (size_t)c * dqk + kq + 8, 0.25f * dQ[q][nt][2]);
        }
        if (c + 1 < C) {
          atomicAdd(dQg + (size_t)(c + 1) * dqk + kq, 0.25f * dQ[q][nt][1]);
          atomicAdd(dQg + (size_t)(c + 1) * dqk + kq + 8, 0.25f * dQ[q][nt][3]);
        }
      }
    __syncwarp();                        // every lane is done with this buffer before the next request overwrites it
  }

  // ---- this job's rows of dK and dV (valid rows only; the others keep the zeros the caller put there)
  float* dKr = P.dK + ((size_t)u * P.L + n0) * dqk + h * DQH;
  float* dVr = P.dV + ((size_t)u * P.L + n0) * d + h * DVH;
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int r0 = mt * 16 + g, r1 = r0 + 8;
#pragma unroll
    for (int j = 0; j < 2 * DQ16; ++j) {
      const int c = j * 8 + 2 * t;
      if (r0 < cnt) *reinterpret_cast<float2*>(dKr + (size_t)r0 * dqk + c) = make_float2(0.5f * dKacc[mt][j][0], 0.5f * dKacc[mt][j][1]);
      if (r1 < cnt) *reinterpret_cast<float2*>(dKr + (size_t)r1 * dqk + c) = make_float2(0.5f * dKacc[mt][j][2], 0.5f * dKacc[mt][j][3]);
    }
#pragma unroll
    for (int j = 0; j < 2 * DV16; ++j) {
      const int c = j * 8 + 2 * t;
      if (r0 < cnt) *reinterpret_cast<float2*>(dVr + (size_t)r0 * d + c) = make_float2(dVacc[mt][j][0], dVacc[mt][j][1]);
      if (r1 < cnt) *reinterpret_cast<float2*>(dVr + (size_t)r1 * d + c) = make_float2(dVacc[mt][j][2], dVacc[mt][j][3]);
    }
  }
}

// ---------------------------------------------------------------------------------------------------------------------
// The recomputed forward of the same step, H'[c, seg, h] = sum_n g[c, n] v_n (Eq. 10-12), with the same bf16 operands: one
// block per (user, segment, head) stages the segment's K_h and V_h rows in shared memory (zero rows up to a multiple of 16)
// and its warps take the user's candidates 16 at a time: scores = Qb K_h^T per 16 items, gates from the accumulator layout
// straight into the A operand of g V_h.  Output fp32 (what the GSTA backward reads).
struct FwdMmaParams {
  const bf16 *Qb, *Kb, *Vb;
  const int32_t *lengths, *cand_offsets;
  float* Hp;                                     // fp32 H' (null: not wanted)
  bf16* Hb;                                      // bf16 H' for the attention kernels below (null: not wanted)
  int L, d, dqk, H, S, Lp, N, rows;              // rows = staged rows per block (min(S, L) rounded up to 16)
};

template <int DQ16, int DV16>
__global__ void __launch_bounds__(kBwdWarps * 32) sta_fwd_mma_kernel(const FwdMmaParams P) {
  constexpr int DQH = 16 * DQ16, DVH = 16 * DV16;
  constexpr int KS = 2 * DQH + 16, VS = 2 * DVH + 16;          // bytes per staged row
  extern __shared__ __align__(16) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int u = blockIdx.y, seg = blockIdx.x / P.H, h = blockIdx.x - seg * P.H;
  const int len = P.lengths[u], off0 = P.cand_offsets[u], off1 = P.cand_offsets[u + 1];
  if (len <= 0 || len > P.L || off0 < 0 || off1 <= off0 || off1 > P.N) return;
  const int C = off1 - off0;
  const int n0 = seg * P.S, n_end = min(min((seg + 1) * P.S, P.L), len);
  if (n0 >= n_end) return;
  const int cnt = n_end - n0, chunks = (cnt + 15) >> 4, d = P.d, dqk = P.dqk;
  const uint32_t Ksm = smem_addr(smem), Vsm = Ksm + P.rows * KS;
  {
    const bf16* Kr = P.Kb + ((size_t)u * P.L + n0) * dqk + h * DQH;
    const bf16* Vr = P.Vb + ((size_t)u * P.L + n0) * d + h * DVH;
    for (int x = tid; x < chunks * 16 * 2 * DQ16; x += kBwdWarps * 32) {
      const int row = x / (2 * DQ16), ch = x - row * (2 * DQ16);
      cp16(Ksm + row * KS + ch * 16, Kr + (size_t)min(row, cnt - 1) * dqk + ch * 8, row < cnt ? 16u : 0u);
    }
    for (int x = tid; x < chunks * 16 * 2 * DV16; x += kBwdWarps * 32) {
      const int row = x / (2 * DV16), ch = x - row * (2 * DV16);
      cp16(Vsm + row * VS + ch * 16, Vr + (size_t)min(row, cnt - 1) * d + ch * 8, row < cnt ? 16u : 0u);
    }
    cp_commit();
    cp_wait<0>();
    __syncthreads();
  }
  const int mi = lane >> 3, lr = lane & 7;
  const uint32_t k_plain = Ksm + ((mi >> 1) * 8 + lr) * KS + (mi & 1) * 16;      // B(k = key component, n = item)
  const uint32_t v_trans = Vsm + ((mi & 1) * 8 + lr) * VS + (mi >> 1) * 16;      // B(k = item, n = value component)
  const bf16* Qg = P.Qb + (size_t)off0 * dqk + h * DQH;
  for (int c0 = warp * 16; c0 < C; c0 += kBwdWarps * 16) {
    uint32_t Qa[DQ16][4];
    const int r0 = c0 + g, r1 = r0 + 8;
#pragma unroll
    for (int k = 0; k < DQ16; ++k) {
      const int c = k * 16 + 2 * t;
      Qa[k][0] = r0 < C ? *reinterpret_cast<const uint32_t*>(Qg + (size_t)r0 * dqk + c) : 0u;
      Qa[k][1] = r1 < C ? *reinterpret_cast<const uint32_t*>(Qg + (size_t)r1 * dqk + c) : 0u;
      Qa[k][2] = r0 < C ? *reinterpret_cast<const uint32_t*>(Qg + (size_t)r0 * dqk + c + 8) : 0u;
      Qa[k][3] = r1 < C ? *reinterpret_cast<const uint32_t*>(Qg + (size_t)r1 * dqk + c + 8) : 0u;
    }
    float acc[2 * DV16][4];
#pragma unroll
    for (int j = 0; j < 2 * DV16; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
    for (int ic = 0; ic < chunks; ++ic) {
      float E[2][4] = {};
#pragma unroll
      for (int k = 0; k < DQ16; ++k) {
        uint32_t b[4];
        ldsm_x4(b, k_plain + ic * 16 * KS + k * 32);
        mma16816(E[0], Qa[k][0], Qa[k][1], Qa[k][2], Qa[k][3], b[0], b[1]);
        mma16816(E[1], Qa[k][0], Qa[k][1], Qa[k][2], Qa[k][3], b[2], b[3]);
      }
      uint32_t gA[4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float gg[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) gg[e] = fmaf(tanh_fast(E[nt][e]), 0.5f, 0.5f);
        gA[2 * nt] = pack2(gg[0], gg[1]);
        gA[2 * nt + 1] = pack2(gg[2], gg[3]);
      }
#pragma unroll
      for (int k = 0; k < DV16; ++k) {
        uint32_t b[4];
        ldsm_x4_t(b, v_trans + ic * 16 * VS + k * 32);
        mma16816(acc[2 * k], gA[0], gA[1], gA[2], gA[3], b[0], b[1]);
        mma16816(acc[2 * k + 1], gA[0], gA[1], gA[2], gA[3], b[2], b[3]);
      }
    }
    const size_t at = ((size_t)off0 * P.Lp + seg) * d + h * DVH, row = (size_t)P.Lp * d;
#pragma unroll
    for (int j = 0; j < 2 * DV16; ++j) {
      const int c = j * 8 + 2 * t;
      if (P.Hp) {
        if (r0 < C) *reinterpret_cast<float2*>(P.Hp + at + (size_t)r0 * row + c) = make_float2(acc[j][0], acc[j][1]);
        if (r1 < C) *reinterpret_cast<float2*>(P.Hp + at + (size_t)r1 * row + c) = make_float2(acc[j][2], acc[j][3]);
      }
      if (P.Hb) {
        if (r0 < C) *reinterpret_cast<uint32_t*>(P.Hb + at + (size_t)r0 * row + c) = pack2(acc[j][0], acc[j][1]);
        if (r1 < C) *reinterpret_cast<uint32_t*>(P.Hb + at + (size_t)r1 * row + c) = pack2(acc[j][2], acc[j][3]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------------------
// The attention of a recomputed GSTA layer on the same MMAs: per candidate e_{j,h} = s_j . Qt_h, a = softmax over the
// non-empty segments, m_h = sum_j a_{j,h} s_j, with the segment vectors in bf16 (the copy sta_fwd_mma_kernel writes), Qt
// and the weights a rounded to bf16, fp32 accumulation.  One warp per candidate: it stages 32 segment vectors at a time
// in its own shared memory (cp.async; rows past the candidate's last non-empty segment are zero rows) and Qt as eight head
// rows (heads past H are zero rows); scores = S Qt^T (segments on the MMA rows, heads on the eight columns), the softmax
// over the rows with lane-group reductions, then m^T = S^T a with S^T read by transposing ldmatrix and a taken from the
// accumulator layout through movmatrix.  More than 32 segments: the scores of all chunks first (they stay in registers),
// then a second pass over the chunks for m.
constexpr int kAttnWarps = 4;

__device__ __forceinline__ int nonempty_segments(const int32_t* lengths, const int32_t* cand_offsets, int U, int L, int S,
                                                 int Lp, int c) {
  int lo = 0, hi = U - 1;
  while (lo < hi) {                               // the last user whose first candidate is <= c
    const int mid = (lo + hi + 1) >> 1;
    if (cand_offsets[mid] <= c) lo = mid; else hi = mid - 1;
  }
  const int len = lengths[lo];
  if (len <= 0 || len > L) return 0;
  return min((len + S - 1) / S, Lp);
}

struct AttnFwdParams {
  const bf16* Hb;
  const float* Qt;
  const int32_t *lengths, *cand_offsets;
  float *Aw, *Mh;
  int N, U, L, S, Lp, H;
};

template <int D16, int NCH>
__global__ void __launch_bounds__(kAttnWarps * 32) gsta_attn_fwd_mma_kernel(const AttnFwdParams P) {
  constexpr int d = 16 * D16, SP = 2 * d + 16, kS = 32 * SP, kQ = 8 * SP;      // bytes: row pitch, S chunk, Qt rows
  extern __shared__ __align__(16) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int c = blockIdx.x * kAttnWarps + warp;
  if (c >= P.N) return;
  const int H = P.H, Lp = P.Lp;
  unsigned char* mine = smem + warp * (kS + kQ);
  const uint32_t Ssm = smem_addr(mine), Qsm = Ssm + kS;
  for (int i = lane; i < 8 * (d / 2); i += 32) {                   // Qt rows as bf16 pairs; heads past H: zeros
    const int h = i / (d / 2), x2 = i - h * (d / 2);
    uint32_t v = 0u;
    if (h < H) {
      const float2 q = *reinterpret_cast<const float2*>(P.Qt + ((size_t)c * H + h) * d + 2 * x2);
      v = pack2(q.x, q.y);
    }
    *reinterpret_cast<uint32_t*>(mine + kS + h * SP + x2 * 4) = v;
  }
  const int nv = nonempty_segments(P.lengths, P.cand_offsets, P.U, P.L, P.S, Lp, c);
  const int nch = (nv + 31) >> 5;
  const bf16* Sg = P.Hb + (size_t)c * Lp * d;
  auto stage = [&](int ch) {
#pragma unroll
    for (int k = 0; k < 2 * D16; ++k) {
      const int x = lane + 32 * k, r = x / (2 * D16), cc = x - r * (2 * D16), j = 32 * ch + r;
      cp16(Ssm + r * SP + cc * 16, Sg + (size_t)min(j, Lp - 1) * d + cc * 8, j < nv ? 16u : 0u);
    }
    cp_commit();
    cp_wait<0>();
    __syncwarp();
  };
  const int mi = lane >> 3, lr = lane & 7;
  const uint32_t a_plain = Ssm + ((mi & 1) * 8 + lr) * SP + (mi >> 1) * 16;      // A = S:   + mt 16 SP + k 32
  const uint32_t a_trans = Ssm + ((mi >> 1) * 8 + lr) * SP + (mi & 1) * 16;      // A = S^T: + mt 16 SP + mf 32
  const uint32_t q_rows = Qsm + lr * SP + (mi & 1) * 16;                         // B = Qt (x2): + k 32
  float e[NCH][2][4];
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int x = 0; x < 4; ++x) e[ch][mt][x] = 0.f;
    if (ch < nch) {
      stage(ch);
#pragma unroll
      for (int k = 0; k < D16; ++k) {
        uint32_t b[2];
        ldsm_x2(b, q_rows + k * 32);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          uint32_t a[4];
          ldsm_x4(a, a_plain + mt * 16 * SP + k * 32);
          mma16816(e[ch][mt], a[0], a[1], a[2], a[3], b[0], b[1]);
        }
      }
      __syncwarp();
    }
  }
  // softmax over the non-empty segments (rows), per head (columns 2t, 2t + 1)
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const bool in = 32 * ch + 16 * mt + 8 * hf + g < nv;
        if (!in) e[ch][mt][2 * hf] = e[ch][mt][2 * hf + 1] = -INFINITY;
        mx0 = fmaxf(mx0, e[ch][mt][2 * hf]);
        mx1 = fmaxf(mx1, e[ch][mt][2 * hf + 1]);
      }
  mx0 = group_max(mx0);
  mx1 = group_max(mx1);
  float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const float p0 = nv > 0 ? expf(e[ch][mt][2 * hf] - mx0) : 0.f, p1 = nv > 0 ? expf(e[ch][mt][2 * hf + 1] - mx1) : 0.f;
        e[ch][mt][2 * hf] = p0;
        e[ch][mt][2 * hf + 1] = p1;
        sum0 += p0;
        sum1 += p1;
      }
  sum0 = group_sum(sum0);
  sum1 = group_sum(sum1);
  const float inv0 = sum0 > 0.f ? 1.f / sum0 : 0.f, inv1 = sum1 > 0.f ? 1.f / sum1 : 0.f;
  float* Aw = P.Aw + (size_t)c * H * Lp;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int j = 32 * ch + 16 * mt + 8 * hf + g;
        const float a0 = e[ch][mt][2 * hf] * inv0, a1 = e[ch][mt][2 * hf + 1] * inv1;
        e[ch][mt][2 * hf] = a0;
        e[ch][mt][2 * hf + 1] = a1;
        if (j < Lp) {
          if (2 * t < H) Aw[(size_t)(2 * t) * Lp + j] = a0;
          if (2 * t + 1 < H) Aw[(size_t)(2 * t + 1) * Lp + j] = a1;
        }
      }
  // m^T [features] x [heads] = S^T a
  float macc[D16][4];
#pragma unroll
  for (int mf = 0; mf < D16; ++mf)
#pragma unroll
    for (int x = 0; x < 4; ++x) macc[mf][x] = 0.f;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
    if (ch < nch) {
      if (nch > 1) stage(ch);                                    // (a single chunk is still there)
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t b0 = movmatrix_t(pack2(e[ch][mt][0], e[ch][mt][1])), b1 = movmatrix_t(pack2(e[ch][mt][2], e[ch][mt][3]));
#pragma unroll
        for (int mf = 0; mf < D16; ++mf) {
          uint32_t a[4];
          ldsm_x4_t(a, a_trans + mt * 16 * SP + mf * 32);
          mma16816(macc[mf], a[0], a[1], a[2], a[3], b0, b1);
        }
      }
      __syncwarp();
    }
  }
  float* Mh = P.Mh + (size_t)c * H * d;
#pragma unroll
  for (int mf = 0; mf < D16; ++mf) {
    const int f0 = mf * 16 + g, f1 = f0 + 8;
    if (2 * t < H) {
      Mh[(size_t)(2 * t) * d + f0] = macc[mf][0];
      Mh[(size_t)(2 * t) * d + f1] = macc[mf][2];
    }
    if (2 * t + 1 < H) {
      Mh[(size_t)(2 * t + 1) * d + f0] = macc[mf][1];
      Mh[(size_t)(2 * t + 1) * d + f1] = macc[mf][3];
    }
  }
}

// The backward of the kernel above, same layout of the work: da_{j,h} = s_j . dm_h (S dm^T), de = a (da - sum_j a da),
// dQt_h = sum_j de_{j,h} s_j (S^T de, de through movmatrix), and the update of dH', ds_j += sum_h de_{j,h} Qt_h + a_{j,h} dm_h,
// as one product [de | a] [Qt ; dm] per 16 segments: its A operand is the two accumulator-layout tiles side by side
// (eight de heads, eight a heads), its B operand Qt and dm read by transposing ldmatrix.  The layer processed first
// writes dH' (zeros for the empty segments), the others add.
struct AttnBwdParams {
  const bf16* Hb;
  const float *Qt, *dM, *Aw;
  const int32_t *lengths, *cand_offsets;
  float *dQt, *dHp;
  bf16* dSb;                                     // non-null for the layer processed last: dH' leaves as this bf16 array only
  int N, U, L, S, Lp, H, overwrite;
};

template <int D16, int NCH>
__global__ void __launch_bounds__(kAttnWarps * 32) gsta_attn_bwd_mma_kernel(const AttnBwdParams P) {
  constexpr int d = 16 * D16, SP = 2 * d + 16, kS = 32 * SP, kQ = 8 * SP;
  extern __shared__ __align__(16) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int c = blockIdx.x * kAttnWarps + warp;
  if (c >= P.N) return;
  const int H = P.H, Lp = P.Lp;
  unsigned char* mine = smem + warp * (kS + 2 * kQ);
  const uint32_t Ssm = smem_addr(mine), Qsm = Ssm + kS, Msm = Qsm + kQ;
  for (int i = lane; i < 8 * (d / 2); i += 32) {                   // Qt and dm rows as bf16 pairs; heads past H: zeros
    const int h = i / (d / 2), x2 = i - h * (d / 2);
    uint32_t vq = 0u, vm = 0u;
    if (h < H) {
      const float2 q = *reinterpret_cast<const float2*>(P.Qt + ((size_t)c * H + h) * d + 2 * x2);
      const float2 m = *reinterpret_cast<const float2*>(P.dM + ((size_t)c * H + h) * d + 2 * x2);
      vq = pack2(q.x, q.y);
      vm = pack2(m.x, m.y);
    }
    *reinterpret_cast<uint32_t*>(mine + kS + h * SP + x2 * 4) = vq;
    *reinterpret_cast<uint32_t*>(mine + kS + kQ + h * SP + x2 * 4) = vm;
  }
  const int nv = nonempty_segments(P.lengths, P.cand_offsets, P.U, P.L, P.S, Lp, c);
  const int nch = (nv + 31) >> 5;
  const bf16* Sg = P.Hb + (size_t)c * Lp * d;
  auto stage = [&](int ch) {
#pragma unroll
    for (int k = 0; k < 2 * D16; ++k) {
      const int x = lane + 32 * k, r = x / (2 * D16), cc = x - r * (2 * D16), j = 32 * ch + r;
      cp16(Ssm + r * SP + cc * 16, Sg + (size_t)min(j, Lp - 1) * d + cc * 8, j < nv ? 16u : 0u);
    }
    cp_commit();
    cp_wait<0>();
    __syncwarp();
  };
  const int mi = lane >> 3, lr = lane & 7;
  const uint32_t a_plain = Ssm + ((mi & 1) * 8 + lr) * SP + (mi >> 1) * 16;
  const uint32_t a_trans = Ssm + ((mi >> 1) * 8 + lr) * SP + (mi & 1) * 16;
  const uint32_t m_rows = Msm + lr * SP + (mi & 1) * 16;                          // B = dm (x2): + k 32
  const uint32_t qm_trans = ((mi & 1) ? Msm : Qsm) + lr * SP + (mi >> 1) * 16;    // B = [Qt ; dm]^T: + 32 per 16 features
  // the weights a in the accumulator layout (rows = segments g, g + 8; columns = heads 2t, 2t + 1)
  float a[NCH][2][4], de[NCH][2][4];
  const float* Aw = P.Aw + (size_t)c * H * Lp;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int j = 32 * ch + 16 * mt + 8 * (x >> 1) + g, h = 2 * t + (x & 1);
        a[ch][mt][x] = (j < nv && h < H) ? Aw[(size_t)h * Lp + j] : 0.f;
        de[ch][mt][x] = 0.f;
      }
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
    if (ch < nch) {
      stage(ch);
#pragma unroll
      for (int k = 0; k < D16; ++k) {
        uint32_t b[2];
        ldsm_x2(b, m_rows + k * 32);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          uint32_t af[4];
          ldsm_x4(af, a_plain + mt * 16 * SP + k * 32);
          mma16816(de[ch][mt], af[0], af[1], af[2], af[3], b[0], b[1]);        // (da for now)
        }
      }
      __syncwarp();
    }
  float dot0 = 0.f, dot1 = 0.f;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        dot0 = fmaf(a[ch][mt][2 * hf], de[ch][mt][2 * hf], dot0);
        dot1 = fmaf(a[ch][mt][2 * hf + 1], de[ch][mt][2 * hf + 1], dot1);
      }
  dot0 = group_sum(dot0);
  dot1 = group_sum(dot1);
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        de[ch][mt][2 * hf] = a[ch][mt][2 * hf] * (de[ch][mt][2 * hf] - dot0);
        de[ch][mt][2 * hf + 1] = a[ch][mt][2 * hf + 1] * (de[ch][mt][2 * hf + 1] - dot1);
      }
  float qacc[D16][4];
#pragma unroll
  for (int mf = 0; mf < D16; ++mf)
#pragma unroll
    for (int x = 0; x < 4; ++x) qacc[mf][x] = 0.f;
  float* dS = P.dHp + (size_t)c * Lp * d;
  bf16* dSb = P.dSb ? P.dSb + (size_t)c * Lp * d : nullptr;
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
    if (ch < nch) {
      if (nch > 1) stage(ch);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t e0 = pack2(de[ch][mt][0], de[ch][mt][1]), e1 = pack2(de[ch][mt][2], de[ch][mt][3]);
        const uint32_t w0 = pack2(a[ch][mt][0], a[ch][mt][1]), w1 = pack2(a[ch][mt][2], a[ch][mt][3]);
        const uint32_t b0 = movmatrix_t(e0), b1 = movmatrix_t(e1);
#pragma unroll
        for (int mf = 0; mf < D16; ++mf) {
          uint32_t af[4];
          ldsm_x4_t(af, a_trans + mt * 16 * SP + mf * 32);
          mma16816(qacc[mf], af[0], af[1], af[2], af[3], b0, b1);
        }
        // ds rows of these 16 segments: [de | a] [Qt ; dm]
        const int j0 = 32 * ch + 16 * mt + g, j1 = j0 + 8;
#pragma unroll
        for (int nf = 0; nf < D16; ++nf) {
          uint32_t b[4];
          ldsm_x4_t(b, qm_trans + nf * 32);
          float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
          mma16816(c0, e0, e1, w0, w1, b[0], b[1]);
          mma16816(c1, e0, e1, w0, w1, b[2], b[3]);
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int j = hf ? j1 : j0;
            if (j >= nv) continue;
            const size_t at = (size_t)j * d + nf * 16 + 2 * t;
            float2 u = make_float2(c0[2 * hf], c0[2 * hf + 1]), v = make_float2(c1[2 * hf], c1[2 * hf + 1]);
            if (!P.overwrite) {
              const float2 pu = *reinterpret_cast<const float2*>(dS + at), pv = *reinterpret_cast<const float2*>(dS + at + 8);
              u.x += pu.x; u.y += pu.y; v.x += pv.x; v.y += pv.y;
            }
            if (dSb) {
              *reinterpret_cast<uint32_t*>(dSb + at) = pack2(u.x, u.y);
              *reinterpret_cast<uint32_t*>(dSb + at + 8) = pack2(v.x, v.y);
            } else {
              *reinterpret_cast<float2*>(dS + at) = u;
              *reinterpret_cast<float2*>(dS + at + 8) = v;
            }
          }
        }
      }
      __syncwarp();
    }
  if (P.overwrite && !dSb)                                         // empty segments receive no gradient (their bf16 rows are never read)
    for (int i = nv * (d / 4) + lane; i < Lp * (d / 4); i += 32)
      *reinterpret_cast<float4*>(dS + (size_t)i * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
  float* dQt = P.dQt + (size_t)c * H * d;
#pragma unroll
  for (int mf = 0; mf < D16; ++mf) {
    const int f0 = mf * 16 + g, f1 = f0 + 8;
    if (2 * t < H) {
      dQt[(size_t)(2 * t) * d + f0] = qacc[mf][0];
      dQt[(size_t)(2 * t) * d + f1] = qacc[mf][2];
    }
    if (2 * t + 1 < H) {
      dQt[(size_t)(2 * t + 1) * d + f0] = qacc[mf][1];
      dQt[(size_t)(2 * t + 1) * d + f1] = qacc[mf][3];
    }
  }
}

struct MmaShape {
  int mt, dq16, dv16;
};
bool mma_shape(const Plan& p, MmaShape* s) {
  if (p.dqh % 16 || p.dvh % 16) return false;
  s->dq16 = p.dqh / 16;
  s->dv16 = p.dvh / 16;
  s->mt = (p.S <= 16 || s->dv16 == 4) ? 1 : 2;       // (two row tiles of 64-wide value slices would not fit the registers)
  return (s->dq16 == 1 || s->dq16 == 2) && (s->dv16 == 1 || s->dv16 == 2 || s->dv16 == 4);
}

template <int MT, int DQ16, int DV16>
int launch_mma(const BwdMmaParams& P, int U, cudaStream_t st) {
  constexpr int smem = kBwdWarps * 2 * 16 * ((2 * 16 * DQ16 + 16) + (2 * 16 * DV16 + 16));
  auto kernel = sta_bwd_mma_kernel<MT, DQ16, DV16>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  LaunchScope ls("bwd_sta_mma", st);
  kernel<<<dim3((P.jobs + kBwdWarps - 1) / kBwdWarps, U), kBwdWarps * 32, smem, st>>>(P);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

constexpr size_t kFwdSmemMax = 160 * 1024;
size_t fwd_smem(const Plan& p) {
  const size_t rows = (size_t)(std::min(p.S, p.L) + 15) / 16 * 16;
  return rows * (2 * p.dqh + 16 + 2 * p.dvh + 16);
}

template <int DQ16, int DV16>
int launch_fwd(const FwdMmaParams& P, int U, size_t smem, cudaStream_t st) {
  auto kernel = sta_fwd_mma_kernel<DQ16, DV16>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("bwd_sta_fwd_mma", st);
  kernel<<<dim3(P.Lp * P.H, U), kBwdWarps * 32, smem, st>>>(P);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

int cast(const float* src, bf16* dst, size_t n, float scale, cudaStream_t st) {
  if (n == 0) return LASER_OK;
  LaunchScope ls("bwd_cast_bf16", st);
  const size_t n4 = n / 4;
  const int blocks = (int)std::min<size_t>((n4 + 255) / 256, 148 * 16);
  cast_bf16_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(dst), n4, scale);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

struct MmaScratch {
  bf16 *Qb, *Kb, *Vb, *dSb, *Hb;
  size_t total;
};
MmaScratch carve_mma(const Plan& p, char* base) {
  MmaScratch s;
  size_t off = 0;
  auto take = [&](size_t n) {
    bf16* ptr = base ? reinterpret_cast<bf16*>(base + off) : nullptr;
    off = align_up(off + n * sizeof(bf16)) + kGuardBytes;
    return ptr;
  };
  const size_t UL = (size_t)p.U * p.L;
  s.Qb = take((size_t)p.N * p.dqk);
  s.Kb = take(UL * p.dqk);
  s.Vb = take(UL * p.d);
  s.dSb = take((size_t)p.N * p.Lp * p.d);
  s.Hb = take((size_t)p.N * p.Lp * p.d);
  s.total = off;
  return s;
}

}  // namespace

bool sta_bwd_mma_supported(const Plan& p) {
  MmaShape s;
  if (!mma_shape(p, &s)) return false;
  const long long R = (std::min(p.S, p.L) + 16 * s.mt - 1) / (16 * s.mt);
  return p.U <= 65535 && (long long)p.Lp * R * p.H <= 0x7fffffffLL && p.maxC >= 8;
}

size_t sta_bwd_mma_scratch_bytes(const Plan& p) { return sta_bwd_mma_supported(p) ? carve_mma(p, nullptr).total : 0; }

int sta_mma_operands(const Plan& p, const float* Qf, const float* Kf, const float* Vf, char* scratch, cudaStream_t st) {
  const MmaScratch s = carve_mma(p, scratch);
  const size_t UL = (size_t)p.U * p.L;
  int rc;
  if ((rc = cast(Qf, s.Qb, (size_t)p.N * p.dqk, 0.5f, st)) != LASER_OK) return rc;
  if (Kf && (rc = cast(Kf, s.Kb, UL * p.dqk, 1.f, st)) != LASER_OK) return rc;
  return Vf ? cast(Vf, s.Vb, UL * p.d, 1.f, st) : (int)LASER_OK;
}

void sta_mma_operand_arrays(const Plan& p, char* scratch, __nv_bfloat16** Kb, __nv_bfloat16** Vb) {
  const MmaScratch s = carve_mma(p, scratch);
  *Kb = s.Kb;
  *Vb = s.Vb;
}

bool sta_fwd_mma_supported(const Plan& p) {
  return sta_bwd_mma_supported(p) && fwd_smem(p) <= kFwdSmemMax && (long long)p.Lp * p.H <= 0x7fffffffLL;
}

bool gsta_attn_mma_supported(const Plan& p) {
  return sta_fwd_mma_supported(p) && (p.d == 32 || p.d == 64 || p.d == 128) && p.H <= 8 && p.Lp <= 128;
}

template <int D16>
int launch_attn_fwd(const AttnFwdParams& P, cudaStream_t st) {
  constexpr size_t smem = (size_t)kAttnWarps * 40 * (2 * 16 * D16 + 16);
  const int nch = (P.Lp + 31) / 32;
  auto kernel = nch <= 1 ? gsta_attn_fwd_mma_kernel<D16, 1> : nch <= 2 ? gsta_attn_fwd_mma_kernel<D16, 2> : gsta_attn_fwd_mma_kernel<D16, 4>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("bwd_attn_fwd_mma", st);
  kernel<<<(P.N + kAttnWarps - 1) / kAttnWarps, kAttnWarps * 32, smem, st>>>(P);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

int gsta_attn_fwd_mma(const Plan& p, const float* Qt, const int32_t* lengths, const int32_t* cand_offsets, float* Aw,
                      float* Mh, char* scratch, cudaStream_t st) {
  const MmaScratch s = carve_mma(p, scratch);
  AttnFwdParams P;
  P.Hb = s.Hb; P.Qt = Qt; P.lengths = lengths; P.cand_offsets = cand_offsets; P.Aw = Aw; P.Mh = Mh;
  P.N = p.N; P.U = p.U; P.L = p.L; P.S = p.S; P.Lp = p.Lp; P.H = p.H;
  if (p.d == 32) return launch_attn_fwd<2>(P, st);
  if (p.d == 64) return launch_attn_fwd<4>(P, st);
  if (p.d == 128) return launch_attn_fwd<8>(P, st);
  return LASER_ERR_UNSUPPORTED;
}

template <int D16>
int launch_attn_bwd(const AttnBwdParams& P, cudaStream_t st) {
  constexpr size_t smem = (size_t)kAttnWarps * 48 * (2 * 16 * D16 + 16);
  const int nch = (P.Lp + 31) / 32;
  auto kernel = nch <= 1 ? gsta_attn_bwd_mma_kernel<D16, 1> : nch <= 2 ? gsta_attn_bwd_mma_kernel<D16, 2> : gsta_attn_bwd_mma_kernel<D16, 4>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("bwd_attn_bwd_mma", st);
  kernel<<<(P.N + kAttnWarps - 1) / kAttnWarps, kAttnWarps * 32, smem, st>>>(P);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

int gsta_attn_bwd_mma(const Plan& p, const float* Qt, const float* Aw, const float* dM, const int32_t* lengths,
                      const int32_t* cand_offsets, float* dQt, float* dHp, bool overwrite, bool last, char* scratch,
                      cudaStream_t st) {
  const MmaScratch s = carve_mma(p, scratch);
  AttnBwdParams P;
  P.dSb = last ? s.dSb : nullptr;
  P.Hb = s.Hb; P.Qt = Qt; P.dM = dM; P.Aw = Aw; P.lengths = lengths; P.cand_offsets = cand_offsets; P.dQt = dQt; P.dHp = dHp;
  P.N = p.N; P.U = p.U; P.L = p.L; P.S = p.S; P.Lp = p.Lp; P.H = p.H; P.overwrite = overwrite ? 1 : 0;
  if (p.d == 32) return launch_attn_bwd<2>(P, st);
  if (p.d == 64) return launch_attn_bwd<4>(P, st);
  if (p.d == 128) return launch_attn_bwd<8>(P, st);
  return LASER_ERR_UNSUPPORTED;
}

int sta_fwd_mma(const Plan& p, const int32_t* lengths, const int32_t* cand_offsets, float* Hp, bool bf16_copy, char* scratch,
                cudaStream_t st) {
  MmaShape sh;
  if (!mma_shape(p, &sh) || !sta_fwd_mma_supported(p)) return LASER_ERR_UNSUPPORTED;
  const MmaScratch s = carve_mma(p, scratch);
  FwdMmaParams P;
  P.Qb = s.Qb; P.Kb = s.Kb; P.Vb = s.Vb;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.Hp = Hp;
  P.Hb = bf16_copy ? s.Hb : nullptr;
  P.L = p.L; P.d = p.d; P.dqk = p.dqk; P.H = p.H; P.S = p.S; P.Lp = p.Lp; P.N = p.N;
  P.rows = (std::min(p.S, p.L) + 15) / 16 * 16;
  const size_t smem = fwd_smem(p);
#define LASER_FWD_CASE(DQ, DV) \
  if (sh.dq16 == DQ && sh.dv16 == DV) return launch_fwd<DQ, DV>(P, p.U, smem, st);
  LASER_FWD_CASE(1, 1) LASER_FWD_CASE(1, 2) LASER_FWD_CASE(1, 4)
  LASER_FWD_CASE(2, 1) LASER_FWD_CASE(2, 2) LASER_FWD_CASE(2, 4)
#undef LASER_FWD_CASE
  return LASER_ERR_UNSUPPORTED;
}

int sta_bwd_mma(const Plan& p, const float* dHp, const int32_t* lengths, const int32_t* cand_offsets, float* dQf,
                float* dK, float* dV, char* scratch, cudaStream_t st) {
  MmaShape sh;
  if (!mma_shape(p, &sh)) return LASER_ERR_UNSUPPORTED;
  const MmaScratch s = carve_mma(p, scratch);
  int rc;
  if (dHp && (rc = cast(dHp, s.dSb, (size_t)p.N * p.Lp * p.d, 1.f, st)) != LASER_OK) return rc;
  BwdMmaParams P;
  P.Qb = s.Qb; P.Kb = s.Kb; P.Vb = s.Vb; P.dSb = s.dSb;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.dQf = dQf; P.dK = dK; P.dV = dV;
  P.L = p.L; P.d = p.d; P.dqk = p.dqk; P.H = p.H; P.S = p.S; P.Lp = p.Lp; P.N = p.N;
  P.R = (std::min(p.S, p.L) + 16 * sh.mt - 1) / (16 * sh.mt);
  P.jobs = p.Lp * P.R * p.H;
#define LASER_MMA_CASE(MT, DQ, DV) \
  if (sh.mt == MT && sh.dq16 == DQ && sh.dv16 == DV) return launch_mma<MT, DQ, DV>(P, p.U, st);
  LASER_MMA_CASE(1, 1, 1) LASER_MMA_CASE(1, 1, 2) LASER_MMA_CASE(1, 1, 4)
  LASER_MMA_CASE(1, 2, 1) LASER_MMA_CASE(1, 2, 2) LASER_MMA_CASE(1, 2, 4)
  LASER_MMA_CASE(2, 1, 1) LASER_MMA_CASE(2, 1, 2)
  LASER_MMA_CASE(2, 2, 1) LASER_MMA_CASE(2, 2, 2)
#undef LASER_MMA_CASE
  return LASER_ERR_UNSUPPORTED;
}

}  // namespace laser
