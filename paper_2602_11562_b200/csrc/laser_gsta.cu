// Fused GSTA kernel (Eq. 7 and the residual update t_l = t_{l-1} + o_l) for bf16 inputs.
//
// One block owns 16 consecutive candidates (the 16 rows of every warp-level MMA) and runs all M layers for them:
//
//   A   Q   = T W_q^l                              [16 x d]    batched over the 16 candidates
//   B   Qt_h = Q[:, head h] W_k^l[:, head h]^T / tau  [16 x d] per head: (s_j W_k)_h . q_h = s_j . Qt_h
//   C   per candidate: scores e_{h,j} = Qt_h . s_j over its non-empty segments j, softmax over j, m_h = sum_j a_{h,j} s_j.
//       The candidate's segment vectors are staged in shared memory (cp.async, two buffers per warp, 16 vectors per
//       chunk); every vector is read from global memory once per layer and used for both contractions, with an online
//       softmax across chunks.
//   D   o[:, head h] = m_h W_v^l[:, head h];  T += o
//
// This is Eq. 7 re-associated (exact in real arithmetic): the key / value projections are applied to the query and to
// the attention-weighted sum instead of to every segment vector, which cuts the cost per candidate and layer from
// 4 L' d^2 to 6 d^2 + 4 H L' d flops.  Operands of every MMA are bf16, accumulators and the running target T are fp32.
// The weights reach the MMAs as B fragments straight from a fragment-ordered image in global memory (built once per
// call by gsta_prep_kernel), so they need no shared memory.
#include "laser_common.cuh"
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
  bf16* z;
  int* status;
};

// Fragment-ordered weight images.  Entry (layer, matrix, kt, p, lane) holds the B fragments of k-tile kt for the two
// 8-column tiles 2p and 2p+1: {b0, b1 of tile 2p, b0, b1 of tile 2p+1}.  For W_q and W_v the MMA's B is W itself
// (B[k][n] = W[k][n]); for W_k it is the transpose (B[k][n] = W_k[n][k]).
__global__ void __launch_bounds__(256) gsta_prep_kernel(GstaParams P) {
  const int D16 = P.d >> 4;
  const int per_mat = D16 * D16 * 32;
  const int total = P.M * 3 * per_mat;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int lane = i & 31;
    int r = i >> 5;
    const int p = r % D16; r /= D16;
    const int kt = r % D16; r /= D16;
    const int m = r % 3;
    const int l = r / 3;
    const uint16_t* W = reinterpret_cast<const uint16_t*>(P.Wg) + (size_t)(l * 3 + m) * P.d * P.d;
    const int g = lane >> 2, t = lane & 3;
    uint32_t v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int n = (2 * p + (q >> 1)) * 8 + g;
      const int k = kt * 16 + 2 * t + (q & 1) * 8;
      uint32_t lo, hi;
      if (m == 1) { lo = W[(size_t)n * P.d + k]; hi = W[(size_t)n * P.d + k + 1]; }
      else { lo = W[(size_t)k * P.d + n]; hi = W[(size_t)(k + 1) * P.d + n]; }
      v[q] = lo | (hi << 16);
    }
    P.img[i] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

template <int D16>
__global__ void __launch_bounds__(kGThreads, 2) gsta_mma_kernel(GstaParams P) {
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
  const int c_base = blockIdx.x * kGT;

  // ---- set-up: candidate -> user -> number of non-empty segments; T = candidates; zero row
  if (tid < kGT) {
    const int c = c_base + tid;
    int nv = 0;
    if (c < P.N) {
      if (P.cand_offsets[0] > c || P.cand_offsets[P.U] <= c) {
        report_status(P.status, LASER_ERR_BAD_INPUT);
      } else {
        int lo = 0, hi = P.U;   // cand_offsets[lo] <= c < cand_offsets[hi]
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (P.cand_offsets[mid] <= c) lo = mid; else hi = mid;
        }
        const int len = P.lengths[lo];
        if (len < 0 || len > P.L) report_status(P.status, LASER_ERR_BAD_INPUT);
        else nv = min((len + P.S - 1) / P.S, P.Lp);
      }
    }
    nv_s[tid] = nv;
  }
  for (int i = tid; i < kGT * d; i += kGThreads) {
    const int r = i / d, c = i - r * d;
    Ts[r * TS + c] = c_base + r < P.N ? __bfloat162float(P.cands[(size_t)(c_base + r) * d + c]) : 0.f;
  }
  for (int i = tid; i < RS / 4; i += kGThreads) reinterpret_cast<uint32_t*>(zrow)[i] = 0u;
  __syncthreads();

  // ---- chunk pipeline of this warp: (layer, candidate slot ci -> candidate warp + kGW ci, chunk) in processing order
  uint8_t* my_stage = stage + (size_t)warp * 2 * kChunk * RS;
  int f_layer = 0, f_ci = 0, f_ch = 0;
  bool f_valid = false;
  int first_ci = -1;
#pragma unroll
  for (int ci = kGT / kGW - 1; ci >= 0; --ci)
    if (nv_s[warp + kGW * ci] > 0) first_ci = ci;
  if (first_ci >= 0 && P.M > 0) { f_valid = true; f_ci = first_ci; }

  auto issue = [&](int buf) {   // stage chunk (f_ci, f_ch) into buffer `buf`, then step the fetch cursor
    const int c = warp + kGW * f_ci;
    const int nv = nv_s[c];
    const bf16* src = P.Hp + ((size_t)(c_base + c) * P.Lp + f_ch * kChunk) * d;
    const uint32_t dst = smem_addr(my_stage + (size_t)buf * kChunk * RS);
    const int rows = min(kChunk, nv - f_ch * kChunk);
    static_assert((kChunk * 2 * D16) % 32 == 0, "a chunk is a whole number of 16-byte pieces per lane");
#pragma unroll
    for (int i = 0; i < kChunk * 2 * D16 / 32; ++i) {      // kChunk rows of 2 D16 16-byte pieces
      const int piece = i * 32 + lane;
      const int r = piece / (2 * D16), q = piece - r * (2 * D16);
      const bool ok = r < rows;
      cp16(dst + r * RS + q * 16, ok ? (const void*)(src + (size_t)r * d + q * 8) : (const void*)P.Hp, ok ? 16u : 0u);
    }
    if (++f_ch * kChunk >= nv) {
      f_ch = 0;
      do { ++f_ci; } while (f_ci < kGT / kGW && nv_s[warp + kGW * f_ci] == 0);
      if (f_ci >= kGT / kGW) {
        f_ci = first_ci;
        if (++f_layer >= P.M) f_valid = false;
      }
    }
  };
  int buf = 0;
  if (f_valid) issue(0);
  cp_commit();

  const uint32_t ldsm_row = (lane & 7) + ((lane >> 3) & 1) * 8;   // row supplied by this lane (A-operand order)
  const uint32_t ldsm_kc = lane >> 4;                             // 16-byte k-chunk supplied by this lane

  for (int l = 0; l < P.M; ++l) {
    const uint4* imgq = P.img + (size_t)(l * 3 + 0) * D16 * D16 * 32;
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
      for (int p = warp; p < D16; p += kGW) {
        float acc[2][4] = {};
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) {
          const uint4 b = __ldg(imgq + (kt * D16 + p) * 32 + lane);
          mma16816(acc[0], ta[kt][0], ta[kt][1], ta[kt][2], ta[kt][3], b.x, b.y);
          mma16816(acc[1], ta[kt][0], ta[kt][1], ta[kt][2], ta[kt][3], b.z, b.w);
        }
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
      for (int p = warp; p < D16; p += kGW) {
        float acc[2][4] = {};
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) {
          const uint4 b = __ldg(imgk + (kt * D16 + p) * 32 + lane);
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
    for (int ci = 0; ci < kGT / kGW; ++ci) {
      const int c = warp + kGW * ci;
      const int nv = nv_s[c];
      if (nv == 0) {   // no segment to attend to: m = 0 (o_l = 0)
        for (int i = lane; i < H * (d / 2); i += 32) {
          const int h = i / (d / 2), q = i - h * (d / 2);
          *reinterpret_cast<uint32_t*>(Qt + (c * H + h) * RS + q * 4) = 0u;
        }
        continue;
      }
      // A fragments of Qt_c: rows = heads (rows >= H read the zero row), only rows 0-7 are non-zero
      uint32_t qa[D16][2];
      {
        const int h = lane & 7;
        const uint8_t* rowp = h < H ? Qt + (c * H + h) * RS : zrow;
#pragma unroll
        for (int kt = 0; kt < D16; ++kt) ldsm_x2(qa[kt], smem_addr(rowp + (kt * 2 + ((lane >> 3) & 1)) * 16));
      }
      float macc[2 * D16][4];
#pragma unroll
      for (int j = 0; j < 2 * D16; ++j) macc[j][0] = macc[j][1] = macc[j][2] = macc[j][3] = 0.f;
      float run_max = -INFINITY, run_sum = 0.f;

      const int nch = (nv + kChunk - 1) / kChunk;
      for (int ch = 0; ch < nch; ++ch) {
        if (f_valid) issue(buf ^ 1);
        cp_commit();
        cp_wait<1>();
        __syncwarp();
        const uint32_t sb = smem_addr(my_stage + (size_t)buf * kChunk * RS);
        const int rows = min(kChunk, nv - ch * kChunk);

        // scores e[h][j] for the chunk's (up to) 16 segments: 2 column tiles of 8 segments; even and odd k-tiles
        // accumulate separately so that four MMA chains are in flight
        float e[2][4], e2[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int q = 0; q < 4; ++q) e[nt][q] = e2[nt][q] = 0.f;
        {
          const uint32_t a = sb + ((lane & 7) + ((lane >> 4) & 1) * 8) * RS + ((lane >> 3) & 1) * 16;
#pragma unroll
          for (int kt = 0; kt < D16; ++kt) {
            uint32_t b[4];
            ldsm_x4(b, a + kt * 32);
            if (kt & 1) {
              mma16816(e2[0], qa[kt][0], 0u, qa[kt][1], 0u, b[0], b[1]);
              mma16816(e2[1], qa[kt][0], 0u, qa[kt][1], 0u, b[2], b[3]);
            } else {
              mma16816(e[0], qa[kt][0], 0u, qa[kt][1], 0u, b[0], b[1]);
              mma16816(e[1], qa[kt][0], 0u, qa[kt][1], 0u, b[2], b[3]);
            }
          }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            e[nt][q] += e2[nt][q];
            if (nt * 8 + 2 * t + q >= rows) e[nt][q] = -INFINITY;
            mx = fmaxf(mx, e[nt][q]);
          }
        mx = quad_max(mx);                       // the chunk holds at least one valid segment, so mx is finite
        const float new_max = fmaxf(run_max, mx);
        const float scale = __expf(run_max - new_max);
        run_max = new_max;
        float psum = 0.f;
        uint32_t pa[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const float p0 = __expf(e[q][0] - new_max), p1 = __expf(e[q][1] - new_max);
          pa[q] = pack2(p0, p1);
          psum += bf16_lo(pa[q]) + bf16_hi(pa[q]);   // normalise by exactly the weights the MMA uses
        }
        run_sum = run_sum * scale + psum;
#pragma unroll
        for (int j = 0; j < 2 * D16; ++j) { macc[j][0] *= scale; macc[j][1] *= scale; }

        // m += P S   (rows = heads, k = the chunk's segments, columns = d)
        {
          const uint32_t a = sb + ((lane & 7) + ((lane >> 3) & 1) * 8) * RS + (lane >> 4) * 16;
#pragma unroll
          for (int jp = 0; jp < D16; ++jp) {
            uint32_t b[4];
            ldsm_x4_t(b, a + jp * 32);
            mma16816(macc[2 * jp], pa[0], 0u, pa[1], 0u, b[0], b[1]);
            mma16816(macc[2 * jp + 1], pa[0], 0u, pa[1], 0u, b[2], b[3]);
          }
        }
        __syncwarp();   // every lane is done with this buffer before the next iteration refills it
        buf ^= 1;
      }
      const float inv = 1.f / quad_sum(run_sum);
      if (g < H) {
#pragma unroll
        for (int j = 0; j < 2 * D16; ++j)
          *reinterpret_cast<uint32_t*>(Qt + (c * H + g) * RS + (j * 8 + 2 * t) * 2) = pack2(macc[j][0] * inv, macc[j][1] * inv);
      }
    }
    __syncthreads();

    // ---------------------------------------------------------------- D: o[:, head h] = m_h W_v[:, head h];  T += o
    for (int p = warp; p < D16; p += kGW) {
      const int h = (p * 16) / dvh;
      float acc[2][4] = {};
#pragma unroll
      for (int kt = 0; kt < D16; ++kt) {
        uint32_t a[4];
        ldsm_x4(a, smem_addr(Qt + ((int)ldsm_row * H + h) * RS + (kt * 2 + ldsm_kc) * 16));
        const uint4 b = __ldg(imgv + (kt * D16 + p) * 32 + lane);
        mma16816(acc[0], a[0], a[1], a[2], a[3], b.x, b.y);
        mma16816(acc[1], a[0], a[1], a[2], a[3], b.z, b.w);
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
    if (c_base + r < P.N) {
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
  LASER_CUDA_OK(cudaFuncSetAttribute(gsta_mma_kernel<D16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("gsta_mma", st);
  gsta_mma_kernel<D16><<<(P.N + kGT - 1) / kGT, kGThreads, smem, st>>>(P);
  return LASER_OK;
}

}  // namespace

bool gsta_mma_supported(const Plan& p) {
  if (p.dtype != LASER_BF16) return false;
  if (p.d % 16 || p.d < 16 || p.d > 128) return false;
  if (p.H > 8 || p.dvh % 16) return false;
  return true;
}

size_t gsta_mma_image_bytes(const Plan& p) { return (size_t)p.M * 3 * p.d * p.d * 2; }

int gsta_mma(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets, const void* cands,
             const void* Wg, void* z, char* ws, cudaStream_t st) {
  if (p.N == 0) return LASER_OK;
  GstaParams P;
  P.N = p.N; P.U = p.U; P.L = p.L; P.S = p.S; P.Lp = p.Lp; P.H = p.H; P.M = p.M; P.d = p.d;
  P.inv_tau = p.inv_tau;
  P.Hp = (const bf16*)Hprime; P.cands = (const bf16*)cands; P.Wg = (const bf16*)Wg;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.img = reinterpret_cast<uint4*>(ws + p.off_gimg);
  P.z = (bf16*)z;
  P.status = reinterpret_cast<int*>(ws + p.off_status);
  if (p.M > 0) {
    const int total = p.M * 3 * (p.d / 16) * (p.d / 16) * 32;
    LaunchScope ls("gsta_prep", st);
    gsta_prep_kernel<<<(total + 255) / 256, 256, 0, st>>>(P);
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
