// Backward pass of STA + GSTA: the vector-Jacobian product of z with respect to the items, the candidates and every
// weight matrix.  The paper trains the model (section "Experimental Settings") without printing backward formulas; what
// is computed here is the chain rule through Eq. 7 (layers last to first) and then through Eq. 10-12 and Eq. 8-9.
//
// Inputs are read in their dtype, everything else is fp32.  Two versions: FP32 ALUs throughout (either dtype), and, for
// bf16 batches, the batched matrix products on the tensor cores with TF32 operands (gemm_tf32_kernel) plus the gate
// contractions, the recomputed H' and the GSTA attention with bf16 operands (laser_backward_mma.cu).  The forward intermediates are recomputed and kept (projections, H', and per GSTA layer
// the running target, Q, the key-folded query Qt_h = W_k[:, h] Q_h / tau, the attention weights and the weighted sums
// m_h = sum_j a_j s_j), all dense steps are batched matrix products over the N candidates (or the U L item rows), and
// three kernels do what is not a matrix product:
//   gsta_attn_fwd   per candidate: e_{j,h} = s_j . Qt_h, a = softmax_j, m_h = sum_j a_{j,h} s_j
//   gsta_attn_bwd   per candidate: da_j = s_j . dm_h, de = a (da - sum a da), dQt_h = sum_j de_j s_j,
//                   ds_j += de_j Qt_h + a_j dm_h
//   sta_bwd         per (user, 32 items of a segment), looping over the user's candidates: gate g = Sigmoid(q_h . k_n),
//                   dg = ds_i[h] . v_n, dv_n += g ds_i[h], de = dg g (1 - g), dk_n += de q_h, dq_h += de k_n
// With the re-association of the forward (keys and values of a segment vector are never formed):
//   o_h = m_h W_v[:, h]  =>  dm_h = do_h W_v[:, h]^T,  dW_v[:, h] += m_h^T do_h
//   Qt_h = Q_h W_k[:, h]^T / tau  =>  dQ_h = dQt_h W_k[:, h] / tau,  dW_k[:, h] += dQt_h^T Q_h / tau
// Sums over candidates that end in one weight matrix are split over blocks and finished with floating-point atomics, so
// the last bits of the weight gradients and of d_cands' STA part depend on the order in which blocks finish.
#include "laser_common.cuh"
#include "laser_mma.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;

// ------------------------------------------------------------------------------------------------ batched products
// C[m][n] (+)= alpha * sum_k A(m, k) B(k, n);  A(m, k) = ta ? A[k lda + m] : A[m lda + k],  B(k, n) = tb ? B[n ldb + k]
// : B[k ldb + n].  64 x 64 tiles of C, k-steps of 16; gridDim.z splits K and the partial sums are added atomically
// (C then has to hold its initial value before the launch).  `batch` independent products of the same shape (one per
// head) go out in one launch: product b reads A + b sa, B + b sb and writes C + b sc.
constexpr int kTM = 64, kTN = 64, kTK = 16, kGemmThreads = 256;

template <typename TA, typename TB>
__global__ void __launch_bounds__(kGemmThreads)
gemm_kernel(int M, int N, int K, const TA* __restrict__ A, int lda, int ta, const TB* __restrict__ B, int ldb, int tb,
            float* __restrict__ C, int ldc, float alpha, int accumulate, int k_per_split, int tiles_n, int sa, int sb,
            int sc) {
  __shared__ __align__(16) float As[kTK][kTM + 4], Bs[kTK][kTN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int batch = blockIdx.y;                                 // independent products: operands sa, sb, sc elements apart
  A += (size_t)batch * sa;
  B += (size_t)batch * sb;
  C += (size_t)batch * sc;
  // grid.x enumerates the tiles of C with the column tile running fastest: blocks that share a row tile of A run together
  const int tile_m = blockIdx.x / tiles_n, m0 = tile_m * kTM, n0 = (blockIdx.x - tile_m * tiles_n) * kTN;
  const int k_lo = blockIdx.z * k_per_split, k_hi = min(K, k_lo + k_per_split);
  float acc[4][4] = {};
  for (int k0 = k_lo; k0 < k_hi; k0 += kTK) {
    for (int i = tid; i < kTK * kTM; i += kGemmThreads) {
      int kk, mm;
      if (ta) { kk = i / kTM; mm = i - kk * kTM; } else { mm = i / kTK; kk = i - mm * kTK; }
      const int m = m0 + mm, k = k0 + kk;
      float v = 0.f;
      if (m < M && k < k_hi) v = to_f32<TA>(ta ? A[(size_t)k * lda + m] : A[(size_t)m * lda + k]);
      As[kk][mm] = v;
    }
    for (int i = tid; i < kTK * kTN; i += kGemmThreads) {
      int kk, nn;
      if (tb) { nn = i / kTK; kk = i - nn * kTK; } else { kk = i / kTN; nn = i - kk * kTN; }
      const int n = n0 + nn, k = k0 + kk;
      float v = 0.f;
      if (n < N && k < k_hi) v = to_f32<TB>(tb ? B[(size_t)n * ldb + k] : B[(size_t)k * ldb + n]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTK; ++kk) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float* c = C + (size_t)m * ldc + n;
      const float v = alpha * acc[i][j];
      if (gridDim.z > 1) atomicAdd(c, v);
      else *c = accumulate ? *c + v : v;
    }
  }
}

// The same product on the tensor cores: mma.sync m16n8k8 with TF32 operands (bf16 inputs are exact in TF32, fp32 ones are
// rounded to nearest when they are staged), fp32 accumulation.  64 x 64 tiles of C, k-steps of 32, eight warps of 32 x 16.
// An operand whose contraction index is contiguous in memory is staged row by row ([64][kWK + 4]), the other k-major
// ([kWK][64 + 8]): both paddings make the fragment reads conflict-free.  Full, aligned tiles are staged with 16-byte (fp32)
// or 8-byte (bf16) loads, partial or unaligned ones element by element.
constexpr int kWK = 32, kRowLd = kWK + 4, kColLd = 64 + 8, kStage = 64 * kRowLd;
static_assert(kWK * kColLd <= kStage, "both layouts fit one staging array");

__device__ __forceinline__ uint32_t tf32_of(float v) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
  return r;
}
// Raw bits of four consecutive elements (fp32: four words; bf16: two words) and of one element, as they come from
// memory, and their TF32 operand form.  Loading and converting are separate steps so that a tile fetched ahead costs no
// wait until it is stored to shared memory.
__device__ __forceinline__ uint4 raw4(const float* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ uint4 raw4(const bf16* p) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  return make_uint4(v.x, v.y, 0u, 0u);
}
__device__ __forceinline__ uint32_t raw1(const float* p) { return __float_as_uint(*p); }
__device__ __forceinline__ uint32_t raw1(const bf16* p) { return *reinterpret_cast<const unsigned short*>(p); }
template <typename TX> __device__ __forceinline__ uint4 tf32_of4(uint4 r);
template <> __device__ __forceinline__ uint4 tf32_of4<float>(uint4 r) {
  return make_uint4(tf32_of(__uint_as_float(r.x)), tf32_of(__uint_as_float(r.y)), tf32_of(__uint_as_float(r.z)),
                    tf32_of(__uint_as_float(r.w)));
}
template <> __device__ __forceinline__ uint4 tf32_of4<bf16>(uint4 r) {
  return make_uint4(r.x << 16, r.x & 0xFFFF0000u, r.y << 16, r.y & 0xFFFF0000u);
}
template <typename TX> __device__ __forceinline__ uint32_t tf32_of1(uint32_t r);
template <> __device__ __forceinline__ uint32_t tf32_of1<float>(uint32_t r) { return tf32_of(__uint_as_float(r)); }
template <> __device__ __forceinline__ uint32_t tf32_of1<bf16>(uint32_t r) { return r << 16; }
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A 64 x kWK tile of an operand X, rows r0 .. (bound R), contraction indices k0 .. (bound k_hi), with
// X(r, k) = k_major ? X[k ld + r] : X[r ld + k], travels in two steps so that the global loads of the next tile are in
// flight while the current one is multiplied: fetch_tile brings a thread's eight elements into registers as they are,
// put_tile rounds them to TF32 and stores them.  Shared layout: k_major ? [k][kColLd] : [r][kRowLd].  Aligned tiles with
// all 32 contraction indices in range move as two 16-byte (fp32) or 8-byte (bf16) loads and two 16-byte stores per thread
// (groups of four past the last row are zeros), the others element by element.
__device__ __forceinline__ bool tile_is_full(bool aligned, int r0, int R, int k0, int k_hi) {
  (void)r0;                                // rows past R are left out group by group (R is then a multiple of 4)
  return aligned && R % 4 == 0 && k0 + kWK <= k_hi;
}
template <typename TX>
__device__ __forceinline__ void fetch_tile(uint32_t (&v)[8], const TX* __restrict__ X, int ld, int k_major, int r0, int R,
                                           int k0, int k_hi, bool aligned, int tid) {
  if (tile_is_full(aligned, r0, R, k0, k_hi)) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int i = tid + kGemmThreads * j;
      const int r = r0 + (k_major ? (i & 15) * 4 : (i >> 3));
      const TX* src = k_major ? X + (size_t)(k0 + (i >> 4)) * ld + r : X + (size_t)r * ld + k0 + (i & 7) * 4;
      const uint4 q = r < R ? raw4(src) : make_uint4(0u, 0u, 0u, 0u);
      v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
    }
    return;
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int i = tid + kGemmThreads * e;
    const int rr = k_major ? (i & 63) : (i / kWK), kk = k_major ? (i >> 6) : (i % kWK);
    const int r = r0 + rr, k = k0 + kk;
    v[e] = (r < R && k < k_hi) ? raw1(k_major ? X + (size_t)k * ld + r : X + (size_t)r * ld + k) : 0u;
  }
}
template <typename TX>
__device__ __forceinline__ void put_tile(uint32_t* __restrict__ sm, const uint32_t (&v)[8], int k_major, bool full, int tid) {
  if (full) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int i = tid + kGemmThreads * j;
      uint32_t* dst = k_major ? sm + (i >> 4) * kColLd + (i & 15) * 4 : sm + (i >> 3) * kRowLd + (i & 7) * 4;
      *reinterpret_cast<uint4*>(dst) = tf32_of4<TX>(make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]));
    }
    return;
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int i = tid + kGemmThreads * e;
    const int rr = k_major ? (i & 63) : (i / kWK), kk = k_major ? (i >> 6) : (i % kWK);
    sm[k_major ? kk * kColLd + rr : rr * kRowLd + kk] = tf32_of1<TX>(v[e]);
  }
}

template <typename TA, typename TB>
__global__ void __launch_bounds__(kGemmThreads, 2)
gemm_tf32_kernel(int M, int N, int K, const TA* __restrict__ A, int lda, int ta, const TB* __restrict__ B, int ldb, int tb,
                 float* __restrict__ C, int ldc, float alpha, int accumulate, int k_per_split, int aligned_a, int aligned_b,
                 int tiles_n, int sa, int sb, int sc) {
  __shared__ __align__(16) uint32_t As[kStage], Bs[kStage];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int batch = blockIdx.y;
  A += (size_t)batch * sa;
  B += (size_t)batch * sb;
  C += (size_t)batch * sc;
  const int tile_m = blockIdx.x / tiles_n, m0 = tile_m * 64, n0 = (blockIdx.x - tile_m * tiles_n) * 64;
  const int k_lo = blockIdx.z * k_per_split, k_hi = min(K, k_lo + k_per_split);
  const int wm = (warp >> 2) * 32, wn = (warp & 3) * 16;
  // element offsets of this lane's fragment entries: A(m, k) with m = wm + g, k = t;  B(k, n) with k = t, n = wn + g
  const int a_m = ta ? 1 : kRowLd, a_k = ta ? kColLd : 1, b_n = tb ? kRowLd : 1, b_k = tb ? 1 : kColLd;
  const int a_off = (wm + g) * a_m + t * a_k, b_off = (wn + g) * b_n + t * b_k;
  float acc[2][2][4] = {};
  uint32_t va[8], vb[8];                  // A(m, k): k-major storage when transposed;  B(k, n): k-major when NOT transposed
  fetch_tile<TA>(va, A, lda, ta, m0, M, k_lo, k_hi, aligned_a != 0, tid);
  fetch_tile<TB>(vb, B, ldb, !tb, n0, N, k_lo, k_hi, aligned_b != 0, tid);
  for (int k0 = k_lo; k0 < k_hi; k0 += kWK) {
    put_tile<TA>(As, va, ta, tile_is_full(aligned_a != 0, m0, M, k0, k_hi), tid);
    put_tile<TB>(Bs, vb, !tb, tile_is_full(aligned_b != 0, n0, N, k0, k_hi), tid);
    __syncthreads();
    if (k0 + kWK < k_hi) {
      fetch_tile<TA>(va, A, lda, ta, m0, M, k0 + kWK, k_hi, aligned_a != 0, tid);
      fetch_tile<TB>(vb, B, ldb, !tb, n0, N, k0 + kWK, k_hi, aligned_b != 0, tid);
    }
#pragma unroll
    for (int kb = 0; kb < kWK; kb += 8) {
      uint32_t a[2][4], b[2][2];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t* pa = As + a_off + mt * 16 * a_m + kb * a_k;
        a[mt][0] = pa[0];
        a[mt][1] = pa[8 * a_m];
        a[mt][2] = pa[4 * a_k];
        a[mt][3] = pa[8 * a_m + 4 * a_k];
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const uint32_t* pb = Bs + b_off + nt * 8 * b_n + kb * b_k;
        b[nt][0] = pb[0];
        b[nt][1] = pb[4 * b_k];
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) mma_tf32(acc[mt][nt], a[mt], b[nt][0], b[nt][1]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int m = m0 + wm + mt * 16 + g + (e >> 1) * 8, n = n0 + wn + nt * 8 + 2 * t + (e & 1);
        if (m >= M || n >= N) continue;
        float* c = C + (size_t)m * ldc + n;
        const float v = alpha * acc[mt][nt][e];
        if (gridDim.z > 1 || accumulate) atomicAdd(c, v);      // (one add per element when K is not split: the result is
        else *c = v;                                           //  the same, and the thread does not wait for the old value)
      }
}

// Products with very many rows and a small second operand, C[M x N] (+)= alpha A[M x K] B(K, N) with N, K <= 128: what
// the generic kernel above does badly (a block lives for K / 32 steps, reads B again for every tile of rows and never has
// more than one step in flight).  Here a block stays: it stages B once (TF32, k-major, pitch N + 8), then walks tiles of
// 128 rows, whose A rows arrive by cp.async as they are (fp32 or bf16, row pitch of K + 4 words or K + 8 halves) into one
// of two buffers while the previous tile is multiplied; A is rounded to TF32 when a fragment is read.  Eight warps of
// 32 rows x N / 2 columns.
constexpr int kRowsTile = 128;
template <typename TA> struct RowsPitch;
template <> struct RowsPitch<float> { static __host__ __device__ int elems(int K) { return K + 4; } };
template <> struct RowsPitch<bf16> { static __host__ __device__ int elems(int K) { return K + 8; } };
__device__ __forceinline__ uint32_t frag_of(const float* p) { return tf32_of(*p); }
__device__ __forceinline__ uint32_t frag_of(const bf16* p) {
  return static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(p)) << 16;
}

template <typename TA, typename TB, int N>
__global__ void __launch_bounds__(kGemmThreads)
rows_gemm_kernel(int M, int K, const TA* __restrict__ A, int lda, const TB* __restrict__ B, int ldb, int tb,
                 float* __restrict__ C, bf16* __restrict__ C16, int ldc, float alpha, int accumulate, int n_tiles) {
  constexpr int WN = N / 2, NTW = WN / 8, BP = N + 8;
  extern __shared__ __align__(16) unsigned char rg_smem[];
  uint32_t* Bs = reinterpret_cast<uint32_t*>(rg_smem);                       // [K][BP]
  const int ap = RowsPitch<TA>::elems(K);
  TA* As = reinterpret_cast<TA*>(rg_smem + (size_t)K * BP * sizeof(uint32_t));    // [2][128][ap]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  constexpr int kPer16 = 16 / (int)sizeof(TA);                               // elements per 16-byte copy
  const int chunks_per_row = K / kPer16, chunks = kRowsTile * chunks_per_row;
  auto stage = [&](int tile, int buf) {
    TA* dst = As + (size_t)buf * kRowsTile * ap;
    const int r0 = tile * kRowsTile;
    for (int x = tid; x < chunks; x += kGemmThreads) {
      const int rr = x / chunks_per_row, ch = x - rr * chunks_per_row;
      const int r = r0 + rr;
      mma::cp16(mma::smem_addr(dst + (size_t)rr * ap + ch * kPer16), A + (size_t)min(r, M - 1) * lda + ch * kPer16,
                r < M ? 16u : 0u);
    }
    mma::cp_commit();
  };
  int tile = blockIdx.x;
  if (tile < n_tiles) stage(tile, 0);
  for (int i = tid; i < K * N; i += kGemmThreads) {
    const int k = i / N, n = i - k * N;
    Bs[k * BP + n] = tf32_of(to_f32<TB>(tb ? B[(size_t)n * ldb + k] : B[(size_t)k * ldb + n]));
  }
  const int wr = (warp >> 1) * 32, wc = (warp & 1) * WN;
  int buf = 0;
  for (; tile < n_tiles; tile += gridDim.x, buf ^= 1) {
    const int next = tile + gridDim.x;
    if (next < n_tiles) {
      stage(next, buf ^ 1);
      mma::cp_wait<1>();
    } else {
      mma::cp_wait<0>();
    }
    __syncthreads();
    const TA* At = As + (size_t)buf * kRowsTile * ap;
    float acc[2][NTW][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
    for (int kb = 0; kb < K; kb += 8) {
      uint32_t a[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const TA* pa = At + (size_t)(wr + mt * 16 + g) * ap + kb + t;
        a[mt][0] = frag_of(pa);
        a[mt][1] = frag_of(pa + 8 * ap);
        a[mt][2] = frag_of(pa + 4);
        a[mt][3] = frag_of(pa + 8 * ap + 4);
      }
      const uint32_t* pb = Bs + (kb + t) * BP + wc + g;
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const uint32_t b0 = pb[nt * 8], b1 = pb[4 * BP + nt * 8];
        mma_tf32(acc[0][nt], a[0], b0, b1);
        mma_tf32(acc[1][nt], a[1], b0, b1);
      }
    }
    const int r0 = tile * kRowsTile + wr;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = r0 + mt * 16 + g + h * 8;
        if (r >= M) continue;
        const size_t at = (size_t)r * ldc + wc + 2 * t;
        float* c = C + at;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          const float v0 = alpha * acc[mt][nt][2 * h], v1 = alpha * acc[mt][nt][2 * h + 1];
          if (C16) {                               // (the result is wanted as bf16 only)
            *reinterpret_cast<uint32_t*>(C16 + at + nt * 8) = mma::pack2(v0, v1);
          } else if (accumulate) {
            atomicAdd(c + nt * 8, v0);
            atomicAdd(c + nt * 8 + 1, v1);
          } else {
            *reinterpret_cast<float2*>(c + nt * 8) = make_float2(v0, v1);
          }
        }
      }
    __syncthreads();                     // the buffer just read is the next one to be filled
  }
}

int bwd_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  return n;
}

template <typename TA, typename TB>
bool rows_gemm_fits(int M, int N, int K, const TA* A, int lda, const float* C, int ldc) {
  constexpr int per16 = 16 / (int)sizeof(TA);
  return M >= 32768 && (N == 32 || N == 64 || N == 128) && K >= 8 && K <= 128 && K % per16 == 0 && K % 8 == 0 &&
         lda % per16 == 0 && reinterpret_cast<uintptr_t>(A) % 16 == 0 && ldc % 2 == 0 &&
         reinterpret_cast<uintptr_t>(C) % 8 == 0;
}

template <typename TA, typename TB, int N>
int launch_rows_gemm(cudaStream_t st, int M, int K, const TA* A, int lda, const TB* B, int ldb, bool tb, float* C, int ldc,
                     float alpha, bool accumulate, bf16* C16 = nullptr) {
  const size_t smem = (size_t)K * (N + 8) * sizeof(uint32_t) + 2 * (size_t)kRowsTile * RowsPitch<TA>::elems(K) * sizeof(TA);
  auto kernel = rows_gemm_kernel<TA, TB, N>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int n_tiles = (M + kRowsTile - 1) / kRowsTile;
  const int per_sm = smem <= 100 * 1024 ? 2 : 1;
  LaunchScope ls("bwd_gemm_rows", st);
  kernel<<<std::min(n_tiles, per_sm * bwd_sm_count()), kGemmThreads, smem, st>>>(M, K, A, lda, B, ldb, tb ? 1 : 0, C, C16, ldc,
                                                                              alpha, accumulate ? 1 : 0, n_tiles);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

// Reductions over very many rows into a small matrix, C[MO x N] += alpha sum_r A[r][m] B[r][n] (the weight gradients
// dW = X^T dY): a block stays, takes one contiguous slice of the rows, streams 32 rows of A and of B at a time (cp.async,
// two buffers, as they are: the row index is the contraction index, so both land k-major) and keeps its MO x N partial
// sum in registers until the end: one atomic add per element and block instead of one per element and 256 rows.
template <typename TA, typename TB, int MO, int N>
__global__ void __launch_bounds__(kGemmThreads)
cols_gemm_kernel(int R, const TA* __restrict__ A, int lda, const TB* __restrict__ B, int ldb, float* __restrict__ C, int ldc,
                 float alpha, int rows_per_block) {
  constexpr int WARPS_M = MO / 32, WARPS_N = 8 / WARPS_M, WN = N / WARPS_N, NTW = WN / 8;
  constexpr int AP = MO + 16 / (int)sizeof(TA) * 2, BPT = N + 32 / (int)sizeof(TB);     // pitches in elements
  static_assert(WN % 8 == 0 && NTW >= 1, "warp tiles of whole 8-column MMA tiles");
  extern __shared__ __align__(16) unsigned char cg_smem[];
  TA* As = reinterpret_cast<TA*>(cg_smem);                                    // [2][32][AP]
  TB* Bs = reinterpret_cast<TB*>(cg_smem + 2 * 32 * AP * sizeof(TA));         // [2][32][BPT]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int r_lo = blockIdx.x * rows_per_block, r_hi = min(R, r_lo + rows_per_block);
  constexpr int a16 = 16 / (int)sizeof(TA), b16 = 16 / (int)sizeof(TB);
  constexpr int a_chunks = 32 * MO / a16, b_chunks = 32 * N / b16;
  auto stage = [&](int r0, int buf) {
    TA* da = As + buf * 32 * AP;
    TB* db = Bs + buf * 32 * BPT;
    for (int x = tid; x < a_chunks; x += kGemmThreads) {
      const int rr = x / (MO / a16), ch = x - rr * (MO / a16), r = r0 + rr;
      mma::cp16(mma::smem_addr(da + rr * AP + ch * a16), A + (size_t)min(r, R - 1) * lda + ch * a16, r < r_hi ? 16u : 0u);
    }
    for (int x = tid; x < b_chunks; x += kGemmThreads) {
      const int rr = x / (N / b16), ch = x - rr * (N / b16), r = r0 + rr;
      mma::cp16(mma::smem_addr(db + rr * BPT + ch * b16), B + (size_t)min(r, R - 1) * ldb + ch * b16, r < r_hi ? 16u : 0u);
    }
    mma::cp_commit();
  };
  const int wm = (warp / WARPS_N) * 32, wn = (warp % WARPS_N) * WN;
  float acc[2][NTW][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
  if (r_lo < r_hi) stage(r_lo, 0);
  int buf = 0;
  for (int r0 = r_lo; r0 < r_hi; r0 += 32, buf ^= 1) {
    if (r0 + 32 < r_hi) {
      stage(r0 + 32, buf ^ 1);
      mma::cp_wait<1>();
    } else {
      mma::cp_wait<0>();
    }
    __syncthreads();
    const TA* Ak = As + buf * 32 * AP;
    const TB* Bk = Bs + buf * 32 * BPT;
#pragma unroll
    for (int kb = 0; kb < 32; kb += 8) {
      uint32_t a[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const TA* pa = Ak + (kb + t) * AP + wm + mt * 16 + g;
        a[mt][0] = frag_of(pa);
        a[mt][1] = frag_of(pa + 8);
        a[mt][2] = frag_of(pa + 4 * AP);
        a[mt][3] = frag_of(pa + 4 * AP + 8);
      }
      const TB* pb = Bk + (kb + t) * BPT + wn + g;
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const uint32_t b0 = frag_of(pb + nt * 8), b1 = frag_of(pb + 4 * BPT + nt * 8);
        mma_tf32(acc[0][nt], a[0], b0, b1);
        mma_tf32(acc[1][nt], a[1], b0, b1);
      }
    }
    __syncthreads();
  }
  if (r_lo >= r_hi) return;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int m = wm + mt * 16 + g + (e >> 1) * 8, n = wn + nt * 8 + 2 * t + (e & 1);
        atomicAdd(C + (size_t)m * ldc + n, alpha * acc[mt][nt][e]);
      }
}

template <typename TA, typename TB>
bool cols_gemm_fits(int M, int N, int K, const TA* A, int lda, const TB* B, int ldb) {
  return K >= 32768 && (M == 64 || M == 128) && (N == 32 || N == 64 || N == 128) &&
         lda % (16 / (int)sizeof(TA)) == 0 && ldb % (16 / (int)sizeof(TB)) == 0 &&
         reinterpret_cast<uintptr_t>(A) % 16 == 0 && reinterpret_cast<uintptr_t>(B) % 16 == 0;
}

template <typename TA, typename TB, int MO, int N>
int launch_cols_gemm(cudaStream_t st, int R, const TA* A, int lda, const TB* B, int ldb, float* C, int ldc, float alpha) {
  constexpr int AP = MO + 16 / (int)sizeof(TA) * 2, BPT = N + 32 / (int)sizeof(TB);
  const size_t smem = 2 * 32 * ((size_t)AP * sizeof(TA) + (size_t)BPT * sizeof(TB));
  auto kernel = cols_gemm_kernel<TA, TB, MO, N>;
  LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int blocks_max = 2 * bwd_sm_count();
  const int per = ((R + blocks_max - 1) / blocks_max + 31) / 32 * 32;
  LaunchScope ls("bwd_gemm_cols", st);
  kernel<<<(R + per - 1) / per, kGemmThreads, smem, st>>>(R, A, lda, B, ldb, C, ldc, alpha, per);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

template <typename TA, typename TB, int MO>
int launch_cols_gemm_n(cudaStream_t st, int N, int R, const TA* A, int lda, const TB* B, int ldb, float* C, int ldc,
                       float alpha) {
  if (N == 32) return launch_cols_gemm<TA, TB, MO, 32>(st, R, A, lda, B, ldb, C, ldc, alpha);
  if (N == 64) return launch_cols_gemm<TA, TB, MO, 64>(st, R, A, lda, B, ldb, C, ldc, alpha);
  return launch_cols_gemm<TA, TB, MO, 128>(st, R, A, lda, B, ldb, C, ldc, alpha);
}

// Where a product runs: the stream, and whether on the tensor cores (TF32) or on the FP32 ALUs.
struct GemmCtx {
  cudaStream_t st;
  bool tf32;
};

template <typename TX>
bool aligned_for_vector_loads(const TX* X, int ld) {
  return ld % 4 == 0 && reinterpret_cast<uintptr_t>(X) % (4 * sizeof(TX)) == 0;
}

template <typename TA, typename TB>
int gemm(const GemmCtx& gx, int M, int N, int K, const TA* A, int lda, bool ta, const TB* B, int ldb, bool tb, float* C,
         int ldc, float alpha, bool accumulate, bool split_k, int batch = 1, int sa = 0, int sb = 0, int sc = 0) {
  if (M <= 0 || N <= 0 || K <= 0 || batch <= 0) return LASER_OK;
  cudaStream_t st = gx.st;
  if (gx.tf32 && !ta && !split_k && batch == 1 && rows_gemm_fits<TA, TB>(M, N, K, A, lda, C, ldc)) {
    if (N == 32) return launch_rows_gemm<TA, TB, 32>(st, M, K, A, lda, B, ldb, tb, C, ldc, alpha, accumulate);
    if (N == 64) return launch_rows_gemm<TA, TB, 64>(st, M, K, A, lda, B, ldb, tb, C, ldc, alpha, accumulate);
    return launch_rows_gemm<TA, TB, 128>(st, M, K, A, lda, B, ldb, tb, C, ldc, alpha, accumulate);
  }
  if (gx.tf32 && ta && !tb && split_k && batch == 1 && cols_gemm_fits<TA, TB>(M, N, K, A, lda, B, ldb)) {
    if (M == 64) return launch_cols_gemm_n<TA, TB, 64>(st, N, K, A, lda, B, ldb, C, ldc, alpha);
    return launch_cols_gemm_n<TA, TB, 128>(st, N, K, A, lda, B, ldb, C, ldc, alpha);
  }
  const int kstep = gx.tf32 ? kWK : kTK;
  int splits = 1, per = K;
  if (split_k) {                     // reductions over many rows into a small matrix (C must hold its initial value)
    // slices of at least 256 rows, longer when that still leaves about four blocks per SM (fewer atomic adds per product)
    const long long tiles = (long long)((M + kTM - 1) / kTM) * ((N + kTN - 1) / kTN) * batch;
    per = (int)std::min<long long>(std::max<long long>(256, ((long long)K * tiles / 592 + 31) / 32 * 32), 1 << 20);
    splits = (K + per - 1) / per;
    if (splits > 65535) { splits = 65535; per = (K + splits - 1) / splits; per = (per + kstep - 1) / kstep * kstep; splits = (K + per - 1) / per; }
  }
  const int tiles_n = (N + kTN - 1) / kTN;
  const long long tiles = (long long)((M + kTM - 1) / kTM) * tiles_n;
  if (batch > 65535 || tiles > 0x7fffffffLL) return LASER_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)tiles, batch, splits);
  LaunchScope ls(gx.tf32 ? "bwd_gemm_tf32" : "bwd_gemm", st);
  if (gx.tf32)
    gemm_tf32_kernel<TA, TB><<<grid, kGemmThreads, 0, st>>>(
        M, N, K, A, lda, ta ? 1 : 0, B, ldb, tb ? 1 : 0, C, ldc, alpha, accumulate ? 1 : 0, per,
        aligned_for_vector_loads(A, lda) && sa % 4 == 0 ? 1 : 0, aligned_for_vector_loads(B, ldb) && sb % 4 == 0 ? 1 : 0,
        tiles_n, sa, sb, sc);
  else
    gemm_kernel<TA, TB><<<grid, kGemmThreads, 0, st>>>(M, N, K, A, lda, ta ? 1 : 0, B, ldb, tb ? 1 : 0, C, ldc, alpha,
                                                      accumulate ? 1 : 0, per, tiles_n, sa, sb, sc);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

// C16 [M x N] (bf16) = A [M x K] B [K x N] on the persistent rows kernel, for results that are only ever read as bf16 MMA
// operands; LASER_ERR_UNSUPPORTED when the shape does not fit that kernel (the caller then takes the fp32 product and a copy).
template <typename TA, typename TB>
int gemm_rows_bf16(const GemmCtx& gx, int M, int N, int K, const TA* A, int lda, const TB* B, int ldb, bf16* C16, int ldc) {
  if (!gx.tf32 || !rows_gemm_fits<TA, TB>(M, N, K, A, lda, reinterpret_cast<const float*>(C16), ldc) ||
      reinterpret_cast<uintptr_t>(C16) % 4 != 0)
    return LASER_ERR_UNSUPPORTED;
  if (N == 32) return launch_rows_gemm<TA, TB, 32>(gx.st, M, K, A, lda, B, ldb, false, nullptr, ldc, 1.f, false, C16);
  if (N == 64) return launch_rows_gemm<TA, TB, 64>(gx.st, M, K, A, lda, B, ldb, false, nullptr, ldc, 1.f, false, C16);
  return launch_rows_gemm<TA, TB, 128>(gx.st, M, K, A, lda, B, ldb, false, nullptr, ldc, 1.f, false, C16);
}

template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, size_t n) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = to_f32<T>(src[i]);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

constexpr int kAttnThreads = 128;

// Non-empty segments of candidate c's user (0 for invalid shapes, which the forward kernels report).
__device__ __forceinline__ int segments_of(const int* lengths, const int* cand_offsets, int U, int L, int S, int Lp, int c) {
  int lo = 0, hi = U - 1;
  while (lo < hi) {                               // the last user whose first candidate is <= c
    const int mid = (lo + hi + 1) >> 1;
    if (cand_offsets[mid] <= c) lo = mid; else hi = mid - 1;
  }
  const int len = lengths[lo];
  if (len <= 0 || len > L) return 0;
  return min((len + S - 1) / S, Lp);
}

// VEC consecutive features of a row (VEC = 4 when d is a multiple of 4: one 16-byte access; else 1).
template <int VEC>
__device__ __forceinline__ void load_vec(float (&v)[VEC], const float* p) {
  if constexpr (VEC == 4) {
    const float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  } else {
    v[0] = *p;
  }
}
template <int VEC>
__device__ __forceinline__ void store_vec(float* p, const float (&v)[VEC]) {
  if constexpr (VEC == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  else *p = v[0];
}

// dot[k] = s_j . W[h0 + k] for HG heads at a time (HG = 4, 2 or 1 divides H: no head of a group is ever missing),
// W = [H][d] in shared memory; lanes split the features.
template <int VEC, int HG>
__device__ __forceinline__ void row_dots(const float* __restrict__ sj, const float* __restrict__ W, int d, int H, int h0,
                                         int lane, float (&dot)[HG]) {
#pragma unroll
  for (int k = 0; k < HG; ++k) dot[k] = 0.f;
  for (int x = VEC * lane; x < d; x += 32 * VEC) {
    float sv[VEC];
    load_vec<VEC>(sv, sj + x);
#pragma unroll
    for (int k = 0; k < HG; ++k) {
      float wv[VEC];
      load_vec<VEC>(wv, W + (h0 + k) * d + x);
#pragma unroll
      for (int v = 0; v < VEC; ++v) dot[k] = fmaf(sv[v], wv[v], dot[k]);
    }
  }
#pragma unroll
  for (int k = 0; k < HG; ++k) dot[k] = warp_sum(dot[k]);
}

// One block per candidate: e_{j,h} = s_j . Qt_h (Qt holds W_k[:, h] Q_h / tau), a = softmax over the non-empty segments,
// m_h = sum_j a_{j,h} s_j.  Writes a [N, H, Lp] and m [N, H, d].  The warps split the segments (a warp reads a segment
// vector once for HG heads, each lane VEC consecutive features); the per-warp partial sums of m meet in shared memory.
template <int VEC, int HG>
__global__ void __launch_bounds__(kAttnThreads)
gsta_attn_fwd_kernel(const float* __restrict__ Hp, const float* __restrict__ Qt, const int* __restrict__ lengths,
                     const int* __restrict__ cand_offsets, float* __restrict__ Aw, float* __restrict__ Mh, int U, int L,
                     int S, int Lp, int H, int d) {
  extern __shared__ __align__(16) float sm[];
  constexpr int nw = kAttnThreads / 32;
  float* qt = sm;                 // [H][d]
  float* red = qt + H * d;        // [nw][H][d]: per-warp partial sums of m
  float* e = red + nw * H * d;    // [H][Lp]
  const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nv = segments_of(lengths, cand_offsets, U, L, S, Lp, c);
  const float* s = Hp + (size_t)c * Lp * d;
  for (int i = tid; i < H * d; i += kAttnThreads) qt[i] = Qt[(size_t)c * H * d + i];
  __syncthreads();
  for (int j = warp; j < nv; j += nw)
    for (int h0 = 0; h0 < H; h0 += HG) {
      float dot[HG];
      row_dots<VEC, HG>(s + (size_t)j * d, qt, d, H, h0, lane, dot);
#pragma unroll
      for (int k = 0; k < HG; ++k)
        if (lane == 0) e[(h0 + k) * Lp + j] = dot[k];
    }
  __syncthreads();
  for (int h = warp; h < H; h += nw) {
    float mx = -INFINITY;
    for (int j = lane; j < nv; j += 32) mx = fmaxf(mx, e[h * Lp + j]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < nv; j += 32) {
      const float pw = expf(e[h * Lp + j] - mx);
      e[h * Lp + j] = pw;
      sum += pw;
    }
    sum = warp_sum(sum);
    const float inv = sum > 0.f ? 1.f / sum : 0.f;
    for (int j = lane; j < Lp; j += 32) {
      const float a = j < nv ? e[h * Lp + j] * inv : 0.f;
      e[h * Lp + j] = a;
      Aw[((size_t)c * H + h) * Lp + j] = a;
    }
  }
  __syncthreads();
  for (int x = VEC * lane; x < d; x += 32 * VEC)
    for (int h0 = 0; h0 < H; h0 += HG) {
      float acc[HG][VEC];
#pragma unroll
      for (int k = 0; k < HG; ++k)
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[k][v] = 0.f;
      const float* sp = s + (size_t)warp * d + x;          // row j of the segment vectors, and column j of the weights
      const float* ep = e + h0 * Lp + warp;
#pragma unroll 2
      for (int j = warp; j < nv; j += nw, sp += nw * d, ep += nw) {
        float sv[VEC];
        load_vec<VEC>(sv, sp);
#pragma unroll
        for (int k = 0; k < HG; ++k) {
          const float a = ep[k * Lp];
#pragma unroll
          for (int v = 0; v < VEC; ++v) acc[k][v] = fmaf(a, sv[v], acc[k][v]);
        }
      }
#pragma unroll
      for (int k = 0; k < HG; ++k)
        store_vec<VEC>(red + ((size_t)warp * H + h0 + k) * d + x, acc[k]);
    }
  __syncthreads();
  for (int i = tid; i < H * d; i += kAttnThreads) {
    float m = 0.f;
#pragma unroll
    for (int w = 0; w < nw; ++w) m += red[(size_t)w * H * d + i];
    Mh[(size_t)c * H * d + i] = m;
  }
}

// One block per candidate: the backward of the kernel above.  dM = dLoss/dm [N, H, d] in; dQt = dLoss/dQt [N, H, d] out;
// dHp [N, Lp, d] accumulates dLoss/ds_j over the layers: the layer processed first (overwrite != 0) writes every entry
// (zeros for the empty segments), the others add.  Same split of the work as in the forward kernel.
template <int VEC, int HG>
__global__ void __launch_bounds__(kAttnThreads)
gsta_attn_bwd_kernel(const float* __restrict__ Hp, const float* __restrict__ Qt, const float* __restrict__ Aw,
                     const float* __restrict__ dM, const int* __restrict__ lengths, const int* __restrict__ cand_offsets,
                     float* __restrict__ dQt, float* __restrict__ dHp, int U, int L, int S, int Lp, int H, int d,
                     int overwrite) {
  extern __shared__ __align__(16) float sm[];
  constexpr int nw = kAttnThreads / 32;
  float* qt = sm;                 // [H][d]
  float* dm = qt + H * d;         // [H][d]
  float* red = dm + H * d;        // [nw][H][d]: per-warp partial sums of dQt
  float* a = red + nw * H * d;    // [H][Lp]
  float* de = a + H * Lp;         // [H][Lp]: first da, then de
  const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nv = segments_of(lengths, cand_offsets, U, L, S, Lp, c);
  const float* s = Hp + (size_t)c * Lp * d;
  for (int i = tid; i < H * d; i += kAttnThreads) {
    qt[i] = Qt[(size_t)c * H * d + i];
    dm[i] = dM[(size_t)c * H * d + i];
  }
  for (int i = tid; i < H * Lp; i += kAttnThreads) a[i] = Aw[(size_t)c * H * Lp + i];
  __syncthreads();
  for (int j = warp; j < nv; j += nw)
    for (int h0 = 0; h0 < H; h0 += HG) {
      float dot[HG];
      row_dots<VEC, HG>(s + (size_t)j * d, dm, d, H, h0, lane, dot);
#pragma unroll
      for (int k = 0; k < HG; ++k)
        if (lane == 0) de[(h0 + k) * Lp + j] = dot[k];
    }
  __syncthreads();
  for (int h = warp; h < H; h += nw) {
    float dotp = 0.f;
    for (int j = lane; j < nv; j += 32) dotp = fmaf(a[h * Lp + j], de[h * Lp + j], dotp);
    dotp = warp_sum(dotp);
    for (int j = lane; j < nv; j += 32) de[h * Lp + j] = a[h * Lp + j] * (de[h * Lp + j] - dotp);
  }
  __syncthreads();
  float* dS = dHp + (size_t)c * Lp * d;
  for (int x = VEC * lane; x < d; x += 32 * VEC) {
    for (int h0 = 0; h0 < H; h0 += HG) {
      // dQt_h[x] = sum_j de_{j,h} s_j[x]: this warp's segments
      float acc[HG][VEC];
#pragma unroll
      for (int k = 0; k < HG; ++k)
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[k][v] = 0.f;
      const float* sp = s + (size_t)warp * d + x;
      const float* dep = de + h0 * Lp + warp;
#pragma unroll 2
      for (int j = warp; j < nv; j += nw, sp += nw * d, dep += nw) {
        float sv[VEC];
        load_vec<VEC>(sv, sp);
#pragma unroll
        for (int k = 0; k < HG; ++k) {
          const float dej = dep[k * Lp];
#pragma unroll
          for (int v = 0; v < VEC; ++v) acc[k][v] = fmaf(dej, sv[v], acc[k][v]);
        }
      }
#pragma unroll
      for (int k = 0; k < HG; ++k)
        store_vec<VEC>(red + ((size_t)warp * H + h0 + k) * d + x, acc[k]);
      // ds_j[x] += sum_h de_{j,h} Qt_h[x] + a_{j,h} dm_h[x]
      float qx[HG][VEC], mx[HG][VEC];
#pragma unroll
      for (int k = 0; k < HG; ++k) {
        load_vec<VEC>(qx[k], qt + (h0 + k) * d + x);
        load_vec<VEC>(mx[k], dm + (h0 + k) * d + x);
      }
      float* out = dS + (size_t)warp * d + x;
      const float* ap = a + h0 * Lp + warp;
      dep = de + h0 * Lp + warp;
      const bool fresh = overwrite && h0 == 0;
#pragma unroll 2
      for (int j = warp; j < nv; j += nw, out += nw * d, dep += nw, ap += nw) {
        float g[VEC];
        if (fresh) {
#pragma unroll
          for (int v = 0; v < VEC; ++v) g[v] = 0.f;
        } else {
          load_vec<VEC>(g, out);
        }
#pragma unroll
        for (int k = 0; k < HG; ++k) {
          const float dej = dep[k * Lp], aj = ap[k * Lp];
#pragma unroll
          for (int v = 0; v < VEC; ++v) g[v] = fmaf(dej, qx[k][v], fmaf(aj, mx[k][v], g[v]));
        }
        store_vec<VEC>(out, g);
      }
    }
    if (overwrite) {                                        // empty segments receive no gradient
      float zero[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) zero[v] = 0.f;
      for (int j = nv + warp; j < Lp; j += nw) store_vec<VEC>(dS + (size_t)j * d + x, zero);
    }
  }
  __syncthreads();
  for (int i = tid; i < H * d; i += kAttnThreads) {
    float q = 0.f;
#pragma unroll
    for (int w = 0; w < nw; ++w) q += red[(size_t)w * H * d + i];
    dQt[(size_t)c * H * d + i] = q;
  }
}

// One block per (user, 32 consecutive items of one segment), thread (item n, head h); the block walks the user's
// candidates, kCandsPerStep at a time between two block-wide barriers.  Qf holds q / gamma, so the score is Qf_h . k_n
// and dQf is the gradient with respect to q / gamma.  dK, dV rows of this chunk are written once (no other block touches
// them); dQf is summed over the chunks atomically: the per-item terms de_n of a step go through shared memory and thread
// (candidate, head, component) adds up its 32 items while the next step's rows are loaded.
constexpr int kChunk = 32;
constexpr int kCandsPerStep = 4;
// DQH, DVH > 0: the head widths are compile-time constants and thread (item, head) keeps its key / value slices and
// their gradient accumulators in registers (shared memory then holds only the keys for the query-side sums and the
// step's candidate rows); 0, 0: any widths, everything in shared memory.
template <int DQH, int DVH>
__global__ void sta_bwd_kernel(const float* __restrict__ Qf, const float* __restrict__ Kf, const float* __restrict__ Vf,
                               const float* __restrict__ dHp, const int* __restrict__ lengths,
                               const int* __restrict__ cand_offsets, float* __restrict__ dQf, float* __restrict__ dKf,
                               float* __restrict__ dVf, int L, int d, int dqk, int H, int S, int Lp, int N,
                               int chunks_per_seg) {
  constexpr bool kRegs = DQH > 0;
  constexpr int kR = kRegs ? DQH : 1, kV = kRegs ? DVH : 1;
  extern __shared__ __align__(16) float sm[];
  const int u = blockIdx.y, seg = blockIdx.x / chunks_per_seg, ck = blockIdx.x - seg * chunks_per_seg;
  const int len = lengths[u], off0 = cand_offsets[u], off1 = cand_offsets[u + 1];
  if (len <= 0 || len > L || off0 < 0 || off1 <= off0 || off1 > N) return;
  const int n0 = seg * S + ck * kChunk, n_end = min(min((seg + 1) * S, L), len);
  if (n0 >= n_end) return;
  const int cnt = min(kChunk, n_end - n0);
  const int dqh = kRegs ? DQH : dqk / H, dvh = kRegs ? DVH : d / H, kld = dqk + 1, vld = d + 1;
  float* Ks = sm;                                                  // [32][dqk + 1]
  float* Vs = Ks + kChunk * kld;                                   // [32][d + 1]      (shared-memory variant only)
  float* dKs = Vs + (kRegs ? 0 : kChunk * vld);                    // [32][dqk + 1]    (shared-memory variant only)
  float* dVs = dKs + (kRegs ? 0 : kChunk * kld);                   // [32][d + 1]      (shared-memory variant only)
  float* qs = dVs + (kRegs ? 0 : kChunk * vld);                    // [kCandsPerStep][dqk]
  float* ds = qs + kCandsPerStep * dqk;                            // [kCandsPerStep][d]
  float* des = ds + kCandsPerStep * d;                             // [kCandsPerStep][H][33]: de of (candidate, head, item)
  const int tid = threadIdx.x, nt = blockDim.x, n = tid & 31, h = tid >> 5;
  for (int i = tid; i < kChunk * dqk; i += nt) {
    const int r = i / dqk, a = i - r * dqk;
    Ks[r * kld + a] = r < cnt ? Kf[((size_t)u * L + n0 + r) * dqk + a] : 0.f;
    if (!kRegs) dKs[r * kld + a] = 0.f;
  }
  if (!kRegs) {
    for (int i = tid; i < kChunk * d; i += nt) {
      const int r = i / d, a = i - r * d;
      Vs[r * vld + a] = r < cnt ? Vf[((size_t)u * L + n0 + r) * d + a] : 0.f;
      dVs[r * vld + a] = 0.f;
    }
  }
  float kreg[kR], vreg[kV], dk[kR], dv[kV];
  if (kRegs) {
    const bool live = h < H && n < cnt;
    const float4* kp = reinterpret_cast<const float4*>(Kf + ((size_t)u * L + n0 + n) * dqk + h * dqh);
    const float4* vp = reinterpret_cast<const float4*>(Vf + ((size_t)u * L + n0 + n) * d + h * dvh);
#pragma unroll
    for (int a = 0; a < kR / 4; ++a) {
      const float4 x = live ? kp[a] : make_float4(0.f, 0.f, 0.f, 0.f);
      kreg[4 * a] = x.x; kreg[4 * a + 1] = x.y; kreg[4 * a + 2] = x.z; kreg[4 * a + 3] = x.w;
    }
#pragma unroll
    for (int v = 0; v < kV / 4; ++v) {
      const float4 x = live ? vp[v] : make_float4(0.f, 0.f, 0.f, 0.f);
      vreg[4 * v] = x.x; vreg[4 * v + 1] = x.y; vreg[4 * v + 2] = x.z; vreg[4 * v + 3] = x.w;
    }
#pragma unroll
    for (int a = 0; a < kR; ++a) dk[a] = 0.f;
#pragma unroll
    for (int v = 0; v < kV; ++v) dv[v] = 0.f;
  }
  // the query-side sums of the step whose de terms sit in `des`: candidates c_lo .. c_lo + n_c - 1
  auto reduce_dq = [&](int c_lo, int n_c) {
    for (int i = tid; i < n_c * dqk; i += nt) {
      const int cc = i / dqk, col = i - cc * dqk, hh = col / dqh;
      const float* e = des + (cc * H + hh) * 33;
      float acc = 0.f;
#pragma unroll 8
      for (int r = 0; r < kChunk; ++r) acc = fmaf(e[r], Ks[r * kld + col], acc);
      atomicAdd(dQf + (size_t)(c_lo + cc) * dqk + col, acc);
    }
  };
  int prev_lo = 0, prev_n = 0;
  for (int c = off0; c < off1; c += kCandsPerStep) {
    const int n_c = min(kCandsPerStep, off1 - c);
    __syncthreads();                       // the previous step's de terms are complete; its q and ds rows are free
    if (prev_n > 0) reduce_dq(prev_lo, prev_n);
    for (int i = tid; i < n_c * dqk; i += nt) qs[i] = Qf[(size_t)c * dqk + i];
    for (int i = tid; i < n_c * d; i += nt) {
      const int cc = i / d, x = i - cc * d;
      ds[i] = dHp[((size_t)(c + cc) * Lp + seg) * d + x];
    }
    __syncthreads();                       // (also: the previous step's sums have been read out of `des`)
    if (h < H) {
      for (int cc = 0; cc < n_c; ++cc) {
        const float* q = qs + cc * dqk + h * dqh;
        const float* g_out = ds + cc * d + h * dvh;
        float e = 0.f, dg = 0.f;
        if (kRegs) {
          float qv[kR], gv[kV];
#pragma unroll
          for (int a = 0; a < kR / 4; ++a) {
            const float4 x = reinterpret_cast<const float4*>(q)[a];
            qv[4 * a] = x.x; qv[4 * a + 1] = x.y; qv[4 * a + 2] = x.z; qv[4 * a + 3] = x.w;
          }
#pragma unroll
          for (int v = 0; v < kV / 4; ++v) {
            const float4 x = reinterpret_cast<const float4*>(g_out)[v];
            gv[4 * v] = x.x; gv[4 * v + 1] = x.y; gv[4 * v + 2] = x.z; gv[4 * v + 3] = x.w;
          }
#pragma unroll
          for (int a = 0; a < kR; ++a) e = fmaf(qv[a], kreg[a], e);
#pragma unroll
          for (int v = 0; v < kV; ++v) dg = fmaf(gv[v], vreg[v], dg);
          const float g = n < cnt ? 1.f / (1.f + expf(-e)) : 0.f;
          const float de = dg * g * (1.f - g);
#pragma unroll
          for (int v = 0; v < kV; ++v) dv[v] = fmaf(g, gv[v], dv[v]);
#pragma unroll
          for (int a = 0; a < kR; ++a) dk[a] = fmaf(de, qv[a], dk[a]);
          des[(cc * H + h) * 33 + n] = de;
        } else {
          for (int a = 0; a < dqh; ++a) e = fmaf(q[a], Ks[n * kld + h * dqh + a], e);
          for (int v = 0; v < dvh; ++v) dg = fmaf(g_out[v], Vs[n * vld + h * dvh + v], dg);
          const float g = n < cnt ? 1.f / (1.f + expf(-e)) : 0.f;
          const float de = dg * g * (1.f - g);
          for (int v = 0; v < dvh; ++v) dVs[n * vld + h * dvh + v] = fmaf(g, g_out[v], dVs[n * vld + h * dvh + v]);
          for (int a = 0; a < dqh; ++a) dKs[n * kld + h * dqh + a] = fmaf(de, q[a], dKs[n * kld + h * dqh + a]);
          des[(cc * H + h) * 33 + n] = de;
        }
      }
    }
    prev_lo = c;
    prev_n = n_c;
  }
  __syncthreads();
  if (prev_n > 0) reduce_dq(prev_lo, prev_n);
  if (kRegs) {
    if (h < H && n < cnt) {
      float4* kp = reinterpret_cast<float4*>(dKf + ((size_t)u * L + n0 + n) * dqk + h * dqh);
      float4* vp = reinterpret_cast<float4*>(dVf + ((size_t)u * L + n0 + n) * d + h * dvh);
#pragma unroll
      for (int a = 0; a < kR / 4; ++a) kp[a] = make_float4(dk[4 * a], dk[4 * a + 1], dk[4 * a + 2], dk[4 * a + 3]);
#pragma unroll
      for (int v = 0; v < kV / 4; ++v) vp[v] = make_float4(dv[4 * v], dv[4 * v + 1], dv[4 * v + 2], dv[4 * v + 3]);
    }
  } else {
    for (int i = tid; i < cnt * dqk; i += nt) {
      const int r = i / dqk, a = i - r * dqk;
      dKf[((size_t)u * L + n0 + r) * dqk + a] = dKs[r * kld + a];
    }
    for (int i = tid; i < cnt * d; i += nt) {
      const int r = i / d, a = i - r * d;
      dVf[((size_t)u * L + n0 + r) * d + a] = dVs[r * vld + a];
    }
  }
}

// H' in fp32 for the backward's forward recomputation, head widths known at compile time: one block per (segment, 32
// candidates, user), thread (candidate, head) with its query slice and its accumulators in registers; the segment's
// items pass through shared memory 32 at a time and every lane reads them as 128-bit broadcasts.  (Other head widths
// use the forward's own FP32 kernel.)
template <int DQH, int DVH>
__global__ void sta_fwd32_kernel(const float* __restrict__ Qf, const float* __restrict__ Kf, const float* __restrict__ Vf,
                                 const int* __restrict__ lengths, const int* __restrict__ cand_offsets,
                                 float* __restrict__ Hp, int L, int d, int dqk, int H, int S, int Lp, int N) {
  extern __shared__ __align__(16) float sm[];
  float* Ks = sm;                        // [32][dqk]
  float* Vs = Ks + kChunk * dqk;         // [32][d]
  const int u = blockIdx.z, seg = blockIdx.x;
  const int len = lengths[u], off0 = cand_offsets[u], off1 = cand_offsets[u + 1];
  if (len < 0 || len > L || off0 < 0 || off1 < off0 || off1 > N) return;
  const int c0 = off0 + blockIdx.y * 32;
  if (c0 >= off1) return;
  const int tid = threadIdx.x, nt = blockDim.x, ci = tid & 31, h = tid >> 5, c = c0 + ci;
  const bool live = c < off1 && h < H;
  float q[DQH], acc[DVH];
#pragma unroll
  for (int a = 0; a < DQH / 4; ++a) {
    const float4 x = live ? reinterpret_cast<const float4*>(Qf + (size_t)c * dqk + h * DQH)[a] : make_float4(0.f, 0.f, 0.f, 0.f);
    q[4 * a] = x.x; q[4 * a + 1] = x.y; q[4 * a + 2] = x.z; q[4 * a + 3] = x.w;
  }
#pragma unroll
  for (int v = 0; v < DVH; ++v) acc[v] = 0.f;
  const int n_begin = seg * S, n_end = min(min(n_begin + S, L), len);
  for (int nb = n_begin; nb < n_end; nb += kChunk) {
    const int cnt = min(kChunk, n_end - nb);
    __syncthreads();
    for (int i = tid; i < cnt * dqk / 4; i += nt)
      reinterpret_cast<float4*>(Ks)[i] = reinterpret_cast<const float4*>(Kf + ((size_t)u * L + nb) * dqk)[i];
    for (int i = tid; i < cnt * d / 4; i += nt)
      reinterpret_cast<float4*>(Vs)[i] = reinterpret_cast<const float4*>(Vf + ((size_t)u * L + nb) * d)[i];
    __syncthreads();
    if (live) {
      for (int n = 0; n < cnt; ++n) {
        const float4* kp = reinterpret_cast<const float4*>(Ks + n * dqk + h * DQH);
        const float4* vp = reinterpret_cast<const float4*>(Vs + n * d + h * DVH);
        float e = 0.f;
#pragma unroll
        for (int a = 0; a < DQH / 4; ++a) {
          const float4 x = kp[a];
          e = fmaf(q[4 * a], x.x, e); e = fmaf(q[4 * a + 1], x.y, e); e = fmaf(q[4 * a + 2], x.z, e); e = fmaf(q[4 * a + 3], x.w, e);
        }
        const float g = 1.f / (1.f + expf(-e));
#pragma unroll
        for (int v = 0; v < DVH / 4; ++v) {
          const float4 x = vp[v];
          acc[4 * v] = fmaf(g, x.x, acc[4 * v]); acc[4 * v + 1] = fmaf(g, x.y, acc[4 * v + 1]);
          acc[4 * v + 2] = fmaf(g, x.z, acc[4 * v + 2]); acc[4 * v + 3] = fmaf(g, x.w, acc[4 * v + 3]);
        }
      }
    }
  }
  if (live) {
    float4* out = reinterpret_cast<float4*>(Hp + ((size_t)c * Lp + seg) * d + h * DVH);
#pragma unroll
    for (int v = 0; v < DVH / 4; ++v) out[v] = make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
  }
}

template <int DQH, int DVH>
int launch_sta_fwd32(const Plan& p, const float* Qf, const float* Kf, const float* Vf, const int32_t* lengths,
                     const int32_t* cand_offsets, float* Hp, cudaStream_t st) {
  const size_t smem = (size_t)kChunk * (p.dqk + p.d) * sizeof(float);
  const int ctiles = (p.maxC + 31) / 32;
  if (p.U > 65535 || ctiles > 65535 || smem > 200 * 1024) return LASER_ERR_UNSUPPORTED;
  LASER_CUDA_OK(cudaFuncSetAttribute(sta_fwd32_kernel<DQH, DVH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  LaunchScope ls("bwd_sta_fwd", st);
  sta_fwd32_kernel<DQH, DVH><<<dim3(p.Lp, ctiles, p.U), 32 * p.H, smem, st>>>(Qf, Kf, Vf, lengths, cand_offsets, Hp, p.L,
                                                                               p.d, p.dqk, p.H, p.S, p.Lp, p.N);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

struct BwdScratch {
  float *Hp, *dHp, *T, *Q, *Qt, *A, *Mh, *dT, *dM, *dQt, *dQ, *dQf, *dK, *dV;
  size_t total;
};

// Carves the backward's own scratch (after the forward plan's regions).
BwdScratch carve_scratch(const Plan& p, char* base) {
  BwdScratch s;
  size_t off = 0;
  auto take = [&](size_t n_floats) {
    float* ptr = base ? reinterpret_cast<float*>(base + off) : nullptr;
    off = align_up(off + n_floats * sizeof(float)) + kGuardBytes;
    return ptr;
  };
  const size_t N = p.N, d = p.d, H = p.H, Lp = p.Lp, M = p.M, UL = (size_t)p.U * p.L;
  s.Hp = take(N * Lp * d);
  s.dHp = take(N * Lp * d);
  s.T = take((M + 1) * N * d);
  s.Q = take(M * N * d);
  s.Qt = take(M * N * H * d);
  s.A = take(M * N * H * Lp);
  s.Mh = take(M * N * H * d);
  s.dT = take(N * d);
  s.dM = take(N * H * d);
  s.dQt = take(N * H * d);
  s.dQ = take(N * d);
  s.dQf = take(N * p.dqk);
  s.dK = take(UL * p.dqk);
  s.dV = take(UL * d);
  s.total = off;
  return s;
}

template <typename T>
int backward_t(const Plan& p, const T* items, const int32_t* lengths, const T* cands, const int32_t* cand_offsets,
               const T* Wq, const T* Wk, const T* Wv, const T* Wg, const float* dz, float* d_items, float* d_cands,
               float* dWq, float* dWk, float* dWv, float* dWg, char* ws, cudaStream_t st, bool tensor) {
  const int N = p.N, d = p.d, H = p.H, Lp = p.Lp, M = p.M, dqk = p.dqk, dvh = p.dvh, U = p.U, L = p.L;
  const size_t UL = (size_t)U * L;
  // (d_items: with candidates present its first matrix product writes every row, padding included)
  if (N == 0 || U == 0) LASER_CUDA_OK(cudaMemsetAsync(d_items, 0, UL * d * sizeof(float), st));
  LASER_CUDA_OK(cudaMemsetAsync(dWq, 0, (size_t)d * dqk * sizeof(float), st));
  LASER_CUDA_OK(cudaMemsetAsync(dWk, 0, (size_t)d * dqk * sizeof(float), st));
  LASER_CUDA_OK(cudaMemsetAsync(dWv, 0, (size_t)d * d * sizeof(float), st));
  if (M > 0) LASER_CUDA_OK(cudaMemsetAsync(dWg, 0, (size_t)M * 3 * d * d * sizeof(float), st));
  if (N == 0 || U == 0) return LASER_OK;
  BwdScratch s = carve_scratch(p, ws + p.total);
  float* Qf = reinterpret_cast<float*>(ws + p.off_q);
  float* Kf = reinterpret_cast<float*>(ws + p.off_k);
  float* Vf = reinterpret_cast<float*>(ws + p.off_v);
  const GemmCtx gx = {st, tensor};
  int rc;
#define BWD_OK(...) do { rc = (__VA_ARGS__); if (rc != LASER_OK) return rc; } while (0)

  // ---- forward, kept in fp32: projections and H' (the FP32-ALU forward kernels), then the GSTA layers
  char* mma_scratch = ws + p.total + s.total;
  const bool mma = tensor && sta_bwd_mma_supported(p);     // (users with very few candidates keep the FP32 gate kernels)
  const bool attn_mma = mma && gsta_attn_mma_supported(p); // the recomputed GSTA attention on the MMAs as well
  if (tensor) {
    // (sta_fwd_mma writes every row of H' that is read later: all candidates of every non-empty segment)
    if (!(mma && sta_fwd_mma_supported(p))) LASER_CUDA_OK(cudaMemsetAsync(s.Hp, 0, (size_t)N * Lp * d * sizeof(float), st));
    // projections as three matrix products over all rows (padding rows included: their K and V are never read)
    BWD_OK(gemm<T, T>(gx, N, dqk, d, cands, d, false, Wq, dqk, false, Qf, dqk, p.inv_gamma, false, false));
    // K and V: as bf16 straight into the MMA kernels' operand arrays when nothing reads them in fp32
    bool kv_ready = false;
    if (mma && sta_fwd_mma_supported(p)) {
      bf16 *Kb, *Vb;
      sta_mma_operand_arrays(p, mma_scratch, &Kb, &Vb);
      const int r1 = gemm_rows_bf16<T, T>(gx, (int)UL, dqk, d, items, d, Wk, dqk, Kb, dqk);
      const int r2 = r1 == LASER_OK ? gemm_rows_bf16<T, T>(gx, (int)UL, d, d, items, d, Wv, d, Vb, d) : r1;
      if (r2 != LASER_OK && r2 != LASER_ERR_UNSUPPORTED) return r2;
      kv_ready = r2 == LASER_OK;
    }
    if (!kv_ready) {
      BWD_OK(gemm<T, T>(gx, (int)UL, dqk, d, items, d, false, Wk, dqk, false, Kf, dqk, 1.f, false, false));
      BWD_OK(gemm<T, T>(gx, (int)UL, d, d, items, d, false, Wv, d, false, Vf, d, 1.f, false, false));
    }
    if (mma) BWD_OK(sta_mma_operands(p, Qf, kv_ready ? nullptr : Kf, kv_ready ? nullptr : Vf, mma_scratch, st));
    if (mma && sta_fwd_mma_supported(p)) BWD_OK(sta_fwd_mma(p, lengths, cand_offsets, attn_mma ? nullptr : s.Hp, attn_mma, mma_scratch, st));
    else if (p.dqh == 16 && dvh == 16 && p.H <= 32) BWD_OK(launch_sta_fwd32<16, 16>(p, Qf, Kf, Vf, lengths, cand_offsets, s.Hp, st));
    else if (p.dqh == 16 && dvh == 32 && p.H <= 32) BWD_OK(launch_sta_fwd32<16, 32>(p, Qf, Kf, Vf, lengths, cand_offsets, s.Hp, st));
    else BWD_OK(simt_sta_f32(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, s.Hp, ws, st));
  } else if (p.dqh == 16 && (dvh == 16 || dvh == 32) && p.H <= 32) {
    // (a candidate tile of a user with more candidates than max_cands_per_user declares would stay unwritten: zero first)
    LASER_CUDA_OK(cudaMemsetAsync(s.Hp, 0, (size_t)N * Lp * d * sizeof(float), st));
    BWD_OK(simt_project(p, items, lengths, cands, Wq, Wk, Wv, ws, st));
    if (dvh == 16) BWD_OK(launch_sta_fwd32<16, 16>(p, Qf, Kf, Vf, lengths, cand_offsets, s.Hp, st));
    else BWD_OK(launch_sta_fwd32<16, 32>(p, Qf, Kf, Vf, lengths, cand_offsets, s.Hp, st));
  } else {
    BWD_OK(simt_sta_f32(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, s.Hp, ws, st));
  }
  const size_t Nd = (size_t)N * d, NHd = Nd * H;
  {
    LaunchScope ls("bwd_to_f32", st);
    to_f32_kernel<T><<<296, 256, 0, st>>>(cands, s.T, Nd);
  }
  constexpr int attn_warps = kAttnThreads / 32;
  const size_t attn_smem_f = ((size_t)(1 + attn_warps) * H * d + (size_t)H * Lp) * sizeof(float);
  const size_t attn_smem_b = ((size_t)(2 + attn_warps) * H * d + 2 * (size_t)H * Lp) * sizeof(float);
  if (attn_smem_b > 200 * 1024) return LASER_ERR_UNSUPPORTED;
  // 16-byte accesses when rows allow; heads in groups of four, two or one, whichever divides H
  const bool v4 = d % 4 == 0;
  auto attn_fwd = H % 4 == 0 ? (v4 ? gsta_attn_fwd_kernel<4, 4> : gsta_attn_fwd_kernel<1, 4>)
                  : H % 2 == 0 ? (v4 ? gsta_attn_fwd_kernel<4, 2> : gsta_attn_fwd_kernel<1, 2>)
                               : (v4 ? gsta_attn_fwd_kernel<4, 1> : gsta_attn_fwd_kernel<1, 1>);
  auto attn_bwd = H % 4 == 0 ? (v4 ? gsta_attn_bwd_kernel<4, 4> : gsta_attn_bwd_kernel<1, 4>)
                  : H % 2 == 0 ? (v4 ? gsta_attn_bwd_kernel<4, 2> : gsta_attn_bwd_kernel<1, 2>)
                               : (v4 ? gsta_attn_bwd_kernel<4, 1> : gsta_attn_bwd_kernel<1, 1>);
  LASER_CUDA_OK(cudaFuncSetAttribute(attn_fwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_f));
  LASER_CUDA_OK(cudaFuncSetAttribute(attn_bwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_b));
  for (int l = 0; l < M; ++l) {
    const T *Wql = Wg + (size_t)(l * 3) * d * d, *Wkl = Wql + (size_t)d * d, *Wvl = Wkl + (size_t)d * d;
    float *Tl = s.T + l * Nd, *Tn = Tl + Nd, *Ql = s.Q + l * Nd, *Qtl = s.Qt + l * NHd, *Al = s.A + (size_t)l * N * H * Lp,
          *Ml = s.Mh + l * NHd;
    BWD_OK(gemm<float, T>(gx, N, d, d, Tl, d, false, Wql, d, false, Ql, d, 1.f, false, false));
    // Qt_h = Q_h W_k[:, h]^T / tau, every head
    BWD_OK(gemm<float, T>(gx, N, d, dvh, Ql, d, false, Wkl, d, true, Qtl, H * d, p.inv_tau, false, false, H, dvh, dvh, d));
    if (attn_mma) {
      BWD_OK(gsta_attn_fwd_mma(p, Qtl, lengths, cand_offsets, Al, Ml, mma_scratch, st));
    } else {
      LaunchScope ls("bwd_attn_fwd", st);
      attn_fwd<<<N, kAttnThreads, attn_smem_f, st>>>(s.Hp, Qtl, lengths, cand_offsets, Al, Ml, U, L, p.S, Lp,
                                                                 H, d);
    }
    LASER_CUDA_OK(cudaMemcpyAsync(Tn, Tl, Nd * sizeof(float), cudaMemcpyDeviceToDevice, st));
    // t += o,  o_h = m_h W_v[:, h], every head
    BWD_OK(gemm<float, T>(gx, N, dvh, d, Ml, H * d, false, Wvl, d, false, Tn, d, 1.f, true, false, H, d, dvh, dvh));
  }

  // ---- backward through the GSTA layers
  LASER_CUDA_OK(cudaMemcpyAsync(s.dT, dz, Nd * sizeof(float), cudaMemcpyDeviceToDevice, st));
  if (M == 0) LASER_CUDA_OK(cudaMemsetAsync(s.dHp, 0, (size_t)N * Lp * d * sizeof(float), st));
  for (int l = M - 1; l >= 0; --l) {
    const T *Wql = Wg + (size_t)(l * 3) * d * d, *Wkl = Wql + (size_t)d * d, *Wvl = Wkl + (size_t)d * d;
    float *Tl = s.T + l * Nd, *Ql = s.Q + l * Nd, *Qtl = s.Qt + l * NHd, *Al = s.A + (size_t)l * N * H * Lp,
          *Ml = s.Mh + l * NHd;
    float *gWq = dWg + (size_t)(l * 3) * d * d, *gWk = gWq + (size_t)d * d, *gWv = gWk + (size_t)d * d;
    // dW_v[:, h] += m_h^T do_h;  dm_h = do_h W_v[:, h]^T, every head
    BWD_OK(gemm<float, float>(gx, d, dvh, N, Ml, H * d, true, s.dT, d, false, gWv, d, 1.f, true, true, H, d, dvh, dvh));
    BWD_OK(gemm<float, T>(gx, N, d, dvh, s.dT, d, false, Wvl, d, true, s.dM, H * d, 1.f, false, false, H, dvh, dvh, d));
    if (attn_mma) {
      BWD_OK(gsta_attn_bwd_mma(p, Qtl, Al, s.dM, lengths, cand_offsets, s.dQt, s.dHp, l == M - 1, l == 0, mma_scratch, st));
    } else {
      LaunchScope ls("bwd_attn_bwd", st);
      attn_bwd<<<N, kAttnThreads, attn_smem_b, st>>>(s.Hp, Qtl, Al, s.dM, lengths, cand_offsets, s.dQt, s.dHp,
                                                                 U, L, p.S, Lp, H, d, l == M - 1 ? 1 : 0);
    }
    // dQ_h = dQt_h W_k[:, h] / tau;  dW_k[:, h] += dQt_h^T Q_h / tau, every head
    BWD_OK(gemm<float, T>(gx, N, dvh, d, s.dQt, H * d, false, Wkl, d, false, s.dQ, d, p.inv_tau, false, false, H, d, dvh, dvh));
    BWD_OK(gemm<float, float>(gx, d, dvh, N, s.dQt, H * d, true, Ql, d, false, gWk, d, p.inv_tau, true, true, H, d, dvh, dvh));
    BWD_OK(gemm<float, float>(gx, d, d, N, Tl, d, true, s.dQ, d, false, gWq, d, 1.f, true, true));        // dW_q += T^T dQ
    BWD_OK(gemm<float, T>(gx, N, d, d, s.dQ, d, false, Wql, d, true, s.dT, d, 1.f, true, false));            // dT += dQ W_q^T
  }

  // ---- backward through the segment aggregation and the gates
  LASER_CUDA_OK(cudaMemsetAsync(s.dQf, 0, (size_t)N * dqk * sizeof(float), st));
  LASER_CUDA_OK(cudaMemsetAsync(s.dK, 0, UL * dqk * sizeof(float), st));
  LASER_CUDA_OK(cudaMemsetAsync(s.dV, 0, UL * d * sizeof(float), st));
  if (mma) {
    // (with the attention on the MMAs and at least one layer, dH' has arrived in bf16 already)
    BWD_OK(sta_bwd_mma(p, attn_mma && M > 0 ? nullptr : s.dHp, lengths, cand_offsets, s.dQf, s.dK, s.dV, mma_scratch, st));
  } else {
    const int cps = (min(p.S, L) + kChunk - 1) / kChunk;
    const int dqh = dqk / H;
    const int variant = (dqh == 16 && dvh == 32) ? 2 : (dqh == 16 && dvh == 16) ? 1 : 0;   // register-resident head slices
    const size_t step_floats = (size_t)kCandsPerStep * (dqk + d + H * 33);
    const size_t smem = ((variant ? (size_t)kChunk * (dqk + 1) : 2 * (size_t)kChunk * (dqk + 1 + d + 1)) + step_floats) *
                        sizeof(float);
    if (smem > 200 * 1024 || (long long)Lp * cps > 0x7fffffffLL || U > 65535 || H > 32) return LASER_ERR_UNSUPPORTED;
    auto kernel = variant == 2 ? sta_bwd_kernel<16, 32> : variant == 1 ? sta_bwd_kernel<16, 16> : sta_bwd_kernel<0, 0>;
    LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LaunchScope ls("bwd_sta", st);
    kernel<<<dim3(Lp * cps, U), 32 * H, smem, st>>>(Qf, Kf, Vf, s.dHp, lengths, cand_offsets, s.dQf, s.dK, s.dV, L, d, dqk,
                                                    H, p.S, Lp, N, cps);
    LASER_CUDA_OK(cudaGetLastError());
  }

  // ---- backward through the projections (Qf = T W_q / gamma)
  BWD_OK(gemm<T, float>(gx, d, dqk, N, cands, d, true, s.dQf, dqk, false, dWq, dqk, p.inv_gamma, true, true));
  BWD_OK(gemm<float, T>(gx, N, d, dqk, s.dQf, dqk, false, Wq, dqk, true, s.dT, d, p.inv_gamma, true, false));
  BWD_OK(gemm<T, float>(gx, d, dqk, (int)UL, items, d, true, s.dK, dqk, false, dWk, dqk, 1.f, true, true));
  BWD_OK(gemm<T, float>(gx, d, d, (int)UL, items, d, true, s.dV, d, false, dWv, d, 1.f, true, true));
  BWD_OK(gemm<float, T>(gx, (int)UL, d, dqk, s.dK, dqk, false, Wk, dqk, true, d_items, d, 1.f, false, false));
  BWD_OK(gemm<float, T>(gx, (int)UL, d, d, s.dV, d, false, Wv, d, true, d_items, d, 1.f, true, false));
  LASER_CUDA_OK(cudaMemcpyAsync(d_cands, s.dT, Nd * sizeof(float), cudaMemcpyDeviceToDevice, st));
#undef BWD_OK
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace

size_t backward_scratch_bytes(const Plan& p) { return carve_scratch(p, nullptr).total + sta_bwd_mma_scratch_bytes(p); }

bool backward_tensor_supported(const Plan& p) { return p.dtype == LASER_BF16; }

int backward(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
             const void* Wq, const void* Wk, const void* Wv, const void* Wg, const float* dz, float* d_items,
             float* d_cands, float* dWq, float* dWk, float* dWv, float* dWg, char* ws, cudaStream_t st, bool tensor) {
  if ((unsigned long long)p.U * p.L > 0x7fffffffULL) return LASER_ERR_UNSUPPORTED;
  if (tensor && !backward_tensor_supported(p)) return LASER_ERR_UNSUPPORTED;
  if (p.dtype == LASER_F32)
    return backward_t<float>(p, (const float*)items, lengths, (const float*)cands, cand_offsets, (const float*)Wq,
                             (const float*)Wk, (const float*)Wv, (const float*)Wg, dz, d_items, d_cands, dWq, dWk, dWv,
                             dWg, ws, st, false);
  return backward_t<bf16>(p, (const bf16*)items, lengths, (const bf16*)cands, cand_offsets, (const bf16*)Wq,
                          (const bf16*)Wk, (const bf16*)Wv, (const bf16*)Wg, dz, d_items, d_cands, dWq, dWk, dWv, dWg, ws,
                          st, tensor);
}

}  // namespace laser
