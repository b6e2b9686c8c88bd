// FP32-ALU kernels for STA and GSTA: fp32 arithmetic for either I/O dtype.  This is the path of the fp32
// configuration (tf32 tensor cores carry a 10-bit mantissa and cannot hold a 1e-4 bound) and a second,
// independent GPU implementation for any shape the tensor-core path does not take.
#include "laser_common.cuh"

namespace laser {
namespace {

constexpr int kProjRows = 32;     // rows per projection block
constexpr int kProjThreads = 128;
constexpr int kStaCands = 32;     // candidates per STA block
constexpr int kStaItems = 32;     // items per chunk
constexpr int kStaThreads = 128;
constexpr int kStaMaxJ = 64;      // columns per thread = d/4 <= 64  (d <= 256)
constexpr int kGstaThreads = 128;

// Y0 = scale0 * X W0 (and optionally Y1 = X W1) for rows [0, nrows(g)) of every group g of `rows_per_group`
// rows.  Eq. 4 / Eq. 8-9: Q = t W_q, K = H W_k, V = H W_v.
template <typename T>
__global__ void __launch_bounds__(kProjThreads)
proj_simt_kernel(const T* __restrict__ X, int rows_per_group, const int* __restrict__ lengths, int d,
                 const T* __restrict__ W0, int n0, float* __restrict__ Y0, float scale0,
                 const T* __restrict__ W1, int n1, float* __restrict__ Y1, const int* __restrict__ row_off, int n_groups,
                 int* __restrict__ status) {
  extern __shared__ float xs[];   // [kProjRows][d]
  chain_wait();                   // (the kernels of this path are chained like the others: launch latencies overlap)
  chain_release();
  const int g = blockIdx.y;
  const int r0 = blockIdx.x * kProjRows;
  int nrows = rows_per_group;
  if (lengths) {
    int len = lengths[g];
    nrows = len < 0 ? 0 : (len > rows_per_group ? 0 : len);   // out-of-range lengths are reported by the STA kernel
    if (row_off && nrows > 0 && (row_off[g] < 0 || row_off[g] > row_off[n_groups] - nrows)) {   // packed rows out of range
      if (threadIdx.x == 0 && blockIdx.x == 0) report_status(status, LASER_ERR_BAD_INPUT);
      nrows = 0;
    }
  }
  if (r0 >= nrows) return;
  const int rcount = min(kProjRows, nrows - r0);
  const size_t base = (size_t)g * rows_per_group + r0;                       // rows of the (padded) outputs
  const size_t in_base = row_off ? (size_t)row_off[g] + r0 : base;          // rows of the input (packed or padded)
  for (int idx = threadIdx.x; idx < kProjRows * d; idx += kProjThreads) {
    int r = idx / d, c = idx - r * d;
    xs[idx] = r < rcount ? to_f32<T>(X[(in_base + r) * d + c]) : 0.f;
  }
  __syncthreads();
  for (int col = threadIdx.x; col < n0 + n1; col += kProjThreads) {
    const bool first = col < n0;
    const T* W = first ? W0 : W1;
    const int n = first ? n0 : n1;
    const int cc = first ? col : col - n0;
    float* Y = first ? Y0 : Y1;
    const float sc = first ? scale0 : 1.f;
    float acc[kProjRows];
#pragma unroll
    for (int r = 0; r < kProjRows; ++r) acc[r] = 0.f;
#pragma unroll 8                    // (eight weight loads in flight: the loop is latency-bound at small d)
    for (int k = 0; k < d; ++k) {
      const float w = to_f32<T>(W[(size_t)k * n + cc]);
#pragma unroll
      for (int r = 0; r < kProjRows; ++r) acc[r] = fmaf(xs[r * d + k], w, acc[r]);
    }
    for (int r = 0; r < rcount; ++r) Y[(base + r) * n + cc] = acc[r] * sc;
  }
}

__device__ __forceinline__ float sigmoid_accurate(float x) {
  // 1 / (1 + e^-x) with the accurate expf; e^-x overflowing to +inf gives exactly 0.
  return 1.f / (1.f + expf(-x));
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

// One block = (segment, 32-candidate tile, user).  Gates (Eq. 5 / Eq. 10) for a 32x32 (candidate, item) chunk go to
// shared memory, then every thread accumulates gate * value for its candidate and its interleaved columns (Eq. 12).
// kSoftmax selects the ablation variant: the weights of a segment's valid items are exp(score) normalised to sum to one
// per (candidate, head), computed online over the 32-item chunks (running maximum, running sum, rescaled accumulators).
template <typename T, bool kSoftmax>
__global__ void __launch_bounds__(kStaThreads)
sta_simt_kernel(const float* __restrict__ Q, const float* __restrict__ K, const float* __restrict__ V,
                const int* __restrict__ lengths, const int* __restrict__ cand_offsets, T* __restrict__ Hp,
                int L, int d, int dqk, int H, int S, int Lp, int N, int* __restrict__ status) {
  extern __shared__ float sm[];
  chain_wait();
  chain_release();
  const int u = blockIdx.z, seg = blockIdx.x;
  const int off0 = cand_offsets[u], off1 = cand_offsets[u + 1];
  const int len = lengths[u];
  // (a user with more candidates than the grid was sized for, i.e. than max_cands_per_user, would leave rows unwritten)
  if (off0 < 0 || off1 < off0 || off1 > N || len < 0 || len > L || off1 - off0 > (int)gridDim.y * kStaCands) {
    if (threadIdx.x == 0) report_status(status, LASER_ERR_BAD_INPUT);
    return;
  }
  const int c0 = off0 + blockIdx.y * kStaCands;
  if (c0 >= off1) return;
  const int nc = min(kStaCands, off1 - c0);
  const int dqh = dqk / H, dvh = d / H;
  const int qld = dqk + 1;
  float* Qs = sm;                              // [32][dqk+1]
  float* Ks = Qs + kStaCands * qld;            // [32][dqk+1]
  float* Vs = Ks + kStaItems * qld;            // [32][d]
  float* G = Vs + kStaItems * d;               // [H][32][33]
  float* st_m = G + H * kStaCands * 33;        // softmax variant: running maximum   [H][32]
  float* st_z = st_m + H * kStaCands;          //                  running sum       [H][32]
  float* st_s = st_z + H * kStaCands;          //                  this chunk's rescale factor [H][32]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = tid >> 2, cg = tid & 3;        // accumulate phase: candidate, column group
  const int nj = (d + 3 - cg) / 4;             // columns cg, cg+4, ...
  float acc[kStaMaxJ];
  int goff[kStaMaxJ];
#pragma unroll
  for (int j = 0; j < kStaMaxJ; ++j) {
    acc[j] = 0.f;
    int col = cg + 4 * j;
    goff[j] = col < d ? ((col / dvh) * kStaCands + c) * 33 : 0;
  }

  for (int idx = tid; idx < kStaCands * dqk; idx += kStaThreads) {
    int r = idx / dqk, a = idx - r * dqk;
    Qs[r * qld + a] = r < nc ? Q[(size_t)(c0 + r) * dqk + a] : 0.f;
  }
  if (kSoftmax) {
    for (int idx = tid; idx < H * kStaCands; idx += kStaThreads) {
      st_m[idx] = -INFINITY;
      st_z[idx] = 0.f;
    }
  }

  const int n_begin = seg * S;
  const int n_end = min(min(n_begin + S, L), len);
  const float* Ku = K + (size_t)u * L * dqk;
  const float* Vu = V + (size_t)u * L * d;
  for (int nb = n_begin; nb < n_end; nb += kStaItems) {
    const int cnt = min(kStaItems, n_end - nb);
    __syncthreads();   // previous chunk fully consumed (and Qs visible on the first trip)
    for (int idx = tid; idx < kStaItems * dqk; idx += kStaThreads) {
      int r = idx / dqk, a = idx - r * dqk;
      Ks[r * qld + a] = r < cnt ? Ku[(size_t)(nb + r) * dqk + a] : 0.f;
    }
    for (int idx = tid; idx < kStaItems * d; idx += kStaThreads) {
      int r = idx / d, a = idx - r * d;
      Vs[idx] = r < cnt ? Vu[(size_t)(nb + r) * d + a] : 0.f;
    }
    __syncthreads();
    // gates: item = lane, candidate = warp + 4k
    for (int cc = warp; cc < kStaCands; cc += kStaThreads / 32) {
      for (int h = 0; h < H; ++h) {
        float dot = 0.f;
        for (int a = 0; a < dqh; ++a) dot = fmaf(Qs[cc * qld + h * dqh + a], Ks[lane * qld + h * dqh + a], dot);
        if (!kSoftmax) {
          G[(h * kStaCands + cc) * 33 + lane] = lane < cnt ? sigmoid_accurate(dot) : 0.f;
        } else {
          const float m_old = st_m[h * kStaCands + cc], z_old = st_z[h * kStaCands + cc];
          const float m_new = fmaxf(m_old, warp_max(lane < cnt ? dot : -INFINITY));   // finite: the chunk has an item
          const float pw = lane < cnt ? expf(dot - m_new) : 0.f;
          const float psum = warp_sum(pw);
          G[(h * kStaCands + cc) * 33 + lane] = pw;
          __syncwarp();
          if (lane == 0) {
            const float sc = expf(m_old - m_new);           // 0 on the first chunk (m_old = -inf)
            st_s[h * kStaCands + cc] = sc;
            st_z[h * kStaCands + cc] = z_old * sc + psum;
            st_m[h * kStaCands + cc] = m_new;
          }
        }
      }
    }
    __syncthreads();
    if (kSoftmax) {
#pragma unroll
      for (int j = 0; j < kStaMaxJ; ++j)
        if (j < nj) acc[j] *= st_s[goff[j] / 33];
    }
    // (the column loop is unrolled over the accumulator registers; its bound follows the width in use, so that a narrow
    // d does not pay for 64 predicated steps per item)
    if (nj <= 8) {
      for (int n = 0; n < cnt; ++n) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (j < nj) acc[j] = fmaf(G[goff[j] + n], Vs[n * d + cg + 4 * j], acc[j]);
      }
    } else if (nj <= 16) {
      for (int n = 0; n < cnt; ++n) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (j < nj) acc[j] = fmaf(G[goff[j] + n], Vs[n * d + cg + 4 * j], acc[j]);
      }
    } else if (nj <= 32) {
      for (int n = 0; n < cnt; ++n) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j < nj) acc[j] = fmaf(G[goff[j] + n], Vs[n * d + cg + 4 * j], acc[j]);
      }
    } else {
      for (int n = 0; n < cnt; ++n) {
#pragma unroll
        for (int j = 0; j < kStaMaxJ; ++j)
          if (j < nj) acc[j] = fmaf(G[goff[j] + n], Vs[n * d + cg + 4 * j], acc[j]);
      }
    }
  }
  if (c < nc) {
    T* out = Hp + ((size_t)(c0 + c) * Lp + seg) * d;
#pragma unroll
    for (int j = 0; j < kStaMaxJ; ++j) {
      if (j < nj) {
        float v = acc[j];
        if (kSoftmax) {
          const float z = st_z[goff[j] / 33];
          v = z > 0.f ? v / z : 0.f;                        // a segment without valid items stays a zero row
        }
        out[cg + 4 * j] = from_f32<T>(v);
      }
    }
  }
}


// One block per candidate.  Eq. 7 in the reassociated form (exact in real arithmetic):
//   q = t W_q;  qt_h = W_k[:, head h] q_h  (so that (s_j W_k)_h . q_h = s_j . qt_h);  e_{j,h} = s_j . qt_h / tau;
//   a = softmax_j(e);  m_h = sum_j a_{j,h} s_j;  o[head h] = m_h W_v[:, head h];  t += o.
template <typename T>
__global__ void __launch_bounds__(kGstaThreads)
gsta_simt_kernel(const T* __restrict__ Hp, const int* __restrict__ lengths, const int* __restrict__ cand_offsets,
                 const T* __restrict__ cands, const T* __restrict__ Wg, T* __restrict__ z, int U, int L, int d, int H,
                 int S, int Lp, int M, int N, float inv_tau, int* __restrict__ status) {
  extern __shared__ float sm[];
  chain_wait();
  chain_release();
  const int cand = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int nwarps = kGstaThreads / 32;
  // user of this candidate: the largest u with cand_offsets[u] <= cand (skipping users without candidates)
  int lo = 0, hi = U;   // invariant: cand_offsets[lo] <= cand < cand_offsets[hi]
  if (cand_offsets[0] > cand || cand_offsets[U] <= cand) {
    if (tid == 0) report_status(status, LASER_ERR_BAD_INPUT);
    return;
  }
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cand_offsets[mid] <= cand) lo = mid; else hi = mid;
  }
  const int len = lengths[lo];
  if (len < 0 || len > L) {
    if (tid == 0) report_status(status, LASER_ERR_BAD_INPUT);
    return;
  }
  const int nv = min((len + S - 1) / S, Lp);
  const int dh = d / H;
  float* Hs = sm;                 // [Lp][d]
  float* t = Hs + (size_t)Lp * d; // [d]
  float* q = t + d;               // [d]
  float* qt = q + d;              // [H][d]
  float* mh = qt + H * d;         // [H][d]
  float* e = mh + H * d;          // [H][Lp]

  for (int i = tid; i < d; i += kGstaThreads) t[i] = to_f32<T>(cands[(size_t)cand * d + i]);
  const T* Hc = Hp + (size_t)cand * Lp * d;
  for (int i = tid; i < nv * d; i += kGstaThreads) Hs[i] = to_f32<T>(Hc[i]);
  __syncthreads();

  for (int l = 0; l < M && nv > 0; ++l) {
    const T* Wq = Wg + (size_t)(l * 3 + 0) * d * d;
    const T* Wk = Wg + (size_t)(l * 3 + 1) * d * d;
    const T* Wv = Wg + (size_t)(l * 3 + 2) * d * d;
    for (int j = tid; j < d; j += kGstaThreads) {
      float a = 0.f;
#pragma unroll 8
      for (int i = 0; i < d; ++i) a = fmaf(t[i], to_f32<T>(Wq[(size_t)i * d + j]), a);
      q[j] = a;
    }
    __syncthreads();
    // qt[h][i] = sum_{j in head h} Wk[i][j] q[j]: one warp per row i, lanes over j
    for (int i = warp; i < d; i += nwarps) {
      for (int h = 0; h < H; ++h) {
        float a = 0.f;
        for (int j = h * dh + lane; j < (h + 1) * dh; j += 32) a = fmaf(to_f32<T>(Wk[(size_t)i * d + j]), q[j], a);
        a = warp_sum(a);
        if (lane == 0) qt[h * d + i] = a;
      }
    }
    __syncthreads();
    // scores: one warp per segment j
    for (int j = warp; j < nv; j += nwarps) {
      for (int h = 0; h < H; ++h) {
        float a = 0.f;
        for (int i = lane; i < d; i += 32) a = fmaf(Hs[j * d + i], qt[h * d + i], a);
        a = warp_sum(a);
        if (lane == 0) e[h * Lp + j] = a * inv_tau;
      }
    }
    __syncthreads();
    // softmax over the non-empty segments: one warp per head
    for (int h = warp; h < H; h += nwarps) {
      float mx = -INFINITY;
      for (int j = lane; j < nv; j += 32) mx = fmaxf(mx, e[h * Lp + j]);
      mx = warp_max(mx);
      float s = 0.f;
      for (int j = lane; j < nv; j += 32) {
        float w = expf(e[h * Lp + j] - mx);
        e[h * Lp + j] = w;
        s += w;
      }
      s = warp_sum(s);
      const float inv = 1.f / s;
      for (int j = lane; j < nv; j += 32) e[h * Lp + j] *= inv;
    }
    __syncthreads();
    for (int i = tid; i < d; i += kGstaThreads) {
      for (int h = 0; h < H; ++h) {
        float a = 0.f;
        for (int j = 0; j < nv; ++j) a = fmaf(e[h * Lp + j], Hs[j * d + i], a);
        mh[h * d + i] = a;
      }
    }
    __syncthreads();
    for (int col = tid; col < d; col += kGstaThreads) {
      const int h = col / dh;
      float a = 0.f;
#pragma unroll 8
      for (int i = 0; i < d; ++i) a = fmaf(mh[h * d + i], to_f32<T>(Wv[(size_t)i * d + col]), a);
      q[col] = a;   // o_l
    }
    __syncthreads();
    for (int i = tid; i < d; i += kGstaThreads) t[i] += q[i];
    __syncthreads();
  }
  for (int i = tid; i < d; i += kGstaThreads) z[(size_t)cand * d + i] = from_f32<T>(t[i]);
}

// T: dtype of the inputs; TO: dtype of H' (T itself, or float when the caller keeps fp32 intermediates)
// Eq. 8-9 in fp32: Q / gamma, K, V into the workspace (off_q, off_k, off_v).
template <typename T>
int simt_project_t(const Plan& p, const T* items, const int32_t* lengths, const T* cands, const T* Wq, const T* Wk,
                   const T* Wv, char* ws, cudaStream_t st) {
  int* status = reinterpret_cast<int*>(ws + p.off_status);
  float* Qf = reinterpret_cast<float*>(ws + p.off_q);
  float* Kf = reinterpret_cast<float*>(ws + p.off_k);
  float* Vf = reinterpret_cast<float*>(ws + p.off_v);
  if (p.N == 0 || p.U == 0) return LASER_OK;
  if (p.U > 65535) return LASER_ERR_UNSUPPORTED;           // users index grid.y of the second launch
  const size_t proj_smem = (size_t)kProjRows * p.d * sizeof(float);
  {
    dim3 grid((p.N + kProjRows - 1) / kProjRows, 1);
    LaunchScope ls("proj_simt_q", st);
    LASER_CUDA_OK(launch_chained(proj_simt_kernel<T>, grid, dim3(kProjThreads), proj_smem, st, cands, p.N,
                                 (const int*)nullptr, p.d, Wq, p.dqk, Qf, p.inv_gamma, (const T*)nullptr, 0,
                                 (float*)nullptr, (const int*)nullptr, 0, status));
  }
  {
    dim3 grid((p.L + kProjRows - 1) / kProjRows, p.U);
    LaunchScope ls("proj_simt_kv", st);
    LASER_CUDA_OK(launch_chained(proj_simt_kernel<T>, grid, dim3(kProjThreads), proj_smem, st, items, p.L,
                                 (const int*)lengths, p.d, Wk, p.dqk, Kf, 1.f, Wv, p.d, Vf, (const int*)p.item_offsets,
                                 p.U, status));
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

template <typename T, typename TO>
int simt_sta_t(const Plan& p, const T* items, const int32_t* lengths, const T* cands, const int32_t* cand_offsets,
               const T* Wq, const T* Wk, const T* Wv, TO* Hp, char* ws, cudaStream_t st, bool softmax) {
  int* status = reinterpret_cast<int*>(ws + p.off_status);
  float* Qf = reinterpret_cast<float*>(ws + p.off_q);
  float* Kf = reinterpret_cast<float*>(ws + p.off_k);
  float* Vf = reinterpret_cast<float*>(ws + p.off_v);
  if (p.N == 0 || p.U == 0) return LASER_OK;
  // users and candidate tiles index grid.y / grid.z of the launches below
  if (p.U > 65535 || (p.maxC + kStaCands - 1) / kStaCands > 65535) return LASER_ERR_UNSUPPORTED;
  const int rc = simt_project_t<T>(p, items, lengths, cands, Wq, Wk, Wv, ws, st);
  if (rc != LASER_OK) return rc;
  {
    const size_t smem = ((size_t)(kStaCands + kStaItems) * (p.dqk + 1) + (size_t)kStaItems * p.d +
                         (size_t)p.H * kStaCands * (33 + 3)) * sizeof(float);
    if (smem > 200 * 1024) return LASER_ERR_UNSUPPORTED;
    dim3 grid(p.Lp, (p.maxC + kStaCands - 1) / kStaCands, p.U);
    if (softmax) {
      LASER_CUDA_OK(cudaFuncSetAttribute(sta_simt_kernel<TO, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      LaunchScope ls("sta_simt_softmax", st);
      LASER_CUDA_OK(launch_chained(sta_simt_kernel<TO, true>, grid, dim3(kStaThreads), smem, st, (const float*)Qf,
                                   (const float*)Kf, (const float*)Vf, (const int*)lengths, (const int*)cand_offsets, Hp,
                                   p.L, p.d, p.dqk, p.H, p.S, p.Lp, p.N, status));
    } else {
      LASER_CUDA_OK(cudaFuncSetAttribute(sta_simt_kernel<TO, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      LaunchScope ls("sta_simt", st);
      LASER_CUDA_OK(launch_chained(sta_simt_kernel<TO, false>, grid, dim3(kStaThreads), smem, st, (const float*)Qf,
                                   (const float*)Kf, (const float*)Vf, (const int*)lengths, (const int*)cand_offsets, Hp,
                                   p.L, p.d, p.dqk, p.H, p.S, p.Lp, p.N, status));
    }
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

template <typename T>
int simt_gsta_t(const Plan& p, const T* Hp, const int32_t* lengths, const int32_t* cand_offsets, const T* cands,
                const T* Wg, T* z, char* ws, cudaStream_t st) {
  int* status = reinterpret_cast<int*>(ws + p.off_status);
  if (p.N == 0) return LASER_OK;
  const size_t smem = ((size_t)p.Lp * p.d + (size_t)(2 + 2 * p.H) * p.d + (size_t)p.H * p.Lp) * sizeof(float);
  if (smem > 200 * 1024) return LASER_ERR_UNSUPPORTED;
  LASER_CUDA_OK(cudaFuncSetAttribute(gsta_simt_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  {
    LaunchScope ls("gsta_simt", st);
    LASER_CUDA_OK(launch_chained(gsta_simt_kernel<T>, dim3(p.N), dim3(kGstaThreads), smem, st, Hp, (const int*)lengths,
                                 (const int*)cand_offsets, cands, Wg, z, p.U, p.L, p.d, p.H, p.S, p.Lp, p.M, p.N,
                                 p.inv_tau, status));
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

}  // namespace

static int simt_sta_any(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                        const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime,
                        char* ws, cudaStream_t st, bool softmax) {
  if (p.d > 4 * kStaMaxJ) return LASER_ERR_UNSUPPORTED;
  if (p.dtype == LASER_F32)
    return simt_sta_t<float, float>(p, (const float*)items, lengths, (const float*)cands, cand_offsets, (const float*)Wq,
                                    (const float*)Wk, (const float*)Wv, (float*)Hprime, ws, st, softmax);
  using B = __nv_bfloat16;
  return simt_sta_t<B, B>(p, (const B*)items, lengths, (const B*)cands, cand_offsets, (const B*)Wq, (const B*)Wk,
                          (const B*)Wv, (B*)Hprime, ws, st, softmax);
}

// The projections alone (fp32 Q / gamma, K, V in the workspace), for callers with an attention kernel of their own.
int simt_project(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const void* Wq,
                 const void* Wk, const void* Wv, char* ws, cudaStream_t st) {
  if (p.dtype == LASER_F32)
    return simt_project_t<float>(p, (const float*)items, lengths, (const float*)cands, (const float*)Wq, (const float*)Wk,
                                 (const float*)Wv, ws, st);
  using B = __nv_bfloat16;
  return simt_project_t<B>(p, (const B*)items, lengths, (const B*)cands, (const B*)Wq, (const B*)Wk, (const B*)Wv, ws, st);
}

// STA with H' kept in fp32 whatever the I/O dtype (the backward pass recomputes the forward this way); the projections
// stay in the workspace as fp32 Q / gamma, K, V.
int simt_sta_f32(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
                 const void* Wq, const void* Wk, const void* Wv, float* Hprime32, char* ws, cudaStream_t st) {
  if (p.d > 4 * kStaMaxJ) return LASER_ERR_UNSUPPORTED;
  if (p.dtype == LASER_F32)
    return simt_sta_t<float, float>(p, (const float*)items, lengths, (const float*)cands, cand_offsets, (const float*)Wq,
                                    (const float*)Wk, (const float*)Wv, Hprime32, ws, st, false);
  using B = __nv_bfloat16;
  return simt_sta_t<B, float>(p, (const B*)items, lengths, (const B*)cands, cand_offsets, (const B*)Wq, (const B*)Wk,
                              (const B*)Wv, Hprime32, ws, st, false);
}

int simt_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
             const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st) {
  return simt_sta_any(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws, st, false);
}

int simt_sta_softmax(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                     const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws,
                     cudaStream_t st) {
  return simt_sta_any(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws, st, true);
}

int simt_gsta(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets, const void* cands,
              const void* Wg, void* z, char* ws, cudaStream_t st) {
  if (p.dtype == LASER_F32)
    return simt_gsta_t<float>(p, (const float*)Hprime, lengths, cand_offsets, (const float*)cands, (const float*)Wg,
                              (float*)z, ws, st);
  using B = __nv_bfloat16;
  return simt_gsta_t<B>(p, (const B*)Hprime, lengths, cand_offsets, (const B*)cands, (const B*)Wg, (B*)z, ws, st);
}

}  // namespace laser
