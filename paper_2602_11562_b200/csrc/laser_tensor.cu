// Tensor-core path (bf16 operands, fp32 accumulation) for sm_100a: tcgen05.mma with TMEM accumulators, bulk-TMA
// staging through mbarrier rings, warp-specialised roles.
//
//   tc_prep_kernel   validates lengths / offsets, builds the unit and candidate-tile prefix arrays, zeroes the segment
//                    value sums, and writes the transposed weight images in UMMA canonical layout.
//   tc_proj_kernel   Eq. 8-9: K = X W_k, V = X W_v (and Q = T W_q / (2 gamma)) on the tensor cores.  Outputs are written
//                    tile by tile in exactly the shared-memory layout the attention kernel's MMAs consume, so that
//                    kernel stages them with plain bulk copies.
//   tc_sta_kernel    Eq. 10-12 fused: per (user, 128-candidate tile, segment) and head,
//                      scores = Q_h K_h^T (MMA, TMEM)  ->  P = 1 + tanh(scores) (registers)  ->  O_h += P V_h (MMA, TMEM)
//                    and H' = O / 2.  Uses Sigmoid(x) = (1 + tanh(x/2)) / 2 with 1 / (2 gamma) folded into Q: one
//                    transcendental and one add per gate.  Masked items have zero K and V rows, so they contribute
//                    exactly nothing.  No score ever leaves the SM.
#include <cuda.h>
#include <string.h>

#include "laser_common.cuh"
#include "laser_gsta_img.cuh"
#include "laser_ptx.cuh"
#include "laser_tmap.cuh"

namespace laser {
namespace {

using bf16 = __nv_bfloat16;
using namespace ptx;

constexpr int kCandTile = 128;        // candidates per tile = MMA M = TMEM lanes
constexpr int kProjThreads = 256;     // two warps per TMEM lane quadrant: they split the accumulator columns
constexpr int kProjTmemCols = 256;    // K / Q accumulator at column 0, V^T accumulator at column 128
constexpr int kGateGroups = 4;        // gate warpgroups; each owns one score / gate buffer in TMEM
constexpr int kStaThreads = (9 + 4 * kGateGroups) * 32;
constexpr int kStaTmemCols = 512;
constexpr int kKvStages = 4;

struct TcParams {
  int U, L, d, dqk, H, S, Lp, N, dqh, dvh, maxC;
  int IT, NT, NTG, NG, n_tiles;       // items per tile, tiles per segment, tiles per projection unit, units per segment
  int cand_tiles_max;
  int n_obuf;                         // output accumulators in TMEM (2 when a second one fits, else 1)
  int o_col1;                         // TMEM column of the second output accumulator
  float q_scale;                      // 1 / (2 gamma)
  const bf16 *items, *cands, *Wq, *Wk, *Wv;
  const int *lengths, *cand_offsets;
  const int* item_off;                // packed item layout: first row of every user ([U + 1]); null = padded [U, L, d]
  bf16 *Qblk, *Kblk, *Vtblk;
  int *unit_start, *tile_off;         // [U+1] prefix of attention units / candidate tiles per user
  int* proj_start;                    // [U+1] prefix of projection units (groups of item tiles that hold valid items)
  int* counters;                      // [0] attention units, [1] candidate tiles, [2] projection units
  int4* sta_begin;                    // [sta_grid]  first attention unit of every block: (user, candidate tile, segment, -)
  int4* proj_begin;                   // [proj_grid] first projection unit of every block: (user, segment, tile group, user's length)
  int4* ctile;                        // [candidate tiles] (user, tile within the user, user's first candidate, its candidates)
  int sta_grid, proj_grid;
  const bf16* Wg;                     // GSTA weights whose images this set-up also builds (null: none)
  uint4* gimg;
  int* gnseg;                         // per-candidate segment counts for the GSTA kernel (built with the images)
  int* gorder;                        // launch order of the GSTA kernel's blocks (null: not wanted), its sort keys, and
  int* gorder_keys;                   // the candidates per block of that kernel
  int gcpb;
  int M;
  bf16 *imgK, *imgQ, *imgV;           // W_k^T, W_q^T [dqk x d], W_v^T [128 x d] in canonical K-major layout
  int* status;
  bf16* Hp;
};

// Sanitised view of one user: invalid lengths / offsets behave like an empty user (and are reported by tc_prep_kernel).
struct UserShape {
  int len, c0, nc, nseg, ctiles;
};
__device__ __forceinline__ UserShape user_shape(const TcParams& P, int u) {
  UserShape s;
  int len = P.lengths[u], c0 = P.cand_offsets[u], c1 = P.cand_offsets[u + 1];
  bool bad = len < 0 || len > P.L || c0 < 0 || c1 < c0 || c1 > P.N || c1 - c0 > P.maxC;
  if (!bad && P.item_off) {                      // packed rows: the user's valid prefix must lie inside the array
    const int r0 = P.item_off[u];
    bad = r0 < 0 || r0 > P.item_off[P.U] - len;
  }
  s.len = bad ? 0 : len;
  s.c0 = bad ? 0 : c0;
  s.nc = bad ? 0 : c1 - c0;
  s.nseg = (s.len + P.S - 1) / P.S;
  s.ctiles = (s.nc + kCandTile - 1) / kCandTile;
  return s;
}

// Projection units of a user: every segment with valid items is cut into groups of NTG item tiles (<= 128 rows);
// only groups that hold at least one valid item count.
__device__ __forceinline__ int proj_units_of(const TcParams& P, const UserShape& s) {
  if (s.nseg == 0) return 0;
  const int last_items = s.len - (s.nseg - 1) * P.S;
  const int last_tiles = min(P.NT, (last_items + P.IT - 1) / P.IT);
  return (s.nseg - 1) * P.NG + (last_tiles + P.NTG - 1) / P.NTG;
}

// Canonical K-major (no swizzle) element offset of (row, k) in a [rows x kdim] operand: 8x8-element core matrices of
// 64 contiguous elements, core matrices of one 8-row group adjacent along k.
__device__ __forceinline__ int canon_off(int row, int k, int kdim) {
  return ((row >> 3) * (kdim >> 3) + (k >> 3)) * 64 + (row & 7) * 8 + (k & 7);
}

// ------------------------------------------------------------------------------------------------------- prep
__global__ void __launch_bounds__(1024) tc_prep_kernel(TcParams P) {
  const int tid = threadIdx.x;
  chain_wait();
  chain_release();
  if (blockIdx.x == 0) {
    __shared__ int sa[1024], sb[1024], sc[1024];
    const int per = (P.U + 1023) / 1024;
    const int n_act = max(1, (P.U + per - 1) / per);      // threads that own users: the scan runs over these only
    const int last = n_act - 1;
    const int u0 = min(tid * per, P.U), u1 = min(u0 + per, P.U);
    int a = 0, b = 0, c = 0;
    bool bad = false;
    for (int u = u0; u < u1; ++u) {
      const int len = P.lengths[u], c0 = P.cand_offsets[u], c1 = P.cand_offsets[u + 1];
      bad |= len < 0 || len > P.L || c0 < 0 || c1 < c0 || c1 > P.N || c1 - c0 > P.maxC;
      const UserShape s = user_shape(P, u);
      bad |= s.len != len && len >= 0 && len <= P.L;      // (the packed-row check of user_shape)
      a += s.ctiles;
      b += s.ctiles * s.nseg;
      c += proj_units_of(P, s);
    }
    if (bad) report_status(P.status, LASER_ERR_BAD_INPUT);
    sa[tid] = a;
    sb[tid] = b;
    sc[tid] = c;
    __syncthreads();
    for (int off = 1; off < n_act; off <<= 1) {
      int va = 0, vb = 0, vc = 0;
      if (tid >= off) { va = sa[tid - off]; vb = sb[tid - off]; vc = sc[tid - off]; }
      __syncthreads();
      sa[tid] += va;
      sb[tid] += vb;
      sc[tid] += vc;
      __syncthreads();
    }
    int pa = sa[tid] - a, pb = sb[tid] - b, pc = sc[tid] - c;   // exclusive prefixes
    for (int u = u0; u < u1; ++u) {
      const UserShape s = user_shape(P, u);
      for (int jt = 0; jt < s.ctiles; ++jt) P.ctile[pa + jt] = make_int4(u, jt, s.c0, s.nc);
      P.tile_off[u] = pa;
      P.unit_start[u] = pb;
      P.proj_start[u] = pc;
      pa += s.ctiles;
      pb += s.ctiles * s.nseg;
      pc += proj_units_of(P, s);
    }
    if (tid == last) {
      P.tile_off[P.U] = sa[last];
      P.unit_start[P.U] = sb[last];
      P.proj_start[P.U] = sc[last];
      P.counters[0] = sb[last];
      P.counters[1] = sa[last];
      P.counters[2] = sc[last];
    }
    // First unit of every block of the two main kernels (block b of G owns units [n b / G, n (b + 1) / G)): find the
    // scan chunk in shared memory, then the user inside the chunk.
    const int n_att = sb[last], n_proj = sc[last];
    for (int b = tid; b < P.sta_grid + P.proj_grid; b += 1024) {
      const bool att = b < P.sta_grid;
      const int* incl = att ? sb : sc;
      const int n = att ? n_att : n_proj, G = att ? P.sta_grid : P.proj_grid, bb = att ? b : b - P.sta_grid;
      const int id = (int)(((long long)n * bb) / G);
      int4 out = make_int4(-1, 0, 0, 0);
      if (id < n) {
        int lo = 0, hi = last;                     // smallest chunk k with incl[k] > id
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (incl[mid] > id) hi = mid; else lo = mid + 1;
        }
        int base = lo > 0 ? incl[lo - 1] : 0;      // units before the chunk
        int u = min(lo * per, P.U);
        UserShape s = user_shape(P, u);
        for (;;) {
          const int cnt = att ? s.ctiles * s.nseg : proj_units_of(P, s);
          if (id < base + cnt) break;
          base += cnt;
          s = user_shape(P, ++u);
        }
        const int local = id - base;
        if (att) out = make_int4(u, local / s.nseg, local % s.nseg, 0);
        else out = make_int4(u, local / P.NG, local % P.NG, s.len);
      }
      if (att) P.sta_begin[bb] = out; else P.proj_begin[bb] = out;
    }
    return;
  }
  if (P.gorder && blockIdx.x == gridDim.x - 1) {   // one extra block when the GSTA kernel wants its blocks sorted
    gsta_build_order(P.lengths, P.cand_offsets, P.U, P.N, P.L, P.S, P.Lp, P.gcpb, P.gorder, P.gorder_keys);
    return;
  }
  // remaining blocks: weight images, grid-stride
  const int nthreads = (gridDim.x - 1 - (P.gorder ? 1 : 0)) * blockDim.x;
  const int g = (blockIdx.x - 1) * blockDim.x + tid;
  const int nK = P.dqk * P.d;
  for (int i = g; i < nK; i += nthreads) {       // i = k * dqk + j  (coalesced read of W[k][j])
    const int k = i / P.dqk, j = i - k * P.dqk;
    const int o = canon_off(j, k, P.d);
    P.imgK[o] = P.Wk[i];
    P.imgQ[o] = P.Wq[i];
  }
  const int nV = kCandTile * P.d;
  for (int i = g; i < nV; i += nthreads) {       // i = k * 128 + j ; rows j >= d are zero
    const int k = i / kCandTile, j = i - k * kCandTile;
    P.imgV[canon_off(j, k, P.d)] = j < P.d ? P.Wv[(size_t)k * P.d + j] : __float2bfloat16_rn(0.f);
  }
  if (P.Wg) {
    gsta_build_images(P.Wg, P.gimg, P.d, P.M, g, nthreads);
    gsta_build_nseg(P.lengths, P.cand_offsets, P.U, P.N, P.L, P.S, P.Lp, P.status, P.gnseg, g >> 5, nthreads >> 5, tid & 31);
  }
}

// H' rows of segments without valid items are zero rows (only needed when the caller wants H').
__global__ void __launch_bounds__(256) tc_zero_empty_kernel(TcParams P) {
  const int u = blockIdx.y, seg = blockIdx.x;
  chain_wait();
  chain_release();
  const UserShape s = user_shape(P, u);
  if (seg < s.nseg || s.nc == 0) return;
  const int vec = P.d / 8;   // 16-byte chunks per row
  for (int i = threadIdx.x; i < s.nc * vec; i += blockDim.x) {
    const int c = i / vec, q = i - c * vec;
    *reinterpret_cast<uint4*>(P.Hp + ((size_t)(s.c0 + c) * P.Lp + seg) * P.d + q * 8) = make_uint4(0, 0, 0, 0);
  }
}

// ------------------------------------------------------------------------------------------------------- projection
// One unit = up to 128 item rows of one segment (K rows and V^T columns of whole item tiles), or one 128-candidate
// tile (Q rows).  Every block takes a contiguous range of the item units (no empty ones: tc_prep_kernel counted them)
// and runs them through a two-deep pipeline: while unit n is multiplied (two MMA groups into TMEM: rows x d_qk for K,
// d x rows for V^T) and drained by the eight warps (warp w reads TMEM lanes 32 (w mod 4) .. +31 and one half of the
// columns), the rows of unit n + 1 are already on their way into the other staging buffer: tiled TMA loads in the
// 128-byte swizzled layout when the item layout allows, else cp.async into the canonical K-major layout.  Afterwards the blocks share out the candidate tiles (Q = T W_q / 2 gamma) the same way.
struct ProjUnit {
  int u, seg, t0, rows, seg_items;      // item unit: tiles t0.. of segment seg; rows = staged rows; valid items of seg
  int jt, c0, nc;                       // candidate unit: tile jt of user u, whose candidates are [c0, c0 + nc)
};

__global__ void __launch_bounds__(kProjThreads) tc_proj_kernel(TcParams P, const __grid_constant__ CUtensorMap tmap_items,
                                                              int use_tma) {
  extern __shared__ __align__(1024) uint8_t proj_smem[];
  __shared__ uint64_t bar_img, bar_mma, bar_x[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ int s_kcol[16];            // per 8-column group of K / Q: (head << 8) | (8-column chunk within the head)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quad = warp & 3, half = warp >> 2;
  const int d = P.d, dqk = P.dqk, IT = P.IT;
  bf16* imgK = reinterpret_cast<bf16*>(proj_smem);          // W_k^T, later W_q^T
  bf16* imgV = imgK + dqk * d;
  bf16* Xbuf = imgV + kCandTile * d;                       // [2][128 x d]

  if (tid == 0) {
    mbar_init(&bar_img, 1);
    mbar_init(&bar_mma, 1);
    mbar_init(&bar_x[0], 1);
    mbar_init(&bar_x[1], 1);
    s_abort = 0;
    fence_mbar_init();
  }
  if (tid < (dqk >> 3)) {
    const int col = tid * 8, h = col / P.dqh;
    s_kcol[tid] = (h << 8) | ((col - h * P.dqh) >> 3);
  }
  if (warp == 0) {
    tmem_alloc(&s_tmem, kProjTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;
  const uint32_t bK = dqk * d * 2, bV = kCandTile * d * 2;
  if (smem_u32(Xbuf) & 1023u) use_tma = 0;   // (the swizzled layout needs 1024-byte aligned buffers; else plain copies)
  chain_wait();                         // the set-up kernel's images, prefixes and start cursors are complete
  chain_release();

  if (tid == 0) {
    mbar_arrive_expect_tx(&bar_img, bK + bV);
    bulk_g2s(imgK, P.imgK, bK, &bar_img);
    bulk_g2s(imgV, P.imgV, bV, &bar_img);
  }

  const uint32_t sbo = (d >> 3) * 128, lbo = 128;
  const uint32_t tmem_lane = tmem + ((uint32_t)(quad * 32) << 16);
  uint32_t mma_phase = 0;

  // staging: a 16-byte piece is (8-row group, 8-column chunk, row in group); this thread copies pieces
  // (tid >> 3) + 32 i of row (tid & 7) in their group, i.e. it walks (group, chunk) with a fixed stride
  const int cpr = d >> 3;                              // 8-column chunks per row
  const int step_g = 32 / cpr, step_c = 32 % cpr;
  const int g0 = (tid >> 3) / cpr, c0 = (tid >> 3) % cpr;
  auto stage = [&](const ProjUnit& pu, bool is_item, bf16* X) {
    const int n_groups = pu.rows >> 3;
    const bf16* base;
    int row_limit;                                         // rows at or past it are staged as zeros
    if (is_item) {
      const int n0 = pu.seg * P.S + pu.t0 * IT;            // unit row r is item n0 + r
      if (P.item_off) {                                    // packed rows: never read past the user's valid prefix
        base = P.items + ((size_t)P.item_off[pu.u] + n0) * d;
        row_limit = pu.seg_items - pu.t0 * IT;
      } else {
        base = P.items + ((size_t)pu.u * P.L + n0) * d;
        row_limit = P.L - n0;
      }
    } else {
      base = P.cands + (size_t)(pu.c0 + pu.jt * kCandTile) * d;
      row_limit = pu.nc - pu.jt * kCandTile;
    }
    int gq = g0, c = c0;
    while (gq < n_groups) {
      const int r = (gq << 3) + (tid & 7);
      const bool in = r < row_limit;
      cp_async16(X + (gq * cpr + c) * 64 + (tid & 7) * 8, in ? base + (size_t)r * d + c * 8 : base, in ? 16u : 0u);
      gq += step_g;
      c += step_c;
      if (c >= cpr) { c -= cpr; ++gq; }
    }
  };
  // K / Q epilogue: this thread owns row r0 of the unit
  const int r0 = quad * 32 + lane;
  const int r0_tile = r0 / IT, r0_in = r0 - r0_tile * IT;
  const int cpr_k = P.dqh >> 3;                        // 8-element chunks per head row
  const int n16k = dqk >> 4, k_lo = half ? (n16k + 1) >> 1 : 0, k_hi = half ? n16k : (n16k + 1) >> 1;
  // V^T epilogue: this thread owns value feature j
  const int j = quad * 32 + lane;
  const int jh = j / P.dvh, jj = j - jh * P.dvh;
  const int npr = P.dvh >> 3;                          // 8-row groups per head

  // multiply the staged unit and drain the accumulators
  // x_bar: null when the rows were staged with cp.async (canonical layout, already complete); else the mbarrier of
  // the TMA copies that bring them in the 128-byte swizzled layout (two 64-column halves of 128 rows, 16 KB apart).
  auto run_unit = [&](const ProjUnit& pu, bool is_item, bf16* X, uint64_t* x_bar, uint32_t x_phase) -> bool {
    if (warp == 0) {                                         // warp-uniform loop, one elected lane issues
      const bool staged = x_bar == nullptr || mbar_wait(x_bar, x_phase, abortp);
      __syncwarp();
      tc_fence_after();
      const uint32_t xa = smem_u32(X);
      const uint64_t wd = smem_desc(smem_u32(imgK), lbo, sbo), vd = smem_desc(smem_u32(imgV), lbo, sbo);
      const int ksteps = d >> 4;
      const uint32_t id1 = idesc_bf16(128, dqk), id2 = idesc_bf16(128, pu.rows);
      auto xdesc = [&](int ks) -> uint64_t {
        return x_bar ? smem_desc_sw128(xa + (uint32_t)(ks >> 2) * (kCandTile * 128)) + (uint64_t)((ks & 3) * 2)
                     : smem_desc(xa, lbo, sbo) + (uint64_t)(ks * 16);
      };
      if (staged && elect_one()) {
        for (int ks = 0; ks < ksteps; ++ks) mma_ss(tmem, xdesc(ks), wd + ks * 16, id1, ks > 0);
        if (is_item)
          for (int ks = 0; ks < ksteps; ++ks) mma_ss(tmem + 128, vd + ks * 16, xdesc(ks), id2, ks > 0);
        tc_commit(&bar_mma);
      }
      __syncwarp();
    }
    const bool ok = __syncthreads_and(mbar_wait(&bar_mma, mma_phase, abortp));
    mma_phase ^= 1;
    if (!ok) return false;
    tc_fence_after();
    const int rows = pu.rows;

    // ---- K (or Q) rows.  TMEM lane = row of the unit; this warp's half of the columns, 16 per load.
    if (quad * 32 < rows) {
      const float scale = is_item ? 1.f : P.q_scale;
      bool valid;
      bf16* dst_row;                                       // start of row r0 inside head 0's block of its tile
      size_t head_stride;
      if (is_item) {
        const int pos = (pu.t0 + r0_tile) * IT + r0_in;
        valid = r0 < rows && pos < pu.seg_items;
        dst_row = P.Kblk + ((size_t)pu.u * P.n_tiles + pu.seg * P.NT + pu.t0 + r0_tile) * ((size_t)IT * dqk) +
                  (r0_in >> 3) * (cpr_k * 64) + (r0_in & 7) * 8;
        head_stride = (size_t)IT * P.dqh;
      } else {
        valid = pu.jt * kCandTile + r0 < pu.nc;
        dst_row = P.Qblk + (size_t)(P.tile_off[pu.u] + pu.jt) * (kCandTile * dqk) + (r0 >> 3) * (cpr_k * 64) + (r0 & 7) * 8;
        head_stride = (size_t)kCandTile * P.dqh;
      }
      for (int c16 = k_lo; c16 < k_hi; ++c16) {
        uint32_t v[16];
        tmem_ld16(tmem_lane + c16 * 16, v);
        tc_wait_ld();
        if (r0 < rows) {
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            const int info = s_kcol[c16 * 2 + hf];
            uint4 o = make_uint4(0, 0, 0, 0);
            if (valid) {
              o.x = pack_bf16x2(__uint_as_float(v[hf * 8 + 0]) * scale, __uint_as_float(v[hf * 8 + 1]) * scale);
              o.y = pack_bf16x2(__uint_as_float(v[hf * 8 + 2]) * scale, __uint_as_float(v[hf * 8 + 3]) * scale);
              o.z = pack_bf16x2(__uint_as_float(v[hf * 8 + 4]) * scale, __uint_as_float(v[hf * 8 + 5]) * scale);
              o.w = pack_bf16x2(__uint_as_float(v[hf * 8 + 6]) * scale, __uint_as_float(v[hf * 8 + 7]) * scale);
            }
            *reinterpret_cast<uint4*>(dst_row + (info >> 8) * head_stride + (info & 255) * 64) = o;
          }
        }
      }
    }
    // ---- V^T.  TMEM lane = value feature j; columns = rows of the unit, this warp's half of them.
    if (is_item && quad * 32 < d) {
      const int n16 = rows >> 4;
      const int lo16 = half ? (n16 + 1) >> 1 : 0, hi16 = half ? n16 : (n16 + 1) >> 1;
      auto store_v = [&](int c16, const uint32_t (&v)[16]) {
        const int rr = c16 * 16;                          // unit row of the first of these 16 columns
        const int tt = rr / IT, in_tile = rr - tt * IT;   // IT is a multiple of 16: the 16 columns share a tile
        const int n_valid = pu.seg_items - ((pu.t0 + tt) * IT + in_tile);   // valid items among them (<= 0 .. >= 16)
        bf16* dst = P.Vtblk + ((size_t)pu.u * P.n_tiles + pu.seg * P.NT + pu.t0 + tt) * ((size_t)IT * d) +
                    (size_t)jh * IT * P.dvh + ((in_tile >> 3) * npr + (jj >> 3)) * 64 + (jj & 7) * 8;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int cnt = n_valid - hf * 8;
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float a = __uint_as_float(v[hf * 8 + 2 * e]), b = __uint_as_float(v[hf * 8 + 2 * e + 1]);
            if (cnt < 8) {                                // ragged end of the segment: masked items are exact zeros
              if (2 * e >= cnt) a = 0.f;
              if (2 * e + 1 >= cnt) b = 0.f;
            }
            pk[e] = pack_bf16x2(a, b);
          }
          *reinterpret_cast<uint4*>(dst + hf * npr * 64) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      };
      int c16 = lo16;
      for (; c16 + 2 <= hi16; c16 += 2) {                   // two accumulator loads in flight per wait
        uint32_t v0[16], v1[16];
        tmem_ld16(tmem_lane + 128 + c16 * 16, v0);
        tmem_ld16(tmem_lane + 128 + c16 * 16 + 16, v1);
        tc_wait_ld();
        if (j < d) {
          store_v(c16, v0);
          store_v(c16 + 1, v1);
        }
      }
      if (c16 < hi16) {
        uint32_t v0[16];
        tmem_ld16(tmem_lane + 128 + c16 * 16, v0);
        tc_wait_ld();
        if (j < d) store_v(c16, v0);
      }
    }
    tc_fence_before();
    return true;
  };

  // ---- item units: this block's contiguous range, two-deep pipeline
  bool ok = true;
  const int n_proj = P.counters[2];
  const int G = gridDim.x, bidx = blockIdx.x;
  const int lo = (int)(((long long)n_proj * bidx) / G), hi = (int)(((long long)n_proj * (bidx + 1)) / G);
  if (hi <= lo) ok = __syncthreads_and(mbar_wait(&bar_img, 0, abortp));
  else {
    // cursor over (user, segment, tile group)
    int cu, cseg, cgrp, c_nseg, c_len, c_last_groups;
    auto set_len = [&](int len) {
      c_len = len;
      c_nseg = (len + P.S - 1) / P.S;
      const int last_items = c_nseg > 0 ? len - (c_nseg - 1) * P.S : 0;
      c_last_groups = (min(P.NT, (last_items + IT - 1) / IT) + P.NTG - 1) / P.NTG;
    };
    auto load_user = [&]() { set_len(user_shape(P, cu).len); };
    {
      const int4 b = P.proj_begin[bidx];                     // this block's first unit and its user's (sanitised) length,
      cu = b.x; cseg = b.y; cgrp = b.z;                      // as found by tc_prep_kernel: one load before the first copy
      set_len(b.w);
    }
    auto make_unit = [&]() {
      ProjUnit pu;
      pu.u = cu; pu.seg = cseg; pu.t0 = cgrp * P.NTG;
      pu.seg_items = min(P.S, c_len - cseg * P.S);
      const int t1 = min(min(P.NT, pu.t0 + P.NTG), (pu.seg_items + IT - 1) / IT);   // tiles with valid items only
      pu.rows = (t1 - pu.t0) * IT;
      pu.jt = 0; pu.c0 = 0; pu.nc = 0;
      return pu;
    };
    auto step = [&]() {
      const int groups = cseg == c_nseg - 1 ? c_last_groups : P.NG;
      if (++cgrp < groups) return;
      cgrp = 0;
      if (++cseg < c_nseg) return;
      cseg = 0;
      do {
        ++cu;
        if (cu >= P.U) return;
        load_user();
      } while (c_nseg == 0);
    };

    ProjUnit cur = make_unit();
    int buf = 0;
    if (use_tma) {
      // One thread asks the TMA unit for the rows of a unit: per item tile and 64-column half one tiled copy (IT rows of
      // 128 bytes, 128-byte swizzle), all completing on the buffer's mbarrier.  Rows past the end of the item array
      // arrive as zeros; rows past the user's block are another user's (finite) rows and are masked like padding.
      auto fetch = [&](const ProjUnit& pu, int b) {
        const uint32_t dst = smem_u32(Xbuf + (size_t)b * kCandTile * d);
        const int row0 = pu.u * P.L + pu.seg * P.S + pu.t0 * IT;
        mbar_arrive_expect_tx(&bar_x[b], (uint32_t)pu.rows * d * 2);
        for (int t = 0; t * IT < pu.rows; ++t)
          for (int kh = 0; kh * 64 < d; ++kh)
            tma_load_2d(dst + kh * (kCandTile * 128) + t * IT * 128, &tmap_items, kh * 64, row0 + t * IT, &bar_x[b]);
      };
      uint32_t x_phase[2] = {0, 0};
      bool in_flight = true;                // a unit was requested and not yet multiplied
      if (tid == 0) fetch(cur, 0);          // (before the wait for the weight images: the two round trips overlap)
      ok = __syncthreads_and(mbar_wait(&bar_img, 0, abortp));
      for (int n = lo; n < hi && ok; ++n) {
        ProjUnit nxt = cur;
        in_flight = n + 1 < hi;
        if (in_flight) {
          step();
          nxt = make_unit();
          if (tid == 0) fetch(nxt, buf ^ 1);   // (its last readers, the MMAs of unit n - 1, have completed)
        }
        __syncthreads();                    // TMEM of unit n - 1 drained
        ok = run_unit(cur, true, Xbuf + (size_t)buf * kCandTile * d, &bar_x[buf], x_phase[buf]);
        x_phase[buf] ^= 1;
        cur = nxt;
        buf ^= 1;
      }
      // giving up with a copy still on its way: let it land (bounded) before the block may exit
      if (!ok && in_flight && tid == 0)
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(&bar_x[buf], x_phase[buf]); ++i) __nanosleep(64);
    } else {
      ok = __syncthreads_and(mbar_wait(&bar_img, 0, abortp));
      if (ok) stage(cur, true, Xbuf);
      asm volatile("cp.async.commit_group;" ::: "memory");
      for (int n = lo; n < hi && ok; ++n) {
        ProjUnit nxt = cur;
        if (n + 1 < hi) {
          step();
          nxt = make_unit();
          stage(nxt, true, Xbuf + (size_t)(buf ^ 1) * kCandTile * d);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        fence_proxy_async_smem();
        __syncthreads();                    // unit n staged by every thread; TMEM of unit n - 1 drained
        ok = run_unit(cur, true, Xbuf + (size_t)buf * kCandTile * d, nullptr, 0);
        cur = nxt;
        buf ^= 1;
      }
    }
  }

  // ---- candidate tiles, dealt round-robin over the blocks (W_q^T replaces W_k^T in shared memory)
  const int n_ctiles = P.counters[1];
  if (ok && bidx < n_ctiles) {
    __syncthreads();                      // every MMA that read W_k^T or the staging buffer has completed (drained)
    if (tid == 0) {
      mbar_arrive_expect_tx(&bar_img, bK);
      bulk_g2s(imgK, P.imgQ, bK, &bar_img);
    }
    auto cand_unit = [&](int ct) {          // (user, tile, first candidate, candidates), tabulated by tc_prep_kernel
      const int4 e = P.ctile[ct];
      ProjUnit pu;
      pu.u = e.x; pu.seg = 0; pu.t0 = 0; pu.rows = kCandTile; pu.seg_items = 0;
      pu.jt = e.y; pu.c0 = e.z; pu.nc = e.w;
      return pu;
    };
    ProjUnit pu = cand_unit(bidx);
    stage(pu, false, Xbuf);                 // the first tile's rows travel together with W_q^T
    ok = __syncthreads_and(mbar_wait(&bar_img, 1, abortp));
    for (int ct = bidx; ct < n_ctiles && ok; ct += G) {
      if (ct != bidx) {
        pu = cand_unit(ct);
        __syncthreads();                    // staging buffer and TMEM of the previous unit are free
        stage(pu, false, Xbuf);
      }
      cp_async_wait_all();
      fence_proxy_async_smem();
      __syncthreads();
      ok = run_unit(pu, false, Xbuf, nullptr, 0);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kProjTmemCols);
  if (tid == 0 && s_abort) report_status(P.status, LASER_ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------------- attention
// Walks the attention units (user, candidate tile, segment) of a contiguous id range in order.  The user's shape is
// cached, so a step inside one user costs a few integer instructions.
struct UnitWalker {
  int u, j, seg;
  int nseg, ctiles, c0, nc, last_items, last_tiles;
  __device__ void load_user(const TcParams& P) {
    const UserShape s = user_shape(P, u);
    nseg = s.nseg; ctiles = s.ctiles; c0 = s.c0; nc = s.nc;
    last_items = s.nseg > 0 ? s.len - (s.nseg - 1) * P.S : 0;       // items of the last non-empty segment
    last_tiles = min(P.NT, (last_items + P.IT - 1) / P.IT);
  }
  __device__ void init(const TcParams& P) {       // this block's first unit, as found by tc_prep_kernel
    const int4 b = P.sta_begin[blockIdx.x];
    u = b.x; j = b.y; seg = b.z;
    load_user(P);
  }
  __device__ void next(const TcParams& P) {
    if (++seg < nseg) return;
    seg = 0;
    if (++j < ctiles) return;
    j = 0;
    do {
      ++u;
      if (u >= P.U) return;
      load_user(P);
    } while (nseg == 0 || ctiles == 0);
  }
  // tiles of the current segment that hold at least one valid item
  __device__ int ntiles(const TcParams& P) const { return seg == nseg - 1 ? last_tiles : P.NT; }
  // columns of tile t that can hold a non-zero gate: its valid items rounded up to the MMA k-step (16)
  __device__ int tile_items(const TcParams& P, int t) const {
    return min(P.IT, (seg == nseg - 1 ? last_items : P.S) - t * P.IT);
  }
  __device__ int tile_cols(const TcParams& P, int t) const { return (tile_items(P, t) + 15) & ~15; }
};

struct StaBars {
  uint64_t q_full[2], q_empty[2];
  uint64_t kv_full[kKvStages], kv_empty[kKvStages];
  uint64_t s_full[kGateGroups], s_free[kGateGroups], p_full[kGateGroups], p_free[kGateGroups];
  uint64_t o_full[2], o_empty[2];
  uint64_t done[kGateGroups];
};

constexpr int kProducerWarp = 8 + 4 * kGateGroups;
constexpr int kItMax = 64;                          // items per tile: one 64-column fp32 score buffer per warpgroup
constexpr uint32_t kColS = 0;                       // TMEM: scores  [kGateGroups][kItMax] fp32
constexpr uint32_t kColP = kGateGroups * kItMax;    //       gates   [kGateGroups][kItMax / 2] packed bf16 pairs
constexpr uint32_t kColO = kColP + kGateGroups * (kItMax / 2);   // outputs [n_obuf][d] fp32

// Roles of the 25 warps of a block (one block per SM):
//   warps 0-3   MMA issuers, one per gate warpgroup (the warp runs the loop, one elected lane issues)
//   warps 4-7   epilogue: H' = O / 2 per finished segment, staged in shared memory, written by bulk stores
//               (with at most two heads, warps 16-19 are a second epilogue group: one group per output accumulator)
//   warps 8-23  four gate warpgroups: P = 1 + tanh(S)
//   warp 24     bulk-copy producer (Q tile per (user, candidate tile), K / V^T tile per item tile, mbarrier rings) and
//               TMEM allocation
// A gate-unit is one (item tile, head).  Head h always belongs to warpgroup / issuer h % 4, which owns one score buffer
// and one gate buffer in TMEM.  Per unit: the issuer writes S = Q_h K_h^T; the warpgroup reads it (releasing the score
// buffer for the issuer's next unit as soon as the last column is in registers), writes P = 1 + tanh(S) as packed bf16;
// the issuer accumulates O_h += P V_h.  All MMAs into a head's accumulator come from one thread, in order.
//
// kSoftmax selects the softmax-aggregation variant (the paper's ablation of the sigmoid gate): the weights of a segment's
// valid items are exp(q_h . k_{n,h} / gamma) normalised to one per (candidate, head).  A gate thread owns one candidate
// row of the score buffer, so the row sums are plain per-thread accumulations over the tiles of the segment; they reach
// the epilogue through shared memory (a ring of four segments), and the epilogue divides each head's columns by its sum
// instead of halving them.  The exponent is shifted by the row's maximum over the first 32 valid items of the segment
// (any shift cancels in the quotient; this one keeps the sum >= 1) and capped at 2^60 above that shift.
constexpr int kSumSlots = 4;
constexpr float kExpCap = 60.f;
template <bool kSoftmax>
__global__ void __launch_bounds__(kStaThreads, 1) tc_sta_kernel(TcParams P) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  __shared__ StaBars bars;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int d = P.d, dqk = P.dqk, IT = P.IT, H = P.H;
  const int n_groups = H < kGateGroups ? H : kGateGroups;     // warpgroups / issuers that own at least one head
  const uint32_t q_bytes = kCandTile * dqk * 2, k_bytes = IT * dqk * 2, v_bytes = IT * d * 2;
  const uint32_t out_row = d * 2 + 16;            // bytes per staged output row (padding spreads the banks)
  uint8_t* Qs = smem_raw;                         // [2][q_bytes]
  uint8_t* Ks = Qs + 2 * q_bytes;                 // [kKvStages][k_bytes]
  uint8_t* Vs = Ks + kKvStages * k_bytes;         // [kKvStages][v_bytes]
  uint8_t* Os = Vs + kKvStages * v_bytes;         // [2][kCandTile][out_row]  staged H' rows
  float* Sums = reinterpret_cast<float*>(Os + 2 * kCandTile * out_row);   // [kSumSlots][H][kCandTile] (kSoftmax only)

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars.q_full[i], 1);
      mbar_init(&bars.q_empty[i], n_groups);      // every issuer releases the old Q tile
      mbar_init(&bars.o_full[i], n_groups);       // every issuer finishes its heads of the segment
      mbar_init(&bars.o_empty[i], 4);
    }
    for (int i = 0; i < kGateGroups; ++i) {
      mbar_init(&bars.s_full[i], 1);
      mbar_init(&bars.s_free[i], 4);
      mbar_init(&bars.p_full[i], 4);
      mbar_init(&bars.p_free[i], 1);
      mbar_init(&bars.done[i], 1);
    }
    for (int i = 0; i < kKvStages; ++i) {
      mbar_init(&bars.kv_full[i], 1);
      mbar_init(&bars.kv_empty[i], H);            // one arrival per (tile, head)
    }
    s_abort = 0;
    fence_mbar_init();
  }
  if (warp == kProducerWarp) {
    tmem_alloc(&s_tmem, kStaTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;
  const int n_obuf = P.n_obuf;
  const bool two_epilogues = n_groups <= 2 && n_obuf == 2;    // gate warpgroup 2 has no head: it drains accumulator 1
  chain_wait();                         // K, V^T and Q tiles are complete
  chain_release();

  // this block's contiguous range of units
  const int n_units = P.counters[0];
  const int G = gridDim.x, b = blockIdx.x;
  const int unit_lo = (int)(((long long)n_units * b) / G);
  const int unit_hi = (int)(((long long)n_units * (b + 1)) / G);
  const int my_units = unit_hi - unit_lo;

  if (my_units > 0) {
    if (warp == kProducerWarp) {
      // ------------------------------------------------------------------ bulk-copy producer
      if (lane == 0) {
        UnitWalker w;
        w.init(P);
        int pu = -1, pj = -1;
        uint32_t qcount = 0, st = 0, kv_par = 1;      // kv_par: parity that means "stage st is free"
        uint32_t kv_armed = 0, kv_full_par = 0;       // per stage (bit): requested at least once; parity of its last request
        bool ok = true;
        for (int it = 0; it < my_units && ok; ++it, w.next(P)) {
          if (w.u != pu || w.j != pj) {
            const int qs = qcount & 1;
            ok = mbar_wait(&bars.q_empty[qs], ((qcount >> 1) & 1) ^ 1, abortp);
            if (!ok) break;
            mbar_arrive_expect_tx(&bars.q_full[qs], q_bytes);
            bulk_g2s(Qs + qs * q_bytes, P.Qblk + (size_t)(P.tile_off[w.u] + w.j) * (kCandTile * dqk), q_bytes,
                     &bars.q_full[qs]);
            ++qcount;
            pu = w.u;
            pj = w.j;
          }
          const int nt = w.ntiles(P);
          const size_t tile0 = (size_t)w.u * P.n_tiles + w.seg * P.NT;
          for (int t = 0; t < nt && ok; ++t) {
            ok = mbar_wait(&bars.kv_empty[st], kv_par, abortp);
            if (!ok) break;
            mbar_arrive_expect_tx(&bars.kv_full[st], k_bytes + v_bytes);
            bulk_g2s(Ks + st * k_bytes, P.Kblk + (tile0 + t) * ((size_t)IT * dqk), k_bytes, &bars.kv_full[st]);
            bulk_g2s(Vs + st * v_bytes, P.Vtblk + (tile0 + t) * ((size_t)IT * d), v_bytes, &bars.kv_full[st]);
            kv_armed |= 1u << st;
            kv_full_par = (kv_full_par & ~(1u << st)) | ((kv_par ^ 1u) << st);
            if (++st == kKvStages) { st = 0; kv_par ^= 1; }
          }
        }
        if (!ok) {
          // giving up with copies possibly still on their way into this block's shared memory: let every requested
          // stage and Q tile land (bounded) before the block releases its resources
          for (uint32_t i = 0; i < (uint32_t)kKvStages; ++i)
            if (kv_armed >> i & 1u) mbar_drain(&bars.kv_full[i], kv_full_par >> i & 1u);
          for (uint32_t i = 0; i < 2 && i < qcount; ++i) {
            const uint32_t n = qcount - 1 - i;                    // the last two Q requests: buffer n & 1, round n >> 1
            mbar_drain(&bars.q_full[n & 1], (n >> 1) & 1);
          }
        }
      }
    } else if (warp < kGateGroups) {
      // ------------------------------------------------------------------ MMA issuer of warpgroup `warp`
      // The whole warp runs the loop, so that addresses and descriptors stay warp-uniform; one elected lane issues.
      if (warp < n_groups) {
        const int wgi = warp;
        const bool leader = elect_one();
        const uint32_t id1 = idesc_bf16(128, IT);        // scores: 128 candidates x IT items, K = dqh
        const uint32_t id2 = idesc_bf16(128, P.dvh);     // O_h: 128 candidates x dvh, K = the tile's items
        const uint32_t qk_sbo = (P.dqh >> 3) * 128;      // 8-row groups of a [rows x dqh] head block
        const uint32_t v_lbo = (P.dvh >> 3) * 128;       // V^T head block: k-chunks (8 items) are dvh/8 core matrices apart
        const int ks1 = P.dqh >> 4;
        const uint64_t q_desc0 = smem_desc(smem_u32(Qs), 128, qk_sbo);
        const uint64_t k_desc0 = smem_desc(smem_u32(Ks), 128, qk_sbo);
        const uint64_t v_desc0 = smem_desc(smem_u32(Vs), v_lbo, 128);
        const uint32_t q_head = (kCandTile * P.dqh * 2) >> 4, k_head = (IT * P.dqh * 2) >> 4;   // in 16-byte units
        const uint32_t v_head = (IT * P.dvh * 2) >> 4, v_step = (2 * v_lbo) >> 4;
        const uint32_t tS = tmem + kColS + wgi * kItMax, tP = tmem + kColP + wgi * (kItMax / 2);

        struct Cursor {
          UnitWalker w;
          int it, t, h, nt;
          uint32_t st, kv_par;                            // K / V stage of the current tile and its "full" parity
        };
        auto advance = [&](Cursor& c) -> bool {           // to this issuer's next gate-unit; false past the end
          c.h += kGateGroups;
          if (c.h < H) return true;
          c.h = wgi;
          if (++c.st == kKvStages) { c.st = 0; c.kv_par ^= 1; }
          if (++c.t < c.nt) return true;
          c.t = 0;
          if (++c.it >= my_units) return false;
          c.w.next(P);
          c.nt = c.w.ntiles(P);
          return true;
        };
        auto wait_all = [&](uint64_t* bar, uint32_t parity) {
          return __all_sync(0xffffffffu, mbar_wait(bar, parity, abortp)) != 0;
        };
        int qu = -1, qj = -1;
        uint32_t qcount = 0, sf_par = 0, p_par = 0, ob = 0, o_par = 1;
        uint64_t q_desc = q_desc0;
        bool ok = true;

        // Scores of a unit in two steps: everything that does not need the score buffer (the Q tile, the K tile, the
        // descriptors) first, so that once the warpgroup hands the buffer back only the MMA itself remains.
        uint64_t qd = 0, kd = 0;
        auto prepare_scores = [&](const Cursor& c) {
          if (c.w.u != qu || c.w.j != qj) {               // first unit on a new candidate tile
            if (qu >= 0 && leader) tc_commit(&bars.q_empty[(qcount - 1) & 1]);   // my score MMAs on the old Q tile are issued
            ok = wait_all(&bars.q_full[qcount & 1], (qcount >> 1) & 1);
            if (!ok) return;
            q_desc = q_desc0 + (uint64_t)((qcount & 1) * (q_bytes >> 4));
            ++qcount;
            qu = c.w.u;
            qj = c.w.j;
          }
          ok = wait_all(&bars.kv_full[c.st], c.kv_par);
          if (!ok) return;
          qd = q_desc + c.h * q_head;
          kd = k_desc0 + (uint64_t)(c.st * (k_bytes >> 4) + c.h * k_head);
        };
        auto fire_scores = [&]() {
          tc_fence_after();
          if (leader) {
            for (int ks = 0; ks < ks1; ++ks) mma_ss(tS, qd + ks * 16, kd + ks * 16, id1, ks > 0);
            tc_commit(&bars.s_full[wgi]);
          }
          __syncwarp();
        };
        auto issue_values = [&](const Cursor& c) {
          ok = wait_all(&bars.p_full[wgi], p_par);
          if (!ok) return;
          p_par ^= 1;
          if (c.t == 0 && c.h == wgi) {                   // my first unit of the segment: the accumulator must be drained
            ok = wait_all(&bars.o_empty[ob], o_par);
            if (!ok) return;
          }
          tc_fence_after();
          const uint32_t dO = tmem + (ob ? (uint32_t)P.o_col1 : kColO) + c.h * P.dvh;
          const uint64_t vd = v_desc0 + (uint64_t)(c.st * (v_bytes >> 4) + c.h * v_head);
          const int ks2 = c.w.tile_cols(P, c.t) >> 4;     // k-steps that hold valid items
          const bool last = c.t == c.nt - 1 && c.h + kGateGroups >= H;      // my last unit of the segment
          if (leader) {
#pragma unroll 4
            for (int ks = 0; ks < ks2; ++ks) mma_ts(dO, tP + ks * 8, vd + ks * v_step, id2, (c.t | ks) != 0);
            tc_commit(&bars.p_free[wgi]);
            tc_commit(&bars.kv_empty[c.st]);              // this unit's scores were consumed before its gates existed
            if (last) tc_commit(&bars.o_full[ob]);
          }
          __syncwarp();
          if (last && (int)++ob == n_obuf) { ob = 0; o_par ^= 1; }
        };

        Cursor cur;
        cur.w.init(P);
        cur.it = 0; cur.t = 0; cur.h = wgi; cur.nt = cur.w.ntiles(P); cur.st = 0; cur.kv_par = 0;
        prepare_scores(cur);
        if (ok) fire_scores();
        while (ok) {
          Cursor nxt = cur;
          const bool more = advance(nxt);
          if (more) {                                     // next scores as soon as the warpgroup has read the current ones
            prepare_scores(nxt);
            if (!ok) break;
            ok = wait_all(&bars.s_free[wgi], sf_par);
            if (!ok) break;
            sf_par ^= 1;
            fire_scores();
          }
          issue_values(cur);
          if (!more) break;
          cur = nxt;
        }
        // every MMA issued by the leader has completed once `done` flips (also awaited, bounded, by a block that gave up:
        // its tensor memory must not be released under MMAs that still write to it)
        if (leader) tc_commit(&bars.done[wgi]);
        __syncwarp();
        mbar_drain(&bars.done[wgi], 0);
      }
    } else if (warp >= 8 && warp < kProducerWarp && !(two_epilogues && ((warp - 8) >> 2) == 2)) {
      // ------------------------------------------------------------------ gate warps: P = 1 + tanh(scores)
      const int wg = (warp - 8) >> 2;                       // warpgroup wg owns buffers wg and heads wg, wg + 4, ...
      const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
      const uint32_t tS = tmem + lane_base + kColS + wg * kItMax;
      const uint32_t tP = tmem + lane_base + kColP + wg * (kItMax / 2);
      UnitWalker w;
      w.init(P);
      uint32_t s_par = 0, pf_par = 1;
      int my_heads = 0;
      for (int h = wg; h < H; h += kGateGroups) ++my_heads;
      bool ok = wg < n_groups;
      auto release_scores = [&]() {                         // every score column of the unit is in registers
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.s_free[wg]);
      };
      // softmax variant: per head of this warpgroup (at most two), this row's exponent shift and running sum
      const float k2 = 2.f * 1.4426950408889634f;           // the scores hold q.k / (2 gamma); weights are 2^(k2 s - shift)
      float sh0 = 0.f, sh1 = 0.f, rs0 = 0.f, rs1 = 0.f;
      const int row = (warp & 3) * 32 + lane;
      for (int it = 0; it < my_units && ok; ++it, w.next(P)) {
        const int nt = w.ntiles(P);
        for (int t = 0; t < nt && ok; ++t) {
          const int cols = w.tile_cols(P, t);               // columns past this hold zero K rows: their gates are 0
          const int items = w.tile_items(P, t);
          for (int hh = 0; hh < my_heads && ok; ++hh) {
            ok = __all_sync(0xffffffffu, mbar_wait(&bars.s_full[wg], s_par, abortp));
            if (!ok) break;
            s_par ^= 1;
            tc_fence_after();
            bool first = true;
            float shift = hh ? sh1 : sh0, rsum = (t == 0) ? 0.f : (hh ? rs1 : rs0);
            // weights of `n` score columns starting at column c: packed bf16 pairs, summed as the MMA will see them
            auto weights = [&](const uint32_t* v, uint32_t* o, int c, int n) {
              if (t == 0 && c == 0) {
                float mx = -INFINITY;
#pragma unroll
                for (int e = 0; e < 16; ++e) if (e < n && e < items) mx = fmaxf(mx, __uint_as_float(v[e]));
#pragma unroll
                for (int e = 16; e < 32; ++e) if (e < n && e < items) mx = fmaxf(mx, __uint_as_float(v[e]));
                shift = mx * k2;
              }
              const bool whole = c + n <= items;
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                if (2 * e < n) {
                  float p0, p1;
                  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p0) : "f"(fminf(fmaf(__uint_as_float(v[2 * e]), k2, -shift), kExpCap)));
                  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p1) : "f"(fminf(fmaf(__uint_as_float(v[2 * e + 1]), k2, -shift), kExpCap)));
                  if (!whole) {                             // padding columns of the segment's last 16-column group
                    if (c + 2 * e >= items) p0 = 0.f;
                    if (c + 2 * e + 1 >= items) p1 = 0.f;
                  }
                  const uint32_t pk = pack_bf16x2(p0, p1);
                  rsum += __uint_as_float(pk << 16) + __uint_as_float(pk & 0xFFFF0000u);
                  o[e] = pk;
                }
              }
            };
            int c = 0;
            for (; c + 32 <= cols; c += 32) {
              uint32_t v[32], o[16];
              tmem_ld32(tS + c, v);
              tc_wait_ld();
              if (c + 32 >= cols) release_scores();
              if (kSoftmax) {
                weights(v, o, c, 32);
              } else {
#pragma unroll
                for (int e = 0; e < 16; ++e)
                  o[e] = pack_bf16x2(1.f + tanh_approx(__uint_as_float(v[2 * e])), 1.f + tanh_approx(__uint_as_float(v[2 * e + 1])));
              }
              if (first) {                                  // the previous unit's gates have been multiplied
                ok = __all_sync(0xffffffffu, mbar_wait(&bars.p_free[wg], pf_par, abortp));
                pf_par ^= 1;
                first = false;
                tc_fence_after();
              }
              tmem_st16(tP + (c >> 1), o);
            }
            if (c < cols) {   // 16-column tail
              uint32_t v[32], o[16];
              {
                uint32_t v16[16];
                tmem_ld16(tS + c, v16);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = v16[e];
              }
              release_scores();
              if (kSoftmax) {
                weights(v, o, c, 16);
              } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  o[e] = pack_bf16x2(1.f + tanh_approx(__uint_as_float(v[2 * e])), 1.f + tanh_approx(__uint_as_float(v[2 * e + 1])));
              }
              if (first) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars.p_free[wg], pf_par, abortp));
                pf_par ^= 1;
                first = false;
                tc_fence_after();
              }
              uint32_t o8[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) o8[e] = o[e];
              tmem_st8(tP + (c >> 1), o8);
            }
            if (kSoftmax) {
              if (hh) { sh1 = shift; rs1 = rsum; } else { sh0 = shift; rs0 = rsum; }
              if (t == nt - 1) Sums[((it & (kSumSlots - 1)) * H + wg + kGateGroups * hh) * kCandTile + row] = rsum;
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars.p_full[wg]);
          }
        }
      }
    } else if (warp >= 4) {
      // ------------------------------------------------------------------ epilogue: H' = O / 2
      // Warps 4-7; with at most two heads, warps 16-19 (whose gate warpgroup has no head) are a second epilogue group:
      // the two output accumulators alternate segment by segment, so group e drains accumulator e, every other unit.
      const int q = warp & 3, eg = warp >= 8 ? 1 : 0;
      const uint32_t lane_base = (uint32_t)(q * 32) << 16;
      const int m = q * 32 + lane;
      UnitWalker w;
      w.init(P);
      uint32_t ob = two_epilogues ? (uint32_t)eg : 0u, o_par = 0;
      bool ok = true;
      for (int it = 0; it < my_units && ok; ++it, w.next(P)) {
        if (two_epilogues && (it & 1) != eg) continue;
        uint8_t* row = Os + ((size_t)(it & 1) * kCandTile + m) * out_row;
        if (two_epilogues) bulk_wait_read<0>();            // my previous store has left this group's staging buffer
        else bulk_wait_read<1>();                          // my store from this staging buffer (two units ago) has left it
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(&bars.o_full[ob], o_par, abortp));
        if (!ok) break;
        tc_fence_after();
        const uint32_t tO = tmem + lane_base + (ob ? (uint32_t)P.o_col1 : kColO);
        auto hand_back = [&]() {                           // the accumulator is in registers
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars.o_empty[ob]);
        };
        // sigmoid gates: H' = O / 2; softmax variant: the 16 columns' head divides by its row sum
        const float* sums = Sums + (size_t)((it & (kSumSlots - 1)) * H) * kCandTile + m;
        auto factor = [&](int c) { return kSoftmax ? 1.f / sums[(c / P.dvh) * kCandTile] : 0.5f; };
        auto stage16 = [&](int c, const uint32_t (&v)[16], float f) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint4 o;
            o.x = pack_bf16x2(f * __uint_as_float(v[half * 8 + 0]), f * __uint_as_float(v[half * 8 + 1]));
            o.y = pack_bf16x2(f * __uint_as_float(v[half * 8 + 2]), f * __uint_as_float(v[half * 8 + 3]));
            o.z = pack_bf16x2(f * __uint_as_float(v[half * 8 + 4]), f * __uint_as_float(v[half * 8 + 5]));
            o.w = pack_bf16x2(f * __uint_as_float(v[half * 8 + 6]), f * __uint_as_float(v[half * 8 + 7]));
            *reinterpret_cast<uint4*>(row + (c + half * 8) * 2) = o;
          }
        };
        int c = 0;
        for (; c + 32 <= d; c += 32) {                     // two accumulator loads in flight per wait
          uint32_t v0[16], v1[16];
          const float f0 = factor(c), f1 = factor(c + 16);   // (the sums are read before the accumulator is handed back)
          tmem_ld16(tO + c, v0);
          tmem_ld16(tO + c + 16, v1);
          tc_wait_ld();
          if (c + 32 >= d) hand_back();
          stage16(c, v0, f0);
          stage16(c + 16, v1, f1);
        }
        if (c < d) {
          uint32_t v0[16];
          const float f0 = factor(c);
          tmem_ld16(tO + c, v0);
          tc_wait_ld();
          hand_back();
          stage16(c, v0, f0);
        }
        const int ci = w.j * kCandTile + m;
        if (ci < w.nc) {                                   // my candidate's row of this segment: one contiguous store
          fence_proxy_async_smem();
          bulk_s2g(P.Hp + ((size_t)(w.c0 + ci) * P.Lp + w.seg) * d, row, d * 2);
        }
        bulk_commit();
        if (two_epilogues) o_par ^= 1;                     // (this group's accumulator again, next phase)
        else if ((int)++ob == n_obuf) { ob = 0; o_par ^= 1; }
      }
      bulk_wait<0>();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kProducerWarp) tmem_dealloc(tmem, kStaTmemCols);
  if (tid == 0 && s_abort) report_status(P.status, LASER_ERR_TIMEOUT);
}

// Self-test of the give-up path of the bounded waits: one block sets itself up like the kernels above (an mbarrier,
// tensor memory), then every warp waits, with a poll budget of `poll_limit`, for a barrier phase that nothing will ever
// complete.  The wait runs out by construction; the block then leaves the way an aborting production block does: flag
// raised, tensor memory released, LASER_ERR_TIMEOUT in the status word.
__global__ void __launch_bounds__(128) tc_wait_selftest_kernel(int* status, uint32_t poll_limit) {
  __shared__ uint64_t bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (tid == 0) {
    mbar_init(&bar, 1);
    s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&s_tmem, 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  volatile int* abortp = &s_abort;
  mbar_wait(&bar, 0, abortp, poll_limit);      // no arrival, no copy: gives up after poll_limit polls
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 32);
  if (tid == 0 && s_abort) report_status(status, LASER_ERR_TIMEOUT);
}

int sm_count() {                         // of the current device (a process may drive several)
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  return n;
}

TcParams make_params(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                     const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hp, char* ws) {
  TcParams P = {};
  P.U = p.U; P.L = p.L; P.d = p.d; P.dqk = p.dqk; P.H = p.H; P.S = p.S; P.Lp = p.Lp; P.N = p.N;
  P.dqh = p.dqh; P.dvh = p.dvh; P.maxC = p.maxC;
  P.IT = p.tg.IT; P.NT = p.tg.NT; P.n_tiles = p.tg.n_tiles; P.cand_tiles_max = p.tg.cand_tiles_max;
  // a second output accumulator: behind the first when both fit, else (at most two heads: warpgroups 2 and 3 idle) in
  // the score buffers those warpgroups would use
  if ((int)kColO + 2 * p.d <= kStaTmemCols) { P.n_obuf = 2; P.o_col1 = (int)kColO + p.d; }
  else if (p.H <= 2 && p.d <= 2 * kItMax) { P.n_obuf = 2; P.o_col1 = 2 * kItMax; }
  else { P.n_obuf = 1; P.o_col1 = (int)kColO; }
  P.NTG = P.IT <= 64 ? (128 / P.IT < P.NT ? 128 / P.IT : P.NT) : 1;
  P.NG = (P.NT + P.NTG - 1) / P.NTG;
  P.q_scale = 0.5f * p.inv_gamma;
  P.items = (const bf16*)items; P.cands = (const bf16*)cands;
  P.Wq = (const bf16*)Wq; P.Wk = (const bf16*)Wk; P.Wv = (const bf16*)Wv;
  P.lengths = lengths; P.cand_offsets = cand_offsets;
  P.item_off = p.item_offsets;
  P.Qblk = (bf16*)(ws + p.off_tq); P.Kblk = (bf16*)(ws + p.off_tk); P.Vtblk = (bf16*)(ws + p.off_tv);
  P.unit_start = (int*)(ws + p.off_twork);
  P.tile_off = P.unit_start + (p.U + 1);
  P.proj_start = P.tile_off + (p.U + 1);
  P.counters = (int*)(ws + p.off_tcount);
  P.sta_begin = reinterpret_cast<int4*>(ws + p.off_tcount + 64 * sizeof(int));
  P.proj_begin = P.sta_begin + 1024;
  P.ctile = reinterpret_cast<int4*>(ws + p.off_tctile);
  P.sta_grid = sm_count() < 1024 ? sm_count() : 1024;
  P.proj_grid = 2 * sm_count() < 1024 ? 2 * sm_count() : 1024;
  P.imgK = (bf16*)(ws + p.off_timg);
  P.imgQ = P.imgK + (size_t)p.dqk * p.d;
  P.imgV = P.imgQ + (size_t)p.dqk * p.d;
  P.status = (int*)(ws + p.off_status);
  P.Hp = (bf16*)Hp;
  return P;
}

}  // namespace

bool tensor_supported(const Plan& p) {
  if (p.dtype != LASER_BF16) return false;
  if (p.d % 16 || p.d < 16 || p.d > 128) return false;
  if (p.dqh % 16 || p.dqk > 128) return false;
  if (p.dvh % 16) return false;
  TensorGeom g;
  tensor_geometry(p, &g);
  // shared memory of the attention kernel (Q double buffer, K / V^T ring, staged output) and of the projection kernel
  const size_t sta_smem = (size_t)2 * kCandTile * p.dqk * 2 + (size_t)kKvStages * g.IT * (p.dqk + p.d) * 2 +
                          (size_t)2 * kCandTile * (p.d * 2 + 16);
  const size_t proj_smem = ((size_t)p.dqk * p.d + 3 * (size_t)kCandTile * p.d) * 2;
  if (sta_smem > 220 * 1024 || proj_smem > 220 * 1024) return false;
  if ((long long)p.U * g.n_tiles >= (1ll << 30)) return false;
  if ((long long)p.U * p.Lp * 4 >= (1ll << 30)) return false;
  return true;
}

void tensor_geometry(const Plan& p, TensorGeom* g) {
  const int it_max = 64;   // one 64-column fp32 score buffer per gate warpgroup in TMEM
  g->NT = (p.S + it_max - 1) / it_max;
  const int per = (p.S + g->NT - 1) / g->NT;
  g->IT = (per + 15) / 16 * 16;
  g->n_tiles = p.Lp * g->NT;
  const long long a = (long long)p.N / kCandTile + p.U;
  const long long b = (long long)p.U * ((p.maxC + kCandTile - 1) / kCandTile);
  g->cand_tiles_max = (int)(a < b ? a : b);
}

namespace {
// Tensor map of the padded item array as a [U * L, d] bf16 matrix for tc_proj_kernel's tiled TMA loads: boxes of 64
// columns (128 bytes, the swizzle span) by IT rows, 128-byte swizzle, zeros outside the array.  False when the driver
// entry point is missing or refuses the shape; the kernel then stages the rows with plain asynchronous copies.
bool encode_item_map(const Plan& p, int IT, const void* items, CUtensorMap* map) {
  return encode_bf16_rows_map(items, (unsigned long long)p.U * p.L, p.d, IT, map);
}
}  // namespace

// Shared memory of the attention kernel: Q double buffer, K / V^T ring, staged output rows, and for the softmax variant
// the ring of row sums.
static size_t sta_smem_bytes(const Plan& p, int IT, bool softmax) {
  return (size_t)2 * kCandTile * p.dqk * 2 + (size_t)kKvStages * IT * (p.dqk + p.d) * 2 +
         (size_t)2 * kCandTile * (p.d * 2 + 16) + (softmax ? (size_t)kSumSlots * p.H * kCandTile * sizeof(float) : 0);
}

bool tensor_softmax_supported(const Plan& p) {
  if (!tensor_supported(p)) return false;
  TensorGeom g;
  tensor_geometry(p, &g);
  return sta_smem_bytes(p, g.IT, true) <= 220 * 1024;
}

int tensor_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
               const void* Wq, const void* Wk, const void* Wv, void* Hprime, char* ws, cudaStream_t st,
               const void* Wg_images, bool softmax) {
  if (p.N == 0 || p.U == 0) return LASER_OK;
  const bool user_wants_hp = Hprime != (void*)(ws + p.off_hp);
  TcParams P = make_params(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws);
  P.Wg = (const bf16*)Wg_images;
  P.gimg = reinterpret_cast<uint4*>(ws + p.off_gimg);
  P.gnseg = reinterpret_cast<int*>(ws + p.off_gimg + gsta_nseg_offset(p));
  P.M = p.M;
  P.gorder = nullptr;
  if (P.Wg && gsta_wants_order(p)) {
    P.gorder = reinterpret_cast<int*>(ws + p.off_gimg + gsta_order_offset(p));
    P.gorder_keys = P.gorder + (p.N + 7) / 8;
    P.gcpb = gsta_candidates_per_block(p);
  }
  const int sms = sm_count();
  {
    LaunchScope ls("tc_prep", st);
    LASER_CUDA_OK(launch_chained(tc_prep_kernel, dim3(1 + 32 + (P.gorder ? 1 : 0)), dim3(1024), 0, st, P));
  }
  {
    const size_t smem = ((size_t)p.dqk * p.d + 3 * (size_t)kCandTile * p.d) * 2;   // W_k^T | W_q^T, W_v^T, two staging buffers
    LASER_CUDA_OK(cudaFuncSetAttribute(tc_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LaunchScope ls("tc_proj", st);
    alignas(64) CUtensorMap item_map;
    memset(&item_map, 0, sizeof(item_map));
    // (packed rows, and item tiles under 32 rows, i.e. copies under 4 KB, stay on plain asynchronous copies)
    const int use_tma = !P.item_off && P.IT >= 32 && encode_item_map(p, P.IT, items, &item_map) ? 1 : 0;
    LASER_CUDA_OK(launch_chained(tc_proj_kernel, dim3(P.proj_grid), dim3(kProjThreads), smem, st, P, item_map, use_tma));
  }
  if (user_wants_hp) {
    LaunchScope ls("tc_zero_empty", st);
    LASER_CUDA_OK(launch_chained(tc_zero_empty_kernel, dim3(p.Lp, p.U), dim3(256), 0, st, P));
  }
  {
    const size_t smem = sta_smem_bytes(p, P.IT, softmax);
    if (smem > 220 * 1024) return LASER_ERR_UNSUPPORTED;
    auto kernel = softmax ? tc_sta_kernel<true> : tc_sta_kernel<false>;
    LASER_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    LaunchScope ls(softmax ? "sta_tc_softmax" : "sta_tc", st);
    LASER_CUDA_OK(launch_chained(kernel, dim3(P.sta_grid), dim3(kStaThreads), smem, st, P));
  }
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

int tensor_wait_selftest(char* ws, int poll_limit, cudaStream_t st) {
  LaunchScope ls("tc_wait_selftest", st);
  tc_wait_selftest_kernel<<<1, 128, 0, st>>>(reinterpret_cast<int*>(ws), (uint32_t)poll_limit);
  LASER_CUDA_OK(cudaGetLastError());
  return LASER_OK;
}

int tensor_gsta(const Plan& p, const void* Hprime, const int32_t* lengths, const int32_t* cand_offsets,
                const void* cands, const void* Wg, void* z, char* ws, cudaStream_t st, bool images_ready) {
  if (gsta_mma_supported(p)) return gsta_mma(p, Hprime, lengths, cand_offsets, cands, Wg, z, ws, st, images_ready);
  return simt_gsta(p, Hprime, lengths, cand_offsets, cands, Wg, z, ws, st);
}

}  // namespace laser
