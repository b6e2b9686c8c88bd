// extern "C" entry points: argument validation, path selection, workspace carve-up, dispatch.
#include <math.h>
#include <string.h>

#include <algorithm>

#include "laser_common.cuh"

namespace laser {

constexpr int kMaxProfiled = 256;          // (a backward call launches about a hundred kernels)
static thread_local int g_launches = 0;
static thread_local bool g_profile = false;
static thread_local int g_prof_n = 0;
static thread_local const char* g_prof_name[kMaxProfiled];
static thread_local cudaEvent_t g_prof_ev[2 * kMaxProfiled];
static thread_local bool g_prof_ev_made = false;

void reset_launch_count() { g_launches = 0; g_prof_n = 0; }

LaunchScope::LaunchScope(const char* name, cudaStream_t st) : st_(st), slot_(-1) {
  ++g_launches;
  if (!g_profile || g_prof_n >= kMaxProfiled) return;
  if (!g_prof_ev_made) {
    for (int i = 0; i < 2 * kMaxProfiled; ++i)
      if (cudaEventCreate(&g_prof_ev[i]) != cudaSuccess) return;
    g_prof_ev_made = true;
  }
  slot_ = g_prof_n++;
  g_prof_name[slot_] = name;
  cudaEventRecord(g_prof_ev[2 * slot_], st_);
}
LaunchScope::~LaunchScope() {
  if (slot_ >= 0) cudaEventRecord(g_prof_ev[2 * slot_ + 1], st_);
}

static int resolve_path(const Plan& p, int requested) {
  if (requested == LASER_PATH_AUTO) {
    if (p.dtype == LASER_F32) return LASER_PATH_SIMT;
    if (p.maxC <= 1 && stream_supported(p)) return LASER_PATH_STREAM;
    if (tensor_supported(p)) return LASER_PATH_TENSOR;
    return LASER_PATH_SIMT;
  }
  if (requested == LASER_PATH_SIMT) return LASER_PATH_SIMT;
  if (requested == LASER_PATH_TENSOR) return tensor_supported(p) ? (int)LASER_PATH_TENSOR : (int)LASER_ERR_UNSUPPORTED;
  if (requested == LASER_PATH_STREAM) return (p.maxC <= 1 && stream_supported(p)) ? (int)LASER_PATH_STREAM : (int)LASER_ERR_UNSUPPORTED;
  return LASER_ERR_INVALID_ARG;
}

int make_plan(const laser_config* c, Plan* p) {
  if (!c || !p) return LASER_ERR_INVALID_ARG;
  memset(p, 0, sizeof(*p));
  if (c->num_users < 0 || c->max_len < 1 || c->d_model < 1 || c->d_qk < 1 || c->num_heads < 1 || c->seg_size < 1 ||
      c->num_gsta_layers < 0 || c->total_cands < 0 || c->max_cands_per_user < 0)
    return LASER_ERR_INVALID_ARG;
  if (c->dtype != LASER_F32 && c->dtype != LASER_BF16) return LASER_ERR_INVALID_ARG;
  if (c->d_model % c->num_heads || c->d_qk % c->num_heads) return LASER_ERR_INVALID_ARG;
  if (c->max_cands_per_user > c->total_cands) return LASER_ERR_INVALID_ARG;
  if (c->total_cands > 0 && (c->max_cands_per_user == 0 || c->num_users == 0)) return LASER_ERR_INVALID_ARG;
  p->U = c->num_users; p->L = c->max_len; p->d = c->d_model; p->dqk = c->d_qk; p->H = c->num_heads;
  p->S = c->seg_size; p->M = c->num_gsta_layers; p->dtype = c->dtype; p->N = c->total_cands;
  p->maxC = c->max_cands_per_user;
  p->Lp = (p->L + p->S - 1) / p->S;
  p->dqh = p->dqk / p->H; p->dvh = p->d / p->H;
  const float gamma = c->sta_gamma > 0.f ? c->sta_gamma : sqrtf((float)p->dqh);
  const float tau = c->gsta_scale > 0.f ? c->gsta_scale : sqrtf((float)p->dvh);
  p->inv_gamma = 1.f / gamma; p->inv_tau = 1.f / tau;
  p->esize = p->dtype == LASER_F32 ? 4 : 2;
  if ((size_t)p->N * p->Lp * p->d >= ((size_t)1 << 40)) return LASER_ERR_UNSUPPORTED;

  const int path = resolve_path(*p, c->path);
  if (path < 0) return path;
  p->path = path;

  // carve-up: every region starts 256-byte aligned and is followed by kGuardBytes that nothing may touch
  size_t off = 0;
  auto carve = [&](size_t bytes) {
    const size_t at = off;
    if (p->n_regions < kMaxRegions) {
      p->reg_off[p->n_regions] = at;
      p->reg_size[p->n_regions] = bytes;
      ++p->n_regions;
    }
    off = align_up(off + bytes) + kGuardBytes;
    return at;
  };
  p->off_status = carve(kStatusWords * sizeof(int));
  p->off_hp = carve((size_t)p->N * p->Lp * p->d * p->esize);
  if (path == LASER_PATH_SIMT) {
    p->off_q = carve((size_t)p->N * p->dqk * sizeof(float));
    p->off_k = carve((size_t)p->U * p->L * p->dqk * sizeof(float));
    p->off_v = carve((size_t)p->U * p->L * p->d * sizeof(float));
  } else if (path == LASER_PATH_TENSOR) {
    tensor_geometry(*p, &p->tg);
    const TensorGeom& g = p->tg;
    const size_t q_tiles = (size_t)g.cand_tiles_max;
    p->off_tq = carve(q_tiles * 128 * p->dqk * 2);
    p->off_tk = carve((size_t)p->U * g.n_tiles * g.IT * p->dqk * 2);
    p->off_tv = carve((size_t)p->U * g.n_tiles * g.IT * p->d * 2);
    p->off_twork = carve(((size_t)p->U + 1) * 3 * sizeof(int));
    p->off_tcount = carve(64 * sizeof(int) + 2 * 1024 * 4 * sizeof(int));   // counters + per-block start tables
    p->off_tctile = carve((size_t)g.cand_tiles_max * 4 * sizeof(int));       // (user, tile, first candidate, candidates) per candidate tile
    p->off_timg = carve(((size_t)2 * p->dqk * p->d + (size_t)128 * p->d) * 2);
    if (gsta_mma_supported(*p)) p->off_gimg = carve(gsta_mma_image_bytes(*p));
  } else if (path == LASER_PATH_STREAM) {
    p->off_su = carve(stream_scratch_bytes(*p));
    p->off_gimg = carve(gsta_mma_image_bytes(*p));
  }
  p->total = off;
  return LASER_OK;
}

static bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

static int check_ptrs(std::initializer_list<const void*> ptrs) {
  for (const void* q : ptrs) {
    if (!q) return LASER_ERR_INVALID_ARG;
    if (!aligned16(q)) return LASER_ERR_INVALID_ARG;
  }
  return LASER_OK;
}

static int check_ws(const Plan& p, const void* ws, size_t bytes) {
  if (!ws) return LASER_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) return LASER_ERR_INVALID_ARG;
  if (bytes < p.total) return LASER_ERR_WORKSPACE;
  return LASER_OK;
}

static int clear_status(const Plan& p, char* ws, cudaStream_t st) {
  LASER_CUDA_OK(cudaMemsetAsync(ws + p.off_status, 0, kStatusWords * sizeof(int), st));
  return LASER_OK;
}

// Wg_images: GSTA weights whose images the STA set-up may build on the side (null when GSTA does not follow).
static int run_sta(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                   const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hp, char* ws,
                   cudaStream_t st, const void* Wg_images) {
  switch (p.path) {
    case LASER_PATH_SIMT: return simt_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hp, ws, st);
    case LASER_PATH_TENSOR: return tensor_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hp, ws, st, Wg_images);
    case LASER_PATH_STREAM: return stream_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hp, ws, st, Wg_images);
    default: return LASER_ERR_UNSUPPORTED;
  }
}

static int run_gsta(const Plan& p, const void* Hp, const int32_t* lengths, const int32_t* cand_offsets,
                    const void* cands, const void* Wg, void* z, char* ws, cudaStream_t st, bool images_ready) {
  switch (p.path) {
    case LASER_PATH_SIMT: return simt_gsta(p, Hp, lengths, cand_offsets, cands, Wg, z, ws, st);
    case LASER_PATH_TENSOR: return tensor_gsta(p, Hp, lengths, cand_offsets, cands, Wg, z, ws, st, images_ready);
    case LASER_PATH_STREAM: return gsta_mma(p, Hp, lengths, cand_offsets, cands, Wg, z, ws, st, images_ready);
    default: return LASER_ERR_UNSUPPORTED;
  }
}

static int forward_impl(const Plan& p, const void* items, const int32_t* lengths, const void* cands,
                        const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, const void* Wg,
                        void* Hprime, void* z, char* ws, cudaStream_t st) {
  int rc = clear_status(p, ws, st);
  if (rc != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  void* Hp = Hprime ? Hprime : (void*)(ws + p.off_hp);
  const bool side_images = p.M > 0 && p.path != LASER_PATH_SIMT && gsta_mma_supported(p);
  rc = run_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hp, ws, st, side_images ? Wg : nullptr);
  if (rc != LASER_OK) return rc;
  return run_gsta(p, Hp, lengths, cand_offsets, cands, Wg, z, ws, st, side_images);
}

}  // namespace laser

using namespace laser;

extern "C" {

size_t laser_workspace_bytes(const laser_config* cfg) {
  Plan p;
  if (make_plan(cfg, &p) != LASER_OK) return 0;
  return p.total;
}

int laser_sta_forward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                      const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime,
                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ws(p, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({items, cands, Wq, Wk, Wv, Hprime})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  return run_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws, st, nullptr);
}

int laser_gsta_forward(const laser_config* cfg, const void* Hprime, const int32_t* lengths,
                       const int32_t* cand_offsets, const void* cands, const void* Wgsta, void* z, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ws(p, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({Hprime, cands, z})) != LASER_OK) return rc;
  if (p.N > 0 && p.M > 0 && (rc = check_ptrs({Wgsta})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  return run_gsta(p, Hprime, lengths, cand_offsets, cands, Wgsta, z, ws, st, false);
}

int laser_forward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                  const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, const void* Wgsta,
                  void* Hprime, void* z, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ws(p, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({items, cands, Wq, Wk, Wv, z})) != LASER_OK) return rc;
  if (p.N > 0 && p.M > 0 && (rc = check_ptrs({Wgsta})) != LASER_OK) return rc;
  if (Hprime && !aligned16(Hprime)) return LASER_ERR_INVALID_ARG;
  return forward_impl(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, Hprime, z,
                      static_cast<char*>(workspace), static_cast<cudaStream_t>(cuda_stream));
}

int laser_forward_packed(const laser_config* cfg, const void* items_packed, const int32_t* item_offsets,
                         const int32_t* lengths, const void* cands, const int32_t* cand_offsets, const void* Wq,
                         const void* Wk, const void* Wv, const void* Wgsta, void* Hprime, void* z, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ws(p, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets || !item_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({items_packed, cands, Wq, Wk, Wv, z})) != LASER_OK) return rc;
  if (p.N > 0 && p.M > 0 && (rc = check_ptrs({Wgsta})) != LASER_OK) return rc;
  if (Hprime && !aligned16(Hprime)) return LASER_ERR_INVALID_ARG;
  p.item_offsets = item_offsets;
  return forward_impl(p, items_packed, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, Hprime, z,
                      static_cast<char*>(workspace), static_cast<cudaStream_t>(cuda_stream));
}

int laser_fusion_forward(const laser_config* cfg, const void* Hprime, const void* z, const int32_t* lengths,
                         const int32_t* cand_offsets, int32_t num_recent, void* fused, void* workspace,
                         size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if (num_recent < 0) return LASER_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))) return LASER_ERR_INVALID_ARG;
  if (workspace_bytes < kAlign) return LASER_ERR_WORKSPACE;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({Hprime, z, fused})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  return fusion_forward(p, Hprime, z, lengths, cand_offsets, num_recent, fused, ws, st);
}

// The variant has a tensor-core version (bf16 shapes the tensor path supports) and the FP32-ALU one; there is no
// one-candidate streaming version, so LASER_PATH_AUTO means "tensor cores if supported" and LASER_PATH_STREAM falls back
// to the FP32 ALUs.
static int softmax_plan(const laser_config* cfg, Plan* p) {
  if (!cfg) return LASER_ERR_INVALID_ARG;
  laser_config c = *cfg;
  if (c.path == LASER_PATH_AUTO || c.path == LASER_PATH_TENSOR) {
    const int requested = c.path;
    c.path = LASER_PATH_TENSOR;
    if (make_plan(&c, p) == LASER_OK && tensor_softmax_supported(*p)) return LASER_OK;
    if (requested == LASER_PATH_TENSOR) return LASER_ERR_UNSUPPORTED;
  }
  c.path = LASER_PATH_SIMT;
  return make_plan(&c, p);
}

size_t laser_sta_softmax_workspace_bytes(const laser_config* cfg) {
  Plan p;
  if (softmax_plan(cfg, &p) != LASER_OK) return 0;
  return p.total;
}

int laser_sta_softmax_forward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                              const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime,
                              void* workspace, size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = softmax_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ws(p, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({items, cands, Wq, Wk, Wv, Hprime})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  if (p.path == LASER_PATH_TENSOR)
    return tensor_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws, st, nullptr, true);
  return simt_sta_softmax(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hprime, ws, st);
}

// The backward pass works on the fp32 intermediates and the workspace layout of the FP32-ALU path, on the padded item
// layout; *tensor says whether its contractions run on the tensor cores (bf16 batches of supported head widths, unless
// cfg->path asks for the FP32 ALUs; LASER_PATH_TENSOR on anything else is LASER_ERR_UNSUPPORTED).
static int backward_plan(const laser_config* cfg, Plan* p, bool* tensor) {
  if (!cfg) return LASER_ERR_INVALID_ARG;
  laser_config c = *cfg;
  c.path = LASER_PATH_SIMT;
  const int rc = make_plan(&c, p);
  if (rc != LASER_OK) return rc;
  *tensor = cfg->path != LASER_PATH_SIMT && backward_tensor_supported(*p);
  if (cfg->path == LASER_PATH_TENSOR && !*tensor) return LASER_ERR_UNSUPPORTED;
  return LASER_OK;
}

size_t laser_backward_workspace_bytes(const laser_config* cfg) {
  Plan p;
  bool tensor;
  if (backward_plan(cfg, &p, &tensor) != LASER_OK) return 0;
  return p.total + backward_scratch_bytes(p);
}

int laser_backward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                   const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, const void* Wgsta,
                   const float* dz, float* d_items, float* d_cands, float* dWq, float* dWk, float* dWv, float* dWgsta,
                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  bool tensor;
  int rc = backward_plan(cfg, &p, &tensor);
  if (rc != LASER_OK) return rc;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))) return LASER_ERR_INVALID_ARG;
  if (workspace_bytes < p.total + backward_scratch_bytes(p)) return LASER_ERR_WORKSPACE;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if ((rc = check_ptrs({Wq, Wk, Wv, dWq, dWk, dWv})) != LASER_OK) return rc;
  if (p.U > 0 && (rc = check_ptrs({items, d_items})) != LASER_OK) return rc;
  if (p.N > 0 && (rc = check_ptrs({cands, dz, d_cands})) != LASER_OK) return rc;
  if (p.M > 0 && (rc = check_ptrs({Wgsta, dWgsta})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  return backward(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wgsta, dz, d_items, d_cands, dWq, dWk, dWv, dWgsta,
                  ws, st, tensor);
}

size_t laser_ffn_workspace_bytes(const laser_config* cfg, int32_t d_hidden) {
  Plan p;
  if (make_plan(cfg, &p) != LASER_OK || d_hidden < 1) return 0;
  return p.total + ffn_scratch_bytes(p, d_hidden);
}

static int check_ffn(const Plan& p, const laser_ffn_params* f, const void* workspace, size_t workspace_bytes) {
  if (!f || f->d_hidden < 1) return LASER_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))) return LASER_ERR_INVALID_ARG;
  if (workspace_bytes < p.total + ffn_scratch_bytes(p, f->d_hidden)) return LASER_ERR_WORKSPACE;
  if (p.N > 0) {
    const int rc = check_ptrs({f->W1, f->b1, f->W2, f->b2, f->ln_gain, f->ln_shift});
    if (rc != LASER_OK) return rc;
    if (!ffn_supported(p, f->d_hidden)) return LASER_ERR_UNSUPPORTED;
  }
  return LASER_OK;
}

int laser_ffn_forward(const laser_config* cfg, const laser_ffn_params* ffn, void* Hprime, const int32_t* lengths,
                      const int32_t* cand_offsets, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ffn(p, ffn, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({Hprime})) != LASER_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  return ffn_forward(p, ffn, Hprime, lengths, cand_offsets, ws, ws + p.total, st);
}

int laser_forward_ffn(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                      const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, const void* Wgsta,
                      const laser_ffn_params* ffn, void* Hprime, void* z, void* workspace, size_t workspace_bytes,
                      void* cuda_stream) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if ((rc = check_ffn(p, ffn, workspace, workspace_bytes)) != LASER_OK) return rc;
  if (!lengths || !cand_offsets) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (rc = check_ptrs({items, cands, Wq, Wk, Wv, z})) != LASER_OK) return rc;
  if (p.N > 0 && p.M > 0 && (rc = check_ptrs({Wgsta})) != LASER_OK) return rc;
  if (Hprime && !aligned16(Hprime)) return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  if ((rc = clear_status(p, ws, st)) != LASER_OK) return rc;
  if (p.N == 0) return LASER_OK;
  void* Hp = Hprime ? Hprime : (void*)(ws + p.off_hp);
  const bool side_images = p.M > 0 && p.path != LASER_PATH_SIMT && gsta_mma_supported(p);
  rc = run_sta(p, items, lengths, cands, cand_offsets, Wq, Wk, Wv, Hp, ws, st, side_images ? Wgsta : nullptr);
  if (rc != LASER_OK) return rc;
  rc = ffn_forward(p, ffn, Hp, lengths, cand_offsets, ws, ws + p.total, st);
  if (rc != LASER_OK) return rc;
  return run_gsta(p, Hp, lengths, cand_offsets, cands, Wgsta, z, ws, st, side_images);
}

namespace {
struct HostStage {
  size_t items, lengths, cands, offs, item_offs, wq, wk, wv, wg, z, total;
  size_t b_items, b_lengths, b_cands, b_offs, b_wq, b_wk, b_wv, b_wg, b_z;
};
HostStage host_stage(const Plan& p) {
  HostStage s;
  s.b_items = (size_t)p.U * p.L * p.d * p.esize;
  s.b_lengths = (size_t)p.U * sizeof(int32_t);
  s.b_cands = (size_t)p.N * p.d * p.esize;
  s.b_offs = (size_t)(p.U + 1) * sizeof(int32_t);
  s.b_wq = s.b_wk = (size_t)p.d * p.dqk * p.esize;
  s.b_wv = (size_t)p.d * p.d * p.esize;
  s.b_wg = (size_t)p.M * 3 * p.d * p.d * p.esize;
  s.b_z = (size_t)p.N * p.d * p.esize;
  size_t off = p.total;
  s.items = off; off = align_up(off + s.b_items);
  s.lengths = off; off = align_up(off + s.b_lengths);
  s.cands = off; off = align_up(off + s.b_cands);
  s.offs = off; off = align_up(off + s.b_offs);
  s.item_offs = off; off = align_up(off + s.b_offs);
  s.wq = off; off = align_up(off + s.b_wq);
  s.wk = off; off = align_up(off + s.b_wk);
  s.wv = off; off = align_up(off + s.b_wv);
  s.wg = off; off = align_up(off + s.b_wg);
  s.z = off; off = align_up(off + s.b_z);
  s.total = off;
  return s;
}

// How the item rows travel to the device.  The lengths are known on the host, so rows past a user's valid prefix need
// not cross the bus; the valid rows land in a gap-free device array, which the kernels then read through per-user row
// offsets exactly as for laser_forward_packed.  Three routes:
//   kGather  items_h is pinned (or registered) host memory with a device alias: one kernel reads the valid rows straight
//            from it.  Taken when it saves at least kGatherWorth bytes.
//   kRuns    one copy per run of users whose valid rows are contiguous in the padded host array (a run ends after the
//            first user shorter than L).  Every copy has a fixed cost on the host (several microseconds, i.e. some
//            hundred KB of bus time), so this is taken only when it saves at least kCopyWorth bytes per copy.
//   kPadded  the padded array travels in one piece.
enum HostRouteKind { kPadded, kRuns, kGather };
struct HostItemRoute {
  HostRouteKind kind;
  size_t bytes;                          // item bytes that travel
  const void* alias;                     // kGather: device alias of items_h
};
constexpr size_t kCopyWorth = 384 * 1024, kGatherWorth = 256 * 1024;
constexpr int kGatherThreads = 256;

HostItemRoute host_item_route(const Plan& p, const void* items_h, const int32_t* lengths_h) {
  HostItemRoute r;
  const size_t row = (size_t)p.d * p.esize, padded = (size_t)p.U * p.L * row;
  r.kind = kPadded;
  r.bytes = padded;
  r.alias = nullptr;
  if (p.U == 0 || p.N == 0) return r;
  long long rows = 0;
  size_t copies = 0;
  bool contiguous = false;               // the previous user's rows end where this user's begin
  for (int u = 0; u < p.U; ++u) {
    const int len = std::min(std::max(lengths_h[u], 0), p.L);   // invalid lengths are reported by the device
    if (len > 0 && !contiguous) ++copies;
    contiguous = len == p.L;
    rows += len;
  }
  if (rows > 0x7fffffffLL) return r;
  const size_t need = (size_t)rows * row;
  if (items_h && row % 16 == 0 && (reinterpret_cast<uintptr_t>(items_h) & 15) == 0 && need + kGatherWorth < padded) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, items_h) == cudaSuccess) {
      if (attr.type == cudaMemoryTypeHost && attr.devicePointer) {
        r.kind = kGather;
        r.alias = attr.devicePointer;
      }
    } else {
      cudaGetLastError();                // (no device, or a runtime that rejects pageable pointers: not an error here)
    }
  }
  if (r.kind == kPadded && need + copies * kCopyWorth < padded) r.kind = kRuns;
  if (r.kind != kPadded) r.bytes = need;
  return r;
}

// First row of every user in the gap-free array: exclusive prefix sums of the lengths, clamped to [0, L] as the host
// clamps them when it sizes its copies.  One block; computed on the device so that the host never has to hand a
// pageable table to an asynchronous copy (which would make it wait for the stream on every call).
__global__ void __launch_bounds__(1024) host_row_offsets_kernel(const int32_t* lengths, int U, int L, int32_t* row_off) {
  chain_wait();
  __shared__ int part[1024];
  const int tid = threadIdx.x, per = (U + 1023) / 1024;
  const int u0 = min(tid * per, U), u1 = min(u0 + per, U);
  int sum = 0;
  for (int u = u0; u < u1; ++u) sum += min(max(lengths[u], 0), L);
  part[tid] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {
    const int v = tid >= off ? part[tid - off] : 0;
    __syncthreads();
    part[tid] += v;
    __syncthreads();
  }
  int run = part[tid] - sum;
  for (int u = u0; u < u1; ++u) {
    row_off[u] = run;
    run += min(max(lengths[u], 0), L);
  }
  if (tid == 1023) row_off[U] = part[1023];
}

// kGather: block (u, j) copies rows j * rows_per_block ... of user u's valid prefix, 16 bytes per thread and step, from
// the padded host array (through its device alias) to the user's place in the gap-free device array.
__global__ void __launch_bounds__(kGatherThreads) host_gather_kernel(const uint4* __restrict__ src,
                                                                     uint4* __restrict__ dst, const int32_t* lengths,
                                                                     const int32_t* row_off, int L, int vec,
                                                                     int rows_per_block) {
  chain_wait();                          // (the next kernel starts once this grid has drained: nothing to overlap with)
  const int u = blockIdx.x;
  const int len = min(max(lengths[u], 0), L);              // as the host clamped it when it built row_off
  const int r0 = blockIdx.y * rows_per_block;
  if (r0 >= len) return;
  const int n = min(rows_per_block, len - r0) * vec;
  const uint4* s = src + ((size_t)u * L + r0) * vec;
  uint4* d = dst + ((size_t)row_off[u] + r0) * vec;
#pragma unroll 4
  for (int i = threadIdx.x; i < n; i += kGatherThreads) d[i] = s[i];
}
}  // namespace

int laser_host_transfer_bytes(const laser_config* cfg, const void* items_h, const int32_t* lengths_h,
                              size_t* h2d_bytes, size_t* d2h_bytes) {
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if (!lengths_h || !h2d_bytes || !d2h_bytes) return LASER_ERR_INVALID_ARG;
  const HostStage s = host_stage(p);
  *h2d_bytes = s.b_lengths + s.b_offs;
  *d2h_bytes = 0;
  if (p.N > 0) {
    const HostItemRoute r = host_item_route(p, items_h, lengths_h);
    *h2d_bytes += r.bytes + s.b_cands + s.b_wq + s.b_wk + s.b_wv + s.b_wg;
    *d2h_bytes = s.b_z;
  }
  return LASER_OK;
}

size_t laser_host_workspace_bytes(const laser_config* cfg) {
  Plan p;
  if (make_plan(cfg, &p) != LASER_OK) return 0;
  return host_stage(p).total;
}

int laser_forward_host(const laser_config* cfg, const void* items_h, const int32_t* lengths_h, const void* cands_h,
                       const int32_t* cand_offsets_h, const void* Wq_h, const void* Wk_h, const void* Wv_h,
                       const void* Wgsta_h, void* z_h, void* workspace, size_t workspace_bytes, void* cuda_stream,
                       int blocking) {
  reset_launch_count();
  Plan p;
  int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))) return LASER_ERR_INVALID_ARG;
  const HostStage s = host_stage(p);
  if (workspace_bytes < s.total) return LASER_ERR_WORKSPACE;
  if (!lengths_h || !cand_offsets_h) return LASER_ERR_INVALID_ARG;
  if (p.N > 0 && (!items_h || !cands_h || !Wq_h || !Wk_h || !Wv_h || !z_h || (p.M > 0 && !Wgsta_h)))
    return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  auto h2d = [&](size_t off, const void* src, size_t bytes) -> cudaError_t {
    if (!bytes) return cudaSuccess;
    return cudaMemcpyAsync(ws + off, src, bytes, cudaMemcpyHostToDevice, st);
  };
  LASER_CUDA_OK(h2d(s.lengths, lengths_h, s.b_lengths));
  LASER_CUDA_OK(h2d(s.offs, cand_offsets_h, s.b_offs));
  if (p.N > 0) {
    const HostItemRoute route = host_item_route(p, items_h, lengths_h);
    if (route.kind == kPadded) LASER_CUDA_OK(h2d(s.items, items_h, s.b_items));
    else {
      {
        LaunchScope ls("host_row_offsets", st);
        LASER_CUDA_OK(launch_chained(host_row_offsets_kernel, dim3(1), dim3(1024), 0, st,
                                     reinterpret_cast<const int32_t*>(ws + s.lengths), p.U, p.L,
                                     reinterpret_cast<int32_t*>(ws + s.item_offs)));
      }
      const size_t row = (size_t)p.d * p.esize;
      if (route.kind == kGather) {
        const int per = std::max(64, (p.L + 65534) / 65535);            // rows per block; grid.y <= 65535
        LaunchScope ls("host_gather", st);
        LASER_CUDA_OK(launch_chained(host_gather_kernel, dim3(p.U, (p.L + per - 1) / per), dim3(kGatherThreads), 0, st,
                                     static_cast<const uint4*>(route.alias), reinterpret_cast<uint4*>(ws + s.items),
                                     reinterpret_cast<const int32_t*>(ws + s.lengths),
                                     reinterpret_cast<const int32_t*>(ws + s.item_offs), p.L, (int)(row / 16), per));
      } else {
        const char* src = static_cast<const char*>(items_h);
        size_t first_row = 0;              // of the run in the gap-free array
        for (int u = 0; u < p.U;) {        // one copy per run of users whose valid rows are contiguous on the host
          size_t rows = 0;
          int e = u;
          for (;; ++e) {
            const int len = std::min(std::max(lengths_h[e], 0), p.L);
            rows += (size_t)len;
            if (len != p.L || e + 1 == p.U) break;
          }
          LASER_CUDA_OK(h2d(s.items + first_row * row, src + (size_t)u * p.L * row, rows * row));
          first_row += rows;
          u = e + 1;
        }
      }
      p.item_offsets = reinterpret_cast<const int32_t*>(ws + s.item_offs);
    }
    LASER_CUDA_OK(h2d(s.cands, cands_h, s.b_cands));
    LASER_CUDA_OK(h2d(s.wq, Wq_h, s.b_wq));
    LASER_CUDA_OK(h2d(s.wk, Wk_h, s.b_wk));
    LASER_CUDA_OK(h2d(s.wv, Wv_h, s.b_wv));
    LASER_CUDA_OK(h2d(s.wg, Wgsta_h, s.b_wg));
  }
  rc = forward_impl(p, ws + s.items, reinterpret_cast<const int32_t*>(ws + s.lengths), ws + s.cands,
                    reinterpret_cast<const int32_t*>(ws + s.offs), ws + s.wq, ws + s.wk, ws + s.wv, ws + s.wg, nullptr,
                    ws + s.z, ws, st);
  if (rc != LASER_OK) return rc;
  if (s.b_z) LASER_CUDA_OK(cudaMemcpyAsync(z_h, ws + s.z, s.b_z, cudaMemcpyDeviceToHost, st));
  if (blocking) return laser_check_status(workspace, cuda_stream);
  return LASER_OK;
}

int laser_check_status(const void* workspace, void* cuda_stream) {
  if (!workspace) return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LASER_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LASER_ERR_CUDA;
  return word;
}

int laser_last_launch_count(void) { return g_launches; }

int laser_profile_enable(int on) {
  g_profile = on != 0;
  return LASER_OK;
}

int laser_profile_read(int max_kernels, float* ms_out, const char** names_out) {
  if (max_kernels < 0 || (max_kernels > 0 && (!ms_out || !names_out))) return LASER_ERR_INVALID_ARG;
  const int n = g_prof_n < max_kernels ? g_prof_n : max_kernels;
  for (int i = 0; i < n; ++i) {
    if (cudaEventSynchronize(g_prof_ev[2 * i + 1]) != cudaSuccess) return LASER_ERR_CUDA;
    if (cudaEventElapsedTime(&ms_out[i], g_prof_ev[2 * i], g_prof_ev[2 * i + 1]) != cudaSuccess) return LASER_ERR_CUDA;
    names_out[i] = g_prof_name[i];
  }
  return n;
}

int laser_workspace_regions(const laser_config* cfg, int max_regions, size_t* offsets, size_t* sizes) {
  Plan p;
  const int rc = make_plan(cfg, &p);
  if (rc != LASER_OK) return rc;
  if (max_regions < 0 || (max_regions > 0 && (!offsets || !sizes))) return LASER_ERR_INVALID_ARG;
  for (int i = 0; i < p.n_regions && i < max_regions; ++i) {
    offsets[i] = p.reg_off[i];
    sizes[i] = p.reg_size[i];
  }
  return p.n_regions;
}

int laser_selftest_wait_timeout(void* workspace, size_t workspace_bytes, int32_t poll_limit, void* cuda_stream) {
  reset_launch_count();
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1))) return LASER_ERR_INVALID_ARG;
  if (workspace_bytes < kStatusWords * sizeof(int)) return LASER_ERR_WORKSPACE;
  if (poll_limit < 1 || poll_limit > 4096) return LASER_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  LASER_CUDA_OK(cudaMemsetAsync(workspace, 0, kStatusWords * sizeof(int), st));
  return tensor_wait_selftest(static_cast<char*>(workspace), poll_limit, st);
}

const char* laser_status_string(int status) {
  switch (status) {
    case LASER_OK: return "ok";
    case LASER_ERR_INVALID_ARG: return "invalid argument";
    case LASER_ERR_UNSUPPORTED: return "shape or path not supported";
    case LASER_ERR_WORKSPACE: return "workspace too small";
    case LASER_ERR_CUDA: return "CUDA runtime error";
    case LASER_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case LASER_ERR_BAD_INPUT: return "a length or candidate offset is out of range";
    default: return "unknown status";
  }
}

}  // extern "C"
