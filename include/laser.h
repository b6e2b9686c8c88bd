/*
 * laser.h -- C ABI of the B200 (sm_100a) forward pass of LASER's Segmented Target Attention (STA)
 * followed by Global Stacked Target Attention (GSTA).
 *
 * What is computed (paper sections "Fine-grained Target-aware Compression", "Global Target Attention over
 * Compressed Sequence" and "Global Attention with Segmented Aggregation"):
 *
 *   STA   For user u with items x_0..x_{len-1} in R^d and each of its candidates t in R^d:
 *           q = t W_q,  k_n = x_n W_k,  v_n = x_n W_v                                   (Eq. 4 / Eq. 8-9)
 *           alpha_{n,h} = Sigmoid(q_h . k_{n,h} / gamma)          one gate per item and head   (Eq. 5 / Eq. 10)
 *           s_i[head h] = sum over the items n of segment i (n < len) of alpha_{n,h} v_{n,h}   (Eq. 11-12)
 *         Segment i holds items [i*S, (i+1)*S) (Eq. 3); L' = ceil(L / S); H' = [s_0 .. s_{L'-1}] in R^{L' x d}.
 *   GSTA  t_0 = t;  for l = 1..M, per head: a = softmax_j((t_{l-1} W_q^l)_h . (s_j W_k^l)_h / tau) over the
 *         non-empty segments j, o_l[head h] = sum_j a_j (s_j W_v^l)_h,  t_l = t_{l-1} + o_l;  z = t_M.   (Eq. 7)
 *
 * Conventions where the paper gives none: heads split the columns of W_q, W_k ([d, d_qk]) and of W_v and
 * the GSTA weights ([d, d]) into H contiguous slices, head outputs are concatenated, there is no output
 * projection and no bias; an item at or beyond a user's length contributes exactly nothing (whatever the
 * padded rows contain, as long as it is finite); a segment without valid items yields a zero row of H' and
 * takes no part in the GSTA softmax; a user of length 0 yields H' = 0 and z = t.  laser_forward runs the two
 * stages back to back; laser_forward_ffn puts the FFN / LayerNorm of Eq. 6 between them.
 *
 * General rules for every entry point
 *   - Unless stated otherwise every pointer is a DEVICE pointer to memory owned by the caller; the library
 *     never allocates, frees or keeps a pointer after the call returns, and never synchronises (except
 *     laser_check_status and laser_forward_host's final wait when `blocking` is non-zero).
 *   - All arrays are dense row-major with the innermost index contiguous; base pointers must be 16-byte
 *     aligned.  Floating-point arrays (items, candidates, weights, H', z) all have the config's dtype.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t cast to void*; NULL = the legacy default stream).
 *   - Return value: LASER_OK, or a negative laser_status for an error the host can see (bad argument,
 *     unsupported shape, workspace too small, a CUDA launch error).  Nothing is launched after such an
 *     error.  Errors that only the device can see (a length outside [0, L], candidate offsets that are not
 *     non-decreasing within [0, N], a bounded wait that ran out) are written to a status word at the
 *     start of the workspace, make the affected kernels skip the offending work, and are returned by
 *     laser_check_status.
 *   - Weights are right-multiplied: y = x W, W stored [in, out].
 *   - There is no CPU fallback: a shape outside the supported envelope returns LASER_ERR_UNSUPPORTED.
 *   - Calls that use the same workspace must not overlap on the GPU; distinct workspaces may run
 *     concurrently on distinct streams.
 */
#ifndef LASER_H_
#define LASER_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LASER_API __attribute__((visibility("default")))
#else
#define LASER_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { LASER_F32 = 0, LASER_BF16 = 1 } laser_dtype;

typedef enum {
  LASER_OK = 0,
  LASER_ERR_INVALID_ARG = -1,
  LASER_ERR_UNSUPPORTED = -2,
  LASER_ERR_WORKSPACE = -3,
  LASER_ERR_CUDA = -4,
  LASER_ERR_TIMEOUT = -5,   /* a bounded device-side wait gave up (device-reported) */
  LASER_ERR_BAD_INPUT = -6  /* a length or candidate offset out of range (device-reported) */
} laser_status;

/* Which kernels carry the path.  AUTO picks: F32 -> SIMT; BF16 -> STREAM when no user has more than one
 * candidate, otherwise TENSOR. */
typedef enum {
  LASER_PATH_AUTO = 0,
  LASER_PATH_SIMT = 1,    /* FP32-ALU kernels, fp32 arithmetic for either dtype (the only F32 path)       */
  LASER_PATH_TENSOR = 2,  /* BF16: tcgen05 / TMEM / TMA kernels, bf16 operands, fp32 accumulation         */
  LASER_PATH_STREAM = 3   /* BF16, at most one candidate per user: one HBM-streaming pass over the items  */
} laser_path;

typedef struct laser_config {
  int32_t num_users;          /* U >= 0                                                                   */
  int32_t max_len;            /* L >= 1: rows of each user's item block (its row stride)                  */
  int32_t d_model;            /* d: embedding width of items, candidates, H' and z                        */
  int32_t d_qk;               /* STA query/key width, = num_heads * d_qh (the paper's d_q; 16 per head)   */
  int32_t num_heads;          /* H >= 1, divides d_model and d_qk                                         */
  int32_t seg_size;           /* S >= 1, the paper's w;  L' = ceil(L / S)                                 */
  int32_t num_gsta_layers;    /* M >= 0, the paper's L_stack                                              */
  int32_t dtype;              /* laser_dtype                                                              */
  int32_t total_cands;        /* N = cand_offsets[U]                                                      */
  int32_t max_cands_per_user; /* an upper bound of cand_offsets[u+1] - cand_offsets[u] (sizes launch grids) */
  int32_t path;               /* laser_path                                                               */
  float sta_gamma;            /* gamma of Eq. 5;  <= 0 selects sqrt(d_qk / H)                             */
  float gsta_scale;           /* tau, the divisor of Eq. 7;  <= 0 selects sqrt(d / H)                     */
} laser_config;

/* Bytes of device scratch that laser_sta_forward / laser_gsta_forward / laser_forward need for `cfg`
 * (the maximum over the three; includes room for an internal H' when laser_forward is not given one).
 * Returns 0 if cfg is NULL or invalid.  Host-only, launches nothing. */
LASER_API size_t laser_workspace_bytes(const laser_config* cfg);

/* STA (Eq. 3-5 in the global form Eq. 8-12).
 *   items        [U, L, d]   item embeddings; rows >= lengths[u] of user u are ignored (must be finite)
 *   lengths      [U] int32   valid prefix length of each user, 0..L
 *   cands        [N, d]      candidate (target) embeddings
 *   cand_offsets [U+1] int32 user u owns candidates [cand_offsets[u], cand_offsets[u+1])
 *   Wq, Wk       [d, d_qk];  Wv [d, d]
 *   Hprime       [N, L', d]  OUT: every row is written (zero rows for empty segments)
 *   workspace    device scratch of at least laser_workspace_bytes(cfg) bytes, 256-byte aligned
 */
LASER_API int laser_sta_forward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                      const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, void* Hprime,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* GSTA (Eq. 7 and the residual update t_l = t_{l-1} + o_l), M = cfg->num_gsta_layers layers over a
 * caller-supplied H'.
 *   Hprime  [N, L', d]    segment vectors (rows of empty segments are not read)
 *   Wgsta   [M, 3, d, d]  per layer W_q^l, W_k^l, W_v^l
 *   z       [N, d]        OUT
 */
LASER_API int laser_gsta_forward(const laser_config* cfg, const void* Hprime, const int32_t* lengths,
                       const int32_t* cand_offsets, const void* cands, const void* Wgsta, void* z,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* STA followed by GSTA.  Hprime may be NULL (H' is then kept in the workspace or never materialised);
 * when non-NULL it receives the same values laser_sta_forward would write. */
LASER_API int laser_forward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                  const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv, const void* Wgsta,
                  void* Hprime, void* z, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* laser_forward for item embeddings stored without padding (a packed, CSR-style layout): user u's rows are
 * items_packed[item_offsets[u] .. item_offsets[u] + lengths[u]), so a batch of ragged sequences costs memory for its
 * valid items only.  The paper does not fix a memory layout; everything computed is as for laser_forward.
 *   items_packed  [item_offsets[U], d]
 *   item_offsets  [U+1] int32 (DEVICE), non-decreasing; user u's valid prefix must fit before item_offsets[U]
 *                 (a violation is reported as LASER_ERR_BAD_INPUT through the status word and that user is skipped)
 * cfg->max_len still bounds every length and fixes L' = ceil(max_len / S). */
LASER_API int laser_forward_packed(const laser_config* cfg, const void* items_packed, const int32_t* item_offsets,
                                   const int32_t* lengths, const void* cands, const int32_t* cand_offsets,
                                   const void* Wq, const void* Wk, const void* Wv, const void* Wgsta, void* Hprime,
                                   void* z, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Multi-resolution feature fusion (section "Multi-resolution Feature Fusion"): per candidate the concatenation
 *   fused = [ z | max over the non-empty segments j of s_j (element-wise) | s_0 | ... | s_{r-1} ]     in R^{(2 + r) d}
 * of the GSTA output, the max-pooled compact sequence and the r most recent segment vectors.  Segment 0 holds the most
 * recent items; empty segments take no part in the max (a user without segments gets zeros there), and a recent slot
 * j beyond the user's non-empty segments (or beyond L') is a zero vector.
 *   Hprime      [N, L', d]        segment vectors (rows of empty segments are not read)
 *   z           [N, d]            GSTA output
 *   num_recent  r >= 0
 *   fused       [N, (2 + r) * d]  OUT
 *   workspace   at least 256 bytes, 256-byte aligned: only the status word at its start is used
 * Works for either dtype and any path; d * sizeof(element) must be a multiple of 16. */
LASER_API int laser_fusion_forward(const laser_config* cfg, const void* Hprime, const void* z, const int32_t* lengths,
                                   const int32_t* cand_offsets, int32_t num_recent, void* fused, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream);

/* Feed-forward refinement of the segment vectors (Eq. 6):  s_i <- LN(FFN(s_i) + s_i)  for every non-empty segment of
 * every candidate.  The paper fixes the residual + layer-norm form and the expansion ratio r (d_hidden = r d, r = 4 in
 * its cost model); this library takes FFN(s) = max(s W1 + b1, 0) W2 + b2 and LN(y) = (y - mean) / sqrt(var + eps) *
 * gain + shift over the d features (biased variance).  Rows of empty segments are left as they are.
 * All pointers are DEVICE pointers in the config's dtype, 16-byte aligned, owned by the caller. */
typedef struct laser_ffn_params {
  int32_t d_hidden;      /* r * d >= 1 (the tcgen05 kernel needs a multiple of 128; other widths run on the FP32 ALUs) */
  float ln_eps;          /* <= 0 selects 1e-5                                                                          */
  const void* W1;        /* [d, d_hidden]                                                                              */
  const void* b1;        /* [d_hidden]                                                                                 */
  const void* W2;        /* [d_hidden, d]                                                                              */
  const void* b2;        /* [d]                                                                                        */
  const void* ln_gain;   /* [d]                                                                                        */
  const void* ln_shift;  /* [d]                                                                                        */
} laser_ffn_params;

/* Bytes of device scratch laser_ffn_forward and laser_forward_ffn need: laser_workspace_bytes(cfg) plus the row
 * prefix and the weight images of the FFN.  Returns 0 if cfg is NULL / invalid or d_hidden < 1.  Host-only. */
LASER_API size_t laser_ffn_workspace_bytes(const laser_config* cfg, int32_t d_hidden);

/* Eq. 6 in place on a caller-supplied H'.
 *   Hprime  [N, L', d]  IN / OUT: rows of non-empty segments are replaced by LN(FFN(s) + s)
 *   workspace           at least laser_ffn_workspace_bytes(cfg, ffn->d_hidden) bytes, 256-byte aligned
 * BF16 with d a multiple of 16 (<= 128) and d_hidden a multiple of 128 runs on the tensor cores (bf16 operands and
 * hidden activations, fp32 accumulation and normalisation) unless cfg->path is LASER_PATH_SIMT or the bias / layer-norm
 * vectors no longer fit beside the tiles in shared memory (at d = 128: d_hidden > 512); everything else runs in fp32
 * on the ALUs.  LASER_ERR_UNSUPPORTED when neither kernel takes the shape. */
LASER_API int laser_ffn_forward(const laser_config* cfg, const laser_ffn_params* ffn, void* Hprime,
                                const int32_t* lengths, const int32_t* cand_offsets, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/* The paper's full compression stack: STA (Eq. 8-12), then Eq. 6 on every segment vector, then GSTA (Eq. 7).
 * Arguments as for laser_forward plus `ffn`; Hprime (optional) receives the refined segment vectors.
 *   workspace  at least laser_ffn_workspace_bytes(cfg, ffn->d_hidden) bytes */
LASER_API int laser_forward_ffn(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                                const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv,
                                const void* Wgsta, const laser_ffn_params* ffn, void* Hprime, void* z, void* workspace,
                                size_t workspace_bytes, void* cuda_stream);

/* The softmax-aggregation variant of STA (the component-ablation table's row on the sigmoid aggregation, where the
 * gate is swapped for an ordinary softmax over the segment): inside every segment the weights of the valid items are exp(q_h . k_{n,h} / gamma)
 * normalised to sum to one per (candidate, head); everything else (projections of Eq. 4, heads, ragged lengths, zero
 * rows for empty segments) is as in laser_sta_forward.  Two versions: on the tensor cores (bf16 shapes the tensor
 * path supports; cfg->path LASER_PATH_AUTO or LASER_PATH_TENSOR, the latter answering LASER_ERR_UNSUPPORTED for other
 * shapes) and on the FP32 ALUs (every other case, LASER_PATH_STREAM included: the variant has no one-candidate
 * version).  The tensor-core version rounds Q and K to bf16 before the product and evaluates exp with the row's
 * maximum over the first 32 valid items of the segment as the shift; a logit more than 41 nats above that shift is
 * treated as 41 nats above it.
 *   workspace  at least laser_sta_softmax_workspace_bytes(cfg) bytes, 256-byte aligned */
LASER_API size_t laser_sta_softmax_workspace_bytes(const laser_config* cfg);
LASER_API int laser_sta_softmax_forward(const laser_config* cfg, const void* items, const int32_t* lengths,
                                        const void* cands, const int32_t* cand_offsets, const void* Wq, const void* Wk,
                                        const void* Wv, void* Hprime, void* workspace, size_t workspace_bytes,
                                        void* cuda_stream);

/* Backward pass of laser_forward: given dz = dLoss/dz [N, d], the gradients of the loss with respect to every input of
 * the forward, i.e. the chain rule through Eq. 7 and its residual updates (layers last to first), then through the
 * segment sums and gates (Eq. 10-12) and the projections (Eq. 8-9).  The paper trains the model (section "Experimental
 * Settings") and prints no backward formulas; readings are those of the forward (an item at or past its user's length
 * receives a zero gradient row, an empty segment passes no gradient).  All gradients are fp32 device arrays, whatever
 * cfg->dtype; the inputs are read in cfg->dtype.  The forward is recomputed and every intermediate kept in the workspace;
 * padded item layout only.  Two versions, chosen by cfg->path:
 *   LASER_PATH_SIMT                 FP32 ALUs throughout, either dtype: every gradient within 1e-4 of its largest entry.
 *   LASER_PATH_AUTO / _STREAM       fp32 batches as above.  bf16 batches on the tensor cores: every batched matrix product
 *                                   with TF32 operands and fp32 accumulation, and, when max_cands_per_user >= 8 and the head
 *                                   widths d_qk / H and d / H are multiples of 16 (d_qk / H at most 32, d / H at most 64), the
 *                                   five contractions through the gates, the recomputed H' and (d in {32, 64, 128}, at most 8
 *                                   heads and 128 segments) the GSTA attention with bf16 operands, as the forward's
 *                                   tensor-core path rounds them: every gradient within 2e-2 of its largest entry while the
 *                                   attention logits stay within a few nats (at tens of nats the bf16 rounding of a
 *                                   segment vector alone moves a softmax weight by several per cent: ask for the FP32 ALUs).
 *   LASER_PATH_TENSOR               as LASER_PATH_AUTO for bf16 batches; LASER_ERR_UNSUPPORTED for fp32 batches.
 *   dz          [N, d] fp32            IN
 *   d_items     [U, L, d] fp32         OUT (rows of padding are zero)
 *   d_cands     [N, d] fp32            OUT
 *   dWq, dWk    [d, d_qk] fp32         OUT
 *   dWv         [d, d] fp32            OUT
 *   dWgsta      [M, 3, d, d] fp32      OUT (may be NULL when M = 0)
 *   workspace   at least laser_backward_workspace_bytes(cfg) bytes, 256-byte aligned; its first word is the status word
 * Sums over candidates that end in one weight matrix (and the query-side part of d_cands) are finished with
 * floating-point atomics: their last bits may differ from call to call. */
LASER_API size_t laser_backward_workspace_bytes(const laser_config* cfg);
LASER_API int laser_backward(const laser_config* cfg, const void* items, const int32_t* lengths, const void* cands,
                             const int32_t* cand_offsets, const void* Wq, const void* Wk, const void* Wv,
                             const void* Wgsta, const float* dz, float* d_items, float* d_cands, float* dWq, float* dWk,
                             float* dWv, float* dWgsta, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* STA without any workspace argument, for callers that cannot allocate device memory (no counterpart in the
 * paper: this is a deployment convenience of this library).  Think of a plug-in inside a serving process
 * whose GPU memory belongs entirely to the host framework's pool, or of a request thread that must never hit
 * cudaMalloc's device-wide synchronisation: such a caller has inputs and an output buffer, but no scratch.
 * This entry point computes exactly what laser_sta_forward computes with path = LASER_PATH_SIMT, and keeps
 * the fp32 Q / K / V scratch in an array compiled into the library (LASER_STATIC_SCRATCH_BYTES per GPU that
 * loads the library, held until the process exits).  It never calls cudaMalloc / cudaFree or any allocating
 * routine.
 *   - Size limit: 256 + 4*(N*d_qk + U*L*(d_qk + d)) bytes (each term rounded up to 256) must fit in
 *     LASER_STATIC_SCRATCH_BYTES, otherwise LASER_ERR_WORKSPACE is returned and nothing is launched.
 *   - cfg->path is ignored; items .. Hprime are as for laser_sta_forward.
 *   - status_out: optional DEVICE int32; if non-NULL the device-side status word of this call (LASER_OK or
 *     LASER_ERR_BAD_INPUT) is copied to it on the stream after the kernels.
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents (only the status
 *     word is cleared per call): two calls that overlap on the GPU (different streams or threads) race.
 *     Serialise them on one stream or with events. */
#define LASER_STATIC_SCRATCH_BYTES (8u << 20)
LASER_API int laser_sta_forward_static(const laser_config* cfg, const void* items, const int32_t* lengths,
                                       const void* cands, const int32_t* cand_offsets, const void* Wq,
                                       const void* Wk, const void* Wv, void* Hprime, int32_t* status_out,
                                       void* cuda_stream);

/* Device scratch laser_forward_host needs: laser_workspace_bytes(cfg) plus staging for every input and z. */
LASER_API size_t laser_host_workspace_bytes(const laser_config* cfg);

/* laser_forward for callers whose data lives in HOST memory (the end-to-end path): copies the inputs to
 * the device, runs laser_forward without H' output, copies z back.  Rows of items_h at or past a user's length
 * need not cross the bus: when that saves enough, only each user's valid prefix travels, into a gap-free
 * device array that the kernels read as in laser_forward_packed.  If items_h is pinned (or registered) host
 * memory, one kernel reads the valid rows straight from it; otherwise there is one copy per run of users whose
 * valid rows are contiguous in items_h.  z is bit-identical whatever the route.
 *   items_h, lengths_h, cands_h, cand_offsets_h, Wq_h, Wk_h, Wv_h, Wgsta_h : HOST pointers, same shapes
 *       and dtype as above (pinned memory makes the copies asynchronous; pageable memory also works)
 *   z_h        HOST pointer, OUT [N, d]
 *   workspace  DEVICE scratch of at least laser_host_workspace_bytes(cfg) bytes
 *   blocking   non-zero: wait for the stream and return the device status too; zero: return after enqueue
 *              (z_h is valid once the stream has drained)
 */
LASER_API int laser_forward_host(const laser_config* cfg, const void* items_h, const int32_t* lengths_h,
                       const void* cands_h, const int32_t* cand_offsets_h, const void* Wq_h, const void* Wk_h,
                       const void* Wv_h, const void* Wgsta_h, void* z_h, void* workspace, size_t workspace_bytes,
                       void* cuda_stream, int blocking);

/* Bytes laser_forward_host moves for this batch: host to device (every input; of the items only what the
 * route chosen for this pointer and these lengths transfers) and device to host (z).  Launches nothing.
 *   items_h    HOST pointer as it would be passed to laser_forward_host (only its kind and alignment matter;
 *              null: treated as pageable memory)
 *   lengths_h  HOST pointer, [U]
 *   h2d_bytes, d2h_bytes  HOST pointers, OUT
 * Returns LASER_OK, or LASER_ERR_INVALID_ARG / LASER_ERR_UNSUPPORTED as laser_forward_host would. */
LASER_API int laser_host_transfer_bytes(const laser_config* cfg, const void* items_h, const int32_t* lengths_h,
                                        size_t* h2d_bytes, size_t* d2h_bytes);

/* Diagnostics.
 *
 * laser_workspace_regions: the regions of the carve-up of a laser_workspace_bytes(cfg) workspace, in order, as byte
 * offsets and bytes in use.  A call with this configuration writes inside these regions only: each is followed by at
 * least 256 bytes that no kernel touches, so a test can fill the workspace with a pattern, run a call and find the
 * pattern intact everywhere else (the place of a memory checker on machines that have none).
 *   offsets, sizes  HOST pointers, OUT, room for max_regions entries each (may be null when max_regions is 0)
 * Returns the number of regions (which may exceed max_regions), or a negative status for an invalid configuration.
 *
 * laser_selftest_wait_timeout: exercises the give-up path of the bounded device-side waits (every wait on a copy or on
 * the tensor cores in this library has a poll budget).  One small block waits, with a budget of poll_limit polls
 * (1 .. 4096), for a barrier that nothing ever completes, gives up, releases its tensor memory and reports
 * LASER_ERR_TIMEOUT through the status word exactly as a production block would; the context stays usable and the next
 * call on the same workspace runs normally.  Nothing faults, traps or hangs.
 *   workspace  DEVICE pointer, 256-byte aligned, at least 256 bytes; its first word receives the status
 * Returns LASER_OK once the block is enqueued (LASER_ERR_INVALID_ARG / LASER_ERR_WORKSPACE / LASER_ERR_CUDA otherwise);
 * laser_check_status(workspace, stream) then returns LASER_ERR_TIMEOUT. */
LASER_API int laser_workspace_regions(const laser_config* cfg, int max_regions, size_t* offsets, size_t* sizes);
LASER_API int laser_selftest_wait_timeout(void* workspace, size_t workspace_bytes, int32_t poll_limit, void* cuda_stream);

/* Waits for `cuda_stream`, reads the device status word at the start of `workspace` and returns it
 * (LASER_OK, LASER_ERR_TIMEOUT, LASER_ERR_BAD_INPUT) or LASER_ERR_CUDA if the stream reports an error. */
LASER_API int laser_check_status(const void* workspace, void* cuda_stream);

/* Number of kernels the last successful call on this host thread enqueued (launch accounting for benchmarks). */
LASER_API int laser_last_launch_count(void);

/* Per-kernel timing for benchmarks (state is per host thread).  laser_profile_enable(1) makes every later
 * forward call on this thread bracket each of its kernel launches with CUDA events recorded on the call's
 * stream (the first such call creates the events); laser_profile_enable(0) turns that off again.
 * laser_profile_read waits for the last profiled call's kernels and writes, for up to `max_kernels` of them
 * in launch order, the duration in milliseconds to ms_out[i] (HOST) and a static name to names_out[i] (HOST);
 * it returns how many entries it wrote, or a negative laser_status. */
LASER_API int laser_profile_enable(int on);
LASER_API int laser_profile_read(int max_kernels, float* ms_out, const char** names_out);

/* Static description of a laser_status value. */
LASER_API const char* laser_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* LASER_H_ */
