/* maskkv.h - C ABI of the MaskKV compress-and-attend path for NVIDIA B200 (sm_100a).
 *
 * The path, per transformer layer of a diffusion LLM (paper: "Mask Tokens as Prophet", Section
 * "The MaskKV Framework"):
 *
 *   maskkv_score    Stage 1, Eq. 6-7: the mask-token queries vote on the prompt keys through softmax
 *                   attention; also the two attention-mass sums of Eq. 14.
 *   maskkv_budget   Stage 2, Eq. 14-15: per-head budgets from the prompt preference, plus the exclusive
 *                   prefix sum that lays out the ragged cache.  (maskkv_layer_budgets: Eq. 9-13, host.)
 *   maskkv_select   Eq. 16: per head, keep the top-k prompt tokens.
 *   maskkv_compact  gather the kept K/V rows into the ragged per-head cache.
 *   maskkv_attend   a later denoising step: attention over [compacted prompt segment ; live keys]
 *                   (appendix, proof step 3: out_m = sum_j softmax(q_m k_j / sqrt(d_k)) V_j).
 *
 * Conventions that hold for every function:
 *   - Return value: 0 (MASKKV_OK) or a negative MASKKV_E_* code.  Nothing throws, aborts or prints.
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; the library neither frees nor keeps
 *     them past the call.  Pointers named *_host (and the *_cu arrays of the descriptor) are HOST
 *     pointers that only need to stay valid until the call returns.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default stream) and the
 *     call returns without synchronising.  The only synchronising call is maskkv_check_status.
 *   - Device pointers to tensors (Q/K/V/O, scores, kept_idx, the caches, workspaces) must be 16-byte aligned, the small
 *     int32 / float arrays (budgets, offsets, masses, cumulative lengths) 4-byte aligned (MASKKV_E_ALIGN otherwise);
 *     head_dim is contiguous.
 *   - Arguments are validated before anything is launched.  A failed validation launches nothing.
 *   - Outputs are fully written for every valid (request, head) segment and untouched elsewhere.
 *     The same inputs give bit-identical outputs on every call (no order-dependent float atomics).
 *   - No call allocates device memory; scratch comes from the caller's workspace
 *     (maskkv_workspace_bytes).  maskkv_create allocates one 256-byte status block.
 *   - Requests are independent.  A batch of layers can be run in one call by treating
 *     (layer, request) as the request axis.
 *
 * Tensor layouts (T = MASKKV_F32 or MASKKV_BF16, chosen by desc.dtype for every Q/K/V/O tensor):
 *   q_mask, q_live, out    T   [sum_M][H   ][d]   token stride q_token_stride, head stride q_head_stride
 *   k_prompt, v_prompt     T   [sum_N][H_kv][d]   token stride kv_token_stride, head stride kv_head_stride
 *   k_mask, k_live, v_live T   [sum_M][H_kv][d]   same kv strides
 *   scores                 f32 [H_kv][sum_N]      I_j of Eq. 7, one contiguous segment per (head, request)
 *   mass_p, mass_m         f32 [R][H_kv]          S_{m->p}, S_{m->m} of Eq. 14
 *   budgets                i32 [R][H_kv]          k_{l,h} of Eq. 15
 *   offsets                i32 [R*H_kv + 1]       exclusive prefix sum of budgets; segment s = r*H_kv + h
 *   kept_idx               i32 [capacity]         request-local prompt indices, ascending within a segment
 *   kc, vc                 T   [capacity][d]      compacted cache; rows of segment s are contiguous
 *   lse                    f32 [H][sum_M]         log of the softmax denominator (optional)
 * sum_N = prompt_cu[R], sum_M = live_cu[R].  Strides are in elements.
 */
#ifndef MASKKV_H_
#define MASKKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MASKKV_OK = 0,
  MASKKV_E_INVALID = -1,      /* null pointer, negative size, inconsistent descriptor */
  MASKKV_E_UNSUPPORTED = -2,  /* dtype / head_dim / device the library has no kernel for */
  MASKKV_E_ALIGN = -3,        /* a device pointer or stride breaks the 16-byte rule */
  MASKKV_E_WORKSPACE = -4,    /* workspace missing or smaller than maskkv_workspace_bytes */
  MASKKV_E_CAPACITY = -5,     /* capacity too small for what the host can bound */
  MASKKV_E_CUDA = -6,         /* a CUDA runtime or driver call failed */
  MASKKV_E_TIMEOUT = -7       /* reported by maskkv_check_status: a bounded device wait expired */
};

enum { MASKKV_F32 = 0, MASKKV_BF16 = 1 };

/* Bits of the device status word returned by maskkv_check_status. */
enum {
  MASKKV_FLAG_TIMEOUT = 1u,   /* a bounded mbarrier wait gave up; that launch's outputs are invalid */
  MASKKV_FLAG_CAPACITY = 2u,  /* maskkv_budget clipped budgets to fit `capacity` */
  MASKKV_FLAG_BOUNDS = 4u,    /* an index read from device memory was out of range and was skipped */
  MASKKV_FLAG_FALLBACK = 8u   /* a bf16 call the tensor-core kernels should have served ran on the FP32-pipe kernels
                                 instead (tensor map not encodable, launch refused): results are valid, the call
                                 was one to two orders of magnitude slower.  Not raised when MASKKV_FORCE_SIMT asks
                                 for those kernels. */
};

typedef struct maskkv_ctx maskkv_ctx;

/* Opens the library on CUDA device `device` (which must be compute capability 10.x, else
 * MASKKV_E_UNSUPPORTED).  Allocates the status block and resolves the tensor-map encoder.
 * The context may be used from one host thread at a time. */
int maskkv_create(maskkv_ctx** out, int device);
int maskkv_destroy(maskkv_ctx* ctx);

/* Static, human-readable name of a return code. */
const char* maskkv_status_string(int code);

/* Waits for `stream`, then returns the device status flags accumulated since the last call in
 * *flags_out (may be NULL) and clears them.  Returns MASKKV_E_TIMEOUT if the TIMEOUT flag was set,
 * MASKKV_E_CUDA if the stream reported an error, else MASKKV_OK. */
int maskkv_check_status(maskkv_ctx* ctx, void* stream, uint32_t* flags_out);

/* Self-test of the bounded waits (every wait on a barrier inside the tensor-core kernels gives up after about one
 * second instead of spinning forever): enqueues one thread that waits for a signal nothing sends.  The kernel returns
 * after the limit with MASKKV_FLAG_TIMEOUT raised, so the next maskkv_check_status returns MASKKV_E_TIMEOUT and the
 * context stays usable.  For tests of the error path; it touches no caller memory. */
int maskkv_selftest_wait_expiry(maskkv_ctx* ctx, void* stream);

/* Measurement aid (the paper has no counterpart): enqueues a kernel that does nothing but evaluate base-2 exponentials
 * on the special-function unit - the instruction that bounds maskkv_score, which exponentiates every logit once per
 * sweep (Eq. 6) - on every SM, `iters` rounds per thread (1 .. 2^20).  *n_exp_out (host) receives the number of
 * exponentials the launch evaluates; the caller times the launch with events on `stream` and divides, which gives the
 * measured peak that maskkv_score's exponential throughput is compared with.  `scratch_dev`: one float of device memory
 * (never written in practice).  Returns MASKKV_E_INVALID on a NULL pointer or an `iters` out of range. */
int maskkv_selftest_exp_rate(maskkv_ctx* ctx, int iters, float* scratch_dev, int64_t* n_exp_out, void* stream);

/* Text of the most recent CUDA runtime error behind a MASKKV_E_CUDA return of this context ("" if none). */
const char* maskkv_last_cuda_error(const maskkv_ctx* ctx);

/* Number of kernels this context has launched so far (host counter; for benchmarks and for checking
 * that a failed validation launched nothing). */
uint64_t maskkv_launch_count(const maskkv_ctx* ctx);
/* Of those, the launches of tcgen05 (tensor-core) kernels: bf16 scoring sweeps and bf16 attention. */
uint64_t maskkv_tensor_core_launch_count(const maskkv_ctx* ctx);

typedef struct {
  int32_t dtype;              /* MASKKV_F32 | MASKKV_BF16 */
  int32_t n_q_heads;          /* H */
  int32_t n_kv_heads;         /* H_kv, divides H */
  int32_t head_dim;           /* d: 64 or 128 */
  int32_t n_requests;         /* R >= 1 */
  float softmax_scale;        /* <= 0 selects 1/sqrt(head_dim) (Eq. 6) */
  const int32_t* prompt_cu;   /* HOST [R+1] cumulative prompt lengths, prompt_cu[0] = 0 */
  const int32_t* live_cu;     /* HOST [R+1] cumulative mask/live lengths */
  const int32_t* prompt_cu_dev; /* DEVICE copies of the two arrays */
  const int32_t* live_cu_dev;
  int64_t q_token_stride, q_head_stride;     /* elements; 0 selects the packed layout */
  int64_t kv_token_stride, kv_head_stride;
} maskkv_desc_t;

/* Bytes of scratch that maskkv_score and maskkv_select may need for this descriptor (the larger of
 * the two).  Never fails; returns 0 for an invalid descriptor. */
size_t maskkv_workspace_bytes(const maskkv_ctx* ctx, const maskkv_desc_t* desc);

/* Eq. 9-13, host only: splits the total budget k_p (in per-head units, i.e. n_layers x the nominal
 * per-head budget) over the layers.  importance_host [n_layers] is the offline layer-importance
 * profile (Eq. 8); is_boundary_host [n_layers] marks the boundary group (NULL = first and last layer).
 * k_group values stay real until the floor of Eq. 13; floors are floor(x + 1e-6) in double precision.
 * Writes k_l_out_host [n_layers]. */
int maskkv_layer_budgets(int64_t k_p, double beta, int32_t n_layers, const double* importance_host,
                         const uint8_t* is_boundary_host, int32_t* k_l_out_host);

/* Eq. 8, the calibration step that produces the offline profile consumed by maskkv_layer_budgets:
 *   importance = 1 - (1/n) sum_i cos_sim(h_in[i], h_out[i])
 * over the n_tokens rows of one layer's attention sub-layer input / output hidden states (T = dtype, [n_tokens][hidden],
 * row strides in elements, 0 = packed; hidden * sizeof(T) and the strides must be multiples of 16 bytes).  A row with a
 * zero vector counts as cosine 0.  Writes one float to importance_out_dev.  Needs
 * maskkv_layer_importance_workspace_bytes(ctx) bytes of scratch (8-byte aligned).  Deterministic: the same inputs
 * give the same bits on every call. */
size_t maskkv_layer_importance_workspace_bytes(const maskkv_ctx* ctx);
int maskkv_layer_importance(maskkv_ctx* ctx, int32_t dtype, const void* h_in_dev, const void* h_out_dev,
                            int64_t n_tokens, int32_t hidden, int64_t in_row_stride, int64_t out_row_stride,
                            float* importance_out_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* The response-token refresh rule of the feature cache the method is built on (appendix, "Response tokens"): which of
 * the n_tokens response rows must be recomputed at this denoising step,
 *   S_shift = { i : cos_sim(v_cur[i], v_prev[i]) < delta },
 * v_cur / v_prev = the value features of the rows at this step and the previous one (T = dtype, [n_tokens][width], all
 * heads of a token side by side; row strides in elements, 0 = packed; width * sizeof(T) and the strides multiples of
 * 16 bytes).  refresh_all != 0 marks a periodic-refresh step (t mod T_r = 0, decided by the caller): every row is
 * taken.  A row with a zero vector counts as cosine 0.  Outputs: idx_out_dev [n_tokens] receives the refreshed row
 * numbers in ascending order (entries past the count are unspecified), count_out_dev [1] their number, cos_out_dev
 * [n_tokens] the cosines (optional, may be NULL).  The comparison is made on the fp32 cosine.  No workspace. */
int maskkv_refresh_set(maskkv_ctx* ctx, int32_t dtype, const void* v_cur_dev, const void* v_prev_dev, int64_t n_tokens,
                       int32_t width, int64_t cur_row_stride, int64_t prev_row_stride, float delta, int32_t refresh_all,
                       float* cos_out_dev, int32_t* idx_out_dev, int32_t* count_out_dev, void* stream);

/* Mask-only projection (appendix, "Mask-only Projection"): the vocabulary projection of the final hidden states at
 * the masked positions only,
 *   logits[m][v] = sum_k hidden[positions[m]][k] * w_vocab[v][k],   m < n_mask, v < vocab,
 * bf16 operands, fp32 accumulation on the tensor cores.  hidden_dev [n_tokens][width] and w_vocab_dev [vocab][width]
 * are bf16 (dtype must be MASKKV_BF16; anything else returns MASKKV_E_UNSUPPORTED), row strides in elements
 * (0 = packed), width and the strides multiples of 8 elements, bases 16-byte aligned.  positions_dev [n_mask] holds
 * the masked token rows (any order, repeats allowed; a position outside [0, n_tokens) gives a zero row and raises
 * MASKKV_FLAG_BOUNDS); NULL means rows 0..n_mask-1 of hidden_dev, read in place.  logits_out_dev [n_mask][vocab] is
 * fp32 (out_dtype MASKKV_F32, out_row_stride a multiple of 4) or bf16 rounded to nearest even (MASKKV_BF16, a
 * multiple of 8), 16-byte aligned, row stride in elements (0 = vocab).  Needs
 * maskkv_mask_project_workspace_bytes(n_mask, width) bytes of scratch (256-byte aligned; 0 when positions_dev is
 * NULL) for the packed rows.  Asynchronous on `stream`; n_mask = 0 launches nothing. */
size_t maskkv_mask_project_workspace_bytes(int64_t n_mask, int32_t width);
int maskkv_mask_project(maskkv_ctx* ctx, int32_t dtype, const void* hidden_dev, int64_t n_tokens, int32_t width,
                        int64_t hidden_row_stride, const int32_t* positions_dev, int32_t n_mask, const void* w_vocab_dev,
                        int32_t vocab, int64_t w_row_stride, int32_t out_dtype, void* logits_out_dev,
                        int64_t out_row_stride, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Eq. 6-7 and the sums of Eq. 14.  For every request r and KV head h: softmax (fp32) of
 * scale * q_i . k_j over the request's N_r prompt keys followed by its M_r mask keys, for each of the
 * H/H_kv query heads that share h; scores[h][prompt_cu[r] + j] = sum over those heads and mask rows i of
 * w_i * A_ij; mass_p = the same sum over prompt j; mass_m = over mask j.  row_weights_dev (f32 [sum_M],
 * NULL = all ones) weights each voting row.  The M x N weight matrix is never written to memory. */
int maskkv_score(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev,
                 const void* k_prompt_dev, const void* k_mask_dev, const float* row_weights_dev,
                 float* scores_dev, float* mass_p_dev, float* mass_m_dev, void* workspace_dev,
                 size_t workspace_bytes, void* stream);

/* maskkv_score with one more output, for the voter sets other than the mask tokens that the paper compares in its
 * voting ablations (all tokens, the prompt tokens, a trailing window of the prompt): scores_live_dev [H_kv][sum_M]
 * (may be NULL) receives the column sums over the live keys, scores_live[h][live_cu[r] + j] = sum over the voting rows
 * of A[i][N_r + j].  The call scores every key of K_full = [k_prompt ; k_mask] from the rows of q_mask, so any voter set
 * is a matter of which tokens are passed where: the voters' queries as q_mask with their own keys as k_mask, every
 * other token's keys as k_prompt (possibly none: scores_dev may then be NULL).  The importance of a prompt token is
 * then read from scores_live if it votes and from scores if it does not.  Everything else as in maskkv_score. */
int maskkv_score_all_keys(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev, const void* k_prompt_dev,
                          const void* k_mask_dev, const float* row_weights_dev, float* scores_dev, float* scores_live_dev,
                          float* mass_p_dev, float* mass_m_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* maskkv_score for callers that cannot hand over a workspace.  (The paper has no counterpart: this is a
 * packaging variant of the call above, same arithmetic, same outputs.)
 *
 * Who needs it: code that runs where device allocation is off limits - inside a serving loop whose memory
 * pool is fixed and fully handed out at start-up, in a plugin that is given tensors but no allocator, or
 * next to a stream-ordered allocator whose pool must not be touched from a side library.  Such a caller
 * cannot call cudaMalloc (or ask torch for a buffer) to create the scratch maskkv_score wants.
 *
 * The scratch is instead a fixed array of maskkv_score_noalloc_max_bytes() = 8 MiB that is part of the
 * library image: each GPU that loads the library reserves those bytes until the process exits, used or not.
 * The call allocates nothing and frees nothing.  If maskkv_workspace_bytes(desc) exceeds the array the call
 * returns MASKKV_E_WORKSPACE and launches nothing (8 MiB covers a single request of up to about 57,000 prompt
 * keys at 32 heads x 256 mask rows; batches need the regular call).
 *
 * The first call on each device looks up the array's device address (a one-time, host-side set-up step);
 * make that first call outside any stream capture.  All calls on a device share the one array, and it keeps
 * whatever the previous call left in it - harmless, because every word the kernels read they first write in
 * the same call - but two calls that overlap on the GPU (different streams, or the same stream from two
 * contexts) would overwrite each other's partial results: serialise them.  Inputs and outputs are the
 * caller's, exactly as for maskkv_score. */
int maskkv_score_noalloc(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_mask_dev,
                         const void* k_prompt_dev, const void* k_mask_dev, const float* row_weights_dev,
                         float* scores_dev, float* mass_p_dev, float* mass_m_dev, void* stream);
size_t maskkv_score_noalloc_max_bytes(void);

/* Eq. 14-15, clamp and prefix sum, all on the device (no host synchronisation):
 *   P = mass_p / (mass_p + mass_m); Phat = P / sum_h P (ascending h);
 *   x = alpha*k_l + ((1-alpha)*(H_kv*k_l))*Phat; k = floor(x + 1e-6) clamped to [0, N_r]
 * in IEEE double precision without fused multiply-add, so equal inputs give equal integers on any
 * conforming implementation.  k_l applies to every request unless k_l_per_request_dev (i32 [R]) is
 * given.  If the running total would exceed `capacity` (rows available in kept_idx / kc / vc) the
 * segment that crosses it is clipped, later ones get 0, and MASKKV_FLAG_CAPACITY is raised. */
int maskkv_budget(maskkv_ctx* ctx, const maskkv_desc_t* desc, int32_t k_l,
                  const int32_t* k_l_per_request_dev, double alpha, const float* mass_p_dev,
                  const float* mass_m_dev, int64_t capacity, int32_t* budgets_dev, int32_t* offsets_dev,
                  void* stream);

/* Eq. 16.  For segment s = (r, h): kept_idx[offsets[s] .. offsets[s+1]) receives the indices of the
 * budgets[s] largest scores of scores[h][prompt_cu[r] .. prompt_cu[r+1]) under the total order
 * (score descending, index ascending; NaN below every number), written in ascending index order.
 * Exact: no tolerance is involved. */
int maskkv_select(maskkv_ctx* ctx, const maskkv_desc_t* desc, const float* scores_dev,
                  const int32_t* budgets_dev, const int32_t* offsets_dev, int32_t* kept_idx_dev,
                  void* workspace_dev, size_t workspace_bytes, void* stream);

/* kc[offsets[s] + t] = k_prompt[prompt_cu[r] + kept_idx[offsets[s] + t]][h][:], same for v: a byte copy.
 * `capacity` is the number of rows kc/vc/kept_idx hold; rows at or beyond it are never touched.
 * k_prompt_dev / v_prompt_dev only have to be addresses the device can read: this call is the path's only reader of
 * v_prompt, so a caller whose prompt values live in pinned (device-mapped) host memory can pass that pointer and have
 * the kept rows alone cross the bus. */
int maskkv_compact(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* k_prompt_dev,
                   const void* v_prompt_dev, const int32_t* kept_idx_dev, const int32_t* offsets_dev,
                   int64_t capacity, void* kc_dev, void* vc_dev, void* stream);

/* One attention step of the live region.  For request r and query head h (KV head h / (H/H_kv)):
 * softmax of scale * q_i . k over the rows [offsets[s], offsets[s+1]) of kc followed by the request's
 * M_r live keys (no mask, own key included); out = weights x [vc rows ; v_live].  bf16: fp32 accumulation
 * and softmax; the tensor-core kernels round the weights to bf16 before the second product (the FP32-pipe kernels that
 * serve fp32 problems, and bf16 ones under MASKKV_FORCE_SIMT, keep them in fp32).
 * `capacity` is the number of rows kc/vc hold: nothing beyond it is read, and offsets that point past it are clipped
 * with MASKKV_FLAG_BOUNDS raised (FP32-pipe kernels) or read as zero rows (tensor-core kernels, through the tensor
 * map's bounds).  lse_dev (f32 [H][sum_M]) may be NULL. */
int maskkv_attend(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_live_dev,
                  const void* k_live_dev, const void* v_live_dev, const void* kc_dev, const void* vc_dev,
                  const int32_t* offsets_dev, int64_t capacity, void* out_dev, float* lse_dev, void* stream);

/* The attention step with partial refresh: the feature cache the method builds on recomputes, at most steps, only the
 * response rows whose value features drifted (maskkv_refresh_set), so only those rows have queries - while the keys and
 * values are still the compacted prompt cache followed by ALL live rows of the request.  q_rows_dev [rows][H][d] holds
 * the queries of the refreshed rows, request after request, rows_cu / rows_cu_dev (host and device copies, int32
 * [n_requests + 1], rows_cu[0] = 0) their cumulative counts; a request may have none.  out_rows_dev has the layout of
 * q_rows_dev, lse_rows_dev (may be NULL) is f32 [H][rows].  Which live row a query belongs to does not matter (no
 * mask).  Both rows_cu pointers NULL: the queries are the live rows themselves, i.e. maskkv_attend.  Everything else
 * as in maskkv_attend. */
int maskkv_attend_rows(maskkv_ctx* ctx, const maskkv_desc_t* desc, const void* q_rows_dev, const int32_t* rows_cu,
                       const int32_t* rows_cu_dev, const void* k_live_dev, const void* v_live_dev, const void* kc_dev,
                       const void* vc_dev, const int32_t* offsets_dev, int64_t capacity, void* out_rows_dev,
                       float* lse_rows_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MASKKV_H_ */
