/*
 * libspo -- the data-parallel hot path of Single-stream Policy Optimization (SPO)
 * on NVIDIA B200 (sm_100a).  Plain C ABI.
 *
 * Conventions (every entry point):
 *   - Every pointer named d_* or documented "device" is device memory owned by the
 *     caller; the library allocates nothing and frees nothing.  Pointers must be
 *     16-byte aligned unless stated otherwise.  NULL is allowed only where marked
 *     "optional".
 *   - Work is enqueued on the caller's stream (`stream` is a cudaStream_t passed as
 *     void*; NULL = the default stream).  No call synchronises the host.
 *   - The return value is a host-side status (SPO_OK or a negative SPO_ERR_*),
 *     produced by argument checks and launch errors only.  Conditions found on
 *     the device (an id out of range, too few uniforms, a non-finite input, a
 *     bounded wait that ran out) are OR-ed as SPO_DEV_* bits into the caller's
 *     `d_status` word (device int32, must be zeroed by the caller beforehand);
 *     the offending element is skipped, nothing traps.  d_status may be NULL.
 *   - The device must be compute capability 10.x; otherwise SPO_ERR_UNSUPPORTED_ARCH.
 *   - Tracker table layout: `ab` is [N][2] fp32, interleaved (alpha, beta) per prompt.
 *   - Token rows are packed: sequence s owns rows cu_seqlens[s] .. cu_seqlens[s+1]-1.
 */
#ifndef SPO_H_
#define SPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host-side status */
#define SPO_OK                        0
#define SPO_ERR_INVALID_ARG          -1   /* NULL where required, negative size, bad flag */
#define SPO_ERR_BAD_SHAPE            -2   /* size outside what the kernels support */
#define SPO_ERR_BAD_ALIGNMENT        -3
#define SPO_ERR_UNSUPPORTED_DTYPE    -4
#define SPO_ERR_UNSUPPORTED_ARCH     -5
#define SPO_ERR_WORKSPACE_TOO_SMALL  -6
#define SPO_ERR_CUDA                 -7   /* see spo_last_cuda_error() */

/* device-side status bits (OR-ed into *d_status) */
#define SPO_DEV_ID_OUT_OF_RANGE       1   /* prompt id or target token outside its table */
#define SPO_DEV_NONFINITE             2   /* NaN/Inf reward, divergence or table entry */
#define SPO_DEV_UNIFORMS_EXHAUSTED    4   /* fewer than B distinct prompts accepted */
#define SPO_DEV_TIMEOUT               8   /* a bounded wait inside a kernel ran out */
#define SPO_DEV_ZERO_TOTAL_WEIGHT    16   /* all sampling weights are zero */

/* element types of H / W / dH */
#define SPO_DTYPE_F32   0
#define SPO_DTYPE_BF16  1

/* token weights in the objective's expectation E_{s,t} (the paper does not say how responses of
 * different length are weighted): every unmasked token alike (default), or every response alike
 * with its tokens sharing the response's weight */
#define SPO_AGG_TOKEN_MEAN  0
#define SPO_AGG_SEQ_MEAN    1

/* objective evaluated by the loss calls.  Sec. 3.2 defines the first and names the other two as
 * compatible with the SPO advantage without writing them out; they follow their own publications:
 *   PPO_CLIP  sum_t u_t min(ratio_t a, clip(ratio_t, 1-clip_lo, 1+clip_hi) a)          (the default)
 *   CISPO     sum_t u_t w_t a logp_t with w_t = clip(ratio_t, 1-clip_lo, 1+clip_hi) held constant
 *             (no gradient through the weight): coef_t = -u_t w_t a for every unmasked token
 *   GSPO      one ratio per response, r_i = exp(mean over its unmasked tokens of logp_t - logp_old_t);
 *             (1/S_act) sum_i min(r_i a_i, clip(r_i) a_i); coef_t = -a_i r_i [unclipped_i] / (S_act n_i);
 *             agg_mode does not apply.  Needs every token of a response before any coef exists, so
 *             spo_loss_fwd_bwd runs it as forward-then-backward (see there) */
#define SPO_SUR_PPO_CLIP  0
#define SPO_SUR_CISPO     1
#define SPO_SUR_GSPO      2

/* selectors for spo_workspace_bytes */
#define SPO_WS_SAMPLE      0
#define SPO_WS_ADVANTAGES  1
#define SPO_WS_LOSS_FWD    2
#define SPO_WS_LOSS_BWD    3
#define SPO_WS_UPDATE_REPEATS 4
#define SPO_WS_ACTIVE_ROWS    5
#define SPO_WS_LOSS_BWD_ROWS  6
#define SPO_WS_LOSS_FWD_BWD   7
#define SPO_WS_LOSS_FWD_BWD_ROWS 8

/*
 * Hyper-parameters.  Defaults (spo_default_params) are the values the paper prints:
 * rho_min 0.875, rho_max 0.96, clip_lo 0.2, clip_hi 0.28 (appendix "Training and
 * Evaluation Details"), eps_explore 0.05 (Sec. 3.3).  The paper names D_half but
 * gives no value; the default here is 0.1.  norm_eps and norm_ddof settle what the
 * paper leaves open about the batch standard deviation (population, +1e-8).
 */
typedef struct spo_params {
  float   rho_min;
  float   rho_max;
  float   d_half;
  float   eps_explore;
  float   clip_lo;
  float   clip_hi;
  float   norm_eps;
  int32_t norm_ddof;
  int32_t agg_mode;       /* SPO_AGG_*: how E_{s,t} of the objective weights tokens */
  /* Data-parallel training: when the mini-batch is spread over several ranks, the denominators of
   * the objective are those of the whole mini-batch.  0 = use this call's own counts. */
  int32_t global_tokens;     /* unmasked tokens of the whole mini-batch (n_tok) */
  int32_t global_responses;  /* responses with an unmasked token in the whole mini-batch (S_act) */
  int32_t surrogate;         /* SPO_SUR_*: which objective the loss calls evaluate */
  /* Second clip of dual-clip PPO (not in the paper; 0 = off, the default).  With c = dual_clip > 1 a
   * negative advantage's term becomes max(min(ratio a, clip(ratio) a), c a): once ratio > c the term
   * is the constant c a and carries no gradient.  Applies to SPO_SUR_PPO_CLIP (per token) and
   * SPO_SUR_GSPO (per response); SPO_SUR_CISPO has its own truncation and ignores it. */
  float   dual_clip;
  /* Tolerances of the near-zero-advantage counts (Sec. 4, signal efficiency: the share of raw
   * advantages with |A| <= tau, tracked at tau = 1e-4 and tau = 0.02). */
  float   near_zero_tau_lo;  /* 1e-4 */
  float   near_zero_tau_hi;  /* 0.02 */
} spo_params;

int32_t spo_default_params(spo_params* p /* host, out */);

/*
 * Algorithm 2 (SPO Initialization): N0 = 1/(1-rho_min); alpha0 = N0*v0; beta0 = N0*(1-v0).
 *   ab  device out [N][2];  v0  device in [N] initial estimates in [0,1].
 */
int32_t spo_tracker_init(float* ab, const float* v0, int64_t N,
                         const spo_params* params, void* stream);

/*
 * Prioritised sampling (Sec. 3.3, Eq. "sampling_coef"; Algorithm 1, the two
 * sampling steps): w(x) = sqrt(v(1-v)) + eps_explore with v = alpha/(alpha+beta)
 * (0.5 for an empty entry), then B distinct prompts drawn by weight.
 *
 * The draw is successive weighted sampling without replacement, made
 * reproducible bit for bit: weights are computed in fp32 by a fixed sequence of
 * individually rounded operations (nothing fused): n=a+b, t=a*b, x=t*(n*n);
 * for 2^-100 <= x <= 2^100 and a > 0 (any entry a tracker produces with both parameters
 * positive): y0 = the float with bits 0x5f3759df - (bits(x) >> 1), three Newton steps
 * y <- y*(1.5 - (0.5*x)*(y*y)), s = t*y (= sqrt(t)/n to 3e-7 relative); an empty entry has
 * s = 0.5, an entry with a or b zero s = 0, any other magnitude s = sqrt((a/n)*(b/n));
 * w = s+eps; q_i = floor(w_i * 2^32) (uint64); C_i = q_0+..+q_i; Wtot = C_{N-1};
 * for the k-th uniform U_k = floor(u_k * 2^32), t_k = floor(U_k*Wtot / 2^32),
 * candidate = first i with C_i > t_k; candidates are accepted in order k unless
 * already accepted, until B are accepted.
 *
 *   ab        device in  [N][2]
 *   uniforms  device in  [M] fp32 in [0,1); M >= B (M = 2B is ample for N >> B)
 *   out_ids   device out [B] int32, in acceptance order
 *   out_w     device out [N] fp32 weights, optional (the ids do not depend on whether it is given;
 *             given the same uniforms and these weights, the ids are fully determined by the
 *             integer arithmetic above)
 *   ws        device scratch, spo_workspace_bytes(SPO_WS_SAMPLE, ..., N, B, M) bytes (for tables of up
 *             to 2^20 prompts it includes 4 bytes per prompt: the call is organised for latency there,
 *             four short launches; larger tables are scanned at HBM speed)
 * Limits: 1 <= N < 2^31, 1 <= B <= M <= 2^20.
 * Device status: SPO_DEV_UNIFORMS_EXHAUSTED if fewer than B distinct candidates
 * (the tail of out_ids is then filled with -1), SPO_DEV_ZERO_TOTAL_WEIGHT,
 * SPO_DEV_NONFINITE for a negative or non-finite table entry (weight treated as 0).
 */
int32_t spo_sample_prompts(const float* ab, int64_t N, const float* uniforms, int32_t M, int32_t B,
                           int32_t* out_ids, float* out_w, void* ws, size_t ws_bytes,
                           const spo_params* params, int32_t* d_status, void* stream);

/*
 * Advantage with the pre-update baseline and global normalisation (Sec. 3.2;
 * Algorithm 1, "Compute raw advantage" and "Normalize advantages"):
 *   A_j = r_j - v(ids_j);  mu, sigma over the B values;  A~_j = (A_j - mu)/(sigma + norm_eps)
 * with sigma^2 = sum (A-mu)^2 / (B - norm_ddof).  Must be called BEFORE
 * spo_tracker_update for the same batch: the baseline is the table as it stood.
 *
 *   ids     device in  [B] int32 in [0,N)
 *   r       device in  [B] fp32 rewards
 *   a_raw   device out [B] fp32, optional
 *   a_norm  device out [B] fp32
 *   stats   device out [8] fp32 = (mu, sigma, B, M2 = sum (A-mu)^2, n_lo, n_hi, 0, 0), optional;
 *           n_lo / n_hi = how many raw advantages satisfy |A| <= near_zero_tau_lo / _hi (Sec. 4,
 *           signal efficiency; counts are exact up to 2^24).  (mu, M2, B) of several ranks merge
 *           exactly (pairwise: M2 = M2a + M2b + (mub-mua)^2 Ba Bb/(Ba+Bb)); the counts add.
 *   ws      device scratch, spo_workspace_bytes(SPO_WS_ADVANTAGES, ..., B, ...) bytes
 * An id outside [0,N) sets SPO_DEV_ID_OUT_OF_RANGE and contributes A = 0; a negative or non-finite
 * table entry sets SPO_DEV_NONFINITE and contributes A = 0 as well.
 */
int32_t spo_advantages(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                       float* a_raw, float* a_norm, float* stats, void* ws, size_t ws_bytes,
                       const spo_params* params, int32_t* d_status, void* stream);

/*
 * Second half of spo_advantages for a batch whose statistics were merged elsewhere (data-parallel
 * ranks each call spo_advantages for a_raw and stats, merge (mu, M2, B) on the host, then call
 * this): a_norm_j = (a_raw_j - mu) / (sigma + norm_eps)  (Sec. 3.2, global normalisation).
 * a_raw and a_norm may be the same buffer.
 */
int32_t spo_advantages_apply(const float* a_raw, int32_t B, float mu, float sigma, float* a_norm,
                             const spo_params* params, void* stream);

/*
 * spo_advantages with no scratch argument and no allocation anywhere.  (The paper has no
 * counterpart to this call: it computes exactly what spo_advantages computes and exists
 * only for the memory situation described here.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a
 * trainer whose framework has already handed every free byte of HBM to its own caching
 * allocator, a plug-in that is given input and output buffers but no allocator handle,
 * a step function that must never touch cudaMalloc because an allocation there would
 * synchronise the device or fail outright.  Such a caller cannot produce the `ws`
 * buffer that spo_advantages asks for large batches.
 *
 * Here the block partials of the two-pass path live in a fixed 32 KB array inside the
 * library's device image (each GPU that loads the library holds it until the process
 * exits).  Consequences the caller must know:
 *   - B may not exceed SPO_ADVANTAGES_STATIC_MAX_B; a larger B returns SPO_ERR_BAD_SHAPE
 *     and launches nothing.
 *   - The first call on a device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array.  Each call overwrites the part it later reads, so
 *     stale contents are harmless, but two calls whose kernels overlap on the GPU (two
 *     streams, two host threads) race on it: serialise them.
 *   - It calls no cudaMalloc/cudaFree or any allocating routine; inputs and outputs are
 *     still the caller's, with the same meaning, alignment and status bits as
 *     spo_advantages.  Always takes the two-kernel path, whatever B is.
 */
#define SPO_ADVANTAGES_STATIC_MAX_B  4194304
int32_t spo_advantages_static(const float* ab, int64_t N, const int32_t* ids, const float* r, int32_t B,
                              float* a_raw, float* a_norm, float* stats,
                              const spo_params* params, int32_t* d_status, void* stream);

/*
 * KL-adaptive tracker update (Sec. 3.1, the update equation; Algorithm 1, "Update tracker"):
 *   rho = clamp(2^(-D/D_half), rho_min, rho_max); alpha <- rho*alpha + r; beta <- rho*beta + (1-r)
 * at row ids[j], in place.  ids must be distinct within a call (what sampling
 * without replacement yields); duplicates race.
 *
 *   kl           device in: [B] per batch entry (kl_is_table = 0) or [N] per prompt,
 *                gathered by id (kl_is_table = 1)
 * A NaN divergence or reward sets SPO_DEV_NONFINITE and leaves the row untouched.
 */
int32_t spo_tracker_update(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                           int32_t kl_is_table, int32_t B,
                           const spo_params* params, int32_t* d_status, void* stream);

/*
 * spo_advantages and spo_tracker_update for the same batch in one pass over the table (Algorithm 1:
 * "Compute raw advantage", "Update tracker", "Normalize advantages"): every entry ids[j] is read
 * once, A_j = r_j - v(ids_j) is formed from the value as read (the pre-update baseline of Sec. 3.2),
 * the entry is updated in place from that same value (Sec. 3.1) and the batch statistics and
 * normalised advantages follow as in spo_advantages.  Results equal the two calls made in the
 * paper's order; the table entry crosses the memory system once per step instead of twice.
 * ids must be distinct (as for spo_tracker_update).  Arguments, scratch size (SPO_WS_ADVANTAGES)
 * and status bits as in the two calls; an element with a bad id, table entry or reward contributes
 * A = 0 and leaves its entry untouched, a NaN divergence leaves the entry untouched.
 */
int32_t spo_advantages_update(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                              int32_t kl_is_table, int32_t B, float* a_raw, float* a_norm, float* stats,
                              void* ws, size_t ws_bytes, const spo_params* params, int32_t* d_status, void* stream);

/*
 * Tracker update for batch SPO (appendix "Batch Extensions": every prompt rolled out G times per
 * batch against a shared baseline): like spo_tracker_update, but `ids` may repeat.  The entries
 * of one prompt are applied one after the other in batch order (the update equation of Sec. 3.1
 * composed G times), the same result as G successive calls; the outcome does not depend on
 * thread scheduling.  spo_advantages already accepts repeated ids (every copy reads the same
 * pre-update estimate), so a batch-SPO step is spo_advantages, then this call.
 *
 *   ws   device scratch, spo_workspace_bytes(SPO_WS_UPDATE_REPEATS, ..., B, ...) bytes
 * Limit: B <= 65536 (one thread block walks the rounds).  Status bits as spo_tracker_update.
 */
int32_t spo_tracker_update_repeats(float* ab, int64_t N, const int32_t* ids, const float* r, const float* kl,
                                   int32_t kl_is_table, int32_t B, void* ws, size_t ws_bytes,
                                   const spo_params* params, int32_t* d_status, void* stream);

/*
 * Policy loss forward (Sec. 3.2, the PPO-Clip objective with Clip-Higher bounds,
 * evaluated from final hidden states).  Per token row t:
 *   z = W h_t (never stored), lse = log sum_v exp z_v, logp = z[y_t] - lse,
 *   ratio = exp(logp - logp_old_t), a = a_norm[seq(t)],
 *   s_t = min(ratio*a, clip(ratio, 1-clip_lo, 1+clip_hi)*a),
 *   loss = - sum_t u_t s_t with token weights u_t that sum to one: u_t = mask_t / n_tok,
 *   n_tok = sum_t mask_t (SPO_AGG_TOKEN_MEAN), or u_t = mask_t / (S_act * n_seq(t)) with n_s the
 *   unmasked tokens of response s and S_act the responses that have any (SPO_AGG_SEQ_MEAN);
 *   loss = 0 if n_tok = 0.  With params->global_tokens / global_responses set, n_tok and S_act are
 *   those values (the whole data-parallel mini-batch) and `loss` is this rank's share: the ranks'
 *   losses and dW add up to the mini-batch's, dH rows are final;
 *   coef_t = d loss / d logp_t = -u_t * a * ratio * [gradient passes the clip].
 *   params->surrogate selects one of the other objectives (SPO_SUR_*, above) instead.
 *
 *   H           device in  [T][d], row-major, dtype as given (bf16: d % 64 == 0)
 *   W           device in  [V][d], row-major, same dtype
 *   y           device in  [T] int32 target token of each row
 *   logp_old    device in  [T] fp32
 *   mask        device in  [T] uint8, optional (NULL = all ones)
 *   cu_seqlens  device in  [S+1] int32, cu_seqlens[0] = 0, cu_seqlens[S] = T
 *   a_norm      device in  [S] fp32 normalised advantage per response
 *   loss        device out [1] fp32
 *   logp, lse, coef   device out [T] fp32 each
 *   seq_sums    device out [S][3] fp32 = per response (sum mask*logp,
 *               sum mask*(logp_old-logp), sum mask), optional
 *   entropy     device out [T] fp32, optional: entropy of each row's next-token distribution,
 *               -sum_v p log p = lse - sum_v p z, in nats (a diagnostic: Sec. 3.2 speaks of retaining
 *               policy entropy; it does not enter the objective).  Asking for it adds one multiply-add
 *               per logit to the contraction's epilogue; NULL costs nothing.
 *   ws          device scratch, spo_workspace_bytes(SPO_WS_LOSS_FWD, T, d, V, 0, S, 0) bytes
 *               (the B argument of that query carries the number of responses S)
 * A target outside [0,V) gives the row logp = -inf and coef = 0; it sets SPO_DEV_ID_OUT_OF_RANGE unless
 * the row is masked out (masked rows may carry an ignore-index target such as -100).
 */
int32_t spo_loss_fwd(const void* H, const void* W, int32_t dtype,
                     const int32_t* y, const float* logp_old, const uint8_t* mask,
                     const int32_t* cu_seqlens, const float* a_norm,
                     int64_t T, int32_t d, int32_t V, int32_t S,
                     float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                     void* ws, size_t ws_bytes,
                     const spo_params* params, int32_t* d_status, void* stream);

/*
 * Policy loss backward: with p = exp(z - lse) recomputed tile by tile,
 *   g[t,v] = grad_loss * coef_t * (1[v = y_t] - p[t,v]);  dH = g W;  dW (+)= g^T H.
 * lse and coef are the forward's outputs for the same H, W, y.
 *
 *   dH        device out [T][d], dtype dH_dtype (bf16 or fp32)
 *   dW        device out [V][d] fp32; overwritten, or added to when dW_accumulate != 0
 *   ws        device scratch, spo_workspace_bytes(SPO_WS_LOSS_BWD, T, d, V, ...) bytes.
 *             For bf16 it holds a bounded chunk of g (a few thousand token rows
 *             by V, bf16), never the whole [T][V] matrix.
 */
int32_t spo_loss_bwd(const void* H, const void* W, int32_t dtype, const int32_t* y,
                     const float* lse, const float* coef, float grad_loss,
                     int64_t T, int32_t d, int32_t V,
                     void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                     void* ws, size_t ws_bytes,
                     const spo_params* params, int32_t* d_status, void* stream);

/*
 * Policy loss forward and backward in one pass: every output of spo_loss_fwd (loss, logp, lse,
 * coef, seq_sums; Sec. 3.2, the PPO-Clip objective) and of spo_loss_bwd (dH, dW) for the same
 * inputs, with three LM-head-sized contractions per token instead of four.  The loss is the last
 * node of the training graph, so its upstream gradient (`grad_loss`, e.g. 1 or a loss scale) is
 * known before the forward runs; that is what lets the two halves share their logits.
 *
 * bf16: token rows are processed in chunks (the chunk of spo_loss_bwd).  A short launch first
 * contracts every row with the first 512 vocabulary rows; the largest of those logits plus 40 binary
 * orders is the row's reference exponent ref_t.  The logits of a chunk are then contracted once; the
 * epilogue sums e = 2^(z log2(e) - ref_t) over the row (no running maximum is needed: fp32 and bf16
 * keep their relative precision at any magnitude) and stores every e as bf16.  With l_t = sum_v e the
 * softmax is e / l_t, so lse_t = (ref_t + log2 l_t) ln 2 and the logit gradient factors as
 *   g[t,v] = rowscale_t (e[t,v] - l_t 1[v = y_t]),   rowscale_t = -grad_loss coef_t / l_t:
 * after the chunk's rows are finalised the one target entry per row is patched in the stored chunk,
 * dH = rowscale (e W) takes the factor in its epilogue and dW = e^T (rowscale H) reads a scaled bf16
 * copy of the chunk's rows of H; the stored chunk is never rewritten.
 * loss, logp, lse and coef never see the bf16 rounding of e; dH and dW carry it
 * (and dW the rounding of rowscale H) in place of spo_loss_bwd's own bf16 rounding of g.
 * Range: a row whose largest logit exceeds the largest of its first 512 by more than 100 nats
 * overflows the stored exponentials; such a row sets SPO_DEV_NONFINITE, gets lse = Inf, logp = -Inf,
 * coef = 0 and takes no part in the gradients (use the two calls for such inputs).
 * fp32: the two SIMT halves run back to back (nothing to share).
 *
 *   arguments   as in spo_loss_fwd and spo_loss_bwd; lse and coef are outputs here.
 *               SPO_SUR_GSPO with bf16 inputs: a response's ratio needs the log-probs of all its tokens,
 *               which may lie in later chunks, so the call runs the forward to the end and then the
 *               chunked backward (four contractions, the cost of the two calls).
 *   ws          device scratch, spo_workspace_bytes(SPO_WS_LOSS_FWD_BWD, T, d, V, 0, S, 0) bytes:
 *               two chunk buffers (a few thousand token rows by V each, bf16), scaled bf16 copies of those
 *               chunks' rows of H, 36 bytes per token row and the forward's partials
 * Status bits as spo_loss_fwd.
 */
int32_t spo_loss_fwd_bwd(const void* H, const void* W, int32_t dtype,
                         const int32_t* y, const float* logp_old, const uint8_t* mask,
                         const int32_t* cu_seqlens, const float* a_norm,
                         int64_t T, int32_t d, int32_t V, int32_t S, float grad_loss,
                         float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                         void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                         void* ws, size_t ws_bytes,
                         const spo_params* params, int32_t* d_status, void* stream);

/*
 * spo_loss_fwd_bwd for data-parallel ranks (Algorithm 1's mini-batch update spread over several GPUs:
 * every rank holds part of the responses, W is replicated, and the ranks' dW must be summed).  dW is
 * only final once its last contraction has run; this variant cuts that last launch into slabs of
 * vocabulary rows and records a CUDA event behind each, so that the caller can start reducing slab k
 * over the ranks on another stream (wait for events[k], then all-reduce rows row_begin[k] ..
 * row_begin[k+1]-1 of dW) while slab k+1 is still being contracted; only the last slab's reduction is
 * left exposed.  Results are those of spo_loss_fwd_bwd, bit for bit.
 *
 *   spo_dw_slab_rows   host only: writes row_begin[0..n] (row_begin[0] = 0, row_begin[n] = V) for a
 *                      request of n_wanted slabs (1 .. SPO_MAX_DW_SLABS) and returns n <= n_wanted
 *                      (slabs hold whole rounds of row tiles), or a negative status.
 *   events             host array of n_wanted cudaEvent_t (created by the caller, e.g. with timing
 *                      disabled); events[0..n) are recorded on `stream`.  Inputs for which the last
 *                      contraction is not cut (fp32, SPO_SUR_GSPO, T = 0) record them all at the end.
 * All other arguments as in spo_loss_fwd_bwd.  The library creates, waits on and destroys nothing.
 */
#define SPO_MAX_DW_SLABS 64
#define SPO_MAX_DW_SHARDS 16
int32_t spo_dw_slab_rows(int32_t V, int32_t d, int32_t n_wanted, int64_t* row_begin /* host, [n_wanted+1] */);
int32_t spo_loss_fwd_bwd_slabs(const void* H, const void* W, int32_t dtype,
                               const int32_t* y, const float* logp_old, const uint8_t* mask,
                               const int32_t* cu_seqlens, const float* a_norm,
                               int64_t T, int32_t d, int32_t V, int32_t S, float grad_loss,
                               float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                               void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                               void* ws, size_t ws_bytes,
                               const spo_params* params, int32_t* d_status, void* stream,
                               int32_t n_wanted, void* const* events /* host, [n_wanted] */);

/*
 * spo_loss_fwd_bwd with the reduce-scatter of dW fused into its last contraction (data-parallel ranks whose
 * optimizer is sharded over the vocabulary rows of W; Algorithm 1's mini-batch update spread over GPUs).
 * The vocabulary rows are cut into n_shards equal shards of rows_per_shard rows (the last may be shorter);
 * shard k lives in the memory of rank k (shard[k]: fp32 [rows_per_shard][d]; for k != own rank a pointer to
 * PEER device memory mapped into this process).  The epilogue of the call's LAST dW contraction adds each
 * finished tile of dW (the sum over all chunks of this rank's tokens) straight into the shard that owns its
 * rows with vector store-reductions (`red.global.add` — over NVLink for a peer's shard; nothing is loaded
 * from a peer and nothing waits on a peer), so the exchange overlaps the contraction tile by tile and no
 * collective library call touches dW.  After every rank's call has completed (a barrier the caller
 * provides: stream synchronise + process-group barrier), shard[own rank] holds the mini-batch's dW rows.
 *   - Every shard must be zeroed by its owner, and that zeroing visible to all ranks, before any rank's call.
 *   - dW is scratch here (it ends up holding the partial sums of the chunks before the last); dW_accumulate
 *     still means "dW already holds a term to include".
 *   - Summation order across ranks is not fixed: results are reproducible up to fp32 addition order.
 *   - Inputs for which the last contraction is not this kernel (fp32, SPO_SUR_GSPO, T = 0) are followed by
 *     a plain kernel that adds dW into the shards the same way.
 * All other arguments and outputs as spo_loss_fwd_bwd.
 */
typedef struct spo_dw_shards {
  int32_t n_shards;                       /* 1 .. SPO_MAX_DW_SHARDS */
  int64_t rows_per_shard;                 /* n_shards * rows_per_shard >= V */
  float*  shard[SPO_MAX_DW_SHARDS];       /* device pointers (own or peer memory), 16-byte aligned */
} spo_dw_shards;
int32_t spo_loss_fwd_bwd_scatter(const void* H, const void* W, int32_t dtype,
                                 const int32_t* y, const float* logp_old, const uint8_t* mask,
                                 const int32_t* cu_seqlens, const float* a_norm,
                                 int64_t T, int32_t d, int32_t V, int32_t S, float grad_loss,
                                 float* loss, float* logp, float* lse, float* coef, float* seq_sums, float* entropy,
                                 void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                                 void* ws, size_t ws_bytes,
                                 const spo_params* params, int32_t* d_status, void* stream,
                                 const spo_dw_shards* shards /* host */);

/*
 * Diagnostic (no counterpart in the paper): runs the kernels' bounded mbarrier wait on a barrier
 * that nothing ever signals, with a limit of `limit_us` microseconds (1 .. 1 000 000).  A healthy
 * build sets SPO_DEV_TIMEOUT in *d_status, writes 1 to *reached_end (device int32, optional) and the
 * kernel returns normally; the context stays usable.  It shows that a stuck pipeline stage ends in a
 * status bit, not in a hang.  One tiny launch on `stream`.
 */
int32_t spo_selftest_bounded_wait(uint32_t limit_us, int32_t* reached_end, int32_t* d_status, void* stream);

/*
 * Backward over the rows that carry gradient only.  A token whose coef is zero -- masked out of the
 * loss (e.g. tool output inside a response) or clipped on the side that stops the gradient --
 * contributes nothing to dH or dW, so the three contractions of spo_loss_bwd can run on the other
 * rows alone; their cost falls in proportion.  Two calls, because the number of such rows has to
 * reach the host to size the second one (the library itself never synchronises):
 *
 *   spo_loss_active_rows: rows[0..count) = ascending indices t with coef[t] != 0, *d_count = count.
 *     rows    device out [T] int32;  d_count  device out [1] int32
 *     ws      device scratch, spo_workspace_bytes(SPO_WS_ACTIVE_ROWS, T, ...) bytes
 *   (the caller reads *d_count back, e.g. after a stream synchronise)
 *   spo_loss_bwd_rows: same results as spo_loss_bwd(H, W, ..., T, ...): dH[t] for the listed rows,
 *     zeros elsewhere; dW as in spo_loss_bwd.  bf16 H / W only.
 *     rows    device in [T_act] from the first call;  T_act  host value of *d_count
 *     ws      device scratch, spo_workspace_bytes(SPO_WS_LOSS_BWD_ROWS, T_act, d, V, ...) bytes
 *             (holds the gathered rows of H and dH besides the chunk buffer)
 */
int32_t spo_loss_active_rows(const float* coef, int64_t T, int32_t* rows, int32_t* d_count,
                             void* ws, size_t ws_bytes, void* stream);
int32_t spo_loss_bwd_rows(const void* H, const void* W, int32_t dtype, const int32_t* y,
                          const float* lse, const float* coef, float grad_loss,
                          int64_t T, int32_t d, int32_t V, const int32_t* rows, int64_t T_act,
                          void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                          void* ws, size_t ws_bytes, const spo_params* params, int32_t* d_status, void* stream);

/*
 * One-pass loss over the unmasked rows only.  In tool-integrated reasoning the tokens a tool wrote
 * sit inside the response but carry no loss (mask = 0): they enter neither the objective of Sec. 3.2
 * nor its gradients, so none of the three contractions has to see them and the cost of the call
 * falls in proportion to the masked share.  Two calls, because the number of unmasked rows has to
 * reach the host to size the second one (the library itself never synchronises):
 *
 *   spo_loss_mask_rows: rows[0..count) = ascending indices t with mask[t] != 0, *d_count = count.
 *     mask    device in [T] uint8;  rows  device out [T] int32;  d_count  device out [1] int32
 *     ws      device scratch, spo_workspace_bytes(SPO_WS_ACTIVE_ROWS, T, ...) bytes
 *   (the caller reads *d_count back, e.g. after a stream synchronise)
 *   spo_loss_fwd_bwd_rows: what spo_loss_fwd_bwd(H, W, ..., mask, ...) gives for loss, seq_sums,
 *     dW, and for logp / lse / coef / dH at the listed rows; at all other rows logp, lse, coef and
 *     dH are ZERO (spo_loss_fwd_bwd reports logp and lse of masked rows too; use it if you need them).
 *     The listed rows of H, y and logp_old are gathered into a packed batch of T_act rows whose
 *     sequence boundaries are the counts of listed rows per response, and the one-pass path runs on
 *     that batch.  bf16 H / W only.  Every listed row counts as unmasked.
 *     rows    device in [T_act] from the first call;  T_act  host value of *d_count
 *     ws      device scratch, spo_workspace_bytes(SPO_WS_LOSS_FWD_BWD_ROWS, T_act, d, V, 0, S, 0) bytes
 *             (holds the gathered rows of H and dH besides the one-pass scratch)
 */
int32_t spo_loss_mask_rows(const uint8_t* mask, int64_t T, int32_t* rows, int32_t* d_count,
                           void* ws, size_t ws_bytes, void* stream);
int32_t spo_loss_fwd_bwd_rows(const void* H, const void* W, int32_t dtype,
                              const int32_t* y, const float* logp_old,
                              const int32_t* cu_seqlens, const float* a_norm,
                              int64_t T, int32_t d, int32_t V, int32_t S,
                              const int32_t* rows, int64_t T_act, float grad_loss,
                              float* loss, float* logp, float* lse, float* coef, float* seq_sums,
                              void* dH, int32_t dH_dtype, float* dW, int32_t dW_accumulate,
                              void* ws, size_t ws_bytes,
                              const spo_params* params, int32_t* d_status, void* stream);

/*
 * Diagnostics of one policy update over the unmasked tokens, from the forward's logp (no counterpart
 * in the paper's equations; these are the quantities its training curves are read by, and none
 * enters the objective).  out (device, [8] fp32):
 *   [0] n_tok   [1] mean importance ratio   [2] share of tokens whose gradient the clip stops
 *   (ratio beyond the bound that matters for the sign of their advantage; zero advantage: not stopped)
 *   [3] mean of logp_old - logp (sampled estimate of KL(old || new))   [4] mean of ratio - 1 - log ratio
 *   (a non-negative estimate of the same)   [5] largest ratio   [6] smallest ratio
 *   [7] share of tokens whose ratio lies outside [1-clip_lo, 1+clip_hi].  All zeros when n_tok = 0.
 * One block, fixed reduction order; a few tens of microseconds at 250 k tokens.
 */
int32_t spo_loss_stats(const float* logp, const float* logp_old, const uint8_t* mask,
                       const int32_t* cu_seqlens, const float* a_norm, int64_t T, int32_t S,
                       float* out, const spo_params* params, void* stream);

/* Scratch size in bytes for one call of the selected entry point (host only, no CUDA call
 * except a device-property query).  Arguments that the selected call does not use are ignored. */
size_t spo_workspace_bytes(int32_t which, int64_t T, int32_t d, int32_t V,
                           int64_t N, int32_t B, int32_t M);

const char* spo_status_string(int32_t status);
int32_t     spo_last_cuda_error(void);   /* cudaError_t of the last SPO_ERR_CUDA on this thread */
int32_t     spo_version(void);

#ifdef __cplusplus
}
#endif
#endif  /* SPO_H_ */
