/*
 * arrol.h - C ABI of the B200 (sm_100a) prune-and-rebatch library for online rollout pruning.
 *
 * The four compute calls follow the method's problem statement:
 *   arrol_score_partial  quality head on the policy's hidden state at the detection length, score -> [0,1]
 *                        -> binned posterior                      (Section 4.2; Appendix A.4)
 *   arrol_select         per-group correctness-balancing selection, exactly K of G kept
 *                                                                  (Section 4.1, Theorem 1's rule)
 *   arrol_compact        filter pruned rollouts and re-batch the survivors, with group-relative
 *                        advantages on the survivors               (Section 4.3 (ii); Algorithm 1; Section 3)
 *   arrol_token_logprob  selected-token log-probability of every survivor token from the lm_head,
 *                        vocabulary-chunked, logits never stored   (Section 3; Algorithm 1 "log-probs on R'")
 *
 * Conventions for every call unless a parameter says otherwise:
 *   - Pointers are DEVICE pointers owned by the caller.  The library keeps no reference to them once the
 *     call's work has completed on `stream`, never frees them, and allocates nothing after arrol_create.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls are asynchronous:
 *     the return value reports argument validation and launch errors only.  Conditions found on the device
 *     (destination too small, target id outside the vocabulary, a bounded wait that ran out) are recorded in
 *     a status word and read with arrol_poll_status; the device never traps.
 *   - Return value: ARROL_OK (0) or a negative arrol_status.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x arrol_create fails.
 */
#ifndef ARROL_H_
#define ARROL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct arrol_ctx arrol_ctx; /* opaque: device id, SM count, status word, small scratch */

typedef enum { ARROL_F32 = 0, ARROL_BF16 = 1 } arrol_dtype;

typedef enum {
    ARROL_OK = 0,
    ARROL_ERR_INVALID_ARG = -1,   /* NULL where data is required, negative size, misaligned pointer/stride */
    ARROL_ERR_UNSUPPORTED = -2,   /* valid but outside the supported range (G > 32, d not a multiple of 8, ...) */
    ARROL_ERR_WORKSPACE = -3,     /* workspace missing or smaller than arrol_token_logprob_workspace says */
    ARROL_ERR_CAPACITY = -4,      /* device: survivors need more than dst_capacity_tokens rows */
    ARROL_ERR_CUDA = -5,          /* a CUDA runtime/driver call failed */
    ARROL_ERR_DEVICE_STATUS = -6, /* device: target id >= V, or an internal bounded wait expired */
    ARROL_ERR_NO_DEVICE = -7      /* no usable sm_100 device */
} arrol_status;

/* Device status bits accumulated in the context's status word (see arrol_poll_status). */
#define ARROL_DEV_CAPACITY 1u      /* arrol_compact: T > dst_capacity_tokens, nothing was gathered */
#define ARROL_DEV_BAD_TARGET 2u    /* arrol_token_logprob: a target id >= V (its logp is set to 0) */
#define ARROL_DEV_WAIT_EXPIRED 4u  /* arrol_token_logprob: a pipeline wait hit its iteration limit */
#define ARROL_DEV_BAD_STATE 8u     /* arrol_calib_update: the state's header does not match (B, cap); state untouched */
#define ARROL_DEV_BAD_INDEX 16u    /* a source row outside the bound set with arrol_set_source_rows; access skipped */

int arrol_version(void);                    /* major*10000 + minor*100 + patch */
const char* arrol_status_string(int status); /* static string, never NULL */

/* Creates a context on CUDA device `device` (made current for the calling thread during the call).
 * Allocates the context's device status word, a 16 MB scratch buffer and a 64 MB row-packing buffer (MLP head),
 * 65 MB of pinned host memory, a second stream and a few events (used by arrol_prune_rebatch_host); nothing is
 * allocated later.  Calls that use the context's buffers (MLP-head scoring, the policy loss, the head training
 * step) must be ordered on the device with respect to one another, e.g. by issuing them on one stream. */
int arrol_create(arrol_ctx** out, int device);
int arrol_destroy(arrol_ctx* ctx);

/* Waits for `stream`, copies the device status word to *dev_status_bits (host pointer, may be NULL),
 * clears it, and returns ARROL_OK if it was 0, else ARROL_ERR_CAPACITY / ARROL_ERR_DEVICE_STATUS.
 * Order it after all work on the context: the word is read and then cleared on `stream`, so a bit that a kernel on
 * another stream sets between the two is lost. */
int arrol_poll_status(arrol_ctx* ctx, void* stream, uint32_t* dev_status_bits);

/* ---- Binned posterior table: host helpers (Appendix A.4).  All pointers are HOST pointers. ----------
 * arrol_calib_counts: c_b^+ / c_b^- = number of historical positive / negative rollouts whose normalised
 *   score s' falls in bin b(s') = min(B-1, floor(B s')).  sprime [n] in [0,1], y [n] in {0,1}.
 * arrol_build_q_lut: Laplace-smoothed likelihoods P(b|Y) = (c_b + alpha) / (sum c + alpha B) and the Bayes
 *   posterior q_b = pi P(b|1) / (pi P(b|1) + (1-pi) P(b|0)), pi = n+/(n+ + n-) (0.5 when both are empty),
 *   computed in double and rounded once to float.  q_lut [B] is what arrol_score_partial consumes. */
int arrol_calib_counts(const double* sprime, const uint8_t* y, int64_t n, int B, int64_t* cpos, int64_t* cneg);
int arrol_build_q_lut(const int64_t* cpos, const int64_t* cneg, int B, double alpha, float* q_lut);

/* ---- Quality head (Section 4.2 "Quality Score Prediction"; Appendix A.4) --------------------------- */
typedef struct arrol_head {
    int32_t d;       /* hidden width; multiple of 8                                                    */
    int32_t h;       /* 0: linear head d -> 1.  > 0: d -> h -> 1 with exact (erf) GELU; multiple of 4  */
    int32_t dtype;   /* arrol_dtype of hidden, W1, b1, w2, b2                                          */
    int32_t reserved;
    const void* W1;  /* device [h, d] row-major; [d] when h == 0                                        */
    const void* b1;  /* device [h] or NULL (= 0); when h == 0: [1] bias or NULL                          */
    const void* w2;  /* device [h]; ignored when h == 0                                                 */
    const void* b2;  /* device [1] or NULL; ignored when h == 0                                         */
} arrol_head;

typedef struct arrol_calib {
    int32_t B;          /* number of bins (128 in the paper); ignored when q_lut == NULL                 */
    int32_t reserved;
    const float* q_lut; /* device [B] posterior per bin, or NULL: q = sigmoid(score)                     */
} arrol_calib;

/* For each rollout i < N: x = row row_index[i] (row i when row_index is NULL) of `hidden`
 * ([rows, row_stride_elems] row-major, head->dtype, 16-byte aligned rows);
 *   score[i] = head(x);  prob[i] = s' = 1 / (1 + exp(-score[i]));
 *   bin[i] = min(B-1, floor(B s'));  q[i] = q_lut[bin[i]]   (q[i] = s' when there is no table).
 * Outputs: score, prob, q float [N] (required); bin int32 [N] or NULL.  fp32 accumulation.
 * A bf16 MLP head runs its first layer on the tensor cores (bf16 products, fp32 accumulation); rows picked by
 * row_index are first packed into the context's buffer.
 * row_index holds int64 row numbers; it must stay valid until the work completes.
 * Errors: INVALID_ARG for NULL/negative/misaligned arguments, UNSUPPORTED for d % 8 != 0, h % 4 != 0,
 * h > 4096, or N larger than the context scratch allows for the MLP head (65536). N == 0 is a no-op. */
int arrol_score_partial(arrol_ctx* ctx, const void* hidden, int64_t row_stride_elems, const int64_t* row_index,
                        int32_t N, const arrol_head* head, const arrol_calib* calib, float* score, float* prob,
                        int32_t* bin, float* q, void* stream);

/* ---- Per-group selection (Section 4.1; Theorem 1: j^ = argmin_j |mu_{-j} - rho|) -------------------
 * q [P*G] float, group-major (rollouts of prompt p are q[p*G .. p*G+G-1]).  For each group, while more than
 * K members remain (n of them, sum Sigma): remove the member minimising |q_j - (Sigma - rho (n-1))|, which
 * is the member whose removal leaves the group mean closest to rho; of equal candidates the one with the
 * highest index is removed, so the lower index survives.  Keys are evaluated in double, one rounding per
 * operation, so the result is reproducible bit for bit.  keep [P*G] uint8 receives 1 (kept) / 0 (pruned).
 * mode must be 0.  Supported: 1 <= K <= G <= 32.  q must be finite.  P == 0 is a no-op. */
int arrol_select(arrol_ctx* ctx, const float* q, int32_t P, int32_t G, int32_t K, double rho, int32_t mode,
                 uint8_t* keep, void* stream);

/* ---- Filter + re-batch with advantages (Section 4.3 (ii); Algorithm 1; Section 3) -------------------
 * Inputs:  keep [N] uint8; lengths [N] int32 (tokens of rollout i, >= 0); src_tok_off [N] int64 (first source
 *   row of rollout i); src_tokens int32 [source rows] or NULL; src_rows [source rows, row_bytes] or NULL
 *   (opaque payload per token, e.g. a hidden-state row; row_bytes a multiple of 16, base 16-byte aligned);
 *   rewards [N] float; G = group size (N % G == 0).
 * Outputs: survivor_idx [<= N] int32, ascending original indices of kept rollouts (S of them);
 *   cu_seqlens [<= N+1] int64, exclusive prefix sum of the survivors' lengths (cu_seqlens[S] = T);
 *   d_num [2] int64 = {S, T};  adv [<= N] float, A = (R - mean) / (std + eps) over the kept rollouts of the
 *   survivor's group, std with divisor (n - ddof) (0 when n - ddof <= 0; exactly 0 when all kept rewards of
 *   the group are equal);  dst_tokens [cap] / dst_rows [cap, row_bytes]: row cu_seqlens[s] + t receives source
 *   row src_tok_off[survivor_idx[s]] + t;  tok_adv [cap] float or NULL: adv of the token's rollout;
 *   tok_seq [cap] int32 or NULL: survivor ordinal s of the token.   cap = dst_capacity_tokens.
 * If T > dst_capacity_tokens the scan outputs (survivor_idx, cu_seqlens, d_num, adv) are still written, nothing
 * is gathered, and ARROL_DEV_CAPACITY is recorded.  T never leaves the device: no host synchronisation.
 * dst_* may be NULL when the matching src_* is NULL. */
int arrol_compact(arrol_ctx* ctx, const uint8_t* keep, const int32_t* lengths, const int64_t* src_tok_off,
                  int32_t N, int32_t G, const int32_t* src_tokens, const void* src_rows, int32_t row_bytes,
                  const float* rewards, float eps, int32_t ddof, int64_t dst_capacity_tokens, int32_t* dst_tokens,
                  void* dst_rows, int64_t* cu_seqlens, int32_t* survivor_idx, float* adv, float* tok_adv,
                  int32_t* tok_seq, int64_t* d_num, void* stream);

/* ---- Selected-token log-probability (Section 3: log pi_theta(o_t | o_<t); Algorithm 1) -------------
 * hidden [T_max, d] bf16 row-major; W_vocab [V, d] bf16 row-major (the layout of an nn.Linear / tied
 * embedding weight); targets [T_max] int32.  T = min(*d_T, T_max) when d_T != NULL (device int64), else T_max.
 * For t < T:  z_v = inv_temperature * sum_k hidden[t,k] W_vocab[v,k]  (bf16 products, fp32 accumulation on
 * the tensor cores);  lse[t] = log sum_v exp z_v (running max / sum over vocabulary chunks, fp32);
 * logp[t] = z_{targets[t]} - lse[t].  targets[t] < 0 marks an ignored position: logp[t] = 0.  A target >= V sets
 * logp[t] = 0 and records ARROL_DEV_BAD_TARGET.  Rows t >= T of the outputs are not written.
 * logp float [T_max]; lse float [T_max] or NULL.  Both pointers 16-byte aligned; d % 8 == 0; inv_temperature > 0.
 * workspace: device scratch of at least arrol_token_logprob_workspace(ctx, T_max, d, V) bytes, 256-byte
 * aligned (holds per-split running maxima / sums when the vocabulary is split across thread blocks); its
 * contents need not be initialised and are undefined afterwards.  The size is monotone in T_max: a workspace sized
 * for T_max also serves calls on fewer tokens with the same d and V. */
size_t arrol_token_logprob_workspace(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V);
/* Number of vocabulary splits a launch on T_max tokens uses (1 = every block walks the whole vocabulary). */
int32_t arrol_token_logprob_splits(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V);
/* Form of the kernel for these sizes: 2 = pairs of thread blocks on 256-row token tiles (tcgen05 cta_group::2), 1 = one
 * block per 128-row tile.  Pairs are used wherever they need no more vocabulary splits than single blocks (hidden
 * widths up to about 2,700 on a 148-SM part); see ARROL_HOOK_LOGPROB_PAIR.  0 for invalid arguments. */
int32_t arrol_token_logprob_form(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V);
int arrol_token_logprob(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                        int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                        float* logp, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* ---- Selected-token log-probability straight from the pre-prune buffer (Section 4.3 (ii): the frontend "filters
 * out pruned rollouts and re-batches the surviving ones to compute log-probabilities"; Algorithm 1) -------------
 * arrol_token_logprob on the survivors WITHOUT a packed copy of their hidden rows: packed token t of survivor s
 * (cu_seqlens[s] <= t < cu_seqlens[s+1]) is row src_tok_off[survivor_idx[s]] + (t - cu_seqlens[s]) of src_rows, and
 * the kernel's loads follow that mapping, so arrol_compact can be called without the hidden-row plane
 * (src_rows = dst_rows = NULL) and [T, d] never exists in memory.
 *   src_rows [source_rows, d] bf16 row-major, 16-byte aligned; source_rows <= 2^31 - 129;
 *   cu_seqlens [>= S_max + 1] int64, survivor_idx [>= S_max] int32, d_num [2] int64 = {S, T}: the outputs of
 *   arrol_compact (S is clamped to S_max, T to T_max);  src_tok_off [N] int64: the array given to arrol_compact;
 *   targets [T_max] int32 in packed order (arrol_compact's dst_tokens);  logp, lse, d, V, inv_temperature as in
 *   arrol_token_logprob.  workspace: arrol_token_logprob_gathered_workspace(ctx, S_max, T_max, d, V) bytes, 256-byte
 *   aligned: the split records of arrol_token_logprob plus S_max * 128 * d * 2 bytes, into which a first small
 *   kernel copies the token tiles that cross a survivor boundary (at most one per survivor); every other tile is
 *   read in place.
 * Results equal arrol_token_logprob on the packed rows bit for bit.  Source rows are trusted to lie inside
 * [0, source_rows) (see arrol_set_source_rows for arrol_compact's check of the same offsets). */
size_t arrol_token_logprob_gathered_workspace(arrol_ctx* ctx, int32_t S_max, int64_t T_max, int32_t d, int32_t V);
int arrol_token_logprob_gathered(arrol_ctx* ctx, const void* src_rows, int64_t source_rows, const void* W_vocab,
                                 const int32_t* targets, const int64_t* cu_seqlens, const int32_t* survivor_idx,
                                 const int64_t* src_tok_off, const int64_t* d_num, int32_t S_max, int64_t T_max,
                                 int32_t d, int32_t V, float inv_temperature, float* logp, float* lse,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* ---- Prune step in one call (Algorithm 1: quality check at the detection length, filter, re-batch) ----------
 * arrol_score_partial -> arrol_select -> arrol_compact issued back to back on `stream` with N = P * G; every field
 * has the meaning, layout and nullability of the argument of the same name in those calls.  Asynchronous.
 * The kernels are launched with programmatic stream serialization (each sets up while its predecessor finishes and
 * reads global memory only after the predecessor has completed).  The call allocates nothing and never
 * synchronises, so it may be captured into a CUDA graph and replayed. */
typedef struct arrol_prune_step_args {
    /* scoring */
    const void* hidden;
    int64_t row_stride_elems;
    const int64_t* row_index;
    arrol_head head;
    arrol_calib calib;
    float *score, *prob, *q;
    int32_t* bin;
    /* selection */
    int32_t P, G, K, ddof;
    double rho;
    uint8_t* keep;
    /* compaction */
    const int32_t* lengths;
    const int64_t* src_tok_off;
    const int32_t* src_tokens;
    const void* src_rows;
    const float* rewards;
    int64_t dst_capacity_tokens;
    int32_t row_bytes;
    float eps;
    int32_t* dst_tokens;
    void* dst_rows;
    int64_t* cu_seqlens;
    int32_t* survivor_idx;
    float* adv;
    float* tok_adv;
    int32_t* tok_seq;
    int64_t* d_num;
} arrol_prune_step_args;
int arrol_prune_step(arrol_ctx* ctx, const arrol_prune_step_args* args, void* stream);

/* ---- Online calibrator and the deployed stochastic rule (Appendix A.4; Algorithm 1, backend) ----------
 * The calibrator state lives in ONE caller-provided device buffer of arrol_calib_state_bytes(B, cap) bytes
 * (16-byte aligned): two first-in-first-out rings of `cap` bin indices (positive / negative rollouts), their
 * histogram counts c_b^+ / c_b^-, the posterior table q_lut [B] and the bias delta.  B <= 1024.
 *
 * arrol_calib_init: empty rings, zero counts, q_lut = 0.5, delta = 0.
 * arrol_calib_update: pushes the rollouts i < N with mask[i] != 0 (all when mask is NULL) in index order: rollout i
 *   goes to the positive ring if rewards[i] > 0.5, else to the negative ring, as bin index bin[i] (the output of
 *   arrol_score_partial); a full ring drops its oldest entry.  Then rebuilds
 *     q_b = pi P(b|1) / (pi P(b|1) + (1-pi) P(b|0)),  P(b|Y) = (c_b + alpha) / (sum c + alpha B),  pi = n+/(n+ + n-)
 *   and solves delta by 64 bisection steps on [-(1+lambda), 1+lambda] so that
 *     sum_b (c_b^+ + c_b^-) clip(kappa + delta + lambda (rho - q_b), p_min, p_max) / (n+ + n-) = kappa
 *   (delta = 0 while both rings are empty).  fp64, one rounding per operation, fixed order: reproducible bit for bit.
 *   (B, cap) must be the pair the state was initialised with: otherwise the state is left untouched and
 *   ARROL_DEV_BAD_STATE is recorded.
 * arrol_calib_q_lut / arrol_calib_delta: device addresses of the table and of delta inside the state (pointer
 *   arithmetic on the host; no device access), to be passed to arrol_score_partial / arrol_select_stochastic.
 * arrol_calib_layout: byte offsets {c+, c-, q_lut, ring+, ring-, total} inside the state, for inspection.
 * arrol_select_stochastic: p_i = clip(kappa + delta + lambda (rho - q_i), p_min, p_max) in fp64;
 *   keep[i] = (u[i] < p_i), u [N] float uniforms in [0,1) supplied by the caller; rollouts with eligible[i] == 0
 *   (ended before the detection length, never evaluated) are kept with p = 1.  delta is read from d_delta
 *   (device) when it is not NULL, else the host value `delta` is used.  p_out [N] float or NULL. */
typedef struct arrol_survival {
    double kappa;   /* target keep rate            */
    double lambda;  /* strength of the correction  */
    double rho;     /* target positive ratio       */
    double p_min, p_max;
} arrol_survival;

size_t arrol_calib_state_bytes(int32_t B, int64_t cap);
int arrol_calib_layout(int32_t B, int64_t cap, size_t* offsets6 /* host [6] */);
int arrol_calib_init(arrol_ctx* ctx, void* state, size_t state_bytes, int32_t B, int64_t cap, double alpha,
                     void* stream);
int arrol_calib_update(arrol_ctx* ctx, void* state, int32_t B, int64_t cap, const int32_t* bin, const float* rewards,
                       const uint8_t* mask, int32_t N, const arrol_survival* params, void* stream);
const float* arrol_calib_q_lut(void* state, int32_t B, int64_t cap);
const double* arrol_calib_delta(void* state);
int arrol_select_stochastic(arrol_ctx* ctx, const float* q, const float* u, const uint8_t* eligible, int64_t N,
                            const arrol_survival* params, const double* d_delta, double delta, uint8_t* keep,
                            float* p_out, void* stream);

/* ---- Policy update on the survivors (Section 3: clipped objective; Algorithm 1 "main RL loss", "Backprop") ----
 * arrol_policy_loss: for every packed survivor token t < T (T, S read from d_num = {S, T}, device):
 *     r = exp(logp[t] - logp_old[t]),  term = min(r A, clip(r, 1 - eps_low, 1 + eps_high) A),  A = tok_adv[t];
 *     loss = - sum_t w_t term_t  (+ beta sum_t w_t (exp(ref - logp) - (ref - logp) - 1) when logp_ref != NULL);
 *     agg_mode 0 (GRPO): w_t = 1 / (S * length of the token's rollout), rollout = tok_seq[t], lengths from cu_seqlens;
 *     agg_mode 1 (DAPO): w_t = 1 / T.
 *   Outputs: grad_logp [T_max] float = d loss / d logp (d term / d logp = r A when r A <= clip(r) A, else 0);
 *   loss: device double [1].  fp32 per token, fp64 fixed-order reduction.  Uses the context scratch: calls on one
 *   context must be issued on one stream at a time.
 * arrol_lm_head_backward: given grad_logp [T_max] and lse [T_max] (from arrol_token_logprob on the same inputs),
 *     dz_{t,v} = grad_logp[t] inv_temperature ([v = targets[t]] - exp(z_{t,v} - lse[t])),  z recomputed on the tensor
 *     cores;  dH [T_max, d] float = dz W_vocab (rows t >= T are zero or left untouched);  dW [V, d] float = dz^T hidden
 *     (overwritten).  Positions with targets[t] < 0 or >= V carry no gradient.  dz is rounded to bf16 before the two
 *     contractions.  hidden, W_vocab, targets, T_max, d_T, d, V as in arrol_token_logprob; dH, dW 16-byte aligned.
 *   hidden rows t in [T, T_max) are never read by the contractions (the last, partly live block of rows goes
 *   through a zero-padded copy), so they may hold anything.
 *   workspace: arrol_lm_head_backward_workspace(ctx, T_max, d, V) bytes, 256-byte aligned (one chunk of 9,472 tokens
 *   of dz in bf16 and one 64-row block of hidden): 9472 * 2 * V + 128 * d bytes (V rounded up to 8). */
int arrol_policy_loss(arrol_ctx* ctx, const float* logp, const float* logp_old, const float* logp_ref,
                      const float* tok_adv, const int32_t* tok_seq, const int64_t* cu_seqlens, const int64_t* d_num,
                      int64_t T_max, float eps_low, float eps_high, float beta, int32_t agg_mode, float* grad_logp,
                      double* loss, void* stream);
size_t arrol_lm_head_backward_workspace(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V);
int arrol_lm_head_backward(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                           const float* grad_logp, const float* lse, int64_t T_max, const int64_t* d_T, int32_t d,
                           int32_t V, float inv_temperature, float* dH, float* dW, void* workspace,
                           size_t workspace_bytes, void* stream);

/* ---- Trace confidence (Section 3 "Trace Confidence") ---------------------------------------------------------
 * arrol_token_logprob_conf: arrol_token_logprob with one more output from the same launch, the token confidence
 *     token_conf[t] = H_t = - sum_{v < V} log P_t(v) = V lse[t] - sum_v z_{t,v}     (float [T_max], rows t < T)
 *   accumulated in the same epilogue (one more add per logit).  All other arguments as arrol_token_logprob.
 * arrol_trace_confidence: per packed trace s < S (S read from d_num = {S, T}; bounds from cu_seqlens):
 *     mode 0: trace_conf[s] = mean of token_conf over the trace;
 *     mode 1: trace_conf[s] = minimum over the trace of the mean of token_conf over a sliding window of `window`
 *             tokens (a trace shorter than the window has one window, the whole trace);
 *     mode 2: trace_conf[s] = mean of the lowest ceil(0.1 n) of the n = len - window + 1 sliding-window means (the
 *             "bottom 10 % of the windows"; fewer than ten windows give the minimum).
 *   An empty trace gives 0.  trace_conf float [S_max]; cu_seqlens holds at least S_max + 1 entries; S is clamped to
 *   S_max, so a count in d_num larger than the arrays is never followed.  fp64 accumulation. */
int arrol_token_logprob_conf(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                             int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                             float* logp, float* lse, float* token_conf, void* workspace, size_t workspace_bytes,
                             void* stream);
int arrol_trace_confidence(arrol_ctx* ctx, const float* token_conf, const int64_t* cu_seqlens, const int64_t* d_num,
                           int32_t S_max, int32_t window, int32_t mode, float* trace_conf, void* stream);

/* ---- Quality-head training step (Section 4.2; Section 4.3 (iii)) ------------------------------------------
 * Cross-entropy of the head's logit against the rollout's final reward, gradients into the head only:
 *     y_i = rewards[i] > 0.5;  over the n rollouts with mask[i] != 0 (all when mask is NULL; e.g. the survivors, the
 *     only rollouts that ran to a final reward):
 *     loss = (1/n) sum_i [log(1 + exp(s_i)) - y_i s_i],   ds_i = (sigmoid(s_i) - y_i) / n,
 *     linear head: dW1 [d] = sum_i ds_i x_i, db1 [1] = sum_i ds_i;
 *     MLP head:    dw2 [h] = sum_i ds_i gelu(u_i), db2 [1] = sum_i ds_i, du_i = ds_i w2 gelu'(u_i),
 *                  dW1 [h, d] = du^T X, db1 [h] = sum_i du_i.
 * hidden / row_stride_elems / row_index / N / head as in arrol_score_partial (the scores are recomputed here).
 * Outputs are float (loss: device double [1]) and are overwritten; dw2, db2 are ignored for a linear head.
 * fp32 arithmetic, fixed-order reductions.  N <= 65536.  N == 0 or an all-zero mask gives zero loss and gradients.
 * workspace: arrol_head_grad_workspace(ctx, N, d, h) bytes, 256-byte aligned.  Uses the context scratch for the
 * linear head's scores: one stream at a time per context. */
size_t arrol_head_grad_workspace(arrol_ctx* ctx, int32_t N, int32_t d, int32_t h);
int arrol_head_grad(arrol_ctx* ctx, const void* hidden, int64_t row_stride_elems, const int64_t* row_index, int32_t N,
                    const arrol_head* head, const float* rewards, const uint8_t* mask, float* dW1, float* db1,
                    float* dw2, float* db2, double* loss, void* workspace, size_t workspace_bytes, void* stream);

/* ---- Test-time rank-weighted vote (Section 4.4) -----------------------------------------------------------
 * score [P*G] float: quality-head scores of G completed candidates per prompt (group-major); answer [P*G] int32:
 * an id of each candidate's final answer (equal ids = equal answers; < 0 = no answer, does not vote).
 * weight[i] = rank of candidate i inside its group / (G - 1): ranks by ascending score, equal scores in index
 * order, so the lowest score gets 0 and the highest 1 (a single candidate gets 1).  Every distinct answer sums the
 * weights of its candidates; winner[p] = the answer with the largest sum (of equal sums the one appearing first),
 * -1 when the group has no answer; winner_weight[p] = its sum.  Sums are compared as integer rank sums.  G <= 32. */
int arrol_rank_vote(arrol_ctx* ctx, const float* score, const int32_t* answer, int32_t P, int32_t G, float* weight,
                    int32_t* winner, float* winner_weight, void* stream);

/* ---- Whole step from host buffers (Algorithm 1, frontend lines "filter ... rebatch ... log-probs on R'") --
 * Convenience call for callers whose per-step data lives in host memory.  Only what the step needs is uploaded:
 * the small per-rollout arrays, the N hidden rows at the detection length (gathered into a pinned staging block of
 * the context and sent as one copy into d_hidden as a packed [N, d] block, for the head), and - once
 * arrol_score_partial and arrol_select have produced the keep mask, which is read back to plan the copies - the
 * survivors' hidden rows and token ids, copied straight into their packed positions in d_dst_rows / d_dst_tokens.
 * arrol_compact then produces the scan and the advantages, and arrol_token_logprob runs
 * per chunk of tokens as soon as the chunk's rows have landed (uploads on the context's second stream overlap the
 * tensor-core work).  Results are copied back and the stream is synchronised: the call is synchronous (one
 * synchronisation in the middle, one at the end) and allocates no device memory.
 * The quality head reads, for rollout i, source row src_tok_off[i] + cutoff - 1 (its hidden state at the
 * detection length).  Pointers prefixed h_ are HOST pointers (pinned memory gives full copy speed and real overlap),
 * d_ are DEVICE buffers provided by the caller with at least the stated sizes.  Model state (head, calib, W_vocab)
 * is device-resident.  P*G <= 1,048,576; head.d must equal d, d % 8 == 0; the workspace must be 256-byte aligned and
 * large enough (ARROL_ERR_WORKSPACE before anything is copied).  After the call d_hidden holds the N scored rows. */
typedef struct arrol_host_step {
    int32_t P, G, K, cutoff;       /* prompts, group size, survivors per group, detection length (>= 1)         */
    int32_t d, V;                  /* hidden width, vocabulary                                                  */
    int32_t ddof, reserved;
    double rho;                    /* target positive ratio                                                     */
    float eps, inv_temperature;
    int64_t T_src;                 /* source rows (sum of stored rollout lengths)                               */
    int64_t dst_capacity_tokens;   /* capacity of the packed buffers, in tokens                                 */
    /* inputs, host */
    const void* h_hidden;          /* [T_src, d] bf16                                                           */
    const int32_t* h_src_tokens;   /* [T_src]                                                                   */
    const int32_t* h_lengths;      /* [P*G]                                                                     */
    const int64_t* h_src_tok_off;  /* [P*G]                                                                     */
    const float* h_rewards;        /* [P*G]                                                                     */
    /* model state, device */
    arrol_head head;               /* dtype must be ARROL_BF16                                                  */
    arrol_calib calib;
    const void* W_vocab;           /* [V, d] bf16                                                               */
    /* staging and outputs, device */
    void* d_hidden;                /* [P*G, d] bf16: receives the scored rows                                   */
    int32_t* d_src_tokens;         /* unused (may be NULL): token ids are uploaded packed into d_dst_tokens     */
    int32_t* d_lengths;            /* [P*G]                                                                     */
    int64_t* d_src_tok_off;        /* [P*G]                                                                     */
    int64_t* d_row_index;          /* unused (may be NULL)                                                      */
    float* d_rewards;              /* [P*G]                                                                     */
    float *d_score, *d_prob, *d_q; /* [P*G] each                                                                */
    uint8_t* d_keep;               /* [P*G]                                                                     */
    int32_t* d_survivor_idx;       /* [P*G]                                                                     */
    int64_t* d_cu_seqlens;         /* [P*G + 1]                                                                 */
    float* d_adv;                  /* [P*G]                                                                     */
    int64_t* d_num;                /* [2]                                                                       */
    int32_t* d_dst_tokens;         /* [cap]                                                                     */
    void* d_dst_rows;              /* [cap, d] bf16                                                             */
    float* d_logp;                 /* [cap]                                                                     */
    void* d_workspace;             /* arrol_token_logprob_workspace(ctx, cap, d, V) bytes, 256-byte aligned     */
    size_t workspace_bytes;
    /* results, host */
    float* h_logp;                 /* [cap]; entries >= T are not meaningful                                    */
    float* h_adv;                  /* [P*G]; first S entries                                                    */
    int64_t* h_cu_seqlens;         /* [P*G + 1]; first S + 1 entries                                            */
    int32_t* h_survivor_idx;       /* [P*G]; first S entries                                                    */
    int64_t* h_num;                /* [2] = {S, T}                                                              */
} arrol_host_step;

/* Returns ARROL_OK, a validation/launch error, or the device status translated as by arrol_poll_status. */
int arrol_prune_rebatch_host(arrol_ctx* ctx, const arrol_host_step* step, void* stream);

/* ---- MLP-head scoring that allocates nothing ---------------------------------------------------------
 * (The paper has no counterpart to this call: it is a packaging variant of arrol_score_partial, added for
 * integration, and computes exactly the same outputs for an MLP head.)
 *
 * Who needs it: code that may not allocate device memory at the point where it scores rollouts.  Examples are a
 * serving or training process whose memory plan is frozen after start-up (all device memory already handed to
 * a pool or arena, so a raw cudaMalloc may fail or is forbidden by policy), a plug-in loaded into a host
 * application that owns the device heap, and latency-critical loops where an allocation's implicit device
 * synchronisation is not acceptable.  arrol_create allocates (status word, scratch), so such callers cannot
 * even make a context; this call therefore takes no context and runs on the calling thread's current device.
 *
 * How: the per-tile partial scores that arrol_score_partial keeps in the context scratch live here in a fixed
 * array inside the library image (128 KiB of device global memory on every GPU that loads the library, held
 * until the process exits).  Limits that follow from the fixed size: head->h > 0 (MLP head only),
 * N <= 4096 rollouts and head->h <= 512 per call; larger values return ARROL_ERR_UNSUPPORTED.  All other
 * arguments, layouts, alignment rules and outputs are those of arrol_score_partial.
 *
 * The first call on each device resolves the array's device address (a one-time, per-device set-up inside this
 * call, guarded by a mutex); make that first call before starting any stream capture on that device.
 * The call itself never calls cudaMalloc, cudaFree or any allocating library routine.
 * Every call on a device shares the one array, which keeps whatever the previous call left in it.  Nothing in it
 * has to start at zero: each call overwrites every entry it later reads.  Two calls that overlap in time on the
 * same GPU (different streams, or different host threads) race on the array and corrupt each other's scores;
 * issue them on one stream or order them yourself. */
int arrol_score_partial_static(const void* hidden, int64_t row_stride_elems, const int64_t* row_index, int32_t N,
                               const arrol_head* head, const arrol_calib* calib, float* score, float* prob,
                               int32_t* bin, float* q, void* stream);

/* ---- Index checks on request (no counterpart in the paper) -----------------------------------------------------
 * The compute calls trust row_index and src_tok_off + lengths, because their signatures carry no size of the source
 * buffers.  After arrol_set_source_rows(ctx, R) with R > 0 (the number of rows of `hidden` / src_tokens / src_rows),
 * every call on the context checks them on the device instead of following them:
 *   arrol_score_partial / arrol_prune_step: a row number outside [0, R) is never read; that rollout is scored as if
 *     its hidden row were zero;
 *   arrol_compact: if any kept rollout has src_tok_off < 0 or src_tok_off + length > R, the scan outputs are written
 *     and nothing is gathered (as for a capacity overflow);
 * and ARROL_DEV_BAD_INDEX is recorded in the status word.  R = 0 (the default) switches the checks off.  The other
 * calls (arrol_head_grad, arrol_token_logprob, ...) are not covered. */
int arrol_set_source_rows(arrol_ctx* ctx, int64_t source_rows);

/* Number of kernels this context has launched so far (host-side count; -1 for a NULL context). */
int64_t arrol_launch_count(arrol_ctx* ctx);

/* ---- Test hook (no counterpart in the paper) --------------------------------------------------------------------
 * Every pipeline wait inside the tensor-core kernels is bounded: when one runs out the block records
 * ARROL_DEV_WAIT_EXPIRED, lets its copies and MMAs in flight finish, frees its tensor memory and returns, and the
 * context stays usable.  In correct operation no wait ever runs out, so this hook lets a test exercise that path of
 * arrol_token_logprob without a fault or a hang:
 *   ARROL_HOOK_SPIN_LIMIT            value = tries per wait (0 restores the normal limit of 2^26)
 *   ARROL_HOOK_MUTE_LOGPROB_PRODUCER value != 0: the kernel's producer issues no copies, so the other roles' waits
 *                                    run out after the limit above; outputs of such a call are not written.
 *   ARROL_HOOK_LOGPROB_TIMING_BUFFER value = device address of a buffer of 4 x uint64 per work item (0 = off), and
 *   ARROL_HOOK_LOGPROB_TIMING_ITEMS  value = its capacity in work items: while set, every work item (token tile x
 *                                    vocabulary split) i < capacity of an arrol_token_logprob launch records
 *                                    {globaltimer at start, globaltimer at end, SM clock at start, SM clock at end}
 *                                    of its epilogue, from which a benchmark derives the SM clock the kernel ran at
 *                                    (cycles / nanoseconds) without reading or setting any GPU clock control.
 *   ARROL_HOOK_LOGPROB_SPLITS        value = vocabulary splits per token tile (1..64; 0 = chosen from the sizes, the
 *                                    default); set it before sizing the workspace, which depends on it.
 *   ARROL_HOOK_LOGPROB_PAIR          form of the log-prob kernel.  0: one thread block per 128-row token tile (tcgen05
 *                                    cta_group::1, cooperative launch).  1: clusters of two thread blocks that share
 *                                    one 256-row tile (tcgen05 cta_group::2; the same results bit for bit at equal
 *                                    split counts, 1.5-3 % faster at equal split counts).  2 (the default): pairs where
 *                                    they need no more vocabulary splits than single blocks, single blocks elsewhere
 *                                    (with more splits the pairs draw more power and, under the board's power cap,
 *                                    end up slower in long runs).  Pairs wait for one another per wave, so no more
 *                                    of them are launched than cudaOccupancyMaxActiveClusters says are resident at
 *                                    once (asked once per context).  Set it before sizing the workspace.
 * Returns INVALID_ARG for an unknown key or a limit outside [0, 2^26]. */
#define ARROL_HOOK_SPIN_LIMIT 1
#define ARROL_HOOK_MUTE_LOGPROB_PRODUCER 2
#define ARROL_HOOK_LOGPROB_TIMING_BUFFER 3
#define ARROL_HOOK_LOGPROB_TIMING_ITEMS 4
#define ARROL_HOOK_LOGPROB_PAIR 5
#define ARROL_HOOK_LOGPROB_SPLITS 6
int arrol_test_hook(arrol_ctx* ctx, int32_t key, int64_t value);

#ifdef __cplusplus
}
#endif
#endif /* ARROL_H_ */
