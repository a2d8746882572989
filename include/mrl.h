/*
 * mrl.h -- C ABI of libmrl: the token-level policy-loss pass that every learner of
 * Mutual RL (GRPO base update with PRP / XGRPO / SGT experience sharing) runs on each
 * optimisation step, as hand-written CUDA for NVIDIA B200 (sm_100a).
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 * ---------------------------------------------------------------------------
 *  - Plain C.  Every function returns an int status (MRL_OK = 0 or an MRL_ERR_* code) and
 *    never throws.  mrl_status_string() names a code.
 *  - Pointers marked [device] are CUDA device pointers, valid on the current device, owned by
 *    the caller, alive until the work enqueued by the call has finished.  Pointers marked
 *    [host] are read during the call only.  Nothing is allocated, freed or retained.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work
 *    is enqueued on it; the call does not synchronise and may return before the work runs.
 *  - Argument errors are detected on the host before anything is enqueued (MRL_ERR_INVALID_ARG,
 *    MRL_ERR_UNSUPPORTED_DTYPE, MRL_ERR_WORKSPACE_TOO_SMALL).  A failed launch gives MRL_ERR_CUDA.
 *  - Errors that only the device can see never fault: the kernel ORs a bit into the caller's
 *    `status` word [device, int32[1], nullable], treats the offending row as masked and goes
 *    on.  The library never clears `status`; zero it before the first call and read it after
 *    your own synchronisation.  Bits: MRL_DEV_BAD_TOKEN_ID (an id outside [0, V)),
 *    MRL_DEV_TIMEOUT (a bounded wait inside a kernel ran out -- on the fused LM head's own asynchronous
 *    copies or tensor-core work, or on the exchange between the two CTAs that share a logits row of
 *    512 KB or more; outputs of that call are then unspecified), MRL_DEV_BAD_WORD_MAP (word alignment).
 *  - `workspace` [device] is scratch of at least mrl_workspace_bytes(...) bytes, 256-byte
 *    aligned, contents unspecified before and after.  Calls that share a workspace must not
 *    overlap on the device.
 *  - Threads.  Calls from several host threads are fine as long as they do not share a workspace, with these
 *    exceptions, which keep per-device state inside the library and must not be called concurrently for one device:
 *    mrl_policy_loss_fwd_bwd_host (its copy streams and events), mrl_policy_loss_fwd_bwd_static (its scratch array),
 *    and the profiling hook (process-wide).
 *  - Row-major everywhere.  "Row t" is one response-token position: its logits row predicts
 *    ids[t] (the caller has already applied the next-token shift and dropped prompt rows).
 *  - Notation follows the paper: P prompts, M policies, G (the paper's K) rollouts per policy
 *    and prompt, S sequences, N rows, V vocabulary, H hidden size.
 */
#ifndef MRL_H_
#define MRL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MRL_VERSION 104

/* return codes */
#define MRL_OK 0
#define MRL_ERR_INVALID_ARG 1
#define MRL_ERR_BAD_TOKEN_ID 2       /* reserved for host-side id checks; device checks use the status word */
#define MRL_ERR_UNSUPPORTED_DTYPE 3
#define MRL_ERR_WORKSPACE_TOO_SMALL 4
#define MRL_ERR_CUDA 5
#define MRL_ERR_TIMEOUT 6
#define MRL_ERR_UNSUPPORTED_SHAPE 7
#define MRL_ERR_STATIC_SCRATCH_TOO_SMALL 8   /* mrl_policy_loss_fwd_bwd_static only: N or S above its fixed limits */

/* bits of the device status word */
#define MRL_DEV_BAD_TOKEN_ID 1
#define MRL_DEV_TIMEOUT 2
#define MRL_DEV_BAD_WORD_MAP 4

/* element types of logits / dlogits */
#define MRL_F32 0
#define MRL_BF16 1

/* mrl_adv_params.mode: which normalisation of the group-centred reward (Sec. 3; App. A) */
#define MRL_ADV_MEAN_ONLY 0     /* A = r - mean                                  (Sec. 3, A-tilde)    */
#define MRL_ADV_GROUP_ZNORM 1   /* A = (r - mean) / (std_group + eps)            (Sec. 3, A-tilde-zn) */
#define MRL_ADV_BATCH_ZNORM 2   /* A = (r - mean_group) / (std_batch + eps)      (App. A)             */

/* mrl_adv_params.sgt_pick: how y* is chosen among the peer successes (App. B) */
#define MRL_PICK_NONE 0
#define MRL_PICK_FIRST 1        /* lowest flat index m*G+g */
#define MRL_PICK_SHORTEST 2     /* smallest seq_len, ties to the lowest flat index ("shorter-response heuristic") */
#define MRL_PICK_ALL 3          /* every peer success */
#define MRL_PICK_SEEDED 4       /* the (splitmix64(seed*2^32 + p) mod n_success)-th success in flat order ("random choice") */

/* mrl_loss_params.agg_mode */
#define MRL_AGG_TOKEN_MEAN 0            /* one masked mean over all tokens */
#define MRL_AGG_SEQ_MEAN_TOKEN_MEAN 1   /* Eq. (1): E_tok within each sequence, then the mean over sequences */

/* mrl_loss_params.ratio_level */
#define MRL_RATIO_TOKEN 0      /* rho_t = exp(logp_t - logp_old_t), clipped per token               (Sec. 3, Eq. (1)) */
#define MRL_RATIO_SEQUENCE 1   /* w = exp(sum_t logp_t - sum_t logp_old_t) over a response, clipped per
                                  response; loss = - mean over responses of min(w A, clip(w) A)  (App. H) */

/* mrl_loss_params.kl_estimator: per-token estimate of KL(pi_theta || pi_ref) from the sampled token alone,
 * d = logp_t - logp_ref_t.  The paper states a per-token KL to a reference, as its own loss term (Eq. (1): beta R(theta);
 * App. A: coefficient 1e-3) and not which estimator; these are the three usual ones. */
#define MRL_KL_K1 0   /* d */
#define MRL_KL_K2 1   /* d^2 / 2 */
#define MRL_KL_K3 2   /* exp(-d) - 1 + d: non-negative, and like k1 its expectation under pi_theta is the KL exactly */

/* mrl_loss_params.flags */
#define MRL_FLAG_ACCUMULATE_LOSS 1u   /* loss[0..1] and stats += this call (micro-batch accumulation, App. A) */
#define MRL_FLAG_SKIP_ZERO_ROWS 2u    /* rows whose gradient multiplier is known to be zero before reading the
                                         logits (A = 0 or weight 0, and no NLL weight, no KL term) are not read:
                                         logp = 0, dlogits row = 0, they still count in the denominators.  Fused
                                         LM head: such rows report logp = 0 as well and blocks of 256 rows made of
                                         them (or of masked rows) are left out of the forward product; blocks
                                         without any gradient are left out of the backward products with or
                                         without this flag (the results do not depend on it) */
#define MRL_FLAG_ACCUMULATE_DW 4u     /* fused LM head: dW is float32 [V, H] and is added to, not overwritten */
#define MRL_FLAG_PAIR_TILES 8u        /* fused LM head: 256-row tiles worked by pairs of CTAs (tcgen05 cta_group::2).
                                         Same results.  Faster for a product timed alone; inside a long
                                         power-capped step the default tiles (one CTA each: 128 rows, 256 rows for the
                                         long-K dW product) were faster on B200 */

/* `which` of mrl_workspace_bytes */
#define MRL_WS_TOKEN_LOGPROBS 0
#define MRL_WS_POLICY_LOSS 1
#define MRL_WS_FUSED_LMHEAD 2
#define MRL_WS_THL_WORD_ALIGN 3         /* N = total number of words of the batch; V, H, dtype, S unused */

typedef struct mrl_adv_params {
  int32_t mode;             /* MRL_ADV_* */
  int32_t ddof;             /* 0: population std (divide by n), 1: sample std (n - 1) */
  float eps;                /* added to the std (Sec. 3) */
  float sgt_success_thr;    /* success iff r >  this (App. A: 0.8) */
  float sgt_negative_thr;   /* negative iff r < this (App. A: 0.2) */
  int32_t sgt_pick;         /* MRL_PICK_* */
  uint64_t seed;            /* MRL_PICK_SEEDED only (low 32 bits used) */
} mrl_adv_params;

typedef struct mrl_loss_params {
  float eps_lo;             /* clip band is [1 - eps_lo, 1 + eps_hi]; the paper uses 0.2 for both */
  float eps_hi;
  int32_t agg_mode;         /* MRL_AGG_* */
  uint32_t flags;           /* MRL_FLAG_* */
  double pg_denominator;    /* TOKEN_MEAN: number of valid tokens of the whole step when the step is fed in
                               several calls; <= 0: the valid tokens of this call */
  double seq_denominator;   /* SEQ_MEAN_TOKEN_MEAN: number of sequences of the whole step; <= 0: S */
  float nll_coeff;          /* lambda_SGT / n_gated (Eq. (2), App. B); 0 disables the NLL term */
  int32_t ratio_level;      /* MRL_RATIO_*; 0 (token level) is the default */
  float* entropy;           /* [device] float32 [N], nullable: entropy - sum_v p_v log p_v of softmax(z_t) at every valid
                               row that is read, 0 elsewhere -- the policy-entropy diagnostic of Sec. 6 / App. B,
                               taken from the same pass (one more FMA per logit; on the fused LM head one more
                               float per row and column tile of scratch traffic) */
  const float* logp_ref;    /* [device] float32 [N], nullable: no KL term.  Reference policy's log-prob of ids[t] */
  float kl_coeff;           /* beta of Eq. (1); App. A uses 1e-3 */
  int32_t kl_estimator;     /* MRL_KL_* */
  float* kl_loss;           /* [device] float32 [1]; required with logp_ref.  Receives beta * sum_t c_t k(d_t), c_t the
                               aggregation coefficient of the token (agg_mode; without tok_weight); added to under
                               MRL_FLAG_ACCUMULATE_LOSS.  The gradient outputs include this term's gradient,
                               beta c_t k'(d_t) through logp_t.  Rows stay live under MRL_FLAG_SKIP_ZERO_ROWS while
                               the term is on */
} mrl_loss_params;

/*
 * mrl_group_advantages -- group-relative advantages and the SGT rescue gate.
 *
 * Defined by: Sec. 3 (r-bar, A-tilde, A-tilde-zn); App. A (group mean then batch whitening);
 * Sec. 5.1 (PRP: advantages normalised over the unified pool of own and peer rollouts);
 * App. H, value-level coupling (XGRPO: mu_pool, sigma_pool over all M*K rewards of the prompt);
 * Sec. 5.3, App. A, App. B (SGT: gate = the learner has no success among its G rollouts and a
 * peer has one; success r > 0.8, negative r < 0.2; one peer success per learner and prompt).
 *
 *   rewards        [device] float32 [P, M, G]
 *   seq_len        [device] int32   [P, M, G] response lengths; nullable unless sgt_pick = SHORTEST
 *   learner        index in [0, M) of the policy the gate is evaluated for
 *   ap             [host]
 *   adv_own        [device] float32 [P, M, G]  each policy normalised within its own group; nullable
 *   adv_pool       [device] float32 [P, M, G]  normalised over the M*G rewards of the prompt; nullable
 *   rescue         [device] uint8   [P]        1 where the gate fires for `learner`; nullable
 *   pick           [device] int32   [P]        flat index m*G+g of the selected peer success, -1 if
 *                                              none (lowest selected index for PICK_ALL); nullable
 *   nll_seq_weight [device] float32 [P, M, G]  1.0 on selected rollouts, else 0; nullable
 *   n_gated        [device] int32   [1]        number of selected rollouts; nullable
 *
 * BATCH_ZNORM divides adv_own by the std of the group-centred values of that policy's whole
 * batch (its P*G values) and adv_pool by the std over all P*M*G pool-centred values.
 * All outputs are overwritten.  Integer outputs are exact; thresholds are compared in float32.
 * Limits: 1 <= M*G <= 1024.  Returns MRL_ERR_INVALID_ARG for sizes outside the limits, a
 * learner outside [0, M), an unknown mode, or SHORTEST without seq_len.  P = 0 is a no-op.
 */
int mrl_group_advantages(const float* rewards, const int32_t* seq_len, int32_t P, int32_t M, int32_t G,
                         int32_t learner, const mrl_adv_params* ap, float* adv_own, float* adv_pool,
                         uint8_t* rescue, int32_t* pick, float* nll_seq_weight, int32_t* n_gated,
                         void* stream);

/*
 * mrl_token_logprobs -- the token log-prob trace l_theta(x, y) of Sec. 3:
 *   lse_t = log sum_v exp(z[t, v]),  logp_t = z[t, ids_t] - lse_t.
 *
 *   logits [device] dtype [N, ld], ld >= V elements between rows (read once)
 *   dtype  MRL_BF16 or MRL_F32
 *   ids    [device] int32 [N]
 *   mask   [device] uint8 [N], nullable = all ones; rows with mask 0 are not read
 *   logp   [device] float32 [N]; 0 on masked rows and rows with a bad id
 *   lse    [device] float32 [N], nullable; 0 on those rows
 *   workspace: mrl_workspace_bytes(MRL_WS_TOKEN_LOGPROBS, ...) (currently 0; may be NULL then)
 *
 * float32 accumulation; results are bitwise reproducible from run to run.
 * N = 0 is a no-op.  V < 1, ld < V, N < 0, a null required pointer -> MRL_ERR_INVALID_ARG.
 */
int mrl_token_logprobs(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                       const int32_t* ids, const uint8_t* mask, float* logp, float* lse,
                       int32_t* status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * mrl_policy_loss_fwd_bwd -- the logits-in pass: log-probs, importance ratio, clipped
 * surrogate, masked aggregation and the gradient with respect to the logits, with each logits
 * row read from HBM once and each dlogits row written once.
 *
 * Defined by: Sec. 3 (w = exp(l_theta - l_old); Eq. (1)); Sec. 5.1 (PRP: the same update on
 * peer text, with the learner-snapshot or the THL-aligned trace as `logp_old`); Sec. 5.3 Eq. (2)
 * and App. B (SGT: lambda * NLL of the selected peer success, averaged per token and over the
 * gated examples); App. H, proof of Prop. 1 (softmax score e_i - pi).
 *
 * With m_t the validity of row t (mask and id in range), len_s the valid tokens of sequence s:
 *   c_t  = m_t / D                (TOKEN_MEAN,  D = pg_denominator)
 *        = m_t / (S_d * len_s)    (SEQ_MEAN_TOKEN_MEAN, S_d = seq_denominator)
 *   cn_t = nll_coeff * m_t * nll_weight_t / len_s
 *   rho_t = exp(logp_t - logp_old_t),  A_t = adv_seq[sequence of t],  u_t = tok_weight_t
 *   loss[0] = - sum_t c_t u_t min(rho_t A_t, clip(rho_t, 1-eps_lo, 1+eps_hi) A_t)
 *   loss[1] = - sum_t cn_t logp_t
 *   g_t = c_t u_t A_t rho_t [t unclipped] + cn_t
 *   dlogits[t, v] = g_t (softmax(z_t)[v] - [v == ids_t])
 * t is clipped iff (A_t > 0 and rho_t > 1+eps_hi) or (A_t < 0 and rho_t < 1-eps_lo); equality is
 * unclipped.  Rows with c_t u_t A_t = 0 add exactly 0 to loss[0].
 *
 * With lp->logp_ref (Eq. (1)'s beta R(theta); App. A: a per-token KL to a reference, its own loss term):
 *   d_t = logp_t - logp_ref_t,  k = the estimator lp->kl_estimator (MRL_KL_*)
 *   lp->kl_loss[0] = kl_coeff * sum_t c_t k(d_t),   g_t -= kl_coeff * c_t k'(d_t)     (every valid row; both
 *   ratio levels; the total loss is loss[0] + loss[1] + kl_loss[0])
 *
 * With ratio_level = MRL_RATIO_SEQUENCE (App. H, data-level coupling) the ratio is taken per response:
 *   w_s = exp(sum over the valid rows of s of (logp_t - logp_old_t)),  S_d = seq_denominator (<= 0: S)
 *   loss[0] = - (1 / S_d) sum_s min(w_s A_s, clip(w_s) A_s)   over responses with a valid row
 *   g_t = A_s w_s / S_d [s unclipped] + cn_t   for every valid row of s
 * agg_mode and pg_denominator are not used, tok_weight must be NULL (MRL_ERR_INVALID_ARG otherwise),
 * SKIP_ZERO_ROWS is ignored, and the gradient is a second launch that reads the logits again.  Every
 * response must be whole inside one call.  stats[1] counts the valid rows of clipped responses.
 *
 *   logits     [device] dtype [N, ld]
 *   ids, mask  as in mrl_token_logprobs
 *   cu_seqlens [device] int32 [S+1], non-decreasing, cu[0] = 0, cu[S] = N: sequence s owns rows
 *              [cu[s], cu[s+1])
 *   adv_seq    [device] float32 [S]
 *   logp_old   [device] float32 [N] behaviour-policy trace; nullable = equal to logp (rho = 1)
 *   tok_weight [device] float32 [N] stop-gradient weight u_t (PRP density weight); nullable = 1
 *   nll_weight [device] float32 [N] SGT weight (1 on rows of a selected y*); nullable = 0
 *   lp         [host]
 *   dlogits    [device] dtype [N, ld_out]; may equal `logits` with ld_out = ld (in place);
 *              nullable = forward only.  Every row is written (zeros where g_t = 0).  In place is also the
 *              faster way to call (measured 3-4 % on B200: the stores then land on lines L2 already holds).
 *   logp       [device] float32 [N], nullable
 *   loss       [device] float32 [2]: policy-gradient term, NLL term
 *   stats      [device] int64 [4], nullable: valid rows, clipped rows (valid, A != 0), rows
 *              read from HBM, rows with a bad id
 *   workspace: mrl_workspace_bytes(MRL_WS_POLICY_LOSS, N, V, 0, dtype, S)
 *
 * float32 row arithmetic on the input dtype, float64 for the final N-term sums (fixed order:
 * bitwise reproducible from run to run).  dlogits is rounded to nearest even.  The fast path (one CTA per row:
 * the row is streamed from HBM once and read a second time from L2) takes bf16 or float32 rows with V >= 4096 and
 * either 32-byte aligned logits / dlogits with V, ld, ld_out multiples of 32 bytes' worth of elements, or the same
 * with 16 bytes; anything else takes a general kernel with the same results.  Rows of 512 KB or more are shared by
 * two CTAs; rows much longer than 1 MB no longer fit L2 while in flight and are then read from HBM twice.
 * N = 0: loss (and stats) are zeroed unless ACCUMULATE_LOSS.
 */
int mrl_policy_loss_fwd_bwd(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                            const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens,
                            int32_t S, const float* adv_seq, const float* logp_old,
                            const float* tok_weight, const float* nll_weight,
                            const mrl_loss_params* lp, void* dlogits, int64_t ld_out, float* logp,
                            float* loss, int64_t* stats, int32_t* status, void* workspace,
                            size_t workspace_bytes, void* stream);

/*
 * mrl_policy_loss_fwd_bwd_host -- mrl_policy_loss_fwd_bwd for a batch that lives in HOST memory.
 *
 * Defined by: the same passages as mrl_policy_loss_fwd_bwd; App. A (the step is fed in log-prob micro-batches
 * and the loss is accumulated across them).  The batch is cut into micro-batches of whole sequences of at most
 * `slab_rows` rows; for each one its logits are copied to a staging buffer, the pass runs in place there, and the
 * gradient is copied back, the three legs on three streams over three staging buffers so that copies in both
 * directions overlap the kernels.  Results are those of mrl_policy_loss_fwd_bwd called once on the whole batch
 * (per-row outputs bit for bit; the loss up to the order of its float sums).
 *
 * Every `h_` argument, and lp->entropy, lp->logp_ref, lp->kl_loss, is a HOST pointer (page-locked memory is needed
 * for the copies to overlap; pageable memory works and serialises).  Shapes and meaning are those of the device
 * entry point.  h_cu_seqlens -- and h_ids / h_mask when agg_mode is TOKEN_MEAN and lp->pg_denominator <= 0 -- are
 * read on the host before the call returns; everything else is read and written asynchronously and the outputs
 * are valid once the caller has synchronised `stream`.  The host buffers must stay untouched until then.
 *
 *   slab_rows  capacity of one staging buffer in rows; no sequence may be longer (MRL_ERR_UNSUPPORTED_SHAPE)
 *   h_dlogits  [host] dtype [N, ld_out]; nullable = forward only.  Must not overlap h_logits unless identical
 *              with ld_out = ld (in place)
 *   h_loss     [host] float32 [2]; h_stats [host] int64 [4], nullable; h_status [host] int32 [1], nullable
 *   workspace  [device] >= mrl_host_pipeline_workspace_bytes(N, ld, dtype, S, slab_rows), 256-byte aligned:
 *              three staging buffers of slab_rows * ld elements, the per-row arrays, the loss scratch
 *   lp         [host] MRL_FLAG_ACCUMULATE_LOSS must be clear (the call returns the whole step's loss)
 *
 * ld * sizeof(element) must be a multiple of 32 bytes (MRL_ERR_UNSUPPORTED_SHAPE otherwise).  The library keeps
 * two copy streams and a few events per device, created at the first call and never freed; calls on one device
 * share them, so they must not overlap in time.  Errors: as mrl_policy_loss_fwd_bwd.
 */
int mrl_policy_loss_fwd_bwd_host(const void* h_logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                 const int32_t* h_ids, const uint8_t* h_mask, const int32_t* h_cu_seqlens,
                                 int32_t S, const float* h_adv_seq, const float* h_logp_old,
                                 const float* h_tok_weight, const float* h_nll_weight, const mrl_loss_params* lp,
                                 void* h_dlogits, int64_t ld_out, float* h_logp, float* h_loss, int64_t* h_stats,
                                 int32_t* h_status, int64_t slab_rows, void* workspace, size_t workspace_bytes,
                                 void* stream);
size_t mrl_host_pipeline_workspace_bytes(int64_t N, int64_t ld, int32_t dtype, int32_t S, int64_t slab_rows);

/*
 * mrl_policy_loss_fwd_bwd_static -- mrl_policy_loss_fwd_bwd for callers that cannot allocate.
 * The paper has no counterpart; this is a packaging variant of the entry point above.
 *
 * Who needs it: code that runs where device allocation is not available to it -- a plugin handed
 * nothing but the host framework's tensors and a stream, a real-time or pre-sized service whose
 * memory budget is frozen after start-up, a process in which cudaMalloc would force a device-wide
 * synchronisation in the middle of a pipelined step.  Such a caller has no way to provide the
 * `workspace` the ordinary entry point asks for.  Here the scratch is a fixed array inside the
 * library image (MRL_STATIC_SCRATCH_BYTES, held on every GPU that loads the library until the
 * process ends), so the call allocates nothing: no cudaMalloc / cudaFree, no allocating library
 * routine.  The caller still owns and passes every input and output.
 *
 * Arguments, results and arithmetic are exactly those of mrl_policy_loss_fwd_bwd (the same kernels
 * run) without `workspace` / `workspace_bytes`.  Limits: N <= MRL_STATIC_MAX_ROWS and
 * S <= MRL_STATIC_MAX_SEQS; anything larger returns MRL_ERR_STATIC_SCRATCH_TOO_SMALL before any
 * work is enqueued (split the step into several calls with MRL_FLAG_ACCUMULATE_LOSS and
 * pg_denominator set, as for micro-batches).
 *
 * The first call on each device looks up the device address of the array (a one-time set-up that
 * may load the module); make that first call outside any stream capture.  All calls on a device
 * share the one array: two calls whose work overlaps on the GPU (different streams, no ordering)
 * race on it.  The array keeps the previous call's contents; each call clears what it needs zeroed.
 */
#define MRL_STATIC_MAX_ROWS 65536
#define MRL_STATIC_MAX_SEQS 65536
#define MRL_STATIC_SCRATCH_BYTES (4u << 20)
int mrl_policy_loss_fwd_bwd_static(const void* logits, int32_t dtype, int64_t N, int32_t V, int64_t ld,
                                   const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens,
                                   int32_t S, const float* adv_seq, const float* logp_old,
                                   const float* tok_weight, const float* nll_weight,
                                   const mrl_loss_params* lp, void* dlogits, int64_t ld_out, float* logp,
                                   float* loss, int64_t* stats, int32_t* status, void* stream);

/*
 * mrl_fused_lmhead_loss_fwd_bwd -- the hidden-in pass: the same loss with z = hidden W^T formed
 * tile by tile on the tensor cores and reduced on the fly, so the [N, V] logits are never
 * stored; backward gives dHidden = dZ W and dW = dZ^T hidden.
 *
 * Defined by: the same passages as mrl_policy_loss_fwd_bwd (the paper's l_theta is the log-softmax
 * of the learner's output layer; it says nothing about the LM head itself).
 *
 *   hidden  [device] bf16 [N, H]   (contiguous, 16-byte aligned, H % 64 == 0)
 *   W       [device] bf16 [V, H]   (contiguous, 16-byte aligned)
 *   ids .. lp  as in mrl_policy_loss_fwd_bwd
 *   dHidden [device] bf16 [N, H], overwritten
 *   dW      [device] bf16 [V, H], overwritten; with MRL_FLAG_ACCUMULATE_DW float32 [V, H], added to
 *   logp, loss, stats, status  as above
 *   workspace: mrl_workspace_bytes(MRL_WS_FUSED_LMHEAD, N, V, H, MRL_BF16, S)
 *
 * bf16 operands, float32 accumulation; dZ is rounded to bf16 before the two backward products.
 */
int mrl_fused_lmhead_loss_fwd_bwd(const void* hidden, const void* W, int64_t N, int32_t H, int32_t V,
                                  const int32_t* ids, const uint8_t* mask, const int32_t* cu_seqlens,
                                  int32_t S, const float* adv_seq, const float* logp_old,
                                  const float* tok_weight, const float* nll_weight,
                                  const mrl_loss_params* lp, void* dHidden, void* dW, float* logp,
                                  float* loss, int64_t* stats, int32_t* status, void* workspace,
                                  size_t workspace_bytes, void* stream);

/*
 * mrl_thl_word_align_logprobs -- THL policy-distribution alignment: a peer's per-token log-prob trace mapped onto
 * the learner's tokenisation of the same text, the denominator of PRP's THL-aligned variant.
 *
 * Defined by: Sec. 4.2 (Z_w = sum of the source log-probs of word w; every target token of w gets
 * Z_w / max(1, C_w), C_w the number of target tokens of w); App. D, Alg. 3 (a sequence with no source token
 * mapped to a word is left at ignore_value; a target word without source tokens gets 0; tokens mapped to no word
 * get ignore_value); App. H, Thm. 1 (per-word mass is conserved wherever C_w > 0).
 *
 * Tokens are packed, response tokens only (the algorithm's masks already applied).  Sequence i owns source
 * tokens [src_cu[i], src_cu[i+1]), target tokens [tgt_cu[i], tgt_cu[i+1]) and word ids [0, word_cu[i+1] - word_cu[i]).
 *
 *   src_logp   [device] float32 [N_src]  source-policy log-probs
 *   src_word   [device] int32   [N_src]  word id of each source token (App. D, Alg. 1), negative = no word
 *   tgt_word   [device] int32   [N_tgt]  the same for the learner's tokens
 *   src_cu, tgt_cu, word_cu  [device] int32 [B+1], non-decreasing, starting at 0
 *   N_src, N_tgt lengths of the source and target token arrays (src_cu[B] and tgt_cu[B])
 *   total_words  word_cu[B] (sizes the workspace)
 *   out        [device] float32 [N_tgt]  aligned trace; every element is written
 *   src_total  [device] float32 [B], nullable: sum of all source log-probs of the sequence (L_mu of Thm. 1)
 *   tgt_total  [device] float32 [B], nullable: sum of the aligned values written (L~_mu); the difference of the
 *              two is the residual R_THL of Thm. 1
 *   workspace: mrl_workspace_bytes(MRL_WS_THL_WORD_ALIGN, total_words, 0, 0, 0, 0)
 *
 * Equal word ids must be contiguous within a sequence (what a span-by-span tokenisation yields); then every sum
 * is taken in token order by one thread and results are bitwise reproducible.  A word id seen in two separate
 * runs or outside the sequence's range sets MRL_DEV_BAD_WORD_MAP in `status` (such tokens count as "no word" /
 * their word's value is then unspecified).  So does an offset array that decreases or reaches past N_src, N_tgt or
 * total_words: each sequence's ranges are cut to the arrays, nothing outside them is read or written, and the outputs
 * of that sequence are unspecified.  float32 sums.  B = 0 is a no-op.
 */
int mrl_thl_word_align_logprobs(const float* src_logp, const int32_t* src_word, const int32_t* src_cu,
                                const int32_t* tgt_word, const int32_t* tgt_cu, const int32_t* word_cu, int32_t B,
                                int64_t N_src, int64_t N_tgt, int64_t total_words, float ignore_value, float* out,
                                float* src_total,
                                float* tgt_total, int32_t* status, void* workspace, size_t workspace_bytes,
                                void* stream);

/*
 * mrl_profile_dominant_kernel -- instrumentation for benchmarks; the paper has no counterpart.
 * Registers n pairs of CUDA events (cudaEvent_t passed as void*, created and owned by the caller).
 * From then on every launch of an entry point's dominant kernel (the per-row kernel of
 * mrl_token_logprobs / mrl_policy_loss_fwd_bwd; each tensor-core kernel of the fused LM head)
 * records start_events[i % n] just before and stop_events[i % n] just after it on the call's
 * stream, i counting such launches since registration.  n = 0 (or null arrays) unregisters.
 * The arrays [host] must stay alive while registered.  Process-wide and not thread-safe.
 */
int mrl_profile_dominant_kernel(void** start_events, void** stop_events, int32_t n);

/* Name of the dominant kernel launched last while events were registered (a static string; "" before the first
 * such launch): lets a benchmark say which kernel its timings and counters belong to.  Not thread-safe. */
const char* mrl_profile_last_kernel(void);

/* Scratch bytes an entry point needs for the given sizes (0 if none).  Pure host arithmetic. */
size_t mrl_workspace_bytes(int32_t which, int64_t N, int32_t V, int32_t H, int32_t dtype, int32_t S);

/* Static, NUL-terminated name of a return code. */
const char* mrl_status_string(int code);

/* MRL_VERSION of the loaded library. */
int mrl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MRL_H_ */
