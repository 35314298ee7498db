/*
 * oapl.h -- C ABI of the B200 (sm_100a) OAPL LM-head library.
 *
 * The library computes, for a batch of sampled responses, the trainer policy's
 * sequence log-probabilities ln pi(y_i|x) through the LM head, the group value
 * estimate of Eq. 2, the squared-regression objective of Eq. 3 of the OAPL paper
 * ("Method" section), and the gradient of Eq. 3 with respect to the hidden states
 * and the LM-head weight (Algorithm 1 takes gradient steps on Eq. 3), without ever
 * forming the [N, V] logits tensor.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the parameter comment says "host".
 *   - The caller owns every buffer.  The library allocates nothing, frees nothing
 *     and never synchronises the device (oapl_get_last_status excepted); all work
 *     is enqueued on `stream` (a cudaStream_t passed as void*).
 *   - Return value: OAPL_OK (0) or a negative oapl_status.  On an argument error
 *     nothing is enqueued.  Errors that only the device can see (a target outside
 *     [0,V) on a live row, decreasing seq_id, a pipeline wait that gave up) are
 *     recorded in the workspace and read back with oapl_get_last_status.
 *   - The current CUDA device must be the one that owns the buffers.
 */
#ifndef OAPL_H_
#define OAPL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  OAPL_OK = 0,
  OAPL_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, beta <= 0 or not finite */
  OAPL_ERR_MISALIGNED = -2,          /* H, W, dH, dW or workspace not 16-byte aligned */
  OAPL_ERR_WORKSPACE_TOO_SMALL = -3, /* ws_bytes < oapl_workspace_bytes(problem, flags) */
  OAPL_ERR_UNSUPPORTED_SHAPE = -4,   /* d not a multiple of 64, or sizes beyond int32 index range */
  OAPL_ERR_BAD_TARGET = -5,          /* device: mask==1 and target outside [0,V) */
  OAPL_ERR_BAD_SEQ_ORDER = -6,       /* device: seq_id decreasing or outside [0,S) */
  OAPL_ERR_NONFINITE_INPUT = -7,     /* device: non-finite reward, or group_id outside [0,P) */
  OAPL_ERR_DEVICE_TIMEOUT = -8,      /* device: a bounded pipeline wait expired */
  OAPL_ERR_CUDA = -9,                /* a CUDA runtime/driver call failed */
  OAPL_ERR_BAD_STATE = -10,          /* oapl_loss_bwd without a matching oapl_loss_fwd in ws */
  OAPL_ERR_SEQUENCE_TOO_LONG = -11,  /* device: oapl_loss_fwd_bwd met a sequence longer than its staging capacity */
  OAPL_ERR_OUT_OF_RANGE = -12,       /* device: a row's staged exponentials overflowed or vanished (single-call
                                        paths: some logit exceeds the target's by more than ~128, or H / W hold
                                        non-finite values); use oapl_loss_fwd + oapl_loss_bwd for such inputs */
  OAPL_ERR_BOUND_EXCEEDED = -13      /* device: the batch needs more ranges than the bounds passed in
                                        oapl_call_options allow (more live rows, or a longer sequence) */
} oapl_status;

/*
 * Environment variables, read by every call that uses them (tuning and testing; defaults in
 * parentheses):
 *   OAPL_STAGE_ROWS    rows of staged exponentials per range in the single-call paths (65536)
 *   OAPL_CHUNK_ROWS    rows per logit-gradient chunk of oapl_loss_bwd (18944)
 *   OAPL_SPLITS        vocabulary splits per wave of the logits sweeps (chosen from the L2 budget)
 *   OAPL_L2_BUDGET_MB  L2 budget for the hidden-state blocks of one wave of a sweep (48)
 *   OAPL_ACC_SKEW      K-steps by which the second accumulator of a sweep tile trails the first (4)
 *   OAPL_NVTX          1 = NVTX ranges around the phases a call enqueues, for a timeline profiler (0)
 *   OAPL_SYNC_EVERY    K-steps between the lock-step meetings of the CTA pairs (32; 0 = never)
 * They change workspace sizes and schedules, never results beyond summation order across splits.
 */

/* flags */
#define OAPL_FLAG_NONE 0
#define OAPL_FLAG_FUSED 1 /* oapl_workspace_bytes: size the workspace for oapl_loss_fwd_bwd */

/*
 * One batch, as the paper states the problem (Eq. 2 / Eq. 3): for every prompt x a
 * group of rollouts y_i with rewards r(x, y_i) and the inference engine's
 * log-probabilities; the trainer policy enters through the hidden states H and the
 * LM-head weight W.  Row n of H predicts targets[n]; rows of one sequence are
 * contiguous; only rows with mask==1 (response tokens) count in ln pi(y|x).
 */
typedef struct {
  int64_t N;               /* row positions (padded or packed; the mask decides)             */
  int32_t d;               /* hidden size, multiple of 64                                    */
  int32_t V;               /* vocabulary size, >= 1                                          */
  int32_t S;               /* sequences (rollouts)                                           */
  int32_t P;               /* prompts (groups)                                               */
  const void* H;           /* [N, d] bf16 row-major, 16-byte aligned                         */
  const void* W;           /* [V, d] bf16 row-major, 16-byte aligned; logits = H . W^T       */
  const int32_t* targets;  /* [N]; in [0,V) where mask==1; not read where mask==0            */
  const uint8_t* mask;     /* [N]; 1 = response token                                        */
  const int32_t* seq_id;   /* [N]; non-decreasing, in [0,S)                                  */
  const int32_t* group_id; /* [S]; in [0,P); members of a group need not be adjacent         */
  const float* reward;     /* [S]; finite                                                    */
  const float* logp_inf;   /* [N]; inference-policy token log-probs; read only where mask==1 */
  float beta_v;            /* temperature of Eq. 2 (the paper's beta_1), > 0                 */
  float beta_loss;         /* temperature of Eq. 3 (the paper's beta_2), > 0                 */
  float loss_scale;        /* lambda: 1 = Eq. 3's plain double sum; 1/S = mean per rollout   */
} oapl_problem;

/*
 * Bytes of device workspace the calls below need for `problem` (host call; reads
 * only N, d, V, S, P).  Returns 0 on invalid sizes.  The size grows with N*d and
 * with V (a bounded row-chunk of bf16 logit gradients), never with N*V.
 */
size_t oapl_workspace_bytes(const oapl_problem* problem /*host*/, int flags);

/*
 * ln pi(y_t | x, y_<t) for every row and ln pi(y_i|x) for every sequence: the log
 * of the policy's next-token distribution at the sampled token, summed over the
 * response tokens (the quantity pi(y_i|x) that enters Eq. 3).
 *   token_logp [N] f32: 0 where mask==0.       seq_logp [S] f32 or NULL.
 * Reads H, W, targets, mask, seq_id of `problem`; the other fields may be null.
 */
int oapl_token_logprobs(const oapl_problem* problem /*host*/, float* token_logp, float* seq_logp,
                        void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * Eq. 2: vhat[p] = beta_v * ln( (1/G_p) * sum_{i in group p} exp(reward[i]/beta_v) ),
 * evaluated in max-shifted form; G_p is the member count; a group without members
 * gets 0.  reward [S], group_id [S], vhat [P].  No workspace.
 */
int oapl_value_estimate(const float* reward, const int32_t* group_id, int32_t S, int32_t P,
                        float beta_v, float* vhat, void* stream);

/*
 * Eq. 3 forward: token log-probs -> masked per-sequence log-ratio D_i against
 * logp_inf -> Eq. 2 -> advantage A_i = r_i - vhat -> residual
 * delta_i = beta_loss*D_i - A_i -> loss = loss_scale * sum_i delta_i^2.
 *   loss [1], seq_logp [S], vhat [P], delta [S] (may be NULL), token_logp [N] (may be NULL).
 * Leaves in `ws` what oapl_loss_bwd needs (per-row log-sum-exp, per-sequence
 * coefficients 2*loss_scale*beta_loss*delta_i).
 */
int oapl_loss_fwd(const oapl_problem* problem /*host*/, float* loss, float* seq_logp, float* vhat,
                  float* delta, float* token_logp, void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * Gradient of Eq. 3: with p = softmax(logits) and c_i the coefficient of the row's
 * sequence, g[n,v] = c_i * mask_n * ([v == target_n] - p[n,v]);  dH = g . W,
 * dW = g^T . H.  Must follow oapl_loss_fwd on the same problem and workspace.
 *   dH [N, d] bf16 (rows with mask==0 are written as 0);
 *   dW [V, d] f32; overwritten, or added to when accumulate_dW != 0.
 */
int oapl_loss_bwd(const oapl_problem* problem /*host*/, void* dH, float* dW, int accumulate_dW,
                  void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * Eq. 3 forward and gradient in one call, without recomputing the logits in the backward.
 * Same inputs and outputs as oapl_loss_fwd followed by oapl_loss_bwd (same definitions:
 * Eq. 2, Eq. 3 and g = c_i * mask * (onehot - softmax)), but the work is organised by ranges
 * of whole sequences: for each range the logits pass stores e = exp(z - zref_row) as bf16
 * (zref_row = target logit + 40), the per-sequence coefficients of the range follow from
 * its log-probabilities, and since g = -c_i * e' / sum_v e (e' = e with the target entry
 * lowered by sum_v e) both gradient contractions read the staged e' directly:
 * dH = rowscale(e'.W), dW += e'^T.(scaled H).  Executed work is 6*N*d*V flops instead of 8.
 *
 * Workspace: oapl_workspace_bytes(problem, OAPL_FLAG_FUSED).  It holds e for 65536 rows
 * (2 bytes * round_up(V,512) each; OAPL_STAGE_ROWS in the environment changes the count), so
 * it does not grow with N*V; a sequence with more live rows than that cannot be staged and
 * raises OAPL_ERR_SEQUENCE_TOO_LONG in the status word (outputs are then not meaningful;
 * use the two separate calls).  A target whose probability under the policy is below
 * about e^-128 is outside the range of the staged exponentials: the row's sum overflows and
 * the status word becomes OAPL_ERR_OUT_OF_RANGE.
 */
int oapl_loss_fwd_bwd(const oapl_problem* problem /*host*/, float* loss, float* seq_logp, float* vhat,
                      float* delta /*may be NULL*/, float* token_logp /*may be NULL*/, void* dH, float* dW,
                      int accumulate_dW, void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * oapl_loss_fwd_bwd with what the caller knows about the batch on the host, and with a hook
 * for the data-parallel trainer step (the paper trains with a global batch spread over several
 * GPUs, "Experimental Details"; groups are independent in Eq. 2 / Eq. 3, so ranks hold whole
 * groups and exchange only the sum of dW).
 *
 * The number of live rows exists only on the device, so the call enqueues as many range slots
 * as the row count N could need; slots past the last range return at once.  A caller that
 * built the batch knows better:
 *   live_rows_bound     upper bound on the rows with mask==1 (0 = unknown: N is used);
 *   max_seq_rows_bound  upper bound on the live rows of any one sequence (0 = unknown).
 * They only reduce the number of (empty) launches.  Bounds that turn out too small are detected
 * on the device: the status word becomes OAPL_ERR_BOUND_EXCEEDED and the outputs are not
 * meaningful.
 *   dW_ready_event      a cudaEvent_t (as void*) or NULL.  It is recorded on `stream` right after
 *                       the last launch that writes dW; at that point the last range's dH
 *                       contraction has not started yet.  A second stream that waits for the event
 *                       can start the all-reduce of dW over the ranks under that contraction.
 *                       loss, seq_logp and dH are complete only when `stream` is.
 * options == NULL behaves like oapl_loss_fwd_bwd.
 */
typedef struct {
  int64_t live_rows_bound;
  int32_t max_seq_rows_bound;
  void* dW_ready_event;
} oapl_call_options;

int oapl_loss_fwd_bwd_ex(const oapl_problem* problem /*host*/, float* loss, float* seq_logp, float* vhat,
                         float* delta /*may be NULL*/, float* token_logp /*may be NULL*/, void* dH, float* dW,
                         int accumulate_dW, void* ws, size_t ws_bytes, int flags,
                         const oapl_call_options* options /*host, may be NULL*/, void* stream);

/*
 * The paper's baseline objective on the same LM-head pass: GRPO reweighted by token-level
 * importance ratios (the display in the Background section),
 *     J = 1/G sum_{y in group} 1/|y| sum_t  w_t * min( r_t A, clip(r_t, 1-eps, 1+eps) A ),
 *     w_t = pi_old(y_t|.) / pi_vllm(y_t|.)   (data: no gradient),
 *     r_t = pi(y_t|.) / pi_old(y_t|.),       A = the rollout's normalised advantage.
 *
 * oapl_group_advantage: A_i = (r_i - mean_p) / (std_p + eps) over the members of the
 * rollout's group p (population standard deviation; the paper only says "normalized
 * advantage").  reward [S], group_id [S], advantage [S]; a group without members writes
 * nothing.  eps >= 0.
 *
 * oapl_grpo_loss_fwd_bwd: loss = -loss_scale * sum_i 1/|y_i| sum_t w_t * min(...) (minimised),
 * and its gradient: per response token c_t = dloss/dlp_t = -loss_scale/|y_i| * w_t * A_i * r_t
 * where the unclipped branch is the minimum and 0 where the clipped (constant) branch is;
 * g[n,v] = c_n * ([v == target_n] - p[n,v]),  dH = g . W,  dW = g^T . H.  It runs on the
 * staged pipeline of oapl_loss_fwd_bwd (no logits tensor, no recompute) with per-token instead
 * of per-sequence coefficients.
 *   problem:    H, W, targets, mask, seq_id, logp_inf (= ln pi_vllm per token), loss_scale and
 *               the sizes are read; group_id, reward and the betas are not.
 *   logp_old    [N] f32: ln pi_old per token, read where mask==1.
 *   advantage   [S] f32.     clip_eps >= 0 (the paper's clip ratio 0.2).
 *   loss [1]; seq_logp [S] or NULL; token_logp [N] or NULL; clip_frac [1] or NULL: the fraction
 *   of response tokens on the clipped branch; dH [N,d] bf16; dW [V,d] f32 (overwritten, or
 *   added to when accumulate_dW != 0).
 *   ws: oapl_workspace_bytes(problem, OAPL_FLAG_FUSED) bytes; same limits as oapl_loss_fwd_bwd.
 */
int oapl_group_advantage(const float* reward, const int32_t* group_id, int32_t S, int32_t P, float eps,
                         float* advantage, void* stream);
int oapl_grpo_loss_fwd_bwd(const oapl_problem* problem /*host*/, const float* logp_old,
                           const float* advantage, float clip_eps, float* loss, float* seq_logp,
                           float* token_logp, float* clip_frac, void* dH, float* dW, int accumulate_dW,
                           void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * The optimizer step that follows the gradient in a trainer step, for the LM-head weight:
 * AdamW with gradient clipping by norm, the optimizer of the paper's "Experimental Details"
 * tables (math: lr 1e-6, betas 0.9/0.95, weight decay 1e-2, clip threshold 1e-3; code
 * generation: betas 0.9/0.999, threshold 1.0).  With g = dW * min(1, clip_norm / (||grad|| + 1e-6)),
 * where ||grad||^2 = sum(dW^2) + *other_sq_norm (the squared gradient norm of the model's other
 * parameters, device scalar or NULL), step t >= 1:
 *     m = beta1 m + (1-beta1) g;   v = beta2 v + (1-beta2) g^2;
 *     theta = theta (1 - lr weight_decay) - lr (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps).
 * theta is the fp32 `master` copy [n] when given (W then receives its bf16 rounding), else the
 * bf16 W itself.  W [n] bf16 (8-byte aligned), dW / m / v / master [n] f32 (16-byte aligned),
 * all updated in place; n = V*d.  clip_norm <= 0 disables clipping.  grad_norm [1] or NULL
 * receives ||grad||.  ws: oapl_adamw_workspace_bytes() bytes of device scratch (partial sums).
 * Two HBM-bound passes: dW is read twice, every other array once (34 bytes per element with a
 * master copy).
 */
size_t oapl_adamw_workspace_bytes(void);
int oapl_adamw_step(void* W, float* master, const float* dW, float* m, float* v, int64_t n, int64_t step,
                    float lr, float beta1, float beta2, float eps, float weight_decay, float clip_norm,
                    const float* other_sq_norm, float* grad_norm, void* ws, size_t ws_bytes, void* stream);

/*
 * Policy entropy of the trainer policy on the response tokens, the training-dynamics
 * diagnostic of the paper's experiments (the entropy curves of OAPL against GRPO in the
 * "Training dynamics" figure and the "sequence entropy" discussed beside it):
 *     H_n = - sum_v p[n,v] ln p[n,v] = lse_n - sum_v p[n,v] z[n,v],   p = softmax(z).
 * Every forward of this library (oapl_token_logprobs, oapl_loss_fwd, oapl_loss_fwd_bwd)
 * accumulates sum_v exp(z - ref) z next to the log-sum-exp in the same pass over the
 * logits and leaves H_n per response token in the workspace; this call only reads it back:
 *   token_entropy [N] f32 or NULL: H_n, 0 where mask==0;
 *   seq_entropy   [S] f32 or NULL: mean of H_n over the sequence's response tokens
 *                                  (0 for a sequence without any);
 *   mean_entropy  [1] f32 or NULL: mean of H_n over all response tokens of the batch.
 * `problem`, `ws`, `ws_bytes` and `flags` are those of the forward call (OAPL_FLAG_FUSED for
 * oapl_loss_fwd_bwd).  Without a preceding forward on `ws` the status word becomes
 * OAPL_ERR_BAD_STATE and nothing is written.
 */
int oapl_entropy(const oapl_problem* problem /*host*/, float* token_entropy, float* seq_entropy,
                 float* mean_entropy, void* ws, size_t ws_bytes, int flags, void* stream);

/*
 * Scalars a trainer logs next to the loss, from the quantities of Eq. 2 / Eq. 3 that the last
 * loss forward (oapl_loss_fwd, oapl_loss_fwd_bwd, oapl_loss_fwd_bwd_ex) left in `ws`; nothing is
 * recomputed.  With D_i = ln pi(y_i|x) - ln pi_vllm(y_i|x) and A_i = r_i - vhat[g_i]:
 *   stats[0] response tokens of the batch         stats[4] mean A_i over all rollouts
 *   stats[1] mean |D_i| over the rollouts with    stats[5] fraction of the groups (with members)
 *            response tokens                               whose rewards are all equal (A_i = 0)
 *   stats[2] max |D_i| over the same rollouts     stats[6] mean reward
 *   stats[3] sum_i D_i / response tokens          stats[7] 0
 * stats: 8 floats on the device; vhat [P]: the forward's output.  `problem`, `ws`, `ws_bytes`
 * and `flags` are those of the forward (OAPL_FLAG_FUSED for the single calls).  Without a
 * preceding loss forward on `ws` the status word becomes OAPL_ERR_BAD_STATE.
 */
int oapl_batch_stats(const oapl_problem* problem /*host*/, const float* vhat, float* stats, void* ws,
                     size_t ws_bytes, int flags, void* stream);

/* Synchronises `stream` and returns the status word the device recorded in `ws`
 * since the last forward call (OAPL_OK if none). */
int oapl_get_last_status(void* ws, void* stream);

/* Number of live rows (mask==1) counted by the last forward call on `ws`;
 * synchronises `stream`.  Negative oapl_status on error. */
int64_t oapl_get_live_rows(void* ws, void* stream);

/* Number of ranges of whole sequences the last single call (oapl_loss_fwd_bwd,
 * oapl_loss_fwd_bwd_ex, oapl_grpo_loss_fwd_bwd) on `ws` planned; synchronises `stream`. */
int oapl_get_range_count(void* ws, void* stream);

/* Kernel launches enqueued by this library in this process so far. */
uint64_t oapl_launch_count(void);

const char* oapl_status_string(int status);

/*
 * oapl_token_logprobs for callers that cannot provide a workspace.  (The paper has no
 * counterpart; this is a property of the library, not of the method.)
 *
 * Who needs it: code that is not allowed to allocate device memory where it calls us --
 * a plug-in inside a framework that owns the allocator, a serving loop whose memory was
 * fixed at start-up, or a section in which the CUDA allocator must not be entered.  The
 * scratch memory lives in a fixed device array inside the library (about 4.8 MB per GPU
 * that loads the library, held until the process exits), so sizes are limited:
 *     N <= 2048,  d <= 1024 (multiple of 64),  S <= 2048,  any V >= 1.
 * Larger problems return OAPL_ERR_UNSUPPORTED_SHAPE and print the limits to stderr.
 * The call itself allocates and frees nothing.
 *
 *   token_logp [N] f32, seq_logp [S] f32 or NULL: as in oapl_token_logprobs.
 *   device_status: device int32 or NULL; receives the device-detected status word
 *                  (OAPL_OK, OAPL_ERR_BAD_TARGET, OAPL_ERR_BAD_SEQ_ORDER, ...) in stream order.
 *
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call before starting any stream capture.  All calls on one
 * GPU share the one array and it keeps the previous call's contents; the call clears the
 * parts that must start at zero, but two calls whose work overlaps on the GPU (different
 * streams without ordering, or several host threads) race on it and give wrong results:
 * order them.
 */
int oapl_token_logprobs_static(const oapl_problem* problem /*host*/, float* token_logp, float* seq_logp,
                               int32_t* device_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Testing and timing aids.  Nothing below is part of the method; a trainer does not need it.
 * ------------------------------------------------------------------------------------------ */

/*
 * Host logic only: the number of range slots the single call enqueues for a batch of at most
 * live_rows_bound live rows in S sequences of at most max_seq_rows_bound live rows each
 * (0 = unknown) and a staging capacity of stage_rows rows -- an upper bound on the number of
 * ranges the greedy packing of whole sequences can produce.
 */
int oapl_range_slots(int64_t live_rows_bound, int64_t max_seq_rows_bound, int32_t stage_rows, int32_t S);

/*
 * Optional timing of the contraction launches (off by default).  oapl_profile_enable(1)
 * switches it on for the CURRENT device: from then on every contraction launch on that device
 * is bracketed by a CUDA event pair on its stream (launches on other devices run untimed).
 * oapl_profile_read waits for those events and sums the elapsed milliseconds and the launch
 * counts per kind into host arrays of `kinds` entries: 0 = logits + online log-sum-exp,
 * 1 = logit-gradient chunk, 2 = dH, 3 = dW, 4 = bring-up GEMM, 5 = logits + staged
 * exponentials; then clears the record.  At most 65536 launches are recorded between two
 * reads; *launches_dropped (host, may be NULL) receives how many were not.  Not thread-safe.
 */
int oapl_profile_enable(int on);
int oapl_profile_read(float* ms_by_kind /*host*/, int* launches_by_kind /*host*/, int kinds,
                      int* launches_dropped /*host*/);
/*
 * While the timing is enabled, CTA 0 of every contraction launch also adds its SM cycle count
 * and its elapsed nanoseconds to two per-kind device counters.  This call (with the device the
 * timing was enabled on current) synchronises the device, writes cycles/nanoseconds as MHz per
 * kind (0 where the kind did not run) -- the SM clock that kind of launch ran at, which on a
 * power-capped part differs from kind to kind -- and clears the counters.  kinds <= 8.
 */
int oapl_profile_read_clocks(float* sm_mhz_by_kind /*host*/, int kinds);
/* The rule the launches apply (host logic only, no CUDA call): 1 when a launch on
 * `current_device` is timed given that the timing was enabled on `enabled_device` (-1 = off). */
int oapl_profile_applies(int enabled_device, int current_device);

/*
 * Bring-up aid for the tensor-core main loop shared by every contraction above:
 * C[M, N] (f32 row-major, ld = N) = A . B with bf16 operands, through the same
 * TMA/tcgen05 pipeline.  a_mn == 0: A is [M, K] row-major (K contiguous);
 * a_mn == 1: A is stored [K, M] row-major (M contiguous).  b_mn == 0: B is stored
 * [N, K] row-major; b_mn == 1: B is stored [K, N] row-major.  wide == 0: 256 x 256 tiles
 * with alternating accumulators; wide == 1: 256 x 512 tiles (the shape of every product
 * contraction).  K % 64 == 0, M % 8 == 0, N % 8 == 0.
 * `err` points to TWO device ints: err[0] (cleared by the caller) is set by the kernel to
 * OAPL_ERR_DEVICE_TIMEOUT when a pipeline wait gave up; err[1] is the counter of the CTA pairs'
 * lock-step meetings (cleared by the call; OAPL_SYNC_EVERY=0 switches the meetings off).
 *
 * Test of the give-up path: wait_cycles > 0 replaces the limit of every pipeline wait (SM
 * cycles; 0 = the product limit of 4e9), and skip_step = k > 0 makes the load warps leave out the
 * loads of pipeline step k - 1, so that the wait for them runs out: every role then leaves its
 * loop, the kernel frees its tensor memory and returns, and err[0] holds the timeout status
 * (C is not meaningful).  skip_step needs 0 < wait_cycles <= 1e8.  Nothing faults and the
 * context stays usable.
 */
int oapl_debug_gemm(const void* A, const void* B, float* C, int M, int N, int K, int a_mn,
                    int b_mn, int wide, long long wait_cycles, int skip_step, int* err, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OAPL_H_ */
