/*
 * e3 -- vocabulary-side hot path of entropy-holding RL for LLMs, for NVIDIA B200 (sm_100a).
 *
 * One C ABI, plain pointers and sizes.  Every rollout token and every training
 * token passes through a per-row temperature softmax over the vocabulary; this
 * library computes, in one streaming pass over the logits,
 *   - the Shannon entropy of softmax(z / tau)               (paper: Eq. "entropy", App. A)
 *   - the log-probability of a given or a sampled token     (Sec. 3.1, importance ratio)
 *   - a reproducible Gumbel-max sample                      (Sec. 2 / Sec. 5.1: tokens are drawn from softmax(z/tau))
 * plus the masked mean entropy that drives the temperature scheduler (Sec. 4.2),
 * the group-relative advantage (Eq. "adv") over ragged rollout groups, and two
 * tiny host functions: Algorithm 1 (rollout budget) and Eq. "tp_adj" with annealing.
 *
 * Conventions for every device call
 *   - "device" pointers are CUDA device pointers owned by the caller; the
 *     library allocates and frees no device memory.  What it keeps between calls, per process:
 *     a counter that gives every row call its own id (the tag of the partial row states in the
 *     workspace), a per-device record of each kernel's launch set-up (filled on first use), and
 *     for e3_masked_mean_entropy_static the address of its built-in scratch.  No result depends on them.
 *   - Pointers: every pointer must be aligned to its element type (else E3_ERR_ALIGNMENT);
 *     workspaces to 16 bytes.  Optional outputs are NULL when not wanted.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).  Calls never synchronise, print or abort.  The kernels are launched with
 *     programmatic stream serialization: their set-up may overlap the tail of the work before them in
 *     the stream; they touch memory only after that work has completed.
 *   - The return value reports what the host can see (bad sizes, NULL
 *     pointers, launch failure).  Problems only the device can see (NaN or
 *     +inf logit, a row of -inf only, tau < 0 or not finite) mark that row:
 *     token -1, log-prob, entropy and gap NaN.  Other rows are unaffected.
 *   - Every wait inside a kernel is bounded (two seconds).  If one ever runs out, the thread block
 *     concerned gives up: its unfinished rows read token -1 / NaN and bit E3_STATUS_TIMEOUT is OR-ed
 *     into the caller's status word (`out_status`, optional, never cleared by the library).  The host
 *     sees it after synchronising; e3_status has E3_ERR_TIMEOUT for callers that want to pass it on.
 *     After a timeout, clear a workspace (cudaMemsetAsync) before a captured graph that uses it is
 *     replayed.
 *   - Results are bit-reproducible for identical arguments.
 *   - Stream capture: every call may be captured into a CUDA graph and replayed (the row calls wipe
 *     their partial row states when a row is finished, so a replay never meets an old one).
 *   - rows == 0 / n == 0 / n_groups == 0 are valid no-ops.
 */
#ifndef E3_H_
#define E3_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define E3_API __attribute__((visibility("default")))
#else
#define E3_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  E3_OK = 0,
  E3_ERR_INVALID_ARG = 1, /* NULL required pointer, negative size, V < 1 or V >= 2^31, row_stride < V, ... */
  E3_ERR_DTYPE = 2,       /* dtype is neither E3_F32 nor E3_BF16 */
  E3_ERR_ALIGNMENT = 3,   /* a pointer is not aligned to its element type */
  E3_ERR_WORKSPACE = 4,   /* workspace missing or smaller than e3_workspace_bytes() says */
  E3_ERR_INFEASIBLE = 5,  /* Algorithm 1: needs G_min <= G <= G_max */
  E3_ERR_CUDA = 6,        /* a CUDA runtime call failed (no device, launch error) */
  E3_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out: never returned by a call (calls do not
                             synchronise); the code for a caller that found E3_STATUS_TIMEOUT in its status word */
} e3_status;

/* Bits of the device status word (`out_status` of the row calls). */
#define E3_STATUS_TIMEOUT 1

typedef enum { E3_F32 = 0, E3_BF16 = 1 } e3_dtype;

/* Sampler of e3_sample.  Both draw exactly from softmax(z / tau) up to the
 * resolution of their uniforms (2^-40 and 2^-32). */
typedef enum {
  E3_SAMPLER_TOKEN = 0, /* one Gumbel per vocabulary entry: tok = argmax_i (z_i/tau + g_i) */
  E3_SAMPLER_BLOCK = 1, /* one Gumbel per block of E3_SAMPLE_BLOCK consecutive entries applied to the
                           block's log-sum-exp, then inverse CDF inside the winning block */
  E3_SAMPLER_TOKEN_AUDIT = 2 /* the draw of E3_SAMPLER_TOKEN, token for token, computed the slow way: the fast
                           path's fp32 scores (good to about 2e-4) are trusted only when the leader is
                           ahead by a margin a thousand times wider than needed, so most rows are settled by
                           the fp64 path that normally only sees near-ties.  For validation. */
} e3_sampler;
#define E3_SAMPLE_BLOCK 256

typedef enum {
  E3_CALL_SAMPLE = 0,
  E3_CALL_TOKEN_LOGP_ENTROPY = 1,
  E3_CALL_MASKED_MEAN_ENTROPY = 2,
  E3_CALL_GRPO_OBJECTIVE = 3,
  E3_CALL_SEQUENCE_MEAN_ENTROPY = 4
} e3_call;

/* Human-readable name of a status code (static string). */
E3_API const char *e3_status_string(e3_status s);

/* Bytes of device scratch a call uses for the given problem size.  For
 * E3_CALL_MASKED_MEAN_ENTROPY `rows` is the number of tokens n, for E3_CALL_GRPO_OBJECTIVE the number of
 * responses n_seq, for E3_CALL_SEQUENCE_MEAN_ENTROPY the number of sequences n_seq; V, dt are ignored for these.  E3_CALL_SAMPLE: 256 KiB for the partial states of cut rows plus,
 * for E3_SAMPLER_BLOCK, the per-lane sums the second kernel reads (about 1/32 of the bytes of the logits);
 * E3_CALL_TOKEN_LOGP_ENTROPY: 256 KiB plus the partial sums of the fused mean entropy.
 * Scratch contents on entry never matter.  A workspace must not be shared by calls that can run
 * at the same time (different streams without ordering).  It must be 16-byte aligned. */
E3_API size_t e3_workspace_bytes(e3_call which, int64_t rows, int64_t V, e3_dtype dt);

/*
 * Rollout step.  For every row r: p = softmax(logits[r, 0..V) / temps[r])
 * (App. A); out_ent[r] = -sum p ln p (Eq. "entropy"); out_tok[r] = one token
 * drawn from p with the Gumbel-max construction; out_logp[r] = ln p[out_tok[r]].
 *
 *   logits      device, row-major [rows, V], element type `dt`, row r starts at
 *               element r * row_stride (row_stride >= V, in elements).  Rows whose
 *               start is 16-byte aligned take the vectorised path; others a slower one.
 *   temps       device float [rows].  tau > 0 samples; tau == 0 is greedy
 *               (lowest-index arg-max, logp = 0, ent = 0); tau < 0, NaN, inf mark the row invalid.
 *   seed, counter, row_base
 *               the draw is a pure function of (seed, counter, row_base + r, vocabulary index):
 *               Philox4x32-10 with key = seed and counter words
 *               (call index, row_base + r, counter low word, counter high bits << 8 | stream tag).
 *               counter < 2^56: the decode step; row_base: index of this call's first row in the
 *               whole batch, so that a batch split over several calls or devices draws the same tokens.
 *               Sampler 0: u_i = (c_i + (x_i + 1/2) 2^-32) / 256 with c_i byte (i mod 16) of call i/16 of
 *               stream 0 and x_i word (i mod 4) of call i/4 of stream 1; g_i = -ln(-ln u_i);
 *               ties go to the lower index.
 *               Sampler 1: u_b = (x_b + 1/2) 2^-32, x_b word (b mod 4) of call b/4 of stream 2, for block b;
 *               the in-block draw uses word 0 of call 0 of stream 3.
 *               row_base >= 0 and row_base + rows <= 2^32 (the row number is one 32-bit counter word), else
 *               E3_ERR_INVALID_ARG.
 *   out_tok     device int32 [rows], required.   out_logp, out_ent: device float [rows], each may be NULL.
 *   out_gap     device float [rows] or NULL: the mean logit gap of App. A in units of tau,
 *               beta sum_i p_i Delta_i with Delta_i = z_max - z_i (so that H = ln sum_i exp(-beta Delta_i) + gap);
 *               0 for greedy rows.  Asking for it selects a kernel variant that also tracks z_max.
 *   out_status  device int32 or NULL: status word, see the conventions above.
 *   workspace   device scratch of e3_workspace_bytes(E3_CALL_SAMPLE, ...) bytes.  It holds the partial states
 *               of rows that are split between thread blocks so that every block streams the same number
 *               of bytes, and what the two kernels of E3_SAMPLER_BLOCK hand to each other.  For the other
 *               samplers NULL (or fewer than 256 KiB) is accepted: rows are then never split, which costs
 *               throughput when there are fewer than a few thousand rows.  E3_SAMPLER_BLOCK needs the full
 *               size (E3_ERR_WORKSPACE).
 * -inf logits are allowed (probability 0, never drawn).
 */
E3_API e3_status e3_sample(const void *logits, e3_dtype dt, int64_t rows, int64_t V, int64_t row_stride,
                    const float *temps, uint64_t seed, uint64_t counter, int64_t row_base, e3_sampler sampler,
                    int32_t *out_tok, float *out_logp, float *out_ent, float *out_gap, int32_t *out_status,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * Training-side pass.  For every row with mask[r] != 0:
 * out_logp[r] = ln softmax(logits[r] / tau_r)[targets[r]], out_ent[r] = entropy of that
 * distribution.  The paper divides the logits by the sampling temperature in the training
 * forward as well (Sec. 4.2), so the call takes tau: temps[r] when temps != NULL, else temp_scalar.
 * Here tau must be > 0 and finite.  Rows with mask[r] == 0 get 0 in both outputs and their
 * logits are not read.  A target outside [0, V) gives out_logp = NaN (entropy still valid).
 *
 *   targets     device int32 [rows];  mask: device uint8 [rows] or NULL (= all ones)
 *   out_logp, out_ent, out_gap   device float [rows], each may be NULL (out_gap as in e3_sample; 0 on masked rows)
 *   out_ent_sum, out_count   both NULL, or both device double scalars: the batch entropy of the scheduler
 *               (Sec. 4.2) from the same call: out_ent_sum = sum_r mask[r] out_ent[r] accumulated in fp64 in
 *               the fixed order of e3_masked_mean_entropy, out_count = sum_r mask[r]; out_ent_sum / out_count
 *               equals that call's mean bit for bit.  Needs out_ent and the workspace
 *               (E3_ERR_INVALID_ARG / E3_ERR_WORKSPACE).  The reduction runs as two small kernels behind
 *               the row kernel, chained by programmatic dependent launch.
 *   workspace   e3_workspace_bytes(E3_CALL_TOKEN_LOGP_ENTROPY, rows, V, dt) bytes; NULL or fewer than
 *               256 KiB is accepted when the fused mean is not asked for (rows are then never split).
 * Other arguments as in e3_sample.
 */
E3_API e3_status e3_token_logp_entropy(const void *logits, e3_dtype dt, int64_t rows, int64_t V, int64_t row_stride,
                                const int32_t *targets, const uint8_t *mask,
                                const float *temps, float temp_scalar,
                                float *out_logp, float *out_ent, float *out_gap,
                                double *out_ent_sum, double *out_count, int32_t *out_status,
                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward of e3_token_logp_entropy.  The objective of Sec. 3.1 depends on the logits through
 * ln pi(o_t), and the entropy-regularised objective discussed in Sec. 4.2 also through the entropy H;
 * with p = softmax(logits[r] / tau_r), beta = 1/tau_r (App. A) the chain rule through the softmax gives,
 * for every row with mask[r] != 0,
 *   dlogits[r, i] = beta ( g_logp[r] (1[i == targets[r]] - p_i)  -  g_ent[r] p_i (ln p_i + H_r) ).
 * Rows with mask[r] == 0 get zeros.  A row whose temperature, target or forward outputs are not usable
 * (tau <= 0 or not finite, target outside [0, V), logp or ent NaN) gets NaN.
 *
 *   logits, dt, rows, V, row_stride, targets, mask, temps, temp_scalar   as in the forward call
 *   logp, ent     device float [rows]: the forward call's outputs for the same arguments (the row's
 *                 normaliser is taken from them: ln p_i = (z_i - z_tok)/tau + logp)
 *   g_logp, g_ent device float [rows]: upstream gradients; NULL = all zero
 *   dlogits       device, same element type as logits, row r starts at element r * dlogits_stride
 *                 (dlogits_stride >= V); must not overlap logits.  Rows and strides that are 16-byte
 *                 aligned on both sides take the vectorised path.
 * No workspace.  One pass: V entries read and V written per row.
 */
E3_API e3_status e3_token_logp_entropy_backward(const void *logits, e3_dtype dt, int64_t rows, int64_t V,
                                         int64_t row_stride, const int32_t *targets, const uint8_t *mask,
                                         const float *temps, float temp_scalar, const float *logp, const float *ent,
                                         const float *g_logp, const float *g_ent, void *dlogits,
                                         int64_t dlogits_stride, void *stream);

/*
 * Batch entropy H_t of the scheduler (Sec. 4.2: "average entropy" of a batch), read as the mean
 * over all response tokens: out_mean = sum_j mask[j] ent[j] / sum_j mask[j], accumulated in
 * fp64 in a fixed order.  out_count = sum_j mask[j].  count == 0 gives mean NaN.
 *
 *   ent         device float [n];  mask: device uint8 [n] or NULL (= all ones)
 *   out_mean, out_count   device double scalars, required
 *   workspace   device scratch of e3_workspace_bytes(E3_CALL_MASKED_MEAN_ENTROPY, n, 0, 0) bytes;
 *               contents on entry do not matter.
 */
E3_API e3_status e3_masked_mean_entropy(const float *ent, const uint8_t *mask, int64_t n,
                                 double *out_mean, double *out_count,
                                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * The other reading of "average entropy" (Sec. 4.2 does not say which): the mean over sequences of each
 * sequence's mean token entropy.  Tokens are laid out [n_seq, seq_len]; mask marks the response tokens.
 *   out_mean  = (1 / S) sum_s ( sum_t mask[s,t] ent[s,t] / sum_t mask[s,t] ), over the S sequences that have a token
 *   out_count = S.   S == 0 gives mean NaN.
 * Long responses weigh as much as short ones here, while e3_masked_mean_entropy weighs every token equally.
 * fp64, fixed order (one thread block per sequence, then one block over the sequences in index order).
 *   ent, mask   device float / uint8 [n_seq * seq_len], mask may be NULL (= all ones);  n_seq < 2^31
 *   workspace   e3_workspace_bytes(E3_CALL_SEQUENCE_MEAN_ENTROPY, n_seq, 0, 0) bytes of device scratch, 8-byte aligned
 */
E3_API e3_status e3_sequence_mean_entropy(const float *ent, const uint8_t *mask, int64_t n_seq, int64_t seq_len,
                                          double *out_mean, double *out_count,
                                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same mean entropy for callers that have no scratch memory to give.  (The paper has no
 * counterpart for this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a plugin or callback
 * executing inside somebody else's stream or inference engine, a real-time loop that must not
 * touch the allocator, a process whose memory pool was sized up front and handed out completely.
 * Such callers cannot call cudaMalloc and often have no spare buffer for
 * e3_masked_mean_entropy's workspace.  Here the per-block partial sums live in a fixed
 * 16 KiB array inside the library image; every GPU that loads the library holds those 16 KiB
 * until the process exits.  The call itself allocates and frees nothing.
 *
 *   ent, mask, n, out_mean, out_count, stream: as in e3_masked_mean_entropy (device pointers).
 *   n may not exceed E3_STATIC_MEAN_MAX_TOKENS; a larger n returns E3_ERR_WORKSPACE (the
 *   built-in scratch is not sized for it) and launches nothing.
 *
 * The first call on each device looks up the array's device address (one runtime query, made
 * with that device current).  Make that first call outside any stream capture.
 * All calls on a device share the one array, and it keeps whatever the previous call left in it.
 * That is harmless for calls that run one after another (each call overwrites every entry it
 * later reads), but two calls whose kernels overlap on the GPU -- different streams, no
 * ordering between them -- race on it and give wrong means.  Serialise them.
 * Results equal e3_masked_mean_entropy's bit for bit.
 */
#define E3_STATIC_MEAN_MAX_TOKENS (INT64_C(1) << 26)
E3_API e3_status e3_masked_mean_entropy_static(const float *ent, const uint8_t *mask, int64_t n,
                                               double *out_mean, double *out_count, void *stream);

/*
 * Group-relative advantage (Eq. "adv"): inside each rollout group g = rows
 * [group_offsets[g], group_offsets[g+1]):  A_i = (r_i - mean) / (std + eps).
 * Groups may have any size (the rollout budget of Algorithm 1 makes them ragged).
 * std is the sample standard deviation (divide by n-1) when unbiased != 0, else the population one.
 * A group with identical rewards gives exactly 0, as Sec. 4.2 assumes (also with eps == 0, where the
 * quotient would be 0/0).  eps must be >= 0 and finite.  A group of one gives 0; an empty group writes nothing.
 *
 *   rewards        device float [group_offsets[n_groups]]
 *   group_offsets  device int64 [n_groups + 1], non-decreasing, [0] == 0
 *   out_adv        device float, same length as rewards
 *   out_group_flags  NULL or device uint8 [n_groups]: bit 0 = all rewards equal, bit 1 = all rewards zero
 */
E3_API e3_status e3_group_advantage(const float *rewards, const int64_t *group_offsets, int64_t n_groups,
                             float eps, int unbiased, float *out_adv, uint8_t *out_group_flags, void *stream);

/*
 * The GRPO objective of Sec. 3.1 without its KL term (the paper does not use it), over one batch:
 *   J = mean over questions q of (1/G_q) sum_{i in q} (1/|o_i|) sum_{t <= |o_i|}
 *         min( r_{i,t} A_i , clip(r_{i,t}, 1 - clip_eps, 1 + clip_eps) A_i ),
 *   r_{i,t} = exp(logp[i,t] - logp_old[i,t]).
 * Tokens are laid out [n_seq, seq_len]; mask marks the |o_i| response tokens of response i; adv[i] is the
 * group-relative advantage of response i (e3_group_advantage), the same for all its tokens; question q
 * owns the responses [group_offsets[q], group_offsets[q+1]) (sizes differ under the dynamic budget).  A
 * response without tokens contributes 0 but counts in G_q.
 *
 *   logp, logp_old   device float [n_seq * seq_len] (e3_token_logp_entropy outputs of the current and the old policy)
 *   mask             device uint8 [n_seq * seq_len] or NULL (= all ones)
 *   adv              device float [n_seq];  group_offsets: device int64 [n_groups + 1], non-decreasing,
 *                    [0] == 0, [n_groups] == n_seq (a response outside every group contributes nothing)
 *   out_g_logp       NULL or device float [n_seq * seq_len]: dJ/dlogp per token; 0 on tokens outside the mask and
 *                    where the clipped term is the smaller one (A > 0 and r > 1 + eps, or A < 0 and r < 1 - eps).
 *                    This is the g_logp of e3_token_logp_entropy_backward (J is maximised: negate for a loss).
 *   out_objective    device double scalar, required;  out_clip_frac: NULL or device double scalar, the fraction of
 *                    response tokens whose clipped term is active
 *   workspace        e3_workspace_bytes(E3_CALL_GRPO_OBJECTIVE, n_seq, 0, 0) bytes of device scratch, 8-byte aligned
 * All arithmetic is fp64 in a fixed order: results are reproducible, and the clip decision does not depend
 * on fp32 rounding.
 */
E3_API e3_status e3_grpo_objective(const float *logp, const float *logp_old, const uint8_t *mask, int64_t n_seq,
                            int64_t seq_len, const float *adv, const int64_t *group_offsets, int64_t n_groups,
                            float clip_eps, float *out_g_logp, double *out_objective, double *out_clip_frac,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * Algorithm 1 (Dynamic Rollout Budget), host only.  k[i] in [0, 1] is the normalised difficulty
 * rank of question i; out_G[i] receives its rollout count with sum out_G = B * G and
 * G_min <= out_G[i] <= G_max.  Steps as printed: start at G_min, add floor(N_rem k_i / sum k)
 * (capped at G_max), hand the remainder out in descending order of k (ties: lower index first).
 * greedy_mode 0 fills each question to G_max in turn; 1 gives one rollout per question per sweep.
 * sum k == 0 gives every question G.  All pointers are host pointers.
 * Errors: E3_ERR_INFEASIBLE unless G_min <= G <= G_max; E3_ERR_INVALID_ARG for k outside [0,1] or NaN.
 */
E3_API e3_status e3_allocate_budget(const double *k, int64_t B, int32_t G, int32_t G_min, int32_t G_max,
                             int greedy_mode, int32_t *out_G);

/*
 * Difficulty model of Sec. 4.1, host only.  For every question of the dataset (D of them) the caller
 * keeps the cumulative rollout count n_c[i] and the cumulative reward r_c[i] (plain arrays it owns,
 * zero at the start of training; they are the whole state and can be stored as they are).
 *
 * e3_difficulty_accumulate adds one batch: question question_ids[b] was rolled out G[b] times and
 * rewards holds those sum(G) rewards, group after group (the layout of e3_group_advantage).
 * Nothing is changed when an argument is rejected (id outside [0, D), negative G).
 *
 * e3_difficulty_rank, called at the end of an iteration over the dataset, ranks the questions by their
 * average reward r_c[i] / n_c[i] in descending order and writes k[i] = rank(q_i) / D: the question with
 * the highest average reward gets 1/D, the hardest gets 1.  Equal averages keep dataset order; a question
 * that was never rolled out counts as average reward 0.  out_k feeds e3_allocate_budget.
 */
E3_API e3_status e3_difficulty_accumulate(int64_t D, int64_t *n_c, double *r_c, const int64_t *question_ids,
                                   const int32_t *G, const float *rewards, int64_t B);
E3_API e3_status e3_difficulty_rank(int64_t D, const int64_t *n_c, const double *r_c, double *out_k);

/*
 * Curriculum on the budget bounds (Sec. 4.1, settings of Sec. 5.2): G_min = G_max = G at the start; after
 * every finished iteration over the dataset G_max grows and G_min shrinks by `step` (2 in the paper's runs)
 * until G_max_limit / G_min_limit.  epochs_done = number of finished iterations.  Host only.
 * E3_ERR_INFEASIBLE unless G_min_limit <= G <= G_max_limit.
 */
E3_API e3_status e3_budget_curriculum(int32_t G, int32_t step, int32_t G_min_limit, int32_t G_max_limit,
                               int64_t epochs_done, int32_t *G_min, int32_t *G_max);

/* Scheduler state, owned by the caller; plain data, can be copied or stored as is. */
typedef struct {
  double tau;      /* current temperature tau_t (> 0) */
  double H_init;   /* entropy level to hold; NaN or <= 0 = not recorded yet */
  int64_t t;       /* training step, advanced by every successful update */
  int64_t t_anneal;/* first step of the annealing phase */
  int64_t t_max;   /* last training step; t_max <= t_anneal switches annealing off */
  double eta;      /* annealing floor: target entropy goes from H_init to eta * H_init */
  int64_t V;       /* vocabulary size |V| in Eq. "tp_adj" (>= 3) */
  double tau_min;  /* clamp, used when tau_max > 0 */
  double tau_max;
} e3_sched;

/*
 * Temperature scheduler (Eq. "tp_adj" and the annealing equation, Sec. 4.2), host only:
 *   alpha = H_target / H_t,  tau_{t+1} = tau_t (1 + tau_t ln(alpha) / (ln|V| + ln ln|V|)),
 *   H_target = H_init for t < t_anneal, else
 *              H_init [eta + (1 - eta) (1/2) (1 + cos(pi (t - t_anneal) / (t_max - t_anneal)))].
 * The first call with H_init unset records H_init = H_t and keeps tau.  On success the state is
 * updated (tau, t) and *tau_next = tau.  H_t <= 0 or not finite, tau <= 0, V < 3, or an update that
 * would leave tau <= 0 return E3_ERR_INVALID_ARG and change nothing.
 */
E3_API e3_status e3_update_temperature(e3_sched *s, double H_t, double *tau_next);

/*
 * The same scheduler with the logit gap Delta of App. A estimated instead of replaced by ln|V| + ln ln|V|
 * (Eq. "tp_relation_1": tau_1 = tau_0 (1 + tau_0 ln(alpha) / Delta)), host only.  App. A models a row as one
 * dominant logit and N-1 others at gap Delta, whose entropy is H = (N-1) x exp(-x) with x = Delta / tau_0.
 * e3_entropy_gap returns the root x >= 1 of that equation for a measured entropy H (NaN when H <= 0, not
 * finite, N < 3 or H > (N-1)/e, where the model has no root).  e3_update_temperature_gap then sets
 *   tau_{t+1} = tau_t (1 + ln(alpha) / x),   alpha = H_target / H_t,
 * with the state, first call, clamp and errors of e3_update_temperature; an H_t without a root is
 * E3_ERR_INVALID_ARG too.
 */
E3_API double e3_entropy_gap(double H, int64_t N);
E3_API e3_status e3_update_temperature_gap(e3_sched *s, double H_t, double *tau_next);

/* Target entropy the scheduler holds at step s->t (H_init before annealing starts). */
E3_API double e3_anneal_target(const e3_sched *s);

/*
 * Test hook, not for production use.  The next row call of this process (e3_sample or
 * e3_token_logp_entropy) leaves the 4 KiB tile number `tile` of its logits (row * ceil(V * esize / 4096)
 * + tile within the row) uncopied, and its waits give up after wait_ns nanoseconds instead of two seconds.
 * The consumer of that tile then runs into the bounded wait: the call returns as usual, the rows of the
 * thread block concerned read token -1 / NaN, and E3_STATUS_TIMEOUT appears in the status word.  One shot.
 */
E3_API void e3_test_arm_stall(int64_t tile, uint64_t wait_ns);

/*
 * Measurement aid: reads `bytes` (a multiple of 16) of device memory at `buf` (16-byte aligned) once, with a
 * plain grid of four thread blocks per SM that only adds the words up -- the practical read-only ceiling
 * of the device, against which the benchmark reports the row kernels.  `scratch`: device memory of at least
 * 8 bytes per thread block (E3_PROBE_SCRATCH_BYTES covers every device), receives one checksum per block.
 * E3_ERR_INVALID_ARG for NULL or misaligned arguments, E3_ERR_WORKSPACE for a scratch that is too small.
 */
#define E3_PROBE_SCRATCH_BYTES 65536
E3_API e3_status e3_probe_read(const void *buf, size_t bytes, void *scratch, size_t scratch_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* E3_H_ */
