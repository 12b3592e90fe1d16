/*
 * echo.h — C ABI of the B200 rollout-generation library.
 *
 * The library implements the step that a rollout worker of the ECHO-2 paper
 * (arXiv 2602.02192) spends its time in: for each prompt x, sample G responses
 * y ~ pi_v(. | x) from the installed policy snapshot v, record the sampler's
 * per-token log-probabilities, and tag every trajectory with v (Section 4.2
 * "Rollout generation"; Algorithm 1, rollout plane).  A newer snapshot can be
 * installed while generation continues on the previous one (Section 4.3: a
 * worker switches its local version only once installation is complete), and
 * rewards are normalised per group for GRPO (Appendix F, group-wise
 * normalisation).
 *
 * Conventions
 *   - Every call returns an int: ECHO_OK (0) or a negative ECHO_ERR_* code.
 *     Nothing throws, aborts or exits.  A failed call leaves the context usable.
 *   - "dev" pointers are CUDA device pointers on the context's device; "host"
 *     pointers are ordinary host memory unless stated otherwise.
 *   - All matrices are row-major.  Weight matrices are bf16, shape [out, in].
 *   - The caller owns every buffer it passes, including the arena and the CUDA
 *     stream.  The library never calls cudaMalloc/cudaFree after echo_create
 *     (echo_create itself allocates only streams and events, no device memory).
 *   - Work is enqueued on the stream given to echo_create.  Device outputs are
 *     valid once that stream (or echo_sync) has been synchronised.
 *   - One context serves one GPU and is not thread-safe; use one context per
 *     thread or serialise calls.
 */
#ifndef ECHO_B200_H
#define ECHO_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- error codes -------------------------------------------------------- */
#define ECHO_OK                 0
#define ECHO_ERR_INVALID       -1   /* null pointer, size out of the configured range, T <= 0, ... */
#define ECHO_ERR_ARENA         -2   /* arena too small or misaligned                                */
#define ECHO_ERR_NO_POLICY     -3   /* rollout requested before any echo_load_policy                */
#define ECHO_ERR_VERSION       -4   /* version not strictly greater than every earlier one          */
#define ECHO_ERR_BUSY          -5   /* an install is still pending: a third live version would
                                       exceed what the weight buffers can hold                      */
#define ECHO_ERR_CUDA          -6   /* a CUDA call failed; text in echo_last_error                  */
#define ECHO_ERR_DEVICE_CHECK  -7   /* a kernel's own range check tripped (status word set)         */
#define ECHO_ERR_TIMEOUT       -8   /* a bounded device-side wait ran out                           */
#define ECHO_ERR_UNSUPPORTED   -9   /* shape the kernels do not cover (e.g. head_dim not 64/128)    */

typedef struct echo_ctx echo_ctx;   /* opaque */

/* Decoder shape and capacity limits, fixed at echo_create. */
typedef struct echo_config {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
  float   rms_eps;            /* e.g. 1e-6 */
  float   rope_theta;         /* e.g. 1e4  */
  int32_t kv_page_size;       /* tokens per KV page; 16 */
  int32_t max_prompts;        /* largest P of one echo_rollout call */
  int32_t max_G;              /* largest group size G               */
  int32_t max_prompt_len;     /* row width of the prompts array     */
  int32_t max_new_tokens;     /* largest T                          */
  int32_t n_weight_buffers;   /* 2: a new snapshot installs while the old one serves
                                 (staleness bound 1); 1: installs block generation  */
  int32_t eos_id;             /* -1: every sequence produces exactly T sampled tokens.  A token id in
                                 [0, vocab): a sequence that emits it is finished; its later positions
                                 hold eos_id with log-probability 0 (Section 5.1 generates up to a
                                 maximum length; responses end earlier at the end token).  Finished
                                 sequences leave the activation rows of the later steps; within one
                                 echo_rollout call nothing takes their place (echo_rollout_queue
                                 admits further prompts instead). */
  float   top_p;              /* nucleus sampling (Section 5.1 samples with top-p 0.95): tokens are ranked
                                 by probability (ties: lower id first), the shortest prefix whose mass
                                 reaches top_p is kept, and the recorded log-probability is renormalised
                                 over it.  0 or 1: no truncation; otherwise in (0, 1). */
  int32_t half_layers;        /* The paper states no precision for its rollout engine (Section 5.1 names the
                                 model family only).  In the first half_layers layers every 16-bit operand
                                 (projection inputs and the installed projection weights, queries, cached
                                 keys and values, attention probabilities) is IEEE half (11-bit significand)
                                 instead of bf16 (8-bit); accumulation, residual stream and softmax are fp32
                                 everywhere.  Same bytes, same tensor-core rate.  bf16 weights convert to
                                 half exactly unless |w| < 2^-17 (then the error is at most 2^-25) or
                                 |w| > 65504 (refused by nothing: it would become inf).  Activations of these
                                 layers must stay below 65504.  0: bf16 everywhere.  In [0, n_layers]. */
  int32_t kv_pages;           /* Pages of the KV pool.  0: enough for max_prompts groups of max_G samples at
                                 the longest prompt and max_new_tokens (no call can run out).  Smaller
                                 values are for echo_rollout_queue, which hands pages to a sequence when it
                                 is admitted and takes them back when it has ended, so that max_prompts can
                                 count more group slots than the pool could hold at full length; at least
                                 one group at full length.  echo_rollout refuses a call whose plan does
                                 not fit the pool (ECHO_ERR_INVALID). */
  int32_t queue_max_live;     /* echo_rollout_queue admits a further group only while the sequences that
                                 have not ended, plus its max_G samples, stay within this number (the
                                 activation rows a decode step's projections run on).  0: no limit
                                 other than slots and pages. */
  int32_t queue_optimistic;   /* 0: echo_rollout_queue gives a sequence the pages of its longest possible
                                 continuation when it is admitted, so the pool can never run dry.
                                 n in 1..8: pages are handed out as positions are reached (every 16 decode
                                 steps, for the 16 to come), a group is admitted while the pool has room
                                 for it plus n - 1 further windows of everything live (a page per sequence
                                 and window; 3 is a sensible value), and when the pool cannot cover the next steps
                                 the most recently admitted groups are evicted: their pages return, their
                                 prompts go back to the head of the queue and they are generated again
                                 from their first token later (the same tokens: noise streams are keyed
                                 by sequence id and token index). */
} echo_config;

/* One snapshot: a pointer per tensor, bf16, row-major [out, in]; each pointer
 * is device memory or page-locked host memory.  Per-layer entries are arrays of
 * n_layers pointers (the arrays themselves live in host memory).
 *   embed [vocab, d]  lm_head [vocab, d]  final_norm [d]
 *   wq [Hq*hd, d]  wk [Hkv*hd, d]  wv [Hkv*hd, d]  wo [d, Hq*hd]
 *   w_gate [F, d]  w_up [F, d]  w_down [d, F]  attn_norm [d]  mlp_norm [d] */
typedef struct echo_weights {
  const void *embed, *lm_head, *final_norm;
  const void *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *w_gate, *const *w_up, *const *w_down;
  const void *const *attn_norm, *const *mlp_norm;
} echo_weights;

/* Counters of the most recent echo_rollout on this context. */
typedef struct echo_stats {
  int64_t version_served;     /* tag of the last rollout                        */
  int64_t tokens_generated;   /* P*G*T of the last rollout                      */
  int64_t kernels_launched;   /* this library's kernel launches in that rollout
                                 (graph replays count the kernels they contain) */
  int64_t decode_steps;       /* T-1                                            */
  int64_t n_pages;            /* KV pages the plan used                         */
  float   install_ms;         /* duration of the last completed install (device) */
  float   prefill_ms;         /* last rollout: prompt prefill + first token (device time; valid once
                                 the rollout has finished, else 0)                                */
  float   decode_ms;          /* last rollout: the T-1 decode steps (device time; same condition)  */
  float   last_step_rows;     /* activation rows of the last decode step's projections: P*G, or fewer
                                 once sequences have ended (with an end token the live sequences are
                                 packed and the row count follows their number downwards) */
  int64_t queue_evictions;    /* echo_rollout_queue with queue_optimistic: groups evicted and generated again */
} echo_stats;

/* Bytes of device memory echo_create needs for this configuration (weight
 * buffers, KV page pool, activations, logits, tables).  0 if cfg is invalid. */
size_t echo_arena_bytes(const echo_config *cfg);

/* Create a context on CUDA device `device`.  `arena` is device memory of at
 * least echo_arena_bytes(cfg) bytes, 256-byte aligned, owned by the caller and
 * kept alive until echo_destroy.  `cuda_stream` is a cudaStream_t (may be 0 for
 * the legacy default stream, which cannot be graph-captured: decode steps are
 * then launched kernel by kernel). */
int echo_create(const echo_config *cfg, int device, void *arena, size_t arena_bytes,
                void *cuda_stream, echo_ctx **out);
int echo_destroy(echo_ctx *ctx);

/* Install snapshot `version` (Section 4.2 "Policy publication"; Section 4.3;
 * Algorithm 1: the worker updates its local version once a newer snapshot is
 * fully installed).  The copy into the inactive weight buffer is enqueued on the
 * library's own copy stream, ordered after every rollout that still reads that
 * buffer, and the call returns at once; generation on the previous version
 * continues meanwhile.  The source tensors must stay alive and unchanged until
 * the install has completed (echo_wait_policy, echo_sync, or a later rollout
 * tagged with this version).  Versions must strictly increase (else
 * ECHO_ERR_VERSION).  With an install pending a further offer is refused with
 * ECHO_ERR_BUSY.  With n_weight_buffers == 1 the install overwrites the only
 * buffer: it is ordered after all enqueued rollouts and the next rollout waits
 * for it. */
int echo_load_policy(echo_ctx *ctx, const echo_weights *w, int64_t version);

/* Block the host until a pending install, if any, has completed. */
int echo_wait_policy(echo_ctx *ctx);

/* Generate G completions of T = max_new_tokens tokens for each of P prompts
 * (Section 4.2 "Rollout generation": y ~ pi_v(. | x); the rollout multiplicity
 * and temperature of Section 5.1).
 *   prompts      dev  int32 [P][cfg.max_prompt_len]   (row p uses its first prompt_lens[p] ids)
 *   prompt_lens  host int32 [P], each in [1, max_prompt_len]
 *   temperature  > 0
 *   seed         keys the Philox4x32-10 streams: key = (seed lo, seed hi),
 *                counter = (v >> 2, j, s, 0), word v & 3 for vocab id v, new-token
 *                index j, sequence id s = p*G + g
 *   out_tokens   dev  int32 [P][G][T]
 *   out_logprobs dev  fp32  [P][G][T]: log-probability of each token under the
 *                temperature-scaled distribution it was drawn from (the sampler
 *                policy of Appendix F's truncated importance ratio)
 *   out_versions host int64 [P][G]: the snapshot version every token of that
 *                trajectory was generated under; filled before the call returns.
 * The version served is the newest whose install had completed when the call
 * began; an install still running does not affect this rollout.  The prompt is
 * prefilled once per prompt into KV pages shared by its G samples.  The call
 * returns after enqueueing; outputs are stream-ordered. */
int echo_rollout(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens,
                 int32_t P, int32_t G, int32_t max_new_tokens, float temperature,
                 uint64_t seed, int32_t *out_tokens, float *out_logprobs,
                 int64_t *out_versions);

/* The same rollout over a QUEUE of prompts longer than the context holds at once (Section 5.1: responses
 * of up to 8192 tokens that end at very different lengths; Section 3.1 counts rollouts per unit time):
 * continuous refill.  The context's max_prompts groups are slots; when every sample of a slot has ended
 * (end token, or all T tokens generated) the next prompt of the queue is prefilled into the slot between
 * two decode steps, while the other slots keep decoding.  Sequence (p, g) keeps the noise stream and the
 * output row of its id p*G + g (plus the sequence base) and counts its token index from the step it was
 * admitted at, so every sequence gets exactly the tokens echo_rollout gives it in a call that holds all
 * n_prompts at once; only the order in which the work runs differs.
 *   prompts      dev  int32 [n_prompts][cfg.max_prompt_len], prompt_lens host int32 [n_prompts];
 *                n_prompts >= 1, not bounded by max_prompts
 *   out_tokens / out_logprobs  dev [n_prompts][G][T]; positions after a sequence's end token hold the
 *                end token / 0, as in echo_rollout
 *   out_versions host int64 [n_prompts][G] (one version for the whole call)
 *   forced_tokens NULL, or dev int32 [n_prompts][G][T]: teacher-forced as in echo_rollout_forced (the
 *                sequences then end where the given tokens hold the end token)
 * The host follows the ended flags once every 16 decode steps (it waits for the GPU at those points), so
 * the call returns when the last steps are enqueued, not before.  Needs the tensor-core decode attention
 * (else ECHO_ERR_UNSUPPORTED).  echo_get_stats().decode_steps reports the steps the queue took. */
int echo_rollout_queue(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens,
                       int32_t n_prompts, int32_t G, int32_t max_new_tokens, float temperature,
                       uint64_t seed, const int32_t *forced_tokens, int32_t *out_tokens,
                       float *out_logprobs, int64_t *out_versions);

/* Teacher-forced variant: step j feeds forced_tokens[p][g][j] (dev int32
 * [P][G][T]) instead of the sampled token.  out_tokens[p][g][j] is the token
 * that would have been sampled at step j, out_logprobs[p][g][j] the
 * log-probability of the forced token.  Same noise streams as echo_rollout. */
int echo_rollout_forced(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens,
                        int32_t P, int32_t G, int32_t max_new_tokens, float temperature,
                        uint64_t seed, const int32_t *forced_tokens, int32_t *out_tokens,
                        float *out_logprobs, int64_t *out_versions);

/* Learner-side scoring (Appendix F: the likelihood ratio and the truncated importance ratio need
 * log pi_theta(y_t | x, y_<t) for whole trajectories from the buffer).  Same result as the
 * out_logprobs of echo_rollout_forced for the same given tokens, but computed in prefill-shaped passes
 * (the prompt once per group, then every sequence's given tokens as rows of large chunks with causal
 * attention): the weights are streamed once per 2048 rows instead of once per decode step.
 *   tokens       dev int32 [P][G][T]: the given trajectories
 *   out_logprobs dev fp32  [P][G][T]: log-probability of tokens[p][g][j] under softmax(z / temperature)
 *                of the installed snapshot (the full distribution: top_p is not applied); with an end
 *                token configured, positions after a sequence's first end token score 0.
 * Arguments otherwise as for echo_rollout; asynchronous on the context's stream. */
int echo_score(echo_ctx *ctx, const int32_t *prompts, const int32_t *prompt_lens, int32_t P, int32_t G,
               int32_t max_new_tokens, float temperature, const int32_t *tokens, float *out_logprobs,
               int64_t *out_versions);

/* Turn-aware response mask (Appendix F, "Turn-Aware Masking"): with u_t = [x_t == turn_start_id] and
 * c_t = u_0 + ... + u_t, m_t = [c_t > 1] * [c_t odd] selects the tokens of assistant turns after the
 * system prompt.  tokens dev int32 [n][T] -> out_mask dev uint8 [n][T].  With shift_to_targets != 0 the
 * mask is aligned with next-token targets y_t = x_{t+1}: out[t] = m_{t+1}, out[T-1] = 0.  The result is
 * the `mask` argument of echo_grpo_surrogate.  Asynchronous on the stream; needs no context. */
int echo_turn_mask(const int32_t *tokens, int32_t n, int32_t T, int32_t turn_start_id, int32_t shift_to_targets,
                   uint8_t *out_mask, void *cuda_stream);

/* echo_rollout with every buffer in HOST memory (prompts, outputs): copies the
 * prompts in, runs the rollout, copies tokens and log-probabilities out and
 * synchronises.  Page-locked buffers make the copies asynchronous. */
int echo_rollout_host(echo_ctx *ctx, const int32_t *prompts_host, const int32_t *prompt_lens,
                      int32_t P, int32_t G, int32_t max_new_tokens, float temperature,
                      uint64_t seed, int32_t *out_tokens_host, float *out_logprobs_host,
                      int64_t *out_versions);

/* GRPO group-wise normalisation (Appendix F): for each of P groups of G rewards,
 * A = (R - mean) / (std + eps), std with the (G-1) divisor as in the listing
 * printed under that equation, eps added to the std.  rewards / out_adv: dev
 * fp32 [P][G] (may alias).  G < 2 is ECHO_ERR_INVALID.  Runs on `cuda_stream`
 * (a cudaStream_t, may be 0); needs no context. */
int echo_group_advantage(const float *rewards, int32_t P, int32_t G, float eps,
                         float *out_adv, void *cuda_stream);

/* Learner-side objective of Appendix F ("GRPO-Style Policy Gradient Objective"), forward value per
 * sequence: with rho_t = exp(logp_new - logp_old), the truncated importance ratio
 * w_t = min(exp(logp_old - logp_sampler), C) and the response mask m_t,
 *   out[i] = sum_t m_t w_t min(rho_t A_i, clip(rho_t, 1 - eps_clip, 1 + eps_clip) A_i) / sum_t m_t
 * (0 for an empty mask; without the KL term: echo_grpo_objective adds it).
 * logp_* dev fp32 [n][T] are log-probabilities of the taken tokens (logp_sampler is what
 * echo_rollout recorded, the other two come from echo_rollout_forced under the respective
 * weights), adv dev fp32 [n] (echo_group_advantage), mask dev uint8 [n][T] or NULL (all ones),
 * out dev fp32 [n].  eps_clip >= 0, C > 0.  Asynchronous on the stream. */
int echo_grpo_surrogate(const float *logp_new, const float *logp_old, const float *logp_sampler,
                        const float *adv, const uint8_t *mask, int32_t n, int32_t T, float eps_clip,
                        float C, float *out, void *cuda_stream);

/* The same objective with its KL regulariser (Appendix F, the equation for J-bar:
 * ... - beta * D_KL(pi_theta || pi_ref)).  The appendix names no estimator; a rollout record holds
 * log-probabilities of the taken tokens only, so the divergence enters as the per-token estimate
 *   k_t = pi_ref(y_t)/pi_theta(y_t) - log(pi_ref(y_t)/pi_theta(y_t)) - 1 = exp(d) - d - 1,
 *   d = logp_ref - logp_new  (non-negative; its mean over y_t ~ pi_theta is the exact divergence),
 * inside the masked mean and under the truncated ratio that multiplies the whole of J-bar:
 *   out[i] = sum_t m_t w_t (min(rho_t A_i, clip(rho_t) A_i) - beta k_t) / sum_t m_t.
 * logp_ref dev fp32 [n][T] (echo_score / echo_rollout_forced under the reference weights); the other
 * arguments as in echo_grpo_surrogate; beta >= 0.  Asynchronous on the stream. */
int echo_grpo_objective(const float *logp_new, const float *logp_old, const float *logp_sampler,
                        const float *logp_ref, const float *adv, const uint8_t *mask, int32_t n,
                        int32_t T, float eps_clip, float C, float beta, float *out, void *cuda_stream);

/* Offset of this context's sequence ids in the noise streams: sequence (p, g) of later rollouts draws
 * from the Philox stream of id base + p*G + g.  Rollout workers are independent and share nothing but
 * the snapshot and the buffer (Section 4.1), so a set of prompts can be cut by prompt over several
 * contexts or GPUs; with base = (index of the context's first prompt) * G every sequence gets the
 * tokens it would get in one call over the whole set.  Default 0. */
int echo_set_sequence_base(echo_ctx *ctx, uint32_t base);

/* Block until everything this context enqueued (rollouts and installs) is done;
 * reports ECHO_ERR_DEVICE_CHECK / ECHO_ERR_TIMEOUT if a kernel flagged one. */
int echo_sync(echo_ctx *ctx);

int echo_get_stats(echo_ctx *ctx, echo_stats *out);

/* Sampled per-kernel timing.  With every_n_steps = n > 0, every n-th decode step of later
 * rollouts is launched kernel by kernel (not as a graph replay) with CUDA events around the
 * attention launches, the dense projections, the sampler and the whole step; 0 turns it off;
 * -1 times the prompt prefill that way instead (reported as step 0; the decode steps run untimed).
 * echo_profile_read waits for the stream and returns, for each sampled step of the most
 * recent rollout, its index in steps[i] (host int32) and four summed durations in
 * milliseconds in ms[4*i + c] (host fp32): c = 0 attention, 1 projections, 2 sampler,
 * 3 whole step.  capacity is the number of steps both arrays can hold; *n_out receives the
 * number of sampled steps (pass steps = ms = NULL to query it). */
int echo_profile_config(echo_ctx *ctx, int32_t every_n_steps);
int echo_profile_read(echo_ctx *ctx, int32_t *steps, float *ms, int32_t capacity, int32_t *n_out);

/* Copy the page table of the most recent rollout to host memory:
 * int32 [P*G][width]; entries past a sequence's last page are -1.  `width` and
 * the number of rows are returned through the pointers; `out` may be NULL to
 * query them.  n is the capacity of `out` in int32 elements. */
int echo_debug_page_table(echo_ctx *ctx, int32_t *out, size_t n, int32_t *rows, int32_t *width);

/* Parity hook: from now on, rollouts on this context copy the fp32 residual stream x as it enters
 * layer `layer` and as it leaves it (the decoder layer of Section 5.1's model family: attention block
 * and MLP block, each added to x) into caller buffers, so that a test can feed one layer's own input
 * to a reference implementation of that layer and compare outputs without the error of the layers
 * before it.  pre_in / pre_out: dev fp32 [n_prompt_tokens][d_model], rows in prefill order (prompt 0's
 * tokens, then prompt 1's, ...).  dec_in / dec_out: dev fp32 [T-1][P*G][d_model], decode step j
 * (the one that feeds token j-1) at index j-1.  Any pointer may be NULL.  layer = -1 turns it off.
 * The buffers must stay valid while rollouts run; d_model must be a multiple of 4. */
int echo_debug_capture(echo_ctx *ctx, int32_t layer, float *pre_in, float *pre_out, float *dec_in, float *dec_out);

/* Read-only streaming probe (measurement aid; the paper has no counterpart): a kernel that reads
 * `bytes` (a multiple of 16) of device memory at `buf` once per pass, with 16-byte loads from every
 * SM, and writes nothing.  Decode attention and weight streaming are read-only streams; a copy, the
 * usual bandwidth yardstick, also writes.  One warm-up pass, then `repeats` (1..1000) passes between
 * two events; *ms_per_pass (host) = their mean duration.  scratch: dev, 4 bytes.  Synchronises. */
int echo_probe_read_bandwidth(const void *buf, size_t bytes, int32_t repeats, void *scratch, float *ms_per_pass,
                              void *cuda_stream);

/* Wait-limit probe.  Every device-side wait of this library (TMA pipelines, accumulator hand-over) is
 * bounded: when the limit runs out the kernel records it, drains and returns, and the host reports
 * ECHO_ERR_TIMEOUT.  This call runs that wait routine alone, in a one-warp kernel, on a barrier that
 * nothing ever signals, with the given limit (1 ns .. 0.1 s) in place of the library's one second:
 * the expected result is ECHO_ERR_TIMEOUT, with the time the warp waited in *waited_ns (host, may be
 * NULL).  scratch: dev, 16 bytes, 8-byte aligned.  Synchronises the stream. */
int echo_debug_wait_limit(uint64_t limit_ns, void *scratch, uint64_t *waited_ns, void *cuda_stream);

/* The KV page plan of a rollout, computed on the host without a context or a GPU (the same
 * routine echo_rollout uses).  prompt_lens host int32 [P].  Writes out_table (host int32
 * [(P*G + P)][*width], capacity in elements): rows 0..P*G-1 are the sequences' page tables
 * (sequence s = p*G + g), rows P*G..P*G+P-1 the pages each prompt's prefill writes; unused
 * entries are -1.  *width = logical pages per row, *n_pages = physical pages used.  Pass
 * out_table = NULL to query width and n_pages. */
int echo_plan_page_table(const int32_t *prompt_lens, int32_t P, int32_t G, int32_t T, int32_t page_size,
                         int32_t *out_table, size_t capacity, int32_t *width, int32_t *n_pages);

/* ---- host-side closed forms of the control plane (no GPU work) -------------
 * Section 3.1, capacity requirement: the aggregate rollout throughput (rollouts/s) that keeps the
 * learner busy when it consumes R trajectories per step of T_train seconds and publishes every
 * kappa steps, with T_bcast seconds from publication to a usable snapshot:
 *   mu_min = kappa R / (kappa T_train - T_bcast).   ECHO_ERR_UNSUPPORTED if kappa T_train <= T_bcast. */
int echo_mu_min(double kappa, double R, double T_train, double T_bcast, double *out);
/* Section 3.1 ("Linking (S, kappa)") / Appendix on staleness: conservative bound
 *   Delta_max <= kappa + ceil((T_bcast + R / mu_pool) / T_train) - 1. */
int echo_staleness_bound(int32_t kappa, double T_bcast, double R, double mu_pool, double T_train,
                         int32_t *out);
/* Section 3.2, greedy provisioning: rank workers by unit throughput cost rho_i = cost_i / mu_i
 * (equal rho: lower index first) and activate the cheapest prefix whose cumulative throughput
 * reaches mu_target.  active[n] (host) receives 0/1; n_active and total_cost may be NULL.
 * ECHO_ERR_UNSUPPORTED (with every worker active) if the whole pool stays below the target. */
int echo_greedy_provision(const double *mu, const double *cost, int32_t n, double mu_target,
                          uint8_t *active, int32_t *n_active, double *total_cost);
/* Section 4.2, replay buffer: a trajectory tagged v is admissible at learner version v_t under
 * the staleness budget S iff v_t - S <= v <= v_t.  Returns 1 or 0. */
int echo_admissible(int64_t v, int64_t v_t, int64_t S);

/* Appendix C.3, "Worker scoring": Score = Decay (0.5 Speed + 0.35 Success + 0.15 Stability) with
 *   Speed = 100 (log10(avg_speed) - 3) / 5 (avg_speed in bits per second: 100 at 100 Mbit/s; clamped to
 *   [0, 100]: the appendix says it saturates at 100, the lower clamp is this library's reading),
 *   Success = 100 success_rate, Stability = 0 after more than 3 consecutive failures, else
 *   100 min(succ_count / 10, 1), Decay = 1 - min(elapsed_s / 600, 0.3). */
int echo_peer_score(double avg_speed, double success_rate, int32_t succ_count, int32_t consecutive_failures,
                    double elapsed_s, double *out);
/* Section 4.3 / Appendix C.3, "Chain assembly": N_ch = floor(B0 / Bw) forwarding chains (at least 1, at
 * most n); the N_ch best-scored workers are the first-hop seeds, the others are appended to the chain
 * tails in rank order, round-robin over the chains (equal scores: lower index first).  chain_of[i] and
 * hop_of[i] (host int32 [n]) receive worker i's chain and its hop (0 = seed, fed by the learner); its
 * parent is the worker of the same chain at hop - 1, its only child the one at hop + 1 (fan-out 1). */
int echo_chain_assemble(const double *score, int32_t n, double B0, double Bw, int32_t *chain_of, int32_t *hop_of,
                        int32_t *n_chains);
/* Section 4.3, chunked store-and-forward streaming along one chain, as a timeline: the time at which
 * the worker at hop `hop` holds the whole snapshot of `bytes` when it is cut into chunks of
 * chunk_bytes (the last may be shorter), every link carries Bw_bytes_per_s, a link forwards a chunk
 * once it has arrived completely upstream, and each hop adds hop_latency_s per chunk.  With equal
 * chunks and no latency: (number of chunks + hop) chunk times - a pipeline fill, then line rate. */
int echo_chain_arrival_time(double bytes, double chunk_bytes, double Bw_bytes_per_s, int32_t hop,
                            double hop_latency_s, double *out);

/* ---- stand-alone kernel entry points (used by the parity tests) ---------- */

/* Philox words and uniforms exactly as the sampler draws them: for vocab ids
 * v in [v0, v0+n), out_words[i] (dev uint32) and out_uniform[i] (dev fp32,
 * w = (float(word) + 0.5f) * 2^-32) for sequence s, new-token index j. */
int echo_debug_noise(uint64_t seed, uint32_t s, uint32_t j, uint32_t v0, uint32_t n,
                     uint32_t *out_words, float *out_uniform, void *cuda_stream);

/* Sampler alone: for r in [0, R): sequence id seq_ids[r] (dev int32, or NULL for
 * seq id r) draws new-token index j from logits row (r / rows_per_logit_row) of
 * dev fp32 logits [.][V]; writes out_tokens[r] (dev int32) and out_logprobs[r]
 * (dev fp32, log-prob of forced[r] if forced != NULL else of the drawn token). */
int echo_sample(const float *logits, int32_t R, int32_t V, int32_t rows_per_logit_row,
                const int32_t *seq_ids, uint32_t j, float temperature, uint64_t seed,
                const int32_t *forced, int32_t *out_tokens, float *out_logprobs,
                void *cuda_stream);

/* echo_sample with nucleus truncation (0 < top_p < 1; top_p = 1 equals echo_sample).  A first
 * kernel finds each logits row's cut (the last member of the nucleus) by histograms of probability
 * mass over score bins, the sampler then draws among the ids at or before the cut and renormalises
 * the log-probability over them; a forced token outside the nucleus scores -inf.  `cut_scratch`:
 * dev, 8 bytes per logits row ((R + rows_per_logit_row - 1) / rows_per_logit_row rows). */
int echo_sample_top_p(const float *logits, int32_t R, int32_t V, int32_t rows_per_logit_row,
                      const int32_t *seq_ids, uint32_t j, float temperature, float top_p, uint64_t seed,
                      const int32_t *forced, int32_t *out_tokens, float *out_logprobs, void *cut_scratch,
                      void *cuda_stream);

/* Decode-step attention alone (paged GQA with the group's prompt pages read once for all G
 * samples).  B = P*G sequences, sequence s = p*G + g.
 *   q           dev bf16 [B][Hq][hd]            (already rotated)
 *   kv_pool     dev bf16 [n_pages][Hkv][2][16][hd]: per page and kv head, 16 K rows then 16 V rows
 *   page_table  dev int32 [B][pt_width]: physical page of each logical page of a sequence
 *   row_pos     dev int32 [B]: position of the newest token of each sequence (keys 0..row_pos)
 *   full_pages  dev int32 [B]: leading pages shared by the whole group (same value for its G
 *               sequences; the shared pages are taken from the group's first sequence)
 *   scratch     dev, echo_decode_attention_scratch_bytes(B, Hq, hd) bytes, 256-byte aligned:
 *               the prefix partial results handed from the first kernel to the second, a status
 *               word and the item counter of the second kernel (cleared by the call itself)
 *   out         dev bf16 [B][Hq][hd]
 *   operand_format  0: q, kv_pool and out hold bf16 values; 1: IEEE half (echo_config.half_layers)
 *   kernel_choice   0: the kernels a rollout uses; bit 0: one suffix CTA per (sequence, kv head) at every
 *               length; bit 1: one prefix CTA per 16-row tile of a group's query rows
 * hd must be 64 or 128, pages hold 16 tokens.  Synchronises the stream and returns
 * ECHO_ERR_DEVICE_CHECK if a page id was out of range. */
size_t echo_decode_attention_scratch_bytes(int32_t B, int32_t Hq, int32_t hd);
int echo_decode_attention(const void *q, const void *kv_pool, int32_t n_pages, const int32_t *page_table,
                          int32_t pt_width, const int32_t *row_pos, const int32_t *full_pages, int32_t P,
                          int32_t G, int32_t Hq, int32_t Hkv, int32_t hd, void *scratch, size_t scratch_bytes,
                          void *out, int32_t operand_format, int32_t kernel_choice, void *cuda_stream);

/* Dense projection alone, on the tcgen05 tensor cores with fp32 accumulation:
 *   epilogue 0:  Y[M][N] (dev fp32)  = X[M][K] (dev bf16) * W[N][K]^T (dev bf16)
 *   epilogue 1:  Y[M][N] (dev fp32) += X * W^T                        (residual add)
 *   epilogue 2:  Y[M][N] (dev bf16)  = silu(X * Wg^T) * (X * Wu^T), W = [Wg; Wu] of shape [2N][K]
 * K must be a multiple of 8, M in [1, 4096]; all pointers 256-byte aligned.  The kernel splits
 * tiles along K across CTAs and needs scratch memory for the partial sums: `workspace` is
 * device memory of at least echo_gemm_workspace_bytes(M) bytes, owned by the caller, used only
 * during the call's kernels.  `impl`: 0 = tensor-core kernel (cluster split-K for few output
 * tiles, persistent stream-K otherwise), 2 = always the persistent stream-K kernel, 100 + s =
 * cluster split-K by s in [1, 8] (partials summed in a fixed order), 200 + s = s independent
 * k-slices per tile that add their partial sums into Y in memory (s = 0: as many as fill the GPU;
 * faster, but the order of the fp32 additions varies from run to run; epilogues 0 and 1),
 * 300 + s = the SM-pair kernel (2-CTA MMAs; more than 64 rows only, else ECHO_ERR_UNSUPPORTED)
 * with s k-slices per tile added into Y in memory (s = 0: as many as give every SM pair a tile),
 * 1 = plain SIMT reference kernel (epilogues 0 and 1 only; needs no workspace).
 * Adding 1000 to `impl` says that W is not row-major but in the block-tiled layout that
 * echo_retile_weights writes (the layout echo_load_policy keeps the policy's matrices in).
 * Adding 2000 says that X and W (and the output of epilogue 2) hold IEEE half values instead of
 * bf16 (the operand format of echo_config.half_layers); the arithmetic is otherwise the same. */
size_t echo_gemm_workspace_bytes(int32_t M);
int echo_gemm_bf16(const void *X, const void *W, void *Y, int32_t M, int32_t N, int32_t K,
                   int32_t epilogue, int32_t impl, void *workspace, size_t workspace_bytes,
                   void *cuda_stream);

/* Block-tiled weight layout (the rollout plane's policy install, Section 4.3, leaves the layout of
 * the installed snapshot to the worker).  A matrix [rows][cols] is stored as 128-row x 64-column
 * blocks, each block contiguous (16 KiB), ordered [row block][column block], partial blocks
 * padded with zeros: element (n, k) is at ((n/128 * ceil(cols/64) + k/64) * 128 + n%128) * 64 + k%64.
 * A gate/up pair for epilogue 2 is two such matrices back to back (gate, then up).
 * echo_retile_weights copies row-major `src` (dev, or host memory the device can address;
 * cols a multiple of 8, 16-byte aligned) into `dst` (dev, echo_tiled_weight_bytes(rows, cols)
 * bytes, 256-byte aligned), asynchronously on the stream. */
size_t echo_tiled_weight_bytes(int64_t rows, int64_t cols);
int echo_retile_weights(const void *src, int64_t rows, int64_t cols, void *dst, size_t dst_bytes,
                        void *cuda_stream);

/* echo_gemm_bf16 for callers that cannot allocate device memory (code that runs inside an
 * allocator hook, a plug-in that is given tensors but no allocator, a process whose device
 * memory another runtime has reserved).  The paper has no counterpart of this call.  Same
 * arithmetic and epilogues as echo_gemm_bf16, but the split-tile scratch is a fixed array
 * inside the library (about 6 MiB of device memory on every GPU that loads the library, held
 * until the process exits), so no workspace is passed and nothing is allocated or freed, by
 * this call or by anything it calls.
 *   - M is limited to 32 activation rows; a larger M returns ECHO_ERR_UNSUPPORTED and does
 *     nothing.  X, W, Y as for echo_gemm_bf16 (Y must be 16-byte aligned).
 *   - The first call on each device looks up the array's device address and sets kernel
 *     attributes; make that first call with the device current and before any stream capture.
 *   - All calls share the one array.  The call clears the part that must start at zero, but
 *     two calls whose kernels can overlap on the GPU (different streams or host threads) race
 *     on it: keep calls on one stream, or order them with events.
 *   - X, W and Y must be 16-byte aligned (else ECHO_ERR_INVALID).
 * The call returns after enqueueing.  echo_gemm_bf16_noalloc_status waits for the stream and reports
 * how the most recent call on the current device ended: ECHO_OK, or ECHO_ERR_TIMEOUT if one of its
 * kernel's bounded waits ran out (Y is then incomplete).  It allocates nothing either. */
int echo_gemm_bf16_noalloc(const void *X, const void *W, void *Y, int32_t M, int32_t N, int32_t K,
                           int32_t epilogue, void *cuda_stream);
int echo_gemm_bf16_noalloc_status(void *cuda_stream);

const char *echo_strerror(int code);
const char *echo_last_error(echo_ctx *ctx);   /* text of the last ECHO_ERR_CUDA on this context */

#ifdef __cplusplus
}
#endif
#endif /* ECHO_B200_H */
