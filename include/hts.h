/*
 * hts.h -- C ABI of the HTS-RL hot-path library for NVIDIA B200 (sm_100a).
 *
 * Two operations of the synchronous actor-critic pipeline of "High-Throughput
 * Synchronous Deep RL" (arXiv 2012.09849) are exported:
 *
 *   hts_policy_step  the batched actor step (Section 4.1, "Asynchronous actors and
 *                    executors"): one forward pass of the policy-value network of
 *                    Appendix F.1 / F.2 over all observations handed in, then one
 *                    sampled action per observation whose randomness depends only
 *                    on (seed, env_id, t), never on how the batch was grouped.
 *   hts_gae          the return / advantage computation over the [T,N] rollout
 *                    storage that feeds the learner (Section 3, "Actor-Critic
 *                    Algorithms": n-step truncated return; GAE generalises it).
 *
 * Conventions that hold for every entry point unless it says otherwise
 *   - Plain C: no exceptions or aborts cross this boundary; every call returns an
 *     hts_status.  Invalid arguments are detected on the host before any launch.
 *   - "DEVICE" pointers are CUDA device memory of the current device, owned by the
 *     caller; the library never frees them and does not keep them after the
 *     stream work of the call.  "HOST" pointers are ordinary host memory.
 *   - Calls taking a `cuda_stream` (a cudaStream_t passed as void*, NULL = legacy
 *     default stream) only enqueue work on that stream and do not synchronise.
 *   - Output buffers must not overlap input buffers or each other.
 *   - A context owns one activation workspace: its steps must be ordered on the GPU
 *     (one stream, or events between streams).  Steps that may overlap need a
 *     context each; contexts are independent, also across threads.
 *   - There is no CPU fallback: without a CUDA device calls return HTS_ERR_CUDA.
 */
#ifndef HTS_H_
#define HTS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hts_ctx hts_ctx; /* opaque: packed weights + activation workspace */

typedef enum {
    HTS_OK = 0,
    HTS_ERR_INVALID_ARG = 1, /* NULL pointer, overlap, n outside 1..max_batch, bad gamma/lambda ... */
    HTS_ERR_SHAPE = 2,       /* network geometry not supported                       */
    HTS_ERR_ALLOC = 3,       /* device or host allocation failed                     */
    HTS_ERR_CUDA = 4,        /* a CUDA runtime call failed (see hts_last_cuda_error) */
    HTS_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out                   */
    HTS_ERR_UNSUPPORTED = 6  /* valid request that this build does not implement     */
} hts_status;

/* weight_dtype */
#define HTS_DTYPE_FP32 0 /* fp32 weights, fp32 CUDA-core arithmetic: the check path   */
#define HTS_DTYPE_BF16 1 /* bf16 weights, tensor-core path with fp32 accumulation     */

/* Network geometry.  The layers are fixed by Appendix F.1 / F.2 of the paper:
 * conv 32@8x8/4 -> conv 64@4x4/2 -> conv 64@3x3/1 -> FC 512 -> {policy over
 * num_actions, scalar value}; no padding, ReLU after the four hidden layers, input
 * scaled by 1/255.  C,H,W describe one uint8 observation (H,W multiples of 4 and
 * large enough that every layer has at least one output); 1 <= num_actions <= 64. */
typedef struct {
    int32_t C, H, W;
    int32_t num_actions;
    int32_t weight_dtype; /* HTS_DTYPE_*                                  */
    int32_t max_batch;    /* largest n any later hts_policy_step may pass */
} hts_net_desc;

/* The twelve parameter tensors, PyTorch layouts, all DEVICE pointers, element type
 * given by weight_dtype (float, or bf16 stored as 16-bit patterns).
 * F = 64*H3*W3 is the flattened conv3 output; FC column f = c*H3*W3 + h*W3 + w.   */
typedef struct {
    const void *conv1_w, *conv1_b; /* [32,C,8,8], [32]  */
    const void *conv2_w, *conv2_b; /* [64,32,4,4], [64] */
    const void *conv3_w, *conv3_b; /* [64,64,3,3], [64] */
    const void *fc_w, *fc_b;       /* [512,F], [512]    */
    const void *pi_w, *pi_b;       /* [A,512], [A]      */
    const void *v_w, *v_b;         /* [1,512], [1]      */
} hts_weights;

/* Create a context for one network geometry on the current device.  Allocates the
 * packed-weight store and an activation workspace sized for max_batch (device
 * memory, freed by hts_policy_destroy).
 * A HTS_DTYPE_BF16 context (tensor-core kernels) takes C in {4, 8, 16} and frames
 * up to 252 pixels wide (the resident activation tiles of the second convolution
 * must fit 227 KB of shared memory) whose first hidden layer, taken 2 x 2 pixels at a
 * time, has at most 2048 positions (252-wide frames up to 532 pixels high); anything else is refused here with
 * HTS_ERR_SHAPE, before any device call, never at step time.  Its frame buffers (obs, state_buffer) must start on a
 * 16-byte boundary (they are staged by TMA); a misaligned pointer is refused with
 * HTS_ERR_INVALID_ARG by the step calls.  Activations between layers are fp16: a
 * hidden activation above 65504 saturates there.  With |w| summed per output unit
 * S1, S2, S3 for the three convolutions and biases b, the largest possible
 * activation is bounded by S3 (S2 (S1 + |b1|) + |b2|) + |b3| (inputs lie in [0, 1]);
 * He-initialised weights of this network give 1.7e4 (4 x 84 x 84 frames) and 3.1e4
 * (16 x 72 x 96 frames), see tests/test_activation_range.py.
 * Errors: INVALID_ARG, SHAPE, ALLOC, CUDA.                                         */
hts_status hts_policy_create(const hts_net_desc *desc, hts_ctx **out);

/* Repack the caller's weights into the library's internal layouts on `cuda_stream`.
 * May be called again at any time (e.g. after each learner update: the parameter
 * hand-over of Section 4.1 "Delayed gradient"); steps enqueued later on the same
 * stream see the new weights.  The caller's buffers are read during the stream
 * work of this call only.                                                        */
hts_status hts_policy_load_weights(hts_ctx *ctx, const hts_weights *w, void *cuda_stream);

/* The batched actor step (Section 4.1; network of Appendix F.1/F.2; outputs are
 * the quantities of Eq. 3/4: log pi(a|s), V(s), H(pi(.|s)) in nats).
 *   obs        DEVICE u8  [n,C,H,W]   raw frames, NCHW
 *   env_ids    DEVICE i32 [n]         global environment index of each row (>= 0;
 *                                      duplicates allowed)
 *   t_per_env  DEVICE i32 [n] or NULL per-row time index; NULL = every row uses `t`
 *   seed                               64-bit run seed
 *   n                                  1..max_batch, any value (no tile multiple needed)
 *   actions    DEVICE i32 [n]   out   Gumbel-max sample: argmax_a logit_a - log(-log u_a),
 *                                      u_a from Philox4x32-10 with counter
 *                                      (env_id, t, a/4, 0), key (seed_lo, seed_hi),
 *                                      word a%4, u = ((word>>9)+0.5)*2^-23; ties -> lowest a
 *   logp, values, entropy  DEVICE f32 [n]  out
 *   logits_or_null  DEVICE f32 [n,A] or NULL  out  raw policy logits (parity tap)
 * Each row's outputs are independent of n, of the row's position and of the other
 * rows.  Errors: INVALID_ARG (NULL, n out of range, overlap), CUDA, UNSUPPORTED
 * (weights not loaded).                                                           */
hts_status hts_policy_step(hts_ctx *ctx, const uint8_t *obs, const int32_t *env_ids,
                           const int32_t *t_per_env, int32_t t, uint64_t seed, int32_t n,
                           int32_t *actions, float *logp, float *values, float *entropy,
                           float *logits_or_null, void *cuda_stream);

/* The executor-facing form of the same step (Section 4.1: executors write states
 * to the state buffer, actors read from it, and their outputs go to the data
 * storage used by the learner): the frames of the batch are gathered from a
 * device-resident state buffer by slot, and each row's outputs are scattered to
 * the same slot of one row of the [T, pool] rollout storage, with no copy in
 * between.  A batch is any subset of the pool in any order (the executor batches
 * of an asynchronous step).
 *   state_buffer  DEVICE u8  [pool,C,H,W]  one frame per environment slot
 *   slots         DEVICE i32 [n]           slot of each row, each in [0, pool)
 *   env_ids, t_per_env, t, seed, n         as in hts_policy_step (env_ids feed the
 *                                          random stream; they need not equal slots)
 *   actions_row, logp_row, values_row, entropy_row
 *                 DEVICE [pool]  out       row t of the storage; only the entries
 *                                          at the n slots are written
 * Outputs equal, bit for bit, those of hts_policy_step on the gathered frames.
 * If two rows name the same slot, one of them is kept.  A slot outside [0, pool)
 * is not dereferenced: that row writes nothing and hts_last_async_error reports
 * INVALID_ARG.  Errors otherwise as hts_policy_step.                            */
hts_status hts_policy_step_indexed(hts_ctx *ctx, const uint8_t *state_buffer, int32_t pool,
                                   const int32_t *slots, const int32_t *env_ids,
                                   const int32_t *t_per_env, int32_t t, uint64_t seed, int32_t n,
                                   int32_t *actions_row, float *logp_row, float *values_row,
                                   float *entropy_row, void *cuda_stream);

/* The learner's re-evaluation of stored transitions (Section 3: the update of Eq. 3/4
 * needs log pi(a_t|s_t), V(s_t) and H(pi(.|s_t)) under the current parameters for the
 * actions that were taken).  Same network pass as hts_policy_step, no sampling.
 *   obs      DEVICE u8  [n,C,H,W]
 *   actions  DEVICE i32 [n]        the stored actions, each in [0, num_actions)
 *   logp, values, entropy  DEVICE f32 [n]  out;  logits_or_null DEVICE f32 [n,A] or NULL
 * For the action hts_policy_step sampled on the same frames and weights the three
 * outputs equal that step's, bit for bit.  An action outside the range is not used
 * as an index: that row writes nothing and hts_last_async_error reports INVALID_ARG. */
hts_status hts_policy_evaluate(hts_ctx *ctx, const uint8_t *obs, const int32_t *actions, int32_t n,
                               float *logp, float *values, float *entropy, float *logits_or_null,
                               void *cuda_stream);

/* The twelve gradient tensors, shaped like hts_weights, all DEVICE f32 (written, not accumulated). */
typedef struct {
    float *conv1_w, *conv1_b;
    float *conv2_w, *conv2_b;
    float *conv3_w, *conv3_b;
    float *fc_w, *fc_b;
    float *pi_w, *pi_b;
    float *v_w, *v_b;
} hts_grads;

/* The gradient the learner applies (Section 3: Eq. 4 is this gradient's estimator; Section 4.1, Eq. 5
 * adds it to the parameters):  grads = d J-hat / d theta  at the context's current weights, with
 *   J-hat = (1/n) sum_i [ S_i - value_coef (R_i - V(s_i))^2 + entropy_coef H(pi(.|s_i)) ]
 *   S_i   = log pi(a_i|s_i) A_i                                  if logp_old is NULL or clip == 0
 *           min(rho_i A_i, clip(rho_i, 1-clip, 1+clip) A_i),  rho_i = exp(log pi(a_i|s_i) - logp_old_i)  otherwise
 * (the advantages are data: no gradient flows through them).  One forward pass over the n frames and one
 * backward pass through the network of Appendix F.1 / F.2; ReLU passes the gradient where its output is
 * positive.  Feed the result to hts_delayed_update (it is an ascent direction).
 *   obs DEVICE u8 [n,C,H,W]; actions DEVICE i32 [n] in [0, num_actions); advantages, returns DEVICE f32 [n];
 *   logp_old DEVICE f32 [n] or NULL; grads: twelve DEVICE f32 buffers, PyTorch layouts, overwritten.
 * Only HTS_DTYPE_FP32 contexts (the learner's master weights are fp32; a bf16 actor context is refreshed
 * from them through hts_delayed_update's bf16 output and hts_policy_load_weights): a bf16 context returns
 * HTS_ERR_UNSUPPORTED.  fp32 CUDA-core arithmetic, every sum in a fixed order; written for a reproducible
 * result, not tuned.  The first call on a context allocates the backward workspace (device memory, freed
 * by hts_policy_destroy).  An action outside the range is not used as an index: that sample contributes
 * nothing and hts_last_async_error reports INVALID_ARG.
 * Errors: INVALID_ARG (NULL, n out of range, clip < 0, non-finite coefficient), UNSUPPORTED, ALLOC, CUDA.  */
hts_status hts_policy_gradient(hts_ctx *ctx, const uint8_t *obs, const int32_t *actions,
                               const float *advantages, const float *returns,
                               const float *logp_old_or_null, float value_coef, float entropy_coef,
                               float clip, int32_t n, const hts_grads *grads, void *cuda_stream);

/* The three sample means the actor-critic update is built from (Section 3), over
 * `count` stored transitions in any layout (e.g. the whole [T,N] storage):
 *   out3[0] = (1/count) sum logp_i (returns_i - values_i)    policy term of Eq. 4 (its
 *             gradient with the advantage held fixed is Eq. 4's first summand)
 *   out3[1] = (1/count) sum (returns_i - values_i)^2         value loss J_V
 *   out3[2] = (1/count) sum entropy_i                        the term Eq. 4 weights by alpha
 *   logp, values, entropy, returns  DEVICE f32 [count];  out3 DEVICE f32 [3]
 * Summed in double precision in an order that depends on count alone.  Uses a small
 * table inside the library: calls on one device must be ordered (one stream, or
 * events between streams), not concurrent.  Errors: INVALID_ARG, CUDA.            */
hts_status hts_a2c_terms(const float *logp, const float *values, const float *entropy,
                         const float *returns, int64_t count, float *out3, void *cuda_stream);

/* The same for proximal policy optimisation, the algorithm HTS-RL is run with on the
 * football scenarios (Section 5, "Ours (PPO)"; objective of Schulman et al. 2017, Eq. 7):
 *   rho_i   = exp(logp_new_i - logp_old_i)   (fp32 exponential; everything after it in fp64)
 *   A_i     = advantages_i, or (advantages_i - mean) / (std + 1e-8) over the batch
 *             (population std) if normalize_advantages != 0
 *   out4[0] = (1/count) sum min(rho_i A_i, clip(rho_i, 1-clip, 1+clip) A_i)   clipped surrogate
 *   out4[1] = (1/count) sum (returns_i - values_i)^2                          value loss
 *   out4[2] = (1/count) sum entropy_i
 *   out4[3] = fraction of samples with |rho_i - 1| > clip
 *   all inputs DEVICE f32 [count]; out4 DEVICE f32 [4]; clip > 0.
 * Summation, ordering and the non-concurrency rule as for hts_a2c_terms.            */
hts_status hts_ppo_terms(const float *logp_new, const float *logp_old, const float *values,
                         const float *entropy, const float *advantages, const float *returns,
                         int64_t count, float clip, int32_t normalize_advantages, float *out4,
                         void *cuda_stream);

/* One learner update with the one-step-delayed gradient (Section 4.1, Eq. 5):
 *   theta <- theta + lr * d,  where grad is the gradient of the objective J-hat that
 * the caller took at the PREVIOUS parameters (the ones the rollout was collected
 * with).  With sq_avg given, d is RMSProp-scaled as in the hyper-parameter tables of
 * Appendix F (momentum 0):  v <- alpha v + (1-alpha) grad^2,  d = grad / (sqrt(v) + eps);
 * with sq_avg NULL, d = grad (Eq. 5 as printed; alpha and eps unused).
 *   theta, grad, sq_avg  DEVICE f32 [count] (theta and sq_avg updated in place)
 *   theta_bf16_or_null   DEVICE bf16 [count] or NULL  out: the new parameters rounded to
 *                        bf16 in the same pass, ready for hts_policy_load_weights
 * The sign is ascent on J-hat; pass the negated gradient of a loss.  0 <= alpha <= 1,
 * eps > 0, lr finite.  Errors: INVALID_ARG, CUDA.                                  */
hts_status hts_delayed_update(float *theta, const float *grad, float *sq_avg_or_null, int64_t count,
                              float lr, float alpha, float eps, void *theta_bf16_or_null,
                              void *cuda_stream);

/* Same operation with HOST buffers: copies obs/env_ids/t_per_env to the device,
 * runs the step, copies the four outputs (and logits if asked) back and waits for
 * them.  Uses staging buffers owned by the context (allocated at create time).
 * Pinned host memory makes the copies asynchronous but is not required.           */
hts_status hts_policy_step_host(hts_ctx *ctx, const uint8_t *obs, const int32_t *env_ids,
                                const int32_t *t_per_env, int32_t t, uint64_t seed, int32_t n,
                                int32_t *actions, float *logp, float *values, float *entropy,
                                float *logits_or_null, void *cuda_stream);

/* Parity tap: convert the hidden activation left in the workspace by the most
 * recent hts_policy_step on this context into fp32 NCHW.
 *   layer 1..3 -> conv outputs [n,32,H1,W1], [n,64,H2,W2], [n,64,H3,W3]; 4 -> FC [n,512]
 *   out  DEVICE f32, n = rows of that step.  Enqueued on cuda_stream.             */
hts_status hts_policy_read_activation(hts_ctx *ctx, int32_t layer, int32_t n, float *out,
                                      void *cuda_stream);

/* Parity tap for the sampler's random stream (Section 4.1: the per-observation
 * pseudo-random number): writes the num_actions uniforms that hts_policy_step
 * uses for each row, computed by the same device function.
 *   env_ids DEVICE i32 [n]; t_per_env DEVICE i32 [n] or NULL; out DEVICE f32 [n,num_actions] */
hts_status hts_action_uniforms(const int32_t *env_ids, const int32_t *t_per_env, int32_t t,
                               uint64_t seed, int32_t n, int32_t num_actions, float *out,
                               void *cuda_stream);

/* Benchmark support: per-kernel device timing of the actor step.  While enabled, every
 * hts_policy_step on this context brackets each of its kernels with CUDA events on the
 * step's stream (up to 4096 steps between two reads; later ones are not recorded).
 * hts_policy_profile(ctx, 1) starts a fresh collection, (ctx, 0) stops recording.
 * hts_policy_profile_read waits for the recorded events and returns, for kernel index
 * 0..4 (hts_policy_kernel_name gives "conv1","conv2","conv3","fc","heads"), the summed
 * device time in milliseconds and the number of launches recorded.                  */
hts_status hts_policy_profile(hts_ctx *ctx, int32_t enable);
hts_status hts_policy_profile_read(hts_ctx *ctx, int32_t kernel, float *total_ms, int32_t *launches);
const char *hts_policy_kernel_name(int32_t kernel);

/* Reads and clears the device status word of the context: HTS_ERR_TIMEOUT if a
 * bounded wait ran out, HTS_ERR_INVALID_ARG if hts_policy_step_indexed met a slot
 * outside the pool or hts_policy_evaluate an action outside the range, HTS_OK if
 * nothing was recorded.  Synchronises with the device.                            */
hts_status hts_last_async_error(hts_ctx *ctx);

/* Self-test of the failure-detection path (the kernels of this library never wait
 * without a limit: a pipeline stage that does not get its data within about a second
 * records a code, the block drains and the kernel returns, and hts_last_async_error
 * reports HTS_ERR_TIMEOUT).  This call enqueues one tiny block that waits, through the
 * same helper, on a barrier nothing arrives on, gives up after `limit_ticks` SM clock
 * ticks (1e3 .. 1e8) and returns normally; afterwards hts_last_async_error(ctx) must
 * report HTS_ERR_TIMEOUT once and the context must still work.  Errors: INVALID_ARG, CUDA. */
hts_status hts_wait_selftest(hts_ctx *ctx, int64_t limit_ticks, void *cuda_stream);

void hts_policy_destroy(hts_ctx *ctx);

/* Advantages and returns over the rollout storage (Section 3: with lambda = 1,
 * returns[t] is the n-step truncated return with n = T - t):
 *   delta_t = r_t + gamma (1-d_t) V_{t+1} - V_t          V_T = bootstrap
 *   A_t     = delta_t + gamma lambda (1-d_t) A_{t+1}     A_T = 0
 *   R_t     = A_t + V_t
 *   rewards, values  DEVICE f32 [T,N] time-major;  dones DEVICE u8 [T,N], non-zero =
 *   the transition taken at step t ended the episode;  bootstrap DEVICE f32 [N];
 *   advantages, returns  DEVICE f32 [T,N] out.   0 <= gamma, lambda <= 1, finite.
 * T >= 1, N >= 1.  Errors: INVALID_ARG, CUDA.                                      */
hts_status hts_gae(const float *rewards, const float *values, const uint8_t *dones,
                   const float *bootstrap, float gamma, float lambda, int32_t T, int32_t N,
                   float *advantages, float *returns, void *cuda_stream);

/* The off-policy-corrected form of the same scan: V-trace targets and the truncated-
 * importance-sampling policy-gradient advantages (the corrections the paper compares
 * its delayed gradient with: Section 2, IMPALA; Appendix C, Table A1 "Truncated I.S.";
 * definition: Espeholt et al. 2018, Section 4.1 Eq. 1 and Section 4.2):
 *   ratio_t = exp(log_rhos_t)   rho_t = min(rho_bar, ratio_t)   c_t = lambda min(c_bar, ratio_t)
 *   delta_t = rho_t (r_t + g_t V_{t+1} - V_t)        g_t = gamma (1-d_t),  V_T = bootstrap
 *   vs_t    = V_t + D_t,   D_t = delta_t + g_t c_t D_{t+1},   D_T = 0
 *   pg_t    = rho_t (r_t + g_t vs_{t+1} - V_t),      vs_T = bootstrap
 *   log_rhos DEVICE f32 [T,N]: log pi(a_t|s_t) - log mu(a_t|s_t) (learner minus behaviour);
 *   rewards, values, dones, bootstrap as for hts_gae;  vs, pg_advantages DEVICE f32 [T,N] out.
 * With log_rhos = 0 and rho_bar, c_bar >= 1 this is hts_gae: vs = returns, pg = advantages.
 * 0 <= gamma, lambda <= 1; rho_bar, c_bar >= 0.  Errors: INVALID_ARG, CUDA.            */
hts_status hts_vtrace(const float *log_rhos, const float *rewards, const float *values,
                      const uint8_t *dones, const float *bootstrap, float gamma, float lambda,
                      float rho_bar, float c_bar, int32_t T, int32_t N, float *vs,
                      float *pg_advantages, void *cuda_stream);

/* Same with HOST buffers; copies in, computes, copies out and waits.  Staging
 * memory is a library-owned device buffer per device that grows on demand (not
 * thread safe) and stays allocated until hts_gae_host_release.                     */
hts_status hts_gae_host(const float *rewards, const float *values, const uint8_t *dones,
                        const float *bootstrap, float gamma, float lambda, int32_t T,
                        int32_t N, float *advantages, float *returns, void *cuda_stream);

/* Frees the staging buffer of hts_gae_host on the current device (waits for the
 * device first).  The next hts_gae_host allocates again.  Errors: CUDA.           */
hts_status hts_gae_host_release(void);

/* The actor step for callers that must not allocate.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits, for example an
 * inference loop inside a process whose device memory is fully handed to another
 * allocator or pool, a plug-in that may not change the host's memory footprint, or a
 * latency-critical loop that cannot afford the implicit device synchronisation of an
 * allocation.  hts_policy_create allocates its workspace with cudaMalloc; this call
 * needs no context and allocates nothing, neither itself nor through a library.
 *
 * What it does: the fp32 check-path arithmetic of hts_policy_step (same kernels, same
 * results bit for bit) on the caller's own fp32 weights, read in place from `w`
 * (PyTorch layouts, DEVICE pointers; desc->weight_dtype must be HTS_DTYPE_FP32,
 * desc->max_batch is ignored).  Inputs and outputs as for hts_policy_step.
 *
 * Scratch: hidden activations and the stacked head weights go to a fixed array of
 * 2^20 floats (4 MiB) that is part of the library image; every GPU that loads the
 * library holds it until the process exits.  A call whose
 *   n*(32*H1*W1 + 64*H2*W2 + 64*H3*W3 + 512) + (A+1)*513
 * floats do not fit (more than 48 observations of 4x84x84 with 18 actions) is refused
 * with HTS_ERR_INVALID_ARG.  The array is shared by all calls and keeps the previous
 * call's contents; the call overwrites every part it reads, so nothing needs clearing,
 * but two calls whose GPU work overlaps (different streams, or threads) race on it:
 * serialise them.  The first call on each device looks up the array's device address
 * (with that device current); make that first call before starting any stream capture.
 * Errors: INVALID_ARG (NULL, n < 1, too large for the scratch), SHAPE, UNSUPPORTED
 * (weights not fp32, device index above 63), CUDA.                                   */
hts_status hts_policy_step_noalloc(const hts_net_desc *desc, const hts_weights *w, const uint8_t *obs,
                                   const int32_t *env_ids, const int32_t *t_per_env, int32_t t,
                                   uint64_t seed, int32_t n, int32_t *actions, float *logp,
                                   float *values, float *entropy, float *logits_or_null,
                                   void *cuda_stream);

/* Number of kernel launches this library has enqueued since it was loaded
 * (all contexts, all streams); for launch accounting by a benchmark.              */
uint64_t hts_launch_count(void);

/* Text of the last CUDA runtime error seen by this library on the calling thread
 * (empty string if none).                                                         */
const char *hts_last_cuda_error(void);

const char *hts_status_string(hts_status s);

#ifdef __cplusplus
}
#endif
#endif /* HTS_H_ */
