/*
 * accerl.h -- C ABI of the int8 Actor policy-inference library for NVIDIA B200 (sm_100a).
 *
 * What the library computes.  In the paper's actor-learner loop every Actor runs, per
 * environment step, one forward pass of the Compressor's quantised policy network on a batch
 * of states and samples one action per state (Introduction, Fig. 1: the "Agent" share of data
 * collection; Section 2.1, Overview).  The compressed policy is an int8 post-training-
 * quantised network whose Conv+ReLU / FC+ReLU pairs are fused into single layers (Section 2.2,
 * paragraphs "Parameter Quantization" and "Static Computational Graph").  The Corrector later
 * needs the behaviour probability pi_smaller(a|x) of the action taken (Section 2.3, Eq. V-trace
 * and Eq. IS).  `accerl_policy_create` takes such a quantised network, `accerl_policy_act`
 * maps a batch of states to logits, sampled actions and behaviour log-probabilities.
 *
 * Arithmetic (fixed; the same on every code path of the library):
 *   input, frames : x = (float)u / 255.0f;  q = clamp(rintf(x / s_input), -128, 127)
 *   input, vectors: q = clamp(rintf(obs / s_input), -128, 127)
 *   contraction   : acc = sum_k w[c,k] * x[k]              int8 x int8 -> int32, zero padding
 *                   (ACCERL_RELU_IN: x is max(x, 0) first)
 *   residual      : acc += skip_mul[c] * x_skip[c, y, x]    int32, before the epilogue
 *   epilogue      : y = fmaf((float)acc, s_in * s_w[c], bias[c]);   s_in * s_w[c] rounded once
 *                   (ACCERL_RELU_OUT: y = max(y, 0))
 *                   q = clamp(rintf(y / s_out), -128, 127)   IEEE divide, ties to even
 *   final layer   : ACCERL_LOGITS stops at y (fp32 logits)
 *   max-pool      : per-channel max over a kh x kw window, stride `stride`, no padding, floor
 *   sampling      : logp = z - logsumexp(z);  cdf_i = sum_{j<=i} exp(logp_j);
 *                   action = first i with u < cdf_i, else A-1;  logp_out = logp[action]
 *
 * Conventions.  All sizes are in elements unless they say bytes.  "host" / "device" in a
 * parameter comment says where the pointer must live.  Nothing is thrown across this ABI and
 * the library never calls exit/abort: every entry point returns an accerl_status, and
 * accerl_last_error() gives a message for the calling thread's last failure.  Invalid
 * arguments are rejected on the host before anything is launched.
 */
#ifndef ACCERL_H_
#define ACCERL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct accerl_policy accerl_policy; /* opaque handle */

typedef enum {
    ACCERL_OK = 0,
    ACCERL_ERR_INVALID_ARG = 1,     /* null pointer, bad size, inconsistent layer chain */
    ACCERL_ERR_UNSUPPORTED = 2,     /* valid description the library has no kernel for */
    ACCERL_ERR_BATCH_TOO_LARGE = 3, /* batch > max_batch given at create */
    ACCERL_ERR_OOM = 4,             /* device or host allocation failed */
    ACCERL_ERR_CUDA = 5,            /* a CUDA runtime / driver call failed */
    ACCERL_ERR_TIMEOUT = 6          /* a bounded device-side wait gave up (status word set) */
} accerl_status;

typedef enum { ACCERL_IN_U8_NCHW = 0, ACCERL_IN_F32 = 1 } accerl_input_kind;
typedef enum { ACCERL_CONV2D = 0, ACCERL_FC = 1, ACCERL_MAXPOOL = 2 } accerl_layer_kind;

/* accerl_layer_desc.flags */
enum {
    ACCERL_RELU_IN = 1,  /* apply max(x, 0) to the int8 input before the contraction */
    ACCERL_RELU_OUT = 2, /* ReLU on the epilogue float, before the clamp */
    ACCERL_LOGITS = 4    /* last layer: fp32 output, no requantisation */
};

/* accerl_policy_create flags */
enum {
    ACCERL_FLAG_KEEP_ACTIVATIONS = 1, /* give every layer its own output buffer so that
                                         accerl_policy_read_activation works (parity taps) */
    ACCERL_FLAG_FORCE_GENERIC = 2,    /* use only the plain CUDA-core kernels (no tensor-core
                                         or fused plans); for cross-checking the fast paths */
    ACCERL_FLAG_TAP_FUSED = 4,        /* only with KEEP_ACTIVATIONS: keep every fusion of the plan
                                         that runs without the taps (input stage inside the first
                                         conv, pooling on accumulators, the single-launch MLP) and
                                         tap the tensors that plan still stores; a tensor it never
                                         stores reads as ACCERL_ERR_UNSUPPORTED.  Without this
                                         bit KEEP_ACTIVATIONS un-fuses those steps so that every
                                         tensor exists. */
    ACCERL_FLAG_VALUE_HEAD = 8,       /* the last layer has one column more than there are actions:
                                         columns [0, A) are the logits, column A is the state value
                                         V(s) (Section 2.2, Eq. KD: the compressed network carries a
                                         value function; Section 2.3, Eq. V-trace uses it).  V is the
                                         same single fma as a logit, takes no part in the softmax and
                                         is returned by accerl_policy_act_ex. */
    ACCERL_FLAG_TEST_NO_FASTDIV = 16, /* test hook: treat every output scale as one for which the
                                         division-free requantiser could not be verified at create.
                                         Layers then run the epilogue that re-does elements near a
                                         rounding tie with the IEEE divide -- what a policy with an
                                         unlucky scale gets for that layer.  Results are the same
                                         bits either way. */
    ACCERL_FLAG_TEST_NO_AFFINE = 32   /* test hook: do not search the single-fma requantiser
                                         constants at create (a layer for which the search finds
                                         none for some channel behaves like this): the epilogues
                                         keep the verified three-step division.  Same bits either
                                         way. */
};

/*
 * One layer.  Conv: input [in_c, in_h, in_w], weights OIHW [out_c][in_c][kh][kw], square
 * `stride`, symmetric zero `pad`.  FC: in_c = K, out_c = N, in_h = in_w = kh = kw = stride = 1,
 * pad = 0; an FC fed by a conv/pool output reads it flattened in (C, H, W) order.  Max-pool:
 * in_c = out_c, kh = kw = window, no weights (w, s_w, bias NULL; s_out must equal s_in).
 * All pointers are HOST pointers; the library copies what they point to during create and
 * never keeps them.
 */
typedef struct {
    int32_t kind; /* accerl_layer_kind */
    uint32_t flags;
    int32_t in_c, in_h, in_w, out_c, kh, kw, stride, pad;
    float s_in, s_out;       /* per-tensor activation scales of this layer's input / output */
    const int8_t *w;         /* host, int8 weights, values in [-127, 127] */
    const float *s_w;        /* host, [out_c] per-output-channel weight scales */
    const float *bias;       /* host, [out_c] fp32 */
    int32_t skip_from;       /* -1, or index of an EARLIER layer whose int8 output (same shape
                                as this layer's output) is added into the accumulators */
    const int32_t *skip_mul; /* host, [out_c] integer multipliers, in [0, 32767]; NULL iff
                                skip_from < 0 */
} accerl_layer_desc;

/*
 * Build a policy on CUDA device `device` (Section 2.2: the Compressor hands the Actor a
 * quantised, fused, static network; this call is the "static graph" step: it validates the
 * chain, repacks weights into the kernels' layouts, precomputes s_in * s_w[c], allocates the
 * activation workspace for `max_batch` states and fixes the launch plan).
 *   out        host, receives the handle (NULL on failure)
 *   in_kind    ACCERL_IN_U8_NCHW: observations are uint8 [B, C, H, W];
 *              ACCERL_IN_F32: observations are fp32 [B, D] with in_shape = {D, 1, 1}
 *   in_shape   host, {C, H, W}
 *   s_input    scale of the quantised input tensor (must equal layers[0].s_in)
 *   layers     host, n_layers descriptors; layer i consumes layer i-1's output; the last layer
 *              must be an FC with ACCERL_LOGITS and out_c = number of actions (1..1024), plus one
 *              with ACCERL_FLAG_VALUE_HEAD
 *   max_batch  largest batch `act` will be called with (>= 1)
 *   flags      ACCERL_FLAG_* bits
 * Synchronises the device once; allocates device memory (freed by accerl_policy_destroy).
 * Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA; *out is NULL then.
 */
accerl_status accerl_policy_create(accerl_policy **out, int32_t in_kind, const int32_t in_shape[3],
                                   float s_input, const accerl_layer_desc *layers,
                                   int32_t n_layers, int32_t max_batch, uint32_t flags,
                                   int32_t device);

/*
 * One layer of an fp32 network, for accerl_policy_create_fp32: the fields of accerl_layer_desc
 * without the quantisation results.  `w` is fp32 OIHW (FC: [out_c][in_c]), `bias` fp32 [out_c];
 * both NULL for a max-pool.  All pointers are HOST pointers, copied during the call.
 */
typedef struct {
    int32_t kind; /* accerl_layer_kind */
    uint32_t flags;
    int32_t in_c, in_h, in_w, out_c, kh, kw, stride, pad;
    const float *w;
    const float *bias;
    int32_t skip_from; /* -1, or the earlier layer whose output is added into the accumulators */
} accerl_layer_fp32;

/*
 * Post-training quantisation on the device, then accerl_policy_create (Section 2.2, paragraph
 * "Parameter Quantization": the Compressor quantises the Learner's fp32 policy for the Actors;
 * paragraph "Structured Pruning" for the optional pruning).  The scheme, each step on the GPU:
 *   pruning (prune_2_4 != 0): of every four consecutive K positions, K = (kh, kw, c_in) with c_in
 *       fastest, keep the two weights of largest magnitude (lower index wins a tie)
 *   weights:     s_w[c] = max_k |w[c, k]| / 127 (1 for an all-zero channel);
 *                q = clamp(rintf(w / s_w[c]), -127, 127)
 *   input:       s_input = max |x| / 127 over the calibration batch (frames: x = u / 255)
 *   activations: layer by layer, s_out = max |y| / 127 over the calibration batch, y the epilogue
 *                float (after the residual add and the ReLU) computed from the already quantised
 *                preceding layers; 1 if the maximum is 0; a max-pool passes its scale through;
 *                the last layer has s_out = 1
 *   residual:    skip_mul[c] = clamp(rintf(s_x / (s_in * s_w[c])), 0, 32767), s_x the scale of the
 *                tensor that is added
 * Every division is the IEEE fp32 one; maxima and integer sums do not depend on evaluation order,
 * so the result is the same bits on every run.
 *   calib_obs_host  host, calib_rows observations in the layout `act` takes (uint8 [rows, C, H, W]
 *                   or fp32 [rows, D])
 *   the other arguments are those of accerl_policy_create; ACCERL_FLAG_VALUE_HEAD as there
 * Create-time work with plain kernels (tens of milliseconds for a thousand frames); transient
 * device memory: the calibration batch's int8 activations plus one int32 tensor of the largest
 * layer output.  Errors: INVALID_ARG, UNSUPPORTED, OOM, CUDA; *out is NULL then.
 */
accerl_status accerl_policy_create_fp32(accerl_policy **out, int32_t in_kind, const int32_t in_shape[3],
                                        const accerl_layer_fp32 *layers, int32_t n_layers,
                                        const void *calib_obs_host, int32_t calib_rows,
                                        int32_t prune_2_4, int32_t max_batch, uint32_t flags,
                                        int32_t device);

/*
 * Read back what accerl_policy_create_fp32 computed for one layer (for storing the quantised
 * policy, or for checking it): int8 weights in OIHW order, per-channel weight scales, residual
 * multipliers, and the layer's input / output activation scales.  Any output pointer may be NULL;
 * w_bytes is the size of w_host.  A max-pool has no weights (nothing is written for it).
 * Errors: INVALID_ARG (also for a handle not built by accerl_policy_create_fp32).
 */
accerl_status accerl_policy_export(const accerl_policy *p, int32_t layer, int8_t *w_host,
                                   size_t w_bytes, float *s_w_host, int32_t *skip_mul_host,
                                   float *s_in_out, float *s_out_out);

/*
 * One Actor step for a batch of states (Introduction, Fig. 1 "Agent"; Section 2.3, Eq. V-trace
 * for the behaviour log-probability): quantise the observations, run every layer, sample.
 *   obs_dev       device, uint8 [batch, C, H, W] or fp32 [batch, D]; 16-byte aligned; read only
 *   uniforms_dev  device, fp32 [batch], each in [0, 1): the random numbers the sampler inverts
 *   batch         1 .. max_batch
 *   logits_dev    device, fp32 [batch, A], written
 *   actions_dev   device, int32 [batch], written; always in [0, A-1]
 *   logp_dev      device, fp32 [batch], written: log pi(action | state), finite and <= 0
 *   cuda_stream   a cudaStream_t (NULL = the default stream)
 * Enqueues kernels on `cuda_stream` and returns without synchronising.  Allocates nothing.
 * The handle owns the workspace the kernels write, so calls on one handle must not overlap on
 * the GPU (use one stream per handle, or one handle per stream).  The caller owns all five
 * buffers.  Errors: INVALID_ARG, BATCH_TOO_LARGE, CUDA (launch failure).
 */
accerl_status accerl_policy_act(accerl_policy *p, const void *obs_dev, const float *uniforms_dev,
                                int32_t batch, float *logits_dev, int32_t *actions_dev,
                                float *logp_dev, void *cuda_stream);

/*
 * accerl_policy_act with the two further per-state outputs the rest of the framework consumes:
 *   value_dev    device, fp32 [batch], written: V(s), the value column of the last layer (Section
 *                2.2, Eq. KD, the term with v_smaller(s); Section 2.3, Eq. V-trace, V(x_s) "estimated
 *                by the compressed policy network").  NULL to skip; non-NULL needs a handle created
 *                with ACCERL_FLAG_VALUE_HEAD (INVALID_ARG otherwise).
 *   entropy_dev  device, fp32 [batch], written: H(pi(.|s)) = -sum_a p_a log p_a of the action
 *                distribution that was sampled from (Section 2.2, Eq. KD, the regulariser; Section
 *                2.4, one of the Monitor's indicators).  NULL to skip.
 * Both come out of the launch that samples; everything else is as in accerl_policy_act.
 */
accerl_status accerl_policy_act_ex(accerl_policy *p, const void *obs_dev, const float *uniforms_dev,
                                   int32_t batch, float *logits_dev, int32_t *actions_dev,
                                   float *logp_dev, float *value_dev, float *entropy_dev,
                                   void *cuda_stream);

/*
 * The Monitor's KL indicators (Section 2.4, Eq. KL): per state
 *   KL(pi_original || pi_smaller) = sum_a pi_original(a|x) log(pi_original(a|x) / pi_smaller(a|x))
 * from the logits two policies produced for the same batch, and optionally its mean and maximum
 * over the batch ("KL mean", "KL max"; the paper switches 8 -> 16 bits when KL max exceeds 14).
 *   logits_original_dev, logits_smaller_dev   device, fp32 [batch, n_actions], read only
 *   kl_dev            device, fp32 [batch], written
 *   kl_mean_max_dev   device, fp32 [2], written: {mean, max}; NULL to skip the reduction
 * Enqueues one or two kernels on `cuda_stream`, returns without synchronising, allocates nothing.
 * The reduction is done in a fixed order (same bits on every run).  Errors: INVALID_ARG, CUDA.
 */
accerl_status accerl_policy_kl(const float *logits_original_dev, const float *logits_smaller_dev,
                               int32_t batch, int32_t n_actions, float *kl_dev,
                               float *kl_mean_max_dev, void *cuda_stream);

/*
 * One Actor step in which every state follows the smaller policy with probability alpha and the
 * original one otherwise (Section 3.2, the linear-alpha strategy between the compressed and the
 * original network; Section 2.4, the Monitor sets alpha): state i uses `smaller` iff
 * select_uniforms_dev[i] < alpha.  Outputs are those of the chosen policy for that state, exactly
 * as accerl_policy_act_ex on that policy alone would give them.
 *   smaller, original    two different handles on the same device with the same observation shape
 *                        and number of actions; batch <= both max_batch
 *   select_uniforms_dev  device, fp32 [batch] in [0, 1): the selector draws (independent of
 *                        uniforms_dev, which the sampler inverts)
 *   alpha                in [0, 1]
 *   use_smaller_dev      device, uint8 [batch], written: 1 where `smaller` was used; NULL to skip
 *   value_dev            needs ACCERL_FLAG_VALUE_HEAD on both handles; NULL to skip
 * Both networks run on the whole batch and a last kernel selects per state, so the cost is the sum
 * of the two steps; results do not depend on which other states share the batch.  The first call
 * allocates, in `smaller`, result buffers for max_batch states (freed with the handle).  Uses both
 * handles' workspaces: no other call on either may overlap with it on the GPU.
 * Errors: INVALID_ARG, BATCH_TOO_LARGE, OOM, CUDA.
 */
accerl_status accerl_policy_act_mixed(accerl_policy *smaller, accerl_policy *original,
                                      const void *obs_dev, const float *uniforms_dev,
                                      const float *select_uniforms_dev, float alpha, int32_t batch,
                                      float *logits_dev, int32_t *actions_dev, float *logp_dev,
                                      float *value_dev, float *entropy_dev, uint8_t *use_smaller_dev,
                                      void *cuda_stream);

/*
 * V-trace targets of the Corrector (Section 2.3, Eq. V-trace, with the clipped importance ratios
 * rho_t = min(rho_hat, pi_original / pi_smaller), c_i = min(c_hat, pi_original / pi_smaller); the
 * paper sets rho_hat = c_hat = 1) for `batch` rollouts of `n_steps` steps, and the advantage of
 * Eq. A3C-V's first line:
 *   v_s   = V(x_s) + sum_{t=s}^{n-1} (prod_{i=s}^{t-1} g_i c_i) rho_t (r_t + g_t V(x_{t+1}) - V(x_t))
 *   adv_s = rho_s (r_s + g_s v_{s+1} - V(x_s)),        V(x_n) = v_n = bootstrap
 * with pi_original / pi_smaller = exp(logp_original - logp_smaller) of the action taken, i.e. of
 * the log-probs accerl_policy_act returns for the behaviour policy and the Learner's policy gives
 * for the same actions.  g_t = gamma, or discounts[t] when that array is given (gamma times "the
 * episode goes on", which cuts the sums at an episode end inside a rollout).
 *   all arrays      device, fp32, time-major [n_steps, batch]; bootstrap_dev [batch]
 *   discounts_dev   NULL, or [n_steps, batch]
 *   vs_dev          written; adv_dev written, NULL to skip
 * One thread per rollout runs the backward recursion the sums telescope into, in double, and
 * rounds the results to float.  Enqueues on `cuda_stream`, returns without synchronising,
 * allocates nothing.  Errors: INVALID_ARG, CUDA.
 */
accerl_status accerl_vtrace(const float *logp_smaller_dev, const float *logp_original_dev,
                            const float *rewards_dev, const float *values_dev,
                            const float *bootstrap_dev, const float *discounts_dev, int32_t n_steps,
                            int32_t batch, float gamma, float rho_hat, float c_hat, float *vs_dev,
                            float *adv_dev, void *cuda_stream);

/*
 * accerl_policy_act with a stopwatch on every kernel launch, for measuring where the Actor's
 * inference time goes (the paper's own method in the Introduction, Fig. 1, one level down):
 * records CUDA events on `cuda_stream` around each launch of the plan, runs the step, waits for
 * it and writes the device time of launch i (milliseconds) to launch_ms_host[i].  The order is
 * that of accerl_policy_info's plan lines; launch_ms_len must be >= launches_per_act.  The
 * events are created on the first call.  Blocks until the step has finished.
 */
accerl_status accerl_policy_act_timed(accerl_policy *p, const void *obs_dev,
                                      const float *uniforms_dev, int32_t batch, float *logits_dev,
                                      int32_t *actions_dev, float *logp_dev, void *cuda_stream,
                                      float *launch_ms_host, int32_t launch_ms_len);

/*
 * The Actor step for callers that must not allocate device memory.  (The paper has no
 * counterpart: this entry point exists for deployment, not for the method.)
 *
 * Who needs it: an Actor that shares its GPU with a Learner or with other Actors whose framework
 * allocators have already claimed the free HBM, a real-time control loop that cannot afford the
 * device-wide synchronisation an allocation may imply, or any host that has been told to keep its
 * device footprint fixed after start-up.  For such callers a workspace sized by `max_batch` at
 * create time, or the staging buffers accerl_policy_act_host allocates on first use, are not an
 * option.  Create the handle with max_batch = 1 (it then owns little beyond the weights) and step
 * through this call: it computes exactly what accerl_policy_act computes, with the plain
 * CUDA-core kernels, but keeps all int8 activations in a fixed array of
 * ACCERL_NOALLOC_SCRATCH_BYTES bytes that is part of the library image.  Every GPU on which the
 * library's kernels get loaded holds that array until the process exits.
 *
 * Same arguments, ownership and alignment rules as accerl_policy_act, except that `batch` is not
 * limited by the handle's max_batch but by the array: a batch whose activations do not fit is
 * rejected with ACCERL_ERR_BATCH_TOO_LARGE and a message that gives both sizes (Nature-CNN, whose
 * plan reuses two buffers of 28 224 + 12 800 bytes per state, fits about 1600 states).  The call enqueues on `cuda_stream`, returns without synchronising, and calls
 * no cudaMalloc / cudaFree or any other allocating routine.
 *
 * First call on a device: the library asks the CUDA runtime for the array's address on that
 * device (once per device, remembered afterwards).  Make this first call during start-up, before
 * any stream capture is begun.  The CUDA runtime loads a library's device code lazily, so the
 * array's memory may only be reserved when this first call (or any earlier kernel of the library
 * on that device, accerl_policy_create included) triggers the load; on a device without 64 MiB to
 * spare that is where ACCERL_ERR_CUDA appears.  From the second call on nothing is reserved.
 *
 * Sharing: all handles and all calls in the process use the same array, and it keeps whatever
 * the previous call left in it.  Nothing in it has to start at zero -- every byte a kernel reads
 * was written earlier in the same call -- so no clearing is done.  Two calls that overlap on the
 * GPU (different streams, or different threads without ordering) race on the array and corrupt
 * each other; order them on one stream or with events.
 */
#define ACCERL_NOALLOC_SCRATCH_BYTES (64u * 1024u * 1024u)
accerl_status accerl_policy_act_noalloc(accerl_policy *p, const void *obs_dev,
                                        const float *uniforms_dev, int32_t batch,
                                        float *logits_dev, int32_t *actions_dev, float *logp_dev,
                                        void *cuda_stream);

/*
 * The same step for callers whose data lives in HOST memory (an Actor process that steps its
 * environments on the CPU, Section 2.1): copies obs and uniforms to device staging buffers owned
 * by the handle, runs accerl_policy_act, copies the three results back and waits for them.
 * All five pointers are host pointers (pinned memory makes the copies asynchronous and faster;
 * pageable memory works).  The staging buffers are allocated on the first call.  Batches of 4096
 * states and more go in eight chunks whose host->device copies run on a stream of the handle's own
 * while the previous chunk computes on `cuda_stream`; the results are those of one call on the
 * whole batch.  Blocks until the results are in the host buffers.
 */
accerl_status accerl_policy_act_host(accerl_policy *p, const void *obs_host,
                                     const float *uniforms_host, int32_t batch,
                                     float *logits_host, int32_t *actions_host, float *logp_host,
                                     void *cuda_stream);

/*
 * Parity tap: copy layer `layer`'s int8 output of the most recent `act` call to the host in
 * canonical NCHW order ([batch, out_c, out_h, out_w]; for FC layers [batch, out_c]).
 * `layer` = -1 reads the quantised input tensor ([batch, C, H, W] or [batch, D]).
 * Needs ACCERL_FLAG_KEEP_ACTIVATIONS; synchronises the device.  The final (logits) layer has
 * no int8 output (INVALID_ARG).  dst_bytes must be at least the tensor's size.  With
 * ACCERL_FLAG_TAP_FUSED a tensor that the fused plan never stores in un-ReLU'd int8 form gives
 * ACCERL_ERR_UNSUPPORTED.
 */
accerl_status accerl_policy_read_activation(accerl_policy *p, int32_t layer, int32_t batch,
                                            int8_t *dst_host_nchw, size_t dst_bytes);

/*
 * Synchronise the stream of the last `act` call and report the device status word: ACCERL_OK,
 * ACCERL_ERR_TIMEOUT if a kernel's bounded wait gave up, ACCERL_ERR_CUDA for a sticky error.
 */
accerl_status accerl_policy_check(accerl_policy *p);

/*
 * Exercise the give-up path of the library's bounded device-side waits (the paper has no
 * counterpart: robustness support).  Enqueues a one-warp kernel that waits on a barrier nothing
 * arrives at, for at most `poll_limit` polls (1 .. 100000, at most 256 ns apart); the wait runs out,
 * the kernel sets the handle's status word and returns normally.  The next accerl_policy_check
 * reports ACCERL_ERR_TIMEOUT and clears the word; the handle and the context stay usable.
 */
accerl_status accerl_policy_selftest_wait(accerl_policy *p, int32_t poll_limit, void *cuda_stream);

/*
 * Describe the handle: number of actions, bytes of device workspace, kernel launches per
 * `act` call and a human-readable plan (one "launch i: ..." line per launch, then a "note: ..."
 * line if a faster plan had to be passed over and why) written as a NUL-terminated string into
 * plan_buf (truncated to plan_buf_bytes).  Any output pointer may be NULL.
 * The plan is fixed at create time for max_batch; `batch` is accepted for symmetry with the act
 * calls and does not change the answer.
 */
accerl_status accerl_policy_info(const accerl_policy *p, int32_t batch, int32_t *n_actions,
                                 size_t *workspace_bytes, int32_t *launches_per_act,
                                 char *plan_buf, size_t plan_buf_bytes);

/*
 * Micro-benchmark of the int8 tensor pipe, the denominator of the tensor-core roofline (the paper
 * has no counterpart: it measures its Actor as a whole, Introduction, Fig. 1; this measures the
 * unit the contraction layers run on).  Launches `ctas` CTAs (one per SM up to the SM count); in
 * each, `issuing_warps` warps issue `mmas_per_warp` tcgen05.mma kind::i8 instructions of shape
 * M = 128, N = n, K = 32 bytes back to back on operands that already sit in shared memory, and
 * wait (bounded) for the pipe to drain.
 *   device              CUDA device index
 *   n                   16 .. 256, a multiple of 16; issuing_warps * n <= 512 (tensor-memory columns)
 *   issuing_warps       1 .. 4
 *   mmas_per_warp       a multiple of 4, up to 2^20
 *   ctas                1 .. 1024
 *   layout              operand layout in shared memory: 128, 64 or 32 = K-major rows of that many
 *                       bytes under the matching swizzle; 0 = no swizzle, 16-byte K chunks in planes
 *                       of [row][16 bytes] (8-row groups 128 bytes apart)
 *   a_shift_rows        0 .. 128: the A operand starts this many rows into its tile, as the
 *                       row-shifted operand views of the convolution kernels do
 *   commit_every        0, or a multiple of 4: a tcgen05.commit (to a barrier nobody waits on)
 *                       after every so many MMAs, as a pipeline that hands accumulators over does
 *   ms_out              host, receives the duration of the best of three launches (CUDA events)
 *   cycles_per_mma_out  host, receives SM cycles per MMA and CTA: mean over CTAs of
 *                       (cycles from first issue to drained pipe) / (issuing_warps * mmas_per_warp)
 * int8 operations per second = ctas * issuing_warps * mmas_per_warp * 2 * 128 * n * 32 / time.
 * Synchronous; allocates and frees a few hundred bytes of device memory; uses the default stream.
 * Errors: INVALID_ARG, UNSUPPORTED (not sm_100), CUDA, TIMEOUT (a bounded wait gave up).
 */
accerl_status accerl_tc_probe_i8(int32_t device, int32_t n, int32_t issuing_warps,
                                 int32_t mmas_per_warp, int32_t ctas, int32_t layout,
                                 int32_t a_shift_rows, int32_t commit_every, float *ms_out,
                                 float *cycles_per_mma_out);

/* Free the handle and its device memory.  Synchronises the device.  NULL is allowed. */
void accerl_policy_destroy(accerl_policy *p);

/* Message for the calling thread's most recent failing call; never NULL. */
const char *accerl_last_error(void);

/* Library version string. */
const char *accerl_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ACCERL_H_ */
