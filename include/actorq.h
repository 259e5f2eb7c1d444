/*
 * actorq.h -- C ABI of the B200 int8 actor-inference library.
 *
 * The library implements the two steps ActorQ puts between a full-precision
 * learner and its actors (paper Section 3.1 and Figure 2b):
 *   1. the quantizer block: post-training quantization of every fp32 weight
 *      tensor of the policy to int8 with the uniform affine quantizer of
 *      Section 3.2 (Eq. 1-2), done again at every policy broadcast;
 *   2. actor policy inference with the quantized policy, here batched over
 *      the observations of many actors, with int8 operands, int32
 *      accumulation, and a single binary32 multiply + round-half-to-even to
 *      move each hidden activation to the next layer's int8 grid.
 *
 * Conventions that hold for every entry point
 *   - Every function returns an actorq_status as int.  Nothing throws, aborts
 *     or traps.  Host-detectable errors (NULL pointers, bad shapes, unsupported
 *     architectures, CUDA API failures) are returned at once.  Errors that only
 *     the device can see (a NaN/Inf weight, an internal wait that ran out) are
 *     recorded in a status word owned by the policy; read it with
 *     actorq_policy_last_device_status after synchronising the stream.
 *   - Pointers named "device" must be CUDA device pointers valid on the
 *     current device; they stay owned by the caller, are only read (inputs)
 *     or written (outputs) by work ordered on `cuda_stream`, and are never
 *     retained after that work finishes.  Pointers named "host" are ordinary
 *     host memory.  `cuda_stream` is a cudaStream_t passed as void* (NULL =
 *     the legacy default stream).
 *   - Calls are asynchronous with respect to the host unless stated.
 *   - A policy must not be re-quantized while a forward that uses it is still
 *     in flight on another stream; ordering the two is the caller's job.
 *
 * Quantizer arithmetic (bit-exact contract, per weight tensor W, n = 8 bits)
 *     lo = min(min W, 0), hi = max(max W, 0)              range contains 0 (Eq. 2)
 *     delta = (hi - lo) / 255         binary32 subtract, then binary32 divide
 *     z = clamp(rne(-lo / delta) - 128, -128, 127)
 *     q = clamp(rne(W / delta) + z, -128, 127)            binary32 divide (Eq. 1)
 *     dequantized value = delta * (q - z)                                (Eq. 3)
 *   rne = round half to even.  An all-zero tensor gets delta = 1, z = 0.
 *   Activation tensors use the same rule on the caller-supplied (min, max) of
 *   each layer's real-valued input, and quantize with one binary32 multiply by
 *   1/delta.  uint8 observations mean u/255: delta = 1/255, z = -128, q = u-128.
 */
#ifndef ACTORQ_H_
#define ACTORQ_H_

#ifdef __cplusplus
extern "C" {
#endif

typedef struct actorq_policy actorq_policy;   /* opaque; created and freed by the library */

typedef enum {
  ACTORQ_OK = 0,
  ACTORQ_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, mismatched architecture  */
  ACTORQ_ERR_UNSUPPORTED = 2,   /* a shape outside the documented limits                      */
  ACTORQ_ERR_NONFINITE = 3,     /* a weight or bias is NaN or Inf (device status)             */
  ACTORQ_ERR_NOMEM = 4,         /* a device or host allocation failed                         */
  ACTORQ_ERR_CUDA = 5,          /* a CUDA runtime call failed                                 */
  ACTORQ_ERR_TIMEOUT = 6,       /* a bounded device-side wait ran out (device status)         */
  ACTORQ_ERR_SCRATCH_LIMIT = 7  /* actorq_policy_forward_noalloc: batch too large for the fixed scratch */
} actorq_status;

typedef enum { ACTORQ_FC = 0, ACTORQ_CONV2D = 1 } actorq_layer_kind;
typedef enum {
  ACTORQ_HEAD_TANH = 0,    /* D4PG actor: out = tanh(y)                                        */
  ACTORQ_HEAD_ARGMAX = 1,  /* DQN: out = Q-values y, actions = lowest index of the row maximum */
  ACTORQ_HEAD_LINEAR = 2   /* out = y                                                          */
} actorq_head;
typedef enum {
  ACTORQ_OBS_F32 = 0,      /* float observations [batch][obs_dim], row-major                   */
  ACTORQ_OBS_U8_DIV255 = 1 /* uint8 frames [batch][C][H][W] meaning u/255                      */
} actorq_obs_dtype;

/* Real-valued range of one layer's INPUT activation (calibration min and max). */
typedef struct { float min, max; } actorq_range;

/* One layer of the fp32 policy as the learner holds it.
 * FC:     y[n] = sum_k W[n][k] x[k] + b[n];  weight is [out_features][in_features] row-major.
 * CONV2D: valid padding, square stride; weight is [out_c][in_c][kh][kw]; the input is
 *         [in_c][in_h][in_w]; the output [out_c][oh][ow] is flattened in (c, h, w) order
 *         when an FC layer follows.  in_features/out_features are ignored for CONV2D.
 * Every layer except the last is followed by ReLU. */
typedef struct {
  int kind;                               /* actorq_layer_kind                               */
  int in_features, out_features;          /* FC                                              */
  int in_c, in_h, in_w, out_c, kh, kw, stride;   /* CONV2D                                   */
  const float *weight;                    /* device, fp32, caller-owned                      */
  const float *bias;                      /* device, fp32 [out] or NULL (= zeros)            */
  int per_channel;                        /* 0: one delta / zero-point for the tensor; 1: one
                                             per output channel (row of an FC weight), Eq. 1-2
                                             applied to each channel on its own -- the scheme
                                             Section 3.2 uses for convolutional layers          */
} actorq_layer_desc;

/*
 * The quantizer block (Section 3.1, Figure 2b; arithmetic of Section 3.2, Eq. 1-2).
 *
 * Quantizes all `n_layers` weight tensors (per-tensor delta and zero-point), builds
 * the tensor-core-ready weight images and the per-layer integer constants
 *     P = s_a * s_w,  M = P / s_out,  bias_q[n] = rne(b[n] / P) clamped to +-2^30,
 * and stores them in *inout_policy.
 *   layers        host array of n_layers descriptors (read during the call only)
 *   input_ranges  host array of n_layers ranges: range of each layer's input; entry 0 is
 *                 ignored when obs_dtype is ACTORQ_OBS_U8_DIV255
 *   head, obs_dtype   actorq_head / actorq_obs_dtype
 *   inout_policy  *inout_policy == NULL: a policy is allocated (this first call may
 *                 synchronise the device while allocating).  Otherwise the policy must
 *                 have been created with the same architecture; it is re-quantized in
 *                 place with no allocation and no host synchronisation (the per-broadcast
 *                 path), else ACTORQ_ERR_INVALID_ARG.
 * Limits: 1 <= n_layers <= 16; the reduction length of every layer (in_features, or
 * in_c*kh*kw) is at most 16384, so that int32 accumulation is exact.
 * Device-side outcome: ACTORQ_ERR_NONFINITE in the status word if any weight or bias is
 * NaN/Inf (the policy's contents are then unspecified until the next successful quantize).
 */
int actorq_quantize_params(const actorq_layer_desc *layers, int n_layers,
                           const actorq_range *input_ranges, int head, int obs_dtype,
                           void *cuda_stream, actorq_policy **inout_policy);

/*
 * The fp16 actor (Section 3.2: policies are quantized "to fp16 and int8"; Section 5 runs actors and
 * communication at q = 16 as well).  Casts the fp32 policy to binary16 instead of quantizing it to int8:
 * every weight is rounded to nearest even binary16, biases stay binary32.  The resulting policy is used
 * through actorq_policy_forward (also the host-buffer and exploration forms) and computes
 *   layer:  y[n] = sum_k a[k] w[n][k] + b[n]   binary16 operands, binary32 accumulation on the tensor cores
 *   hidden: a_next = round_to_binary16(max(y, 0));   last: out = tanh(y) or y, greedy action as for int8
 * with the observations rounded to binary16 on the way in.  Results agree with a reference that sums in
 * double and rounds once to within the accumulation error of binary32 plus, rarely, one binary16 step of a
 * hidden activation (no bit-exact contract: the tensor core's summation order is not specified).
 *   layers / head / obs_dtype / inout_policy   as for actorq_quantize_params (no activation ranges);
 *                 *inout_policy != NULL must be a policy created by this call with the same architecture:
 *                 it is re-cast in place without allocation or host synchronisation (the per-broadcast path).
 * All-FC policies on float observations, every layer at most 8192 wide, the last at most 128:
 * ACTORQ_ERR_UNSUPPORTED otherwise.  The inspection calls for int8 policies (export_layer, forward_debug,
 * blobs, set_fused_variant, forward_noalloc) return ACTORQ_ERR_UNSUPPORTED for such a policy.
 */
int actorq_cast_params_fp16(const actorq_layer_desc *layers, int n_layers, int head, int obs_dtype,
                            void *cuda_stream, actorq_policy **inout_policy);

/*
 * Actor policy inference with the quantized policy (Section 3.1: the actors run the
 * quantized policy; Section 3.2: weights and activations in the same precision),
 * batched over `batch` independent observations.
 *   obs      device; float [batch][obs_dim] or uint8 [batch][C][H][W], 16-byte aligned
 *   out      device; float [batch][out_dim]: tanh(y), or y (Q-values)
 *   actions  device; int [batch]; required for ACTORQ_HEAD_ARGMAX, ignored otherwise
 * Per layer:  acc = sum_k (a_q - z_a)(w_q - z_w) + bias_q   (int32, exact)
 *   hidden:   a_next = clamp(rne((float)acc * M) + z_next, z_next, 127)   (ReLU = lower clamp)
 *   last:     y = (float)acc * P                                           (Eq. 3)
 * batch == 0 is a no-op.  Rows are independent: a row's result does not depend on
 * batch or on the other rows.  The first call with a larger batch than any before may
 * grow a scratch buffer held by the policy (a synchronising allocation) for the
 * architectures that keep intermediate activations in device memory (convolutional
 * policies and layers wider than the fused kernel supports).
 */
int actorq_policy_forward(actorq_policy *policy, const void *obs, long long batch,
                          float *out, int *actions, void *cuda_stream);

/*
 * actorq_policy_forward without any device-memory allocation.  (The paper has no counterpart:
 * this is a deployment variant of the call above, not a step of the method.)
 *
 * Who needs it: an actor-serving loop that must never call cudaMalloc once it is running --
 * because the learner's framework has already claimed the device's memory for its own caching
 * pool so a late raw allocation may fail, or because an allocation synchronises the whole device
 * and would stall the learner's streams in the middle of an update.  actorq_policy_forward may
 * grow a scratch buffer inside the policy the first time it sees a larger batch;  this entry
 * point never does.  It runs the layer-at-a-time kernels (every architecture, MLP or
 * convolutional) and keeps their two int8 activation buffers in one fixed array of
 * ACTORQ_NOALLOC_SCRATCH_BYTES that is built into the library, so each GPU that loads the
 * library gives up that much memory until the process exits.
 *
 * Arguments and results are those of actorq_policy_forward (same arithmetic, bit for bit, up to
 * the single-precision tanh of the head).  Differences:
 *   - batch * (largest per-observation layer input or output, in elements) must not exceed
 *     ACTORQ_NOALLOC_SCRATCH_BYTES / 2; a larger batch returns ACTORQ_ERR_SCRATCH_LIMIT and
 *     nothing is launched.  (DQN 4x84x84 network: 28224 elements -> batch <= 1188.)
 *   - the policy must have been quantized on the device that is current at the call.
 *   - The first call on each device looks up the array's device address (a one-time set-up that
 *     is not stream work).  With CUDA's lazy module loading that first call is also the one that
 *     makes the driver load the module holding the array, i.e. reserve the 64 MiB, which can
 *     synchronise the device or fail if the memory is gone by then: make it once at start-up,
 *     before the learner has claimed the device and before starting any stream capture.
 *   - All calls, on every policy and stream, share the one array, which simply keeps whatever the
 *     previous call left in it (nothing needs to be cleared: each call overwrites all it reads).
 *     Two calls whose kernels can overlap on the GPU therefore race; order them on one stream or
 *     with events.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.
 */
#define ACTORQ_NOALLOC_SCRATCH_BYTES (64ll << 20)
int actorq_policy_forward_noalloc(actorq_policy *policy, const void *obs, long long batch,
                                  float *out, int *actions, void *cuda_stream);

/* Frees the policy and everything it owns.  Synchronises the device.  NULL is a no-op.
 * (The paper has no counterpart; this is resource management for the two calls above.) */
void actorq_free(actorq_policy *policy);

/* ---- quantized communication: the packed policy blob ---------------------------------------
 * Section 5 of the paper ("Quantization ... communication") broadcasts the quantized policy as
 * int8 weights packed into one matrix, 4x smaller than fp32, and observes that the actor-side
 * re-packing of the weights dominates the load time.  Here the quantized policy can be written
 * to ONE caller-owned device buffer (header, per-layer delta / zero-point / constants, int8
 * codes) and read back into another policy of the same architecture -- e.g. after one NCCL
 * broadcast or peer copy of that buffer -- where a single kernel rebuilds the tensor-core images.
 *   actorq_policy_blob_bytes   size of the blob of this architecture (host result)
 *   actorq_policy_export_blob  blob: device, 16-byte aligned, capacity >= blob_bytes; asynchronous
 *   actorq_policy_import_blob  policy: created earlier by actorq_quantize_params with the same
 *                              layers/head/observation type; bytes must equal blob_bytes, else
 *                              ACTORQ_ERR_INVALID_ARG.  A blob of another architecture or a damaged
 *                              header raises ACTORQ_ERR_INVALID_ARG in the device status word.
 * After import the policy computes exactly what the exporting policy computes. */
int actorq_policy_blob_bytes(const actorq_policy *policy, long long *bytes);
int actorq_policy_export_blob(actorq_policy *policy, void *blob, long long capacity, void *cuda_stream);
int actorq_policy_import_blob(actorq_policy *policy, const void *blob, long long bytes, void *cuda_stream);

/* ---- inspection surface used by the parity tests ------------------------------------ */

/* As actorq_policy_export_layer for a layer quantized per output channel (Section 3.2):
 * scales and zero_points (host) receive out_features / out_c entries each.  Returns
 * ACTORQ_ERR_INVALID_ARG for a per-tensor layer.  Synchronises `cuda_stream`. */
int actorq_policy_export_layer_channels(actorq_policy *policy, int layer, signed char *w_q,
                                        float *scales, int *zero_points, void *cuda_stream);

/* Copies layer `layer`'s int8 weight codes, in the caller's original element order, to
 * w_q (device, as many bytes as the fp32 tensor has elements), and writes its delta and
 * zero-point (Eq. 2) to *scale and *zero_point (host).  Synchronises `cuda_stream`. */
int actorq_policy_export_layer(actorq_policy *policy, int layer, signed char *w_q,
                               float *scale, int *zero_point, void *cuda_stream);

/* Runs the same kernels as actorq_policy_forward and additionally writes, for one layer,
 * its int32 accumulators acc (device, [batch][layer outputs], conv layers in (c, h, w)
 * order) and, for a hidden layer, its requantized int8 activations act_q (device, same
 * shape; pass NULL for the last layer).  out/actions as in actorq_policy_forward. */
int actorq_policy_forward_debug(actorq_policy *policy, const void *obs, long long batch,
                                float *out, int *actions, int layer, int *acc,
                                signed char *act_q, void *cuda_stream);

/* Reads and clears the policy's device status word (an actorq_status).  The caller must
 * have synchronised the streams the policy was used on. */
int actorq_policy_last_device_status(actorq_policy *policy);

/* After actorq_policy_last_device_status returned ACTORQ_ERR_TIMEOUT: where the first bounded
 * wait gave up.  info8 (host, 8 ints): [0] 1 if a report exists, [1] thread block, [2] warp,
 * [3] byte offset of the barrier inside the fused kernel's barrier block, [4] phase parity waited
 * for; the rest 0.  Reading clears the report.  (Diagnostics; the paper has no counterpart.) */
int actorq_policy_timeout_info(actorq_policy *policy, int *info8);

/*
 * Inference of an acting policy with exploration noise (Section 5, experimental set-up: "a Gaussian
 * noise layer [on] the output of the policy network on the actor", sigma assigned per actor
 * between 0 and 0.2).  For ACTORQ_HEAD_TANH policies only (ACTORQ_ERR_UNSUPPORTED otherwise):
 *   out[b][n] = clamp(tanh(y[b][n]) + sigma[b] * noise[b][n], -1, 1)
 * with one binary32 multiply and one binary32 add.  The paper does not say whether the noisy action
 * is clipped; it is clipped here to the range of tanh, the range the actions live in.
 *   sigma  device; float [batch], the row's (actor's) standard deviation
 *   noise  device; float [batch][out_dim], standard normal draws supplied by the caller (the
 *          library draws no random numbers)
 * obs / out / batch / stream as for actorq_policy_forward.
 */
int actorq_policy_forward_explore(actorq_policy *policy, const void *obs, long long batch,
                                  const float *sigma, const float *noise, float *out, void *cuda_stream);

/*
 * The same with the noise drawn inside the library (the paper's actors draw their own noise; Section 5
 * does not say how).  Row b, column n of the call gets the standard normal z of a counter-based
 * generator keyed by (seed, first_row + b, n), so an actor's noise does not depend on the batch its
 * observation travels in, and shards of one batch draw consistently when each passes its first row:
 *   (x0..x3) = Philox-4x32-10(counter = (row mod 2^32, row div 2^32, n div 4, 0), key = (seed mod 2^32, seed div 2^32))
 *   (x0, x1) serves columns 4j, 4j + 1 and (x2, x3) columns 4j + 2, 4j + 3 of block j = n div 4:
 *   u1 = ((xa >> 9) + 1/2) 2^-23,  u2 = ((xb >> 9) + 1/2) 2^-23,
 *   z = sqrt(-2 ln u1) cos(2 pi u2) for even n, ... sin(2 pi u2) for odd n            (Box-Muller)
 *   out[b][n] = clamp(tanh(y[b][n]) + sigma[b] * z, -1, 1)
 * The integer part is exact; the logarithm, square root and sine / cosine are single-precision
 * library functions (a few ulp).  For policies the resident-weights kernel takes, the draw happens in
 * that kernel's head; otherwise in one small kernel behind the forward.  ACTORQ_HEAD_TANH only.
 */
int actorq_policy_forward_explore_seeded(actorq_policy *policy, const void *obs, long long batch, const float *sigma,
                                         unsigned long long seed, long long first_row, float *out, void *cuda_stream);

/*
 * The same inference for callers whose observations live in HOST memory, as the paper's actors'
 * do (Section 3.1: actors run on CPU cores and feed the policy from their environments):
 *   obs_host      host; float [batch][obs_dim] or uint8 [batch][C][H][W]
 *   out_host      host; float [batch][out_dim]
 *   actions_host  host; int [batch]; required for ACTORQ_HEAD_ARGMAX, ignored otherwise
 * The batch is cut into chunks of about 8 MB of observations; a chunk's copy in, its forward (on
 * cuda_stream) and its copy out run on three streams ordered by events, so with PINNED host buffers
 * the copies of neighbouring chunks overlap the compute and the call runs at the speed of the
 * slower of the two (pageable buffers work, without the overlap).  Results are those of
 * actorq_policy_forward on the same rows, bit for bit.  The call returns after enqueueing.  The
 * observations must be in obs_host when the call is made (their copies are not ordered behind
 * cuda_stream, so that they can overlap the end of the previous call); the forwards run behind
 * the work enqueued on cuda_stream before the call, and the outputs are complete once cuda_stream has
 * reached the end of the call (synchronise it, or record an event on it, before reading them, and
 * before overwriting obs_host).
 * The policy owns the staging buffers, two copy streams and the events: the first call (and a call
 * with a larger chunk than any before) allocates device memory, which synchronises the device.
 * One policy runs one such call at a time.
 */
int actorq_policy_forward_host(actorq_policy *policy, const void *obs_host, long long batch,
                               float *out_host, int *actions_host, void *cuda_stream);

/* Which fused MLP kernel actorq_policy_forward uses for an all-FC policy (Section 3.1, actor
 * inference): 0 = the library picks (default: for small policies -- every layer at most 256 wide
 * and 256 deep -- the kernel that keeps the whole int8 policy resident in shared memory and two
 * observation tiles in flight per CTA; otherwise the CTA-pair kernel that streams the weights,
 * tcgen05 cta_group::2; the single-CTA kernel where the device cannot co-schedule pairs),
 * 1 = always the single-CTA kernel, 2 = always the streaming CTA-pair kernel (forward then returns
 * ACTORQ_ERR_UNSUPPORTED / ACTORQ_ERR_CUDA if pairs cannot be launched), 3 = one launch per layer on
 * CTA pairs with the int8 activations kept in device memory between layers (the path policies wider
 * than 1024 take by default, e.g. the paper's 2048-wide actor networks, and policies with
 * per-channel layers; accepted for any all-FC fp32-observation policy with hidden width <= 8192 and
 * head <= 128), 4 = always the resident-weights kernel.  All kernels produce identical results;
 * the switch exists for tests and measurements.  Returns ACTORQ_ERR_UNSUPPORTED for policies the
 * requested kernel does not take. */
int actorq_policy_set_fused_variant(actorq_policy *policy, int variant);

/* Runs a one-warp kernel whose only wait can never be satisfied, with the given limit
 * (1 us .. 1 s): after synchronising, actorq_policy_last_device_status reports
 * ACTORQ_ERR_TIMEOUT and actorq_policy_timeout_info names the wait, and the policy stays usable.
 * This is how the bounded-wait path of the tensor-core kernels is tested without hanging a GPU.
 * (Diagnostics; the paper has no counterpart.) */
int actorq_selftest_bounded_wait(actorq_policy *policy, long long limit_ns, void *cuda_stream);

/* The GPU's achieved dense INT8 tensor-core rate, for roofline denominators: launches a kernel that
 * only issues the instruction the layer kernels use (tcgen05.mma.cta_group::2.kind::i8, M = 256,
 * n = 256, K = 32) on every SM pair -- operands resident in shared memory (a_in_tmem = 0; the two
 * accumulators alternate) or the A operand in tensor memory (a_in_tmem = 1) -- with no epilogue and
 * no memory traffic.  mma_groups (1 .. 2^24) = groups of four instructions per SM pair; *ops (host,
 * may be NULL) receives the integer operations of the launch (2 per multiply-accumulate).  The
 * caller times the launch with events on cuda_stream; rate = *ops / time.  The kernel's only wait is
 * bounded (ACTORQ_ERR_TIMEOUT in the policy's status word); keep a launch to a few milliseconds.
 * (Measurement aid; the paper has no counterpart.) */
int actorq_selftest_int8_mma_peak(actorq_policy *policy, long long mma_groups, int a_in_tmem,
                                  long long *ops, void *cuda_stream);

/* Number of kernel launches the last actorq_policy_forward / actorq_quantize_params call on
 * this policy enqueued (for benchmark bookkeeping). */
int actorq_policy_last_launch_count(const actorq_policy *policy);

/* Library version string, e.g. "actorq-b200 0.1 sm_100a". */
const char *actorq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ACTORQ_H_ */
