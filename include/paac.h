/*
 * paac.h -- C boundary of the B200 parallel advantage actor-critic (PAAC) library.
 *
 * One context holds one learner: the parameters theta of a CNN with a softmax
 * policy head and a scalar value head (Section 5.1 of the paper), n_e synthetic
 * environments, and the RMSProp state.  paac_rollout() and paac_update() are the
 * two halves of one pass of Algorithm 1; everything they compute runs in CUDA
 * kernels on the device of the context.  There is no CPU fallback: every entry
 * point that needs the GPU fails with PAAC_ERR_CUDA when it is not there.
 *
 * Conventions
 *   - All functions return an int status (PAAC_OK = 0) unless stated; nothing is
 *     printed, nothing aborts.  paac_strerror() names a status.
 *   - "host" / "device" on a pointer says where the memory lives.
 *   - A context is not thread-safe, and the library keeps per-process caches (tensor maps, kernel
 *     attributes) that are neither locked nor keyed by device: one calling thread and one device per
 *     process (paac_init on a second device returns PAAC_ERR_STATE).  Calls must follow
 *     init -> (rollout -> update)*.
 *   - Work is enqueued on the stream given at init; calls that return data to the
 *     host synchronise that stream, the others do not.
 *   - Indices: t in [0, t_max) is the step inside the current rollout, e in [0, n_e)
 *     the environment, i = t*n_e + e the experience inside the update batch of
 *     B = n_e*t_max.  Frames are uint8 [84][84][4] (row, column, channel).
 *   - Canonical parameter vector (float): layers conv1, conv2, [conv3], fc, policy
 *     head, value head; each layer W then b; conv W as [c_out][k_h][k_w][c_in];
 *     fc W as [out][in] with in enumerated (row, column, channel).
 */
#ifndef PAAC_H_
#define PAAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct paac_ctx paac_ctx;   /* opaque, owned by the library */

/* The two networks of Section 5.1 (layer sizes from the papers it cites):
 * NIPS:   conv 16@8x8/4, conv 32@4x4/2, fc 256
 * NATURE: conv 32@8x8/4, conv 64@4x4/2, conv 64@3x3/1, fc 512      (ReLU, VALID) */
enum { PAAC_ARCH_NIPS = 0, PAAC_ARCH_NATURE = 1 };

/* PAAC_FP32: float storage and arithmetic.
 * PAAC_BF16: bfloat16 weights copies, activations and activation gradients,
 *            float accumulation, float master parameters and optimiser. */
enum { PAAC_FP32 = 0, PAAC_BF16 = 1 };

/* What the learner is (Section 3: the framework does not care how the policy is represented).
 * PAAC_ALGO_A2C:     the parallel advantage actor-critic of Algorithm 1 (Section 4, Eqs. 9-10).
 * PAAC_ALGO_NSTEP_Q: value-based (Section 2.2, Eqs. 2-4): the A outputs of the first head are Q(s, a; theta);
 *                    acting is epsilon-greedy (one Philox uniform u per environment and step: u < epsilon
 *                    explores into action floor((u / epsilon) A), anything else takes the first arg max);
 *                    the value stored for a step is Q(s_t, a_t), the bootstrap value is max_a Q(s_{t_max}, a),
 *                    targets are the same n-step returns, and the loss is the batch mean of
 *                    value_coef (R_t - Q(s_t, a_t))^2 with R constant (Eq. 4 prints the factor -1/2 where the
 *                    derivative of Eq. 3's square has -2: value_coef carries the scale).  The value head is
 *                    carried along unused and receives a zero gradient; entropy_beta is ignored. */
enum { PAAC_ALGO_A2C = 0, PAAC_ALGO_NSTEP_Q = 1 };

/* The synthetic environment inside the library (it stands in for the emulators of the paper's experiments).
 * PAAC_ENV_HASHED:  frames, rewards in {-1, 0, 1} and terminals are hashes of (seed, environment, step, action):
 *                   the workload of the throughput measurements; there is nothing to learn in it.
 * PAAC_ENV_PATTERN: the same hashed frames dimmed to their low six bits, with a band of 84 / n_actions rows set to 255 that names the rewarded
 *                   action of the state (goal = hash(seed, environment, step) mod n_actions); the goal action pays
 *                   +1, any other 0; terminals as above.  A learner can solve it, which the learning-rate rule
 *                   of Section 5.3 (alpha = 0.0007 n_e) is tried on. */
enum { PAAC_ENV_HASHED = 0, PAAC_ENV_PATTERN = 1 };

enum {
  PAAC_OK = 0,
  PAAC_ERR_ARG = 1,        /* null pointer, size or enum out of range */
  PAAC_ERR_WORKSPACE = 2,  /* caller's workspace too small or misaligned */
  PAAC_ERR_CUDA = 3,       /* a CUDA call failed (no device, launch error, ...) */
  PAAC_ERR_NONFINITE = 4,  /* gradient norm was inf/nan: the update was skipped */
  PAAC_ERR_TIMEOUT = 5,    /* a bounded device-side wait gave up */
  PAAC_ERR_STATE = 6,      /* call out of order (update without a fresh rollout, ...) */
  PAAC_ERR_LIMIT = 7,      /* size beyond the fixed capacity of an entry point that cannot allocate */
  PAAC_ERR_RANGE = 8       /* a parameter lies outside the range a kernel's operand format can hold (see
                              paac_set_params) */
};

/* Hyper-parameters.  paac_default_hparams() fills in the values of Section 5.1:
 * gamma 0.99, RMSProp learning rate 0.0224 (= 0.0007 * 32), decay 0.99, epsilon 0.1,
 * clipping threshold 40, entropy weight beta 0.01. */
typedef struct {
  float gamma;          /* discount of the n-step return */
  float lr;             /* RMSProp step size alpha */
  float rms_decay;      /* RMSProp decay of the squared-gradient average */
  float rms_eps;        /* RMSProp epsilon, inside the square root */
  float clip_norm;      /* global L2-norm threshold; <= 0 disables clipping */
  float entropy_beta;   /* weight of the entropy bonus */
  float value_coef;     /* weight of (R - V)^2; Algorithm 1 has no 1/2, so 1 */
  uint32_t term_denom;  /* synthetic environment: a transition is terminal with probability 1/term_denom */
  int precision;        /* PAAC_FP32 or PAAC_BF16 */
  void* workspace;      /* device; caller-owned scratch of >= paac_workspace_bytes(), 256-byte aligned;
                           NULL: the library allocates and owns it */
  size_t workspace_bytes;
  void* stream;         /* cudaStream_t the work is enqueued on; NULL: the default stream */
  int algorithm;        /* PAAC_ALGO_A2C (default) or PAAC_ALGO_NSTEP_Q */
  float epsilon;        /* PAAC_ALGO_NSTEP_Q: exploration probability in [0, 1] (default 0.1) */
  int environment;      /* PAAC_ENV_HASHED (default) or PAAC_ENV_PATTERN */
} paac_hparams;

void paac_default_hparams(paac_hparams* hp /* host, out */);

/* Bytes of device scratch a context of this shape needs (0 on bad arguments). */
size_t paac_workspace_bytes(int arch, int n_e, int t_max, int n_actions, const paac_hparams* hp /* host */);

/* Algorithm 1, first two lines: N = 0, theta Xavier-uniform from `seed` (biases and
 * RMSProp state zero), n_e environments put in their start states.
 * n_e in [1, 65536], t_max in [1, 64], n_actions in [2, 32].  *out is set only on PAAC_OK. */
int paac_init(paac_ctx** out /* host */, int arch, int n_e, int t_max, int n_actions,
              const paac_hparams* hp /* host */, uint64_t seed);

/* Device pointers into the context's buffers, valid until the next paac_rollout()
 * or paac_destroy() on the same context.  Borrowed: never free them. */
typedef struct {
  const uint8_t* frames;      /* device [t_max][n_e][84][84][4]: s_t for t = 0..t_max-1 */
  const uint8_t* next_frames; /* device [n_e][84][84][4]: s_{t_max}, the state the next rollout starts from */
  const int32_t* actions;     /* device [t_max][n_e] */
  const int8_t* rewards;      /* device [t_max][n_e], in {-1, 0, 1}: reward for a_t taken in s_t */
  const uint8_t* terminals;   /* device [t_max][n_e]: 1 if that transition ended an episode */
  const float* values;        /* device [t_max+1][n_e]: V(s_t); row t_max is the bootstrap value */
  const float* logits;        /* device [t_max][n_e][n_actions] */
  const float* uniforms;      /* device [t_max][n_e]: the uniform that picked a_t */
} paac_rollout_view;

/* Algorithm 1, the inner loop and the bootstrap: for t = 0..t_max-1 evaluate the
 * network on s_t for all environments, sample a_t from the softmax policy by
 * inverse CDF with a Philox4x32-10 uniform, step every environment; then evaluate
 * V on the final states.  Asynchronous.  view may be NULL. */
int paac_rollout(paac_ctx* ctx, paac_rollout_view* view /* host, out, nullable */);

typedef struct {
  float policy_loss;   /* -(1/B) sum adv_i log pi(a_i | s_i)                    (0 for PAAC_ALGO_NSTEP_Q) */
  float value_loss;    /* (value_coef/B) sum (R_i - V_i)^2, or (R_i - Q(s_i, a_i))^2 for PAAC_ALGO_NSTEP_Q */
  float entropy;       /* (1/B) sum H(pi(. | s_i))                              (0 for PAAC_ALGO_NSTEP_Q) */
  float grad_norm;     /* global L2 norm before clipping */
  float clip_scale;    /* factor applied to the gradient (1 when not clipped) */
  int32_t status;      /* PAAC_OK, PAAC_ERR_NONFINITE, PAAC_ERR_TIMEOUT or PAAC_ERR_RANGE */
  uint64_t timesteps;  /* N after this update */
} paac_update_stats;

/* Algorithm 1 after the inner loop: returns R_t = r_t + gamma (1 - terminal_t) R_{t+1}
 * from the bootstrap value, advantages R_t - V(s_t) (constants), the batch-mean
 * gradient of  -adv log pi - beta H + value_coef (R - V)^2  (Eqs. 9-10) through the
 * whole network, global-norm clipping, RMSProp, N += n_e * t_max.
 * stats == NULL: asynchronous.  stats != NULL: synchronises and fills it; returns
 * PAAC_ERR_NONFINITE if the update was skipped because the gradient norm was not finite, and
 * PAAC_ERR_TIMEOUT / PAAC_ERR_RANGE if a kernel of this or an earlier call left a device error: the
 * optimiser kernel itself checks the error word and then changes neither parameters nor RMSProp state. */
int paac_update(paac_ctx* ctx, paac_update_stats* stats /* host, out, nullable */);

size_t paac_param_count(const paac_ctx* ctx);

/* Copy the float master parameters (canonical layout) to the host; n must equal
 * paac_param_count().  Synchronises. */
int paac_params(paac_ctx* ctx, float* dst /* host */, size_t n);

/* Release the context and what it owns (never the caller's workspace). */
int paac_destroy(paac_ctx* ctx);

const char* paac_strerror(int status);

/* ---- external-environment mode: the emulators of Algorithm 1's parallel-for live on
 * the host (as in the paper's set-up); frames come in, actions go out ---- */

/* Step t of a rollout with host frames s_t [n_e][84][84][4] (pinned memory advised):
 * copies them in, evaluates the network, samples a_t, copies actions (and values, if
 * values != NULL) out.  t == t_max evaluates the bootstrap value only (actions may be
 * NULL).  Synchronises.  t must run 0, 1, ..., t_max in order.
 * frames may be NULL at t == 0 when the call before it on this context was paac_act_host(t_max) of the previous
 * rollout (with paac_observe_host / paac_update in between or not): s_0 of a rollout is s_{t_max} of the one before
 * (Algorithm 1), and those frames are already on the device, so nothing is copied; the network is evaluated again,
 * with the current parameters.  Anywhere else a NULL frames pointer is PAAC_ERR_ARG. */
int paac_act_host(paac_ctx* ctx, int t, const uint8_t* frames /* host */, int32_t* actions /* host, out */,
                  float* values /* host, out, nullable */);

/* The same step with the state built on the device (Section 5.1: a state is the stack of the four latest
 * pre-processed frames, so three quarters of s_t are already there as part of s_{t-1}): newest [n_e][84][84] uint8
 * (host, pinned memory advised) is the frame that joins the stack; s_t = (the three newest channels of s_{t-1},
 * newest), oldest first.  Where restart[e] != 0 (host, [n_e], nullable = no restarts) environment e has begun a new
 * episode and the new frame fills all four channels.  t = 1 .. t_max (step 0 of a rollout has no new frame: it is the
 * state of the call before, see paac_act_host); calls of the two kinds may be mixed within a rollout.  Copies a
 * quarter of the bytes paac_act_host copies.  Errors as paac_act_host. */
int paac_act_host_newest(paac_ctx* ctx, int t, const uint8_t* newest /* host */, const uint8_t* restart /* host, nullable */,
                         int32_t* actions /* host, out */, float* values /* host, out, nullable */);

/* Outcome of the actions of step t, observed on the host: rewards in {-1,0,1} and
 * terminal flags, [n_e] each.  After step t_max-1 and the bootstrap paac_act_host(t_max),
 * paac_update() may be called. */
int paac_observe_host(paac_ctx* ctx, int t, const int8_t* rewards /* host */, const uint8_t* terminals /* host */);

/* Frame pre-processing of Section 5.1 for real emulators feeding the external-environment mode: of the raw
 * frames one (four times repeated) action produces, the two latest are combined by a per-pixel maximum, turned
 * into pixel intensity, scaled from 210 x 160 to 84 x 84 and appended to the state as its newest channel.
 * Readings where the paper is silent: the maximum is per colour channel; intensity = (77 R + 150 G + 29 B + 128) >> 8;
 * the scaling is the exact area average (every source pixel weighted by the area it shares with the output
 * pixel's box of 2.5 x 40/21 source pixels), rounded half up; channels of a state are its four latest frames,
 * oldest first.
 *   raw_prev, raw_last  device uint8 [n][210][160][3] (row, column, RGB), 16-byte aligned
 *   state_in            device uint8 [n][84][84][4], nullable: the states before this step; NULL (after a reset):
 *                       the new frame fills all four channels
 *   state_out           device uint8 [n][84][84][4]; may be the same buffer as state_in
 *   n in [1, 65535]; stream: cudaStream_t.  Asynchronous; allocates nothing.  Integer arithmetic: results are
 *   the same bits on any machine. */
int paac_preprocess(const uint8_t* raw_prev /* device */, const uint8_t* raw_last /* device */,
                    const uint8_t* state_in /* device, nullable */, uint8_t* state_out /* device */, int n, void* stream);

/* The frame stack of Section 5.1 by itself, on device buffers: state_out = (the three newest channels of state_in,
 * newest), or four copies of newest where restart[e] != 0 (nullable).  state_in / state_out [n][84][84][4] uint8
 * (device, 16-byte aligned; the same buffer may be given for both), newest [n][84][84] uint8 (device, 4-byte
 * aligned), restart [n] uint8 (device).  n = 1 .. 65,535.  Asynchronous on `stream` (a cudaStream_t, 0 = default).
 * The paper states the stack, not a procedure. */
int paac_stack_push(const uint8_t* state_in, const uint8_t* newest, const uint8_t* restart /* nullable */,
                    uint8_t* state_out, int n, void* stream);

/* ---- test and resume hooks ---- */

/* Overwrite the master parameters (and their bf16 copies) from the host. Synchronises.
 * Domain of the first layer in PAAC_BF16 on the Nature network: its forward kernel multiplies fp16 images (the
 * bf16 weight times 2^8 against pixel values as fp16 subnormals), exact for 2^-25 <= |w| <= 255 after the bf16
 * rounding; smaller magnitudes lose low bits (absolute error below 2^-26), larger ones cannot be held.  A vector
 * with a first-layer weight whose bf16 value exceeds 255 in magnitude (or is not finite) is refused with
 * PAAC_ERR_RANGE and nothing is changed.  Should training itself drive such a weight out of range, the update
 * that finds it reports PAAC_ERR_RANGE and the following updates are skipped until the word is cleared
 * (PAAC_DBG_ERROR_WORD). */
int paac_set_params(paac_ctx* ctx, const float* src /* host */, size_t n);

/* Actions to take instead of sampling in the following rollouts: host int32
 * [t_max][n_e], -1 = sample as usual.  NULL clears.  Lets a checker walk in lock
 * step when a uniform falls within rounding of a CDF boundary. */
int paac_force_actions(paac_ctx* ctx, const int32_t* actions /* host, nullable */);

/* Internal tensors readable through paac_debug_read (storage type in brackets;
 * "T" is float in PAAC_FP32 and bfloat16 in PAAC_BF16). */
enum {
  PAAC_DBG_FRAMES = 0,     /* u8  [t_max][n_e][84][84][4] */
  PAAC_DBG_NEXT_FRAMES,    /* u8  [n_e][84][84][4] */
  PAAC_DBG_ACTIONS,        /* i32 [t_max][n_e] */
  PAAC_DBG_REWARDS,        /* i8  [t_max][n_e] */
  PAAC_DBG_TERMINALS,      /* u8  [t_max][n_e] */
  PAAC_DBG_VALUES,         /* f32 [t_max+1][n_e] */
  PAAC_DBG_LOGITS,         /* f32 [t_max][n_e][A] */
  PAAC_DBG_UNIFORMS,       /* f32 [t_max][n_e] */
  PAAC_DBG_COUNTERS,       /* i32 [3][n_e]: episode length, episode return, episodes finished */
  PAAC_DBG_RETURNS,        /* f32 [B] */
  PAAC_DBG_ADVANTAGES,     /* f32 [B] */
  PAAC_DBG_DLOGITS,        /* f32 [B][A] */
  PAAC_DBG_DVALUES,        /* f32 [B] */
  PAAC_DBG_GRAD,           /* f32 [P] gradient of the last update, before clipping */
  PAAC_DBG_RMS,            /* f32 [P] RMSProp state */
  PAAC_DBG_SAMPLED,        /* i32 [t_max][n_e]: the action inverse-CDF sampling gave, before any forcing */
  PAAC_DBG_ERROR_WORD,     /* u32 [1]: sticky device error bits (1, 2, 4: a bounded wait gave up; 8: first-layer
                              weight out of range).  While it is non-zero paac_update leaves parameters and
                              optimiser state untouched and reports the error; a caller that has dealt with the
                              cause (say, restored parameters with paac_set_params) clears it by writing 0.
                              Reading it returns the word together with the status it stands for. */
  PAAC_DBG_ACT0 = 32,      /* T [B][...] stored activation of layer l = which - PAAC_DBG_ACT0
                              (conv layers, then fc) */
  PAAC_DBG_GACT0 = 48      /* T [B][...] gradient w.r.t. the pre-activation of layer l */
};

/* Bytes of tensor `which` (0 if unknown). */
size_t paac_debug_bytes(const paac_ctx* ctx, int which);
/* Copy tensor `which` to the host; bytes must equal paac_debug_bytes(). Synchronises. */
int paac_debug_read(paac_ctx* ctx, int which, void* dst /* host */, size_t bytes);
/* Overwrite tensor `which` from the host (fault injection from the host side, e.g. a
 * poisoned gradient is not possible here since the gradient is recomputed; used for
 * PAAC_DBG_RMS and PAAC_DBG_COUNTERS on resume). Synchronises. */
int paac_debug_write(paac_ctx* ctx, int which, const void* src /* host */, size_t bytes);

/* Run-time options.  PAAC_OPT_CUDA_CORES_ONLY != 0 keeps the bf16 network off the tensor cores
 * (same rounding points, CUDA-core contractions): a second implementation to compare against.
 * PAAC_OPT_TC_WGRAD_LAYERS: bit mask (bit l = layer l, conv1 = 0) of the layers whose weight gradient
 * runs on the tensor cores; the others use the CUDA-core contraction.  Default: all.
 * PAAC_OPT_CUDA_GRAPHS: != 0 (default) lets paac_rollout / paac_update record their kernel sequence into CUDA
 * graphs after two plain iterations and replay them; 0 keeps every call on plain launches.  (Graphs are also
 * bypassed while actions are forced or per-kernel profiling is on.)
 * PAAC_OPT_DEPENDENT_LAUNCH: != 0 (default) launches every kernel with programmatic stream serialization, so
 * that a kernel's CTAs are scheduled while the kernel before it drains (each kernel waits on the device for its
 * predecessor before it touches that kernel's data); 0 launches with plain stream order.  The setting is
 * process-wide.  Results are bit-identical either way.
 * PAAC_OPT_FP32_TENSOR_CORES: != 0 runs every contraction of the CUDA-core path (PAAC_FP32 on either network, and
 * PAAC_BF16 with PAAC_OPT_CUDA_CORES_ONLY) on the tensor cores at float accuracy: each float operand is split into two
 * TF32 pieces (22 significant bits together) and three tcgen05 passes (hi*hi + hi*lo + lo*hi) are accumulated in one
 * float accumulator; what is dropped is below 2^-21 of a product, so results stay within the 1e-4 tolerance of the
 * float path, free-running over ten updates included.  Default 0:
 * with the 20 to 160 rows of the float configurations a 128-row tensor tile is mostly padding.
 * PAAC_OPT_UPDATE_CHUNKS: 1 (default) .. 4.  With more than one, the tensor-core update runs the second layer's data
 * gradient and the first layer's weight gradient alternately over that many groups of states, so that a group's slice
 * of the gradient between them is read back from L2 instead of HBM.  The weight gradient's partial sums are then
 * added in a different grouping: results agree to float rounding, not bit for bit, with the default. */
enum { PAAC_OPT_CUDA_CORES_ONLY = 1, PAAC_OPT_TC_WGRAD_LAYERS = 2, PAAC_OPT_CUDA_GRAPHS = 3, PAAC_OPT_DEPENDENT_LAUNCH = 4,
       PAAC_OPT_FP32_TENSOR_CORES = 5, PAAC_OPT_UPDATE_CHUNKS = 6 };
int paac_set_option(paac_ctx* ctx, int option, int value);

/* Failure-path check that cannot hang: launches one small kernel whose only thread block waits, at most
 * max_polls polls (1 .. 1,000,000, a fraction of a second), on a barrier that nothing ever signals.  The wait
 * runs out, the kernel records that in the context's error word exactly as the network kernels do, releases
 * what it holds and returns; the call synchronises and returns PAAC_ERR_TIMEOUT.  The error word stays set
 * (see PAAC_DBG_ERROR_WORD). */
int paac_debug_wait_probe(paac_ctx* ctx, uint32_t max_polls);

/* Number of kernels the library has launched on this context since init. */
uint64_t paac_launch_count(const paac_ctx* ctx);

/* Per-kernel timing for the time-usage breakdown (the paper's Fig. 2 splits an iteration into
 * environment interaction, action selection and learning).  enable != 0: zero the totals and
 * bracket every following kernel launch with a CUDA event pair on the context's stream;
 * enable == 0: stop.  Synchronises.  Timed runs launch the same kernels, slightly spaced out. */
int paac_profile(paac_ctx* ctx, int enable);
/* Totals since profiling was enabled, one entry per kernel family that ran: names[i] (static
 * strings owned by the library), ms[i] device milliseconds, launches[i].  Arrays are host, sized
 * max_entries.  Returns the number of entries written, or -1 on bad arguments.  Synchronises. */
int paac_profile_read(paac_ctx* ctx, int max_entries, const char** names /* out */, double* ms /* out */,
                      uint64_t* launches /* out */);

/* ---- for callers that may not allocate device memory ----
 *
 * (The paper has no counterpart to this entry point; it exists for deployment constraints.)
 * Some hosts of this library cannot call cudaMalloc at all: a control loop with a frozen memory budget, a
 * process whose device pool belongs to another framework and is fully handed out, a sandbox that only
 * lets pre-built modules touch the GPU.  For them the optimiser step of Algorithm 1 -- global L2-norm
 * clipping followed by RMSProp, as in paac_update -- is offered on plain caller-owned arrays, with the
 * per-slice partial sums of the squared gradient kept in a 16 KB array that is part of the library's
 * device image (each GPU that loads the library holds it until the process exits).  The call allocates
 * and frees nothing, neither through CUDA nor through any library.
 *
 *   theta, rms   device float[n], updated in place      grad   device float[n], read only
 *   theta_bf16   device, nullable: bfloat16 bits of the new theta, [n]
 *   norm_and_scale  device float[2], nullable: gradient norm before clipping, factor applied (0 when
 *                   the norm was not finite and nothing was changed)
 *   stream       cudaStream_t; the two kernels are enqueued on it, the call does not synchronise
 *
 * n may not exceed paac_noalloc_max_params() (16,777,216): beyond that the call returns PAAC_ERR_LIMIT
 * and does nothing.  The first call on each device looks up the device address of the built-in array
 * (cudaGetSymbolAddress) with that device current; make that first call outside any stream capture.
 * All calls on one device share the array, which keeps the last call's sums: every call rewrites the
 * entries it reads before reading them, so nothing has to be cleared, but two calls that overlap on
 * the GPU (on different streams) race on it -- keep them on one stream or order them with events. */
int paac_clip_rmsprop_noalloc(float* theta /* device */, float* rms /* device */, const float* grad /* device */,
                              uint16_t* theta_bf16 /* device, nullable */, size_t n, float lr, float rms_decay,
                              float rms_eps, float clip_norm, float* norm_and_scale /* device, nullable */,
                              void* stream);
size_t paac_noalloc_max_params(void);

#ifdef __cplusplus
}
#endif
#endif /* PAAC_H_ */
