// Host-side launchers of the PAAC kernels.  Every function enqueues work on lc.st and
// counts (and optionally times) each kernel launch through lc; none synchronises.
#pragma once
#include "common.cuh"

namespace paac {

// ---- initialisation and environment (env.cu) -----------------------------------------
void launch_init_params(LaunchCtx& lc, const NetDims& nd, uint64_t seed, float* theta);
void launch_cast_bf16(LaunchCtx& lc, const float* src, bf16* dst, size_t n);
// actions == nullptr: start states (step index 0) for every environment
void launch_env_step(LaunchCtx& lc, uint64_t seed, int n_e, const uint64_t* step_base /* device */, uint32_t t,
                     const int32_t* actions, uint32_t term_denom, uint8_t* next_frames, int8_t* rewards,
                     uint8_t* terminals, int32_t* counters /* [3][n_e] */, int pattern_actions = 0 /* > 0: the learnable
                     environment with that many actions */);

// What is left of the heads after the cluster kernel of the fully connected layer: the two halves' dot products
// hp[2][n_e][32], the head biases, and where logits, values, uniforms and actions go (see launch_heads_fused).
struct HeadsTail {
  const float* hp; const float* bpi; const float* bv; int A;
  float* logits; float* values; const int32_t* forced; int32_t* actions; int32_t* sampled; float* uniforms;
  HeadMode mode;
};
// the same step with the action taken inside the kernel, from the heads' partial sums
void launch_env_step_sampling(LaunchCtx& lc, uint64_t seed, int n_e, const uint64_t* step_base, uint32_t t, uint32_t term_denom,
                              uint8_t* next_frames, int8_t* rewards, uint8_t* terminals, int32_t* counters,
                              const HeadsTail& ht, int pattern_actions = 0);

void launch_advance_step(LaunchCtx& lc, uint64_t* step_base, uint32_t by);

// ---- network on the CUDA cores (net_simt.cu) --------------------------------------------
// act[l]: stored activation of layer l for the n states, storage float (PAAC_FP32) or bf16
// scratch: simt_scratch_floats() floats for the split-k partial sums of the fully connected layer (nullptr: no split)
void simt_forward(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta,
                  const bf16* theta16, const uint8_t* frames, int n, void* const act[], float* scratch);
// from gact[fc] (gradient at the fc pre-activation) down to conv1; fills grad for conv and fc layers
void simt_backward(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta,
                   const bf16* theta16, const uint8_t* frames, int n, void* const act[], void* const gact[],
                   float* grad, float* scratch);
// scratch floats simt_backward / heads_backward (n states) and simt_forward (n_fwd states) need for split-k partials
size_t simt_scratch_floats(int arch, const NetDims& nd, int n, int n_fwd);

// ---- network on the tensor cores (net_tc.cu): Nature CNN, bf16 ------------------------------
bool tc_supported(int arch, int prec);
// fc_scratch: tc_fc_scratch_floats(n) floats for the split-k partial sums of the fully connected layer
size_t tc_fc_scratch_floats(int n);
// with fc_splits != nullptr the end of the fully connected layer is shared with launch_heads_fused: either the layer
// is left as *fc_splits > 0 split-k partial sums in fc_scratch (part[split][n][512]) for that kernel to finish, or
// (*fc_splits == 0) the layer is complete and fc_scratch holds the head dot products of the two halves of the
// hidden units, hp[2][n][32], which that call only has to add up
void tc_forward(LaunchCtx& lc, int arch, const NetDims& nd, const float* theta, const bf16* theta16, const bf16* images,
                const uint8_t* frames, int n, void* const act[], float* fc_scratch, uint32_t* error_word,
                int* fc_splits = nullptr);
// transposed / regrouped bf16 weight images the backward contractions read (refreshed after every
// parameter change), and the data-gradient kernels that use them
size_t tc_weight_image_elems();
// (a first-layer weight whose fp16 image would overflow raises DEV_ERR_RANGE in *error_word)
void tc_relayout_weights(LaunchCtx& lc, const NetDims& nd, const bf16* theta16, bf16* images, uint32_t* error_word);
// one block waits at most max_polls polls on a barrier nobody signals, then records the time-out in *error_word
void launch_wait_probe(LaunchCtx& lc, uint32_t max_polls, uint32_t* error_word);
void tc_backward_dgrad_fc(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err);
void tc_backward_dgrad_conv3(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err);
// out_scale: power of two the gradient handed to the first layer is stored with (tc_conv1_grad_scale() when that
// layer's weight gradient runs on the tensor cores, which expects it so; 1 otherwise)
void tc_backward_dgrad_conv2(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err,
                             float out_scale);
float tc_conv1_grad_scale();
// weight + bias gradient of one layer (0 = conv1 .. 3 = fc) as split-k partial sums in its own region of a
// scratch of tc_scratch_floats(B) floats; the regions are noted in a GradSegments list, and
// tc_backward_finish() adds them up into the gradient vector with one launch and empties the list
struct GradSegment { const float* part; float* dst; int splits, J, CO; float scale; int first_group, groups, wide; };
struct GradSegments { GradSegment seg[12]; int n; int total_groups; };
size_t tc_scratch_floats(int n);
// frame stack: out = (three newest channels of prev, newest plane), or four copies of the plane where restart[e] != 0
void launch_stack_push(LaunchCtx& lc, const uint8_t* prev, const uint8_t* newest, const uint8_t* restart /* nullable */,
                       uint8_t* out, int n);
// the same data gradient followed by the first layer's weight gradient, alternating over `chunks` (at most
// TC_MAX_UPDATE_CHUNKS) groups of states; notes the weight gradient's partial sums in *segs
constexpr int TC_MAX_UPDATE_CHUNKS = 4;
void tc_backward_conv2d_conv1w_chunked(LaunchCtx& lc, const NetDims& nd, const bf16* images, const uint8_t* frames, int n,
                                       void* const act[], void* const gact[], float* grad, float* scratch, int chunks,
                                       GradSegments* segs, uint32_t* err);
void tc_backward_wgrad(LaunchCtx& lc, const NetDims& nd, const uint8_t* frames, int n, void* const act[],
                       void* const gact[], float* grad, float* scratch, int layer, GradSegments* segs, uint32_t* err);
// sumsq_partials != nullptr: every block also leaves the sum of squares of the gradient values it wrote in
// sumsq_partials[block]; returns the number of blocks launched
int tc_backward_finish(LaunchCtx& lc, GradSegments* segs, float* sumsq_partials);
// both heads in one kernel: gradient at the fc pre-activation into g_fc, the heads' parameter gradients as one more
// set of partial sums for tc_backward_finish()
bool tc_heads_backward_supported(const NetDims& nd);
void tc_heads_backward(LaunchCtx& lc, const NetDims& nd, const bf16* theta16, const bf16* h, int n, const float* dz,
                       const float* dV, bf16* g_fc, float* grad, float* scratch, GradSegments* segs);
// single layers of the CUDA-core backward pass (the tensor-core update mixes them in where it has no
// kernel of its own yet)
void simt_backward_layer(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta, const bf16* theta16,
                         const uint8_t* frames, int n, void* const act[], void* const gact[], float* grad,
                         float* scratch, int layer, bool wgrad, bool dgrad);

// ---- heads, sampling, returns, loss gradient (heads.cu) -----------------------------------
// logits/values of n states from the fc activation; if actions != nullptr also samples
void launch_heads(LaunchCtx& lc, int prec, const NetDims& nd, const float* theta,
                  const bf16* theta16, const void* h, int n, float* logits, float* values, uint64_t seed,
                  const uint64_t* step_base /* device */, uint32_t t, const int32_t* forced, int32_t* actions, int32_t* sampled /* action before forcing */,
                  float* uniforms, HeadMode mode);
// the same for the tensor-core path, which leaves the fully connected layer as split-k partial sums
// part[split][n][F]: finishes h (sum, bias, ReLU, bf16) into h_out on the way
bool heads_fused_supported(const NetDims& nd);
void launch_heads_fused(LaunchCtx& lc, const NetDims& nd, const float* theta, const bf16* theta16, const float* part,
                        int splits, bf16* h_out, int n, float* logits, float* values, uint64_t seed,
                        const uint64_t* step_base, uint32_t t, const int32_t* forced, int32_t* actions, int32_t* sampled,
                        float* uniforms, HeadMode mode, uint64_t* advance_step = nullptr, uint32_t advance_by = 0);
// advance_step (only honoured with splits == 0, only valid without sampling): the kernel also adds advance_by to the
// environments' step index, which saves the rollout its last launch
// n-step returns and advantages, the loss gradient at the heads and the loss statistics, in one launch
// mode.algo == PAAC_ALGO_NSTEP_Q: the loss is value_coef * (R - Q(s, a))^2 instead (dV = 0, no policy or entropy term)
void launch_returns_head_grad(LaunchCtx& lc, HeadMode mode, int n_e, int t_max, int A, float gamma, float beta, float value_coef,
                              const int8_t* rewards, const uint8_t* terminals, const float* logits, const float* values,
                              const int32_t* actions, float* R, float* adv, float* dz, float* dV,
                              float* loss_terms /* [3][B] */, DeviceStats* stats);
// gradient of the two heads' parameters and of the fc pre-activation
void heads_backward(LaunchCtx& lc, int prec, const NetDims& nd, const float* theta,
                    const bf16* theta16, const void* h, int n, const float* dz, const float* dV, void* gact_fc,
                    float* grad, float* scratch);

// ---- optimiser (optim.cu) -------------------------------------------------------------------
constexpr int NORM_BLOCKS = 1184;
void launch_clip_rmsprop(LaunchCtx& lc, size_t P, float* theta, float* rms, const float* grad,
                         bf16* theta16 /* nullable */, float lr, float rho, float eps, float clip,
                         float* norm_partials /* [NORM_BLOCKS] */, DeviceStats* stats,
                         int ready_partials = 0 /* > 0: norm_partials[0..ready_partials) already hold the squared norm */);

}  // namespace paac
