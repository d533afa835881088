// C boundary of the PAAC library: context, workspace carving, and the order in which the
// kernels of one pass of Algorithm 1 are enqueued.
#include <new>
#include <string.h>

#include "kernels.h"

using namespace paac;

struct paac_ctx {
  int arch, n_e, t_max, A, prec, B;
  paac_hparams hp;
  uint64_t seed;
  NetDims nd;
  LaunchCtx lc;            // stream, launch counter, optional per-kernel timing
  cudaStream_t st;
  int device;
  bool owns_workspace;
  char* ws;
  size_t ws_bytes;
  uint64_t N;              // timesteps consumed by updates
  uint64_t env_step;       // global step index of the environments (same for all)
  bool rollout_fresh;      // a rollout has completed since the last update
  uint8_t* newest;         // staging for paac_act_host_newest: [n_e][84][84] planes, then [n_e] restart flags
  int host_t;              // external-environment mode: next expected step
  int update_chunks;       // > 1: conv2 data gradient and conv1 weight gradient alternate over this many groups of states
  bool host_next_valid;    // the bootstrap state of the last host-mode rollout sits where step 0 of the next one goes
  bool forced_on;
  int tc_wgrad_mask;       // bit l: layer l's weight gradient runs on the tensor cores
  GradSegments grad_segs;  // partial-sum regions of the update in flight
  uint64_t* step_dev;      // device copy of env_step; kernels read the step index from here
  // Recorded launch sequences.  The kernels of a rollout (and of an update) take the same arguments every
  // second iteration (the two frame buffers alternate), so after two plain iterations each parity is captured
  // once into a CUDA graph and replayed from then on.  Anything that changes the sequence drops the graphs.
  bool graphs_on;          // option: allow recording
  // recorded launch sequences: kind 0 = rollout, 1 = update, 2 + 2 t + v = step t of the external-environment mode
  // (v = 1: with the frame stack built on the device), each for both parities of the frame buffers
  static constexpr int GRAPH_KINDS = 2 + 2 * 65;
  int plain_calls[GRAPH_KINDS][2];   // calls made with plain launches
  cudaGraphExec_t graph[GRAPH_KINDS][2];
  uint64_t graph_launches[GRAPH_KINDS][2];
  bool simt_only;          // keep the bf16 network on the CUDA cores (cross-check of the tensor-core path)

  // device buffers (all inside the workspace)
  float *theta, *grad, *rms;
  bf16* theta16;
  bf16* w_images;          // regrouped bf16 weights read by the tensor-core backward kernels
  uint8_t* frames[2];      // [t_max][n_e][FRAME_BYTES] each; rollouts alternate, the bootstrap state of one
                           // rollout is written straight into slot 0 of the other
  int cur;                 // buffer the last / current rollout used
  void* act[MAX_LAYERS];   // [(t_max+1)*n_e][out_size], slot t_max is bootstrap scratch
  void* gact[MAX_LAYERS];  // [B][out_size]
  float *logits, *values, *uniforms, *R, *adv, *dz, *dV, *loss_terms, *scratch, *norm_partials;
  float gact0_scale;       // power of two gact[0] was stored with by the last update (1 unless the tensor cores took both kernels)
  size_t simt_scratch_off; // floats: where the CUDA-core kernels' split-k scratch starts inside `scratch`
  int32_t *actions, *sampled, *forced, *counters;
  int8_t* rewards;
  uint8_t* terminals;
  DeviceStats* stats;
  size_t elt;              // bytes of one stored activation element
};

namespace {

struct Carver {
  char* base; size_t off;
  template <class T> T* take(size_t count) {
    off = (off + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

bool valid_shape(int arch, int n_e, int t_max, int A, const paac_hparams* hp) {
  if (hp == nullptr) return false;
  if (arch != PAAC_ARCH_NIPS && arch != PAAC_ARCH_NATURE) return false;
  if (hp->precision != PAAC_FP32 && hp->precision != PAAC_BF16) return false;
  if (n_e < 1 || n_e > 65536 || t_max < 1 || t_max > 64 || A < 2 || A > 32) return false;
  if ((long long)n_e * (t_max + 1) > 131072) return false;   // keeps every row index below 2^31
  if (hp->term_denom == 0) return false;
  if (hp->algorithm != PAAC_ALGO_A2C && hp->algorithm != PAAC_ALGO_NSTEP_Q) return false;
  if (!(hp->epsilon >= 0.f && hp->epsilon <= 1.f)) return false;
  if (hp->environment != PAAC_ENV_HASHED && hp->environment != PAAC_ENV_PATTERN) return false;
  return true;
}

// lays the buffers out; with base == nullptr only measures
size_t carve(paac_ctx* c, char* base) {
  Carver k{base, 0};
  const NetDims& nd = c->nd;
  const size_t n_e = c->n_e, T = c->t_max, B = c->B, A = c->A;
  c->theta = k.take<float>(nd.P);
  c->grad = k.take<float>(nd.P);
  c->rms = k.take<float>(nd.P);
  c->theta16 = k.take<bf16>(nd.P);
  c->w_images = k.take<bf16>(tc_supported(c->arch, c->prec) ? tc_weight_image_elems() : 0);
  c->frames[0] = k.take<uint8_t>(T * n_e * FRAME_BYTES);
  c->frames[1] = k.take<uint8_t>(T * n_e * FRAME_BYTES);
  c->newest = k.take<uint8_t>(n_e * (FRAME_H * FRAME_W + 4));          // newest planes from the host, then restart flags
  for (int l = 0; l <= nd.n_conv; ++l) {
    c->act[l] = k.take<char>((T + 1) * n_e * nd.layer[l].out_size * c->elt);
    c->gact[l] = k.take<char>(B * nd.layer[l].out_size * c->elt);
  }
  c->logits = k.take<float>((T + 1) * n_e * A);
  c->values = k.take<float>((T + 1) * n_e);
  c->uniforms = k.take<float>(B);
  c->R = k.take<float>(B);
  c->adv = k.take<float>(B);
  c->dz = k.take<float>(B * A);
  c->dV = k.take<float>(B);
  c->loss_terms = k.take<float>(3 * B);
  {
    // the tensor-core weight gradients keep their partial sums until the finishing kernel has run, so a layer that
    // is taken on the CUDA cores in the same update works in a region of its own behind them
    size_t sc = simt_scratch_floats(c->arch, nd, (int)B, (int)n_e);
    c->simt_scratch_off = 0;
    if (tc_supported(c->arch, c->prec)) {
      c->simt_scratch_off = (tc_scratch_floats((int)B) + 63) / 64 * 64;
      sc += c->simt_scratch_off;
      if (tc_fc_scratch_floats((int)n_e) > sc) sc = tc_fc_scratch_floats((int)n_e);
    }
    c->scratch = k.take<float>(sc);
  }
  c->norm_partials = k.take<float>(NORM_BLOCKS);
  c->actions = k.take<int32_t>(B);
  c->sampled = k.take<int32_t>(B);
  c->forced = k.take<int32_t>(B);
  c->counters = k.take<int32_t>(3 * n_e);
  c->rewards = k.take<int8_t>(B);
  c->terminals = k.take<uint8_t>(B);
  c->stats = k.take<DeviceStats>(1);
  c->step_dev = k.take<uint64_t>(1);
  return (k.off + 255) & ~(size_t)255;
}

void fill_shape(paac_ctx* c, int arch, int n_e, int t_max, int A, const paac_hparams* hp) {
  c->arch = arch; c->n_e = n_e; c->t_max = t_max; c->A = A; c->B = n_e * t_max;
  c->hp = *hp; c->prec = hp->precision;
  c->nd = make_net(arch, A);
  c->elt = hp->precision == PAAC_BF16 ? 2 : 4;
}

int cuda_status(paac_ctx* c) {
  const bool launches_ok = cudaGetLastError() == cudaSuccess;
  return launches_ok && !c->lc.host_failure ? PAAC_OK : PAAC_ERR_CUDA;
}

bool use_tc(const paac_ctx* c) { return tc_supported(c->arch, c->prec) && !c->simt_only; }
HeadMode head_mode(const paac_ctx* c) { return HeadMode{c->hp.algorithm, c->hp.epsilon}; }
int pattern_actions(const paac_ctx* c) { return c->hp.environment == PAAC_ENV_PATTERN ? c->A : 0; }

// bf16 copies of the master parameters, in the canonical layout and regrouped for the backward kernels
void refresh_weight_copies(paac_ctx* c, bool cast) {
  if (cast) launch_cast_bf16(c->lc, c->theta, c->theta16, c->nd.P);
  if (tc_supported(c->arch, c->prec)) tc_relayout_weights(c->lc, c->nd, c->theta16, c->w_images, &c->stats->error_word);
}

// network + heads on the n_e states of `frames`, activations into slot `slot`.  With `tail` the caller is about
// to step the synthetic environments and can take the actions there: if the forward pass left the heads as partial
// sums (see HeadsTail), no sampling kernel is launched, *tail describes what is left, and the result is true.
bool forward_slot(paac_ctx* c, const uint8_t* frames, int slot, bool sample, HeadsTail* tail = nullptr,
                  bool* advanced = nullptr) {
  void* act[MAX_LAYERS];
  for (int l = 0; l <= c->nd.n_conv; ++l)
    act[l] = (char*)c->act[l] + (size_t)slot * c->n_e * c->nd.layer[l].out_size * c->elt;
  const size_t row = (size_t)slot * c->n_e;
  const int32_t* forced = sample && c->forced_on ? c->forced + row : nullptr;
  int32_t* actions = sample ? c->actions + row : nullptr;
  int32_t* sampled = sample ? c->sampled + row : nullptr;
  float* uniforms = sample ? c->uniforms + row : nullptr;
  if (use_tc(c) && heads_fused_supported(c->nd)) {
    int splits = 0;
    tc_forward(c->lc, c->arch, c->nd, c->theta, c->theta16, c->w_images, frames, c->n_e, act, c->scratch,
               &c->stats->error_word, &splits);
    if (tail != nullptr && splits == 0 && sample) {
      *tail = HeadsTail{c->scratch, c->theta + c->nd.pi_b, c->theta + c->nd.v_b, c->A, c->logits + row * c->A,
                        c->values + row, forced, actions, sampled, uniforms, head_mode(c)};
      return true;
    }
    launch_heads_fused(c->lc, c->nd, c->theta, c->theta16, c->scratch, splits, (bf16*)act[c->nd.n_conv], c->n_e,
                       c->logits + row * c->A, c->values + row, c->seed, c->step_dev, (uint32_t)slot, forced, actions,
                       sampled, uniforms, head_mode(c), (advanced && splits == 0 && !sample) ? c->step_dev : nullptr, (uint32_t)c->t_max);
    if (advanced) *advanced = splits == 0 && !sample;      // the sampling kernel has moved the step index on
    return false;
  }
  if (use_tc(c))
    tc_forward(c->lc, c->arch, c->nd, c->theta, c->theta16, c->w_images, frames, c->n_e, act, c->scratch,
               &c->stats->error_word);
  else
    simt_forward(c->lc, c->arch, c->prec, c->nd, c->theta, c->theta16, frames, c->n_e, act, c->scratch + c->simt_scratch_off);
  launch_heads(c->lc, c->prec, c->nd, c->theta, c->theta16, act[c->nd.n_conv], c->n_e,
               c->logits + row * c->A, c->values + row, c->seed, c->step_dev, (uint32_t)slot, forced, actions, sampled,
               uniforms, head_mode(c));
  return false;
}

void drop_graphs(paac_ctx* c) {
  for (int k = 0; k < paac_ctx::GRAPH_KINDS; ++k)
    for (int par = 0; par < 2; ++par) {
      if (c->graph[k][par]) { cudaGraphExecDestroy(c->graph[k][par]); c->graph[k][par] = nullptr; }
      c->plain_calls[k][par] = 0;
    }
}

// Runs `enqueue` (which only launches kernels on c->st) either directly, or -- once this kind/parity has run
// directly before -- records it into a graph and replays the graph.
template <class F> void run_recorded(paac_ctx* c, int kind, int parity, F enqueue) {
  const bool allowed = c->graphs_on && !c->lc.profiling && !c->forced_on;
  if (allowed && c->graph[kind][parity]) {
    if (cudaGraphLaunch(c->graph[kind][parity], c->st) == cudaSuccess) { c->lc.count += c->graph_launches[kind][parity]; return; }
    cudaGetLastError();
    drop_graphs(c);
  }
  if (allowed && c->plain_calls[kind][parity] >= 1) {
    cudaGraph_t g = nullptr;
    if (cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
      const uint64_t before = c->lc.count;
      c->lc.serialize_next = true;
      enqueue();
      const uint64_t launched = c->lc.count - before;
      cudaGraphExec_t exec = nullptr;
      if (cudaStreamEndCapture(c->st, &g) == cudaSuccess && g != nullptr &&
          cudaGraphInstantiate(&exec, g, 0) == cudaSuccess) {
        cudaGraphDestroy(g);
        c->graph[kind][parity] = exec;
        c->graph_launches[kind][parity] = launched;
        if (cudaGraphLaunch(exec, c->st) == cudaSuccess) return;
      }
      if (g) cudaGraphDestroy(g);
      cudaGetLastError();
      c->lc.count = before;
      c->graphs_on = false;        // recording does not work here (e.g. the caller is capturing): plain launches only
      drop_graphs(c);
    } else {
      cudaGetLastError();
      c->graphs_on = false;
    }
  }
  c->lc.serialize_next = true;
  enqueue();
  ++c->plain_calls[kind][parity];
}

}  // namespace

extern "C" {

void paac_default_hparams(paac_hparams* hp) {
  if (!hp) return;
  memset(hp, 0, sizeof(*hp));
  hp->gamma = 0.99f; hp->lr = 0.0224f; hp->rms_decay = 0.99f; hp->rms_eps = 0.1f;
  hp->clip_norm = 40.f; hp->entropy_beta = 0.01f; hp->value_coef = 1.f;
  hp->term_denom = 200; hp->precision = PAAC_FP32;
  hp->algorithm = PAAC_ALGO_A2C; hp->epsilon = 0.1f; hp->environment = PAAC_ENV_HASHED;
}

size_t paac_workspace_bytes(int arch, int n_e, int t_max, int n_actions, const paac_hparams* hp) {
  if (!valid_shape(arch, n_e, t_max, n_actions, hp)) return 0;
  paac_ctx tmp{};
  fill_shape(&tmp, arch, n_e, t_max, n_actions, hp);
  return carve(&tmp, nullptr);
}

int paac_init(paac_ctx** out, int arch, int n_e, int t_max, int n_actions, const paac_hparams* hp, uint64_t seed) {
  if (!out || !valid_shape(arch, n_e, t_max, n_actions, hp)) return PAAC_ERR_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  // the per-process caches (tensor maps, kernel attributes, SM count) belong to the first device used
  static int process_device = -1;
  if (process_device < 0) process_device = dev;
  if (dev != process_device) return PAAC_ERR_STATE;
  paac_ctx* c = new (std::nothrow) paac_ctx{};
  if (!c) return PAAC_ERR_CUDA;
  fill_shape(c, arch, n_e, t_max, n_actions, hp);
  c->tc_wgrad_mask = 0xF;
  c->update_chunks = 1;
  c->gact0_scale = 1.f;
  c->graphs_on = true;
  c->seed = seed; c->device = dev; c->st = (cudaStream_t)hp->stream; c->lc.st = c->st;
  const size_t need = carve(c, nullptr);
  if (hp->workspace) {
    if (hp->workspace_bytes < need || ((uintptr_t)hp->workspace & 255)) { delete c; return PAAC_ERR_WORKSPACE; }
    c->ws = (char*)hp->workspace; c->owns_workspace = false;
  } else {
    if (cudaMalloc((void**)&c->ws, need) != cudaSuccess) { cudaGetLastError(); delete c; return PAAC_ERR_CUDA; }
    c->owns_workspace = true;
  }
  c->ws_bytes = need;
  carve(c, c->ws);
  c->lc.error_word = &c->stats->error_word;
  cudaMemsetAsync(c->ws, 0, need, c->st);
  cudaMemsetAsync(c->forced, 0xFF, (size_t)c->B * sizeof(int32_t), c->st);
  launch_init_params(c->lc, c->nd, seed, c->theta);
  refresh_weight_copies(c, true);
  c->cur = 1;   // the first rollout flips to buffer 0; its start states are written there now
  launch_env_step(c->lc, seed, n_e, c->step_dev, 0u, nullptr, hp->term_denom, c->frames[0], nullptr, nullptr, nullptr,
                  pattern_actions(c));
  if (cudaStreamSynchronize(c->st) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
    if (c->owns_workspace) cudaFree(c->ws);
    delete c;
    return PAAC_ERR_CUDA;
  }
  *out = c;
  return PAAC_OK;
}

int paac_rollout(paac_ctx* c, paac_rollout_view* view) {
  if (!c) return PAAC_ERR_ARG;
  if (c->host_t != 0) return PAAC_ERR_STATE;
  c->host_next_valid = false;
  c->cur ^= 1;
  uint8_t* fr = c->frames[c->cur];
  uint8_t* nxt = c->frames[c->cur ^ 1];
  const size_t fstep = (size_t)c->n_e * FRAME_BYTES;
  run_recorded(c, 0, c->cur, [&]() {
    for (int t = 0; t < c->t_max; ++t) {
      HeadsTail tail;
      const bool deferred = forward_slot(c, fr + t * fstep, t, true, &tail);
      uint8_t* dst = t + 1 < c->t_max ? fr + (t + 1) * fstep : nxt;
      const size_t row = (size_t)t * c->n_e;
      if (deferred)
        launch_env_step_sampling(c->lc, c->seed, c->n_e, c->step_dev, (uint32_t)t, c->hp.term_denom, dst, c->rewards + row,
                                 c->terminals + row, c->counters, tail, pattern_actions(c));
      else
        launch_env_step(c->lc, c->seed, c->n_e, c->step_dev, (uint32_t)t, c->actions + row, c->hp.term_denom, dst,
                        c->rewards + row, c->terminals + row, c->counters, pattern_actions(c));
    }
    bool advanced = false;
    forward_slot(c, nxt, c->t_max, false, nullptr, &advanced);
    if (!advanced) launch_advance_step(c->lc, c->step_dev, (uint32_t)c->t_max);
  });
  c->env_step += c->t_max;
  c->rollout_fresh = true;
  if (view) {
    view->frames = fr; view->next_frames = nxt; view->actions = c->actions; view->rewards = c->rewards;
    view->terminals = c->terminals; view->values = c->values; view->logits = c->logits; view->uniforms = c->uniforms;
  }
  return cuda_status(c);
}

int paac_update(paac_ctx* c, paac_update_stats* stats) {
  if (!c) return PAAC_ERR_ARG;
  if (!c->rollout_fresh) return PAAC_ERR_STATE;
  const paac_hparams& hp = c->hp;
  run_recorded(c, 1, c->cur, [&]() {
    launch_returns_head_grad(c->lc, head_mode(c), c->n_e, c->t_max, c->A, hp.gamma, hp.entropy_beta, hp.value_coef, c->rewards,
                             c->terminals, c->logits, c->values, c->actions, c->R, c->adv, c->dz, c->dV, c->loss_terms,
                             c->stats);
    const int L = c->nd.n_conv;
    if (use_tc(c) && tc_heads_backward_supported(c->nd))
      tc_heads_backward(c->lc, c->nd, c->theta16, (const bf16*)c->act[L], c->B, c->dz, c->dV, (bf16*)c->gact[L], c->grad,
                        c->scratch, &c->grad_segs);
    else
      heads_backward(c->lc, c->prec, c->nd, c->theta, c->theta16, c->act[L], c->B, c->dz, c->dV, c->gact[L],
                     c->grad, c->scratch + c->simt_scratch_off);
    uint32_t* err = &c->stats->error_word;
    c->gact0_scale = 1.f;
    const bool chunked = use_tc(c) && c->update_chunks > 1 && (c->tc_wgrad_mask & 3) == 3;
    for (int l = L; l >= 0; --l) {
      // tensor-core kernels where they exist, the CUDA-core contraction otherwise
      if (chunked && l == 1) {
        // the layer's own weight gradient first, then data gradient and first-layer weight gradient group by group
        tc_backward_wgrad(c->lc, c->nd, c->frames[c->cur], c->B, c->act, c->gact, c->grad, c->scratch, 1, &c->grad_segs, err);
        c->gact0_scale = tc_conv1_grad_scale();
        tc_backward_conv2d_conv1w_chunked(c->lc, c->nd, c->w_images, c->frames[c->cur], c->B, c->act, c->gact, c->grad,
                                          c->scratch, c->update_chunks, &c->grad_segs, err);
        break;
      }
      bool dgrad_done = false;
      if (use_tc(c)) {
        if (l == 3) { tc_backward_dgrad_fc(c->lc, c->w_images, c->B, c->act, c->gact, err); dgrad_done = true; }
        if (l == 2) { tc_backward_dgrad_conv3(c->lc, c->w_images, c->B, c->act, c->gact, err); dgrad_done = true; }
        if (l == 1) {
          // the first layer's tensor-core weight gradient takes its gradient operand times a power of two
          c->gact0_scale = (c->tc_wgrad_mask & 1) ? tc_conv1_grad_scale() : 1.f;
          tc_backward_dgrad_conv2(c->lc, c->w_images, c->B, c->act, c->gact, err, c->gact0_scale);
          dgrad_done = true;
        }
      }
      bool wgrad_done = false;
      if (use_tc(c) && (c->tc_wgrad_mask >> l) & 1) {
        tc_backward_wgrad(c->lc, c->nd, c->frames[c->cur], c->B, c->act, c->gact, c->grad, c->scratch, l, &c->grad_segs, err);
        wgrad_done = true;
      }
      if (!wgrad_done || (l > 0 && !dgrad_done))
        simt_backward_layer(c->lc, c->arch, c->prec, c->nd, c->theta, c->theta16, c->frames[c->cur], c->B, c->act,
                            c->gact, c->grad, c->scratch + c->simt_scratch_off, l, !wgrad_done, l > 0 && !dgrad_done);
    }
    // when every gradient goes through the finishing kernel, it also delivers the squared norm
    const bool all_finished = use_tc(c) && c->tc_wgrad_mask == 0xF && tc_heads_backward_supported(c->nd);
    int ready = 0;
    if (use_tc(c)) ready = tc_backward_finish(c->lc, &c->grad_segs, all_finished ? c->norm_partials : nullptr);
    launch_clip_rmsprop(c->lc, c->nd.P, c->theta, c->rms, c->grad,
                        c->prec == PAAC_BF16 ? c->theta16 : nullptr, hp.lr, hp.rms_decay, hp.rms_eps, hp.clip_norm,
                        c->norm_partials, c->stats, all_finished ? ready : 0);
    if (c->prec == PAAC_BF16) refresh_weight_copies(c, false);
  });
  c->N += (uint64_t)c->B;
  c->rollout_fresh = false;
  if (cuda_status(c) != PAAC_OK) return PAAC_ERR_CUDA;
  if (stats) {
    DeviceStats ds;
    if (cudaMemcpyAsync(&ds, c->stats, sizeof(ds), cudaMemcpyDeviceToHost, c->st) != cudaSuccess ||
        cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
    stats->policy_loss = ds.policy_loss; stats->value_loss = ds.value_loss; stats->entropy = ds.entropy;
    stats->grad_norm = ds.grad_norm; stats->clip_scale = ds.clip_scale; stats->status = ds.status;
    stats->timesteps = c->N;
    if (ds.error_word) return status_of_error_word(ds.error_word);
    if (ds.status != PAAC_OK) return ds.status;
  }
  return PAAC_OK;
}

size_t paac_param_count(const paac_ctx* c) { return c ? c->nd.P : 0; }

// a kernel whose bounded wait gave up leaves a bit in the device error word
static int device_error(paac_ctx* c) {
  uint32_t w = 0;
  if (cudaMemcpyAsync(&w, &c->stats->error_word, sizeof(w), cudaMemcpyDeviceToHost, c->st) != cudaSuccess ||
      cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  return status_of_error_word(w);
}

int paac_params(paac_ctx* c, float* dst, size_t n) {
  if (!c || !dst || n != c->nd.P) return PAAC_ERR_ARG;
  if (cudaMemcpyAsync(dst, c->theta, n * sizeof(float), cudaMemcpyDeviceToHost, c->st) != cudaSuccess ||
      cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  return device_error(c);
}

int paac_set_params(paac_ctx* c, const float* src, size_t n) {
  if (c) c->lc.serialize_next = true;
  if (!c || !src || n != c->nd.P) return PAAC_ERR_ARG;
  if (tc_supported(c->arch, c->prec)) {
    // the forward kernel of the first layer holds its weights as fp16(bf16(w) * 2^8): |bf16(w)| <= 255
    const LayerDims& d = c->nd.layer[0];
    const size_t count = (size_t)d.CO * d.K * d.K * d.C;
    for (size_t i = 0; i < count; ++i) {
      uint32_t u;
      memcpy(&u, &src[d.w_off + i], 4);
      u &= 0x7FFFFFFFu;
      if (u >= 0x7F800000u) return PAAC_ERR_RANGE;                  // inf / nan
      u += 0x7FFFu + ((u >> 16) & 1u);                              // round to nearest even at bit 16
      if ((u >> 16) > 0x437Fu) return PAAC_ERR_RANGE;               // bf16 bits of 255.0
    }
  }
  if (cudaMemcpyAsync(c->theta, src, n * sizeof(float), cudaMemcpyHostToDevice, c->st) != cudaSuccess) {
    cudaGetLastError(); return PAAC_ERR_CUDA;
  }
  refresh_weight_copies(c, true);
  if (cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  return cuda_status(c);
}

int paac_force_actions(paac_ctx* c, const int32_t* actions) {
  if (!c) return PAAC_ERR_ARG;
  if (!actions) { c->forced_on = false; return PAAC_OK; }
  for (int i = 0; i < c->B; ++i)
    if (actions[i] < -1 || actions[i] >= c->A) return PAAC_ERR_ARG;
  if (cudaMemcpyAsync(c->forced, actions, (size_t)c->B * sizeof(int32_t), cudaMemcpyHostToDevice, c->st) != cudaSuccess ||
      cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  c->forced_on = true;
  return PAAC_OK;
}

int paac_destroy(paac_ctx* c) {
  if (!c) return PAAC_ERR_ARG;
  cudaStreamSynchronize(c->st);
  drop_graphs(c);
  c->lc.release();
  if (c->owns_workspace) cudaFree(c->ws);
  cudaGetLastError();
  delete c;
  return PAAC_OK;
}

const char* paac_strerror(int s) {
  switch (s) {
    case PAAC_OK: return "ok";
    case PAAC_ERR_ARG: return "bad argument";
    case PAAC_ERR_WORKSPACE: return "workspace too small or misaligned";
    case PAAC_ERR_CUDA: return "CUDA error (no device, allocation or launch failure)";
    case PAAC_ERR_NONFINITE: return "gradient norm not finite: update skipped";
    case PAAC_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case PAAC_ERR_STATE: return "call out of order";
    case PAAC_ERR_LIMIT: return "size beyond the fixed capacity of a non-allocating entry point";
    case PAAC_ERR_RANGE: return "a parameter lies outside the range a kernel's operand format can hold";
    default: return "unknown status";
  }
}

int paac_debug_wait_probe(paac_ctx* c, uint32_t max_polls) {
  if (c) c->lc.serialize_next = true;
  if (!c || max_polls < 1u || max_polls > 1000000u) return PAAC_ERR_ARG;
  launch_wait_probe(c->lc, max_polls, &c->stats->error_word);
  if (cuda_status(c) != PAAC_OK) return PAAC_ERR_CUDA;
  return device_error(c);
}

uint64_t paac_launch_count(const paac_ctx* c) { return c ? c->lc.count : 0; }

int paac_set_option(paac_ctx* c, int option, int value) {
  if (!c) return PAAC_ERR_ARG;
  if (option == PAAC_OPT_CUDA_CORES_ONLY) { c->simt_only = value != 0; drop_graphs(c); return PAAC_OK; }
  if (option == PAAC_OPT_TC_WGRAD_LAYERS) { c->tc_wgrad_mask = value & 0xF; drop_graphs(c); return PAAC_OK; }
  if (option == PAAC_OPT_CUDA_GRAPHS) { c->graphs_on = value != 0; drop_graphs(c); return PAAC_OK; }
  if (option == PAAC_OPT_DEPENDENT_LAUNCH) { pdl_enabled() = value != 0; drop_graphs(c); return PAAC_OK; }
  if (option == PAAC_OPT_UPDATE_CHUNKS) {
    if (value < 1 || value > TC_MAX_UPDATE_CHUNKS) return PAAC_ERR_ARG;
    c->update_chunks = value; drop_graphs(c); return PAAC_OK;
  }
  if (option == PAAC_OPT_FP32_TENSOR_CORES) { c->lc.fp32_tensor_cores = value != 0; drop_graphs(c); return PAAC_OK; }
  return PAAC_ERR_ARG;
}

int paac_profile(paac_ctx* c, int enable) {
  if (!c) return PAAC_ERR_ARG;
  if (cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  c->lc.collect();
  if (enable) { for (int i = 0; i < KID_COUNT; ++i) { c->lc.ms[i] = 0.0; c->lc.calls[i] = 0; } }
  c->lc.profiling = enable != 0;
  return PAAC_OK;
}

int paac_profile_read(paac_ctx* c, int max_entries, const char** names, double* ms, uint64_t* launches) {
  if (!c || max_entries < 0 || !names || !ms || !launches) return -1;
  if (cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return -1; }
  c->lc.collect();
  int n = 0;
  for (int i = 0; i < KID_COUNT && n < max_entries; ++i) {
    if (c->lc.calls[i] == 0) continue;
    names[n] = kernel_name(i); ms[n] = c->lc.ms[i]; launches[n] = c->lc.calls[i];
    ++n;
  }
  return n;
}

// ---- external-environment mode ------------------------------------------------------------------
// Step t of an external-environment rollout once the host's bytes are on their way: (the frame stack,) the network on
// the state at `dst` -- a recorded sequence from the second time on --, results to the host, bookkeeping.
static int act_host_finish(paac_ctx* c, int t, const uint8_t* prev, uint8_t* dst, int32_t* actions, float* values) {
  const bool sample = t < c->t_max;
  const size_t plane = (size_t)c->n_e * FRAME_H * FRAME_W;
  run_recorded(c, 2 + 2 * t + (prev ? 1 : 0), c->cur, [&]() {
    if (prev) launch_stack_push(c->lc, prev, c->newest, c->newest + plane, dst, c->n_e);
    forward_slot(c, dst, t, sample);
  });
  const size_t row = (size_t)t * c->n_e;
  if (sample) cudaMemcpyAsync(actions, c->actions + row, c->n_e * sizeof(int32_t), cudaMemcpyDeviceToHost, c->st);
  if (values) cudaMemcpyAsync(values, c->values + row, c->n_e * sizeof(float), cudaMemcpyDeviceToHost, c->st);
  if (cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  if (t == c->t_max) {
    launch_advance_step(c->lc, c->step_dev, (uint32_t)c->t_max);
    c->host_t = 0; c->env_step += c->t_max; c->rollout_fresh = true; c->host_next_valid = true;
  }
  else c->host_t = t + 1;
  return cuda_status(c);
}

int paac_act_host(paac_ctx* c, int t, const uint8_t* frames, int32_t* actions, float* values) {
  if (c) c->lc.serialize_next = true;
  if (!c || t < 0 || t > c->t_max || (t < c->t_max && !actions)) return PAAC_ERR_ARG;
  if (t != c->host_t) return PAAC_ERR_STATE;
  // s_0 of a rollout is s_{t_max} of the one before (Algorithm 1): those frames are on the device already
  if (!frames && !(t == 0 && c->host_next_valid)) return PAAC_ERR_ARG;
  const size_t fstep = (size_t)c->n_e * FRAME_BYTES;
  if (t == 0) c->cur ^= 1;
  uint8_t* dst = t < c->t_max ? c->frames[c->cur] + t * fstep : c->frames[c->cur ^ 1];
  if (frames && cudaMemcpyAsync(dst, frames, fstep, cudaMemcpyHostToDevice, c->st) != cudaSuccess) {
    cudaGetLastError(); return PAAC_ERR_CUDA;
  }
  return act_host_finish(c, t, nullptr, dst, actions, values);
}

int paac_act_host_newest(paac_ctx* c, int t, const uint8_t* newest, const uint8_t* restart, int32_t* actions, float* values) {
  if (c) c->lc.serialize_next = true;
  if (!c || !newest || t < 1 || t > c->t_max || (t < c->t_max && !actions)) return PAAC_ERR_ARG;
  if (t != c->host_t) return PAAC_ERR_STATE;
  const size_t fstep = (size_t)c->n_e * FRAME_BYTES, plane = (size_t)c->n_e * FRAME_H * FRAME_W;
  const uint8_t* prev = c->frames[c->cur] + (size_t)(t - 1) * fstep;
  uint8_t* dst = t < c->t_max ? c->frames[c->cur] + t * fstep : c->frames[c->cur ^ 1];
  // the restart flags always live on the device (all zero when the host has none), so that the recorded sequence
  // is the same either way
  const cudaError_t e1 = cudaMemcpyAsync(c->newest, newest, plane, cudaMemcpyHostToDevice, c->st);
  const cudaError_t e2 = restart ? cudaMemcpyAsync(c->newest + plane, restart, c->n_e, cudaMemcpyHostToDevice, c->st)
                                 : cudaMemsetAsync(c->newest + plane, 0, c->n_e, c->st);
  if (e1 != cudaSuccess || e2 != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  return act_host_finish(c, t, prev, dst, actions, values);
}

int paac_observe_host(paac_ctx* c, int t, const int8_t* rewards, const uint8_t* terminals) {
  if (c) c->lc.serialize_next = true;
  if (!c || !rewards || !terminals || t < 0 || t >= c->t_max) return PAAC_ERR_ARG;
  if (t + 1 != c->host_t) return PAAC_ERR_STATE;
  const size_t row = (size_t)t * c->n_e;
  if (cudaMemcpyAsync(c->rewards + row, rewards, c->n_e, cudaMemcpyHostToDevice, c->st) != cudaSuccess ||
      cudaMemcpyAsync(c->terminals + row, terminals, c->n_e, cudaMemcpyHostToDevice, c->st) != cudaSuccess) {
    cudaGetLastError(); return PAAC_ERR_CUDA;
  }
  return PAAC_OK;
}

// ---- debug access -----------------------------------------------------------------------------------
static void* debug_ptr(const paac_ctx* c, int which, size_t* bytes) {
  const size_t n_e = c->n_e, T = c->t_max, B = c->B, A = c->A, P = c->nd.P;
  switch (which) {
    case PAAC_DBG_FRAMES: *bytes = T * n_e * FRAME_BYTES; return c->frames[c->cur];
    case PAAC_DBG_NEXT_FRAMES: *bytes = n_e * FRAME_BYTES; return c->frames[c->cur ^ 1];
    case PAAC_DBG_ACTIONS: *bytes = B * 4; return c->actions;
    case PAAC_DBG_REWARDS: *bytes = B; return c->rewards;
    case PAAC_DBG_TERMINALS: *bytes = B; return c->terminals;
    case PAAC_DBG_VALUES: *bytes = (T + 1) * n_e * 4; return c->values;
    case PAAC_DBG_LOGITS: *bytes = B * A * 4; return c->logits;
    case PAAC_DBG_UNIFORMS: *bytes = B * 4; return c->uniforms;
    case PAAC_DBG_COUNTERS: *bytes = 3 * n_e * 4; return c->counters;
    case PAAC_DBG_RETURNS: *bytes = B * 4; return c->R;
    case PAAC_DBG_ADVANTAGES: *bytes = B * 4; return c->adv;
    case PAAC_DBG_DLOGITS: *bytes = B * A * 4; return c->dz;
    case PAAC_DBG_DVALUES: *bytes = B * 4; return c->dV;
    case PAAC_DBG_GRAD: *bytes = P * 4; return c->grad;
    case PAAC_DBG_RMS: *bytes = P * 4; return c->rms;
    case PAAC_DBG_SAMPLED: *bytes = B * 4; return c->sampled;
    case PAAC_DBG_ERROR_WORD: *bytes = 4; return &c->stats->error_word;
    default: break;
  }
  if (which >= PAAC_DBG_ACT0 && which <= PAAC_DBG_ACT0 + c->nd.n_conv) {
    const int l = which - PAAC_DBG_ACT0;
    *bytes = B * c->nd.layer[l].out_size * c->elt; return c->act[l];
  }
  if (which >= PAAC_DBG_GACT0 && which <= PAAC_DBG_GACT0 + c->nd.n_conv) {
    const int l = which - PAAC_DBG_GACT0;
    *bytes = B * c->nd.layer[l].out_size * c->elt; return c->gact[l];
  }
  *bytes = 0;
  return nullptr;
}

size_t paac_debug_bytes(const paac_ctx* c, int which) {
  if (!c) return 0;
  size_t b = 0;
  debug_ptr(c, which, &b);
  return b;
}

int paac_debug_read(paac_ctx* c, int which, void* dst, size_t bytes) {
  if (!c || !dst) return PAAC_ERR_ARG;
  size_t b = 0;
  void* p = debug_ptr(c, which, &b);
  if (!p || b != bytes) return PAAC_ERR_ARG;
  if (cudaMemcpyAsync(dst, p, b, cudaMemcpyDeviceToHost, c->st) != cudaSuccess ||
      cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  if (which == PAAC_DBG_GACT0 && c->prec == PAAC_BF16 && c->gact0_scale != 1.f) {
    // stored times a power of two for the first layer's weight-gradient kernel: hand out the gradient itself
    uint16_t* h = (uint16_t*)dst;
    const float inv = 1.f / c->gact0_scale;
    for (size_t i = 0; i < b / 2; ++i) {
      uint32_t u = (uint32_t)h[i] << 16;
      float f;
      memcpy(&f, &u, 4);
      f *= inv;                                  // exact: a shift of the exponent (denormal results lose low bits)
      memcpy(&u, &f, 4);
      h[i] = (uint16_t)(u >> 16);
    }
  }
  return device_error(c);
}

int paac_debug_write(paac_ctx* c, int which, const void* src, size_t bytes) {
  if (c) c->lc.serialize_next = true;
  if (!c || !src) return PAAC_ERR_ARG;
  size_t b = 0;
  void* p = debug_ptr(c, which, &b);
  if (!p || b != bytes) return PAAC_ERR_ARG;
  if (cudaMemcpyAsync(p, src, b, cudaMemcpyHostToDevice, c->st) != cudaSuccess ||
      cudaStreamSynchronize(c->st) != cudaSuccess) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  return PAAC_OK;
}

}  // extern "C"
