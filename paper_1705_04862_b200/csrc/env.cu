// Parameter initialisation and the synthetic hashed environment.
#include "kernels.h"

namespace paac {

// Xavier-uniform: element i of weight tensor `layer` is (2u-1)*bound with u the 24-bit
// Philox uniform of counter (i, layer, 0, RNG_STREAM_INIT).  2u-1 is exact in float, so the
// single rounding of the product is the same on any IEEE machine.
__global__ void xavier_kernel(float* w, uint32_t count, float bound, uint32_t layer, uint64_t seed) {
  pdl_entry();
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x) {
    const float u = philox_uniform(i, layer, 0u, RNG_STREAM_INIT, seed);
    w[i] = __fmul_rn(__fsub_rn(__fmul_rn(2.0f, u), 1.0f), bound);
  }
}

static void xavier(LaunchCtx& lc, float* w, size_t count, double fan_in, double fan_out,
                   uint32_t layer, uint64_t seed) {
  const float bound = (float)sqrt(6.0 / (fan_in + fan_out));
  int blocks = (int)((count + 255) / 256);
  if (blocks > 1184) blocks = 1184;
  KernelScope scope(lc, KID_INIT);
  launch_kernel(lc, xavier_kernel, blocks, 256, 0, w, (uint32_t)count, bound, layer, seed);
}

void launch_init_params(LaunchCtx& lc, const NetDims& nd, uint64_t seed, float* theta) {
  cudaMemsetAsync(theta, 0, nd.P * sizeof(float), lc.st);
  uint32_t id = 0;
  for (int l = 0; l < nd.n_conv; ++l, ++id) {
    const LayerDims& d = nd.layer[l];
    const double kk = (double)d.K * d.K;
    xavier(lc, theta + d.w_off, (size_t)d.CO * d.K * d.K * d.C, kk * d.C, kk * d.CO, id, seed);
  }
  const LayerDims& f = nd.layer[nd.n_conv];
  const size_t in = (size_t)f.H * f.W * f.C;
  xavier(lc, theta + f.w_off, in * nd.F, (double)in, (double)nd.F, id++, seed);
  xavier(lc, theta + nd.pi_w, (size_t)nd.A * nd.F, (double)nd.F, (double)nd.A, id++, seed);
  xavier(lc, theta + nd.v_w, (size_t)nd.F, (double)nd.F, 1.0, id++, seed);
}

__global__ void cast_bf16_kernel(const float* src, bf16* dst, size_t n) {
  pdl_entry();
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}
void launch_cast_bf16(LaunchCtx& lc, const float* src, bf16* dst, size_t n) {
  int blocks = (int)((n + 255) / 256);
  if (blocks > 1184) blocks = 1184;
  KernelScope scope(lc, KID_CAST);
  launch_kernel(lc, cast_bf16_kernel, blocks, 256, 0, src, dst, n);
}

// One block per environment.  The block's first thread decides reward and terminal flag of
// the transition (seed, env, step, action) and keeps the episode counters; all threads then
// write the 84x84x4 frame of the state reached, one hashed 32-bit word per pixel (its bytes,
// little endian, are the four channels), as 16-byte stores.
constexpr int ENV_THREADS = 256;
constexpr int FRAME_WORDS = FRAME_H * FRAME_W;   // 7056, a multiple of 4

// With SAMPLE the block's first warp also takes the action first: it finishes the heads of its environment from the
// two partial dot products hp[half][e][k] the fully connected kernel left (k < A policy rows, k = A value row;
// rows 32 floats apart), softmax, inverse-CDF draw from the Philox uniform of (env, step) exactly as the stand-alone
// sampling kernel does, and writes logits, value, uniform and action; the transition then uses that action.
template <bool SAMPLE>
__global__ void __launch_bounds__(ENV_THREADS)
env_step_kernel(uint64_t seed, int n_e, const uint64_t* __restrict__ step_base, uint32_t t,
                const int32_t* actions, uint32_t term_denom,
                uint8_t* __restrict__ next_frames, int8_t* __restrict__ rewards, uint8_t* __restrict__ terminals,
                int32_t* __restrict__ counters, HeadsTail ht, int pattern_actions) {
  // pattern_actions > 0: the learnable environment.  The state at step k of environment e has the goal
  // hash(e, k, 'GOAL') mod A; its frame is the hashed frame with every byte reduced to its low six bits (a dim
  // texture) and rows [band goal, band (goal + 1)), band = 84 / A, set to 255; an action pays 1 if it is the current
  // state's goal and 0 otherwise.
  // Two roles run side by side until the action is known: the first warp takes it (SAMPLE), and the first thread of
  // the second warp prepares everything of the transition that does not depend on it -- the hash chains of this step
  // and the next up to the point where the action enters, and the environment's counters, whose loads would otherwise
  // be waited for after the draw.  One hash step, the reward / terminal bits and the frame's base remain.
  __shared__ uint32_t s_base, s_band_lo, s_band_hi;
  __shared__ int32_t s_action;
  const uint32_t e = blockIdx.x;
  const bool stepping = SAMPLE || actions != nullptr;          // else: the start frames (step 0, tag 0)
  uint32_t pre_step = 0u, pre_next = 0u, step = 0u;
  int32_t len = 0, ret = 0, episodes = 0;
  if (SAMPLE && threadIdx.x < 32) {
    const int lane = threadIdx.x, A = ht.A;
    const float bias = lane < A ? __ldg(ht.bpi + lane) : (lane == A ? __ldg(ht.bv) : 0.f);   // older than the previous kernel
    pdl_entry();
    float sum = -INFINITY;
    if (lane <= A) sum = (ht.hp[(size_t)e * 32 + lane] + ht.hp[((size_t)n_e + e) * 32 + lane]) + bias;
    const float z = lane < A ? sum : -INFINITY;
    const int32_t a = warp_finish_heads(ht.mode, z, __shfl_sync(0xffffffffu, sum, A), lane, A, (size_t)e, ht.logits, ht.values, true,
                                        seed, *step_base + t, ht.forced, ht.actions, ht.sampled, ht.uniforms);
    if (lane == 0) s_action = a;
  } else {
    pdl_entry();
    if (threadIdx.x == 32) {
      if (stepping) {
        step = (uint32_t)(*step_base) + t;                      // global step index of this transition
        pre_step = env_hash_prefix(seed, e, step);
        pre_next = env_hash_prefix(seed, e, step + 1u);
        len = counters[e]; ret = counters[n_e + e]; episodes = counters[2 * n_e + e];
        if (!SAMPLE) s_action = actions[e];
      } else {
        pre_next = env_hash_prefix(seed, e, 0u);
      }
    }
  }
  __syncthreads();
  bool term = false;
  int r = 0;
  if (threadIdx.x == 32) {
    uint32_t tag = 0u;
    if (stepping) {
      const int32_t a = s_action;
      const uint32_t base = hash_mix(pre_step ^ ((uint32_t)a + 1u));
      const uint32_t hr = hash_mix(base ^ HASH_TAG_REWARD) & 15u;
      r = hr == 0u ? 1 : (hr == 1u ? -1 : 0);
      if (pattern_actions > 0)
        r = (uint32_t)a == hash_mix(hash_mix(pre_step) ^ HASH_TAG_GOAL) % (uint32_t)pattern_actions ? 1 : 0;
      const uint32_t hterm = hash_mix(base ^ HASH_TAG_TERMINAL);
      term = (uint32_t)(((uint64_t)hterm * term_denom) >> 32) == 0u;
      tag = term ? 0u : (uint32_t)a + 1u;
    }
    s_base = hash_mix(pre_next ^ tag);
    s_band_lo = s_band_hi = 0u;
    if (pattern_actions > 0) {
      const uint32_t goal = hash_mix(hash_mix(pre_next) ^ HASH_TAG_GOAL) % (uint32_t)pattern_actions;
      const uint32_t band = (uint32_t)(FRAME_H / pattern_actions);
      s_band_lo = band * goal * FRAME_W;                  // in pixel words; a row is 84 words, so four words never straddle it
      s_band_hi = s_band_lo + band * FRAME_W;
    }
  }
  __syncthreads();
  if (threadIdx.x == 32 && stepping) {
    rewards[e] = (int8_t)r;
    terminals[e] = term ? 1 : 0;
    len += 1; ret += r;
    if (term) { counters[2 * n_e + e] = episodes + 1; len = 0; ret = 0; }
    counters[e] = len; counters[n_e + e] = ret;
  }
  const uint32_t base = s_base, band_lo = s_band_lo, band_hi = s_band_hi;
  const uint32_t keep = pattern_actions > 0 ? 0x3F3F3F3Fu : 0xFFFFFFFFu;
  uint4* out = reinterpret_cast<uint4*>(next_frames + (size_t)e * FRAME_BYTES);
  for (int q = threadIdx.x; q < FRAME_WORDS / 4; q += ENV_THREADS) {
    const uint32_t p = (uint32_t)q * 4u + 1u;
    uint4 v;
    v.x = hash_mix(base + HASH_K0 * p);
    v.y = hash_mix(base + HASH_K0 * (p + 1u));
    v.z = hash_mix(base + HASH_K0 * (p + 2u));
    v.w = hash_mix(base + HASH_K0 * (p + 3u));
    v.x &= keep; v.y &= keep; v.z &= keep; v.w &= keep;
    if ((uint32_t)q * 4u >= band_lo && (uint32_t)q * 4u < band_hi) v = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
    out[q] = v;
  }
}

void launch_env_step(LaunchCtx& lc, uint64_t seed, int n_e, const uint64_t* step_base, uint32_t t,
                     const int32_t* actions, uint32_t term_denom, uint8_t* next_frames, int8_t* rewards,
                     uint8_t* terminals, int32_t* counters, int pattern_actions) {
  KernelScope scope(lc, KID_ENV_STEP);
  launch_kernel(lc, env_step_kernel<false>, n_e, ENV_THREADS, 0, seed, n_e, step_base, t, actions, term_denom, next_frames, rewards,
                                                  terminals, counters, HeadsTail{}, pattern_actions);
}

void launch_env_step_sampling(LaunchCtx& lc, uint64_t seed, int n_e, const uint64_t* step_base, uint32_t t, uint32_t term_denom,
                              uint8_t* next_frames, int8_t* rewards, uint8_t* terminals, int32_t* counters,
                              const HeadsTail& ht, int pattern_actions) {
  KernelScope scope(lc, KID_ENV_STEP);
  launch_kernel(lc, env_step_kernel<true>, n_e, ENV_THREADS, 0, seed, n_e, step_base, t, (const int32_t*)nullptr, term_denom,
                next_frames, rewards, terminals, counters, ht, pattern_actions);
}

// the environments' global step index lives on the device, so that a recorded sequence of launches can be
// replayed for the next iteration without new arguments
__global__ void advance_step_kernel(uint64_t* step_base, uint32_t by) {
  pdl_entry(); *step_base += by; }
void launch_advance_step(LaunchCtx& lc, uint64_t* step_base, uint32_t by) {
  KernelScope scope(lc, KID_ENV_STEP);
  launch_kernel(lc, advance_step_kernel, 1, 1, 0, step_base, by);
}

}  // namespace paac
