// Shared device helpers and the context layout of the PAAC library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/paac.h"

namespace paac {

typedef __nv_bfloat16 bf16;

constexpr int FRAME_H = 84, FRAME_W = 84, FRAME_C = 4;
constexpr int FRAME_BYTES = FRAME_H * FRAME_W * FRAME_C;   // 28,224
constexpr int MAX_LAYERS = 4;                              // conv layers + fc

// ---- storage type helpers ---------------------------------------------------
__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f(uint8_t x) { return (float)x; }
template <class T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// ---- Philox4x32-10 (Salmon et al., SC'11) -------------------------------------
__host__ __device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}
constexpr uint32_t RNG_STREAM_INIT = 1u, RNG_STREAM_ACTION = 2u;

// 24-bit uniform in [0,1) from the first output word
__host__ __device__ __forceinline__ float philox_uniform(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t stream,
                                                         uint64_t seed) {
  uint32_t o[4];
  philox4x32_10(c0, c1, c2, stream, (uint32_t)seed, (uint32_t)(seed >> 32), o);
  return (float)(o[0] >> 8) * (1.0f / 16777216.0f);
}

// ---- what the heads mean -----------------------------------------------------------
// PAAC_ALGO_A2C: softmax policy over the A outputs of the first head plus a state value (Algorithm 1).
// PAAC_ALGO_NSTEP_Q: the A outputs are Q(s, a) (Section 2.2 on the framework of Section 3): acting is
// epsilon-greedy, the value stored for a step is Q(s_t, a_t), the bootstrap value is max_a Q.
struct HeadMode { int algo; float eps; };

#ifdef __CUDACC__
// Everything that follows the heads' dot products, done by one full warp for state e.  Lane k < A holds head output
// z_k (the other lanes -inf); v is the value head's output, the same in all lanes.  Writes the A outputs and the
// stored value; with `sample` it also draws the action from the Philox uniform of (e, step) -- inverse CDF of the
// softmax in index order on a float running sum, or epsilon-greedy on the Q-values with the one uniform deciding
// both whether to explore (u < eps) and where (floor((u / eps) A)) --, honours a forced action, and returns the
// action taken (-1 without sampling).
__device__ __forceinline__ int warp_finish_heads(const HeadMode hm, float z, float v, int lane, int A, size_t e,
                                                 float* __restrict__ logits, float* __restrict__ values, bool sample,
                                                 uint64_t seed, uint64_t step, const int32_t* __restrict__ forced,
                                                 int32_t* __restrict__ actions, int32_t* __restrict__ sampled,
                                                 float* __restrict__ uniforms) {
  if (lane < A) logits[e * A + lane] = z;
  float m = z;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (hm.algo == PAAC_ALGO_NSTEP_Q) {
    const uint32_t at_max = __ballot_sync(0xffffffffu, lane < A && z == m);
    const int greedy = at_max ? __ffs(at_max) - 1 : 0;                  // smallest index among equal maxima
    if (!sample) { if (lane == 0) values[e] = m; return -1; }
    const float u = philox_uniform((uint32_t)e, (uint32_t)step, (uint32_t)(step >> 32), RNG_STREAM_ACTION, seed);
    int a = greedy;
    if (u < hm.eps) {
      const int k = (int)__fmul_rn(__fdiv_rn(u, hm.eps), (float)A);     // two single roundings: the same on any machine
      a = k < A - 1 ? k : A - 1;
    }
    const int drawn = a;
    if (forced != nullptr && forced[e] >= 0) a = forced[e];
    const float qa = __shfl_sync(0xffffffffu, z, a);
    if (lane == 0) { sampled[e] = drawn; actions[e] = a; uniforms[e] = u; values[e] = qa; }
    return a;
  }
  if (lane == 0) values[e] = v;
  if (!sample) return -1;
  float ex = lane < A ? expf(z - m) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ex += __shfl_xor_sync(0xffffffffu, ex, o);
  const float lse = m + logf(ex);
  const float p = lane < A ? expf(z - lse) : 0.f;
  const float u = philox_uniform((uint32_t)e, (uint32_t)step, (uint32_t)(step >> 32), RNG_STREAM_ACTION, seed);
  float c = 0.f;
  int a = A - 1;
  bool found = false;
  for (int k = 0; k < A; ++k) {
    c += __shfl_sync(0xffffffffu, p, k);
    if (!found && u < c) { a = k; found = true; }
  }
  const int drawn = a;
  if (forced != nullptr && forced[e] >= 0) a = forced[e];
  if (lane == 0) { sampled[e] = drawn; actions[e] = a; uniforms[e] = u; }
  return a;
}
#endif

// ---- environment hash -----------------------------------------------------------
constexpr uint32_t HASH_K0 = 0x9E3779B9u, HASH_K1 = 0xBB67AE85u, HASH_K2 = 0x6A09E667u;
constexpr uint32_t HASH_TAG_REWARD = 0x52455744u, HASH_TAG_TERMINAL = 0x5445524Du, HASH_TAG_GOAL = 0x474F414Cu;

__host__ __device__ __forceinline__ uint32_t hash_mix(uint32_t x) {
  x ^= x >> 16; x *= HASH_K0; x ^= x >> 15; x *= HASH_K1; x ^= x >> 16;
  return x;
}
// the part of the chain that does not depend on the tag (an action, or 0), and the step that takes the tag in
__host__ __device__ __forceinline__ uint32_t env_hash_prefix(uint64_t seed, uint32_t env, uint32_t step) {
  uint32_t h = hash_mix((uint32_t)seed ^ HASH_K2);
  h = hash_mix(h ^ (uint32_t)(seed >> 32));
  h = hash_mix(h ^ env);
  return hash_mix(h ^ step);
}
__host__ __device__ __forceinline__ uint32_t env_hash_base(uint64_t seed, uint32_t env, uint32_t step, uint32_t tag) {
  return hash_mix(env_hash_prefix(seed, env, step) ^ tag);
}

// ---- network geometry (compile time) ----------------------------------------------
template <int H_, int W_, int C_, int K_, int S_, int CO_>
struct ConvGeom {
  static constexpr int H = H_, W = W_, C = C_, K = K_, S = S_, CO = CO_;
  static constexpr int OH = (H - K) / S + 1, OW = (W - K) / S + 1;
  static constexpr int KK = K * K * C;          // reduction length of the forward contraction
  static constexpr int IN_SIZE = H * W * C, OUT_SIZE = OH * OW * CO;
};
typedef ConvGeom<84, 84, 4, 8, 4, 16> NipsConv1;
typedef ConvGeom<20, 20, 16, 4, 2, 32> NipsConv2;
typedef ConvGeom<84, 84, 4, 8, 4, 32> NatConv1;
typedef ConvGeom<20, 20, 32, 4, 2, 64> NatConv2;
typedef ConvGeom<9, 9, 64, 3, 1, 64> NatConv3;

// run-time copy of the same numbers for host-side sizing
struct LayerDims {
  int H, W, C, K, S, CO, OH, OW;   // fc: K = S = 0, H*W*C = inputs, CO = outputs, OH = OW = 1
  size_t w_off, b_off;             // offsets into the canonical parameter vector
  size_t out_size;                 // elements per state of the stored activation
};

struct NetDims {
  int n_conv;
  LayerDims layer[MAX_LAYERS];     // conv layers then fc
  int F, A;
  size_t pi_w, pi_b, v_w, v_b, P;
};

inline NetDims make_net(int arch, int A) {
  NetDims n{};
  const int nips[2][3] = {{16, 8, 4}, {32, 4, 2}};
  const int nat[3][3] = {{32, 8, 4}, {64, 4, 2}, {64, 3, 1}};
  n.n_conv = arch == PAAC_ARCH_NIPS ? 2 : 3;
  n.F = arch == PAAC_ARCH_NIPS ? 256 : 512;
  n.A = A;
  int H = FRAME_H, W = FRAME_W, C = FRAME_C;
  size_t off = 0;
  for (int l = 0; l < n.n_conv; ++l) {
    const int* s = arch == PAAC_ARCH_NIPS ? nips[l] : nat[l];
    LayerDims& d = n.layer[l];
    d.H = H; d.W = W; d.C = C; d.CO = s[0]; d.K = s[1]; d.S = s[2];
    d.OH = (H - d.K) / d.S + 1; d.OW = (W - d.K) / d.S + 1;
    d.w_off = off; off += (size_t)d.CO * d.K * d.K * C;
    d.b_off = off; off += d.CO;
    d.out_size = (size_t)d.OH * d.OW * d.CO;
    H = d.OH; W = d.OW; C = d.CO;
  }
  LayerDims& f = n.layer[n.n_conv];
  f.H = H; f.W = W; f.C = C; f.K = 0; f.S = 0; f.CO = n.F; f.OH = f.OW = 1;
  f.w_off = off; off += (size_t)H * W * C * n.F;
  f.b_off = off; off += n.F;
  f.out_size = n.F;
  n.pi_w = off; off += (size_t)A * n.F;
  n.pi_b = off; off += A;
  n.v_w = off; off += n.F;
  n.v_b = off; off += 1;
  n.P = off;
  return n;
}

// ---- launch bookkeeping ----------------------------------------------------------------------
// Kernel families, for the launch counter and the optional per-kernel CUDA-event timing.
enum KernelId {
  KID_INIT = 0, KID_ENV_STEP, KID_CONV1_FWD, KID_CONV2_FWD, KID_CONV3_FWD, KID_FC_FWD, KID_HEADS_FWD,
  KID_RETURNS, KID_HEAD_GRAD, KID_HEADS_BWD, KID_FC_WGRAD, KID_FC_DGRAD, KID_CONV3_WGRAD, KID_CONV3_DGRAD,
  KID_CONV2_WGRAD, KID_CONV2_DGRAD, KID_CONV1_WGRAD, KID_WGRAD_REDUCE, KID_SUMSQ, KID_CLIP_RMSPROP, KID_CAST, KID_BIAS_GRAD,
  KID_COUNT
};
inline const char* kernel_name(int id) {
  static const char* names[KID_COUNT] = {
      "init_params", "env_step", "conv1_fwd", "conv2_fwd", "conv3_fwd", "fc_fwd", "heads_fwd_sample", "returns",
      "head_grad", "heads_bwd", "fc_wgrad", "fc_dgrad", "conv3_wgrad", "conv3_dgrad", "conv2_wgrad", "conv2_dgrad",
      "conv1_wgrad", "wgrad_reduce", "grad_sumsq", "clip_rmsprop", "cast_bf16", "bias_grad"};
  return id >= 0 && id < KID_COUNT ? names[id] : "?";
}

struct LaunchCtx {
  cudaStream_t st = nullptr;
  uint64_t count = 0;                 // kernels launched so far
  bool profiling = false;             // record a CUDA event pair around every launch
  bool serialize_next = true;         // the next launch takes plain stream order (no overlap with its predecessor)
  bool host_failure = false;          // a launch could not be prepared on the host (sticky; reported as PAAC_ERR_CUDA)
  bool fp32_tensor_cores = false;     // the float path's contractions go through the three-pass tensor-core kernel
  uint32_t* error_word = nullptr;     // device word the bounded waits of that kernel report to
  static constexpr int MAX_PENDING = 512;
  cudaEvent_t ev[MAX_PENDING][2];
  int ev_kid[MAX_PENDING];
  int n_events = 0, n_created = 0;
  double ms[KID_COUNT] = {};          // accumulated device time per family
  uint64_t calls[KID_COUNT] = {};

  // fold the pending event pairs into ms[]; the stream must be idle
  void collect() {
    for (int i = 0; i < n_events; ++i) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, ev[i][0], ev[i][1]) == cudaSuccess) { ms[ev_kid[i]] += t; calls[ev_kid[i]] += 1; }
    }
    n_events = 0;
  }
  void release() {
    for (int i = 0; i < n_created; ++i) { cudaEventDestroy(ev[i][0]); cudaEventDestroy(ev[i][1]); }
    n_created = n_events = 0;
  }
};

// Brackets one kernel launch: counts it and, when profiling, times it with an event pair.
struct KernelScope {
  LaunchCtx& lc; int slot;
  KernelScope(LaunchCtx& l, int kid) : lc(l), slot(-1) {
    ++lc.count;
    if (!lc.profiling) return;
    if (lc.n_events == LaunchCtx::MAX_PENDING) { cudaStreamSynchronize(lc.st); lc.collect(); }
    slot = lc.n_events++;
    if (slot >= lc.n_created) {
      cudaEventCreate(&lc.ev[slot][0]); cudaEventCreate(&lc.ev[slot][1]);
      lc.n_created = slot + 1;
    }
    lc.ev_kid[slot] = kid;
    cudaEventRecord(lc.ev[slot][0], lc.st);
  }
  ~KernelScope() { if (slot >= 0) cudaEventRecord(lc.ev[slot][1], lc.st); }
};

// ---- programmatic dependent launch ----------------------------------------------------------------------------
// The tensor-core kernels are launched with programmatic stream serialization: their CTAs may be scheduled while
// the kernel before them in the stream is still draining, which hides the launch latency and lets a CTA set itself
// up on an SM as soon as the previous kernel's CTA there has left.  The contract every kernel keeps:
//   pdl_wait() comes before the first access to anything the PREVIOUS kernel in the stream writes or reads-then-
//   overwrites; it returns once that kernel has completed and its writes are visible.  Only work on data that no
//   neighbouring kernel touches (barrier set-up, tensor-memory allocation, weight tiles written several kernels
//   earlier) may precede it;
//   pdl_launch_dependents() comes after pdl_wait(), so at most two kernels ever overlap and everything older than
//   the previous kernel is complete when a kernel starts.
// Launched without the attribute (pdl_enabled() == false) both calls do nothing and stream order is the usual one.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_entry() { pdl_wait(); pdl_launch_dependents(); }

inline bool& pdl_enabled() { static bool on = true; return on; }

// The first launch after serialize_next was set (every API call sets it before it enqueues anything) gets plain
// stream order, so that no kernel's set-up ever overlaps the last kernel of an earlier call (parameter updates
// and weight re-layouts close an update).
template <bool OVERLAP, class... KArgs, class... Args>
inline cudaError_t launch_kernel_impl(LaunchCtx& lc, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = lc.st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = (OVERLAP && pdl_enabled() && !lc.serialize_next) ? 1 : 0;
  lc.serialize_next = false;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
// plain stream order: for kernels that need their predecessor's data from the first instruction on
template <class... KArgs, class... Args>
inline cudaError_t launch_kernel(LaunchCtx& lc, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  return launch_kernel_impl<false>(lc, kern, grid, block, smem, args...);
}
// may start while its predecessor drains: for kernels whose set-up before pdl_wait() is worth overlapping
template <class... KArgs, class... Args>
inline cudaError_t launch_kernel_overlapped(LaunchCtx& lc, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  return launch_kernel_impl<true>(lc, kern, grid, block, smem, args...);
}

// bits of DeviceStats::error_word: 1, 2, 4 = a bounded wait gave up (which kind: see tc_common.cuh);
// 8 = a first-layer weight does not fit the fp16 image the forward kernel multiplies with
constexpr uint32_t DEV_ERR_WAIT_MASK = 7u, DEV_ERR_RANGE = 8u;
inline int status_of_error_word(uint32_t w) {
  return (w & DEV_ERR_WAIT_MASK) ? PAAC_ERR_TIMEOUT : ((w & DEV_ERR_RANGE) ? PAAC_ERR_RANGE : PAAC_OK);
}

// device-side statistics block written by the update kernels
struct DeviceStats {
  float policy_loss, value_loss, entropy, grad_norm, clip_scale;
  int32_t status;
  uint32_t error_word;   // bit set by a kernel whose bounded wait or bounds check gave up
  uint32_t arrivals;     // blocks of the head-gradient kernel that have finished (back to zero when it ends)
};

}  // namespace paac
