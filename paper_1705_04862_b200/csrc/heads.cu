// Policy / value heads with softmax, entropy and Philox inverse-CDF sampling; the reverse
// scan for n-step returns; the loss gradient at the heads.
#include "kernels.h"

namespace paac {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// EPL consecutive elements of a row as floats (EPL = 8 or 16; 16-byte loads)
template <int EPL> __device__ __forceinline__ void load_row_slice(const float* p, float (&v)[EPL]) {
  const float4* q = reinterpret_cast<const float4*>(p);
#pragma unroll
  for (int i = 0; i < EPL / 4; ++i) { const float4 t = __ldg(q + i); v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w; }
}
template <int EPL> __device__ __forceinline__ void load_row_slice(const bf16* p, float (&v)[EPL]) {
  const uint4* q = reinterpret_cast<const uint4*>(p);
#pragma unroll
  for (int i = 0; i < EPL / 8; ++i) {
    const uint4 t = __ldg(q + i);
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { v[8 * i + 2 * j] = __uint_as_float(w[j] << 16); v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u); }
  }
}

// One warp per state; lane l holds elements [l*EPL, (l+1)*EPL) of the fc activation (F = 32*EPL) and of
// each head row.  Lane k ends up holding logit k (A <= 32).  If `actions` is given, the warp also draws
// a_t: u from Philox counter (env, step_lo, step_hi, ACTION stream), then the smallest k with
// u < p_0 + ... + p_k, the running sum taken serially in float in index order.
template <class T, class TW, int EPL>
__global__ void __launch_bounds__(128)
heads_kernel(const T* __restrict__ h, const TW* __restrict__ wpi, const float* __restrict__ bpi,
             const TW* __restrict__ wv, const float* __restrict__ bv, int n, int A,
             float* __restrict__ logits, float* __restrict__ values, uint64_t seed, const uint64_t* __restrict__ step_base, uint32_t t,
             const int32_t* __restrict__ forced, int32_t* __restrict__ actions, int32_t* __restrict__ sampled,
             float* __restrict__ uniforms, HeadMode mode) {
  pdl_entry();
  constexpr int F = 32 * EPL;
  const int lane = threadIdx.x & 31;
  const int e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (e >= n) return;
  float x[EPL], w[EPL];
  load_row_slice<EPL>(h + (size_t)e * F + lane * EPL, x);
  float z = -INFINITY;
  for (int k = 0; k < A; ++k) {
    load_row_slice<EPL>(wpi + (size_t)k * F + lane * EPL, w);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < EPL; ++i) acc = fmaf(w[i], x[i], acc);
    acc = warp_sum(acc) + bpi[k];
    if (lane == k) z = acc;
  }
  // the value row follows the policy biases in the parameter vector, so it is not 16-byte aligned
  float v = 0.f;
#pragma unroll
  for (int i = 0; i < EPL; ++i) v = fmaf(to_f(wv[lane * EPL + i]), x[i], v);
  v = warp_sum(v) + bv[0];
  warp_finish_heads(mode, z, v, lane, A, (size_t)e, logits, values, actions != nullptr, seed,
                    actions != nullptr ? *step_base + t : 0ull, forced, actions, sampled, uniforms);
}

// The same, fused with the end of the fully connected layer of the tensor-core path: the warp first finishes
// its state's 512 hidden units from the split-k partial sums, h = bf16(relu(sum_s part[s][e][:] + bias)), the
// splits added in order, stores them for the backward pass and goes on with the rounded values.  The A dot
// products are reduced together: every lane keeps one partial sum per action, and a butterfly that halves the
// number of live values at each step leaves lane k with logit k after 31 shuffles instead of 5 per action; the
// additions pair up exactly as in warp_sum, so the logits are bit-identical to the unfused kernel's.
// The head weights (A + 1 rows of 512) are brought into shared memory once per block, before the wait on the
// previous kernel: they are older than that kernel.  Row k is stored as two halves, [lane][first 8 of the lane's
// 16 elements] then [lane][last 8], so that a warp's 16-byte reads are contiguous.
constexpr int HF_WARPS = 8;
__global__ void __launch_bounds__(HF_WARPS * 32)
heads_fused_kernel(const float* __restrict__ part, int splits, const float* __restrict__ fc_bias, bf16* __restrict__ h_out,
                   const bf16* __restrict__ wpi, const float* __restrict__ bpi, const bf16* __restrict__ wv,
                   const float* __restrict__ bv, int n, int A, float* __restrict__ logits, float* __restrict__ values,
                   uint64_t seed, const uint64_t* __restrict__ step_base, uint32_t t, const int32_t* __restrict__ forced,
                   int32_t* __restrict__ actions, int32_t* __restrict__ sampled, float* __restrict__ uniforms, HeadMode mode) {
  constexpr int EPL = 16, F = 32 * EPL;
  __shared__ uint4 wsh[33 * 64];                     // row k: 64 chunks of 8 bf16; row A = value head
  const int lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < (A + 1) * 64; i += HF_WARPS * 32) {
    const int k = i >> 6, c = i & 63, l = c >> 1, half = c & 1;          // chunk c of the row = lane l, half
    uint4 v;
    if (k < A) v = __ldg(reinterpret_cast<const uint4*>(wpi + (size_t)k * F) + c);
    else {                                            // the value row is not 16-byte aligned
      uint32_t w4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        w4[j] = (uint32_t)__bfloat16_as_ushort(wv[c * 8 + 2 * j]) | ((uint32_t)__bfloat16_as_ushort(wv[c * 8 + 2 * j + 1]) << 16);
      v = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    }
    wsh[k * 64 + half * 32 + l] = v;
  }
  __syncthreads();
  pdl_entry();          // the head weights above were written several kernels ago
  const int e = blockIdx.x * HF_WARPS + (threadIdx.x >> 5);
  if (e >= n) return;
  float x[EPL];
  {
    float v[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) v[i] = 0.f;
    const float* p0 = part + (size_t)e * F + lane * EPL;
#pragma unroll 7
    for (int s = 0; s < splits; ++s) {
      const float4* q = reinterpret_cast<const float4*>(p0 + (size_t)s * n * F);
#pragma unroll
      for (int i = 0; i < EPL / 4; ++i) {
        const float4 a = __ldg(q + i);
        v[4 * i] += a.x; v[4 * i + 1] += a.y; v[4 * i + 2] += a.z; v[4 * i + 3] += a.w;
      }
    }
    uint32_t o[EPL / 2];
#pragma unroll
    for (int i = 0; i < EPL / 2; ++i) {
      const bf16 lo = __float2bfloat16_rn(fmaxf(v[2 * i] + __ldg(fc_bias + lane * EPL + 2 * i), 0.f));
      const bf16 hi = __float2bfloat16_rn(fmaxf(v[2 * i + 1] + __ldg(fc_bias + lane * EPL + 2 * i + 1), 0.f));
      x[2 * i] = __bfloat162float(lo); x[2 * i + 1] = __bfloat162float(hi);
      o[i] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
    }
    uint4* dst = reinterpret_cast<uint4*>(h_out + (size_t)e * F + lane * EPL);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
  }
  float pr[32];
#pragma unroll
  for (int k = 0; k < 32; ++k) {
    pr[k] = 0.f;
    if (k < A) {
      const uint4 lo = wsh[k * 64 + lane], hi = wsh[k * 64 + 32 + lane];
      const uint32_t w8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        acc = fmaf(__uint_as_float(w8[i] << 16), x[2 * i], acc);
        acc = fmaf(__uint_as_float(w8[i] & 0xFFFF0000u), x[2 * i + 1], acc);
      }
      pr[k] = acc;
    }
  }
  // reduce-scatter: at the step with offset o a lane keeps the half of its values whose index has bit o equal to
  // its own lane bit and adds the partner's copy of them
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float send = up ? pr[i] : pr[i + o];
      const float keep = up ? pr[i + o] : pr[i];
      pr[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  const float z = lane < A ? pr[0] + bpi[lane < A ? lane : 0] : -INFINITY;
  float v = 0.f;
  {
    const uint4 lo = wsh[A * 64 + lane], hi = wsh[A * 64 + 32 + lane];
    const uint32_t w8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v = fmaf(__uint_as_float(w8[i] << 16), x[2 * i], v);
      v = fmaf(__uint_as_float(w8[i] & 0xFFFF0000u), x[2 * i + 1], v);
    }
  }
  v = warp_sum(v) + bv[0];
  warp_finish_heads(mode, z, v, lane, A, (size_t)e, logits, values, actions != nullptr, seed,
                    actions != nullptr ? *step_base + t : 0ull, forced, actions, sampled, uniforms);
}

// The tail of the heads for the cluster path of the fully connected layer, which has already taken the head dot
// products over each half of the hidden units: hp[half][e][k], k < A the policy rows, k = A the value row, rows
// HS_LD floats apart.  One warp per state, lane k holds logit k; softmax and sampling as in heads_kernel.
constexpr int HS_LD = 32, HS_WARPS = 4;
__global__ void __launch_bounds__(HS_WARPS * 32)
heads_sample_kernel(const float* __restrict__ hp, const float* __restrict__ bpi, const float* __restrict__ bv, int n, int A,
                    float* __restrict__ logits, float* __restrict__ values, uint64_t seed,
                    const uint64_t* __restrict__ step_base, uint32_t t, const int32_t* __restrict__ forced,
                    int32_t* __restrict__ actions, int32_t* __restrict__ sampled, float* __restrict__ uniforms,
                    uint64_t* advance_step, uint32_t advance_by, HeadMode mode) {
  const int lane = threadIdx.x & 31;
  const int e = blockIdx.x * HS_WARPS + (threadIdx.x >> 5);
  const float b = lane < A ? __ldg(bpi + lane) : (lane == A ? __ldg(bv) : 0.f);     // biases are older than the previous kernel
  pdl_entry();
  // the last kernel of a rollout also moves the environments' step index on (nothing in this launch reads it then)
  if (advance_step != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *advance_step += advance_by;
  if (e >= n) return;
  float s = -INFINITY;
  if (lane <= A) s = (hp[(size_t)e * HS_LD + lane] + hp[((size_t)n + e) * HS_LD + lane]) + b;
  const float z = lane < A ? s : -INFINITY;
  warp_finish_heads(mode, z, __shfl_sync(0xffffffffu, s, A), lane, A, (size_t)e, logits, values, actions != nullptr, seed,
                    actions != nullptr ? *step_base + t : 0ull, forced, actions, sampled, uniforms);
}

bool heads_fused_supported(const NetDims& nd) { return nd.F == 512 && nd.pi_w % 8 == 0 && nd.A <= 32; }

void launch_heads_fused(LaunchCtx& lc, const NetDims& nd, const float* theta, const bf16* theta16, const float* part,
                        int splits, bf16* h_out, int n, float* logits, float* values, uint64_t seed,
                        const uint64_t* step_base, uint32_t t, const int32_t* forced, int32_t* actions, int32_t* sampled,
                        float* uniforms, HeadMode mode, uint64_t* advance_step, uint32_t advance_by) {
  KernelScope scope(lc, KID_HEADS_FWD);
  if (splits == 0) {          // `part` holds the head dot products of the two halves of the hidden units
    launch_kernel_overlapped(lc, heads_sample_kernel, (n + HS_WARPS - 1) / HS_WARPS, HS_WARPS * 32, 0, part, theta + nd.pi_b,
                             theta + nd.v_b, n, nd.A, logits, values, seed, advance_step ? nullptr : step_base, t, forced,
                             actions, sampled, uniforms, advance_step, advance_by, mode);
    return;
  }
  launch_kernel(lc, heads_fused_kernel, (n + HF_WARPS - 1) / HF_WARPS, HF_WARPS * 32, 0, part, splits, theta + nd.layer[nd.n_conv].b_off, h_out,
                theta16 + nd.pi_w, theta + nd.pi_b, theta16 + nd.v_w, theta + nd.v_b, n, nd.A, logits, values, seed,
                step_base, t, forced, actions, sampled, uniforms, mode);
}

// Element-wise variant of the heads kernel for layouts without 16-byte alignment and for float storage.
// One warp per state.  Lane k ends up holding logit k (A <= 32).  If `actions` is given,
// the warp also draws a_t: u from Philox counter (env, step_lo, step_hi, ACTION stream), then the
// smallest k with u < p_0 + ... + p_k, the running sum taken serially in float in index order.
template <class T, class TW>
__global__ void __launch_bounds__(128)
heads_slow_kernel(const T* __restrict__ h, const TW* __restrict__ wpi, const float* __restrict__ bpi,
             const TW* __restrict__ wv, const float* __restrict__ bv, int n, int F, int A,
             float* __restrict__ logits, float* __restrict__ values, uint64_t seed, const uint64_t* __restrict__ step_base, uint32_t t,
             const int32_t* __restrict__ forced, int32_t* __restrict__ actions, int32_t* __restrict__ sampled,
             float* __restrict__ uniforms, HeadMode mode) {
  pdl_entry();
  const int lane = threadIdx.x & 31;
  const int e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (e >= n) return;
  const T* x = h + (size_t)e * F;
  float z = -INFINITY;
  for (int k = 0; k < A; ++k) {
    float acc = 0.f;
    for (int i = lane; i < F; i += 32) acc = fmaf(to_f(wpi[(size_t)k * F + i]), to_f(x[i]), acc);
    acc = warp_sum(acc) + bpi[k];
    if (lane == k) z = acc;
  }
  float v = 0.f;
  for (int i = lane; i < F; i += 32) v = fmaf(to_f(wv[i]), to_f(x[i]), v);
  v = warp_sum(v) + bv[0];
  warp_finish_heads(mode, z, v, lane, A, (size_t)e, logits, values, actions != nullptr, seed,
                    actions != nullptr ? *step_base + t : 0ull, forced, actions, sampled, uniforms);
}

void launch_heads(LaunchCtx& lc, int prec, const NetDims& nd, const float* theta,
                  const bf16* theta16, const void* h, int n, float* logits, float* values, uint64_t seed,
                  const uint64_t* step_base, uint32_t t, const int32_t* forced, int32_t* actions, int32_t* sampled,
                  float* uniforms, HeadMode mode) {
  const int blocks = (n + 3) / 4;
  KernelScope scope(lc, KID_HEADS_FWD);
  cudaStream_t st = lc.st;
  const float* bpi = theta + nd.pi_b; const float* bv = theta + nd.v_b;
  const bool aligned = nd.pi_w % 8 == 0;      // 16-byte loads of the policy rows
  if (prec == PAAC_BF16 && nd.F == 512 && aligned)
    launch_kernel(lc, heads_kernel<bf16, bf16, 16>, blocks, 128, 0, (const bf16*)h, theta16 + nd.pi_w, bpi, theta16 + nd.v_w, bv, n,
                                                         nd.A, logits, values, seed, step_base, t, forced, actions, sampled, uniforms, mode);
  else if (prec == PAAC_BF16 && nd.F == 256 && aligned)
    launch_kernel(lc, heads_kernel<bf16, bf16, 8>, blocks, 128, 0, (const bf16*)h, theta16 + nd.pi_w, bpi, theta16 + nd.v_w, bv, n,
                                                        nd.A, logits, values, seed, step_base, t, forced, actions, sampled, uniforms, mode);
  else if (prec == PAAC_BF16)
    launch_kernel(lc, heads_slow_kernel<bf16, bf16>, blocks, 128, 0, (const bf16*)h, theta16 + nd.pi_w, bpi, theta16 + nd.v_w, bv,
                                                          n, nd.F, nd.A, logits, values, seed, step_base, t, forced, actions,
                                                          sampled, uniforms, mode);
  else
    launch_kernel(lc, heads_slow_kernel<float, float>, blocks, 128, 0, (const float*)h, theta + nd.pi_w, bpi, theta + nd.v_w, bv,
                                                            n, nd.F, nd.A, logits, values, seed, step_base, t, forced, actions,
                                                            sampled, uniforms, mode);
}

// One warp per experience i = (t, e).  Lane 0 first walks the environment's transitions backwards from the bootstrap
// value down to step t, R_u = r_u + gamma * (1 - terminal_u) * R_{u+1} (one multiply by gamma * keep, one add, the
// same operations in the same order for every t, so all warps of an environment see the same bits), which gives
// R_t and adv_t = R_t - V_t.  Then d/dz and d/dV of
//   (1/B) [ -adv log pi(a) - beta H + c_v (R - V)^2 ]
// with adv and R constants, and the three per-sample loss terms.  The block that finishes last adds the loss terms
// up in a fixed order (a reproducible mean) and resets the arrival counter for the next launch.
__global__ void __launch_bounds__(128)
returns_head_grad_kernel(int algo, int n_e, int t_max, int A, float gamma, float beta, float value_coef,
                         const int8_t* __restrict__ rewards, const uint8_t* __restrict__ terminals,
                         const float* __restrict__ logits, const float* __restrict__ values,
                         const int32_t* __restrict__ actions, float* __restrict__ R, float* __restrict__ adv,
                         float* __restrict__ dz, float* __restrict__ dV, float* loss_terms, DeviceStats* stats) {
  pdl_entry();
  const int B = n_e * t_max;
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  __shared__ bool last;
  __shared__ float sh[3][128], wsum[3][4];
  if (i < B) {
    float ret, ad;
    // everything the row needs is asked for at once (the kernel is a chain of memory latencies otherwise)
    const float z = lane < A ? logits[(size_t)i * A + lane] : -INFINITY;
    const int a = actions[i];
    const float v_i = values[i];
    {
      const int t = i / n_e, e = i - t * n_e;
      float next = values[(size_t)t_max * n_e + e];
      if (t_max <= 32) {
        // lane u fetches transition u, so that the loads are in flight together; the scan itself is serial
        float rw = 0.f, keep = 0.f;
        if (lane >= t && lane < t_max) {
          const size_t j = (size_t)lane * n_e + e;
          rw = (float)rewards[j];
          keep = terminals[j] ? 0.f : 1.f;
        }
        for (int u = t_max - 1; u >= t; --u)
          next = __fadd_rn(__shfl_sync(0xffffffffu, rw, u), __fmul_rn(__fmul_rn(gamma, __shfl_sync(0xffffffffu, keep, u)), next));
      } else {
        for (int u = t_max - 1; u >= t; --u) {
          const size_t j = (size_t)u * n_e + e;
          const float keep = terminals[j] ? 0.f : 1.f;
          next = __fadd_rn((float)rewards[j], __fmul_rn(__fmul_rn(gamma, keep), next));
        }
      }
      ret = next;
      ad = __fsub_rn(next, v_i);
      if (lane == 0) { R[i] = ret; adv[i] = ad; }
    }
    const float m = warp_max(z);
    const float ex = lane < A ? expf(z - m) : 0.f;
    const float lse = m + logf(warp_sum(ex));
    const float lp = z - lse;
    const float p = lane < A ? expf(lp) : 0.f;
    const float H = -warp_sum(lane < A ? p * lp : 0.f);
    const float invB = 1.0f / (float)B;
    if (algo == PAAC_ALGO_NSTEP_Q) {
      // value-based variant: L = value_coef (R - Q(s, a))^2, R constant; only the taken action's output has a gradient
      const float d = __shfl_sync(0xffffffffu, z, a) - ret;
      if (lane < A) dz[(size_t)i * A + lane] = lane == a ? 2.f * value_coef * d * invB : 0.f;
      if (lane == 0) {
        dV[i] = 0.f;
        wsum[0][threadIdx.x >> 5] = 0.f;
        wsum[1][threadIdx.x >> 5] = value_coef * d * d;
        wsum[2][threadIdx.x >> 5] = 0.f;
      }
    } else {
      if (lane < A) {
        const float g = -ad * ((lane == a ? 1.f : 0.f) - p) + beta * p * (lp + H);
        dz[(size_t)i * A + lane] = g * invB;
      }
      const float lp_a = __shfl_sync(0xffffffffu, lp, a);
      if (lane == 0) {
        const float d = v_i - ret;
        dV[i] = 2.f * value_coef * d * invB;
        wsum[0][threadIdx.x >> 5] = -ad * lp_a;
        wsum[1][threadIdx.x >> 5] = value_coef * d * d;
        wsum[2][threadIdx.x >> 5] = H;
      }
    }
  } else if (lane == 0) {
    for (int j = 0; j < 3; ++j) wsum[j][threadIdx.x >> 5] = 0.f;
  }
  // the block's three sums go to loss_terms[j][block]; the last block to arrive adds all blocks' sums in a fixed order
  __syncthreads();
  if (threadIdx.x < 3)
    loss_terms[(size_t)threadIdx.x * gridDim.x + blockIdx.x] =
        ((wsum[threadIdx.x][0] + wsum[threadIdx.x][1]) + wsum[threadIdx.x][2]) + wsum[threadIdx.x][3];
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(&stats->arrivals, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last) return;
  __threadfence();
  float acc[3] = {0.f, 0.f, 0.f};
  for (int k = threadIdx.x; k < (int)gridDim.x; k += 128)
    for (int j = 0; j < 3; ++j) acc[j] += __ldcg(loss_terms + (size_t)j * gridDim.x + k);
  for (int j = 0; j < 3; ++j) sh[j][threadIdx.x] = acc[j];
  __syncthreads();
  for (int s2 = 64; s2 > 0; s2 >>= 1) {
    if (threadIdx.x < s2)
      for (int j = 0; j < 3; ++j) sh[j][threadIdx.x] += sh[j][threadIdx.x + s2];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    stats->policy_loss = sh[0][0] / B;
    stats->value_loss = sh[1][0] / B;
    stats->entropy = sh[2][0] / B;
    stats->arrivals = 0u;
  }
}

void launch_returns_head_grad(LaunchCtx& lc, HeadMode mode, int n_e, int t_max, int A, float gamma, float beta, float value_coef,
                              const int8_t* rewards, const uint8_t* terminals, const float* logits, const float* values,
                              const int32_t* actions, float* R, float* adv, float* dz, float* dV, float* loss_terms,
                              DeviceStats* stats) {
  const int B = n_e * t_max;
  KernelScope scope(lc, KID_HEAD_GRAD);
  launch_kernel(lc, returns_head_grad_kernel, (B + 3) / 4, 128, 0, mode.algo, n_e, t_max, A, gamma, beta, value_coef, rewards, terminals,
                logits, values, actions, R, adv, dz, dV, loss_terms, stats);
}

}  // namespace paac
