// Global-norm clipping fused with RMSProp.
#include "kernels.h"

namespace paac {

constexpr int OPT_THREADS = 256;

// pass 1: block b sums g^2 over its fixed slice of the parameter vector
__global__ void __launch_bounds__(OPT_THREADS)
sumsq_kernel(const float* __restrict__ g, size_t P, float* __restrict__ partials) {
  pdl_entry();
  __shared__ float sh[OPT_THREADS];
  const size_t per = ((P + gridDim.x - 1) / gridDim.x + 3) / 4 * 4;
  const size_t lo = (size_t)blockIdx.x * per, hi = lo + per < P ? lo + per : P;
  float acc = 0.f;
  if (lo < hi) {
    // slice starts are multiples of 4 floats, so 16-byte loads are aligned
    const size_t n4 = (hi - lo) / 4;
    const float4* g4 = reinterpret_cast<const float4*>(g + lo);
    for (size_t i = threadIdx.x; i < n4; i += OPT_THREADS) {
      const float4 v = g4[i];
      acc = fmaf(v.x, v.x, acc); acc = fmaf(v.y, v.y, acc); acc = fmaf(v.z, v.z, acc); acc = fmaf(v.w, v.w, acc);
    }
    for (size_t i = lo + n4 * 4 + threadIdx.x; i < hi; i += OPT_THREADS) acc = fmaf(g[i], g[i], acc);
  }
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int s = OPT_THREADS / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) partials[blockIdx.x] = sh[0];
}

// pass 2: every block re-adds the partials in the same order (so all agree bit for bit),
// forms scale = min(1, clip / norm) and applies
//   m <- rho m + (1 - rho) (scale g)^2,  theta <- theta - lr (scale g) / sqrt(m + eps)
// and refreshes the bf16 copy.  A non-finite norm leaves theta and m untouched, and so does a device error
// left by any earlier kernel (a bounded wait that gave up means some tile or partial sum of this update is
// garbage): the status then names the error.
__global__ void __launch_bounds__(OPT_THREADS)
clip_rmsprop_kernel(size_t P, float* __restrict__ theta, float* __restrict__ rms, const float* __restrict__ g,
                    bf16* __restrict__ theta16, float lr, float rho, float eps, float clip,
                    const float* __restrict__ partials, int n_partials, DeviceStats* stats) {
  pdl_entry();
  __shared__ float sh[OPT_THREADS / 32];
  __shared__ float s_scale;
  // this thread's first elements do not depend on the norm: fetch them before the norm is known
  const size_t n4 = P / 4;
  float4* t4 = reinterpret_cast<float4*>(theta);
  float4* m4 = reinterpret_cast<float4*>(rms);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const size_t i0 = blockIdx.x * (size_t)OPT_THREADS + threadIdx.x;
  float4 gv0 = make_float4(0.f, 0.f, 0.f, 0.f), mv0 = gv0, tv0 = gv0;
  if (i0 < n4) { gv0 = g4[i0]; mv0 = m4[i0]; tv0 = t4[i0]; }
  // the device error word, fetched now so that its latency hides behind the sum of the partials
  uint32_t dev_err = 0u;
  if (threadIdx.x == 0) dev_err = *reinterpret_cast<const volatile uint32_t*>(&stats->error_word);
  float acc = 0.f;
  for (int i = threadIdx.x; i < n_partials; i += OPT_THREADS) acc += partials[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < OPT_THREADS / 32; ++w) total += sh[w];
    const float norm = sqrtf(total);
    float scale = 1.f;
    const bool ok = isfinite(norm) && dev_err == 0u;
    if (ok && clip > 0.f && norm > clip) scale = clip / norm;
    s_scale = ok ? scale : -1.f;
    if (blockIdx.x == 0) {
      stats->grad_norm = norm;
      stats->clip_scale = ok ? scale : 0.f;
      stats->status = ok ? PAAC_OK
                         : ((dev_err & DEV_ERR_WAIT_MASK) ? PAAC_ERR_TIMEOUT
                                                           : ((dev_err & DEV_ERR_RANGE) ? PAAC_ERR_RANGE : PAAC_ERR_NONFINITE));
    }
  }
  __syncthreads();
  const float scale = s_scale;
  if (scale < 0.f) return;
  const float one_m_rho = 1.f - rho;
  for (size_t i = i0; i < n4; i += (size_t)gridDim.x * OPT_THREADS) {
    float4 gv, mv, tv;
    if (i == i0) { gv = gv0; mv = mv0; tv = tv0; }
    else { gv = g4[i]; mv = m4[i]; tv = t4[i]; }
    float* gp = &gv.x; float* mp = &mv.x; float* tp = &tv.x;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float gs = scale * gp[j];
      mp[j] = fmaf(rho, mp[j], one_m_rho * gs * gs);
      tp[j] = tp[j] - lr * gs / sqrtf(mp[j] + eps);
    }
    m4[i] = mv; t4[i] = tv;
    if (theta16 != nullptr) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(tv.x, tv.y), hi = __floats2bfloat162_rn(tv.z, tv.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo); pk.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(theta16)[i] = pk;
    }
  }
  if (blockIdx.x == 0) {
    for (size_t i = n4 * 4 + threadIdx.x; i < P; i += OPT_THREADS) {
      const float gs = scale * g[i];
      const float m = fmaf(rho, rms[i], one_m_rho * gs * gs);
      rms[i] = m;
      const float t = theta[i] - lr * gs / sqrtf(m + eps);
      theta[i] = t;
      if (theta16 != nullptr) theta16[i] = __float2bfloat16_rn(t);
    }
  }
}

void launch_clip_rmsprop(LaunchCtx& lc, size_t P, float* theta, float* rms, const float* grad,
                         bf16* theta16, float lr, float rho, float eps, float clip, float* norm_partials,
                         DeviceStats* stats, int ready_partials) {
  int n_partials = ready_partials;
  if (ready_partials <= 0) {
    KernelScope scope(lc, KID_SUMSQ);
    launch_kernel(lc, sumsq_kernel, NORM_BLOCKS, OPT_THREADS, 0, grad, P, norm_partials);
    n_partials = NORM_BLOCKS;
  }
  KernelScope scope(lc, KID_CLIP_RMSPROP);
  launch_kernel(lc, clip_rmsprop_kernel, NORM_BLOCKS, OPT_THREADS, 0, P, theta, rms, grad, theta16, lr, rho, eps, clip,
                                                              norm_partials, n_partials, stats);
}

}  // namespace paac
