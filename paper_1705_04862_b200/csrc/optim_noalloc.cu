// Global-norm clipping + RMSProp for callers that must not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a real-time control loop that
// was promised a fixed memory footprint, inside a host process whose memory pool is owned by another
// framework and fully handed out, or in a sandbox that only lets pre-built modules touch the device.
// They cannot give the optimiser its scratch (the per-block partial sums of the squared gradient).  This
// file therefore carries that scratch itself, as a file-scope __device__ array that is part of the loaded
// module: every GPU that loads the library holds these 16 KB until the process exits, and no call here
// allocates or frees anything, on the device or through a library.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int NA_SLICE = 4096;                        // parameters per partial sum
constexpr int NA_MAX_SLICES = 4096;                   // capacity of the static scratch
constexpr size_t NA_MAX_PARAMS = (size_t)NA_SLICE * NA_MAX_SLICES;   // 16,777,216
constexpr int NA_THREADS = 256;
constexpr int NA_MAX_DEVICES = 64;

// One partial sum per slice.  Shared by every call on the device and never cleared: each call overwrites
// the entries it will read before reading them, so stale contents are harmless, but two calls that overlap
// on the GPU (different streams) would overwrite each other's sums.
static __device__ __align__(256) float g_noalloc_partials[NA_MAX_SLICES];

// In host code the array's name is only a handle for the runtime; the device address has to be asked for,
// once per device, with that device current.
std::mutex g_setup_mutex;
float* g_partials_addr[NA_MAX_DEVICES] = {};

int partials_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) { cudaGetLastError(); return PAAC_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_partials_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || p == nullptr) { cudaGetLastError(); return PAAC_ERR_CUDA; }
    g_partials_addr[dev] = static_cast<float*>(p);
  }
  *out = g_partials_addr[dev];
  return PAAC_OK;
}

// pass 1: block b writes the sum of squares of slice b
__global__ void __launch_bounds__(NA_THREADS)
noalloc_sumsq_kernel(const float* __restrict__ g, size_t n, float* __restrict__ partials) {
  __shared__ float sh[NA_THREADS];
  const size_t lo = (size_t)blockIdx.x * NA_SLICE, hi = lo + NA_SLICE < n ? lo + NA_SLICE : n;
  float acc = 0.f;
  for (size_t i = lo + threadIdx.x; i < hi; i += NA_THREADS) acc = fmaf(g[i], g[i], acc);
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int s = NA_THREADS / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) partials[blockIdx.x] = sh[0];
}

// pass 2: every block adds the partials in the same order, forms scale = min(1, clip / norm) and updates
// its slice: m <- rho m + (1 - rho)(scale g)^2, theta <- theta - lr (scale g) / sqrt(m + eps)
__global__ void __launch_bounds__(NA_THREADS)
noalloc_update_kernel(float* __restrict__ theta, float* __restrict__ rms, const float* __restrict__ g,
                      uint16_t* __restrict__ theta_bf16, size_t n, float lr, float rho, float eps, float clip,
                      const float* __restrict__ partials, int n_partials, float* __restrict__ norm_and_scale) {
  __shared__ float sh[NA_THREADS];
  __shared__ float s_scale;
  float acc = 0.f;
  for (int i = threadIdx.x; i < n_partials; i += NA_THREADS) acc += partials[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int s = NA_THREADS / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float norm = sqrtf(sh[0]);
    const bool ok = isfinite(norm);
    float scale = 1.f;
    if (ok && clip > 0.f && norm > clip) scale = clip / norm;
    s_scale = ok ? scale : -1.f;
    if (blockIdx.x == 0 && norm_and_scale != nullptr) { norm_and_scale[0] = norm; norm_and_scale[1] = ok ? scale : 0.f; }
  }
  __syncthreads();
  const float scale = s_scale;
  if (scale < 0.f) return;                           // non-finite norm: leave everything as it is
  const float one_m_rho = 1.f - rho;
  const size_t lo = (size_t)blockIdx.x * NA_SLICE, hi = lo + NA_SLICE < n ? lo + NA_SLICE : n;
  for (size_t i = lo + threadIdx.x; i < hi; i += NA_THREADS) {
    const float gs = scale * g[i];
    const float m = fmaf(rho, rms[i], one_m_rho * gs * gs);
    rms[i] = m;
    const float t = theta[i] - lr * gs / sqrtf(m + eps);
    theta[i] = t;
    if (theta_bf16 != nullptr) theta_bf16[i] = __bfloat16_as_ushort(__float2bfloat16_rn(t));
  }
}

}  // namespace

extern "C" int paac_clip_rmsprop_noalloc(float* theta, float* rms, const float* grad, uint16_t* theta_bf16, size_t n,
                                         float lr, float rms_decay, float rms_eps, float clip_norm,
                                         float* norm_and_scale, void* stream) {
  if (!theta || !rms || !grad || n == 0) return PAAC_ERR_ARG;
  if (n > NA_MAX_PARAMS) return PAAC_ERR_LIMIT;
  float* partials = nullptr;
  const int st = partials_for_current_device(&partials);
  if (st != PAAC_OK) return st;
  const int blocks = (int)((n + NA_SLICE - 1) / NA_SLICE);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  noalloc_sumsq_kernel<<<blocks, NA_THREADS, 0, s>>>(grad, n, partials);
  noalloc_update_kernel<<<blocks, NA_THREADS, 0, s>>>(theta, rms, grad, theta_bf16, n, lr, rms_decay, rms_eps,
                                                      clip_norm, partials, blocks, norm_and_scale);
  return cudaGetLastError() == cudaSuccess ? PAAC_OK : PAAC_ERR_CUDA;
}

extern "C" size_t paac_noalloc_max_params(void) { return NA_MAX_PARAMS; }
