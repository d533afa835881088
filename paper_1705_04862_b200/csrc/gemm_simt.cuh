// Generic float-accumulating contraction on the CUDA cores:
//   C(m, n) = sum_k A(m, k) * B(n, k),  k in the split's range,
// with A, B given as index functors (so convolution windows, transposes and
// validity masks need no materialised matrix) and the result handed to an
// epilogue functor.  Used for the fp32 configurations, for the small head
// layers, and as the portable path every tensor-core kernel is checked against.
#pragma once
#include "common.cuh"

namespace paac {

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16, SG_THREADS = 256;

// BM x BN = the output tile: 64 x 64, or 32 / 16 rows for contractions with at most that many rows (the weight
// gradients of layers with 16 or 32 output channels, a batch of four states), or 32 / 16 columns for contractions with
// at most that many columns (the forward pass of those layers), where most of a 64 x 64 tile's multiply-adds would be
// padding.
template <int BM, int BN, class LA, class LB, class EP>
__global__ void __launch_bounds__(SG_THREADS)
gemm_simt_kernel(int M, int N, int K, int k_per_split, LA la, LB lb, EP ep) {
  pdl_entry();
  constexpr int RM = BM / 16, CN = BN / 16;      // rows and columns per thread
  __shared__ float As[SG_BK][BM + 4];
  __shared__ float Bs[SG_BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN, split = blockIdx.z;
  const int k_begin = split * k_per_split;
  const int k_end = min(K, k_begin + k_per_split);
  float acc[RM][CN];
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < CN; ++j) acc[i][j] = 0.f;

  // operand values of one k block, fetched into registers one block ahead of the multiply-adds that use them, so that
  // the loads' latency overlaps the arithmetic of the block before (the order of the additions does not change)
  constexpr int NA = BM * SG_BK / SG_THREADS, NB = BN * SG_BK / SG_THREADS;
  float ra[NA], rb[NB];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < NA; ++i) {
      const int idx = tid + i * SG_THREADS;
      int kk, mm;
      if (LA::K_CONTIG) { kk = idx % SG_BK; mm = idx / SG_BK; } else { mm = idx % BM; kk = idx / BM; }
      const int m = m0 + mm, k = k0 + kk;
      ra[i] = (m < M && k < k_end) ? la(m, k) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      const int idx = tid + i * SG_THREADS;
      int kk, nn;
      if (LB::K_CONTIG) { kk = idx % SG_BK; nn = idx / SG_BK; } else { nn = idx % BN; kk = idx / BN; }
      const int n = n0 + nn, k = k0 + kk;
      rb[i] = (n < N && k < k_end) ? lb(n, k) : 0.f;
    }
  };
  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += SG_BK) {
#pragma unroll
    for (int i = 0; i < NA; ++i) {
      const int idx = tid + i * SG_THREADS;
      if (LA::K_CONTIG) As[idx % SG_BK][idx / SG_BK] = ra[i]; else As[idx / BM][idx % BM] = ra[i];
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      const int idx = tid + i * SG_THREADS;
      if (LB::K_CONTIG) Bs[idx % SG_BK][idx / SG_BK] = rb[i]; else Bs[idx / BN][idx % BN] = rb[i];
    }
    __syncthreads();
    if (k0 + SG_BK < k_end) fetch(k0 + SG_BK);
#pragma unroll
    for (int kk = 0; kk < SG_BK; ++kk) {
      float a[RM], b[CN];
#pragma unroll
      for (int i = 0; i < RM; ++i) a[i] = As[kk][ty * RM + i];
#pragma unroll
      for (int j = 0; j < CN; ++j) b[j] = Bs[kk][tx * CN + j];
#pragma unroll
      for (int i = 0; i < RM; ++i)
#pragma unroll
        for (int j = 0; j < CN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < CN; ++j) {
      const int m = m0 + ty * RM + i, n = n0 + tx * CN + j;
      if (m < M && n < N) ep(m, n, acc[i][j], split);
    }
}

template <class LA, class LB, class EP>
inline void gemm_simt(LaunchCtx& lc, int kid, int M, int N, int K, int splits, LA la, LB lb, EP ep) {
  if (M <= 0 || N <= 0 || K <= 0) return;
  KernelScope scope(lc, kid);
  int kps = (K + splits - 1) / splits;
  kps = (kps + SG_BK - 1) / SG_BK * SG_BK;
  if (M <= 32) {
    dim3 grid(1, (N + SG_BN - 1) / SG_BN, (K + kps - 1) / kps);
    if (M <= 16) launch_kernel(lc, gemm_simt_kernel<16, SG_BN, LA, LB, EP>, grid, SG_THREADS, 0, M, N, K, kps, la, lb, ep);
    else launch_kernel(lc, gemm_simt_kernel<32, SG_BN, LA, LB, EP>, grid, SG_THREADS, 0, M, N, K, kps, la, lb, ep);
    return;
  }
  if (N <= 32) {
    dim3 grid((M + SG_BM - 1) / SG_BM, 1, (K + kps - 1) / kps);
    if (N <= 16) launch_kernel(lc, gemm_simt_kernel<SG_BM, 16, LA, LB, EP>, grid, SG_THREADS, 0, M, N, K, kps, la, lb, ep);
    else launch_kernel(lc, gemm_simt_kernel<SG_BM, 32, LA, LB, EP>, grid, SG_THREADS, 0, M, N, K, kps, la, lb, ep);
    return;
  }
  dim3 grid((M + SG_BM - 1) / SG_BM, (N + SG_BN - 1) / SG_BN, (K + kps - 1) / kps);
  launch_kernel(lc, gemm_simt_kernel<SG_BM, SG_BN, LA, LB, EP>, grid, SG_THREADS, 0, M, N, K, kps, la, lb, ep);
}
// number of k-splits gemm_simt will really launch for a requested count
inline int gemm_simt_splits(int K, int splits) {
  int kps = (K + splits - 1) / splits;
  kps = (kps + SG_BK - 1) / SG_BK * SG_BK;
  return (K + kps - 1) / kps;
}

// ---- operand functors ----------------------------------------------------------------
// x[row][k], rows ld apart
template <class T> struct RowMajorOp {
  static constexpr bool K_CONTIG = true;
  const T* p; int ld;
  __device__ __forceinline__ float operator()(int r, int k) const { return to_f(p[(size_t)r * ld + k]); }
};
// x[k][row]
template <class T> struct ColMajorOp {
  static constexpr bool K_CONTIG = false;
  const T* p; int ld;
  __device__ __forceinline__ float operator()(int r, int k) const { return to_f(p[(size_t)k * ld + r]); }
};
// x[k][row] with one extra row index == n_rows that reads as 1 (folds the bias gradient
// into a weight-gradient contraction)
template <class T> struct ColMajorOnesOp {
  static constexpr bool K_CONTIG = false;
  const T* p; int ld; int n_rows;
  __device__ __forceinline__ float operator()(int r, int k) const {
    return r < n_rows ? to_f(p[(size_t)k * ld + r]) : 1.f;
  }
};

// convolution window: row m = (state, oh, ow), k = (r, s, ci)
template <class G, class T> struct ConvWindowOp {
  static constexpr bool K_CONTIG = true;
  const T* x;
  __device__ __forceinline__ float operator()(int m, int k) const {
    const int b = m / (G::OH * G::OW), rem = m % (G::OH * G::OW), oh = rem / G::OW, ow = rem % G::OW;
    const int r = k / (G::K * G::C), s = (k / G::C) % G::K, ci = k % G::C;
    return to_f(x[((size_t)(b * G::H + oh * G::S + r) * G::W + (ow * G::S + s)) * G::C + ci]);
  }
};
// the same window seen from the weight gradient: row j = (r, s, ci) or the ones row, k = (state, oh, ow)
template <class G, class T> struct ConvWindowTOp {
  static constexpr bool K_CONTIG = false;
  const T* x;
  __device__ __forceinline__ float operator()(int j, int m) const {
    if (j >= G::KK) return 1.f;
    const int b = m / (G::OH * G::OW), rem = m % (G::OH * G::OW), oh = rem / G::OW, ow = rem % G::OW;
    const int r = j / (G::K * G::C), s = (j / G::C) % G::K, ci = j % G::C;
    return to_f(x[((size_t)(b * G::H + oh * G::S + r) * G::W + (ow * G::S + s)) * G::C + ci]);
  }
};
// data gradient: row m = (state, y, x) of the layer input, k = (r, s, co); zero where the
// window (oh, ow) = ((y-r)/S, (x-s)/S) does not exist
template <class G, class T> struct ConvDgradOp {
  static constexpr bool K_CONTIG = true;
  const T* g;
  __device__ __forceinline__ float operator()(int m, int k) const {
    const int b = m / (G::H * G::W), rem = m % (G::H * G::W), y = rem / G::W, x = rem % G::W;
    const int r = k / (G::K * G::CO), s = (k / G::CO) % G::K, co = k % G::CO;
    const int t = y - r, u = x - s;
    if (t < 0 || u < 0 || t % G::S || u % G::S) return 0.f;
    const int oh = t / G::S, ow = u / G::S;
    if (oh >= G::OH || ow >= G::OW) return 0.f;
    return to_f(g[((size_t)(b * G::OH + oh) * G::OW + ow) * G::CO + co]);
  }
};
// Stride-2, 4 x 4 kernel: the input pixels of parity class (py, px) = (y & 1, x & 1) are touched only by the four taps
// (py + 2 i, px + 2 j), so each class is a dense contraction of its own with a quarter of the reduction length and
// no structural zeros.  Row m = (state, y >> 1, x >> 1), k = (i, j, co).
template <class G, class T> struct ConvDgradClassOp {
  static constexpr bool K_CONTIG = true;
  const T* g; int py, px;
  __device__ __forceinline__ float operator()(int m, int k) const {
    constexpr int HH = G::H / 2, WW = G::W / 2;
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    const int i = k / (2 * G::CO), j = (k / G::CO) & 1, co = k % G::CO;
    const int oh = yy - i, ow = xx - j;                       // ((2 yy + py) - (py + 2 i)) / 2
    if (oh < 0 || ow < 0 || oh >= G::OH || ow >= G::OW) return 0.f;
    return to_f(g[((size_t)(b * G::OH + oh) * G::OW + ow) * G::CO + co]);
  }
};
template <class G, class T> struct ConvWeightClassOp {        // row ci, k = (i, j, co) -> tap (py + 2 i, px + 2 j)
  static constexpr bool K_CONTIG = true;
  const T* w; int py, px;
  __device__ __forceinline__ float operator()(int ci, int k) const {
    const int i = k / (2 * G::CO), j = (k / G::CO) & 1, co = k % G::CO;
    return to_f(w[((size_t)(co * G::K + py + 2 * i) * G::K + px + 2 * j) * G::C + ci]);
  }
};
// weights seen from the data gradient: row ci, k = (r, s, co)
template <class G, class T> struct ConvWeightTOp {
  static constexpr bool K_CONTIG = true;
  const T* w;
  __device__ __forceinline__ float operator()(int ci, int k) const {
    const int r = k / (G::K * G::CO), s = (k / G::CO) % G::K, co = k % G::CO;
    return to_f(w[((size_t)(co * G::K + r) * G::K + s) * G::C + ci]);
  }
};

// ---- epilogues ------------------------------------------------------------------------
// out[m][n] = relu(acc * scale + bias[n])
template <class T> struct BiasReluEp {
  T* out; const float* bias; int ld; float scale;
  __device__ __forceinline__ void operator()(int m, int n, float acc, int) const {
    const float z = fmaf(acc, scale, bias[n]);
    out[(size_t)m * ld + n] = from_f<T>(fmaxf(z, 0.f));
  }
};
// out[m][n] = act[m][n] > 0 ? acc : 0   (gradient through the ReLU of the layer below)
template <class T> struct ReluMaskEp {
  T* out; const T* act; int ld;
  __device__ __forceinline__ void operator()(int m, int n, float acc, int) const {
    const size_t i = (size_t)m * ld + n;
    out[i] = to_f(act[i]) > 0.f ? from_f<T>(acc) : from_f<T>(0.f);
  }
};
// the same for one parity class of a stride-2 layer: row m = (state, y >> 1, x >> 1) -> pixel (2 yy + py, 2 xx + px)
template <class G, class T> struct ReluMaskClassEp {
  T* out; const T* act; int py, px;
  __device__ __forceinline__ void operator()(int m, int n, float acc, int) const {
    constexpr int HH = G::H / 2, WW = G::W / 2;
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    const size_t i = ((size_t)(b * G::H + 2 * yy + py) * G::W + 2 * xx + px) * G::C + n;
    out[i] = to_f(act[i]) > 0.f ? from_f<T>(acc) : from_f<T>(0.f);
  }
};
// split-k partial: part[split][m][n]
struct PartialEp {
  float* part; int M, N;
  __device__ __forceinline__ void operator()(int m, int n, float acc, int split) const {
    part[((size_t)split * M + m) * N + n] = acc;
  }
};

// fixed-order sum of the split-k partials part[split][part_rows][cols+1] (last column = bias
// gradient) for rows row0 .. row0+rows-1 into the canonical gradient vector
static __global__ void wgrad_reduce_kernel(const float* part, int splits, int part_rows, int row0, int rows, int cols,
                                           float scale, float* gw, float* gb) {
  pdl_entry();
  const size_t total = (size_t)rows * (cols + 1), stride = (size_t)part_rows * (cols + 1);
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const float* src = part + (size_t)row0 * (cols + 1) + i;
    float s = 0.f;
    for (int p = 0; p < splits; ++p) s += src[(size_t)p * stride];
    const int r = (int)(i / (cols + 1)), c = (int)(i % (cols + 1));
    if (c < cols) gw[(size_t)r * cols + c] = s * scale; else gb[r] = s;
  }
}

}  // namespace paac
