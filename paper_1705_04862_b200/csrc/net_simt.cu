// The network's layers as contractions on the CUDA cores (float accumulate):
// forward with fused bias + ReLU, data gradients with the ReLU mask of the layer
// below fused, weight gradients as split-k partial sums reduced in a fixed order.
#include "gemm_tc3.cuh"
#include "kernels.h"

namespace paac {

static int pick_splits(int M, int N, int K) {
  const int blocks = ((M + SG_BM - 1) / SG_BM) * ((N + SG_BN - 1) / SG_BN);
  int s = (592 + blocks - 1) / blocks;
  const int by_k = (K + 127) / 128;
  if (s > by_k) s = by_k;
  if (s > 512) s = 512;
  if (s < 1) s = 1;
  return gemm_simt_splits(K, s);
}

static void reduce_wgrad(LaunchCtx& lc, const float* part, int splits, int part_rows, int row0,
                         int rows, int cols, float scale, float* gw, float* gb) {
  const size_t total = (size_t)rows * (cols + 1);
  int blocks = (int)((total + 255) / 256);
  if (blocks > 2368) blocks = 2368;
  KernelScope scope(lc, KID_WGRAD_REDUCE);
  launch_kernel(lc, wgrad_reduce_kernel, blocks, 256, 0, part, splits, part_rows, row0, rows, cols, scale, gw, gb);
}

template <class G, class TIn, class T, class TW>
static void conv_fwd(LaunchCtx& lc, int kid, const TIn* x, const TW* w, const float* bias, T* out, int n,
                     float scale) {
  gemm_f32(lc, kid, n * G::OH * G::OW, G::CO, G::KK, 1, ConvWindowOp<G, TIn>{x}, RowMajorOp<TW>{w, G::KK},
            BiasReluEp<T>{out, bias, G::CO, scale});
}
// out[m][n] = relu(sum over splits (in order) of part[split][m][n] + bias[n])
template <class T>
static __global__ void fc_finish_simt_kernel(const float* __restrict__ part, int splits, int M, int N,
                                             const float* __restrict__ bias, T* __restrict__ out) {
  pdl_entry();
  const size_t total = (size_t)M * N;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    // the partial sums are added in double: the pre-activation then differs from an exactly rounded one only by the
    // error inside each short partial sum, and fewer units near zero end up on the other side of the ReLU
    double s = 0.0;
    for (int p = 0; p < splits; ++p) s += (double)part[(size_t)p * total + i];
    out[i] = from_f<T>(fmaxf((float)(s + (double)bias[i % N]), 0.f));
  }
}
// With few states the fully connected layer is a handful of 64 x 64 tiles over a reduction of thousands: the
// reduction is then split over many blocks (partial sums in scratch, added in a fixed order by a finishing kernel)
// so that the weight matrix is streamed by the whole device instead of by four blocks.
template <class T, class TW>
static void fc_fwd(LaunchCtx& lc, int kid, const T* x, const TW* w, const float* bias, T* out, int n,
                   int IN, int F, float* scratch) {
  const int splits = scratch != nullptr ? pick_splits(n, F, IN) : 1;
  if (splits <= 1) {
    gemm_f32(lc, kid, n, F, IN, 1, RowMajorOp<T>{x, IN}, RowMajorOp<TW>{w, IN}, BiasReluEp<T>{out, bias, F, 1.f});
    return;
  }
  gemm_f32(lc, kid, n, F, IN, splits, RowMajorOp<T>{x, IN}, RowMajorOp<TW>{w, IN}, PartialEp{scratch, n, F});
  KernelScope scope(lc, kid);
  int blocks = (n * F + 255) / 256;
  if (blocks > 1184) blocks = 1184;
  launch_kernel(lc, fc_finish_simt_kernel<T>, blocks, 256, 0, scratch, splits, n, F, bias, out);
}
template <class G, class T, class TW>
static void conv_dgrad(LaunchCtx& lc, int kid, const T* g, const TW* w, const T* act_in, T* gin, int n) {
  if constexpr (G::S == 2 && G::K == 4 && G::H % 2 == 0 && G::W % 2 == 0) {
    // four parity classes, each a dense contraction over its own four taps (a quarter of the multiply-adds)
    for (int z = 0; z < 4; ++z)
      gemm_f32(lc, kid, n * (G::H / 2) * (G::W / 2), G::C, 4 * G::CO, 1, ConvDgradClassOp<G, T>{g, z >> 1, z & 1},
                ConvWeightClassOp<G, TW>{w, z >> 1, z & 1}, ReluMaskClassEp<G, T>{gin, act_in, z >> 1, z & 1});
    return;
  }
  gemm_f32(lc, kid, n * G::H * G::W, G::C, G::K * G::K * G::CO, 1, ConvDgradOp<G, T>{g}, ConvWeightTOp<G, TW>{w},
            ReluMaskEp<T>{gin, act_in, G::C});
}
template <class G, class TIn, class T>
static void conv_wgrad(LaunchCtx& lc, int kid, const T* g, const TIn* x, int n, float scale, float* gw,
                       float* gb, float* scratch) {
  const int M = G::CO, N = G::KK + 1, K = n * G::OH * G::OW;
  const int splits = pick_splits(M, N, K);
  gemm_f32(lc, kid, M, N, K, splits, ColMajorOp<T>{g, G::CO}, ConvWindowTOp<G, TIn>{x}, PartialEp{scratch, M, N});
  reduce_wgrad(lc, scratch, splits, M, 0, M, G::KK, scale, gw, gb);
}
template <class T, class TW>
static void fc_dgrad(LaunchCtx& lc, int kid, const T* g, const TW* w, const T* act_in, T* gin, int n,
                     int IN, int F) {
  gemm_f32(lc, kid, n, IN, F, 1, RowMajorOp<T>{g, F}, ColMajorOp<TW>{w, IN}, ReluMaskEp<T>{gin, act_in, IN});
}
template <class T>
static void fc_wgrad(LaunchCtx& lc, int kid, const T* g, const T* x, int n, int IN, int F, float* gw,
                     float* gb, float* scratch) {
  const int M = F, N = IN + 1, K = n;
  const int splits = pick_splits(M, N, K);
  gemm_f32(lc, kid, M, N, K, splits, ColMajorOp<T>{g, F}, ColMajorOnesOp<T>{x, IN, IN}, PartialEp{scratch, M, N});
  reduce_wgrad(lc, scratch, splits, M, 0, M, IN, 1.f, gw, gb);
}

template <class T, class TW>
static void forward_t(LaunchCtx& lc, int arch, const NetDims& nd, const float* theta, const TW* w,
                      const uint8_t* frames, int n, void* const act[], float* scratch) {
  const LayerDims* d = nd.layer;
  const float s255 = 1.0f / 255.0f;
  if (arch == PAAC_ARCH_NIPS) {
    conv_fwd<NipsConv1, uint8_t, T, TW>(lc, KID_CONV1_FWD, frames, w + d[0].w_off, theta + d[0].b_off, (T*)act[0], n, s255);
    conv_fwd<NipsConv2, T, T, TW>(lc, KID_CONV2_FWD, (const T*)act[0], w + d[1].w_off, theta + d[1].b_off, (T*)act[1], n, 1.f);
    fc_fwd<T, TW>(lc, KID_FC_FWD, (const T*)act[1], w + d[2].w_off, theta + d[2].b_off, (T*)act[2], n, 2592, 256, scratch);
  } else {
    conv_fwd<NatConv1, uint8_t, T, TW>(lc, KID_CONV1_FWD, frames, w + d[0].w_off, theta + d[0].b_off, (T*)act[0], n, s255);
    conv_fwd<NatConv2, T, T, TW>(lc, KID_CONV2_FWD, (const T*)act[0], w + d[1].w_off, theta + d[1].b_off, (T*)act[1], n, 1.f);
    conv_fwd<NatConv3, T, T, TW>(lc, KID_CONV3_FWD, (const T*)act[1], w + d[2].w_off, theta + d[2].b_off, (T*)act[2], n, 1.f);
    fc_fwd<T, TW>(lc, KID_FC_FWD, (const T*)act[2], w + d[3].w_off, theta + d[3].b_off, (T*)act[3], n, 3136, 512, scratch);
  }
}

// one layer of the backward pass: its weight gradient and/or the data gradient handed to the layer below
template <class T, class TW>
static void backward_layer_t(LaunchCtx& lc, int arch, const NetDims& nd, const TW* w, const uint8_t* frames, int n,
                             void* const act[], void* const gact[], float* grad, float* scratch, int l, bool wg,
                             bool dg) {
  const LayerDims* d = nd.layer;
  const float s255 = 1.0f / 255.0f;
  const T* g = (const T*)gact[l];
  const T* x = l > 0 ? (const T*)act[l - 1] : nullptr;
  T* gin = l > 0 ? (T*)gact[l - 1] : nullptr;
  float* gw = grad + d[l].w_off; float* gb = grad + d[l].b_off;
  const TW* wl = w + d[l].w_off;
  if (arch == PAAC_ARCH_NIPS) {
    if (l == 2) {
      if (wg) fc_wgrad<T>(lc, KID_FC_WGRAD, g, x, n, 2592, 256, gw, gb, scratch);
      if (dg) fc_dgrad<T, TW>(lc, KID_FC_DGRAD, g, wl, x, gin, n, 2592, 256);
    } else if (l == 1) {
      if (wg) conv_wgrad<NipsConv2, T, T>(lc, KID_CONV2_WGRAD, g, x, n, 1.f, gw, gb, scratch);
      if (dg) conv_dgrad<NipsConv2, T, TW>(lc, KID_CONV2_DGRAD, g, wl, x, gin, n);
    } else if (wg) {
      conv_wgrad<NipsConv1, uint8_t, T>(lc, KID_CONV1_WGRAD, g, frames, n, s255, gw, gb, scratch);
    }
  } else {
    if (l == 3) {
      if (wg) fc_wgrad<T>(lc, KID_FC_WGRAD, g, x, n, 3136, 512, gw, gb, scratch);
      if (dg) fc_dgrad<T, TW>(lc, KID_FC_DGRAD, g, wl, x, gin, n, 3136, 512);
    } else if (l == 2) {
      if (wg) conv_wgrad<NatConv3, T, T>(lc, KID_CONV3_WGRAD, g, x, n, 1.f, gw, gb, scratch);
      if (dg) conv_dgrad<NatConv3, T, TW>(lc, KID_CONV3_DGRAD, g, wl, x, gin, n);
    } else if (l == 1) {
      if (wg) conv_wgrad<NatConv2, T, T>(lc, KID_CONV2_WGRAD, g, x, n, 1.f, gw, gb, scratch);
      if (dg) conv_dgrad<NatConv2, T, TW>(lc, KID_CONV2_DGRAD, g, wl, x, gin, n);
    } else if (wg) {
      conv_wgrad<NatConv1, uint8_t, T>(lc, KID_CONV1_WGRAD, g, frames, n, s255, gw, gb, scratch);
    }
  }
}

void simt_backward_layer(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta, const bf16* theta16,
                         const uint8_t* frames, int n, void* const act[], void* const gact[], float* grad,
                         float* scratch, int layer, bool wgrad, bool dgrad) {
  if (prec == PAAC_BF16)
    backward_layer_t<bf16, bf16>(lc, arch, nd, theta16, frames, n, act, gact, grad, scratch, layer, wgrad, dgrad);
  else
    backward_layer_t<float, float>(lc, arch, nd, theta, frames, n, act, gact, grad, scratch, layer, wgrad, dgrad);
}

void simt_forward(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta,
                  const bf16* theta16, const uint8_t* frames, int n, void* const act[], float* scratch) {
  if (prec == PAAC_BF16) forward_t<bf16, bf16>(lc, arch, nd, theta, theta16, frames, n, act, scratch);
  else forward_t<float, float>(lc, arch, nd, theta, theta, frames, n, act, scratch);
}

void simt_backward(LaunchCtx& lc, int arch, int prec, const NetDims& nd, const float* theta,
                   const bf16* theta16, const uint8_t* frames, int n, void* const act[], void* const gact[],
                   float* grad, float* scratch) {
  for (int l = nd.n_conv; l >= 0; --l)
    simt_backward_layer(lc, arch, prec, nd, theta, theta16, frames, n, act, gact, grad, scratch, l, true, l > 0);
}

size_t simt_scratch_floats(int arch, const NetDims& nd, int n, int n_fwd) {
  size_t best = 0;
  for (int l = 0; l <= nd.n_conv; ++l) {
    const LayerDims& d = nd.layer[l];
    const int M = d.CO;
    const int N = (l < nd.n_conv ? d.K * d.K * d.C : d.H * d.W * d.C) + 1;
    const int K = n * d.OH * d.OW;
    const size_t need = (size_t)pick_splits(M, N, K) * M * N;
    if (need > best) best = need;
  }
  const size_t heads = (size_t)pick_splits(nd.A + 1, nd.F + 1, n) * (nd.A + 1) * (nd.F + 1);
  (void)arch;
  if (heads > best) best = heads;
  // split-k partial sums of the fully connected layer's forward pass, which only ever sees n_fwd states at a time
  const LayerDims& f = nd.layer[nd.n_conv];
  const size_t fwd = (size_t)pick_splits(n_fwd, nd.F, f.H * f.W * f.C) * n_fwd * nd.F;
  return best > fwd ? best : fwd;
}

// ---- heads backward (tiny contractions over the A+1 head units) ------------------------------
struct HeadGradOp {          // row = sample, k = head unit (policy logits then value)
  static constexpr bool K_CONTIG = true;
  const float* dz; const float* dV; int A;
  __device__ __forceinline__ float operator()(int m, int k) const { return k < A ? dz[(size_t)m * A + k] : dV[m]; }
};
struct HeadGradTOp {         // row = head unit, k = sample
  static constexpr bool K_CONTIG = false;
  const float* dz; const float* dV; int A;
  __device__ __forceinline__ float operator()(int u, int b) const { return u < A ? dz[(size_t)b * A + u] : dV[b]; }
};
template <class TW> struct HeadWeightOp {   // row = fc unit i, k = head unit
  static constexpr bool K_CONTIG = false;
  const TW* wpi; const TW* wv; int F, A;
  __device__ __forceinline__ float operator()(int i, int k) const {
    return k < A ? to_f(wpi[(size_t)k * F + i]) : to_f(wv[i]);
  }
};

template <class T, class TW>
static void heads_backward_t(LaunchCtx& lc, const NetDims& nd, const TW* w, const T* h, int n,
                             const float* dz, const float* dV, T* gact_fc, float* grad, float* scratch) {
  const int A = nd.A, F = nd.F;
  gemm_f32(lc, KID_HEADS_BWD, n, F, A + 1, 1, HeadGradOp{dz, dV, A}, HeadWeightOp<TW>{w + nd.pi_w, w + nd.v_w, F, A},
            ReluMaskEp<T>{gact_fc, h, F});
  const int splits = pick_splits(A + 1, F + 1, n);
  gemm_f32(lc, KID_HEADS_BWD, A + 1, F + 1, n, splits, HeadGradTOp{dz, dV, A}, ColMajorOnesOp<T>{h, F, F},
            PartialEp{scratch, A + 1, F + 1});
  reduce_wgrad(lc, scratch, splits, A + 1, 0, A, F, 1.f, grad + nd.pi_w, grad + nd.pi_b);
  reduce_wgrad(lc, scratch, splits, A + 1, A, 1, F, 1.f, grad + nd.v_w, grad + nd.v_b);
}

void heads_backward(LaunchCtx& lc, int prec, const NetDims& nd, const float* theta,
                    const bf16* theta16, const void* h, int n, const float* dz, const float* dV, void* gact_fc,
                    float* grad, float* scratch) {
  if (prec == PAAC_BF16)
    heads_backward_t<bf16, bf16>(lc, nd, theta16, (const bf16*)h, n, dz, dV, (bf16*)gact_fc, grad, scratch);
  else
    heads_backward_t<float, float>(lc, nd, theta, (const float*)h, n, dz, dV, (float*)gact_fc, grad, scratch);
}

}  // namespace paac
