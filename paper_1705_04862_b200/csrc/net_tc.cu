// The bf16 network on the 5th-generation tensor cores: every layer is an implicit GEMM whose
// operand tiles are gathered straight from the NHWC tensors into swizzled shared memory,
// multiplied by tcgen05.mma into a float accumulator in tensor memory, and finished by an
// epilogue that reads the accumulator back with tcgen05.ld.
//
// Kernel anatomy (one output tile of 128 rows per CTA, 160 threads):
//   warps 0-3  producers: each thread owns one of the 128 tile rows; per 64-wide K block it
//              loads its 128 bytes of A (and, for the first BN threads, 128 bytes of B) from
//              global memory, stores them into the stage's 128B-swizzled image, fences the
//              writes towards the async proxy and arrives on the stage's "full" barrier.
//              After the main loop the same warps are the epilogue: warp w reads TMEM lanes
//              32w..32w+31 (its rows) and writes the finished values.
//   warp 4     lane 0 issues the MMAs (four K=16 instructions per stage) and commits each
//              stage to its "empty" barrier, then commits the accumulator barrier.
// Every wait is bounded; a wait that gives up raises a CTA-wide abort flag and an error bit
// the host reads, and all threads still meet at the final barrier so TMEM is released.
#include "kernels.h"
#include "tc_common.cuh"

namespace paac {
using namespace tc;

constexpr int TC_BM = 128, TC_BK = 64, TC_THREADS = 160;

struct TcShared {
  uint64_t full[8], empty[8], acc;
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// ---- A-operand sources: 64 bf16 (128 bytes) of row m for K block kb ---------------------------
// plain row-major matrix x[m][k]
struct PlainSrc {
  const bf16* x; int ld; int M;
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    m = min(m, M - 1);
    const uint4* p = reinterpret_cast<const uint4*>(x + (size_t)m * ld + kb * TC_BK);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};
// convolution window over a bf16 NHWC tensor; k = (r, s, ci); a K block holds 64 / C taps of one kernel row
template <class G> struct ConvSrc {
  const bf16* x; int M;
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    static_assert(64 % G::C == 0 && G::K % (64 / G::C) == 0, "a K block must stay inside one kernel row");
    m = min(m, M - 1);
    const int b = m / (G::OH * G::OW), rem = m % (G::OH * G::OW), oh = rem / G::OW, ow = rem % G::OW;
    const int tap = kb * (64 / G::C), r = tap / G::K, s = tap % G::K;
    const uint4* p = reinterpret_cast<const uint4*>(
        x + ((size_t)(b * G::H + oh * G::S + r) * G::W + (ow * G::S + s)) * G::C);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};
// first layer: uint8 frames [84][84][4]; a kernel row is 8 pixels x 4 channels = 32 bytes, a K block two
// kernel rows.  Pixel values 0..255 are exact in bf16; the 1/255 normalisation is applied in the epilogue.
__device__ __forceinline__ uint32_t u8x2_to_bf16x2(uint32_t lo, uint32_t hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn((float)lo, (float)hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ void u8x16_to_bf16(const uint4& q, uint4& a, uint4& b) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
  uint32_t o[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = u8x2_to_bf16x2(w[i] & 255u, (w[i] >> 8) & 255u);
    o[2 * i + 1] = u8x2_to_bf16x2((w[i] >> 16) & 255u, w[i] >> 24);
  }
  a = make_uint4(o[0], o[1], o[2], o[3]);
  b = make_uint4(o[4], o[5], o[6], o[7]);
}
template <class G> struct FrameSrc {
  const uint8_t* x; int M;
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    static_assert(G::K * G::C == 32, "one kernel row must be 32 bytes");
    m = min(m, M - 1);
    const int b = m / (G::OH * G::OW), rem = m % (G::OH * G::OW), oh = rem / G::OW, ow = rem % G::OW;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int r = kb * 2 + j;
      const uint4* p = reinterpret_cast<const uint4*>(
          x + ((size_t)(b * G::H + oh * G::S + r) * G::W + ow * G::S) * G::C);
      const uint4 q0 = __ldg(p), q1 = __ldg(p + 1);
      u8x16_to_bf16(q0, v[4 * j], v[4 * j + 1]);
      u8x16_to_bf16(q1, v[4 * j + 2], v[4 * j + 3]);
    }
  }
};

// ---- B-operand source: K-major weight matrix w[n][k] -------------------------------------------------
struct WeightSrc {
  const bf16* w; int ld;
  __device__ __forceinline__ void load(int n, int kb, int, uint4 (&v)[8]) const {
    const uint4* p = reinterpret_cast<const uint4*>(w + (size_t)n * ld + kb * TC_BK);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};

// ---- epilogues: 32 accumulator columns n0..n0+31 of row m --------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}
// out[m][n] = bf16(relu(acc * scale + bias[n]))
struct BiasReluEpiTc {
  bf16* out; const float* bias; int ld; float scale; int M;
  __device__ __forceinline__ void operator()(int m, int n0, int, const uint32_t (&r)[32]) const {
    if (m >= M) return;
    uint32_t o[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float a = fmaxf(fmaf(__uint_as_float(r[2 * j]), scale, __ldg(bias + n0 + 2 * j)), 0.f);
      const float b = fmaxf(fmaf(__uint_as_float(r[2 * j + 1]), scale, __ldg(bias + n0 + 2 * j + 1)), 0.f);
      o[j] = pack_bf16x2(a, b);
    }
    uint4* dst = reinterpret_cast<uint4*>(out + (size_t)m * ld + n0);
#pragma unroll
    for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
  }
};

// ---- data-gradient sources: rows of the layer INPUT, k = (tap, co) -------------------------------------
// stride-1 convolution with CO = 64: K block kb is tap (r, s); the row for input pixel (y, x) is the
// 64 output-channel gradients of window (y - r, x - s), or zeros where that window does not exist.
template <class G> struct DgradSrcS1 {
  const bf16* g; int M;
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    static_assert(G::S == 1 && G::CO == 64, "one tap per K block");
    m = min(m, M - 1);
    const int b = m / (G::H * G::W), rem = m % (G::H * G::W), y = rem / G::W, x = rem % G::W;
    const int oh = y - kb / G::K, ow = x - kb % G::K;
    if (oh < 0 || oh >= G::OH || ow < 0 || ow >= G::OW) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
      return;
    }
    const uint4* p = reinterpret_cast<const uint4*>(g + ((size_t)(b * G::OH + oh) * G::OW + ow) * G::CO);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};
// stride-2, 4x4 kernel, CO = 64.  Input pixels are split into four parity classes z = (y&1, x&1); a
// pixel of class z is touched only by the four taps (r, s) = (py + 2i, px + 2j), so each class is its
// own dense contraction with K = 4 taps x 64 and no structural zeros.  Row m = (state, y>>1, x>>1).
template <class G> struct DgradSrcS2 {
  const bf16* g; int M;
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    static_assert(G::S == 2 && G::K == 4 && G::CO == 64 && G::H % 2 == 0 && G::W % 2 == 0, "parity split");
    constexpr int HH = G::H / 2, WW = G::W / 2;
    m = min(m, M - 1);
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    const int oh = yy - (kb >> 1), ow = xx - (kb & 1);
    if (oh < 0 || oh >= G::OH || ow < 0 || ow >= G::OW) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
      return;
    }
    const uint4* p = reinterpret_cast<const uint4*>(g + ((size_t)(b * G::OH + oh) * G::OW + ow) * G::CO);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};
// per-class K-major weights w[z][n][k]
struct ClassWeightSrc {
  const bf16* w; int ld; int class_stride;
  __device__ __forceinline__ void load(int n, int kb, int z, uint4 (&v)[8]) const {
    const uint4* p = reinterpret_cast<const uint4*>(w + (size_t)z * class_stride + (size_t)n * ld + kb * TC_BK);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};

// out[m][n] = act[m][n] > 0 ? bf16(acc) : 0     (gradient through the ReLU of the layer below)
__device__ __forceinline__ void relu_mask_store(bf16* out, const bf16* act, size_t idx, const uint32_t (&r)[32]) {
  const uint4* a4 = reinterpret_cast<const uint4*>(act + idx);
  uint4* dst = reinterpret_cast<uint4*>(out + idx);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint4 a = __ldg(a4 + j);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      // stored activations are >= 0, so "positive" is "non-zero bit pattern other than -0"
      const float lo = (aw[q] & 0x7FFFu) ? __uint_as_float(r[8 * j + 2 * q]) : 0.f;
      const float hi = (aw[q] & 0x7FFF0000u) ? __uint_as_float(r[8 * j + 2 * q + 1]) : 0.f;
      o[q] = pack_bf16x2(lo, hi);
    }
    dst[j] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}
struct ReluMaskEpiTc {
  bf16* out; const bf16* act; int ld; int M;
  __device__ __forceinline__ void operator()(int m, int n0, int, const uint32_t (&r)[32]) const {
    if (m >= M) return;
    relu_mask_store(out, act, (size_t)m * ld + n0, r);
  }
};
// same, scattering parity class z of a stride-2 layer back to its input pixels
template <class G> struct ReluMaskEpiS2 {
  bf16* out; const bf16* act; int M;
  __device__ __forceinline__ void operator()(int m, int n0, int z, const uint32_t (&r)[32]) const {
    if (m >= M) return;
    constexpr int HH = G::H / 2, WW = G::W / 2;
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    const int y = 2 * yy + (z >> 1), x = 2 * xx + (z & 1);
    relu_mask_store(out, act, ((size_t)(b * G::H + y) * G::W + x) * G::C + n0, r);
  }
};

// ---- the kernel ----------------------------------------------------------------------------------------
template <class ASrc, class BSrc, class Epi, int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS)
tc_gemm_kernel(ASrc a_src, BSrc b_src, Epi epi, int num_kb, uint32_t* error_word) {
  static_assert(BN == 32 || BN == 64 || BN == 128, "tile width");
  constexpr uint32_t A_BYTES = TC_BM * 128, B_BYTES = BN * 128, STAGE_BYTES = A_BYTES + B_BYTES;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ TcShared sh;
  const uint32_t tiles = (smem_u32(dyn_smem) + 1023u) & ~1023u;      // swizzle groups need 1024-byte alignment
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * TC_BM, n0 = blockIdx.y * BN, z = blockIdx.z;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], 4); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.acc, 1);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(&sh.tmem_base, BN);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp < 4) {
    // ---------------- producers ----------------
    const int row = threadIdx.x;                 // tile row owned by this thread
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % STAGES;
      uint4 va[8], vb[8];
      a_src.load(m0 + row, kb, z, va);
      if (row < BN) b_src.load(n0 + row, kb, z, vb);
      // all lanes wait on the same phase; leave the loop together or not at all
      const bool ok = mbar_wait(&sh.empty[s], ((kb / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t a_base = tiles + s * STAGE_BYTES, b_base = a_base + A_BYTES;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint32_t off = sw128_offset(row, c);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_base + off), "r"(va[c].x), "r"(va[c].y),
                     "r"(va[c].z), "r"(va[c].w) : "memory");
        if (row < BN)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(b_base + off), "r"(vb[c].x), "r"(vb[c].y),
                       "r"(vb[c].z), "r"(vb[c].w) : "memory");
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.full[s]);
    }
    // ---------------- epilogue ----------------
    if (mbar_wait(&sh.acc, 0, &sh.abort, error_word, ERR_WAIT_ACC)) {
      tcgen05_fence_after();
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + c * 32, r);
        epi(m0 + row, n0 + c * 32, z, r);
      }
    }
  } else if (lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, BN, 0, 0);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % STAGES;
      ok = mbar_wait(&sh.full[s], (kb / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t a_base = tiles + s * STAGE_BYTES, b_base = a_base + A_BYTES;
#pragma unroll
      for (int k = 0; k < TC_BK / 16; ++k) {
        const uint64_t ad = make_smem_desc(a_base + k * 32, 0, 1024, SWIZZLE_128B);
        const uint64_t bd = make_smem_desc(b_base + k * 32, 0, 1024, SWIZZLE_128B);
        mma_bf16(tmem, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
      }
      mma_commit(&sh.empty[s]);
    }
    if (ok) mma_commit(&sh.acc);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 4) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, BN);
  }
}

template <class ASrc, class BSrc, class Epi, int BN, int STAGES>
static void tc_gemm(LaunchCtx& lc, int kid, ASrc a, BSrc b, Epi e, int M, int N, int num_kb, int Z, uint32_t* error_word) {
  constexpr int smem = STAGES * (TC_BM * 128 + BN * 128) + 1024;
  auto kern = tc_gemm_kernel<ASrc, BSrc, Epi, BN, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  KernelScope scope(lc, kid);
  dim3 grid((M + TC_BM - 1) / TC_BM, N / BN, Z);
  kern<<<grid, TC_THREADS, smem, lc.st>>>(a, b, e, num_kb, error_word);
}

// ---- forward ---------------------------------------------------------------------------------------------
bool tc_supported(int arch, int prec) { return arch == PAAC_ARCH_NATURE && prec == PAAC_BF16; }

void tc_forward(LaunchCtx& lc, int arch, const NetDims& nd, const float* theta, const bf16* w, const uint8_t* frames,
                int n, void* const act[], uint32_t* err) {
  const LayerDims* d = nd.layer;
  const float s255 = 1.0f / 255.0f;
  if (arch != PAAC_ARCH_NATURE) return;   // the caller routes the smaller network to the CUDA-core path
  {
    typedef NatConv1 C1; typedef NatConv2 C2; typedef NatConv3 C3;
    const int M1 = n * C1::OH * C1::OW, M2 = n * C2::OH * C2::OW, M3 = n * C3::OH * C3::OW;
    tc_gemm<FrameSrc<C1>, WeightSrc, BiasReluEpiTc, 32, 4>(
        lc, KID_CONV1_FWD, FrameSrc<C1>{frames, M1}, WeightSrc{w + d[0].w_off, C1::KK},
        BiasReluEpiTc{(bf16*)act[0], theta + d[0].b_off, 32, s255, M1}, M1, 32, C1::KK / 64, 1, err);
    tc_gemm<ConvSrc<C2>, WeightSrc, BiasReluEpiTc, 64, 4>(
        lc, KID_CONV2_FWD, ConvSrc<C2>{(const bf16*)act[0], M2}, WeightSrc{w + d[1].w_off, C2::KK},
        BiasReluEpiTc{(bf16*)act[1], theta + d[1].b_off, 64, 1.f, M2}, M2, 64, C2::KK / 64, 1, err);
    tc_gemm<ConvSrc<C3>, WeightSrc, BiasReluEpiTc, 64, 4>(
        lc, KID_CONV3_FWD, ConvSrc<C3>{(const bf16*)act[1], M3}, WeightSrc{w + d[2].w_off, C3::KK},
        BiasReluEpiTc{(bf16*)act[2], theta + d[2].b_off, 64, 1.f, M3}, M3, 64, C3::KK / 64, 1, err);
    tc_gemm<PlainSrc, WeightSrc, BiasReluEpiTc, 128, 4>(
        lc, KID_FC_FWD, PlainSrc{(const bf16*)act[2], 3136, n}, WeightSrc{w + d[3].w_off, 3136},
        BiasReluEpiTc{(bf16*)act[3], theta + d[3].b_off, 512, 1.f, n}, n, 512, 3136 / 64, 1, err);
  }
}

// ---- weight images for the backward contractions ------------------------------------------------------
// From the canonical bf16 copy: wfc_t[i][o] = Wfc[o][i];  w3_d[ci][r][s][co] = W3[co][r][s][ci];
// w2_d[z][ci][i][j][co] = W2[co][py + 2i][px + 2j][ci] with z = 2 py + px.
__global__ void relayout_weights_kernel(const bf16* __restrict__ w2, const bf16* __restrict__ w3,
                                        const bf16* __restrict__ wfc, bf16* __restrict__ w2_d,
                                        bf16* __restrict__ w3_d, bf16* __restrict__ wfc_t) {
  typedef NatConv2 C2; typedef NatConv3 C3;
  constexpr int N2 = 4 * C2::C * 4 * C2::CO, N3 = C3::C * 9 * C3::CO, NF = 3136 * 512;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < N2 + N3 + NF; i += gridDim.x * blockDim.x) {
    if (i < N2) {
      const int co = i % 64, t = (i / 64) % 4, ci = (i / 256) % 32, z = i / (256 * 32);
      const int r = (z >> 1) + 2 * (t >> 1), s = (z & 1) + 2 * (t & 1);
      w2_d[i] = w2[((co * 4 + r) * 4 + s) * 32 + ci];
    } else if (i < N2 + N3) {
      const int j = i - N2, co = j % 64, tap = (j / 64) % 9, ci = j / 576;
      w3_d[j] = w3[(co * 9 + tap) * 64 + ci];
    } else {
      const int j = i - N2 - N3, o = j % 512, in = j / 512;
      wfc_t[j] = wfc[(size_t)o * 3136 + in];
    }
  }
}
size_t tc_weight_image_elems() { return 4 * 32 * 256 + 64 * 576 + (size_t)3136 * 512; }

void tc_relayout_weights(LaunchCtx& lc, const NetDims& nd, const bf16* theta16, bf16* images) {
  const LayerDims* d = nd.layer;
  KernelScope scope(lc, KID_CAST);
  relayout_weights_kernel<<<592, 256, 0, lc.st>>>(theta16 + d[1].w_off, theta16 + d[2].w_off, theta16 + d[3].w_off,
                                                  images, images + 4 * 32 * 256, images + 4 * 32 * 256 + 64 * 576);
}

// ---- backward: data gradients ---------------------------------------------------------------------------
void tc_backward_dgrad_fc(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err) {
  const bf16* wfc_t = images + 4 * 32 * 256 + 64 * 576;
  tc_gemm<PlainSrc, WeightSrc, ReluMaskEpiTc, 64, 4>(
      lc, KID_FC_DGRAD, PlainSrc{(const bf16*)gact[3], 512, n}, WeightSrc{wfc_t, 512},
      ReluMaskEpiTc{(bf16*)gact[2], (const bf16*)act[2], 3136, n}, n, 3136, 512 / 64, 1, err);
}
void tc_backward_dgrad_conv3(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err) {
  typedef NatConv3 C3;
  const int M = n * C3::H * C3::W;
  tc_gemm<DgradSrcS1<C3>, WeightSrc, ReluMaskEpiTc, 64, 4>(
      lc, KID_CONV3_DGRAD, DgradSrcS1<C3>{(const bf16*)gact[2], M}, WeightSrc{images + 4 * 32 * 256, 576},
      ReluMaskEpiTc{(bf16*)gact[1], (const bf16*)act[1], 64, M}, M, 64, 9, 1, err);
}
void tc_backward_dgrad_conv2(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err) {
  typedef NatConv2 C2;
  const int M = n * (C2::H / 2) * (C2::W / 2);
  tc_gemm<DgradSrcS2<C2>, ClassWeightSrc, ReluMaskEpiS2<C2>, 32, 4>(
      lc, KID_CONV2_DGRAD, DgradSrcS2<C2>{(const bf16*)gact[1], M}, ClassWeightSrc{images, 256, 32 * 256},
      ReluMaskEpiS2<C2>{(bf16*)gact[0], (const bf16*)act[0], M}, M, 32, 4, 4, err);
}

}  // namespace paac
