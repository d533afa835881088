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
#include <cuda.h>          // CUtensorMap and its enums only; the encoder is looked up at run time, nothing links to libcuda

#include "kernels.h"
#include "tc_common.cuh"

namespace paac {
using namespace tc;

constexpr int TC_BM = 128, TC_BK = 64, TC_THREADS = 160;
// element offsets of the regrouped weight images (see relayout_weights_kernel)
constexpr size_t TC_IMG_W2 = 0, TC_IMG_W3 = 4 * 32 * 256, TC_IMG_WFC = TC_IMG_W3 + 64 * 576,
                 TC_IMG_W1 = TC_IMG_WFC + (size_t)3136 * 512, TC_IMG_END = TC_IMG_W1 + 32 * 256;


// ---- tensor maps for the plain row-major bf16 matrices (fully connected layer) ---------------------------------
// map of matrix x[rows][cols] (row pitch `ld` elements) for boxes of box_rows x 64 elements with the 128-byte swizzle.
// Maps are cached by their defining values: the matrices live at fixed places of the workspace, so after the first
// iteration every call is a look-up.  Returns nullptr if the driver's encoder is unavailable or refuses.
struct TmapKey { const void* p; uint64_t rows, cols, ld; uint32_t box_rows; };
static const CUtensorMap* tc_tensor_map(const bf16* x, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  static bool looked_up = false;
  constexpr int MAX_MAPS = 64;
  static TmapKey keys[MAX_MAPS];
  static CUtensorMap maps[MAX_MAPS];
  static int n_maps = 0;
  for (int i = 0; i < n_maps; ++i)
    if (keys[i].p == x && keys[i].rows == rows && keys[i].cols == cols && keys[i].ld == ld && keys[i].box_rows == box_rows)
      return &maps[i];
  if (!looked_up) {
    looked_up = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      encode = (EncodeFn)fn;
  }
  if (encode == nullptr) return nullptr;
  static int next = 0;                                   // a full cache is overwritten in turn: launches copy the map
  const int slot = n_maps < MAX_MAPS ? n_maps : next++ % MAX_MAPS;
  const cuuint64_t gdim[2] = {cols, rows}, gstride[1] = {ld * sizeof(bf16)};
  const cuuint32_t box[2] = {64u, box_rows}, estride[2] = {1u, 1u};
  keys[slot].p = nullptr;
  if (encode(&maps[slot], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16*>(x), gdim, gstride, box, estride,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return nullptr;
  keys[slot] = TmapKey{x, rows, cols, ld, box_rows};
  if (n_maps < MAX_MAPS) ++n_maps;
  return &maps[slot];
}

// map of a 3-D bf16 tensor x[d2][d1][64] (strides in bytes) for boxes of box2 x box1 rows of 128 bytes, 128-byte swizzle;
// cached by its defining values like the 2-D maps (a full cache is overwritten in turn: launches copy the map);
// nullptr if the encoder is unavailable
static const CUtensorMap* tc_tensor_map3(const bf16* x, uint64_t d1, uint64_t d2, uint64_t stride1, uint64_t stride2,
                                         uint32_t box1, uint32_t box2) {
  struct Key { const void* p; uint64_t d1, d2, s1, s2; uint32_t b1, b2; };
  constexpr int MAX_MAPS = 32;
  static Key keys[MAX_MAPS];
  static CUtensorMap maps[MAX_MAPS];
  static int n_maps = 0, next = 0;
  for (int i = 0; i < n_maps; ++i)
    if (keys[i].p == x && keys[i].d1 == d1 && keys[i].d2 == d2 && keys[i].s1 == stride1 && keys[i].s2 == stride2 &&
        keys[i].b1 == box1 && keys[i].b2 == box2)
      return &maps[i];
  const int slot = n_maps < MAX_MAPS ? n_maps : next++ % MAX_MAPS;
  CUtensorMap* out = &maps[slot];
  keys[slot].p = nullptr;
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  static bool looked_up = false;
  if (!looked_up) {
    looked_up = true;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      encode = (EncodeFn)fn;
  }
  if (encode == nullptr) return nullptr;
  const cuuint64_t gdim[3] = {64, d1, d2}, gstride[2] = {stride1, stride2};
  const cuuint32_t box[3] = {64u, box1, box2}, estride[3] = {1u, 1u, 1u};
  if (encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(x), gdim, gstride, box, estride,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return nullptr;
  keys[slot] = Key{x, d1, d2, stride1, stride2, box1, box2};
  if (n_maps < MAX_MAPS) ++n_maps;
  return out;
}

struct TcShared {
  uint64_t full[8], empty[8], acc;
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// ---- A-operand sources: 64 bf16 (128 bytes) of row m for K block kb ---------------------------
// plain row-major matrix x[m][k]
// Asynchronous sources split the address of (row m, K block kb) into a per-row part, computed once per tile
// row, and a cheap per-block part: row(m) -> RowRef, at(ref, kb, valid) -> address of the 128 bytes, with
// valid = false meaning "reads as zeros".
struct RowRef { uint32_t base; int32_t yx; };
struct PlainSrc {
  static constexpr bool ASYNC = true;
  const bf16* x; int ld; int M;
  __device__ __forceinline__ RowRef row(int m) const { return RowRef{(uint32_t)min(m, M - 1) * (uint32_t)ld, 0}; }
  __device__ __forceinline__ const bf16* at(const RowRef& r, int kb, bool& valid) const {
    valid = true;
    return x + r.base + kb * TC_BK;
  }
  __device__ __forceinline__ const bf16* ptr(int m, int kb, int, bool& valid) const { return at(row(m), kb, valid); }
  __device__ __forceinline__ void load(int m, int kb, int, uint4 (&v)[8]) const {
    m = min(m, M - 1);
    const uint4* p = reinterpret_cast<const uint4*>(x + (size_t)m * ld + kb * TC_BK);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
};
// convolution window over a bf16 NHWC tensor; k = (r, s, ci); a K block holds 64 / C taps of one kernel row
template <class G> struct ConvSrc {
  static constexpr bool ASYNC = true;
  const bf16* x; int M;
  __device__ __forceinline__ RowRef row(int m) const {
    m = min(m, M - 1);
    const int b = m / (G::OH * G::OW), rem = m % (G::OH * G::OW), oh = rem / G::OW, ow = rem % G::OW;
    return RowRef{(uint32_t)(((b * G::H + oh * G::S) * G::W + ow * G::S) * G::C), 0};
  }
  __device__ __forceinline__ const bf16* at(const RowRef& rr, int kb, bool& valid) const {
    valid = true;
    const int tap = kb * (64 / G::C), r = tap / G::K, s = tap % G::K;
    return x + rr.base + (r * G::W + s) * G::C;
  }
  __device__ __forceinline__ const bf16* ptr(int m, int kb, int, bool& valid) const { return at(row(m), kb, valid); }
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
  static constexpr bool ASYNC = false;     // needs the uint8 -> bf16 conversion, so it goes through registers
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
// A warp's 32 rows x 32 floats (thread = row, registers = columns) go to the global rows dst0 + row * ld through a
// 4 KB staging tile of the warp's own, so that every store instruction writes four whole 128-byte rows instead of
// sixteen bytes of thirty-two different rows.  Bit `row` of row_mask says whether that row exists.
__device__ __forceinline__ void warp_store_rows_f32(uint32_t stg, int lane, const uint32_t (&r)[32], float* dst0, size_t ld,
                                                    uint32_t row_mask) {
#pragma unroll
  for (int q = 0; q < 8; ++q)
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + ((uint32_t)(q ^ (lane & 7)) << 4)),
                 "r"(r[4 * q]), "r"(r[4 * q + 1]), "r"(r[4 * q + 2]), "r"(r[4 * q + 3]) : "memory");
  __syncwarp();
  const int ch = lane & 7, rr0 = lane >> 3;
#pragma unroll
  for (int p = 0; p < 8; ++p) {
    const int rr = p * 4 + rr0;
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(stg + rr * 128 + ((uint32_t)(ch ^ (rr & 7)) << 4)) : "memory");
    if ((row_mask >> rr) & 1u) *reinterpret_cast<uint4*>(dst0 + (size_t)rr * ld + ch * 4) = v;
  }
  __syncwarp();
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
  __device__ __forceinline__ RowRef row(int m) const {
    m = min(m, M - 1);
    const int b = m / (G::H * G::W), rem = m % (G::H * G::W), y = rem / G::W, x = rem % G::W;
    return RowRef{(uint32_t)(b * G::OH * G::OW * G::CO), (y << 8) | x};
  }
  __device__ __forceinline__ const bf16* at(const RowRef& rr, int kb, bool& valid) const {
    const int oh = (rr.yx >> 8) - kb / G::K, ow = (rr.yx & 255) - kb % G::K;
    valid = oh >= 0 && oh < G::OH && ow >= 0 && ow < G::OW;
    return valid ? g + rr.base + (oh * G::OW + ow) * G::CO : g;
  }
  __device__ __forceinline__ const bf16* ptr(int m, int kb, int, bool& valid) const { return at(row(m), kb, valid); }
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
  __device__ __forceinline__ RowRef row(int m) const {
    constexpr int HH = G::H / 2, WW = G::W / 2;
    m = min(m, M - 1);
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    return RowRef{(uint32_t)(b * G::OH * G::OW * G::CO), (yy << 8) | xx};
  }
  __device__ __forceinline__ const bf16* at(const RowRef& rr, int kb, bool& valid) const {
    const int oh = (rr.yx >> 8) - (kb >> 1), ow = (rr.yx & 255) - (kb & 1);
    valid = oh >= 0 && oh < G::OH && ow >= 0 && ow < G::OW;
    return valid ? g + rr.base + (oh * G::OW + ow) * G::CO : g;
  }
  __device__ __forceinline__ const bf16* ptr(int m, int kb, int, bool& valid) const { return at(row(m), kb, valid); }
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
// value words (two bf16 each) survive where the activation word's halves are non-zero
__device__ __forceinline__ uint32_t mask_pair(uint32_t v, uint32_t a) {
  // stored activations are ReLU outputs, never negative: non-zero is the same as greater than zero
  const __nv_bfloat162 a2 = *reinterpret_cast<const __nv_bfloat162*>(&a);
  return v & __hgt2_mask(a2, __floats2bfloat162_rn(0.f, 0.f));
}

// the same with the 32 activations of the slice already in registers (four 16-byte words)
__device__ __forceinline__ void relu_mask_store_pre(bf16* out, size_t idx, const uint32_t (&r)[32], const uint4* a4) {
  uint4* dst = reinterpret_cast<uint4*>(out + idx);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t aw[4] = {a4[j].x, a4[j].y, a4[j].z, a4[j].w};
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float lo = (aw[q] & 0x7FFFu) ? __uint_as_float(r[8 * j + 2 * q]) : 0.f;
      const float hi = (aw[q] & 0x7FFF0000u) ? __uint_as_float(r[8 * j + 2 * q + 1]) : 0.f;
      o[q] = pack_bf16x2(lo, hi);
    }
    dst[j] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}
template <int BN> struct MaskPre { uint4 m[BN / 8]; size_t idx; bool valid; };
struct ReluMaskEpiTc {
  bf16* out; const bf16* act; int ld; int M;
  __device__ __forceinline__ void operator()(int m, int n0, int, const uint32_t (&r)[32]) const {
    if (m >= M) return;
    relu_mask_store(out, act, (size_t)m * ld + n0, r);
  }
  // two-step form: fetch the BN activations of row m starting at column n0 early, use them later
  template <class P> __device__ __forceinline__ void prefetch(int m, int n0, P& p) const {
    p.valid = m < M;
    p.idx = (size_t)m * ld + n0;
    if (!p.valid) return;
    const uint4* a4 = reinterpret_cast<const uint4*>(act + p.idx);
#pragma unroll
    for (int j = 0; j < (int)(sizeof(p.m) / sizeof(uint4)); ++j)
      if (n0 + 8 * j < ld) p.m[j] = __ldg(a4 + j);          // a ragged last tile stops at the end of the row
  }
  template <class P> __device__ __forceinline__ void store(int col, const uint32_t (&r)[32], const P& p) const {
    if (p.valid) relu_mask_store_pre(out, p.idx + col, r, &p.m[col / 8]);
  }
};
// same for the stride-2 layer, whose four parity classes share one A operand and are laid side by side
// along N: column n belongs to class n / C, channel n % C, and goes back to input pixel
// (2 yy + class / 2, 2 xx + class % 2)
template <class G> struct ReluMaskEpiS2 {
  bf16* out; const bf16* act; int M;
  __device__ __forceinline__ void operator()(int m, int n0, int, const uint32_t (&r)[32]) const {
    static_assert(G::C == 32, "one class per 32-column slice");
    if (m >= M) return;
    constexpr int HH = G::H / 2, WW = G::W / 2;
    const int cls = n0 / G::C;
    const int b = m / (HH * WW), rem = m % (HH * WW), yy = rem / WW, xx = rem % WW;
    const int y = 2 * yy + (cls >> 1), x = 2 * xx + (cls & 1);
    relu_mask_store(out, act, ((size_t)(b * G::H + y) * G::W + x) * G::C, r);
  }
};

// ---- the kernel ----------------------------------------------------------------------------------------
template <class ASrc, class BSrc, class Epi, int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS)
tc_gemm_kernel(ASrc a_src, BSrc b_src, Epi epi, int num_kb, uint32_t* error_word) {
  pdl_entry();
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

// ---- persistent variant: weights resident in shared memory, A streamed with cp.async -------------------
// One CTA per SM walks over output tiles t = blockIdx.x, blockIdx.x + gridDim.x, ...; tile t is row tile
// t % tiles_m of class t / tiles_m (classes: the parity classes of a stride-2 data gradient, else one).
// The whole K extent of the CTA's weight slice (BN rows, KB blocks, all classes) is loaded once.
//   warps 0-3  epilogue: tile i is read out of its TMEM buffer while tile i+1 is being multiplied
//   warps 4-7  producers: one tile row per thread, eight 16-byte cp.async per K block straight into the
//              swizzled image; a stage is published LAG blocks later, after the thread's copies of it
//              have landed (cp.async.wait_group) and were fenced towards the async proxy
//   warp 8     lane 0 issues the MMAs and commits stages / accumulators
constexpr int PK_THREADS = 288, PK_LAG = 5;
struct PkShared {
  uint64_t full[8], empty[8], acc_full[2], acc_empty[2], mask_full[2], mask_empty[2];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

template <class ASrc, class Epi, int BN, int KB, int NCLS, int STAGES, int KPS>
__global__ void __launch_bounds__(PK_THREADS, 1)
tc_persistent_kernel(const __grid_constant__ CUtensorMap tm_a, const bf16* __restrict__ w, int n_total, Epi epi, int tiles_m,
                     uint32_t* error_word) {
  static_assert(BN == 32 || BN == 64 || BN == 128, "tile width");
  // KPS K blocks share a stage, i.e. one wait and one commit of the issuing thread: with four instructions per K block
  // a wait per block (a couple of hundred cycles even when satisfied) left the tensor pipe idle half of the time
  static_assert(STAGES >= 2 && STAGES <= 8 && KB % KPS == 0, "pipeline shape");
  constexpr uint32_t A_BLOCK = TC_BM * 128, A_BYTES = KPS * A_BLOCK, B_BLOCK = BN * 128, B_BYTES = NCLS * KB * B_BLOCK;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ PkShared sh;
  const uint32_t b_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const uint32_t a_base0 = b_base + B_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.y * BN;
  const int total_tiles = NCLS * tiles_m;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    tma_prefetch_desc(&tm_a);
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 4); }
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(&sh.tmem_base, 2 * BN);
  // resident weights: chunk index -> (class, k block, row, 16-byte chunk)
  for (int i = threadIdx.x; i < NCLS * KB * BN * 8; i += PK_THREADS) {
    const int c = i & 7, row = (i >> 3) % BN, kb = (i / (8 * BN)) % KB, cls = i / (8 * BN * KB);
    // rows past the last output column (a ragged last tile) repeat the last one; the epilogue drops their results
    const bf16* src = w + ((size_t)(cls * n_total + min(n0 + row, n_total - 1)) * KB + kb) * TC_BK + c * 8;
    cp_async16(b_base + (cls * KB + kb) * B_BLOCK + sw128_offset(row, c), src, 16u);
  }
  cp_async_commit();
  cp_async_wait<0>();
  fence_proxy_async_smem();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp >= 4 && warp < 8) {
    // ---------------- producer: one thread asks the copy engine for the 128 x 64 box of each K block ----------------
    // (rows past the end of the matrix read as zeros)
    if (warp == 4 && lane == 0) {
      int it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const int m0 = (t % tiles_m) * TC_BM;
        for (int kb = 0; kb < KB; kb += KPS, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
          if (!ok) break;
          mbar_arrive_expect_tx(&sh.full[s], A_BYTES);
#pragma unroll
          for (int j = 0; j < KPS; ++j) tma_load_2d(a_base0 + s * A_BYTES + j * A_BLOCK, &tm_a, (kb + j) * TC_BK, m0, &sh.full[s]);
        }
      }
    }
  } else if (warp < 4) {
    // ---------------- epilogue: accumulator -> bf16 through the ReLU mask of the layer below ----------------
    // Two phases, so that global memory only sees whole rows: lane = accumulator row packs its BN values into a
    // staging tile of the warp's own (16-byte chunks swizzled by row); then CH lanes cover one row, the warp
    // reads RPP rows per pass, applies the mask (fetched with the same row-wise pattern before the accumulator
    // was ready) and writes RPP x BN x 2 contiguous bytes per row.
    constexpr int CH = BN / 8, RPP = 32 / CH, ROWB = BN * 2;
    const uint32_t stg = a_base0 + STAGES * A_BYTES + warp * (32 * ROWB);
    const int ch = lane % CH, rr0 = lane / CH;
    const bool col_ok = n0 + ch * 8 < n_total;
    int local = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++local) {
      const int ab = local & 1, m0 = (t % tiles_m) * TC_BM + warp * 32;
      uint4 mk[CH];
#pragma unroll
      for (int p = 0; p < CH; ++p) {
        const int m = m0 + p * RPP + rr0;
        mk[p] = make_uint4(0u, 0u, 0u, 0u);
        if (m < epi.M && col_ok) mk[p] = __ldg(reinterpret_cast<const uint4*>(epi.act + (size_t)m * epi.ld + n0 + ch * 8));
      }
      const bool ok = mbar_wait(&sh.acc_full[ab], (local >> 1) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!__all_sync(0xffffffffu, ok)) break;
      tcgen05_fence_after();
#pragma unroll
      for (int cc = 0; cc < BN / 32; ++cc) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + ab * BN + cc * 32, r);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * ROWB + ((uint32_t)((cc * 4 + q) ^ (lane & (CH - 1))) << 4)),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * q]), __uint_as_float(r[8 * q + 1]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * q + 2]), __uint_as_float(r[8 * q + 3]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * q + 4]), __uint_as_float(r[8 * q + 5]))),
                       "r"(pack_bf16x2(__uint_as_float(r[8 * q + 6]), __uint_as_float(r[8 * q + 7]))) : "memory");
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[ab]);            // the accumulator is free again
#pragma unroll
      for (int p = 0; p < CH; ++p) {
        const int rr = p * RPP + rr0, m = m0 + rr;
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(stg + rr * ROWB + ((uint32_t)(ch ^ (rr & (CH - 1))) << 4)) : "memory");
        if (m < epi.M && col_ok) {
          v.x = mask_pair(v.x, mk[p].x); v.y = mask_pair(v.y, mk[p].y); v.z = mask_pair(v.z, mk[p].z); v.w = mask_pair(v.w, mk[p].w);
          *reinterpret_cast<uint4*>(epi.out + (size_t)m * epi.ld + n0 + ch * 8) = v;
        }
      }
      __syncwarp();                                              // staging tile free for the next tile
    }
  } else if (lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, BN, 0, 0);
    int it = 0, local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++local) {
      const int ab = local & 1, z = t / tiles_m;
      ok = mbar_wait(&sh.acc_empty[ab], ((local >> 1) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!ok) break;
      tcgen05_fence_after();
      for (int kb = 0; kb < KB; kb += KPS, ++it) {
        const int s = it % STAGES;
        ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        tcgen05_fence_after();
#pragma unroll
        for (int j = 0; j < KPS; ++j) {
          const uint32_t a_addr = a_base0 + s * A_BYTES + j * A_BLOCK, b_addr = b_base + (z * KB + kb + j) * B_BLOCK;
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)
            mma_bf16(tmem + ab * BN, make_smem_desc(a_addr + k * 32, 0, 1024, SWIZZLE_128B),
                     make_smem_desc(b_addr + k * 32, 0, 1024, SWIZZLE_128B), idesc, (kb | j | k) != 0 ? 1u : 0u);
        }
        mma_commit(&sh.empty[s]);
      }
      if (ok) mma_commit(&sh.acc_full[ab]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 8) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 2 * BN);
  }
}

// ---- convolutions without im2col: shifted views of one staged row block ----------------------------------
// A 128-byte-swizzled operand image may be entered at any 128-byte row (the swizzle is a function of the
// shared-memory address, not of the descriptor), so when the rows of an image are the pixels of a feature
// map in raster order, the A operand of filter tap (r, s) is simply the same image entered (r * width + s)
// rows further down.  A tile therefore stages its 128 + max-shift rows ONCE and issues one group of MMAs
// per tap, instead of gathering a fresh 128 x 64 block per tap.  The tile rows run over every position of
// the (padded or full-width) raster, including positions that are not outputs (right / bottom margins):
// those accumulate finite garbage that the epilogue drops.
//
// Cfg supplies: PLANES (row blocks staged per tile), NT (taps), STAGE_ROWS (multiple of 8, >= 128 + largest
// shift), src(plane, g, valid) -> address of the 128 bytes of raster row g (valid = false: zeros),
// tap_plane(t), tap_shift(t).  The weights are [BN][NT * 64] K-major, block t belonging to tap t.
constexpr int SH_THREADS = 544;     // warps 0-7 epilogue, 8-15 producers, 16 MMA

// Consecutive MMAs go to NACC different accumulators in turn (any partition of the tap x k products sums to the
// same result), so that an MMA does not have to wait for the one before it; the epilogue adds the NACC pieces.
template <class Cfg, class Epi, int BN, int STAGES, int NACC>
__global__ void __launch_bounds__(SH_THREADS, 1)
tc_shift_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, Cfg cfg, const bf16* __restrict__ w, Epi epi, int tiles,
                uint32_t* error_word) {
  static_assert(BN == 64 || BN == 128, "tile width");
  static_assert(2 * NACC * BN <= 512 && (NACC == 1 || NACC == 2 || NACC == 4), "tensor memory budget");
  static_assert(STAGES >= 2 && STAGES <= 8 && Cfg::STAGE_ROWS % 8 == 0, "pipeline shape");
  constexpr int NT = Cfg::NT, SR = Cfg::STAGE_ROWS, PLANES = Cfg::PLANES;
  constexpr uint32_t PLANE_BYTES = SR * 128, STAGE_BYTES = PLANES * PLANE_BYTES, B_BLOCK = BN * 128, B_BYTES = NT * B_BLOCK;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ PkShared sh;
  const uint32_t b_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const uint32_t a_base0 = b_base + B_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // Two barriers per stage slot (a wait costs the single issuing thread a couple of hundred cycles even when it is
    // already satisfied, and the tensor pipe runs dry meanwhile):
    //   full[s]  the stage's copies have landed AND the accumulator of the tile that will use the slot has been read
    //            out by the epilogue of the tile two before it (the first two tiles find that arrival made here);
    //   empty[s] the tile's instructions have completed: the producers may refill the slot, the epilogue may read.
    static_assert(STAGES >= 2, "the accumulator release of tile i arrives on the slot of tile i + 2");
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], (Cfg::BULK != 0 ? 1 : 256) + 8); mbar_init(&sh.empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.mask_full[i], 256); mbar_init(&sh.mask_empty[i], 8); }
    for (int s = 0; s < 2; ++s)
      for (int e = 0; e < 8; ++e) mbar_arrive(&sh.full[s]);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 16) tmem_alloc(&sh.tmem_base, 2 * NACC * BN);
  for (int i = threadIdx.x; i < NT * BN * 8; i += SH_THREADS) {
    const int c = i & 7, row = (i >> 3) % BN, t = i / (8 * BN);
    cp_async16(b_base + t * B_BLOCK + sw128_offset(row, c), w + ((size_t)row * NT + t) * TC_BK + c * 8, 16u);
  }
  cp_async_commit();
  cp_async_wait<0>();
  fence_proxy_async_smem();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (Cfg::BULK != 0 && warp >= 8 && warp < 16) {
    // ---------------- producer: a stage is one box of the layer input per plane, fetched by tiled bulk copies
    // (128-byte swizzle; rows past the end of the tensor read as zeros) ----------------
    static_assert(Cfg::BULK == 0 || !Epi::MASK, "bulk-copied stages: plain forward layers only");
    if (warp == 8 && lane == 0) {
      tma_prefetch_desc(&tm_a);
      if (Cfg::BULK == 2) tma_prefetch_desc(&tm_b);
      int it = 0;
      for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
        const int s = it % STAGES;
        if (!mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY)) break;
        mbar_arrive_expect_tx(&sh.full[s], STAGE_BYTES);
        if (Cfg::BULK == 1) {
          tma_load_2d(a_base0 + s * STAGE_BYTES, &tm_a, 0, t * TC_BM, &sh.full[s]);
        } else {
          tma_load_3d(a_base0 + s * STAGE_BYTES, &tm_a, 0, 0, (t * TC_BM) / 10, &sh.full[s]);
          tma_load_3d(a_base0 + s * STAGE_BYTES + PLANE_BYTES, &tm_b, 0, 0, (t * TC_BM) / 10, &sh.full[s]);
        }
      }
    }
  } else if (warp >= 8 && warp < 16) {
    // ---------------- producers: eight lanes per 128-byte row, 32 rows per pass ----------------
    const int c = lane & 7, sub = (warp - 8) * 4 + (lane >> 3);
    int it = 0;
    bool alive = true;
    for (int t = blockIdx.x; t < tiles && alive; t += gridDim.x, ++it) {
      const int s = it % STAGES;
      const bool ok = mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
      const uint32_t stage = a_base0 + s * STAGE_BYTES;
      // Source addresses by arithmetic only, all of them before the first copy.  A warp that has asynchronous copies
      // in flight must not read shared memory (a table of raster cells, say): the load is made to wait until every
      // one of those copies has landed, which chains the tiles to the memory latency.
      constexpr int NIT = (PLANES * SR + 31) / 32;
      uint32_t srcs[NIT], vmask = 0;                    // element offsets from the tensor's base (< 2^32 elements)
#pragma unroll
      for (int k = 0; k < NIT; ++k) {
        const int idx = sub + 32 * k;
        srcs[k] = 0u;
        if (idx < PLANES * SR) {
          const int plane = PLANES == 1 ? 0 : idx / SR, ri = PLANES == 1 ? idx : idx % SR;
          bool valid;
          const bf16* ptr;
          if constexpr (Cfg::RASTER > 0) ptr = cfg.src_cell(t * TC_BM + ri, valid);
          else ptr = cfg.src(plane, t * TC_BM + ri, valid);
          srcs[k] = (uint32_t)(ptr - cfg.base());
          vmask |= valid ? 1u << k : 0u;
        }
      }
#pragma unroll
      for (int k = 0; k < NIT; ++k) {
        const int idx = sub + 32 * k;
        if (idx < PLANES * SR) {
          const int plane = PLANES == 1 ? 0 : idx / SR, ri = PLANES == 1 ? idx : idx % SR;
          cp_async16(stage + plane * PLANE_BYTES + ri * 128u + ((uint32_t)(c ^ (ri & 7)) << 4), cfg.base() + srcs[k] + c * 8,
                     (vmask >> k) & 1u ? 16u : 0u);
        }
      }
      // no waiting here: the hardware arrives on the stage's barrier for this thread when its copies have landed
      cp_async_mbar_arrive(&sh.full[s]);
      if constexpr (Epi::MASK) {
        // The activations under the tile (the ReLU mask of its epilogue) travel the same way, into a two-slot ring
        // laid out per epilogue warp: producer warp w fetches what epilogue warp w will read.  The epilogue warps
        // cannot fetch them themselves: a warp with asynchronous copies in flight waits for all of them at its next
        // shared-memory load, which would chain every staging-tile read to the DRAM latency.
        constexpr int COLS = BN / 2, CH = COLS / 8, RPP = 32 / CH, ROWB = COLS * 2;
        const int ms = it & 1, ew = warp - 8, quarter = ew & 3, col0 = (ew >> 2) * COLS, rr0 = lane / CH, ch = lane % CH;
        const bool okm = mbar_wait(&sh.mask_empty[ms], ((it >> 1) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
        if (!__all_sync(0xffffffffu, okm)) { alive = false; break; }
        const uint32_t dst = a_base0 + STAGES * STAGE_BYTES + 8 * (32 * ROWB) + ew * (2 * 32 * ROWB) + ms * (32 * ROWB);
        int b, y, x;
        epi.map.split(t * TC_BM + quarter * 32 + rr0, b, y, x);
        uint32_t at = epi.index(b, y, x, col0 + ch * 8);
#pragma unroll
        for (int p = 0; p < CH; ++p) {
          const bool v = epi.map.is_output(b, y, x);
          cp_async16(dst + (p * RPP + rr0) * ROWB + ch * 16, epi.act + (v ? at : 0u), v ? 16u : 0u);
          epi.map.template advance<Epi>(b, y, x, at, RPP);
        }
        cp_async_mbar_arrive(&sh.mask_full[ms]);
      }
    }
    cp_async_commit();
    cp_async_wait<0>();
  } else if (warp < 8) {
    // ---------------- epilogue: warps e and e + 4 share TMEM lane quarter e & 3 and split the columns ----------------
    constexpr int COLS = BN / 2, CH = COLS / 8, RPP = 32 / CH, ROWB = COLS * 2;   // 16-byte chunks per row part
    const int quarter = warp & 3, col0 = (warp >> 2) * COLS;
    const uint32_t stg = a_base0 + STAGES * STAGE_BYTES + warp * (32 * ROWB);    // this warp's staging tile
    // masked epilogues: the activations under a tile arrive in a two-slot ring of this warp, filled by producer
    // warp (this warp + 8) and handed over through the mask_full / mask_empty barriers
    const uint32_t mring = a_base0 + STAGES * STAGE_BYTES + 8 * (32 * ROWB) + warp * (2 * 32 * ROWB);
    const int rr0 = lane / CH, ch = lane % CH;
    int local = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++local) {
      const int ab = local & 1, pos0 = t * TC_BM + quarter * 32;
      // where this lane's chunks go, before the tile is ready
      uint32_t idx[CH];                                          // element offsets (every tensor here is < 2^32 elements)
      uint32_t valid = 0;
      {
        int b, y, x;
        epi.map.split(pos0 + rr0, b, y, x);
        uint32_t at = epi.index(b, y, x, col0 + ch * 8);
#pragma unroll
        for (int p = 0; p < CH; ++p) {
          idx[p] = at;
          if (epi.map.is_output(b, y, x)) valid |= 1u << p;
          epi.map.template advance<Epi>(b, y, x, at, RPP);
        }
      }
      const bool ok = mbar_wait(&sh.empty[local % STAGES], (local / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!__all_sync(0xffffffffu, ok)) break;
      tcgen05_fence_after();
#pragma unroll
      for (int cc = 0; cc < COLS / 32; ++cc) {
        uint32_t r[32], o[16];
        tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + ab * NACC * BN + col0 + cc * 32, r);
#pragma unroll
        for (int a = 1; a < NACC; ++a) {
          uint32_t r2[32];
          tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + (ab * NACC + a) * BN + col0 + cc * 32, r2);
#pragma unroll
          for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) + __uint_as_float(r2[q]));
        }
        epi.values(col0 + cc * 32, r, o);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * ROWB + ((uint32_t)((cc * 4 + q) ^ (lane & (CH - 1))) << 4)),
                       "r"(o[4 * q]), "r"(o[4 * q + 1]), "r"(o[4 * q + 2]), "r"(o[4 * q + 3]) : "memory");
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.full[(local + 2) % STAGES]);      // the accumulator is free for the tile after next
      if constexpr (Epi::MASK) {                                 // this tile's activations have landed
        const bool okm = mbar_wait(&sh.mask_full[local & 1], (local >> 1) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!__all_sync(0xffffffffu, okm)) break;
      }
#pragma unroll
      for (int p = 0; p < CH; ++p) {
        const int rr = p * RPP + rr0;
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(stg + rr * ROWB + ((uint32_t)(ch ^ (rr & (CH - 1))) << 4)) : "memory");
        if ((valid >> p) & 1u) {
          if constexpr (Epi::MASK) {
            uint4 m;
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(m.x), "=r"(m.y), "=r"(m.z), "=r"(m.w)
                         : "r"(mring + (local & 1) * (32 * ROWB) + rr * ROWB + ch * 16) : "memory");
            v.x = mask_pair(v.x, m.x); v.y = mask_pair(v.y, m.y); v.z = mask_pair(v.z, m.z); v.w = mask_pair(v.w, m.w);
          }
          *reinterpret_cast<uint4*>(epi.out + idx[p]) = v;
        }
      }
      __syncwarp();                                              // staging tile and ring slot free again
      if constexpr (Epi::MASK) { if (lane == 0) mbar_arrive(&sh.mask_empty[local & 1]); }
    }
  } else if (warp == 16 && lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, BN, 0, 0);
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
      const int ab = it & 1, s = it % STAGES;
      ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!ok) break;
      fence_proxy_async_smem();        // the copies observed through the barrier -> visible to the MMA's operand reads
      tcgen05_fence_after();
      // descriptor low words: (address >> 4); every operand slice is a compile-time offset from the stage
      // (with boxes that start at the tile's first oh, the tile's own rows begin a few rows into the stage)
      const uint32_t row0 = Cfg::BULK == 2 ? (uint32_t)((t * TC_BM) % 10) : 0u;
      const uint32_t a_lo = (((a_base0 + s * STAGE_BYTES) >> 4) & 0x3FFFu) + row0 * 8u, b_lo = (b_base >> 4) & 0x3FFFu;
      const uint32_t hi = desc_hi_kmajor_sw128(), d = tmem + ab * NACC * BN;
#pragma unroll
      for (int tap = 0; tap < NT; ++tap) {
        constexpr uint32_t K_STEP = 32 >> 4;
        const uint32_t a_off = (Cfg::tap_plane(tap) * PLANE_BYTES + Cfg::tap_shift(tap) * 128u) >> 4;
        const uint32_t b_off = (tap * B_BLOCK) >> 4;
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k) {
          constexpr int KS = TC_BK / 16;
          const int m = tap * KS + k;                       // m-th MMA of the tile -> accumulator m % NACC
          if (m < NACC) mma_bf16_lo<false>(d + (m % NACC) * BN, a_lo + a_off + k * K_STEP, b_lo + b_off + k * K_STEP, hi, idesc);
          else mma_bf16_lo<true>(d + (m % NACC) * BN, a_lo + a_off + k * K_STEP, b_lo + b_off + k * K_STEP, hi, idesc);
        }
      }
      mma_commit(&sh.empty[s]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 16) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 2 * NACC * BN);
  }
}

// conv3 forward: rows = the 9 x 9 x 64 input pixels in memory order; tap (r, s) is 9 r + s rows down
struct C3FwdCfg {
  static constexpr int PLANES = 1, NT = 9, STAGE_ROWS = 152, RASTER = 0;      // RASTER = 0: rows are plain memory order
  static constexpr int BULK = 1;          // a stage is one contiguous run of 128-byte rows: one tiled bulk copy fetches it
  const bf16* x; int rows;                                   // rows = states * 81
  const bf16* base_host() const { return x; }
  int row_count() const { return rows; }
  __device__ __forceinline__ const bf16* base() const { return x; }
  __device__ __forceinline__ const bf16* src(int, int g, bool& valid) const {
    valid = g < rows;
    return valid ? x + (size_t)g * 64 : x;
  }
  __host__ __device__ static constexpr int tap_plane(int) { return 0; }
  __host__ __device__ static constexpr int tap_shift(int t) { return (t / 3) * 9 + t % 3; }
  // tap pairs one raster position apart (see tc_shift_t_kernel): per kernel row (s = 0, s = 1) and s = 2 alone
  static constexpr int NSTEP = 6;
  __host__ __device__ static constexpr int step_lo(int j) { return 3 * (j / 2) + 2 * (j & 1); }
  __host__ __device__ static constexpr int step_hi(int j) { return (j & 1) ? -1 : 3 * (j / 2) + 1; }
};
// conv2 forward: rows = pairs of horizontally adjacent 32-channel pixels (128 bytes), i.e. the input in memory
// order seen as [state][y][10 pairs]; even and odd image rows go to separate planes, so that tap row r
// lives in plane r & 1, 10 (r >> 1) + (pair offset) rows down, and tile rows run over a 10 x 10 raster
struct C2FwdCfg {
  // A plane is the 3-D tensor [state * 10 + oh][10 pairs][64] (20 pair rows from one oh to the next), so a stage is one
  // box of 16 x 10 rows per plane that starts at the tile's first oh; the tile's own rows begin (first position % 10)
  // rows into it, which the MMA descriptors add.
  static constexpr int PLANES = 2, NT = 8, STAGE_ROWS = 160, RASTER = 0;
  static constexpr int BULK = 2;
  const bf16* x; int states;
  const bf16* base_host() const { return x; }
  __device__ __forceinline__ const bf16* base() const { return x; }
  __device__ __forceinline__ const bf16* src(int plane, int g, bool& valid) const {
    // plane row g = (b, oh, X) is pair row 2 g - X + 10 plane of the input in memory order
    valid = g < states * 100;
    return valid ? x + (size_t)(2 * g - g % 10 + 10 * plane) * 64 : x;
  }
  __host__ __device__ static constexpr int tap_plane(int t) { return (t >> 1) & 1; }
  __host__ __device__ static constexpr int tap_shift(int t) { return 10 * (t >> 2) + (t & 1); }
  // tap pairs one raster position apart: the two pixel pairs of a kernel row
  static constexpr int NSTEP = 4;
  __host__ __device__ static constexpr int step_lo(int j) { return 2 * j; }
  __host__ __device__ static constexpr int step_hi(int j) { return 2 * j + 1; }
};
// conv3 data gradient: the 7 x 7 x 64 output gradient on a zero-padded 11 x 11 raster; input pixel (y, x) is
// raster position 11 y + x and tap (r, s) reads (2 - r) * 11 + (2 - s) rows down
struct C3DgradCfg {
  static constexpr int PLANES = 1, NT = 9, STAGE_ROWS = 152, RASTER = 121;
  static constexpr int BULK = 0;
  const bf16* g3; int states;
  __device__ __forceinline__ const bf16* base() const { return g3; }
  // element offset of raster cell `rem` inside a state's 7 x 7 x 64 gradient, or -1 for a padding cell
  __device__ static __forceinline__ int cell(int rem) {
    const int Y = rem / 11, X = rem % 11;
    return (Y >= 2 && Y <= 8 && X >= 2 && X <= 8) ? ((Y - 2) * 7 + (X - 2)) * 64 : -1;
  }
  __device__ __forceinline__ const bf16* src_cell(int g, bool& valid) const {
    const int b = g / RASTER, off = cell(g - b * RASTER);
    valid = b < states && off >= 0;
    return valid ? g3 + (size_t)b * 49 * 64 + off : g3;
  }
  __host__ __device__ static constexpr int tap_plane(int) { return 0; }
  __host__ __device__ static constexpr int tap_shift(int t) { return (2 - t / 3) * 11 + (2 - t % 3); }
};
// conv2 data gradient (all four parity classes along N): the 9 x 9 x 64 gradient on a zero-padded 11 x 11
// raster; class pixel (yy, xx) is position 11 yy + xx and tap (i, j) reads (1 - i) * 11 + (1 - j) rows down
struct C2DgradCfg {
  static constexpr int PLANES = 1, NT = 4, STAGE_ROWS = 144, RASTER = 121;
  static constexpr int BULK = 0;
  const bf16* g2; int states;
  __device__ __forceinline__ const bf16* base() const { return g2; }
  __device__ static __forceinline__ int cell(int rem) {
    const int Y = rem / 11, X = rem % 11;
    return (Y >= 1 && Y <= 9 && X >= 1 && X <= 9) ? ((Y - 1) * 9 + (X - 1)) * 64 : -1;
  }
  __device__ __forceinline__ const bf16* src_cell(int g, bool& valid) const {
    const int b = g / RASTER, off = cell(g - b * RASTER);
    valid = b < states && off >= 0;
    return valid ? g2 + (size_t)b * 81 * 64 + off : g2;
  }
  __host__ __device__ static constexpr int tap_plane(int) { return 0; }
  __host__ __device__ static constexpr int tap_shift(int t) { return (1 - (t >> 1)) * 11 + (1 - (t & 1)); }
};

// epilogues of the shifted kernels: raster position -> output row, or nothing for a margin position
template <int RASTER, int WIDTH, int OUT_H, int OUT_W> struct RasterMap {
  int states;
  __device__ __forceinline__ void split(int pos, int& b, int& y, int& x) const {
    b = pos / RASTER;
    const int rem = pos - b * RASTER;
    y = rem / WIDTH; x = rem - y * WIDTH;
  }
  // n raster cells further (n < WIDTH)
  __device__ __forceinline__ void advance(int& b, int& y, int& x, int n) const {
    x += n;
    if (x >= WIDTH) { x -= WIDTH; if (++y >= RASTER / WIDTH) { y = 0; ++b; } }
  }
  __device__ __forceinline__ bool is_output(int b, int y, int x) const { return b < states && y < OUT_H && x < OUT_W; }
  // the same step for an epilogue whose output offset is affine in (b, y, x): idx = b * E::SB + y * E::SY + x * E::SX + ...
  template <class E> __device__ __forceinline__ void advance(int& b, int& y, int& x, uint32_t& idx, int n) const {
    x += n; idx += (uint32_t)(n * E::SX);
    if (x >= WIDTH) {
      x -= WIDTH; idx += (uint32_t)(E::SY - WIDTH * E::SX);
      if (++y >= RASTER / WIDTH) { y = 0; ++b; idx += (uint32_t)(E::SB - (RASTER / WIDTH) * E::SY); }
    }
  }
};
// Epilogues of the shifted kernels work in two phases per tile.  First the thread that owns a TMEM lane turns
// its row's accumulators into bf16 (`values`) and parks them in a swizzled shared-memory staging tile.  Then
// the warp re-reads the tile with eight (or four) lanes per row, so that every global access of a warp
// instruction covers whole contiguous rows: `locate` gives the output element of (raster position, column),
// and epilogues with MASK also fetch the activation there and zero the value where the activation is zero
// (the gradient through the ReLU of the layer below).  Row-per-thread global accesses, 32 cache lines per
// instruction, were what bounded these kernels before.
template <class Map, int OUT_H, int OUT_W> struct ShiftBiasReluEpi {
  static constexpr bool MASK = false;
  static constexpr int SX = 64, SY = OUT_W * 64, SB = OUT_H * OUT_W * 64;
  Map map; bf16* out; const float* bias; const bf16* act;       // act unused
  __device__ __forceinline__ void values(int col, const uint32_t (&r)[32], uint32_t (&o)[16]) const {
    const float4* b4 = reinterpret_cast<const float4*>(bias + col);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float4 t = __ldg(b4 + j);
      o[2 * j] = pack_bf16x2(fmaxf(__uint_as_float(r[4 * j]) + t.x, 0.f), fmaxf(__uint_as_float(r[4 * j + 1]) + t.y, 0.f));
      o[2 * j + 1] = pack_bf16x2(fmaxf(__uint_as_float(r[4 * j + 2]) + t.z, 0.f), fmaxf(__uint_as_float(r[4 * j + 3]) + t.w, 0.f));
    }
  }
  __device__ __forceinline__ uint32_t index(int b, int y, int x, int col) const {
    return (uint32_t)(((b * OUT_H + y) * OUT_W + x) * 64 + col);
  }
};
__device__ __forceinline__ void plain_bf16_values(const uint32_t (&r)[32], uint32_t (&o)[16]) {
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j] = pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
}
template <class Map, int OUT_H, int OUT_W> struct ShiftReluMaskEpi {
  static constexpr bool MASK = true;
  static constexpr int SX = 64, SY = OUT_W * 64, SB = OUT_H * OUT_W * 64;
  Map map; bf16* out; const bf16* act;
  __device__ __forceinline__ void values(int, const uint32_t (&r)[32], uint32_t (&o)[16]) const { plain_bf16_values(r, o); }
  __device__ __forceinline__ uint32_t index(int b, int y, int x, int col) const {
    return (uint32_t)(((b * OUT_H + y) * OUT_W + x) * 64 + col);
  }
};
// stride-2 data gradient: accumulator columns 32 c .. 32 c + 31 are parity class c of raster pixel (yy, xx)
// `scale` is a power of two the stored gradient is multiplied by before its bf16 rounding (an exact shift of the
// exponent): the first layer's weight-gradient kernel wants its gradient operand that way (see C1_GRAD_SCALE)
template <class Map> struct ShiftReluMaskEpiS2 {
  static constexpr bool MASK = true;
  static constexpr int SX = 2 * 32, SY = 2 * 20 * 32, SB = 20 * 20 * 32;
  Map map; bf16* out; const bf16* act; float scale;
  __device__ __forceinline__ void values(int, const uint32_t (&r)[32], uint32_t (&o)[16]) const {
#pragma unroll
    for (int j = 0; j < 16; ++j) o[j] = pack_bf16x2(__uint_as_float(r[2 * j]) * scale, __uint_as_float(r[2 * j + 1]) * scale);
  }
  __device__ __forceinline__ uint32_t index(int b, int yy, int xx, int col) const {
    const int cls = col >> 5;
    return (uint32_t)(((b * 20 + 2 * yy + (cls >> 1)) * 20 + 2 * xx + (cls & 1)) * 32 + (col & 31));
  }
};
// ---- the same convolutions with the operand roles exchanged: weights as the A operand, held in tensor memory ----
// An M = 128 instruction costs max(~50, N / 2) cycles, so a 64-channel layer that puts its channels along N runs the
// tensor pipe at under two thirds of its rate and fetches 6 KB of operands from shared memory per instruction.  Here the
// raster positions run along N = 128 and the weights are the A operand: the 128 rows of A are the 64 output channels of
// TWO filter taps that lie one raster position apart (row 2 c = tap `lo`, channel c; row 2 c + 1 = tap `hi`, channel c),
// written once per CTA into tensor memory (tcgen05.st: row -> lane, two bf16 per 32-bit column), from where the
// instruction reads them without touching shared memory.  The B operand of a step is the staged input entered
// shift(lo) rows down.  All steps accumulate into one 128 x 128 accumulator; with L = even lanes and H = odd lanes
//   out[c][p] = L[c][p] + H[c][p + 1]
// (the `hi` tap saw every position one row early).  The epilogue thread that owns TMEM lane l holds 32 consecutive
// positions of its row; lanes 2 c and 2 c + 1 exchange what the other needs with one shuffle per two outputs, the even
// lane finishing the even positions and the odd lane the odd ones.  Column 127 of a tile only feeds column 126, so a
// tile yields 127 positions and tiles advance by 127.  The finished bf16 values are parked position-major in a staging
// tile (128 bytes per position) and leave with whole-row stores, as in tc_shift_kernel.
// Cfg adds: NSTEP, step_lo(j), step_hi(j) (tap indices, -1 = none; shift(hi) = shift(lo) + 1, same plane).
// Roles: warps 0-15 epilogue (warp e: TMEM lane quarter e & 3, columns 32 (e >> 2) ..), warp 16 issues the MMAs, one
// thread of warp 17 asks the copy engine for the stages.  Warps 0-3 also write the weights into tensor memory before
// the first tile.  Forward layers only: with a masked epilogue and gathered stages (the data gradients) this
// arrangement measured slower than tc_shift_kernel -- eight warps are too few for the transposing epilogue and
// twenty-four warps in all too many for the SM's issue slots (71 and 77 us against 64 us for the conv3 data gradient),
// and a zero-padded raster fetched as one tiled box per raster row made the producer the bottleneck (a tiled copy
// costs its issuing warp about 80 cycles whatever its size).
constexpr int ST_TILE = 127;
constexpr int ST_THREADS = 576;      // warps 0-15 epilogue, 16 MMA, 17 bulk-copy producer

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 32 columns of this warp's 32 lanes and, if `more`, the column that follows them
__device__ __forceinline__ void tmem_ld_32x32_next(uint32_t taddr, uint32_t r[32], uint32_t& next, bool more) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  next = 0u;
  if (more) asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(next) : "r"(taddr + 32u) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A's 128 rows in the lanes of a_tmem, 16 bf16 of K in eight 32-bit columns
template <bool ACC>
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "n"(ACC ? 1 : 0)
      : "memory");
}
__device__ __forceinline__ void group_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <class Cfg, class Epi, int STAGES>
__global__ void __launch_bounds__(ST_THREADS, 1)
tc_shift_t_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, Cfg cfg, const bf16* __restrict__ w,
                  Epi epi, int tiles, uint32_t* error_word) {
  static_assert(STAGES >= 2 && STAGES <= 8 && Cfg::STAGE_ROWS % 8 == 0, "pipeline shape");
  static_assert(Cfg::BULK != 0 && !Epi::MASK, "forward layers with bulk-copied stages");
  constexpr int NT = Cfg::NT, NS = Cfg::NSTEP, SR = Cfg::STAGE_ROWS, PLANES = Cfg::PLANES;
  constexpr uint32_t PLANE_BYTES = SR * 128, STAGE_BYTES = PLANES * PLANE_BYTES, STG_BYTES = 128 * 128;
  constexpr uint32_t ACC_COLS = 128, A_COL0 = 2 * ACC_COLS, TMEM_COLS = 512;
  constexpr int EW = 16, ROWS_PER_WARP = 128 / EW;                         // epilogue warps
  static_assert(A_COL0 + NS * 32 <= TMEM_COLS, "tensor memory budget: two accumulators and the weights");
  extern __shared__ uint8_t dyn_smem[];
  __shared__ PkShared sh;
  const uint32_t a_base0 = (smem_u32(dyn_smem) + 1023u) & ~1023u;          // operand stages
  const uint32_t stg0 = a_base0 + STAGES * STAGE_BYTES;                    // two staging tiles (tile parity)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // Two barriers per stage slot instead of four per tile: every wait, even one that is already satisfied, costs
    // the single issuing thread a couple of hundred cycles during which the tensor pipe runs dry.
    //   full[s]  ("ready"): the stage's copies have landed AND the accumulator of the tile that will use the slot
    //            has been read out by the epilogue of the tile two before it (the first two tiles find that
    //            arrival made here);
    //   empty[s] ("done"):  the tile's instructions have completed: the producer may refill the slot and the
    //            epilogue may read the accumulator.
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], 1 + EW); mbar_init(&sh.empty[s], 1); }
    for (int s = 0; s < 2; ++s)
      for (int e = 0; e < EW; ++e) mbar_arrive(&sh.full[s]);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 16) tmem_alloc(&sh.tmem_base, TMEM_COLS);
  // The weights pass through shared memory (the operand stages are not in use yet) so that all threads fetch them in
  // one round of copies: A row a of step j (128 bytes) lands at (j * 128 + a) * 128, 16-byte chunks swizzled by row.
  for (int i = threadIdx.x; i < NS * 128 * 8; i += ST_THREADS) {
    const int q = i & 7, arow = (i >> 3) & 127, j = i >> 10;
    const int tap = (arow & 1) ? Cfg::step_hi(j) : Cfg::step_lo(j);
    cp_async16(a_base0 + (uint32_t)(j * 128 + arow) * 128u + ((uint32_t)(q ^ (arow & 7)) << 4),
               w + ((size_t)(arow >> 1) * NT + (tap >= 0 ? tap : 0)) * TC_BK + q * 8, tap >= 0 ? 16u : 0u);
  }
  cp_async_commit();
  cp_async_wait<0>();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  if (warp < 4) {
    // shared memory -> tensor memory: lane l of quarter `warp` is A row 32 warp + l = (tap lo / hi, channel)
    const uint32_t arow = 32u * warp + lane;
#pragma unroll 2
    for (int j = 0; j < NS; ++j) {
      uint32_t r[32];
#pragma unroll
      for (int q = 0; q < 8; ++q)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r[4 * q]), "=r"(r[4 * q + 1]), "=r"(r[4 * q + 2]), "=r"(r[4 * q + 3])
                     : "r"(a_base0 + ((uint32_t)j * 128u + arow) * 128u + (((uint32_t)q ^ (arow & 7u)) << 4)) : "memory");
      tmem_st_32x32(tmem + ((uint32_t)(32 * warp) << 16) + A_COL0 + j * 32, r);
    }
    tmem_st_wait();
  }
  tcgen05_fence_before();
  __syncthreads();          // the stage area is free for the first tiles from here on
  tcgen05_fence_after();
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp == 17) {
    // ---------------- producer: a stage is one box of the layer input per plane (tiled bulk copies) ----------------
    if (lane == 0) {
      tma_prefetch_desc(&tm_a);
      if (Cfg::BULK == 2) tma_prefetch_desc(&tm_b);
      int it = 0;
      for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
        const int s = it % STAGES;
        if (!mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY)) break;
        mbar_arrive_expect_tx(&sh.full[s], STAGE_BYTES);
        if (Cfg::BULK == 1) {
          tma_load_2d(a_base0 + s * STAGE_BYTES, &tm_a, 0, t * ST_TILE, &sh.full[s]);
        } else {
          tma_load_3d(a_base0 + s * STAGE_BYTES, &tm_a, 0, 0, (t * ST_TILE) / 10, &sh.full[s]);
          tma_load_3d(a_base0 + s * STAGE_BYTES + PLANE_BYTES, &tm_b, 0, 0, (t * ST_TILE) / 10, &sh.full[s]);
        }
      }
    }
  } else if (warp < EW) {
    // ---------------- epilogue: warp e reads TMEM lane quarter e & 3, columns (128 / (EW / 4)) * (e >> 2) .. ----------------
    const int quarter = warp & 3, grp = warp >> 2;
    constexpr int GCOLS = 128 / (EW / 4);                              // columns (= staging rows) of a group of four warps
    const int ch = 16 * quarter + (lane >> 1), par = lane & 1;          // this lane's channel and tap half
    const float bias = __ldg(epi.bias + ch);
    const int rr0 = lane >> 3, c16 = lane & 7;                          // second phase: row within a pass, 16-byte chunk
    bool dead = false;
    int local = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++local) {
      const int ab = local & 1;
      const uint32_t stg = stg0 + (local & 1) * STG_BYTES;
      // where the rows this lane writes in the second phase go: rows GCOLS grp + ROWS_PER_WARP quarter + 4 p + rr0
      uint32_t idx[ROWS_PER_WARP / 4];
      uint32_t valid = 0;
      {
        const int r_first = GCOLS * grp + ROWS_PER_WARP * quarter + rr0;
        int b, y, x;
        epi.map.split(t * ST_TILE + r_first, b, y, x);
        uint32_t at = epi.index(b, y, x, c16 * 8);
#pragma unroll
        for (int p = 0; p < ROWS_PER_WARP / 4; ++p) {
          idx[p] = at;
          if (r_first + 4 * p < ST_TILE && epi.map.is_output(b, y, x)) valid |= 1u << p;
          epi.map.template advance<Epi>(b, y, x, at, 4);
        }
      }
      if (!dead) {
        const bool ok = mbar_wait(&sh.empty[local % STAGES], (local / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
        if (!__all_sync(0xffffffffu, ok)) dead = true;
      }
      if (!dead) {
        tcgen05_fence_after();
#pragma unroll
        for (int cc = 0; cc < GCOLS / 32; ++cc) {
          const int c0 = GCOLS * grp + 32 * cc;
          uint32_t r[32], nxt;
          tmem_ld_32x32_next(tmem + ((uint32_t)(quarter * 32) << 16) + ab * ACC_COLS + c0, r, nxt, c0 + 32 < 128);
          if (cc == GCOLS / 32 - 1) {
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.full[(local + 2) % STAGES]);      // the accumulator is free for the tile after next
          }
          // even lane: out[2 i] = L[2 i] + H[2 i + 1];  odd lane: out[2 i + 1] = L[2 i + 1] + H[2 i + 2].
          // Staging row = position (128 bytes, channel-major); its 16-byte chunks are swizzled by 2 (pos & 3), so that
          // the two rows a store instruction touches use different banks; rows 2 i + par and 2 i + 4 + par share a swizzle,
          // which leaves two base addresses and compile-time offsets.
          const uint32_t row = (uint32_t)(c0 + par);
          const uint32_t sb0 = stg + row * 128u + ((((uint32_t)ch >> 3) ^ ((row & 3u) << 1)) << 4) + ((uint32_t)ch & 7u) * 2u;
          const uint32_t sb1 = stg + row * 128u + ((((uint32_t)ch >> 3) ^ (((row + 2u) & 3u) << 1)) << 4) + ((uint32_t)ch & 7u) * 2u;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float got = __shfl_xor_sync(0xffffffffu, __uint_as_float(r[2 * i + 1]), 1);
            const float mine = __uint_as_float(par ? (i < 15 ? r[2 * i + 2] : nxt) : r[2 * i]);
            const float v = (got + mine) + bias;
            uint16_t hv;
            asm("cvt.rn.relu.bf16.f32 %0, %1;" : "=h"(hv) : "f"(v));                  // bias, ReLU and the bf16 rounding
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(((i & 1) ? sb1 : sb0) + (uint32_t)(i * 256)), "h"(hv) : "memory");
          }
        }
      }
      group_barrier(1 + grp, 128);                                  // the GCOLS rows of this group are complete
      if (!dead) {
#pragma unroll
        for (int p = 0; p < ROWS_PER_WARP / 4; ++p) {
          const uint32_t rr = (uint32_t)(GCOLS * grp + ROWS_PER_WARP * quarter + 4 * p + rr0);
          const uint32_t off = rr * 128u + (((uint32_t)c16 ^ ((rr & 3u) << 1)) << 4);
          uint4 v;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stg + off) : "memory");
          if ((valid >> p) & 1u) *reinterpret_cast<uint4*>(epi.out + idx[p]) = v;
        }
      }
    }
  } else if (warp == 16 && lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, 128, 0, 0);
    const uint32_t hi = desc_hi_kmajor_sw128(), a_t = tmem + A_COL0;
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
      const int ab = it & 1, s = it % STAGES;
      ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!ok) break;
      fence_proxy_async_smem();        // the copies observed through the barrier -> visible to the MMA's operand reads
      tcgen05_fence_after();
      const uint32_t row0 = Cfg::BULK == 2 ? (uint32_t)((t * ST_TILE) % 10) : 0u;
      const uint32_t b_lo = (((a_base0 + s * STAGE_BYTES) >> 4) & 0x3FFFu) + row0 * 8u;
      const uint32_t d = tmem + ab * ACC_COLS;
#pragma unroll
      for (int j = 0; j < NS; ++j) {
        constexpr uint32_t K_STEP = 32 >> 4;
        const uint32_t b_off = (Cfg::tap_plane(Cfg::step_lo(j)) * PLANE_BYTES + Cfg::tap_shift(Cfg::step_lo(j)) * 128u) >> 4;
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k) {
          if (j == 0 && k == 0) mma_bf16_ts<false>(d, a_t, b_lo + b_off, hi, idesc);
          else mma_bf16_ts<true>(d, a_t + (j * 4 + k) * 8, b_lo + b_off + k * K_STEP, hi, idesc);
        }
      }
      mma_commit(&sh.empty[s]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 16) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// ---- plain split-k GEMM with both operands streamed (the fully connected layer, forward) ----------------
// C[m][n] = sum_k A[m][k] W[n][k] for A[M][K], W[N][K] row-major bf16.  Same persistent skeleton; a work item
// is (row tile, 128-column tile, k split), the stage holds the A and the W tile of one K block, and the
// epilogue stores float partial sums part[split][m][n].  fc_finish_kernel adds the splits in order, then
// bias, ReLU and the bf16 rounding.
constexpr int SK_BN = 128, SK_STAGES = 6, SK_LAG = 4;

__global__ void __launch_bounds__(PK_THREADS, 1)
tc_splitk_kernel(const bf16* __restrict__ a, const bf16* __restrict__ w, float* __restrict__ part, int M, int N, int K,
                 int tiles_m, int tiles_n, int splits, int kb_per, uint32_t* error_word) {
  constexpr uint32_t A_BYTES = TC_BM * 128, STAGE_BYTES = A_BYTES + SK_BN * 128;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ PkShared sh;
  const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total = tiles_m * tiles_n * splits, kb_total = K / TC_BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < SK_STAGES; ++s) { mbar_init(&sh.full[s], 4); mbar_init(&sh.empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&sh.acc_full[i], 1); mbar_init(&sh.acc_empty[i], 4); }
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(&sh.tmem_base, 2 * SK_BN);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp >= 4 && warp < 8) {
    // ---------------- producers: lane l copies chunk l & 7 of rows 32 pw + 4 p + (l >> 3) of both tiles ----------------
    const int pw = warp - 4, c = lane & 7, r4 = lane >> 3;
    int it = 0;
    bool alive = true;
    for (int t = blockIdx.x; t < total && alive; t += gridDim.x) {
      const int split = t % splits, nt = (t / splits) % tiles_n, mt = t / (splits * tiles_n);
      const int kb0 = split * kb_per, kb1 = min(kb_total, kb0 + kb_per);
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % SK_STAGES;
        const bool ok = mbar_wait(&sh.empty[s], ((it / SK_STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
        if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
        const uint32_t stage = base + s * STAGE_BYTES + (uint32_t)(32 * pw) * 128u;
#pragma unroll
        for (int p = 0; p < 8; ++p) {
          const uint32_t row = 4 * p + r4, off = row * 128u + ((uint32_t)(c ^ (row & 7)) << 4);
          const int m = min(mt * TC_BM + 32 * pw + (int)row, M - 1), n = nt * SK_BN + 32 * pw + (int)row;
          cp_async16(stage + off, a + (size_t)m * K + kb * TC_BK + c * 8, 16u);
          cp_async16(stage + A_BYTES + off, w + (size_t)n * K + kb * TC_BK + c * 8, 16u);
        }
        cp_async_commit();
        if (it >= SK_LAG) {
          cp_async_wait<SK_LAG>();
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.full[(it - SK_LAG) % SK_STAGES]);
        }
      }
    }
    cp_async_wait<0>();
    fence_proxy_async_smem();
    __syncwarp();
    if (alive && lane == 0)
      for (int j = it > SK_LAG ? it - SK_LAG : 0; j < it; ++j) mbar_arrive(&sh.full[j % SK_STAGES]);
  } else if (warp < 4) {
    // ---------------- epilogue ----------------
    int local = 0;
    for (int t = blockIdx.x; t < total; t += gridDim.x, ++local) {
      const int ab = local & 1, split = t % splits, nt = (t / splits) % tiles_n, mt = t / (splits * tiles_n);
      const int m = mt * TC_BM + threadIdx.x;
      const bool ok = mbar_wait(&sh.acc_full[ab], (local >> 1) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!__all_sync(0xffffffffu, ok)) break;
      tcgen05_fence_after();
#pragma unroll 1
      for (int cc = 0; cc < SK_BN / 32; ++cc) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + ab * SK_BN + cc * 32, r);
        if (m < M) {
          float4* dst = reinterpret_cast<float4*>(part + ((size_t)split * M + m) * N + nt * SK_BN + cc * 32);
#pragma unroll
          for (int q = 0; q < 8; ++q)
            dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]),
                                 __uint_as_float(r[4 * q + 3]));
        }
      }
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[ab]);
    }
  } else if (lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, SK_BN, 0, 0);
    int it = 0, local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total && ok; t += gridDim.x, ++local) {
      const int ab = local & 1, split = t % splits;
      const int kb0 = split * kb_per, kb1 = min(kb_total, kb0 + kb_per);
      ok = mbar_wait(&sh.acc_empty[ab], ((local >> 1) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!ok) break;
      tcgen05_fence_after();
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % SK_STAGES;
        ok = mbar_wait(&sh.full[s], (it / SK_STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_addr = base + s * STAGE_BYTES, b_addr = a_addr + A_BYTES;
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k)
          mma_bf16(tmem + ab * SK_BN, make_smem_desc(a_addr + k * 32, 0, 1024, SWIZZLE_128B),
                   make_smem_desc(b_addr + k * 32, 0, 1024, SWIZZLE_128B), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
        mma_commit(&sh.empty[s]);
      }
      if (ok) mma_commit(&sh.acc_full[ab]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 8) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 2 * SK_BN);
  }
}

// out[m][n..n+7] = bf16(relu(sum_s part[s][m][n] + bias[n]))
__global__ void __launch_bounds__(256) fc_finish_kernel(const float* __restrict__ part, int splits, int M, int N,
                                                        const float* __restrict__ bias, bf16* __restrict__ out) {
  pdl_entry();
  const size_t total = (size_t)M * N / 8;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const size_t e = i * 8;
    const int n = (int)(e % N);
    float v[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) v[q] = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float4* p = reinterpret_cast<const float4*>(part + (size_t)s * M * N + e);
      const float4 lo = __ldg(p), hi = __ldg(p + 1);
      v[0] += lo.x; v[1] += lo.y; v[2] += lo.z; v[3] += lo.w; v[4] += hi.x; v[5] += hi.y; v[6] += hi.z; v[7] += hi.w;
    }
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      o[q] = pack_bf16x2(fmaxf(v[2 * q] + __ldg(bias + n + 2 * q), 0.f), fmaxf(v[2 * q + 1] + __ldg(bias + n + 2 * q + 1), 0.f));
    *reinterpret_cast<uint4*>(out + e) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---- fully connected layer, forward, as one cluster per output tile --------------------------------------------
// h[m][n] = bf16(relu(sum_k A[m][k] W[n][k] + bias[n])) and the head dot products that follow it, in one launch.
// An output tile is 128 rows x 256 columns; the CTAs of a cluster (its size = the number of K slices, chosen on
// the host so that all clusters are resident at once) each multiply a slice of K into a tensor-memory accumulator,
// park it as floats in their own shared memory (on top of the operand stages, which are no longer needed), write
// it from there with whole-row accesses to their slice of part[split][m][n] and meet at a cluster barrier.  The
// slices are read back microseconds later, from L2.  (Reading the parked tiles of the other CTAs directly through
// distributed shared memory was measured two to three times slower than this round trip, in every access order
// tried.)  CTA r of the cluster then owns an equal share of the tile's rows: it adds the slices in split order (so
// the sum does not depend on timing), applies bias, ReLU and the bf16 rounding, stores h for the backward pass
// and, from the rounded values, its share of the A + 1 head dot products (256 of the 512 hidden units) as
// hp[column tile][m][k]; heads_sample_kernel adds the two shares.
// Warps 0-3 move the accumulator, one thread of warp 4 streams the operands (tiled bulk copies), lane 0 of warp 8
// issues the MMAs; all twelve warps share the finishing phase (warps 9-11 are there only for it: with two rows per
// warp a CTA's 21 or 22 rows then take one pass, and a pass costs a round trip to L2 however few rows it has).
constexpr int FCC_BN = 256, FCC_STAGES = 4, FCC_MAX_SPLITS = 8, FCC_THREADS = 384, FCC_HP_LD = 32;
constexpr int FCC_FIN_ROWS = 2 * (FCC_THREADS / 32);      // rows of the finishing phase per pass: 24 >= ceil(128 / 6)
constexpr uint32_t FCC_STAGE_BYTES = TC_BM * 128 + FCC_BN * 128, FCC_ACC_BYTES = TC_BM * FCC_BN * 4;
constexpr uint32_t FCC_HEADW_BYTES = 33 * FCC_BN * 2;
static_assert(FCC_ACC_BYTES <= FCC_STAGES * FCC_STAGE_BYTES, "the parked accumulator reuses the operand stages");

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// all threads of all CTAs of the cluster; release / acquire order the writes before it against the reads after it
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
struct FccShared {
  uint64_t full[FCC_STAGES], empty[FCC_STAGES], acc_full;
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__global__ void __launch_bounds__(FCC_THREADS, 1)
tc_fc_cluster_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                     const float* __restrict__ bias,
                     const bf16* __restrict__ wpi, const bf16* __restrict__ wv, int A, bf16* __restrict__ h_out,
                     float* part, float* __restrict__ hp, int M, int N, int K, int tiles_n, int splits,
                     uint32_t* error_word) {
  extern __shared__ uint8_t dyn_smem[];
  __shared__ FccShared sh;
  const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const uint32_t headw = base + FCC_STAGES * FCC_STAGE_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank(), tile = blockIdx.x / splits;
  const int nt = tile % tiles_n, mt = tile / tiles_n;
  const int kb_total = K / TC_BK, kb_base = kb_total / splits, kb_rem = kb_total % splits;
  const int kb0 = rank * kb_base + min(rank, kb_rem), kb1 = kb0 + kb_base + (rank < kb_rem ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < FCC_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.acc_full, 1);
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_w);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(&sh.tmem_base, FCC_BN);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp >= 4 && warp < 8) {
    // ---------------- producer: one thread asks the copy engine for the two boxes of each K block ----------------
    // (rows of A past M read as zeros)
    if (warp == 4 && lane == 0) {
      int it = 0;
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % FCC_STAGES;
        if (!mbar_wait(&sh.empty[s], ((it / FCC_STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY)) break;
        const uint32_t stage = base + s * FCC_STAGE_BYTES;
        mbar_arrive_expect_tx(&sh.full[s], FCC_STAGE_BYTES);
        tma_load_2d(stage, &tm_a, kb * TC_BK, mt * TC_BM, &sh.full[s]);
        tma_load_2d(stage + TC_BM * 128, &tm_w, kb * TC_BK, nt * FCC_BN, &sh.full[s]);
      }
    }
  } else if (warp == 8) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc = make_idesc_bf16(TC_BM, FCC_BN, 0, 0);
      int it = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1 && ok; ++kb, ++it) {
        const int s = it % FCC_STAGES;
        ok = mbar_wait(&sh.full[s], (it / FCC_STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_addr = base + s * FCC_STAGE_BYTES, b_addr = a_addr + TC_BM * 128;
#pragma unroll
        for (int k = 0; k < TC_BK / 16; ++k)
          mma_bf16(tmem, make_smem_desc(a_addr + k * 32, 0, 1024, SWIZZLE_128B),
                   make_smem_desc(b_addr + k * 32, 0, 1024, SWIZZLE_128B), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
        mma_commit(&sh.empty[s]);
      }
      if (ok) mma_commit(&sh.acc_full);
    }
  } else if (warp < 4) {
    // While the K slice is being multiplied these four warps have nothing to wait for yet: they bring in the head
    // weights of this column tile (row k = policy row k, k < A, 16-byte aligned, or the value row, k = A, which follows
    // the policy biases in the parameter vector and is only 2-byte aligned; 256 bf16 each).  The weights are several
    // kernels old; the block-wide barrier after the accumulator is parked makes them visible to the finishing phase.
    for (int i = threadIdx.x; i < A * (FCC_BN / 8); i += 128) {
      const int k = i / (FCC_BN / 8), c = i % (FCC_BN / 8);
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(wpi + (size_t)k * N + nt * FCC_BN) + c);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(headw + (uint32_t)(k * FCC_BN + 8 * c) * 2u),
                   "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
    }
    for (int c = threadIdx.x; c < FCC_BN / 2; c += 128) {
      const bf16* src = wv + nt * FCC_BN + 2 * c;
      const uint32_t v = (uint32_t)__bfloat16_as_ushort(src[0]) | ((uint32_t)__bfloat16_as_ushort(src[1]) << 16);
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(headw + (uint32_t)(A * FCC_BN + 2 * c) * 2u), "r"(v) : "memory");
    }
    // ---------------- accumulator -> this CTA's shared memory (float, 16-byte chunks swizzled by row) ----------------
    const bool ok = mbar_wait(&sh.acc_full, 0, &sh.abort, error_word, ERR_WAIT_ACC);
    if (__all_sync(0xffffffffu, ok)) {
      tcgen05_fence_after();
      const uint32_t row = (uint32_t)threadIdx.x, dst = base + row * (FCC_BN * 4u);
#pragma unroll 1
      for (int cc = 0; cc < FCC_BN / 32; ++cc) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + cc * 32, r);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((uint32_t)((cc * 8 + q) ^ (row & 7u)) << 4)),
                       "r"(r[4 * q]), "r"(r[4 * q + 1]), "r"(r[4 * q + 2]), "r"(r[4 * q + 3]) : "memory");
      }
      tcgen05_fence_before();
    }
  }
  // The parked tile goes to this split's slice of part[split][m][n] with whole-row accesses (a warp writes 512
  // contiguous bytes); the slices stay in L2 for the few microseconds until they are read back.
  __syncthreads();
  if (threadIdx.x < 256) {
#pragma unroll 4
    for (int i = 0; i < TC_BM * FCC_BN / 4 / 256; ++i) {
      const uint32_t q = (uint32_t)threadIdx.x + 256u * i, row = q >> 6, c = q & 63u;
      const int m = mt * TC_BM + (int)row;
      uint32_t r0, r1, r2, r3;
      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                   : "r"(base + row * (FCC_BN * 4u) + ((c ^ (row & 7u)) << 4)) : "memory");
      if (m < M)
        __stcg(reinterpret_cast<float4*>(part + ((size_t)rank * M + m) * N + nt * FCC_BN) + c,
               make_float4(__uint_as_float(r0), __uint_as_float(r1), __uint_as_float(r2), __uint_as_float(r3)));
    }
    __threadfence();
  }
  // Every CTA of the cluster reaches the barrier whatever happened above (a wait that gave up only raises the
  // error word; the numbers of that launch are then meaningless and the host reports the time-out).
  __syncwarp();
  cluster_sync_all();
  // ---------------- this CTA's share of the tile's rows: sum over the cluster, bias, ReLU, heads ----------------
  // rows [128 rank / splits, 128 (rank + 1) / splits), two per warp; thread (rl, cg) owns the 16-byte chunks
  // cg, cg + 16, cg + 32, cg + 48 of row rl, i.e. columns 4 (cg + 16 j) .. + 3: the sixteen threads of a row read
  // 256 contiguous bytes at a time
  const int row_lo = TC_BM * rank / splits, row_hi = TC_BM * (rank + 1) / splits;
  for (int row0 = row_lo + 2 * warp; row0 < row_hi; row0 += FCC_FIN_ROWS) {
    const int cg = lane & 15;
    const uint32_t row = (uint32_t)(row0 + (lane >> 4));
    const bool live = (int)row < row_hi;
    const int m = live ? mt * TC_BM + (int)row : M;
    float v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = 0.f;
    if (m < M) {
      const float4* src = reinterpret_cast<const float4*>(part + (size_t)m * N + nt * FCC_BN) + cg;
      // the first six slices are asked for in one go (24 loads in flight per thread: the phase is a chain of L2
      // latencies otherwise), a seventh and eighth, if any, after them; the additions keep the slice order
      {
        float4 t[6][4];
#pragma unroll
        for (int s = 0; s < 6; ++s)
#pragma unroll
          for (int j = 0; j < 4; ++j)
            t[s][j] = s < splits ? __ldcg(src + (size_t)s * M * (N / 4) + 16 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < 6; ++s)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            v[4 * j] += t[s][j].x; v[4 * j + 1] += t[s][j].y; v[4 * j + 2] += t[s][j].z; v[4 * j + 3] += t[s][j].w;
          }
      }
      if (splits > 6) {
        float4 t[2][4];
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
          for (int j = 0; j < 4; ++j)
            t[s][j] = 6 + s < splits ? __ldcg(src + (size_t)(6 + s) * M * (N / 4) + 16 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < 2; ++s)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            v[4 * j] += t[s][j].x; v[4 * j + 1] += t[s][j].y; v[4 * j + 2] += t[s][j].z; v[4 * j + 3] += t[s][j].w;
          }
      }
    }
    float x[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = nt * FCC_BN + 4 * (cg + 16 * j);
      const float4 b = __ldg(reinterpret_cast<const float4*>(bias + n));
      const bf16 h0 = __float2bfloat16_rn(fmaxf(v[4 * j] + b.x, 0.f)), h1 = __float2bfloat16_rn(fmaxf(v[4 * j + 1] + b.y, 0.f));
      const bf16 h2 = __float2bfloat16_rn(fmaxf(v[4 * j + 2] + b.z, 0.f)), h3 = __float2bfloat16_rn(fmaxf(v[4 * j + 3] + b.w, 0.f));
      x[4 * j] = __bfloat162float(h0); x[4 * j + 1] = __bfloat162float(h1);
      x[4 * j + 2] = __bfloat162float(h2); x[4 * j + 3] = __bfloat162float(h3);
      if (m < M)
        *reinterpret_cast<uint2*>(h_out + (size_t)m * N + n) =
            make_uint2((uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16),
                       (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16));
    }
    // head dot products over this thread's 16 hidden units: independent sums first, then a butterfly over the 16
    // threads of the row that halves the number of live values at each step and leaves thread cg with heads
    // 2 cg and 2 cg + 1 (the additions pair up in a fixed pattern)
    float pr[FCC_HP_LD];
#pragma unroll
    for (int k = 0; k < FCC_HP_LD; ++k) {
      pr[k] = 0.f;
      if (k <= A) {
        float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t w0, w1;
          asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w0), "=r"(w1)
                       : "r"(headw + (uint32_t)(k * FCC_BN + 4 * (cg + 16 * j)) * 2u) : "memory");
          acc0 = fmaf(__uint_as_float(w0 << 16), x[4 * j], acc0);
          acc1 = fmaf(__uint_as_float(w0 & 0xFFFF0000u), x[4 * j + 1], acc1);
          acc0 = fmaf(__uint_as_float(w1 << 16), x[4 * j + 2], acc0);
          acc1 = fmaf(__uint_as_float(w1 & 0xFFFF0000u), x[4 * j + 3], acc1);
        }
        pr[k] = acc0 + acc1;
      }
    }
#pragma unroll
    for (int o = 8, len = FCC_HP_LD / 2; o > 0; o >>= 1, len >>= 1) {
      const bool up = (cg & o) != 0;
#pragma unroll
      for (int i = 0; i < len; ++i) {
        const float send = up ? pr[i] : pr[i + len];
        const float keep = up ? pr[i + len] : pr[i];
        pr[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
      }
    }
    if (m < M) *reinterpret_cast<float2*>(hp + ((size_t)nt * M + m) * FCC_HP_LD + 2 * cg) = make_float2(pr[0], pr[1]);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 8) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, FCC_BN);
  }
}

static bool tc_fc_cluster_supported(int N, int K, int A) {
  return N % FCC_BN == 0 && K % TC_BK == 0 && K / TC_BK >= FCC_MAX_SPLITS && A + 1 <= FCC_HP_LD;
}

constexpr int FCC_SMEM = FCC_STAGES * FCC_STAGE_BYTES + FCC_HEADW_BYTES + 1024;
static_assert(FCC_SMEM <= 227 * 1024, "shared memory budget");

// The largest cluster size (= number of K slices) with which all `tiles` clusters are resident at once, so that
// the launch is one wave; how many clusters of a size fit depends on how the SMs are grouped on the part.
static int tc_fc_cluster_splits(int tiles) {
  static int max_active[FCC_MAX_SPLITS + 1] = {};          // 0 = not asked yet, -1 = the query failed
  for (int sp = FCC_MAX_SPLITS; sp >= 4; --sp) {
    if (max_active[sp] == 0) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(sp * 16); cfg.blockDim = dim3(FCC_THREADS); cfg.dynamicSmemBytes = FCC_SMEM;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = sp; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      max_active[sp] = cudaOccupancyMaxActiveClusters(&n, tc_fc_cluster_kernel, &cfg) == cudaSuccess && n > 0 ? n : -1;
    }
    if (max_active[sp] >= tiles) return sp;
  }
  return 4;
}

// false (nothing launched) if the tensor maps cannot be made; the caller then takes the split-k kernel
static bool tc_fc_forward_cluster(LaunchCtx& lc, const bf16* a, const bf16* w, const float* bias, const bf16* wpi,
                                  const bf16* wv, int A, bf16* h_out, float* part, float* hp, int M, int N, int K,
                                  uint32_t* err) {
  constexpr int smem = FCC_SMEM;
  const CUtensorMap* tm_a = tc_tensor_map(a, (uint64_t)M, (uint64_t)K, (uint64_t)K, TC_BM);
  const CUtensorMap* tm_w = tc_tensor_map(w, (uint64_t)N, (uint64_t)K, (uint64_t)K, FCC_BN);
  if (tm_a == nullptr || tm_w == nullptr) return false;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(tc_fc_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles_m = (M + TC_BM - 1) / TC_BM, tiles_n = N / FCC_BN;
  const int splits = tc_fc_cluster_splits(tiles_m * tiles_n);
  KernelScope scope(lc, KID_FC_FWD);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles_m * tiles_n * splits); cfg.blockDim = dim3(FCC_THREADS); cfg.dynamicSmemBytes = smem;
  cfg.stream = lc.st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = splits; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = (pdl_enabled() && !lc.serialize_next) ? 2 : 1;
  lc.serialize_next = false;
  cudaLaunchKernelEx(&cfg, tc_fc_cluster_kernel, *tm_a, *tm_w, bias, wpi, wv, A, h_out, part, hp, M, N, K, tiles_n, splits, err);
  return true;
}

// ---- first layer, forward: uint8 frames -> bf16 operand on the fly --------------------------------------
// Same persistent skeleton, with eight producer warps: the frame rows a tile needs are copied once into
// shared memory with cp.async (two tiles ahead); thread (row, half) then expands window rows
// 4*half .. 4*half+3 of its output pixel to bf16 into the two K blocks it owns.  Integers 0..255 are exact in bf16: the bytes are
// spliced into floats 2^23 + n, 2^23 is subtracted, and the upper halves of two results are packed.
// The forward kernel of the first layer multiplies in fp16 instead: a byte n placed in the low half of a 16-bit word
// IS the fp16 subnormal n * 2^-24, so the expansion is two byte permutations per four pixels and nothing else (the
// logic pipe that runs them was the kernel's bound with the ten instructions of the bf16 route).  Its weights are the
// bf16 weights times 2^8 as fp16 (exact down to 2^-25); the epilogue's scale carries the 2^16 / 255.
__device__ __forceinline__ void u8x4_to_f16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  lo = __byte_perm(w, 0u, 0x4140);
  hi = __byte_perm(w, 0u, 0x4342);
}
constexpr float C1_F16_WEIGHT_SCALE = 256.f, C1_F16_OUTPUT_SCALE = 16777216.f / C1_F16_WEIGHT_SCALE / 255.f;     // 2^24 / 2^8 / 255
// The weight-gradient kernel of the first layer plays the same trick in bf16, where it needs no second number format:
// a byte n in the low half of a 16-bit word is the bf16 value n * 2^-133 whether n < 128 (a subnormal) or not (exponent
// field 1, which has the same scale), and the tensor cores multiply these exactly (checked against exact products).
// Such operands times gradients of size 1e-6 would sink below what a float accumulator holds, so the data-gradient
// kernel of the layer above stores the gradient it hands down multiplied by 2^64 -- a shift of the exponent, exact
// before the bf16 rounding as after it -- and the finished sums are multiplied by 2^(133 - 64) / 255.
constexpr float C1_GRAD_SCALE = 18446744073709551616.f;                       // 2^64
constexpr float C1_WGRAD_OUTPUT_SCALE = 590295810358705651712.f / 255.f;      // 2^69 / 255
constexpr float C1_BIAS_OUTPUT_SCALE = 1.f / C1_GRAD_SCALE;
__device__ __forceinline__ void u8x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const float f0 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7440)) - 8388608.f;
  const float f1 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7441)) - 8388608.f;
  const float f2 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7442)) - 8388608.f;
  const float f3 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7443)) - 8388608.f;
  lo = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
  hi = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
}

// Space-to-depth view: with stride 4 and an 8 x 8 kernel, the window of output (oh, ow) is the 2 x 2 group of
// 4 x 4-pixel blocks (oh + i, ow + j), i, j in {0, 1}.  A block is 4 x 4 x 4 channels = 64 values = one 128-byte
// bf16 operand row, so the layer is a 2 x 2, stride-1 convolution over the 21 x 21 raster of blocks and runs
// as shifted views of one staged row block, like the other convolutions.  Every input byte is expanded to bf16
// once per tile instead of once per window that contains it.
//
// With only 32 output channels an MMA would be 32 columns wide, and a narrow MMA costs almost as much as a wide
// one (the 128 x 16 A slice is fetched either way).  So an accumulator row stands for TWO neighbouring raster
// positions 2 i and 2 i + 1 (columns 0-31 and 32-63): blocks at even positions are staged in plane E, blocks at
// odd positions in plane O, and with taps W00, W01, W10, W11 (block shifts 0, 1, 21, 22) the tile is the sum of
// six views, each multiplied by a 64-row weight matrix (left half | right half):
//   E+0: (W00 | 0)   O+0: (W01 | W00)   E+1: (0 | W01)   O+10: (W10 | 0)   E+11: (W11 | W10)   O+11: (0 | W11)
// The six matrices are windows of two block sequences [0, W01, W00, 0] and [0, W11, W10, 0] kept in shared memory.
//
// Roles: warps 0-7 epilogue (warp e: TMEM lane quarter e & 3, position parity e >> 2), warps 8-15 expand the raw
// bytes of a tile to bf16, warp 16 issues the MMAs, warp 17 fetches the frame rows a tile needs with one or two
// bulk copies (a tile's positions lie in at most two states, contiguous rows in each) into a ring of raw slots.
constexpr int C1_THREADS = 576;
constexpr int C1_RASTER = 21, C1_TILE_POS = 256, C1_USED_POS = 278;     // positions 2 i + 23, i <= 127
constexpr int C1_PLANE_ROWS = 144;                                      // >= 128 + 11, multiple of 8
constexpr int C1_RAW_BYTES = 20480;                                     // >= 15 block rows of 4 x 336 bytes
constexpr int C1_RAW_SLOTS = 3;

struct C1Shared {
  uint64_t full[4], empty[4], acc_full[2], acc_empty[2], raw_full[C1_RAW_SLOTS], raw_empty[C1_RAW_SLOTS];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

template <class G, class Epi, int STAGES>
__global__ void __launch_bounds__(C1_THREADS, 1)
tc_conv1_kernel(const uint8_t* __restrict__ frames, const bf16* __restrict__ w, Epi epi, int n_states, int tiles,
                uint32_t* error_word) {
  static_assert(G::K == 8 && G::S == 4 && G::C == 4 && G::CO == 32 && G::H == 84 && G::W == 84, "geometry");
  static_assert(STAGES >= 2 && STAGES <= 4, "pipeline depth");
  constexpr int BN = 64, NPROD = 256, POS = C1_RASTER * C1_RASTER, ROW_BYTES = G::W * G::C;
  constexpr uint32_t PLANE_BYTES = C1_PLANE_ROWS * 128, A_BYTES = 2 * PLANE_BYTES, W_BLOCK = 32 * 128, B_BYTES = 8 * W_BLOCK;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ C1Shared sh;
  const uint32_t b_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const uint32_t a_base0 = b_base + B_BYTES;
  const uint32_t raw_base = a_base0 + STAGES * A_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_pos = n_states * POS;

  if (threadIdx.x == 0) {
    // full[s]: the stage has been expanded AND the accumulator of the tile that will use the slot has been read out by
    // the epilogue of the tile two before it (the first two tiles find that arrival made here); empty[s]: the tile's
    // instructions have completed (producers may refill the slot, the epilogue may read).  One wait and one commit per
    // tile: a wait costs the issuing thread a couple of hundred cycles even when it is already satisfied.
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], NPROD / 32 + 8); mbar_init(&sh.empty[s], 1); }
    for (int s = 0; s < 2; ++s)
      for (int e = 0; e < 8; ++e) mbar_arrive(&sh.full[s]);
    for (int i = 0; i < C1_RAW_SLOTS; ++i) { mbar_init(&sh.raw_full[i], 1); mbar_init(&sh.raw_empty[i], NPROD / 32); }
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 16) tmem_alloc(&sh.tmem_base, 2 * BN);
  // weight blocks: sequence q (0: taps of block row 0, 1: block row 1) = [zeros, tap 2q+1, tap 2q, zeros]
  for (int i = threadIdx.x; i < 8 * 32 * 8; i += C1_THREADS) {
    const int c = i & 7, row = (i >> 3) & 31, blk = i >> 8, q = blk >> 2, k = blk & 3;
    const int tap = 2 * q + (k == 1 ? 1 : 0);
    cp_async16(b_base + blk * W_BLOCK + sw128_offset(row, c), w + ((size_t)row * 4 + tap) * TC_BK + c * 8,
               (k == 1 || k == 2) ? 16u : 0u);
  }
  cp_async_commit();
  cp_async_wait<0>();
  fence_proxy_async_smem();
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  // frame rows of tile t: raster positions qf .. ql, at most fifteen block rows in at most two states
  auto tile_ranges = [&](int t, int& b0, int& r0, int& n0, int& n1) {
    const int qf = t * C1_TILE_POS, ql = min(qf + C1_USED_POS - 1, total_pos - 1);
    b0 = qf / POS;
    const int b1 = ql / POS, yf = (qf % POS) / C1_RASTER, yl = (ql % POS) / C1_RASTER;
    r0 = 4 * yf;
    if (b1 == b0) { n0 = 4 * (yl - yf + 1); n1 = 0; }
    else { n0 = G::H - r0; n1 = 4 * (yl + 1); }
  };

  if (warp >= 8 && warp < 16) {
    // ---------------- producers: raw bytes -> bf16 operand rows ----------------
    const int p = threadIdx.x - 256;
    int local = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++local) {
      const int s = local % STAGES, slot = local % C1_RAW_SLOTS;
      int b0, r0, n0, n1;
      tile_ranges(t, b0, r0, n0, n1);
      const uint32_t stage = a_base0 + s * A_BYTES, raw = raw_base + slot * C1_RAW_BYTES;
      // work item = (position u of the tile, pixel row py of its block): 16 raw bytes -> two operand chunks;
      // thread p takes items p, p + 256, ...: the same py, positions 64 apart (3 block rows + 1 block).
      // Where the items sit in the raw slot is worked out before the waits, whose idle time hides the arithmetic.
      const int py = p & 3;
      int u = p >> 2, b, Y, X;
      {
        const int q = t * C1_TILE_POS + u;
        b = q / POS;
        const int rem = q - b * POS;
        Y = rem / C1_RASTER; X = rem - Y * C1_RASTER;
      }
      uint32_t src[5];
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        if (b >= n_states) { b = n_states - 1; Y = C1_RASTER - 1; X = C1_RASTER - 1; }     // past the end: repeat the last block
        const int slot_row = (b == b0 ? 4 * Y - r0 : n0 + 4 * Y) + py;
        src[k] = raw + (uint32_t)(slot_row * ROW_BYTES + X * 16);
        X += 1; Y += 3;
        if (X >= C1_RASTER) { X -= C1_RASTER; ++Y; }
        if (Y >= C1_RASTER) { Y -= C1_RASTER; ++b; }
      }
      bool ok = mbar_wait(&sh.raw_full[slot], (local / C1_RAW_SLOTS) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      ok = ok && mbar_wait(&sh.empty[s], ((local / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) break;
      uint4 rw[5];
#pragma unroll
      for (int k = 0; k < 5; ++k)
        if (u + 64 * k < C1_USED_POS)
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(rw[k].x), "=r"(rw[k].y), "=r"(rw[k].z), "=r"(rw[k].w)
                       : "r"(src[k]) : "memory");
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        const int uu = u + 64 * k;
        if (uu < C1_USED_POS) {
          uint32_t o[8];
          u8x4_to_f16x4(rw[k].x, o[0], o[1]); u8x4_to_f16x4(rw[k].y, o[2], o[3]);
          u8x4_to_f16x4(rw[k].z, o[4], o[5]); u8x4_to_f16x4(rw[k].w, o[6], o[7]);
          const uint32_t ri = (uint32_t)(uu >> 1), dst = stage + (uu & 1) * PLANE_BYTES + ri * 128u;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((uint32_t)((2 * py) ^ (ri & 7)) << 4)),
                       "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((uint32_t)((2 * py + 1) ^ (ri & 7)) << 4)),
                       "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&sh.full[s]); mbar_arrive(&sh.raw_empty[slot]); }
    }
  } else if (warp < 8) {
    // ---------------- epilogue ----------------
    // Two phases, so that a store instruction covers eight positions (64 bytes each) instead of thirty-two sixteen-
    // byte pieces of thirty-two different lines: lane = accumulator row turns its 32 channels into bf16 and parks them
    // in the warp's staging tile (32 rows of 64 bytes, chunks swizzled by row pair); then four lanes cover a row.
    // The load / store pipe, which the expansion shares, was what every role of this kernel was waiting for.
    const int quarter = warp & 3, h = warp >> 2;
    const uint32_t stg = raw_base + C1_RAW_SLOTS * C1_RAW_BYTES + warp * 2048;
    const int ch = lane & 3, rr0 = lane >> 2;
    const float4 bq0 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 0), bq1 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 1);
    const float4 bq2 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 2), bq3 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 3);
    const float4 bq4 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 4), bq5 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 5);
    const float4 bq6 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 6), bq7 = __ldg(reinterpret_cast<const float4*>(epi.bias) + 7);
    const float bias_r[32] = {bq0.x, bq0.y, bq0.z, bq0.w, bq1.x, bq1.y, bq1.z, bq1.w, bq2.x, bq2.y, bq2.z, bq2.w, bq3.x, bq3.y, bq3.z, bq3.w,
                              bq4.x, bq4.y, bq4.z, bq4.w, bq5.x, bq5.y, bq5.z, bq5.w, bq6.x, bq6.y, bq6.z, bq6.w, bq7.x, bq7.y, bq7.z, bq7.w};
    int local = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++local) {
      const int ab = local & 1;
      // where the four rows this lane writes in the second phase go (rows rr0, rr0 + 8, ...: positions 16 apart)
      uint32_t out_at[4];
      uint32_t valid = 0;
      {
        const int pos = t * C1_TILE_POS + 2 * (quarter * 32 + rr0) + h;
        int b = pos / POS;
        const int rem = pos - b * POS;
        int Y = rem / C1_RASTER, X = rem - Y * C1_RASTER;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          if (b < n_states && Y < G::OH && X < G::OW) valid |= 1u << p;
          out_at[p] = (uint32_t)(((b * G::OH + Y) * G::OW + X) * 32 + ch * 8);
          X += 16;
          if (X >= C1_RASTER) { X -= C1_RASTER; ++Y; }
          if (Y >= C1_RASTER) { Y -= C1_RASTER; ++b; }
        }
      }
      const bool ok = mbar_wait(&sh.empty[local % STAGES], (local / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!__all_sync(0xffffffffu, ok)) break;
      tcgen05_fence_after();
      uint32_t r[32];
      tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + ab * BN + h * 32, r);
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.full[(local + 2) % STAGES]);      // the accumulator is free for the tile after next
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a0 = fmaxf(fmaf(__uint_as_float(r[8 * q + 2 * j]), epi.scale, bias_r[8 * q + 2 * j]), 0.f);
          const float a1 = fmaxf(fmaf(__uint_as_float(r[8 * q + 2 * j + 1]), epi.scale, bias_r[8 * q + 2 * j + 1]), 0.f);
          o[j] = pack_bf16x2(a0, a1);
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 64 + ((uint32_t)(q ^ ((lane >> 1) & 3)) << 4)),
                     "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
      }
      __syncwarp();
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        const int rr = p * 8 + rr0;
        uint4 v;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(stg + rr * 64 + ((uint32_t)(ch ^ ((rr >> 1) & 3)) << 4)) : "memory");
        if ((valid >> p) & 1u) *reinterpret_cast<uint4*>(epi.out + out_at[p]) = v;
      }
      __syncwarp();                                              // staging tile free for the next tile
    }
  } else if (warp == 16) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc = make_idesc_f16(TC_BM, BN);        // fp16 operands (see u8x4_to_f16x4)
      constexpr uint32_t idesc32 = make_idesc_f16(TC_BM, 32);
      const uint32_t hi = desc_hi_kmajor_sw128(), b_lo = (b_base >> 4) & 0x3FFFu;
      int local = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++local) {
        const int ab = local & 1, s = local % STAGES;
        ok = mbar_wait(&sh.full[s], (local / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t a_lo = ((a_base0 + s * A_BYTES) >> 4) & 0x3FFFu, d = tmem + ab * BN;
#pragma unroll
        for (int i = 0; i < 6; ++i) {
          // view v: plane (E = 0, O = 1), rows down, and what it is multiplied with.  The two views that feed both
          // positions of a row take a 64-row window of a block sequence (first block given); the four that feed one
          // position take the 32 rows of their tap alone and go to that position's half of the accumulator: a 32-column
          // MMA fetches a kilobyte less than a 64-column one whose other half is zeros.  A 64-column view comes
          // first, so that it can initialise the whole accumulator.
          constexpr int order[6] = {1, 0, 2, 3, 4, 5};
          constexpr int plane[6] = {0, 1, 0, 1, 0, 1}, shift[6] = {0, 0, 1, 10, 11, 11};
          constexpr int wblk[6] = {2, 1, 1, 6, 5, 5}, dcol[6] = {0, 0, 32, 0, 0, 32};
          constexpr bool wide[6] = {false, true, false, false, true, false};
          const int v = order[i];
          const uint32_t a_off = (plane[v] * PLANE_BYTES + shift[v] * 128u) >> 4, b_off = (wblk[v] * W_BLOCK) >> 4;
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k) {
            if (i == 0 && k == 0) mma_bf16_lo<false>(d, a_lo + a_off, b_lo + b_off, hi, idesc);
            else mma_bf16_lo<true>(d + dcol[v], a_lo + a_off + k * 2, b_lo + b_off + k * 2, hi, wide[v] ? idesc : idesc32);
          }
        }
        mma_commit(&sh.empty[s]);
      }
    }
  } else if (lane == 0) {
    // ---------------- raw loader ----------------
    int local = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++local) {
      const int slot = local % C1_RAW_SLOTS;
      if (!mbar_wait(&sh.raw_empty[slot], ((local / C1_RAW_SLOTS) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY)) break;
      int b0, r0, n0, n1;
      tile_ranges(t, b0, r0, n0, n1);
      const uint32_t dst = raw_base + slot * C1_RAW_BYTES;
      mbar_arrive_expect_tx(&sh.raw_full[slot], (uint32_t)((n0 + n1) * ROW_BYTES));
      bulk_copy_g2s(dst, frames + ((size_t)b0 * G::H + r0) * ROW_BYTES, (uint32_t)(n0 * ROW_BYTES), &sh.raw_full[slot]);
      if (n1 > 0)
        bulk_copy_g2s(dst + n0 * ROW_BYTES, frames + (size_t)(b0 + 1) * G::H * ROW_BYTES, (uint32_t)(n1 * ROW_BYTES),
                      &sh.raw_full[slot]);
    }
  }
  // Every issued bulk copy has been waited for by the producers (or the CTA is aborting after a bounded wait gave
  // up, in which case the copies in flight still land in this CTA's shared memory before it retires).
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 16) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 2 * BN);
  }
}

static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

template <class ASrc, class Epi, int BN, int KB, int NCLS, int STAGES, int KPS>
static void tc_persistent(LaunchCtx& lc, int kid, ASrc a, const bf16* w, int n_total, Epi e, int M, uint32_t* err) {
  const CUtensorMap* tm_a = tc_tensor_map(a.x, (uint64_t)a.M, (uint64_t)KB * TC_BK, (uint64_t)a.ld, TC_BM);
  if (tm_a == nullptr) { lc.host_failure = true; return; }      // no tensor-map encoder: the API call reports PAAC_ERR_CUDA
  constexpr int smem = NCLS * KB * BN * 128 + STAGES * KPS * TC_BM * 128 + 4 * 32 * BN * 2 + 1024;      // weights, stages, staging tiles
  static_assert(smem <= 227 * 1024, "shared memory budget");
  auto kern = tc_persistent_kernel<ASrc, Epi, BN, KB, NCLS, STAGES, KPS>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles_m = (M + TC_BM - 1) / TC_BM, gy = (n_total + BN - 1) / BN;
  int gx = sm_count() / gy;
  if (gx < 1) gx = 1;
  if (gx > NCLS * tiles_m) gx = NCLS * tiles_m;
  KernelScope scope(lc, kid);
  launch_kernel_overlapped(lc, kern, dim3(gx, gy), PK_THREADS, smem, *tm_a, w, n_total, e, tiles_m, err);
}

template <class Cfg, class Epi, int BN, int STAGES, int NACC>
static void tc_shift(LaunchCtx& lc, int kid, Cfg cfg, const bf16* w, Epi e, int positions, uint32_t* err) {
  constexpr int smem = Cfg::NT * BN * 128 + STAGES * Cfg::PLANES * Cfg::STAGE_ROWS * 128 + 8 * 32 * BN +
                       (Epi::MASK ? 2 * 8 * 32 * BN : 0) + 1024;        // weights, stages, staging tiles, activation rings
  static_assert(smem <= 227 * 1024, "shared memory budget");
  auto kern = tc_shift_kernel<Cfg, Epi, BN, STAGES, NACC>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles = (positions + TC_BM - 1) / TC_BM;
  // bulk-copied stages: the layer input as a matrix of 128-byte rows, fetched in boxes of one stage
  static CUtensorMap no_map;
  const CUtensorMap* tm_a = &no_map;
  const CUtensorMap* tm_b = &no_map;
  if constexpr (Cfg::BULK == 1) {
    tm_a = tc_tensor_map(cfg.base_host(), (uint64_t)cfg.row_count(), 64, 64, Cfg::STAGE_ROWS);
  } else if constexpr (Cfg::BULK == 2) {
    // plane p: [states * 10][10 pairs][64], 2560 bytes from one oh to the next, starting 10 p pair rows in
    tm_a = tc_tensor_map3(cfg.base_host(), 10, (uint64_t)cfg.states * 10, 128, 2560, 10, Cfg::STAGE_ROWS / 10);
    tm_b = tc_tensor_map3(cfg.base_host() + 10 * 64, 10, (uint64_t)cfg.states * 10, 128, 2560, 10, Cfg::STAGE_ROWS / 10);
  }
  if (tm_a == nullptr || tm_b == nullptr) { lc.host_failure = true; return; }      // no tensor-map encoder
  KernelScope scope(lc, kid);
  launch_kernel_overlapped(lc, kern, tiles < sm_count() ? tiles : sm_count(), SH_THREADS, smem, *tm_a, *tm_b, cfg, w, e, tiles, err);
}

template <class Cfg, class Epi, int STAGES>
static void tc_shift_t(LaunchCtx& lc, int kid, Cfg cfg, const bf16* w, Epi e, int positions, uint32_t* err) {
  constexpr int smem = STAGES * Cfg::PLANES * Cfg::STAGE_ROWS * 128 + 2 * 128 * 128 + 1024;
  static_assert(smem <= 227 * 1024, "shared memory budget");
  static_assert(smem - 1024 >= Cfg::NSTEP * 128 * 128, "the weights pass through the stage area on their way to tensor memory");
  auto kern = tc_shift_t_kernel<Cfg, Epi, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles = (positions + ST_TILE - 1) / ST_TILE;
  static CUtensorMap no_map;
  const CUtensorMap* tm_a = &no_map;
  const CUtensorMap* tm_b = &no_map;
  if constexpr (Cfg::BULK == 1) {
    tm_a = tc_tensor_map(cfg.base_host(), (uint64_t)cfg.row_count(), 64, 64, Cfg::STAGE_ROWS);
  } else if constexpr (Cfg::BULK == 2) {
    tm_a = tc_tensor_map3(cfg.base_host(), 10, (uint64_t)cfg.states * 10, 128, 2560, 10, Cfg::STAGE_ROWS / 10);
    tm_b = tc_tensor_map3(cfg.base_host() + 10 * 64, 10, (uint64_t)cfg.states * 10, 128, 2560, 10, Cfg::STAGE_ROWS / 10);
  }
  if (tm_a == nullptr || tm_b == nullptr) { lc.host_failure = true; return; }      // no tensor-map encoder
  KernelScope scope(lc, kid);
  launch_kernel_overlapped(lc, kern, tiles < sm_count() ? tiles : sm_count(), ST_THREADS, smem, *tm_a, *tm_b, cfg, w, e, tiles, err);
}

template <class G, class Epi>
static void tc_conv1(LaunchCtx& lc, const uint8_t* frames, const bf16* w_blocks, Epi e, int n_states, uint32_t* err) {
  constexpr int STAGES = 3;
  constexpr int smem = 8 * 32 * 128 + STAGES * 2 * C1_PLANE_ROWS * 128 + C1_RAW_SLOTS * C1_RAW_BYTES + 8 * 2048 + 1024;   // + staging tiles
  static_assert(smem <= 227 * 1024, "shared memory budget");
  auto kern = tc_conv1_kernel<G, Epi, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles = (n_states * C1_RASTER * C1_RASTER + C1_TILE_POS - 1) / C1_TILE_POS;
  const int gx = tiles < sm_count() ? tiles : sm_count();
  KernelScope scope(lc, KID_CONV1_FWD);
  launch_kernel_overlapped(lc, kern, gx, C1_THREADS, smem, frames, w_blocks, e, n_states, tiles, err);
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
  launch_kernel_overlapped(lc, kern, grid, TC_THREADS, smem, a, b, e, num_kb, error_word);
}

constexpr int FC_SPLITS = 7;
size_t tc_fc_scratch_floats(int n) { return (size_t)FCC_MAX_SPLITS * n * 512 + (size_t)2 * n * FCC_HP_LD; }

static void tc_fc_forward(LaunchCtx& lc, const bf16* a, const bf16* w, const float* bias, bf16* out, int M, int N, int K,
                          float* part, uint32_t* err, int* splits_out) {
  constexpr int smem = SK_STAGES * (TC_BM * 128 + SK_BN * 128) + 1024;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(tc_splitk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles_m = (M + TC_BM - 1) / TC_BM, tiles_n = N / SK_BN, kb_total = K / TC_BK;
  const int kb_per = (kb_total + FC_SPLITS - 1) / FC_SPLITS, splits = (kb_total + kb_per - 1) / kb_per;
  const int total = tiles_m * tiles_n * splits;
  {
    KernelScope scope(lc, KID_FC_FWD);
    launch_kernel_overlapped(lc, tc_splitk_kernel, total < sm_count() ? total : sm_count(), PK_THREADS, smem, a, w, part, M, N, K, tiles_m,
                                                                                         tiles_n, splits, kb_per, err);
  }
  if (splits_out) { *splits_out = splits; return; }      // the caller's next kernel adds the partial sums up
  KernelScope scope(lc, KID_FC_FWD);
  const int blocks = (M * N / 8 + 255) / 256;
  launch_kernel(lc, fc_finish_kernel, blocks < 1184 ? blocks : 1184, 256, 0, part, splits, M, N, bias, out);
}

// ---- forward ---------------------------------------------------------------------------------------------
bool tc_supported(int arch, int prec) { return arch == PAAC_ARCH_NATURE && prec == PAAC_BF16; }

void tc_forward(LaunchCtx& lc, int arch, const NetDims& nd, const float* theta, const bf16* w, const bf16* images,
                const uint8_t* frames, int n, void* const act[], float* fc_scratch, uint32_t* err, int* fc_splits) {
  const LayerDims* d = nd.layer;
  if (arch != PAAC_ARCH_NATURE) return;   // the caller routes the smaller network to the CUDA-core path
  {
    typedef NatConv1 C1; typedef NatConv2 C2; typedef NatConv3 C3;
    const int M1 = n * C1::OH * C1::OW, M2 = n * C2::OH * C2::OW, M3 = n * C3::OH * C3::OW;
    tc_conv1<C1, BiasReluEpiTc>(lc, frames, images + TC_IMG_W1, BiasReluEpiTc{(bf16*)act[0], theta + d[0].b_off, 32, C1_F16_OUTPUT_SCALE, M1},
                                n, err);
    {
      typedef RasterMap<100, 10, 9, 9> Map;
      tc_shift_t<C2FwdCfg, ShiftBiasReluEpi<Map, 9, 9>, 4>(
          lc, KID_CONV2_FWD, C2FwdCfg{(const bf16*)act[0], n}, w + d[1].w_off,
          ShiftBiasReluEpi<Map, 9, 9>{Map{n}, (bf16*)act[1], theta + d[1].b_off, nullptr}, n * 100, err);
    }
    {
      typedef RasterMap<81, 9, 7, 7> Map;
      tc_shift_t<C3FwdCfg, ShiftBiasReluEpi<Map, 7, 7>, 6>(
          lc, KID_CONV3_FWD, C3FwdCfg{(const bf16*)act[1], n * 81}, w + d[2].w_off,
          ShiftBiasReluEpi<Map, 7, 7>{Map{n}, (bf16*)act[2], theta + d[2].b_off, nullptr}, n * 81, err);
    }
    (void)M2; (void)M3;
    if (fc_splits != nullptr && tc_fc_cluster_supported(512, 3136, nd.A) &&
        tc_fc_forward_cluster(lc, (const bf16*)act[2], w + d[3].w_off, theta + d[3].b_off, w + nd.pi_w, w + nd.v_w, nd.A,
                              (bf16*)act[3], fc_scratch + (size_t)2 * n * FCC_HP_LD, fc_scratch, n, 512, 3136, err)) {
      // cluster path: h is complete and fc_scratch holds the head dot products as hp[2][n][32] (*fc_splits = 0)
      *fc_splits = 0;
    } else {
      tc_fc_forward(lc, (const bf16*)act[2], w + d[3].w_off, theta + d[3].b_off, (bf16*)act[3], n, 512, 3136, fc_scratch, err,
                    fc_splits);
    }
  }
}

// ---- weight gradients ------------------------------------------------------------------------------------
// dW^T[j][co] = sum_m X[m][j] * G[m][co]: the reduction runs over the rows m = (state, oh, ow), so both
// operands are "MN-major": a shared-memory row holds 64 consecutive j (or co) of ONE m, exactly the 128
// bytes the forward sources deliver (an atom = K block of the forward pass).  Image of one stage (64 rows
// of m): atom column a -> 8 groups of 8 rows -> 128-byte swizzled rows; leading (atom-column) stride 8 KB,
// stride between 8-row groups 1 KB; a K=16 MMA step covers two groups.
// A CTA owns JT row tiles of 128 j each and a contiguous range of 64-row blocks of m (split-k); it writes
// its float partial tile to scratch, and a second kernel adds the partials in a fixed order.
constexpr int WG_ROWS = 64, WG_LAG = 3;

// G rows: BN (64 or 128) bf16 starting at column n0; rows past M read as zero so that the tail of the last
// block adds nothing.  VALID < 64 pads a narrower matrix (conv1: 32 channels) with zero columns.
template <int VALID> struct GradSrc {
  const bf16* g; int ld; int M;
  __device__ __forceinline__ const bf16* ptr(int m, int n0, bool& valid) const {
    valid = m < M;
    return valid ? g + (size_t)m * ld + n0 : g;
  }
  __device__ __forceinline__ void load(int m, int n0, uint4 (&v)[8]) const {
    if (m >= M) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
      return;
    }
    const uint4* p = reinterpret_cast<const uint4*>(g + (size_t)m * ld + n0);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = i < VALID / 8 ? __ldg(p + i) : make_uint4(0u, 0u, 0u, 0u);
  }
};

template <class XSrc, class GSrc, int VALID_N, int JT, int BN, int STAGES>
__global__ void __launch_bounds__(TC_THREADS)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_g, XSrc x_src, GSrc g_src,
                float* __restrict__ partial, float* __restrict__ bias_partial, int n_atoms, int J, int CO, int num_blocks,
                int blocks_per_split, uint32_t* error_word) {
  // plain row-major matrices: one thread fetches a stage as 64 x 64 boxes (rows and columns outside read as zeros)
  constexpr bool TMA = XSrc::ASYNC && VALID_N == 64;
  static_assert(BN == 64 || BN == 128, "tile width");
  static_assert(JT == 1 || JT == 2, "row tiles per CTA");
  constexpr uint32_t ATOM_COL = WG_ROWS * 128;                      // 8 KB: one atom column of a stage
  constexpr uint32_t A_BYTES = 2 * JT * ATOM_COL, B_BYTES = (BN / 64) * ATOM_COL, STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int A_PER_HALF = JT, B_COLS = BN / 64;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ TcShared sh;
  const uint32_t tiles = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, atom0 = blockIdx.y * 2 * JT, n0 = blockIdx.z * BN;
  const int kb0 = split * blocks_per_split, kb1 = min(num_blocks, kb0 + blocks_per_split);
  // The bias gradient sum_m G[m][co] rides along as one more row tile whose operand is constant: row j = 0
  // is all ones, the other rows zero.  Only the CTAs of the first row-tile group compute it.
  constexpr uint32_t TMEM_COLS = (JT + 1) * BN <= 128 ? 128 : ((JT + 1) * BN <= 256 ? 256 : 512);
  const bool do_bias = blockIdx.y == 0;
  const uint32_t ones_base = tiles + STAGES * STAGE_BYTES;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], TMA ? 1 : 4); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.acc, 1);
    if (TMA) { tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_g); }
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(&sh.tmem_base, TMEM_COLS);
  if (do_bias) {
    for (uint32_t i = threadIdx.x; i < 2 * ATOM_COL / 16; i += TC_THREADS) {
      // 16-byte chunk i of the image: element j = 0 of k-row (i / 8) sits in physical chunk (row & 7) of atom column 0
      const uint32_t krow = i >> 3, chunk = i & 7;
      const uint32_t one = (i < ATOM_COL / 16 && chunk == (krow & 7)) ? 0x3F80u : 0u;
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %2, %2};" ::"r"(ones_base + i * 16), "r"(one), "r"(0u) : "memory");
    }
    fence_proxy_async_smem();
  }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp < 4) {
    // ---------------- producers: thread = (row of the block, half) ----------------
    const int row = threadIdx.x & 63, half = threadIdx.x >> 6;
    const uint32_t row_off = (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u;
    for (int kb = kb0; kb < kb1; ++kb) {
      const int it = kb - kb0, s = it % STAGES;
      const bool ok = mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t a_base = tiles + s * STAGE_BYTES, b_base = a_base + A_BYTES;
      const int m = kb * WG_ROWS + row;
      if constexpr (TMA) {
        if (threadIdx.x == 0) {
          mbar_arrive_expect_tx(&sh.full[s], STAGE_BYTES);
#pragma unroll
          for (int col = 0; col < 2 * JT; ++col)
            tma_load_2d(a_base + col * ATOM_COL, &tm_x, (atom0 + col) * 64, kb * WG_ROWS, &sh.full[s]);
#pragma unroll
          for (int gc = 0; gc < B_COLS; ++gc)
            tma_load_2d(b_base + gc * ATOM_COL, &tm_g, n0 + gc * 64, kb * WG_ROWS, &sh.full[s]);
        }
      } else {
        uint4 v[8];
#pragma unroll
        for (int q = 0; q < A_PER_HALF; ++q) {
          const int col = half * A_PER_HALF + q;                      // atom column inside the stage
          const int atom = atom0 + col;
          if (atom < n_atoms) x_src.load(m, atom, 0, v);
          else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
          }
#pragma unroll
          for (int c = 0; c < 8; ++c)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_base + col * ATOM_COL + row_off +
                         ((uint32_t)(c ^ (row & 7)) << 4)), "r"(v[c].x), "r"(v[c].y), "r"(v[c].z), "r"(v[c].w) : "memory");
        }
        if (half < B_COLS) {
          g_src.load(m, n0 + half * 64, v);
#pragma unroll
          for (int c = 0; c < 8; ++c)
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(b_base + half * ATOM_COL + row_off +
                         ((uint32_t)(c ^ (row & 7)) << 4)), "r"(v[c].x), "r"(v[c].y), "r"(v[c].z), "r"(v[c].w) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.full[s]);
      }
    }
    // ---------------- epilogue: float partial tile to scratch ----------------
    if (kb1 > kb0 && mbar_wait(&sh.acc, 0, &sh.abort, error_word, ERR_WAIT_ACC)) {
      tcgen05_fence_after();
#pragma unroll 1
      for (int jt = 0; jt < JT; ++jt) {
        const int j = (atom0 / 2 + jt) * 128 + threadIdx.x;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + jt * BN + c * 32, r);
          if (n0 + c * 32 < CO) {
            const int j0 = j - lane;                              // this warp's rows j0 .. j0 + 31
            const uint32_t rows = j0 + 32 <= J ? 0xFFFFFFFFu : (j0 < J ? (1u << (J - j0)) - 1u : 0u);
            // the operand stages are idle by now (every MMA has completed): their memory serves as staging tiles
            warp_store_rows_f32(tiles + warp * 4096, lane, r, partial + ((size_t)split * J + j0) * CO + n0 + c * 32, CO, rows);
          }
        }
      }
      if (do_bias && warp == 0) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(tmem + JT * BN + c * 32, r);
          if (lane == 0 && n0 + c * 32 < CO) {
#pragma unroll
            for (int q = 0; q < 32; ++q) bias_partial[(size_t)split * CO + n0 + c * 32 + q] = __uint_as_float(r[q]);
          }
        }
      }
    }
  } else if (lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_bf16(TC_BM, BN, 1, 1);
    bool ok = true;
    for (int kb = kb0; kb < kb1 && ok; ++kb) {
      const int it = kb - kb0, s = it % STAGES;
      ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t a_base = tiles + s * STAGE_BYTES, b_base = a_base + A_BYTES;
#pragma unroll
      for (int jt = 0; jt < JT; ++jt) {
#pragma unroll
        for (int t = 0; t < WG_ROWS / 16; ++t) {
          const uint64_t ad = make_smem_desc(a_base + jt * 2 * ATOM_COL + t * 2048, ATOM_COL, 1024, SWIZZLE_128B);
          const uint64_t bd = make_smem_desc(b_base + t * 2048, ATOM_COL, 1024, SWIZZLE_128B);
          mma_bf16(tmem + jt * BN, ad, bd, idesc, (it | t) != 0 ? 1u : 0u);
        }
      }
      if (do_bias) {
#pragma unroll
        for (int t = 0; t < WG_ROWS / 16; ++t) {
          const uint64_t ad = make_smem_desc(ones_base + t * 2048, ATOM_COL, 1024, SWIZZLE_128B);
          const uint64_t bd = make_smem_desc(b_base + t * 2048, ATOM_COL, 1024, SWIZZLE_128B);
          mma_bf16(tmem + JT * BN, ad, bd, idesc, (it | t) != 0 ? 1u : 0u);
        }
      }
      mma_commit(&sh.empty[s]);
    }
    if (ok && kb1 > kb0) mma_commit(&sh.acc);
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 4) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// dW[co][j] = scale * sum over splits of partial[split][j][co].  A block owns 32 consecutive outputs;
// its 8 thread rows each add every 8th split, then the 8 sums are added in a fixed order.
__global__ void __launch_bounds__(256) tc_wgrad_reduce_kernel(const float* __restrict__ partial, int splits, int J, int CO,
                                                              float scale, float* __restrict__ gw) {
  pdl_entry();
  __shared__ float sh[8][33];
  const int total = J * CO, lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  const int i = blockIdx.x * 32 + lane;
  float s = 0.f;
  if (i < total)
    for (int p = part; p < splits; p += 8) s += partial[(size_t)p * total + i];
  sh[part][lane] = s;
  __syncthreads();
  if (part == 0 && i < total) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) t += sh[q][lane];
    const int j = i / CO, co = i % CO;
    gw[(size_t)co * J + j] = t * scale;
  }
}

// bias gradient: the per-split column sums written by the weight-gradient kernel, added in split order
__global__ void tc_bias_final_kernel(const float* __restrict__ part, int blocks, int CO, float* __restrict__ gb) {
  pdl_entry();
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= CO) return;
  float s = 0.f;
  for (int b = 0; b < blocks; ++b) s += part[(size_t)b * CO + c];
  gb[c] = s;
}

// One launch finishes every tensor-core weight gradient of an update: for each segment (a layer's weights, or
// its bias with J = 1) dst[co * J + j] = scale * sum over splits of part[split][j][co], the splits added in a
// fixed order.  The partial sums have co innermost and the gradient has j innermost, so every group of outputs
// goes through a shared-memory tile: reads are whole 128-byte rows of co, writes whole runs of j.
//   many splits: a group is FG_J j x 32 co; warp w adds the splits w, w + 8, ... for these j, the eight warps' sums
//                are then added in warp order;
//   few splits:  a group is 32 j x 32 co; warp w adds all splits, in order, for rows w, w + 8, w + 16, w + 24.
constexpr int FG_J = 2;          // rows of j per group of a many-split segment
__global__ void __launch_bounds__(256) tc_finalize_grads_kernel(GradSegments segs, float* __restrict__ sumsq_partials) {
  pdl_entry();
  __shared__ float sh[8 * 8 * 33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float ss = 0.f;                       // sum of squares of the gradient values this thread writes
  for (int grp = blockIdx.x; grp < segs.total_groups; grp += gridDim.x) {
    int si = 0;
    while (si + 1 < segs.n && grp >= segs.seg[si + 1].first_group) ++si;
    const GradSegment& sg = segs.seg[si];
    const int local = grp - sg.first_group, co_tiles = (sg.CO + 31) / 32;
    const int co0 = (local % co_tiles) * 32, J = sg.J, CO = sg.CO;
    const size_t total = (size_t)J * CO;
    const bool co_ok = co0 + lane < CO;
    if (sg.wide) {
      // a group is FG_J j x 32 co: small, so that the many-split layers spread over all blocks of the grid; warp w
      // adds the splits w, w + 8, ... with 32 loads in flight per thread (its latency, not the bandwidth, sets the
      // pace of a group); the additions keep their order
      constexpr int SPI = 32 / FG_J;                      // splits per iteration and warp
      const int j0 = (local / co_tiles) * FG_J;
      float acc[FG_J];
#pragma unroll
      for (int q = 0; q < FG_J; ++q) acc[q] = 0.f;
      const float* src = sg.part + (size_t)j0 * CO + co0 + lane;
      for (int p = warp; p < sg.splits; p += 8 * SPI) {
        float v[SPI][FG_J];
#pragma unroll
        for (int u = 0; u < SPI; ++u)
#pragma unroll
          for (int q = 0; q < FG_J; ++q)
            v[u][q] = (co_ok && j0 + q < J && p + 8 * u < sg.splits) ? __ldg(src + (size_t)(p + 8 * u) * total + (size_t)q * CO) : 0.f;
#pragma unroll
        for (int u = 0; u < SPI; ++u)
          if (p + 8 * u < sg.splits) {
#pragma unroll
            for (int q = 0; q < FG_J; ++q) acc[q] += v[u][q];
          }
      }
#pragma unroll
      for (int q = 0; q < FG_J; ++q) sh[(warp * FG_J + q) * 33 + lane] = acc[q];
      __syncthreads();
      if (threadIdx.x < 32 * FG_J) {
        const int c = threadIdx.x / FG_J, q = threadIdx.x % FG_J;   // consecutive threads write consecutive j
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += sh[(w * FG_J + q) * 33 + c];
        if (co0 + c < CO && j0 + q < J) { const float v = t * sg.scale; sg.dst[(size_t)(co0 + c) * J + j0 + q] = v; ss = fmaf(v, v, ss); }
      }
      __syncthreads();
    } else {
      const int j0 = (local / co_tiles) * 32;
      float t[4] = {0.f, 0.f, 0.f, 0.f};
      const float* src = sg.part + (size_t)(j0 + warp) * CO + co0 + lane;
      bool ok[4];
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) ok[rr] = co_ok && j0 + warp + 8 * rr < J;
#pragma unroll 4
      for (int p = 0; p < sg.splits; ++p) {
        float v[4];
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) v[rr] = ok[rr] ? __ldg(src + (size_t)p * total + (size_t)(8 * rr) * CO) : 0.f;
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) t[rr] += v[rr];
      }
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) sh[(warp + 8 * rr) * 33 + lane] = t[rr];
      __syncthreads();
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const int c = warp + 8 * rr;
        if (co0 + c < CO && j0 + lane < J) { const float v = sh[lane * 33 + c] * sg.scale; sg.dst[(size_t)(co0 + c) * J + j0 + lane] = v; ss = fmaf(v, v, ss); }
      }
      __syncthreads();
    }
  }
  // this block's share of the squared gradient norm (the optimiser adds the blocks' shares in block order)
  if (sumsq_partials != nullptr) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (lane == 0) sh[warp] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += sh[w];
      sumsq_partials[blockIdx.x] = t;
    }
  }
}

static bool add_segment(GradSegments* segs, const float* part, float* dst, int splits, int J, int CO, float scale) {
  if (segs->n >= (int)(sizeof(segs->seg) / sizeof(segs->seg[0]))) return false;      // the caller reports a host failure
  GradSegment& g = segs->seg[segs->n++];
  g.part = part; g.dst = dst; g.splits = splits; g.J = J; g.CO = CO; g.scale = scale;
  g.wide = splits > 8;
  g.first_group = segs->total_groups;
  g.groups = ((J + (g.wide ? FG_J : 32) - 1) / (g.wide ? FG_J : 32)) * ((CO + 31) / 32);
  segs->total_groups += g.groups;
  return true;
}

static int wg_splits(int num_blocks, int tiles_yz) {
  int s = sm_count() / tiles_yz;                     // one wave: the kernel's shared memory allows one CTA per SM
  if (s > num_blocks) s = num_blocks;
  if (s < 1) s = 1;
  return s;
}
static size_t wg_scratch_floats(int rows, int J, int CO, int tiles_yz) {
  const int num_blocks = (rows + WG_ROWS - 1) / WG_ROWS;
  const int bps = (num_blocks + wg_splits(num_blocks, tiles_yz) - 1) / wg_splits(num_blocks, tiles_yz);
  const int splits = (num_blocks + bps - 1) / bps;
  return (size_t)splits * J * CO + (size_t)splits * CO;
}

template <class XSrc, class GSrc, int JT, int BN, int STAGES, int CO>
static void tc_wgrad(LaunchCtx& lc, int kid, XSrc xs, GSrc gs, int rows, int n_atoms, float scale,
                     float* gw, float* gb, float* scratch, GradSegments* segs, uint32_t* err) {
  constexpr int smem = STAGES * ((2 * JT + BN / 64) * WG_ROWS * 128) + 2 * WG_ROWS * 128 + 1024;
  static_assert(STAGES >= WG_LAG || !XSrc::ASYNC, "pipeline depth");
  auto kern = tc_wgrad_kernel<XSrc, GSrc, (CO < 64 ? CO : 64), JT, BN, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int J = n_atoms * 64;
  const int gy = (n_atoms + 2 * JT - 1) / (2 * JT), gz = (CO + BN - 1) / BN;
  const int num_blocks = (rows + WG_ROWS - 1) / WG_ROWS;
  const int bps = (num_blocks + wg_splits(num_blocks, gy * gz) - 1) / wg_splits(num_blocks, gy * gz);
  const int splits = (num_blocks + bps - 1) / bps;
  float* bias_part = scratch + (size_t)splits * J * CO;
  const CUtensorMap* tm_x = tc_tensor_map(xs.x, (uint64_t)xs.M, (uint64_t)J, (uint64_t)xs.ld, WG_ROWS);
  const CUtensorMap* tm_g = tc_tensor_map(gs.g, (uint64_t)gs.M, (uint64_t)CO, (uint64_t)gs.ld, WG_ROWS);
  if (tm_x == nullptr || tm_g == nullptr) { lc.host_failure = true; return; }      // no tensor-map encoder
  KernelScope scope(lc, kid);
  launch_kernel_overlapped(lc, kern, dim3(splits, gy, gz), TC_THREADS, smem, *tm_x, *tm_g, xs, gs, scratch, bias_part, n_atoms, J, CO,
                           num_blocks, bps, err);
  if (!add_segment(segs, scratch, gw, splits, J, CO, scale) || !add_segment(segs, bias_part, gb, splits, 1, CO, 1.f))
    lc.host_failure = true;
}

// ---- weight gradients of the middle convolutions without im2col ----------------------------------------------
// The same shifted views as in the forward kernels, seen from the reduction side:
//   dW[tap][ci][co] = sum over raster positions m of X[m + shift(tap)][ci] * G[m][co],
// where X is the layer input in raster order and G the output gradient laid on the SAME raster (zero at the
// positions that are not outputs).  A stage holds 128 + max-shift rows of X (per plane) and 128 rows of G, each
// fetched once; both operands are MN-major (a shared-memory row = one raster position, 64 values of ci or co),
// and the A operand of tap t is the X image entered shift(t) rows down.  Two taps share one M = 128 instruction:
// the descriptor's leading-dimension offset, the distance between the first and the second block of 64 rows of
// M, is simply the distance between the two taps' entry rows, so the second half of the accumulator belongs to
// the next tap.  (An odd tap count leaves the upper half of the last accumulator unused.)
// The bias gradient, the column sums of G, is added up by one extra warp from the staged rows.
// A CTA owns a contiguous range of 128-row raster tiles (split-k); partial sums go to scratch as
// part[split][tap * 64 + ci][co] and the finishing kernel adds the splits in a fixed order.
constexpr int SWG_THREADS = 320;      // warps 0-7 producers (and the final epilogue), 8 MMA issuer, 9 bias sums
constexpr int SWG_MAX_SPLITS = 148;

template <int RASTER_, int WIDTH, int OUT_H, int OUT_W> struct GradCells {
  static constexpr int RASTER = RASTER_, STATE = OUT_H * OUT_W * 64;
  // element offset of raster cell `rem` inside a state's OUT_H x OUT_W x 64 gradient, or -1 for a margin cell
  __device__ static __forceinline__ int cell(int rem) {
    const int y = rem / WIDTH, x = rem % WIDTH;
    return (y < OUT_H && x < OUT_W) ? (y * OUT_W + x) * 64 : -1;
  }
};

struct SwgShared {
  uint64_t full[8], empty[8], acc;
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__device__ __forceinline__ void mma_bf16_lo_rt(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

template <class Cfg, class Cells, int STAGES>
__global__ void __launch_bounds__(SWG_THREADS, 1)
tc_shift_wgrad_kernel(Cfg cfg, const bf16* __restrict__ g, int states, float* __restrict__ partial,
                      float* __restrict__ bias_partial, int tiles, int tiles_per_cta, uint32_t* error_word) {
  constexpr int NT = Cfg::NT, NP = (NT + 1) / 2, SR = Cfg::STAGE_ROWS, PLANES = Cfg::PLANES, J = NT * 64;
  constexpr uint32_t PLANE_BYTES = SR * 128, X_BYTES = PLANES * PLANE_BYTES, G_BYTES = TC_BM * 128,
                     STAGE_BYTES = X_BYTES + G_BYTES;
  constexpr uint32_t TMEM_COLS = NP * 64 <= 256 ? 256 : 512;
  static_assert(STAGES >= 2 && STAGES <= 8 && SR % 8 == 0 && NP * 64 <= 512, "pipeline shape");
  extern __shared__ uint8_t dyn_smem[];
  __shared__ SwgShared sh;
  const uint32_t stage0 = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, t0 = split * tiles_per_cta, t1 = min(tiles, t0 + tiles_per_cta);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], 256); mbar_init(&sh.empty[s], 2); }
    mbar_init(&sh.acc, 1);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(&sh.tmem_base, TMEM_COLS);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources and weights that are several kernels old

  if (warp < 8) {
    // ---------------- producers: eight lanes per 128-byte row, 32 rows per pass ----------------
    const int c = lane & 7, sub = warp * 4 + (lane >> 3);
    for (int t = t0; t < t1; ++t) {
      const int it = t - t0, s = it % STAGES;
      const bool ok = mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t stage = stage0 + s * STAGE_BYTES;
      for (int idx = sub; idx < PLANES * SR; idx += 32) {
        const int plane = PLANES == 1 ? 0 : idx / SR, ri = PLANES == 1 ? idx : idx % SR;
        bool valid;
        const bf16* src = cfg.src(plane, t * TC_BM + ri, valid);
        cp_async16(stage + plane * PLANE_BYTES + ri * 128u + ((uint32_t)(c ^ (ri & 7)) << 4), src + c * 8, valid ? 16u : 0u);
      }
      // gradient rows (offsets by arithmetic: no shared-memory reads in a warp with copies in flight)
      int goff[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int pos = t * TC_BM + sub + 32 * k, b = pos / Cells::RASTER, cell = Cells::cell(pos - b * Cells::RASTER);
        goff[k] = (b < states && cell >= 0) ? b * Cells::STATE + cell : -1;                // < 2^31 elements
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int ri = sub + 32 * k;
        cp_async16(stage + X_BYTES + ri * 128u + ((uint32_t)(c ^ (ri & 7)) << 4), g + (goff[k] >= 0 ? goff[k] : 0) + c * 8,
                   goff[k] >= 0 ? 16u : 0u);
      }
      // the hardware arrives on the stage's barrier for this thread once its copies have landed
      cp_async_mbar_arrive(&sh.full[s]);
    }
    cp_async_commit();
    cp_async_wait<0>();
    // ---------------- epilogue: float partial tile to scratch ----------------
    // warps e and e + 4 share TMEM lane quarter e & 3 and take 32 of the 64 columns each
    if (t1 > t0 && mbar_wait(&sh.acc, 0, &sh.abort, error_word, ERR_WAIT_ACC)) {
      tcgen05_fence_after();
      const int quarter = warp & 3, col0 = (warp >> 2) * 32;
#pragma unroll 1
      for (int p = 0; p < NP; ++p) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + p * 64 + col0, r);
        const int j0 = p * 128 + quarter * 32;                   // this warp's rows j0 .. j0 + 31
        const uint32_t rows = j0 + 32 <= J ? 0xFFFFFFFFu : (j0 < J ? (1u << (J - j0)) - 1u : 0u);
        // Every MMA has completed, so the X parts of the operand stages are idle and serve as staging tiles (the G
        // parts are not touched: the bias warp may still be reading the last ones).
        static_assert(X_BYTES >= ((8 + STAGES - 1) / STAGES) * 4096, "room for the staging tiles");
        warp_store_rows_f32(stage0 + (warp % STAGES) * STAGE_BYTES + (warp / STAGES) * 4096, lane, r,
                            partial + ((size_t)split * J + j0) * 64 + col0, 64, rows);
      }
    }
  } else if (warp == 8) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc = make_idesc_bf16(TC_BM, 64, 1, 1);
      const uint32_t hi = desc_hi_kmajor_sw128();                 // stride between 8-row groups 1024 B, 128B swizzle
      bool ok = true;
      for (int t = t0; t < t1 && ok; ++t) {
        const int it = t - t0, s = it % STAGES;
        ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        fence_proxy_async_smem();        // the copies observed through the barrier -> visible to the MMA's operand reads
        tcgen05_fence_after();
        const uint32_t stage = stage0 + s * STAGE_BYTES;
        const uint32_t b_lo0 = ((stage + X_BYTES) >> 4) & 0x3FFFu;
#pragma unroll
        for (int k = 0; k < TC_BM / 16; ++k) {
#pragma unroll
          for (int p = 0; p < NP; ++p) {
            const int ta = 2 * p, tb = 2 * p + 1 < NT ? 2 * p + 1 : -1;
            const uint32_t a_off = Cfg::tap_plane(ta) * PLANE_BYTES + Cfg::tap_shift(ta) * 128u;
            // second half of M: the next tap's entry row (or simply the next row, result unused)
            const uint32_t lbo = tb >= 0 ? (Cfg::tap_plane(tb) * PLANE_BYTES + Cfg::tap_shift(tb) * 128u) - a_off : 128u;
            const uint32_t a_lo = (((stage + a_off + k * 2048u) >> 4) & 0x3FFFu) | ((lbo >> 4) << 16);
            mma_bf16_lo_rt(tmem + p * 64, a_lo, b_lo0 + k * (2048u >> 4), hi, idesc, (it | k) != 0 ? 1u : 0u);
          }
        }
        mma_commit(&sh.empty[s]);
      }
      if (ok && t1 > t0) mma_commit(&sh.acc);
    }
  } else {
    // ---------------- bias gradient: lane l adds up columns 2 l and 2 l + 1 of the staged G rows ----------------
    float acc[4][2] = {};
    bool ok = true;
    for (int t = t0; t < t1 && ok; ++t) {
      const int it = t - t0, s = it % STAGES;
      ok = mbar_wait(&sh.full[s], (it / STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      const uint32_t gbase = stage0 + s * STAGE_BYTES + X_BYTES + (uint32_t)(lane & 3) * 4u;
#pragma unroll 4
      for (int r8 = 0; r8 < TC_BM; r8 += 8) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          uint32_t v;
          asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(gbase + (r8 + r) * 128u + ((uint32_t)((lane >> 2) ^ r) << 4)) : "memory");
          acc[r & 3][0] += __uint_as_float(v << 16);
          acc[r & 3][1] += __uint_as_float(v & 0xFFFF0000u);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[s]);
    }
    if (ok && t1 > t0) {
      bias_partial[(size_t)split * 64 + 2 * lane] = (acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]);
      bias_partial[(size_t)split * 64 + 2 * lane + 1] = (acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == 8) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

static int swg_splits(int positions) {
  const int tiles = (positions + TC_BM - 1) / TC_BM;
  int ctas = sm_count() < SWG_MAX_SPLITS ? sm_count() : SWG_MAX_SPLITS;
  if (ctas > tiles) ctas = tiles;
  const int per = (tiles + ctas - 1) / ctas;
  return (tiles + per - 1) / per;
}

template <class Cfg, class Cells, int STAGES>
static void tc_shift_wgrad(LaunchCtx& lc, int kid, Cfg cfg, const bf16* g, int states, int positions, float* gw, float* gb,
                           float* scratch, GradSegments* segs, uint32_t* err) {
  constexpr int smem = STAGES * (Cfg::PLANES * Cfg::STAGE_ROWS + TC_BM) * 128 + 1024;
  static_assert(smem <= 227 * 1024, "shared memory budget");
  auto kern = tc_shift_wgrad_kernel<Cfg, Cells, STAGES>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  constexpr int J = Cfg::NT * 64;
  const int tiles = (positions + TC_BM - 1) / TC_BM;
  const int splits = swg_splits(positions), per = (tiles + splits - 1) / splits;
  float* bias_part = scratch + (size_t)splits * J * 64;
  KernelScope scope(lc, kid);
  launch_kernel_overlapped(lc, kern, splits, SWG_THREADS, smem, cfg, g, states, scratch, bias_part, tiles, per, err);
  if (!add_segment(segs, scratch, gw, splits, J, 64, 1.f) || !add_segment(segs, bias_part, gb, splits, 1, 64, 1.f))
    lc.host_failure = true;
}

// ---- first layer, weight gradient: space-to-depth, all four block taps in one MMA ----------------------------
// In the block view of the first layer (see the forward kernel) the weight gradient is
//   dW[tap][e][co] = sum over raster positions m of X[m + shift(tap)][e] * G[m][co],   shift = 0, 1, 21, 22,
// X[q] = the 64 values of 4 x 4-pixel block q, G = the output gradient on the 21-wide raster (zero in the margin).
// Both operands are MN-major images whose rows are raster positions.  One M = 128, N = 64 instruction covers all
// four taps: the two halves of M are the X image entered at rows m + 1 and m + 22 (leading-dimension offset of
// 21 rows), and the two halves of N are G[m] and G[m + 1] (each gradient row is staged twice, 64 bytes each):
//   D[a * 64 + e][h * 32 + co] = sum_m X[m + (a ? 22 : 1)][e] * G[m + h][co]  =  tap shift (a ? 22 : 1) - h.
// The right half sees every gradient row one position early, so tile t stands for positions 128 t - 1 .. 128 t + 126
// and the tiles of all CTAs together cover -1 .. total: every (tap, position) pair is counted exactly once.
// Raw frame rows arrive by bulk copy and are expanded to bf16 once per tile, as in the forward kernel.
// Roles, with E = W1_EXPAND_WARPS: warps 0 .. E-1 expand X (warps 0-3 also write the result at the end), warp E issues
// the MMAs, warp E+1 fetches frame rows, warps E+2 and E+11 add up the bias gradient from the staged gradient rows
// (half of the rows each), warps E+3 .. E+10 copy the gradient rows.  Role timers show the expansion busy three
// quarters of the kernel (1200 cycles per tile against 400 for the tile's eight MMAs); sixteen expansion warps
// were measured 8 % slower than eight: the role is bound by issue slots and shared-memory traffic, not by latency.
// The kernel is bound by how many bytes an SM keeps in flight from DRAM, so the gradient rows and the frame rows
// have rings of their own that run several tiles ahead of the expansion.
constexpr int W1_EXPAND_WARPS = 8, W1_THREADS = (W1_EXPAND_WARPS + 12) * 32, W1_STAGES = 4, W1_G_SLOTS = W1_STAGES, W1_G_AHEAD = 3, W1_X_ROWS = 152, W1_USED = 149,
              W1_RAW_BYTES = 12288, W1_RAW_SLOTS = 5;

struct W1Shared {
  uint64_t full[W1_STAGES], empty[W1_STAGES], raw_full[W1_RAW_SLOTS],
           raw_empty[W1_RAW_SLOTS], acc;
  uint32_t tmem_base;
  volatile uint32_t abort;
};

template <class G>
__global__ void __launch_bounds__(W1_THREADS, 1)
tc_conv1_wgrad_kernel(const uint8_t* __restrict__ frames, const bf16* __restrict__ g, float* __restrict__ partial,
                      float* __restrict__ bias_partial, int n_states, int tiles, int tiles_per_cta, uint32_t* error_word) {
  static_assert(G::OH == 20 && G::OW == 20 && G::CO == 32 && G::K == 8 && G::C == 4 && G::S == 4, "geometry");
  constexpr int POS = C1_RASTER * C1_RASTER, ROW_BYTES = G::W * G::C, E = W1_EXPAND_WARPS, NPROD = E * 32;
  constexpr int STEP = NPROD / 4, ITEMS = (W1_USED + STEP - 1) / STEP;          // positions between a thread's items
  constexpr uint32_t X_BYTES = W1_X_ROWS * 128, G_BYTES = TC_BM * 128;
  extern __shared__ uint8_t dyn_smem[];
  __shared__ W1Shared sh;
  const uint32_t stage0 = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const uint32_t g_base = stage0 + W1_STAGES * X_BYTES;
  const uint32_t raw_base = g_base + W1_G_SLOTS * G_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_pos = n_states * POS;
  const int split = blockIdx.x, t0 = split * tiles_per_cta, t1 = min(tiles, t0 + tiles_per_cta);

  if (threadIdx.x == 0) {
    // One barrier pair per slot serves the expanded X rows and the gradient rows alike (both rings have W1_STAGES
    // slots): full[s] gathers the eight expansion warps and the eight copy warps, empty[s] the commit of the tile's
    // instructions and the two bias warps.  The issuing thread then waits once and commits once per tile; with eight
    // short instructions per tile every further wait or commit (a couple of hundred cycles each, even when
    // satisfied) was what set the kernel's pace.
    for (int s = 0; s < W1_STAGES; ++s) { mbar_init(&sh.full[s], NPROD / 32 + 8); mbar_init(&sh.empty[s], 3); }
    for (int i = 0; i < W1_RAW_SLOTS; ++i) { mbar_init(&sh.raw_full[i], 1); mbar_init(&sh.raw_empty[i], NPROD / 32); }
    mbar_init(&sh.acc, 1);
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == E) tmem_alloc(&sh.tmem_base, 64);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;
  pdl_entry();          // everything above touches only this CTA's own resources

  // frame rows of tile t: blocks at positions qf .. ql, at most nine block rows in at most two states
  auto tile_ranges = [&](int t, int& b0, int& r0, int& n0, int& n1) {
    const int qf = min(t * TC_BM, total_pos - 1), ql = min(t * TC_BM + W1_USED - 1, total_pos - 1);
    b0 = qf / POS;
    const int b1 = ql / POS, yf = (qf % POS) / C1_RASTER, yl = (ql % POS) / C1_RASTER;
    r0 = 4 * yf;
    if (b1 == b0) { n0 = 4 * (yl - yf + 1); n1 = 0; }
    else { n0 = G::H - r0; n1 = 4 * (yl + 1); }
  };

  if (warp < E) {
    // ---------------- producers ----------------
    const int p = threadIdx.x;
    for (int t = t0; t < t1; ++t) {
      const int it = t - t0, s = it % W1_STAGES, slot = it % W1_RAW_SLOTS;
      int b0, r0, n0, n1;
      tile_ranges(t, b0, r0, n0, n1);
      bool ok = mbar_wait(&sh.empty[s], ((it / W1_STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t stage = stage0 + s * X_BYTES;
      ok = mbar_wait(&sh.raw_full[slot], (it / W1_RAW_SLOTS) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!__all_sync(0xffffffffu, ok)) break;
      const uint32_t raw = raw_base + slot * W1_RAW_BYTES;
      // X rows: work item = (position u of the tile, pixel row py of its block): 16 raw bytes -> two operand chunks;
      // thread p takes items p, p + NPROD, ...: the same py, positions STEP apart
      const int py = p & 3, u = p >> 2;
      int b, Y, X;
      {
        const int q = t * TC_BM + u;
        b = q / POS;
        const int rem = q - b * POS;
        Y = rem / C1_RASTER; X = rem - Y * C1_RASTER;
      }
      uint4 rw[ITEMS];
#pragma unroll
      for (int k = 0; k < ITEMS; ++k) {
        if (b >= n_states) { b = n_states - 1; Y = C1_RASTER - 1; X = C1_RASTER - 1; }     // past the end: repeat the last block
        const int slot_row = (b == b0 ? 4 * Y - r0 : n0 + 4 * Y) + py;
        if (u + STEP * k < W1_USED)
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(rw[k].x), "=r"(rw[k].y), "=r"(rw[k].z), "=r"(rw[k].w)
                       : "r"(raw + (uint32_t)(slot_row * ROW_BYTES + X * 16)) : "memory");
        X += STEP % C1_RASTER; Y += STEP / C1_RASTER;
        if (X >= C1_RASTER) { X -= C1_RASTER; ++Y; }
        if (Y >= C1_RASTER) { Y -= C1_RASTER; ++b; }
      }
#pragma unroll
      for (int k = 0; k < ITEMS; ++k) {
        const uint32_t ri = (uint32_t)(u + STEP * k);
        if (ri < (uint32_t)W1_USED) {
          uint32_t o[8];
          u8x4_to_f16x4(rw[k].x, o[0], o[1]); u8x4_to_f16x4(rw[k].y, o[2], o[3]);          // bytes as bf16 values n * 2^-133
          u8x4_to_f16x4(rw[k].z, o[4], o[5]); u8x4_to_f16x4(rw[k].w, o[6], o[7]);
          const uint32_t dst = stage + ri * 128u;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((uint32_t)((2 * py) ^ (ri & 7)) << 4)),
                       "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((uint32_t)((2 * py + 1) ^ (ri & 7)) << 4)),
                       "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&sh.full[s]); mbar_arrive(&sh.raw_empty[slot]); }
    }
    // ---------------- epilogue: float partial tile to scratch, rows regrouped to the canonical weight order ----------------
    if (warp < 4 && t1 > t0 && mbar_wait(&sh.acc, 0, &sh.abort, error_word, ERR_WAIT_ACC)) {
      tcgen05_fence_after();
      const int row = threadIdx.x, a = row >> 6, e = row & 63, py = e >> 4, px = (e >> 2) & 3, ci = e & 3;
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + h * 32, r);
        const int i = a, jj = 1 - h;                                    // block tap (i, jj): shift 21 i + jj
        const int jcan = ((4 * i + py) * 8 + 4 * jj + px) * 4 + ci;    // (r, s, ci) of the 8 x 8 x 4 filter
        float4* dst = reinterpret_cast<float4*>(partial + ((size_t)split * 256 + jcan) * 32);
#pragma unroll
        for (int v = 0; v < 8; ++v)
          dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                               __uint_as_float(r[4 * v + 3]));
      }
    }
  } else if (warp == E) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      constexpr uint32_t idesc = make_idesc_bf16(TC_BM, 64, 1, 1);
      const uint32_t hi = desc_hi_kmajor_sw128();
      constexpr uint32_t LBO = 21u * 128u;                 // second half of M: the X image 21 rows further down
      bool ok = true;
      for (int t = t0; t < t1 && ok; ++t) {
        const int it = t - t0, s = it % W1_STAGES, gs = it % W1_G_SLOTS;
        ok = mbar_wait(&sh.full[s], (it / W1_STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
        if (!ok) break;
        fence_proxy_async_smem();        // the copies observed through the barrier -> visible to the MMA's operand reads
        tcgen05_fence_after();
        const uint32_t a_lo0 = (((stage0 + s * X_BYTES) >> 4) & 0x3FFFu) | ((LBO >> 4) << 16);
        const uint32_t b_lo0 = ((g_base + gs * G_BYTES) >> 4) & 0x3FFFu;
#pragma unroll
        for (int k = 0; k < TC_BM / 16; ++k)
          mma_bf16_lo_rt(tmem, a_lo0 + k * (2048u >> 4), b_lo0 + k * (2048u >> 4), hi, idesc, (it | k) != 0 ? 1u : 0u);
        mma_commit(&sh.empty[s]);
      }
      if (ok && t1 > t0) mma_commit(&sh.acc);
    }
  } else if (warp == E + 1) {
    if (lane == 0) {
      // ---------------- raw loader ----------------
      for (int t = t0; t < t1; ++t) {
        const int it = t - t0, slot = it % W1_RAW_SLOTS;
        if (!mbar_wait(&sh.raw_empty[slot], ((it / W1_RAW_SLOTS) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY)) break;
        int b0, r0, n0, n1;
        tile_ranges(t, b0, r0, n0, n1);
        const uint32_t dst = raw_base + slot * W1_RAW_BYTES;
        mbar_arrive_expect_tx(&sh.raw_full[slot], (uint32_t)((n0 + n1) * ROW_BYTES));
        bulk_copy_g2s(dst, frames + ((size_t)b0 * G::H + r0) * ROW_BYTES, (uint32_t)(n0 * ROW_BYTES), &sh.raw_full[slot]);
        if (n1 > 0)
          bulk_copy_g2s(dst + n0 * ROW_BYTES, frames + (size_t)(b0 + 1) * G::H * ROW_BYTES, (uint32_t)(n1 * ROW_BYTES),
                        &sh.raw_full[slot]);
      }
    }
  } else if (warp >= E + 3 && warp < E + 11) {
    // ---------------- gradient rows: image row r = [G[m] | G[m + 1]], m = 128 t - 1 + r ----------------
    // thread p copies chunk p & 7 of rows (p >> 3) + 32 k, W1_G_AHEAD tiles ahead of the tile it publishes
    const int p = threadIdx.x - (E + 3) * 32, c8 = p & 7, half = c8 >> 2, chunk = c8 & 3;
    int b1, Y, X;
    {
      const int mm = t0 * TC_BM - 1 + (p >> 3) + half + POS;       // one state further, so that position -1 is not negative
      b1 = mm / POS;
      const int rem = mm - b1 * POS;
      Y = rem / C1_RASTER; X = rem - Y * C1_RASTER;
    }
    bool alive = true;
    for (int t = t0; t < t1 + W1_G_AHEAD && alive; ++t) {
      // publish first, fetch second: the slot a fetch waits for must not be the one whose consumers are waiting
      // for this very publication
      if (t - W1_G_AHEAD >= t0) {
        cp_async_wait<W1_G_AHEAD - 1>();           // the rows of tile t - W1_G_AHEAD (my share) have landed
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.full[(t - W1_G_AHEAD - t0) % W1_G_SLOTS]);
      }
      if (t < t1) {
        const int it = t - t0, gs = it % W1_G_SLOTS;
        const bool ok = mbar_wait(&sh.empty[gs], ((it / W1_G_SLOTS) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
        if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
        const uint32_t dst = g_base + gs * G_BYTES;
        // Source offsets: the raster cell (state + 1, Y, X) of this thread's first row is carried from tile to tile
        // and stepped by 32 positions from row to row; these few warps have no one to hide a division's latency.
        int off[4];
        {
          int bb = b1, yy = Y, xx = X;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const bool valid = bb >= 1 && bb <= n_states && yy < G::OH && xx < G::OW;
            off[k] = valid ? ((bb - 1) * (G::OH * G::OW) + yy * G::OW + xx) * G::CO + chunk * 8 : -1;     // < 2^31 elements
            xx += 32 - C1_RASTER; ++yy;                       // 32 positions on
            if (xx >= C1_RASTER) { xx -= C1_RASTER; ++yy; }
            if (yy >= C1_RASTER) { yy -= C1_RASTER; ++bb; }
          }
          X += TC_BM - 6 * C1_RASTER; Y += 6;                 // the next tile is 128 = 6 * 21 + 2 positions on
          if (X >= C1_RASTER) { X -= C1_RASTER; ++Y; }
          if (Y >= C1_RASTER) { Y -= C1_RASTER; ++b1; }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int r = (p >> 3) + 32 * k;
          cp_async16(dst + r * 128u + ((uint32_t)(c8 ^ (r & 7)) << 4), g + (off[k] >= 0 ? off[k] : 0), off[k] >= 0 ? 16u : 0u);
        }
      }
      cp_async_commit();                           // one group per iteration, also when there is nothing left to fetch
    }
    cp_async_wait<0>();
  } else {
    // ---------------- bias gradient: the left halves of the staged gradient rows hold every position once ----------------
    // lane l adds channels 8 (l & 3) .. 8 (l & 3) + 7 (one 16-byte chunk) over the rows (l >> 2) + 8 i, i of this warp's parity
    float acc[8] = {};
    bool ok = true;
    const int q = lane & 3, rr = lane >> 2, which = warp == E + 2 ? 0 : 1;
    for (int t = t0; t < t1 && ok; ++t) {
      const int it = t - t0, gs = it % W1_G_SLOTS;
      ok = mbar_wait(&sh.full[gs], (it / W1_G_SLOTS) & 1, &sh.abort, error_word, ERR_WAIT_FULL);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      const uint32_t gaddr = g_base + gs * G_BYTES + (uint32_t)(rr + 8 * which) * 128u + ((uint32_t)(q ^ rr) << 4);
      uint32_t v[TC_BM / 16][4];
#pragma unroll
      for (int i = 0; i < TC_BM / 16; ++i)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i][0]), "=r"(v[i][1]), "=r"(v[i][2]), "=r"(v[i][3])
                     : "r"(gaddr + (uint32_t)i * 2048u) : "memory");
#pragma unroll
      for (int i = 0; i < TC_BM / 16; ++i) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] += __uint_as_float(v[i][j] << 16);
          acc[2 * j + 1] += __uint_as_float(v[i][j] & 0xFFFF0000u);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.empty[gs]);
    }
    // the eight row groups, added in a fixed order
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 4);
      acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 8);
      acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 16);
    }
    if (ok && t1 > t0 && lane < 4) {
#pragma unroll
      for (int j = 0; j < 8; ++j) bias_partial[((size_t)split * 2 + which) * 32 + 8 * q + j] = acc[j];
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == E) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 64);
  }
}

// how many CTAs (= split-k partial sums) the first layer's weight gradient uses for n_states states
static int tc_conv1_wgrad_splits(int n_states) {
  const int tiles = (n_states * C1_RASTER * C1_RASTER + 1 + TC_BM - 1) / TC_BM;      // positions -1 .. total - 1
  int ctas = sm_count() < SWG_MAX_SPLITS ? sm_count() : SWG_MAX_SPLITS;
  if (ctas > tiles) ctas = tiles;
  const int per = (tiles + ctas - 1) / ctas;
  return (tiles + per - 1) / per;
}
// launches the kernel on n_states states; its CTAs leave their weight tiles in partial[cta][256][32] and their two
// bias rows in bias_part[2 cta + i][32]; returns the number of CTAs
template <class G>
static int tc_conv1_wgrad_launch(LaunchCtx& lc, const uint8_t* frames, const bf16* g, int n_states, float* partial,
                                 float* bias_part, uint32_t* err) {
  constexpr int smem = (W1_STAGES * W1_X_ROWS + W1_G_SLOTS * TC_BM) * 128 + W1_RAW_SLOTS * W1_RAW_BYTES + 1024;
  static_assert(smem <= 227 * 1024, "shared memory budget");
  auto kern = tc_conv1_wgrad_kernel<G>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  const int tiles = (n_states * C1_RASTER * C1_RASTER + 1 + TC_BM - 1) / TC_BM;
  const int splits = tc_conv1_wgrad_splits(n_states), per = (tiles + splits - 1) / splits;
  KernelScope scope(lc, KID_CONV1_WGRAD);
  launch_kernel_overlapped(lc, kern, splits, W1_THREADS, smem, frames, g, partial, bias_part, n_states, tiles, per, err);
  return splits;
}
template <class G>
static void tc_conv1_wgrad(LaunchCtx& lc, const uint8_t* frames, const bf16* g, int n_states, float* gw, float* gb,
                           float* scratch, GradSegments* segs, uint32_t* err) {
  float* bias_part = scratch + (size_t)tc_conv1_wgrad_splits(n_states) * 256 * 32;
  const int splits = tc_conv1_wgrad_launch<G>(lc, frames, g, n_states, scratch, bias_part, err);
  // the gradient rows arrive multiplied by C1_GRAD_SCALE (see tc_backward_dgrad_conv2), the pixels as n * 2^-133
  if (!add_segment(segs, scratch, gw, splits, 256, 32, C1_WGRAD_OUTPUT_SCALE) ||
      !add_segment(segs, bias_part, gb, 2 * splits, 1, 32, C1_BIAS_OUTPUT_SCALE))      // two bias warps per CTA, a row each
    lc.host_failure = true;
}

// every layer keeps its own partial-sum region until the finishing kernel has run
static size_t tc_layer_scratch_floats(int n, int layer) {
  switch (layer) {
    case 0: return (size_t)TC_MAX_UPDATE_CHUNKS * SWG_MAX_SPLITS * (256 * 32 + 2 * 32);      // per chunk and CTA: the weight tile and two bias rows
    case 1: return (size_t)SWG_MAX_SPLITS * (512 * 64 + 64);
    case 2: return (size_t)SWG_MAX_SPLITS * (576 * 64 + 64);
    default: return wg_scratch_floats(n, 3136, 512, 13 * 4);      // 256 x 128 tiles of the 3136 x 512 matrix
  }
}
static size_t tc_layer_scratch_offset(int n, int layer) {
  size_t off = 0;
  for (int l = 0; l < layer; ++l) off += (tc_layer_scratch_floats(n, l) + 63) / 64 * 64;
  return off;
}

static size_t tc_heads_scratch_floats();
size_t tc_scratch_floats(int n) { return tc_layer_scratch_offset(n, 4) + tc_heads_scratch_floats(); }

// Enqueues the weight-gradient kernel of `layer` (0 = conv1 .. 3 = fc) and notes in *segs where its partial
// sums are; tc_backward_finish() then turns all noted partial sums into the gradient vector in one launch.
int tc_backward_finish(LaunchCtx& lc, GradSegments* segs, float* sumsq_partials) {
  int blocks = 0;
  if (segs->n > 0) {
    KernelScope scope(lc, KID_WGRAD_REDUCE);
    blocks = segs->total_groups < NORM_BLOCKS ? segs->total_groups : NORM_BLOCKS;
    launch_kernel(lc, tc_finalize_grads_kernel, blocks, 256, 0, *segs, sumsq_partials);
  }
  segs->n = 0; segs->total_groups = 0;
  return blocks;
}

void tc_backward_wgrad(LaunchCtx& lc, const NetDims& nd, const uint8_t* frames, int n, void* const act[],
                       void* const gact[], float* grad, float* scratch, int layer, GradSegments* segsp, uint32_t* err) {
  GradSegments& segs = *segsp;
  const LayerDims* d = nd.layer;
  float* gw = grad + d[layer].w_off; float* gb = grad + d[layer].b_off;
  const bf16* g = (const bf16*)gact[layer];
  float* sc = scratch + tc_layer_scratch_offset(n, layer);
  if (layer == 0) {
    typedef NatConv1 C1;
    tc_conv1_wgrad<C1>(lc, frames, g, n, gw, gb, sc, &segs, err);
  } else if (layer == 1) {
    tc_shift_wgrad<C2FwdCfg, GradCells<100, 10, 9, 9>, 4>(lc, KID_CONV2_WGRAD, C2FwdCfg{(const bf16*)act[0], n}, g, n, n * 100,
                                                          gw, gb, sc, &segs, err);
  } else if (layer == 2) {
    tc_shift_wgrad<C3FwdCfg, GradCells<81, 9, 7, 7>, 5>(lc, KID_CONV3_WGRAD, C3FwdCfg{(const bf16*)act[1], n * 81}, g, n, n * 81,
                                                        gw, gb, sc, &segs, err);
  } else {
    tc_wgrad<PlainSrc, GradSrc<64>, 2, 128, 4, 512>(lc, KID_FC_WGRAD, PlainSrc{(const bf16*)act[2], 3136, n},
                                                    GradSrc<64>{g, 512, n}, n, 49, 1.f, gw, gb, sc, &segs, err);
  }
}

// ---- backward through the two heads, one kernel ---------------------------------------------------------------
// With dz[b][k] the loss gradient at the logits and dV[b] at the value (row k = A of a combined matrix):
//   g_fc[b][i] = (h[b][i] > 0) * sum_k dz[b][k] W[k][i],      dW[k][i] = sum_b dz[b][k] h[b][i],     db[k] = sum_b dz[b][k].
// A thread owns two of the 512 hidden units: their weight columns live in registers, every row costs it one 4-byte
// load of h and NK multiply-adds each way, and the row's dz values are broadcast from shared memory.  A CTA walks a
// contiguous range of rows and leaves its dW / db sums as one more split for the finishing kernel.
constexpr int HB_THREADS = 256, HB_ROWS = 40;      // rows staged at a time: a CTA's whole share at the largest benchmark size

template <int NK>
__global__ void __launch_bounds__(HB_THREADS, 2)
heads_backward_kernel(const bf16* __restrict__ h, const float* __restrict__ dz, const float* __restrict__ dV,
                      const bf16* __restrict__ wpi, const bf16* __restrict__ wv, int n, int A, int rows_per,
                      bf16* __restrict__ g_fc, float* __restrict__ part_w, float* __restrict__ part_b,
                      float* __restrict__ part_vw, float* __restrict__ part_vb) {
  constexpr int F = 512;
  static_assert(NK % 4 == 0, "rows of dz are read as float4");
  __shared__ __align__(16) float dzs[HB_ROWS][NK];
  const int tid = threadIdx.x, col = 2 * tid;
  float w[NK][2], acc[NK][2], accb = 0.f;            // accb: thread k < NK adds up column k of dz
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    acc[k][0] = acc[k][1] = 0.f;
    w[k][0] = w[k][1] = 0.f;
    if (k < A) { w[k][0] = to_f(wpi[(size_t)k * F + col]); w[k][1] = to_f(wpi[(size_t)k * F + col + 1]); }
    else if (k == A) { w[k][0] = to_f(wv[col]); w[k][1] = to_f(wv[col + 1]); }
  }
  pdl_entry();          // the head weights above were written several kernels ago
  const int r0 = blockIdx.x * rows_per, r1 = min(n, r0 + rows_per);
  for (int rb = r0; rb < r1; rb += HB_ROWS) {
    // eight rows of h at a time, the next eight fetched while these are used (the loads' latency was the kernel's
    // bound); the first eight are asked for before the block's dz rows are staged
    uint32_t hv[8], hn[8];
#pragma unroll
    for (int j = 0; j < 8; ++j)
      hv[j] = rb + j < r1 ? __ldg(reinterpret_cast<const uint32_t*>(h + (size_t)(rb + j) * F + col)) : 0u;
    __syncthreads();
    for (int i = tid; i < HB_ROWS * NK; i += HB_THREADS) {
      const int r = rb + i / NK, k = i % NK;
      dzs[i / NK][k] = r < r1 ? (k < A ? dz[(size_t)r * A + k] : (k == A ? dV[r] : 0.f)) : 0.f;
    }
    __syncthreads();
    if (tid < NK)
      for (int r = 0; r < HB_ROWS; ++r) accb += dzs[r][tid];        // rows past the end hold zeros
#pragma unroll 1
    for (int q = 0; q < HB_ROWS && rb + q < r1; q += 8) {
#pragma unroll
      for (int j = 0; j < 8; ++j)
        hn[j] = (q + 8 + j < HB_ROWS && rb + q + 8 + j < r1)
                    ? __ldg(reinterpret_cast<const uint32_t*>(h + (size_t)(rb + q + 8 + j) * F + col)) : 0u;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (rb + q + j >= r1) break;
        const float h0 = __uint_as_float(hv[j] << 16), h1 = __uint_as_float(hv[j] & 0xFFFF0000u);
        float g0 = 0.f, g1 = 0.f;
#pragma unroll
        for (int k4 = 0; k4 < NK; k4 += 4) {
          const float4 d4 = *reinterpret_cast<const float4*>(&dzs[q + j][k4]);
          const float d[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            g0 = fmaf(d[i], w[k4 + i][0], g0); g1 = fmaf(d[i], w[k4 + i][1], g1);
            acc[k4 + i][0] = fmaf(d[i], h0, acc[k4 + i][0]); acc[k4 + i][1] = fmaf(d[i], h1, acc[k4 + i][1]);
          }
        }
        *reinterpret_cast<uint32_t*>(g_fc + (size_t)(rb + q + j) * F + col) =
            pack_bf16x2(h0 > 0.f ? g0 : 0.f, h1 > 0.f ? g1 : 0.f);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) hv[j] = hn[j];
    }
  }
  // partial sums of this CTA in the layout of the parameters themselves: policy rows [action][hidden unit], the
  // value row, the two biases
  const size_t cta = blockIdx.x;
#pragma unroll
  for (int k = 0; k < NK; ++k) {
    if (k < A) *reinterpret_cast<float2*>(part_w + (cta * A + k) * F + col) = make_float2(acc[k][0], acc[k][1]);
    else if (k == A) *reinterpret_cast<float2*>(part_vw + cta * F + col) = make_float2(acc[k][0], acc[k][1]);
  }
  if (tid < A) part_b[cta * A + tid] = accb;
  else if (tid == A) part_vb[cta] = accb;
}

constexpr int HB_MAX_SPLITS = 148;
static size_t tc_heads_scratch_floats() { return (size_t)HB_MAX_SPLITS * (512 * 20 + 20) + 4; }

bool tc_heads_backward_supported(const NetDims& nd) { return nd.F == 512 && nd.A + 1 <= 20; }

void tc_heads_backward(LaunchCtx& lc, const NetDims& nd, const bf16* theta16, const bf16* h, int n, const float* dz,
                       const float* dV, bf16* g_fc, float* grad, float* scratch, GradSegments* segs) {
  const int A = nd.A;
  int ctas = sm_count() < HB_MAX_SPLITS ? sm_count() : HB_MAX_SPLITS;
  if (ctas > n) ctas = n;
  const int rows_per = (n + ctas - 1) / ctas, splits = (n + rows_per - 1) / rows_per;
  float* sc = scratch + tc_layer_scratch_offset(n, 4);
  // the value row's partial sums are stored as float2: their area starts on an even float (splits * A can be odd)
  float* part_w = sc; float* part_b = part_w + (size_t)splits * 512 * A;
  float* part_vw = part_b + (((size_t)splits * A + 3) & ~(size_t)3); float* part_vb = part_vw + (size_t)splits * 512;
  KernelScope scope(lc, KID_HEADS_BWD);
  if (A + 1 <= 8)
    launch_kernel_overlapped(lc, heads_backward_kernel<8>, splits, HB_THREADS, 0, h, dz, dV, theta16 + nd.pi_w, theta16 + nd.v_w, n, A,
                  rows_per, g_fc, part_w, part_b, part_vw, part_vb);
  else
    launch_kernel_overlapped(lc, heads_backward_kernel<20>, splits, HB_THREADS, 0, h, dz, dV, theta16 + nd.pi_w, theta16 + nd.v_w, n, A,
                  rows_per, g_fc, part_w, part_b, part_vw, part_vb);
  // already in parameter order: plain sums
  if (!add_segment(segs, part_w, grad + nd.pi_w, splits, 1, 512 * A, 1.f) || !add_segment(segs, part_b, grad + nd.pi_b, splits, 1, A, 1.f) ||
      !add_segment(segs, part_vw, grad + nd.v_w, splits, 1, 512, 1.f) || !add_segment(segs, part_vb, grad + nd.v_b, splits, 1, 1, 1.f))
    lc.host_failure = true;
}

// ---- weight images for the backward contractions ------------------------------------------------------
// From the canonical bf16 copy: wfc_t[i][o] = Wfc[o][i];  w3_d[ci][r][s][co] = W3[co][r][s][ci];
// w2_d[z][ci][i][j][co] = W2[co][py + 2i][px + 2j][ci] with z = 2 py + px;
// w1_b[co][2i + j][py][px][ci] = W1[co][4i + py][4j + px][ci] (the first layer's weights per 4 x 4 block tap).
constexpr int RL_FC_TILES = (3136 / 64) * (512 / 64), RL_SMALL_BLOCKS = 76;
__global__ void __launch_bounds__(256) relayout_weights_kernel(const bf16* __restrict__ w1, const bf16* __restrict__ w2,
                                        const bf16* __restrict__ w3, const bf16* __restrict__ wfc,
                                        bf16* __restrict__ w2_d, bf16* __restrict__ w3_d, bf16* __restrict__ wfc_t,
                                        bf16* __restrict__ w1_b, uint32_t* __restrict__ error_word) {
  pdl_entry();
  typedef NatConv2 C2; typedef NatConv3 C3;
  constexpr int N2 = 4 * C2::C * 4 * C2::CO, N3 = C3::C * 9 * C3::CO, NF = 3136 * 512, N1 = 32 * 256;
  // Blocks 0 .. RL_FC_TILES - 1 transpose the fully connected matrix, the bulk of the work, one 64 x 64 tile each
  // through shared memory, so that both sides are whole 128-byte rows; the other blocks gather the small images.
  if (blockIdx.x < RL_FC_TILES) {
    __shared__ uint16_t tile[64][66];                              // row pitch of 33 words: column reads spread over the banks
    const int o0 = (blockIdx.x % 8) * 64, in0 = (blockIdx.x / 8) * 64;
    const int r = threadIdx.x >> 2, c = threadIdx.x & 3;
    {
      const uint4* src = reinterpret_cast<const uint4*>(wfc + (size_t)(o0 + r) * 3136 + in0 + 16 * c);
      const uint4 lo = __ldg(src), hi = __ldg(src + 1);
      const uint32_t v[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) *reinterpret_cast<uint32_t*>(&tile[r][16 * c + 2 * e]) = v[e];
    }
    __syncthreads();
    uint32_t v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e)
      v[e] = (uint32_t)tile[16 * c + 2 * e][r] | ((uint32_t)tile[16 * c + 2 * e + 1][r] << 16);
    uint4* dst = reinterpret_cast<uint4*>(wfc_t + (size_t)(in0 + r) * 512 + o0 + 16 * c);
    dst[0] = make_uint4(v[0], v[1], v[2], v[3]);
    dst[1] = make_uint4(v[4], v[5], v[6], v[7]);
    return;
  }
  for (int i = (blockIdx.x - RL_FC_TILES) * blockDim.x + threadIdx.x; i < N2 + N3 + N1; i += (gridDim.x - RL_FC_TILES) * blockDim.x) {
    if (i >= N2 + N3) {
      const int j = i - N2 - N3, ci = j & 3, px = (j >> 2) & 3, py = (j >> 4) & 3, tap = (j >> 6) & 3, co = j >> 8;
      const int r = 4 * (tap >> 1) + py, sx = 4 * (tap & 1) + px;
      // the forward kernel's copy of the first layer is fp16, scaled by 2^8 (see u8x4_to_f16x4)
      const float scaled = __bfloat162float(w1[((co * 8 + r) * 8 + sx) * 4 + ci]) * C1_F16_WEIGHT_SCALE;
      if (!(fabsf(scaled) <= 65504.f)) atomicOr(error_word, DEV_ERR_RANGE);      // beyond fp16 (or not a number)
      reinterpret_cast<__half*>(w1_b)[j] = __float2half_rn(scaled);
      continue;
    }
    if (i < N2) {
      const int co = i % 64, t = (i / 64) % 4, ci = (i / 256) % 32, z = i / (256 * 32);
      const int r = (z >> 1) + 2 * (t >> 1), s = (z & 1) + 2 * (t & 1);
      w2_d[i] = w2[((co * 4 + r) * 4 + s) * 32 + ci];
    } else {
      const int j = i - N2, co = j % 64, tap = (j / 64) % 9, ci = j / 576;
      w3_d[j] = w3[(co * 9 + tap) * 64 + ci];
    }
  }
}
size_t tc_weight_image_elems() { return TC_IMG_END; }

void tc_relayout_weights(LaunchCtx& lc, const NetDims& nd, const bf16* theta16, bf16* images, uint32_t* error_word) {
  const LayerDims* d = nd.layer;
  KernelScope scope(lc, KID_CAST);
  launch_kernel(lc, relayout_weights_kernel, RL_FC_TILES + RL_SMALL_BLOCKS, 256, 0, theta16 + d[0].w_off, theta16 + d[1].w_off, theta16 + d[2].w_off,
                                                  theta16 + d[3].w_off, images + TC_IMG_W2, images + TC_IMG_W3,
                                                  images + TC_IMG_WFC, images + TC_IMG_W1, error_word);
}

// ---- failure-path probe: a bounded wait that is made to run out ------------------------------------------------
// One warp initialises a barrier that expects one arrival, nobody arrives, and every lane waits for its first
// phase with the given poll limit: the wait gives up, the error bit is recorded, the block returns.
__global__ void __launch_bounds__(32) wait_probe_kernel(uint32_t max_polls, uint32_t* error_word) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t abort_flag;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0u; fence_barrier_init(); }
  __syncwarp();
  mbar_wait_limit(&bar, 0, &abort_flag, error_word, ERR_WAIT_FULL, max_polls);
}
void launch_wait_probe(LaunchCtx& lc, uint32_t max_polls, uint32_t* error_word) {
  KernelScope scope(lc, KID_INIT);
  launch_kernel(lc, wait_probe_kernel, 1, 32, 0, max_polls, error_word);
}

// ---- backward: data gradients ---------------------------------------------------------------------------
void tc_backward_dgrad_fc(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err) {
  const bf16* wfc_t = images + 4 * 32 * 256 + 64 * 576;
  tc_persistent<PlainSrc, ReluMaskEpiTc, 128, 8, 1, 2, 2>(
      lc, KID_FC_DGRAD, PlainSrc{(const bf16*)gact[3], 512, n}, wfc_t, 3136,
      ReluMaskEpiTc{(bf16*)gact[2], (const bf16*)act[2], 3136, n}, n, err);
}
void tc_backward_dgrad_conv3(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err) {
  typedef NatConv3 C3;
  const int M = n * C3::H * C3::W;
  typedef RasterMap<121, 11, 9, 9> Map;
  tc_shift<C3DgradCfg, ShiftReluMaskEpi<Map, 9, 9>, 64, 4, 1>(
      lc, KID_CONV3_DGRAD, C3DgradCfg{(const bf16*)gact[2], n}, images + 4 * 32 * 256,
      ShiftReluMaskEpi<Map, 9, 9>{Map{n}, (bf16*)gact[1], (const bf16*)act[1]}, n * 121, err);
  (void)M;
}
float tc_conv1_grad_scale() { return C1_GRAD_SCALE; }

// The conv2 data gradient and the conv1 weight gradient over `chunks` groups of states, alternating, so that a group's
// slice of the gradient at the first layer's output (25.6 KB per state) is read back while it is still in L2.  All groups' partial
// sums lie one behind the other (weight tiles, then bias rows), in group order, and are added up as one segment.
void tc_backward_conv2d_conv1w_chunked(LaunchCtx& lc, const NetDims& nd, const bf16* images, const uint8_t* frames, int n,
                                       void* const act[], void* const gact[], float* grad, float* scratch, int chunks,
                                       GradSegments* segs, uint32_t* err) {
  typedef NatConv1 C1;
  typedef NatConv2 C2;
  typedef RasterMap<121, 11, 10, 10> Map;
  if (chunks > TC_MAX_UPDATE_CHUNKS) chunks = TC_MAX_UPDATE_CHUNKS;
  if (chunks > n) chunks = n;
  const int per = (n + chunks - 1) / chunks;
  int total_splits = 0;
  for (int s0 = 0; s0 < n; s0 += per) total_splits += tc_conv1_wgrad_splits(n - s0 < per ? n - s0 : per);
  float* part = scratch + tc_layer_scratch_offset(n, 0);
  float* bias_part = part + (size_t)total_splits * 256 * 32;
  const size_t a0 = (size_t)C2::H * C2::W * C2::C, g1 = (size_t)C2::OH * C2::OW * C2::CO;      // elements per state
  int done = 0;
  for (int s0 = 0; s0 < n; s0 += per) {
    const int nc = n - s0 < per ? n - s0 : per;
    bf16* gact0 = (bf16*)gact[0] + (size_t)s0 * a0;
    tc_shift<C2DgradCfg, ShiftReluMaskEpiS2<Map>, 128, 3, 1>(
        lc, KID_CONV2_DGRAD, C2DgradCfg{(const bf16*)gact[1] + (size_t)s0 * g1, nc}, images,
        ShiftReluMaskEpiS2<Map>{Map{nc}, gact0, (const bf16*)act[0] + (size_t)s0 * a0, C1_GRAD_SCALE}, nc * 121, err);
    done += tc_conv1_wgrad_launch<C1>(lc, frames + (size_t)s0 * FRAME_BYTES, gact0, nc, part + (size_t)done * 256 * 32,
                                      bias_part + (size_t)done * 2 * 32, err);
  }
  const LayerDims* d = nd.layer;
  if (!add_segment(segs, part, grad + d[0].w_off, total_splits, 256, 32, C1_WGRAD_OUTPUT_SCALE) ||
      !add_segment(segs, bias_part, grad + d[0].b_off, 2 * total_splits, 1, 32, C1_BIAS_OUTPUT_SCALE))
    lc.host_failure = true;
}

void tc_backward_dgrad_conv2(LaunchCtx& lc, const bf16* images, int n, void* const act[], void* const gact[], uint32_t* err,
                             float out_scale) {
  typedef NatConv2 C2;
  const int M = n * (C2::H / 2) * (C2::W / 2);
  typedef RasterMap<121, 11, 10, 10> Map;
  tc_shift<C2DgradCfg, ShiftReluMaskEpiS2<Map>, 128, 3, 1>(
      lc, KID_CONV2_DGRAD, C2DgradCfg{(const bf16*)gact[1], n}, images,
      ShiftReluMaskEpiS2<Map>{Map{n}, (bf16*)gact[0], (const bf16*)act[0], out_scale}, n * 121, err);
  (void)M;
}

}  // namespace paac
