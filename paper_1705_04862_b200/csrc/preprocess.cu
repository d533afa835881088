// Frame pre-processing (Section 5.1 of the paper): per-pixel maximum of the two latest raw frames, pixel intensity,
// 210 x 160 -> 84 x 84, newest channel of the four-frame state.  Integer arithmetic throughout.
#include "common.cuh"
#include "kernels.h"

namespace paac {

constexpr int PP_SH = 210, PP_SW = 160, PP_BAND_OUT = 12, PP_BAND_SRC = 30, PP_BANDS = 7, PP_THREADS = 256;
constexpr int PP_RAW_BYTES = PP_SH * PP_SW * 3, PP_BAND_BYTES = PP_BAND_SRC * PP_SW * 3;       // 100,800 and 14,400
static_assert(PP_BANDS * PP_BAND_OUT == FRAME_H && PP_BANDS * PP_BAND_SRC == PP_SH, "bands tile the frame");
static_assert(PP_BAND_BYTES % 16 == 0 && PP_RAW_BYTES % 16 == 0, "16-byte loads");

// One block per (band of 12 output rows, environment).  84 / 210 = 2 / 5, so a band reads exactly 30 source rows,
// which are one contiguous run of 14,400 bytes in each raw frame: whole 16-byte loads, the channel-wise maximum
// taken four bytes at a time, intensities kept in 4.8 KB of shared memory.  Rows: output row 2 m averages source rows 5 m, 5 m + 1, 5 m + 2 with weights
// 2, 2, 1 and output row 2 m + 1 rows 5 m + 2 .. 5 m + 4 with weights 1, 2, 2.  Columns: in units of 1/21 of a
// source pixel, output column x covers [40 x, 40 x + 40) and source column c covers [21 c, 21 c + 21).  The weights
// add up to 5 x 40, and (sum + 100) / 200 is the area average rounded half up.
__global__ void __launch_bounds__(PP_THREADS)
preprocess_kernel(const uint8_t* __restrict__ raw_prev, const uint8_t* __restrict__ raw_last,
                  const uint8_t* state_in, uint8_t* state_out) {
  __shared__ __align__(16) uint8_t grey[PP_BAND_SRC * PP_SW];
  const int band = blockIdx.x, e = blockIdx.y;
  const size_t src = (size_t)e * PP_RAW_BYTES + (size_t)band * PP_BAND_BYTES;
  const uint4* a4 = reinterpret_cast<const uint4*>(raw_prev + src);
  const uint4* b4 = reinterpret_cast<const uint4*>(raw_last + src);
  // sixteen pixels are 48 bytes, three 16-byte loads per frame: maximum four bytes at a time, then the intensity of
  // each pixel from its three bytes, sixteen results written as one 16-byte word
  for (int i = threadIdx.x; i < PP_BAND_SRC * PP_SW / 16; i += PP_THREADS) {
    uint32_t w[12];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      const uint4 a = __ldg(a4 + 3 * i + k), b = __ldg(b4 + 3 * i + k);
      w[4 * k] = __vmaxu4(a.x, b.x); w[4 * k + 1] = __vmaxu4(a.y, b.y); w[4 * k + 2] = __vmaxu4(a.z, b.z); w[4 * k + 3] = __vmaxu4(a.w, b.w);
    }
    uint32_t g[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      uint32_t c[3];
#pragma unroll
      for (int k = 0; k < 3; ++k) { const int byte = 3 * p + k; c[k] = (w[byte >> 2] >> (8 * (byte & 3))) & 255u; }
      g[p >> 2] |= ((77u * c[0] + 150u * c[1] + 29u * c[2] + 128u) >> 8) << (8 * (p & 3));
    }
    reinterpret_cast<uint4*>(grey)[i] = make_uint4(g[0], g[1], g[2], g[3]);
  }
  __syncthreads();
  for (int o = threadIdx.x; o < PP_BAND_OUT * FRAME_W; o += PP_THREADS) {
    const int yl = o / FRAME_W, x = o - yl * FRAME_W;
    const int m = yl >> 1, odd = yl & 1;
    const int r0 = 5 * m + 2 * odd;                              // three source rows r0 .. r0 + 2
    const int wy0 = odd ? 1 : 2, wy2 = odd ? 2 : 1;              // the middle one always weighs 2
    const int u0 = 40 * x, c0 = u0 / 21;                         // first source column; at most three are touched
    uint32_t acc = 0;
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      const int c = c0 + j;
      const int lo = max(u0, 21 * c), hi = min(u0 + 40, 21 * c + 21);
      if (hi > lo && c < PP_SW) {
        const uint32_t col = wy0 * grey[r0 * PP_SW + c] + 2u * grey[(r0 + 1) * PP_SW + c] + wy2 * grey[(r0 + 2) * PP_SW + c];
        acc += (uint32_t)(hi - lo) * col;
      }
    }
    const uint32_t v = (acc + 100u) / 200u;
    const size_t pix = ((size_t)e * FRAME_H + band * PP_BAND_OUT + yl) * FRAME_W + x;
    uint32_t out;
    if (state_in != nullptr) out = (reinterpret_cast<const uint32_t*>(state_in)[pix] >> 8) | (v << 24);    // channels are bytes, oldest first
    else out = v * 0x01010101u;
    reinterpret_cast<uint32_t*>(state_out)[pix] = out;
  }
}

// The frame stack by itself: out = (the three newest channels of prev, newest), or four copies of newest where the
// environment restarts.  A thread takes four pixels: one 16-byte load of the previous state, one 4-byte load of the
// new plane, one 16-byte store.  prev == out is allowed (every word is read before it is written, by the same thread).
constexpr int SP_THREADS = 256, SP_QUADS = FRAME_H * FRAME_W / 4;          // 1764 groups of four pixels per state
__global__ void __launch_bounds__(SP_THREADS)
stack_push_kernel(const uint8_t* prev, const uint8_t* __restrict__ newest, const uint8_t* __restrict__ restart,
                  uint8_t* out) {
  pdl_entry();
  const uint32_t e = blockIdx.y;
  const bool fresh = restart != nullptr && restart[e] != 0;
  const uint4* src = reinterpret_cast<const uint4*>(prev + (size_t)e * FRAME_BYTES);
  const uint32_t* nw = reinterpret_cast<const uint32_t*>(newest + (size_t)e * FRAME_H * FRAME_W);
  uint4* dst = reinterpret_cast<uint4*>(out + (size_t)e * FRAME_BYTES);
  for (int q = blockIdx.x * SP_THREADS + threadIdx.x; q < SP_QUADS; q += gridDim.x * SP_THREADS) {
    const uint32_t v = nw[q];
    uint4 w;
    if (fresh) {
      w = make_uint4((v & 0xFFu) * 0x01010101u, ((v >> 8) & 0xFFu) * 0x01010101u, ((v >> 16) & 0xFFu) * 0x01010101u,
                     (v >> 24) * 0x01010101u);
    } else {
      const uint4 p = src[q];
      w = make_uint4((p.x >> 8) | (v << 24), (p.y >> 8) | ((v >> 8) << 24), (p.z >> 8) | ((v >> 16) << 24),
                     (p.w >> 8) | ((v >> 24) << 24));
    }
    dst[q] = w;
  }
}

void launch_stack_push(LaunchCtx& lc, const uint8_t* prev, const uint8_t* newest, const uint8_t* restart, uint8_t* out, int n) {
  KernelScope scope(lc, KID_ENV_STEP);
  launch_kernel(lc, stack_push_kernel, dim3(2, n), SP_THREADS, 0, prev, newest, restart, out);
}

}  // namespace paac

extern "C" int paac_stack_push(const uint8_t* state_in, const uint8_t* newest, const uint8_t* restart, uint8_t* state_out,
                               int n, void* stream) {
  using namespace paac;
  if (!state_in || !newest || !state_out || n < 1 || n > 65535) return PAAC_ERR_ARG;
  if (((uintptr_t)state_in | (uintptr_t)state_out) & 15u) return PAAC_ERR_ARG;
  if ((uintptr_t)newest & 3u) return PAAC_ERR_ARG;
  stack_push_kernel<<<dim3(2, n), SP_THREADS, 0, (cudaStream_t)stream>>>(state_in, newest, restart, state_out);
  return cudaGetLastError() == cudaSuccess ? PAAC_OK : PAAC_ERR_CUDA;
}

extern "C" int paac_preprocess(const uint8_t* raw_prev, const uint8_t* raw_last, const uint8_t* state_in,
                               uint8_t* state_out, int n, void* stream) {
  using namespace paac;
  if (!raw_prev || !raw_last || !state_out || n < 1 || n > 65535) return PAAC_ERR_ARG;
  if (((uintptr_t)raw_prev | (uintptr_t)raw_last) & 15u) return PAAC_ERR_ARG;
  if (((uintptr_t)state_out | (uintptr_t)state_in) & 3u) return PAAC_ERR_ARG;
  preprocess_kernel<<<dim3(PP_BANDS, n), PP_THREADS, 0, (cudaStream_t)stream>>>(raw_prev, raw_last, state_in, state_out);
  return cudaGetLastError() == cudaSuccess ? PAAC_OK : PAAC_ERR_CUDA;
}
