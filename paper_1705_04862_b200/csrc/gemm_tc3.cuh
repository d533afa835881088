// The same generic contraction as gemm_simt.cuh on the tensor cores, accurate to float level:
//   C(m, n) = sum_k A(m, k) * B(n, k)
// with every float operand split into two TF32 pieces, x = hi + lo (hi = tf32(x), lo = tf32(x - hi), round to nearest,
// together 22 significant bits), and three tcgen05 passes (kind::tf32) per block of 32 k into a float accumulator in
// tensor memory, the blocks' sums then added in registers:
//   hi*hi + hi*lo + lo*hi      (the dropped lo*lo term and the rounding of lo are below 2^-21 of a product).
// Two bfloat16 pieces (16 bits) are not enough here: errors of 1e-5 flip about one ReLU unit per update of the small
// network and the free-running trajectories leave the float tolerance within three updates.
// Operands come from the same index functors and results go to the same epilogue functors as the CUDA-core
// kernel, so every layer of the float path (forward, data and weight gradients, split-k included) can run through it.
// One CTA per 128 x 64 output tile and k split; 544 threads:
//   warps 0-15 producers: per block of 32 k a thread evaluates two 16-byte chunks (four k of one row) of A and one of B,
//              splits them, and writes them into the hi and the lo image (128-byte rows, 128-byte swizzle); then the
//              thread (= tile row, one of four column groups) adds its sixteen columns of the finished product of
//              the block before to a running sum in registers (round to nearest), and after the last block calls
//              the epilogue functor;
//   warp 16    lane 0 issues twelve MMAs per block (three passes of four K = 8 steps, small terms first) into one of
//              two accumulators, starting each block from zero, and commits.
// Only the twelve steps of one block are summed inside the tensor core, whose accumulation does not round to nearest;
// summed there over a whole contraction (thousands of steps) the result was eight times further from the exact
// one than the CUDA-core kernel's.
// Every wait is bounded.  The contractions of the float configurations are small (4 to 160 rows in the fully connected
// layers), so most of a 128-row tile is padding there: this path exists for its arithmetic, not for speed.
#pragma once
#include "gemm_simt.cuh"
#include "tc_common.cuh"

namespace paac {

constexpr int T3_BM = 128, T3_BN = 64, T3_BK = 32, T3_STAGES = 2;
constexpr int T3_PWARPS = 16, T3_THREADS = (T3_PWARPS + 1) * 32;      // producer warps + the issuing warp
constexpr int T3_GROUPS = T3_PWARPS / 4, T3_COLS = T3_BN / T3_GROUPS;
constexpr uint32_t T3_A_BYTES = T3_BM * 128, T3_B_BYTES = T3_BN * 128, T3_STAGE_BYTES = 2 * T3_A_BYTES + 2 * T3_B_BYTES;
constexpr int T3_SMEM = T3_STAGES * T3_STAGE_BYTES + 1024;

struct T3Shared {
  uint64_t full[T3_STAGES], empty[T3_STAGES], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  volatile uint32_t abort;
};

// Instruction descriptor for kind::tf32: float accumulator, A and B in TF32 format (code 2), both K-major.
__host__ __device__ constexpr uint32_t make_idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
static_assert(T3_COLS == 16, "the accumulator read below takes sixteen columns");
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t r[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
// four floats -> four hi pieces and four lo pieces (32-bit containers)
__device__ __forceinline__ void split_tf32x4(const float (&x)[4], uint4& hi, uint4& lo) {
  uint32_t h[4], l[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    h[j] = to_tf32(x[j]);
    l[j] = to_tf32(x[j] - __uint_as_float(h[j]));
  }
  hi = make_uint4(h[0], h[1], h[2], h[3]);
  lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <class LA, class LB, class EP>
__global__ void __launch_bounds__(T3_THREADS)
gemm_tc3_kernel(int M, int N, int K, int k_per_split, LA la, LB lb, EP ep, uint32_t* error_word) {
  using namespace tc;
  pdl_entry();
  extern __shared__ uint8_t dyn_smem[];
  __shared__ T3Shared sh;
  const uint32_t tiles = (smem_u32(dyn_smem) + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * T3_BM, n0 = blockIdx.y * T3_BN, split = blockIdx.z;
  const int k_begin = split * k_per_split, k_end = min(K, k_begin + k_per_split);
  const int num_kb = (k_end - k_begin + T3_BK - 1) / T3_BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < T3_STAGES; ++s) { mbar_init(&sh.full[s], T3_PWARPS); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.acc_full[a], 1); mbar_init(&sh.acc_empty[a], T3_PWARPS); }
    sh.abort = 0u;
    fence_barrier_init();
  }
  if (warp == T3_PWARPS) tmem_alloc(&sh.tmem_base, 2 * T3_BN);
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp < T3_PWARPS) {
    // ---------------- producers, and the running sum over the k blocks ----------------
    // thread = (tile row, group): the group picks which 16-byte chunks of the row it fills and which accumulator
    // columns it sums; the row is also the thread's lane of tensor memory (warp % 4 selects the 32-lane quarter)
    const int row = threadIdx.x & 127, grp = threadIdx.x >> 7;
    const int m = m0 + row;
    float sum[T3_COLS];
#pragma unroll
    for (int j = 0; j < T3_COLS; ++j) sum[j] = 0.f;
    bool alive = true;
    // adds the finished product of block `kb` (one of the two accumulators) to the running sum and hands the
    // accumulator back to the issuer
    auto collect = [&](int kb) -> bool {
      const int a = kb & 1;
      const bool ok = mbar_wait(&sh.acc_full[a], (kb >> 1) & 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!__all_sync(0xffffffffu, ok)) return false;
      tcgen05_fence_after();
      uint32_t r[T3_COLS];
      tmem_ld_32x16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + a * T3_BN + grp * T3_COLS, r);
#pragma unroll
      for (int j = 0; j < T3_COLS; ++j) sum[j] += __uint_as_float(r[j]);
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.acc_empty[a]);
      return true;
    };
    // Operand values of one k block are fetched into registers one block ahead of their use, so that the loads'
    // latency overlaps the wait for the stage, the read-out of the accumulator and the MMAs of the block before.
    // Which 16-byte chunks (four k of one row) a thread fetches follows the operand's layout in memory, so that a
    // warp's loads are contiguous: eight neighbouring lanes take the eight chunks of one row where k is contiguous,
    // 32 lanes take 32 rows where the row index is.
    constexpr int A_SLOTS = T3_BM * 8 / (T3_PWARPS * 32);          // chunks of A per thread (2); B has one
    static_assert(T3_BN * 8 == T3_PWARPS * 32, "one chunk of B per producer thread");
    int a_row[A_SLOTS], a_chunk[A_SLOTS];
#pragma unroll
    for (int i = 0; i < A_SLOTS; ++i) {
      const int slot = (int)threadIdx.x + i * T3_PWARPS * 32;
      if (LA::K_CONTIG) { a_row[i] = slot >> 3; a_chunk[i] = slot & 7; }
      else { a_row[i] = slot & (T3_BM - 1); a_chunk[i] = slot / T3_BM; }
    }
    const int b_row = LB::K_CONTIG ? (int)threadIdx.x >> 3 : (int)threadIdx.x & (T3_BN - 1);
    const int b_chunk = LB::K_CONTIG ? (int)threadIdx.x & 7 : (int)threadIdx.x / T3_BN;
    float xa[A_SLOTS][4], xb[4];
    auto fetch = [&](int kb) {
      const int k0 = k_begin + kb * T3_BK;
#pragma unroll
      for (int i = 0; i < A_SLOTS; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int k = k0 + 4 * a_chunk[i] + j;
          xa[i][j] = (m0 + a_row[i] < M && k < k_end) ? la(m0 + a_row[i], k) : 0.f;
        }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int k = k0 + 4 * b_chunk + j;
        xb[j] = (n0 + b_row < N && k < k_end) ? lb(n0 + b_row, k) : 0.f;
      }
    };
    if (num_kb > 0) fetch(0);
    for (int kb = 0; kb < num_kb; ++kb) {
      const int s = kb % T3_STAGES;
      const bool ok = mbar_wait(&sh.empty[s], ((kb / T3_STAGES) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_EMPTY);
      if (!__all_sync(0xffffffffu, ok)) { alive = false; break; }
      const uint32_t a_hi = tiles + s * T3_STAGE_BYTES, a_lo = a_hi + T3_A_BYTES, b_hi = a_lo + T3_A_BYTES, b_lo = b_hi + T3_B_BYTES;
      uint4 hi, lo;
#pragma unroll
      for (int i = 0; i < A_SLOTS; ++i) {
        split_tf32x4(xa[i], hi, lo);
        const uint32_t off = sw128_offset((uint32_t)a_row[i], (uint32_t)a_chunk[i]);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_hi + off), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_lo + off), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
      }
      {
        split_tf32x4(xb, hi, lo);
        const uint32_t off = sw128_offset((uint32_t)b_row, (uint32_t)b_chunk);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(b_hi + off), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(b_lo + off), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.full[s]);
      if (kb + 1 < num_kb) fetch(kb + 1);
      if (kb >= 1 && !collect(kb - 1)) { alive = false; break; }
    }
    if (alive && num_kb > 0 && collect(num_kb - 1) && m < M) {
      // ---------------- epilogue ----------------
#pragma unroll
      for (int j = 0; j < T3_COLS; ++j)
        if (n0 + grp * T3_COLS + j < N) ep(m, n0 + grp * T3_COLS + j, sum[j], split);
    }
  } else if (lane == 0) {
    // ---------------- MMA issuer ----------------
    constexpr uint32_t idesc = make_idesc_tf32(T3_BM, T3_BN);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % T3_STAGES, a = kb & 1;
      ok = mbar_wait(&sh.full[s], (kb / T3_STAGES) & 1, &sh.abort, error_word, ERR_WAIT_FULL) &&
           mbar_wait(&sh.acc_empty[a], ((kb >> 1) & 1) ^ 1, &sh.abort, error_word, ERR_WAIT_ACC);
      if (!ok) break;
      tcgen05_fence_after();
      const uint32_t a_hi = tiles + s * T3_STAGE_BYTES, a_lo = a_hi + T3_A_BYTES, b_hi = a_lo + T3_A_BYTES, b_lo = b_hi + T3_B_BYTES;
#pragma unroll
      for (int pass = 0; pass < 3; ++pass) {
        const uint32_t pa = pass == 0 ? a_lo : a_hi, pb = pass == 1 ? b_lo : b_hi;      // small terms first
#pragma unroll
        for (int k = 0; k < T3_BK / 8; ++k)
          mma_tf32(tmem + a * T3_BN, make_smem_desc(pa + k * 32, 0, 1024, SWIZZLE_128B),
                   make_smem_desc(pb + k * 32, 0, 1024, SWIZZLE_128B), idesc, (pass | k) != 0 ? 1u : 0u);
      }
      mma_commit(&sh.empty[s]);
      mma_commit(&sh.acc_full[a]);
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if (warp == T3_PWARPS) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem, 2 * T3_BN);
  }
}

// same split geometry as gemm_simt (the callers size their partial-sum scratch and their reductions by it)
template <class LA, class LB, class EP>
inline void gemm_tc3(LaunchCtx& lc, int kid, int M, int N, int K, int splits, LA la, LB lb, EP ep) {
  if (M <= 0 || N <= 0 || K <= 0) return;
  auto kern = gemm_tc3_kernel<LA, LB, EP>;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T3_SMEM);
    configured = true;
  }
  KernelScope scope(lc, kid);
  int kps = (K + splits - 1) / splits;
  kps = (kps + SG_BK - 1) / SG_BK * SG_BK;
  dim3 grid((M + T3_BM - 1) / T3_BM, (N + T3_BN - 1) / T3_BN, (K + kps - 1) / kps);
  launch_kernel(lc, kern, grid, T3_THREADS, T3_SMEM, M, N, K, kps, la, lb, ep, lc.error_word);
}

// the float path's contractions: on the CUDA cores, or (option) through the three-pass tensor-core kernel
template <class LA, class LB, class EP>
inline void gemm_f32(LaunchCtx& lc, int kid, int M, int N, int K, int splits, LA la, LB lb, EP ep) {
  if (lc.fp32_tensor_cores && lc.error_word != nullptr) gemm_tc3(lc, kid, M, N, K, splits, la, lb, ep);
  else gemm_simt(lc, kid, M, N, K, splits, la, lb, ep);
}

}  // namespace paac
