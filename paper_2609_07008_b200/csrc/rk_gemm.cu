// Batched dense projection  C[M, N] = A[M, K] * B[N, K]^T  (bf16 operands, fp32 accumulation in
// TMEM, bf16 result) used for the per-head up-projection W_uv, the group-aligned slices of the
// first output projection W_a (Eq. offonline) and the shared second projection W_b
// (Eq. factorization).  One CTA per 128 x BN output tile; TMA -> 128B-swizzled shared memory
// -> tcgen05.mma (cta_group::1, M=128, N=BN, K=16) -> tcgen05.ld epilogue.
//
// A batch (blockIdx.z) selects column/row blocks of the 2-D operands: a head's or a group's
// block.  `b_skip` opens a 128-column hole in B's K axis so that the seven Local slices of a
// group's W_a are contracted in one pass while the Global head's slice is skipped.
#include <cuda_bf16.h>

#include "rk_internal.h"

namespace rk {
namespace {

constexpr int kStages = 4;
constexpr int kBM = 128;
constexpr int kBK = 64;

template <int BN>
struct GemmSmem {
  static constexpr uint32_t kABytes = kBM * kBK * 2;  // 16 KB
  static constexpr uint32_t kBBytes = BN * kBK * 2;
  static constexpr uint32_t kStageBytes = kABytes + kBBytes;
  static constexpr uint32_t kOffBars = kStages * kStageBytes;
  static constexpr uint32_t kOffTmemPtr = kOffBars + (2 * kStages + 1) * 8;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
  static constexpr uint32_t kBytes = kOffAbort + 8 + 1024;
};

enum { WG_FULL = 31, WG_EMPTY, WG_ACC };

template <int BN>
__global__ void __launch_bounds__(256, 1) rk_gemm_kernel(const __grid_constant__ GemmParams p) {
  using S = GemmSmem<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  auto full_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * s; };
  auto empty_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * (kStages + s); };
  const uint32_t acc_bar = smem_base + S::kOffBars + 8u * (2 * kStages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + S::kOffTmemPtr);
  const uint64_t limit = p.wait_ns;

  const int n0 = blockIdx.x * BN;
  const int m0 = blockIdx.y * kBM;
  const GemmBatch bt = p.batches[blockIdx.z];
  const int k_chunks = p.K / kBK;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(acc_bar, 1);
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<1>(smem_base + S::kOffTmemPtr, BN);
    tmem_relinquish<1>();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_a);
      tma_prefetch_desc(&p.tm_b);
      bool ok = true;
      for (int kc = 0; kc < k_chunks && ok; ++kc) {
        const int s = kc % kStages;
        const uint32_t use = kc / kStages;
        if (use > 0)
          ok = mbar_wait_bounded<false>(empty_bar(s), (use - 1) & 1u, limit, abort_flag, p.status, WG_EMPTY, kc);
        if (!ok) break;
        mbar_arrive_expect_tx(full_bar(s), S::kStageBytes);
        const int k = kc * kBK;
        const int bk = bt.b_col0 + k + (k >= bt.b_skip ? 128 : 0);
        const uint32_t a_dst = smem_base + s * S::kStageBytes;
        tma_load_2d(a_dst, &p.tm_a, full_bar(s), bt.a_col0 + k, m0);
        tma_load_2d(a_dst + S::kABytes, &p.tm_b, full_bar(s), bk, bt.b_row0 + n0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN, 0, 0);
      bool ok = true;
      for (int kc = 0; kc < k_chunks && ok; ++kc) {
        const int s = kc % kStages;
        ok = mbar_wait_bounded<false>(full_bar(s), (kc / kStages) & 1u, limit, abort_flag, p.status, WG_FULL, kc);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a_addr = smem_base + s * S::kStageBytes;
        const uint32_t b_addr = a_addr + S::kABytes;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_f16<1>(tmem_base, umma_desc_sw128(a_addr + k * 32, 16, 1024), umma_desc_sw128(b_addr + k * 32, 16, 1024),
                      idesc, (kc > 0 || k > 0) ? 1u : 0u);
        umma_commit_1(empty_bar(s));
      }
      if (ok) umma_commit_1(acc_bar);
    }
  } else if (warp >= 4) {
    const int L = threadIdx.x - 128;
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    bool ok = mbar_wait_bounded<false>(acc_bar, 0, limit, abort_flag, p.status, WG_ACC, 0);
    if (ok) {
      tc_fence_after_sync();
      const int row = m0 + L;
      __nv_bfloat16* crow = reinterpret_cast<__nv_bfloat16*>(p.C) + (size_t)(row < p.M ? row : 0) * p.ldc + bt.c_col0 + n0;
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 32) {
        uint32_t o[32];
        tmem_ld_x32(tmem_base + lane_base + cc, o);
        tmem_wait_ld();
        if (row < p.M && n0 + cc < p.N) {
          uint4* dst = reinterpret_cast<uint4*>(crow + cc);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(o[8 * e + 0]), __uint_as_float(o[8 * e + 1]));
            v.y = pack_bf16(__uint_as_float(o[8 * e + 2]), __uint_as_float(o[8 * e + 3]));
            v.z = pack_bf16(__uint_as_float(o[8 * e + 4]), __uint_as_float(o[8 * e + 5]));
            v.w = pack_bf16(__uint_as_float(o[8 * e + 6]), __uint_as_float(o[8 * e + 7]));
            dst[e] = v;
          }
        }
      }
    }
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc<1>(tmem_base, BN);
  }
}

}  // namespace

cudaError_t gemm_setup() {
  cudaError_t e = cudaFuncSetAttribute(rk_gemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)GemmSmem<128>::kBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(rk_gemm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)GemmSmem<256>::kBytes);
}

cudaError_t launch_gemm(const GemmParams& p, int bn, cudaStream_t stream) {
  dim3 grid((p.N + bn - 1) / bn, (p.M + kBM - 1) / kBM, p.n_batches);
  if (bn == 128)
    rk_gemm_kernel<128><<<grid, 256, GemmSmem<128>::kBytes, stream>>>(p);
  else
    rk_gemm_kernel<256><<<grid, 256, GemmSmem<256>::kBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rk
