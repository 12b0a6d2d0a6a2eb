// Batched dense projection  C[M, N] = A[M, K] * B[N, K]^T  (bf16 operands, fp32 accumulation in
// TMEM, bf16 result) used for the per-head up-projection W_uv, the group-aligned slices of the
// first output projection W_a (Eq. offonline) and the shared second projection W_b
// (Eq. factorization).  Persistent CTAs over 128 x BN output tiles; TMA -> 128B-swizzled shared
// memory -> tcgen05.mma (cta_group::1, M=128, N=BN, K=16) into one of two TMEM accumulators ->
// tcgen05.ld epilogue that overlaps the next tile's main loop.
//
// A batch selects column/row blocks of the 2-D operands: a head's or a group's block.  `b_skip`
// opens a 128-column hole in B's K axis so that the seven Local slices of a group's W_a are
// contracted in one pass while the Global head's slice is skipped.
//
// Three kernels live here: rk_gemm_kernel (this general batched form: the Local half of the
// sliced projection, the offline build, small problems), rk_gemm_pair_kernel (W_b on CTA pairs,
// cta_group::2 with M = 256) and rk_proj_fused_kernel (the Global half of the sliced projection,
// both contractions in one kernel with the 128-wide intermediate kept in shared memory).
#include <cuda_bf16.h>

#include "rk_internal.h"

namespace rk {
namespace {

constexpr int kStages = 4;
constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kGemmThreads = 256;

template <int BN>
struct GemmSmem {
  static constexpr uint32_t kABytes = kBM * kBK * 2;  // 16 KB
  static constexpr uint32_t kBBytes = BN * kBK * 2;
  static constexpr uint32_t kStageBytes = kABytes + kBBytes;
  static constexpr uint32_t kOffCStage = kStages * kStageBytes;  // two [128 rows x 128 B] output staging tiles
  static constexpr uint32_t kCStageBytes = kBM * 128;
  static constexpr uint32_t kOffBars = kOffCStage + 2 * kCStageBytes;
  // full[kStages], empty[kStages], acc_full[2], acc_empty[2]
  static constexpr uint32_t kOffTmemPtr = kOffBars + (2 * kStages + 4) * 8;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
  static constexpr uint32_t kBytes = kOffAbort + 8 + 1024;
};

enum { WG_FULL = 31, WG_EMPTY, WG_ACC_FULL, WG_ACC_EMPTY };

// Tile order.  Batched launches (head / group blocks): row block, batch, column tile, so that concurrent
// CTAs fill whole output rows.  Single-batch launches: bands of kBandRows row blocks, inside a band column
// tile first, then row block -- the CTAs of one wave then share kBandRows A row blocks and about
// sm_count / kBandRows B column tiles instead of every column tile of B at once.
constexpr int kBandRows = 16;
__device__ __forceinline__ void tile_coords(int t, int n_tiles_m, int n_tiles_n, int n_batches, int& mb, int& batch,
                                            int& nt) {
  if (n_batches > 1) {
    const int per_row_block = n_tiles_n * n_batches;
    mb = t / per_row_block;
    const int rem = t - mb * per_row_block;
    batch = rem / n_tiles_n;
    nt = rem - batch * n_tiles_n;
    return;
  }
  batch = 0;
  const int per_band = kBandRows * n_tiles_n;
  const int band = t / per_band;
  const int rows_here = min(kBandRows, n_tiles_m - band * kBandRows);  // the last band may be short
  const int rem = t - band * per_band;
  nt = rem / rows_here;
  mb = band * kBandRows + (rem - nt * rows_here);
}

// Persistent: each CTA walks output tiles t = blockIdx.x, + gridDim.x, ... ordered row block, batch, column
// tile (fastest), so the CTAs running at the same time cover a few 128-row blocks over the full output
// width: they share those A rows and the whole of B through L2, and their stores fill whole output rows
// at about the same time instead of 512-byte pieces scattered over every row of the tensor.  Two TMEM
// accumulator buffers let the epilogue of tile i overlap the main loop of tile i + 1.
template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1) rk_gemm_kernel(const __grid_constant__ GemmParams p) {
  using S = GemmSmem<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  auto full_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * s; };
  auto empty_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * (kStages + s); };
  auto acc_full_bar = [&](int b) -> uint32_t { return smem_base + S::kOffBars + 8u * (2 * kStages + b); };
  auto acc_empty_bar = [&](int b) -> uint32_t { return smem_base + S::kOffBars + 8u * (2 * kStages + 2 + b); };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + S::kOffTmemPtr);
  const uint64_t limit = p.wait_ns;

  const int n_tiles_n = (p.N + BN - 1) / BN;
  const int n_tiles_m = (p.M + kBM - 1) / kBM;
  const int tiles_per_row_block = n_tiles_n * p.n_batches;  // all batches and column tiles of one 128-row block
  const int n_tiles = tiles_per_row_block * n_tiles_m;
  const int k_chunks = p.K / kBK;
  constexpr uint32_t kTmemCols = 2 * BN;  // 256 or 512: power of two

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), 1);
      mbar_init(acc_empty_bar(b), 4);  // one arrival per epilogue warp
    }
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<1>(smem_base + S::kOffTmemPtr, kTmemCols);
    tmem_relinquish<1>();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    // ---- TMA producer (whole warp loops, one elected lane issues) ----
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_a);
      tma_prefetch_desc(&p.tm_b);
    }
    uint32_t it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      int mb, batch, nt;
      tile_coords(t, n_tiles_m, n_tiles_n, p.n_batches, mb, batch, nt);
      const int m0 = mb * kBM, n0 = nt * BN;
      const GemmBatch bt = p.batches[batch];
      for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
        const uint32_t s = it % kStages;
        if (it >= (uint32_t)kStages)
          ok = mbar_wait_bounded<false>(empty_bar(s), ((it / kStages) & 1u) ^ 1u, limit, abort_flag, p.status, WG_EMPTY, t);
        if (!ok) break;
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(s), S::kStageBytes);
          const int k = kc * kBK;
          const int bk = bt.b_col0 + k + (k >= bt.b_skip ? 128 : 0);
          const uint32_t a_dst = smem_base + s * S::kStageBytes;
          tma_load_2d(a_dst, &p.tm_a, full_bar(s), bt.a_col0 + k, m0);
          tma_load_2d(a_dst + S::kABytes, &p.tm_b, full_bar(s), bk, bt.b_row0 + n0);
        }
        __syncwarp();
      }
    }
    // drain: the tensor core must have released every stage this CTA filled
    for (uint32_t back = 1; back <= (uint32_t)kStages && ok; ++back) {
      if (it >= back) {
        const uint32_t u = it - back;
        ok = mbar_wait_bounded<false>(empty_bar(u % kStages), (u / kStages) & 1u, limit, abort_flag, p.status, WG_EMPTY, -1);
      }
    }
  } else if (warp == 1) {
    // ---- UMMA issuer (whole warp loops, one elected lane issues 4 MMAs + commit per stage) ----
    constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN, 0, 0);
    uint32_t it = 0, tile_i = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile_i) {
      const uint32_t b = tile_i & 1u;
      if (tile_i >= 2) {
        ok = mbar_wait_bounded<false>(acc_empty_bar(b), ((tile_i >> 1) & 1u) ^ 1u, limit, abort_flag, p.status,
                                      WG_ACC_EMPTY, t);
        if (!ok) break;
        tc_fence_after_sync();
      }
      const uint32_t tmem_acc = tmem_base + b * BN;
      for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
        const uint32_t s = it % kStages;
        ok = mbar_wait_bounded<false>(full_bar(s), (it / kStages) & 1u, limit, abort_flag, p.status, WG_FULL, t);
        if (!ok) break;
        const uint32_t a_addr = smem_base + s * S::kStageBytes;
        const uint32_t b_addr = a_addr + S::kABytes;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_f16<1>(tmem_acc, umma_desc_sw128(a_addr + k * 32, 16, 1024), umma_desc_sw128(b_addr + k * 32, 16, 1024),
                        idesc, (kc > 0 || k > 0) ? 1u : 0u);
          umma_commit_1(empty_bar(s));
          if (kc == k_chunks - 1) umma_commit_1(acc_full_bar(b));
        }
        __syncwarp();
      }
    }
  } else if (warp >= 4) {
    // ---- epilogue: TMEM -> registers -> bf16 -> swizzled shared-memory tile -> TMA store ----
    // One row per thread.  64 output columns at a time go through one of two 16 KB staging tiles, so the
    // stores reach memory as whole 128-byte lines of 128 rows (a thread's own 16-byte stores to rows a
    // whole matrix row apart held the short-K projections at 40 % of the memory rate).
    const int L = threadIdx.x - 128;
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    uint32_t tile_i = 0, chunk_i = 0;
    bool ok = true;
    if (L == 0) tma_prefetch_desc(&p.tm_c);
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile_i) {
      const uint32_t b = tile_i & 1u;
      int mb, batch, nt;
      tile_coords(t, n_tiles_m, n_tiles_n, p.n_batches, mb, batch, nt);
      const int m0 = mb * kBM, n0 = nt * BN;
      const GemmBatch bt = p.batches[batch];
      ok = mbar_wait_bounded<false>(acc_full_bar(b), (tile_i >> 1) & 1u, limit, abort_flag, p.status, WG_ACC_FULL, t);
      // the four warps leave together or not at all: the barriers below have no time limit of their own
      ok = named_barrier_and(1, 128, ok);
      if (!ok) break;
      tc_fence_after_sync();
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 64, ++chunk_i) {
        uint32_t o[64];
        tmem_ld_x32(tmem_base + lane_base + b * BN + cc, o);
        tmem_ld_x32(tmem_base + lane_base + b * BN + cc + 32, o + 32);
        tmem_wait_ld();
        if (cc + 64 >= BN) {  // the accumulator is in registers: hand it back to the tensor core
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acc_empty_bar(b));
        }
        const uint32_t buf = chunk_i & 1u;
        // the store that last read this staging tile (two chunks ago) must have finished reading it
        if (L == 0) bulk_wait_group_read<1>();
        named_barrier_sync(1, 128);
        uint8_t* stage = smem + S::kOffCStage + buf * S::kCStageBytes;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(o[8 * e + 0]), __uint_as_float(o[8 * e + 1]));
          v.y = pack_bf16(__uint_as_float(o[8 * e + 2]), __uint_as_float(o[8 * e + 3]));
          v.z = pack_bf16(__uint_as_float(o[8 * e + 4]), __uint_as_float(o[8 * e + 5]));
          v.w = pack_bf16(__uint_as_float(o[8 * e + 6]), __uint_as_float(o[8 * e + 7]));
          *reinterpret_cast<uint4*>(stage + sw128_offset((uint32_t)L, (uint32_t)e)) = v;
        }
        fence_proxy_async_smem();
        named_barrier_sync(1, 128);
        if (L == 0 && n0 + cc < p.N) {
          tma_store_2d(&p.tm_c, smem_base + S::kOffCStage + buf * S::kCStageBytes, bt.c_col0 + n0 + cc, m0);
          bulk_commit_group();
        }
      }
    }
    if (L == 0) bulk_wait_group<0>();  // the staging tiles must outlive the last stores
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc<1>(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------------------
// CTA-pair form for single-batch launches with N a multiple of 256 (the shared second projection W_b):
// a cluster of two CTAs owns a 256 x 256 output tile, 128 rows each, and one cta_group::2 UMMA
// (M = 256, N = 256, K = 16) per step reads A from both CTAs and one half of the B tile from each.  Every SM
// then streams 16 KB of A and 16 KB of B per k-chunk instead of 16 + 32 KB: a third less L2 -> shared
// memory traffic and shared-memory operand reads per flop at the same MMA rate, which under the board's
// power limit is clock.  No multicast load is involved: each CTA fetches its own half of B with its own TMA.
// ------------------------------------------------------------------------------------------------------
constexpr int kPairStages = 5;
struct PairSmem {
  static constexpr uint32_t kABytes = kBM * kBK * 2;  // this CTA's 128 rows of A: 16 KB
  static constexpr uint32_t kBBytes = 128 * kBK * 2;  // this CTA's 128 of the tile's 256 B rows: 16 KB
  static constexpr uint32_t kStageBytes = kABytes + kBBytes;
  static constexpr uint32_t kOffCStage = kPairStages * kStageBytes;
  static constexpr uint32_t kCStageBytes = kBM * 128;
  static constexpr uint32_t kOffBars = kOffCStage + 2 * kCStageBytes;
  // full[kPairStages], empty[kPairStages], acc_full[2], acc_empty[2]
  static constexpr uint32_t kOffTmemPtr = kOffBars + (2 * kPairStages + 4) * 8;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
  static constexpr uint32_t kBytes = kOffAbort + 8 + 1024;
};

// tile order: bands of kBandRows / 2 row-pair blocks, inside a band column tile first (see tile_coords)
__device__ __forceinline__ void pair_tile_coords(int t, int n_pair_blocks, int n_tiles_n, int& pb, int& nt) {
  constexpr int kBand = kBandRows / 2;
  const int per_band = kBand * n_tiles_n;
  const int band = t / per_band;
  const int rows_here = min(kBand, n_pair_blocks - band * kBand);
  const int rem = t - band * per_band;
  nt = rem / rows_here;
  pb = band * kBand + (rem - nt * rows_here);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
    rk_gemm_pair_kernel(const __grid_constant__ GemmParams p) {
  using S = PairSmem;
  constexpr int BN = 256;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t crank = cluster_ctarank();
  const bool leader = (crank == 0);
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  auto full_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * s; };
  auto empty_bar = [&](int s) -> uint32_t { return smem_base + S::kOffBars + 8u * (kPairStages + s); };
  auto acc_full_bar = [&](int b) -> uint32_t { return smem_base + S::kOffBars + 8u * (2 * kPairStages + b); };
  auto acc_empty_bar = [&](int b) -> uint32_t { return smem_base + S::kOffBars + 8u * (2 * kPairStages + 2 + b); };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + S::kOffTmemPtr);
  const uint64_t limit = p.wait_ns;

  const int n_tiles_n = p.N / BN;
  const int n_pair_blocks = (p.M + 2 * kBM - 1) / (2 * kBM);
  const int n_tiles = n_tiles_n * n_pair_blocks;
  const int k_chunks = p.K / kBK;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(full_bar(s), 1);   // leader's: one arrival (its own expect_tx) + the bytes of both CTAs
      mbar_init(empty_bar(s), 1);  // each CTA's: the pair's commit arrives on both
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), 1);   // each CTA's: the pair's commit arrives on both
      mbar_init(acc_empty_bar(b), 8);  // leader's: the four epilogue warps of both CTAs
    }
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<2>(smem_base + S::kOffTmemPtr, 512);
    tmem_relinquish<2>();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr_smem;

  if (warp == 0) {
    // ---- TMA producer: this CTA's A rows and its half of the B tile; bytes are counted on the leader's barrier ----
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_a);
      tma_prefetch_desc(&p.tm_b);
    }
    const GemmBatch bt = p.batches[0];
    uint32_t it = 0;
    bool ok = true;
    for (int t = pair; t < n_tiles && ok; t += n_pairs) {
      int pb, nt;
      pair_tile_coords(t, n_pair_blocks, n_tiles_n, pb, nt);
      const int m0 = pb * 2 * kBM + (int)crank * kBM, n0 = nt * BN + (int)crank * 128;
      for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
        const uint32_t s = it % kPairStages;
        if (it >= (uint32_t)kPairStages)
          ok = mbar_wait_bounded<false>(empty_bar(s), ((it / kPairStages) & 1u) ^ 1u, limit, abort_flag, p.status, WG_EMPTY, t);
        if (!ok) break;
        if (elect_one()) {
          if (leader) mbar_arrive_expect_tx(full_bar(s), 2 * S::kStageBytes);
          const uint32_t full_remote = mapa_shared(full_bar(s), 0);
          const int k = kc * kBK;
          const uint32_t a_dst = smem_base + s * S::kStageBytes;
          tma_load_2d_pair(a_dst, &p.tm_a, full_remote, bt.a_col0 + k, m0);
          tma_load_2d_pair(a_dst + S::kABytes, &p.tm_b, full_remote, bt.b_col0 + k, bt.b_row0 + n0);
        }
        __syncwarp();
      }
    }
    for (uint32_t back = 1; back <= (uint32_t)kPairStages && ok; ++back) {
      if (it >= back) {
        const uint32_t u = it - back;
        ok = mbar_wait_bounded<false>(empty_bar(u % kPairStages), (u / kPairStages) & 1u, limit, abort_flag, p.status, WG_EMPTY, -1);
      }
    }
  } else if (warp == 1) {
    // ---- UMMA issuer (leader CTA only) ----
    if (leader) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kBM, BN, 0, 0);
      uint32_t it = 0, tile_i = 0;
      bool ok = true;
      for (int t = pair; t < n_tiles && ok; t += n_pairs, ++tile_i) {
        const uint32_t b = tile_i & 1u;
        if (tile_i >= 2) {
          ok = mbar_wait_bounded<true>(acc_empty_bar(b), ((tile_i >> 1) & 1u) ^ 1u, limit, abort_flag, p.status, WG_ACC_EMPTY, t);
          if (!ok) break;
          tc_fence_after_sync();
        }
        const uint32_t tmem_acc = tmem_base + b * BN;
        for (int kc = 0; kc < k_chunks && ok; ++kc, ++it) {
          const uint32_t s = it % kPairStages;
          ok = mbar_wait_bounded<false>(full_bar(s), (it / kPairStages) & 1u, limit, abort_flag, p.status, WG_FULL, t);
          if (!ok) break;
          const uint32_t a_addr = smem_base + s * S::kStageBytes;
          const uint32_t b_addr = a_addr + S::kABytes;
          if (elect_one()) {
            const uint64_t da = umma_desc_sw128(a_addr, 16, 1024), db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_f16<2>(tmem_acc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kc > 0 || k > 0) ? 1u : 0u);
            umma_commit_2_mc(empty_bar(s), 3);
            if (kc == k_chunks - 1) umma_commit_2_mc(acc_full_bar(b), 3);
          }
          __syncwarp();
        }
      }
    }
  } else if (warp >= 4) {
    // ---- epilogue: this CTA's 128 rows of the accumulator (lane = row, 256 columns) ----
    const int L = threadIdx.x - 128;
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    const uint32_t acc_empty_remote = mapa_shared(acc_empty_bar(0), 0);
    uint32_t tile_i = 0, chunk_i = 0;
    bool ok = true;
    if (L == 0) tma_prefetch_desc(&p.tm_c);
    const GemmBatch bt = p.batches[0];
    for (int t = pair; t < n_tiles && ok; t += n_pairs, ++tile_i) {
      const uint32_t b = tile_i & 1u;
      int pb, nt;
      pair_tile_coords(t, n_pair_blocks, n_tiles_n, pb, nt);
      const int m0 = pb * 2 * kBM + (int)crank * kBM, n0 = nt * BN;
      ok = mbar_wait_bounded<false>(acc_full_bar(b), (tile_i >> 1) & 1u, limit, abort_flag, p.status, WG_ACC_FULL, t);
      ok = named_barrier_and(1, 128, ok);
      if (!ok) break;
      tc_fence_after_sync();
#pragma unroll 1
      for (int cc = 0; cc < BN; cc += 64, ++chunk_i) {
        uint32_t o[64];
        tmem_ld_x32(tmem_base + lane_base + b * BN + cc, o);
        tmem_ld_x32(tmem_base + lane_base + b * BN + cc + 32, o + 32);
        tmem_wait_ld();
        if (cc + 64 >= BN) {  // the accumulator is in registers: hand it back to the tensor cores of the pair
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(acc_empty_remote + 8u * b);
        }
        const uint32_t buf = chunk_i & 1u;
        if (L == 0) bulk_wait_group_read<1>();
        named_barrier_sync(1, 128);
        uint8_t* stage = smem + S::kOffCStage + buf * S::kCStageBytes;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(o[8 * e + 0]), __uint_as_float(o[8 * e + 1]));
          v.y = pack_bf16(__uint_as_float(o[8 * e + 2]), __uint_as_float(o[8 * e + 3]));
          v.z = pack_bf16(__uint_as_float(o[8 * e + 4]), __uint_as_float(o[8 * e + 5]));
          v.w = pack_bf16(__uint_as_float(o[8 * e + 6]), __uint_as_float(o[8 * e + 7]));
          *reinterpret_cast<uint4*>(stage + sw128_offset((uint32_t)L, (uint32_t)e)) = v;
        }
        fence_proxy_async_smem();
        named_barrier_sync(1, 128);
        if (L == 0 && m0 < p.M) {
          tma_store_2d(&p.tm_c, smem_base + S::kOffCStage + buf * S::kCStageBytes, bt.c_col0 + n0 + cc, m0);
          bulk_commit_group();
        }
      }
    }
    if (L == 0) bulk_wait_group<0>();
  }
  if (*abort_flag != 0) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc<2>(tmem_base, 512);
  }
}

}  // namespace

bool gemm_uses_pairs(int M, int N, int n_batches) { return n_batches == 1 && N % 256 == 0 && M >= 512; }

cudaError_t gemm_setup() {
  cudaError_t e = cudaFuncSetAttribute(rk_gemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)GemmSmem<128>::kBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(rk_gemm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GemmSmem<256>::kBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(rk_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairSmem::kBytes);
  return e;
}

cudaError_t launch_gemm(const GemmParams& p, int bn, int sm_count, cudaStream_t stream) {
  const long long tiles = (long long)((p.N + bn - 1) / bn) * ((p.M + kBM - 1) / kBM) * p.n_batches;
  if (tiles <= 0) return cudaSuccess;
  if (gemm_uses_pairs(p.M, p.N, p.n_batches)) {  // CTA pairs over 256 x 256 tiles (tm_b's box is 128 rows then)
    const long long pair_tiles = (long long)(p.N / 256) * ((p.M + 2 * kBM - 1) / (2 * kBM));
    const int n_pairs = (int)(pair_tiles < sm_count / 2 ? pair_tiles : sm_count / 2);
    rk_gemm_pair_kernel<<<2 * n_pairs, kGemmThreads, PairSmem::kBytes, stream>>>(p);
    return cudaGetLastError();
  }
  const int grid = (int)(tiles < sm_count ? tiles : sm_count);
  if (bn == 128)
    rk_gemm_kernel<128><<<grid, kGemmThreads, GemmSmem<128>::kBytes, stream>>>(p);
  else
    rk_gemm_kernel<256><<<grid, kGemmThreads, GemmSmem<256>::kBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rk

// ------------------------------------------------------------------------------------------------------
// Fused sliced first projection of the Global heads (Eq. offonline): per (128-row block, group g)
//   o[128 x 128]   = O_g[rows, g] W_uv[head_g]^T            (K = 512, or 576 in the output-phase variant)
//   z[128 x r_o]   = o W_a[g][:, 128 j_g : 128 j_g + 128]^T  (K = 128), written as r_o / 128 column tiles
// with o kept on chip: the first accumulator is converted to bf16 into a shared-memory tile that is the A
// operand of the second contraction, so the 128-wide intermediate never travels to memory and back.  HBM
// traffic is O_g once in and z_on_g once out.  One CTA per SM, persistent over (row block, group) tiles in that
// order; warp 0 TMA producer, warp 1 UMMA issuer, warps 4-11 two epilogue groups of four warps.
// ------------------------------------------------------------------------------------------------------
namespace rk {
namespace {

constexpr int kFpThreads = 384;
constexpr int kFpStages = 4;
struct FpSmem {
  static constexpr uint32_t kStageBytes = 32768;                   // GEMM1: A chunk + W_uv chunk; GEMM2: two W_a chunks
  static constexpr uint32_t kOffO = kFpStages * kStageBytes;       // o tile, bf16 [128 x 128] as two K-major 128B-swizzled chunks
  static constexpr uint32_t kOffCStage = kOffO + 32768;            // four 16 KB output staging tiles (two per epilogue group)
  static constexpr uint32_t kOffBars = kOffCStage + 4 * 16384;
  // full[4], empty[4], acc1_full, acc1_empty, o_ready, o_free, acc2_full[3], acc2_empty[3]
  static constexpr int kBarFull = 0, kBarEmpty = kFpStages, kBarAcc1Full = 2 * kFpStages, kBarAcc1Empty = kBarAcc1Full + 1,
                       kBarOReady = kBarAcc1Empty + 1, kBarOFree = kBarOReady + 1, kBarAcc2Full = kBarOFree + 1,
                       kBarAcc2Empty = kBarAcc2Full + 3, kNumBars = kBarAcc2Empty + 3;
  static constexpr uint32_t kOffTmemPtr = kOffBars + kNumBars * 8;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
  static constexpr uint32_t kBytes = kOffAbort + 8 + 1024;
};
enum { WF_FULL = 41, WF_EMPTY, WF_ACC1_FULL, WF_ACC1_EMPTY, WF_O_READY, WF_O_FREE, WF_ACC2_FULL, WF_ACC2_EMPTY };

__global__ void __launch_bounds__(kFpThreads, 1) rk_proj_fused_kernel(const __grid_constant__ FusedProjParams p) {
  using S = FpSmem;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  auto bar = [&](int i) -> uint32_t { return smem_base + S::kOffBars + 8u * i; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + S::kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + S::kOffTmemPtr);
  const uint64_t limit = p.wait_ns;
  const int n_mb = (p.M + kBM - 1) / kBM;
  const int n_tiles = n_mb * p.n_groups;
  const int k1_chunks = p.K1 / kBK;
  const int n_nt = p.o_rank / 128;  // column tiles of the second contraction

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kFpStages; ++s) {
      mbar_init(bar(S::kBarFull + s), 1);
      mbar_init(bar(S::kBarEmpty + s), 1);
    }
    mbar_init(bar(S::kBarAcc1Full), 1);
    mbar_init(bar(S::kBarAcc1Empty), 8);  // every epilogue warp has read its part of the first accumulator
    mbar_init(bar(S::kBarOReady), 8);     // ... and written its part of o
    mbar_init(bar(S::kBarOFree), 1);      // the second contraction of the tile has finished reading o
    for (int b = 0; b < 3; ++b) {
      mbar_init(bar(S::kBarAcc2Full + b), 1);
      mbar_init(bar(S::kBarAcc2Empty + b), 4);  // the four warps of the group that read it
    }
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<1>(smem_base + S::kOffTmemPtr, 512);
    tmem_relinquish<1>();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr_smem;
  // acc2: a ring of three 128-column buffers, so that the MMAs of the next column tiles run while a tile is being
  // stored (the issuer is up to three column tiles ahead of the epilogue)
  constexpr uint32_t kColAcc1 = 0, kColAcc2 = 128;

  // Order of the ring (producer and issuer walk it alike): the first contraction of the first tile, then for every
  // tile its second contraction's column tiles interleaved one to one with the k-chunks of the NEXT tile's first
  // contraction.  So the next tile's o accumulates while this tile's z is being stored, and the store path (the
  // slowest part: an SM writes about 26 bytes per clock) never waits for a first contraction.
  if (warp == 0) {
    // ---- TMA producer ----
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_a);
      tma_prefetch_desc(&p.tm_b1);
      tma_prefetch_desc(&p.tm_b2);
    }
    uint32_t it = 0;
    bool ok = true;
    auto acquire = [&](int t) -> bool {
      const uint32_t s = it % kFpStages;
      if (it >= (uint32_t)kFpStages)
        return mbar_wait_bounded<false>(bar(S::kBarEmpty + s), ((it / kFpStages) & 1u) ^ 1u, limit, abort_flag, p.status, WF_EMPTY, t);
      return true;
    };
    auto load1 = [&](int t, int kc) -> bool {  // k-chunk kc of tile t's first contraction: A chunk + W_uv chunk
      if (!acquire(t)) return false;
      if (elect_one()) {
        const int mb = t / p.n_groups, g = t - mb * p.n_groups;
        const GemmBatch b1 = p.batches_uv[g];
        const uint32_t s = it % kFpStages, dst = smem_base + s * S::kStageBytes;
        mbar_arrive_expect_tx(bar(S::kBarFull + s), S::kStageBytes);
        tma_load_2d(dst, &p.tm_a, bar(S::kBarFull + s), b1.a_col0 + kc * kBK, mb * kBM);
        tma_load_2d(dst + 16384, &p.tm_b1, bar(S::kBarFull + s), kc * kBK, b1.b_row0);
      }
      __syncwarp();
      ++it;
      return true;
    };
    auto load2 = [&](int t, int nt) -> bool {  // column tile nt of tile t's second contraction: two W_a chunks
      if (!acquire(t)) return false;
      if (elect_one()) {
        const int mb = t / p.n_groups, g = t - mb * p.n_groups;
        const GemmBatch b2 = p.batches_wa[g];
        const uint32_t s = it % kFpStages, dst = smem_base + s * S::kStageBytes;
        mbar_arrive_expect_tx(bar(S::kBarFull + s), S::kStageBytes);
        tma_load_2d(dst, &p.tm_b2, bar(S::kBarFull + s), b2.b_col0, b2.b_row0 + nt * 128);
        tma_load_2d(dst + 16384, &p.tm_b2, bar(S::kBarFull + s), b2.b_col0 + kBK, b2.b_row0 + nt * 128);
      }
      __syncwarp();
      ++it;
      return true;
    };
    if ((int)blockIdx.x < n_tiles)
      for (int kc = 0; kc < k1_chunks && ok; ++kc) ok = load1(blockIdx.x, kc);
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
      const int t_next = t + gridDim.x;
      const int n1 = t_next < n_tiles ? k1_chunks : 0;
      for (int j = 0; (j < n_nt || j < n1) && ok; ++j) {
        if (j < n_nt) ok = load2(t, j);
        if (ok && j < n1) ok = load1(t_next, j);
      }
    }
    for (uint32_t back = 1; back <= (uint32_t)kFpStages && ok; ++back) {
      if (it >= back) {
        const uint32_t u = it - back;
        ok = mbar_wait_bounded<false>(bar(S::kBarEmpty + u % kFpStages), (u / kFpStages) & 1u, limit, abort_flag, p.status, WF_EMPTY, -1);
      }
    }
  } else if (warp == 1) {
    // ---- UMMA issuer ----
    constexpr uint32_t idesc = umma_idesc_bf16(kBM, 128, 0, 0);
    uint32_t it = 0, tile_i = 0, use2 = 0;  // use2: column tiles issued so far (buffer = use2 % 3)
    bool ok = true;
    const uint32_t o_addr = smem_base + S::kOffO;
    auto mma1 = [&](int t, int kc) -> bool {  // one k-chunk of a first contraction into acc1
      const uint32_t s = it % kFpStages;
      if (!mbar_wait_bounded<false>(bar(S::kBarFull + s), (it / kFpStages) & 1u, limit, abort_flag, p.status, WF_FULL, t)) return false;
      const uint32_t a_addr = smem_base + s * S::kStageBytes;
      if (elect_one()) {
        const uint64_t da = umma_desc_sw128(a_addr, 16, 1024), db = umma_desc_sw128(a_addr + 16384, 16, 1024);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_f16<1>(tmem_base + kColAcc1, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kc > 0 || k > 0) ? 1u : 0u);
        umma_commit_1(bar(S::kBarEmpty + s));
        if (kc == k1_chunks - 1) umma_commit_1(bar(S::kBarAcc1Full));
      }
      __syncwarp();
      ++it;
      return true;
    };
    auto mma2 = [&](int t, int nt) -> bool {  // one column tile of a second contraction into the next acc2 buffer
      const uint32_t e = use2 % 3u, u = use2 / 3u;  // u-th use of buffer e
      if (u >= 1) {
        if (!mbar_wait_bounded<false>(bar(S::kBarAcc2Empty + e), (u - 1) & 1u, limit, abort_flag, p.status, WF_ACC2_EMPTY, t)) return false;
        tc_fence_after_sync();
      }
      const uint32_t s = it % kFpStages;
      if (!mbar_wait_bounded<false>(bar(S::kBarFull + s), (it / kFpStages) & 1u, limit, abort_flag, p.status, WF_FULL, t)) return false;
      const uint32_t b_addr = smem_base + s * S::kStageBytes;
      if (elect_one()) {
        const uint64_t da = umma_desc_sw128(o_addr, 16, 1024), db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_f16<1>(tmem_base + kColAcc2 + e * 128u, da + (uint64_t)(((k >> 2) * 16384 + (k & 3) * 32) >> 4),
                      db + (uint64_t)(((k >> 2) * 16384 + (k & 3) * 32) >> 4), idesc, k > 0 ? 1u : 0u);
        umma_commit_1(bar(S::kBarEmpty + s));
        umma_commit_1(bar(S::kBarAcc2Full + e));
        if (nt == n_nt - 1) umma_commit_1(bar(S::kBarOFree));
      }
      __syncwarp();
      ++it;
      ++use2;
      return true;
    };
    if ((int)blockIdx.x < n_tiles)
      for (int kc = 0; kc < k1_chunks && ok; ++kc) ok = mma1(blockIdx.x, kc);
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile_i) {
      const int t_next = t + gridDim.x;
      const int n1 = t_next < n_tiles ? k1_chunks : 0;
      // o of this tile is in shared memory; that also means the epilogue has read acc1, so the next tile's first
      // contraction may overwrite it
      ok = mbar_wait_bounded<false>(bar(S::kBarOReady), tile_i & 1u, limit, abort_flag, p.status, WF_O_READY, t) &&
           mbar_wait_bounded<false>(bar(S::kBarAcc1Empty), tile_i & 1u, limit, abort_flag, p.status, WF_ACC1_EMPTY, t);
      if (!ok) break;
      tc_fence_after_sync();
      for (int j = 0; (j < n_nt || j < n1) && ok; ++j) {
        if (j < n_nt) ok = mma2(t, j);
        if (ok && j < n1) ok = mma1(t_next, j);
      }
    }
  } else if (warp >= 4) {
    // ---- epilogue: group e owns o chunk e (64 columns of the first accumulator) and every other column tile ----
    const int e = (warp - 4) >> 2;
    const int L = (threadIdx.x - 128) & 127;
    const int bar_id = 1 + e;
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    uint32_t tile_i = 0, chunk_i = 0;
    bool ok = true;
    if (L == 0) tma_prefetch_desc(&p.tm_c);
    // o of tile number i (in this CTA's sequence): first accumulator -> bf16 -> shared-memory A tile of the second
    // contraction.  It runs before the group's last column tile of the previous row-block tile, so that the
    // second contraction of the next tile is already under way when the stores of this one end.
    auto convert_o = [&](uint32_t i, int t) -> bool {
      bool good = mbar_wait_bounded<false>(bar(S::kBarAcc1Full), i & 1u, limit, abort_flag, p.status, WF_ACC1_FULL, t);
      if (good && i >= 1)
        good = mbar_wait_bounded<false>(bar(S::kBarOFree), (i - 1) & 1u, limit, abort_flag, p.status, WF_O_FREE, t);
      good = named_barrier_and(bar_id, 128, good);
      if (!good) return false;
      tc_fence_after_sync();
      uint32_t o[64];
      tmem_ld_x32(tmem_base + lane_base + kColAcc1 + 64u * e, o);
      tmem_ld_x32(tmem_base + lane_base + kColAcc1 + 64u * e + 32, o + 32);
      tmem_wait_ld();
      tc_fence_before_sync();
      uint8_t* dst = smem + S::kOffO + e * 16384;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(o[8 * c + 0]), __uint_as_float(o[8 * c + 1]));
        v.y = pack_bf16(__uint_as_float(o[8 * c + 2]), __uint_as_float(o[8 * c + 3]));
        v.z = pack_bf16(__uint_as_float(o[8 * c + 4]), __uint_as_float(o[8 * c + 5]));
        v.w = pack_bf16(__uint_as_float(o[8 * c + 6]), __uint_as_float(o[8 * c + 7]));
        *reinterpret_cast<uint4*>(dst + sw128_offset((uint32_t)L, (uint32_t)c)) = v;
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(S::kBarAcc1Empty));
        mbar_arrive(bar(S::kBarOReady));
      }
      return true;
    };
    if ((int)blockIdx.x < n_tiles) ok = convert_o(0, blockIdx.x);
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile_i) {
      const int mb = t / p.n_groups, g = t - mb * p.n_groups;
      const GemmBatch b2 = p.batches_wa[g];
      const int m0 = mb * kBM;
      const int t_next = t + gridDim.x;
      // ---- z: this group's column tiles ----
      for (int nt = e; nt < n_nt && ok; nt += 2) {
        if (nt + 2 >= n_nt && t_next < n_tiles) {  // before this group's last column tile: the next tile's o
          ok = convert_o(tile_i + 1, t_next);
          if (!ok) break;
        }
        const uint32_t q = tile_i * (uint32_t)n_nt + (uint32_t)nt;  // column tiles are issued in this order
        const uint32_t b = q % 3u, u = q / 3u;
        ok = mbar_wait_bounded<false>(bar(S::kBarAcc2Full + b), u & 1u, limit, abort_flag, p.status, WF_ACC2_FULL, t);
        ok = named_barrier_and(bar_id, 128, ok);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll 1
        for (int cc = 0; cc < 128; cc += 64, ++chunk_i) {
          uint32_t o[64];
          tmem_ld_x32(tmem_base + lane_base + kColAcc2 + 128u * b + cc, o);
          tmem_ld_x32(tmem_base + lane_base + kColAcc2 + 128u * b + cc + 32, o + 32);
          tmem_wait_ld();
          if (cc == 64) {
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(S::kBarAcc2Empty + b));
          }
          const uint32_t buf = 2u * e + (chunk_i & 1u);
          if (L == 0) bulk_wait_group_read<1>();
          named_barrier_sync(bar_id, 128);
          uint8_t* stage = smem + S::kOffCStage + buf * 16384;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(o[8 * c + 0]), __uint_as_float(o[8 * c + 1]));
            v.y = pack_bf16(__uint_as_float(o[8 * c + 2]), __uint_as_float(o[8 * c + 3]));
            v.z = pack_bf16(__uint_as_float(o[8 * c + 4]), __uint_as_float(o[8 * c + 5]));
            v.w = pack_bf16(__uint_as_float(o[8 * c + 6]), __uint_as_float(o[8 * c + 7]));
            *reinterpret_cast<uint4*>(stage + sw128_offset((uint32_t)L, (uint32_t)c)) = v;
          }
          fence_proxy_async_smem();
          named_barrier_sync(bar_id, 128);
          if (L == 0) {
            tma_store_2d(&p.tm_c, smem_base + S::kOffCStage + buf * 16384, b2.c_col0 + nt * 128 + cc, m0);
            bulk_commit_group();
          }
        }
      }
    }
    if (L == 0) bulk_wait_group<0>();
  }
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc<1>(tmem_base, 512);
  }
}

}  // namespace

cudaError_t proj_fused_setup() {
  return cudaFuncSetAttribute(rk_proj_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FpSmem::kBytes);
}

cudaError_t launch_proj_fused(const FusedProjParams& p, int sm_count, cudaStream_t stream) {
  const long long tiles = (long long)((p.M + kBM - 1) / kBM) * p.n_groups;
  if (tiles <= 0) return cudaSuccess;
  const int grid = (int)(tiles < sm_count ? tiles : sm_count);
  rk_proj_fused_kernel<<<grid, kFpThreads, FpSmem::kBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rk
