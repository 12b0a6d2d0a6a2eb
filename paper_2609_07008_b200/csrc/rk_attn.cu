// Absorbed-MLA attention over the packed latent stream for one pass (Global heads x all rows,
// or Local heads x protected rows) -- Algorithm 2: for every document segment rotate the
// query's rope sub-vector by -delta_i (fused into the Q tile in shared memory), attend the
// segment's canonical keys with the causal limit in the canonical frame, and merge segments
// with the running log-sum-exp recurrence (max / sum / rescale) inside the CTA.
//
// Mapping to sm_100a.  A CTA pair (cluster of 2) owns 128 consecutive query rows
// ((token, head) pairs; 64 per CTA) and issues cta_group::2 UMMAs with M=128, N=256:
//   S[64 x 256 keys]  = Q[64 x 576] K^T         9 k-chunks of 64 (8 latent, then the rotated rope)
//   O[64 x 512]      += P[64 x 256] V[256 x 512] two N=256 halves
// In that UMMA shape each CTA's 64 accumulator rows fold onto all 128 TMEM lanes (lanes 0-63:
// columns [0,N/2), lanes 64-127: columns [N/2,N)), so O takes 256 columns and the score buffer S
// 128.  The remaining 128 columns hold latent dims 256-511 of the Q tile (bf16 pairs, the rows in
// both lane halves) and feed the QK^T MMAs of those dims as a tensor-memory A operand; only dims
// 0-255 and the rope chunk of Q stay in shared memory.  The 32 KB that frees pay for a fourth
// 32 KB stage of the K/V ring, which is what keeps the tensor pipe fed while the per-SM L2 -> SMEM
// rate (about 76 B/clk) trails the MMA's appetite within a tile.  S is single-buffered: QK^T of
// the next key tile follows the PV of the previous one in the issue order, and by then the
// softmax warps have long read S into registers (the s_free barrier states it).
// The B operand is split across the pair: for QK^T each CTA streams its 128 keys of the tile,
// for PV its 128 of each 256 output dims.  The same [128 keys x 64 dims] 128B-swizzled TMA box
// serves as K-major B (QK^T) and MN-major B (PV).
//
// Warp roles per CTA (384 threads): warp 0 TMA producer, warp 1 UMMA issuer (leader CTA only),
// warp 2 query relocation, warps 4-11 softmax / correction / epilogue (two warps per TMEM lane
// quarter, each owning half of the columns).  At the start of a row tile the upper Q half lands
// in one ring stage and the softmax warps copy it into TMEM (tcgen05.st) before their first scores.
//
// The kernel is a template: <kPhase = 0> is what the lines above describe.  <kPhase = 1> is the
// output-phase variant, whose value is the whole stored row (latent and rope dims): a second small
// accumulator for the 64 rope dims of O, turned into the next segment's frame at every segment
// switch (RestorePhase of Algorithm 2 folded into the running merge) and by R(delta - pos) in the
// epilogue (the inverse output RoPE of Eq. offonline); see Cfg for how it fits.
#include <cuda_bf16.h>

#include "rk_internal.h"

namespace rk {
namespace {

constexpr int kAttnThreads = 384;       // 4 role warps + 8 softmax warps
constexpr uint32_t kChunkBytes = 16384;  // 128 keys x 64 dims bf16
constexpr uint32_t kStageBytes = 2 * kChunkBytes;
constexpr uint32_t kQChunkBytes = 8192;  // 64 rows x 64 dims bf16

// Two instantiations share this file.  The plain one (values = the 512-wide latent) keeps latent dims
// 256-511 of the Q tile in tensor memory (128 columns); that pays for the fourth stage of the ring.  The
// output-phase one (values = the whole stored row, latent and rope dims; Eq. offonline's inverse output
// RoPE, Algorithm 2's RestorePhase) needs 32 more accumulator columns for the rope part of O, so only 96
// columns are left for Q: latent dims 320-511.  The 8 KB that its fifth shared-memory Q chunk costs come from
// the pristine rope chunk, which in this instantiation lives in the relocation warp's registers (it lands in
// the second rotated-rope buffer and is picked up from there at the start of a row tile).  Both run four stages.
template <bool kPhase>
struct Cfg {
  static constexpr int kStages = 4;                       // ring of 32 KB stages (two 16 KB TMA boxes each)
  static constexpr int kQSmemChunks = kPhase ? 5 : 4;     // 64-dim latent chunks of Q kept in shared memory
  static constexpr int kQTmemChunks = 8 - kQSmemChunks;   // ... kept in tensor memory (32 columns each)
  static constexpr int kStagesPerKeyTile = kPhase ? 10 : 9;  // K: 5, V: 4, rope part of V: 1
  static constexpr int kOW = kPhase ? kDQK : kDLatent;    // width of an output row
  // shared memory map (offsets from a 1024-byte aligned base)
  static constexpr uint32_t kOffQLat = 0;
  // plain: rope chunk as loaded, then 2 rotated rope chunks.  output-phase: no buffer for the chunk as loaded;
  // it lands in the second rotated buffer
  static constexpr uint32_t kOffQRot = kOffQLat + (kQSmemChunks + (kPhase ? 0 : 1)) * kQChunkBytes;
  static constexpr uint32_t kOffQPristine = kPhase ? kOffQRot + kQChunkBytes : kOffQLat + kQSmemChunks * kQChunkBytes;
  static constexpr uint32_t kOffP = kOffQRot + 2 * kQChunkBytes;                     // 4 sub-chunks [64 x 64 keys]
  static constexpr uint32_t kOffRing = kOffP + 4 * kQChunkBytes;
  static constexpr uint32_t kOffBars = kOffRing + kStages * kStageBytes;
  // barrier indices (8 bytes each)
  static constexpr int kBarQFull = 0, kBarQFree = 1, kBarQrReady = 2 /*2*/, kBarQrFree = 4 /*2*/, kBarRingFull = 6,
                       kBarRingEmpty = kBarRingFull + kStages, kBarSFull = kBarRingEmpty + kStages,
                       kBarSFree = kBarSFull + 1, kBarPReady = kBarSFree + 1, kBarPvDone = kBarPReady + 1,
                       kBarQhFull = kBarPvDone + 1, kBarQhDone = kBarQhFull + 1, kNumBars = kBarQhDone + 1;
  static constexpr uint32_t kOffTmemPtr = kOffBars + kNumBars * 8;
  static constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
  static constexpr uint32_t kOffXchg = kOffAbort + 8;         // u64 [2 parity][4 parts][64]: (seq << 32) | value
  static constexpr uint32_t kSmemUsed = kOffXchg + 2 * 4 * 64 * 8;
  static constexpr uint32_t kSmemBytes = kSmemUsed + 1024;    // + alignment slack
};

// TMEM columns
constexpr uint32_t kColO = 0;     // two halves of 128 columns
constexpr uint32_t kColS = 256;   // one 128-column score buffer
constexpr uint32_t kColQ = 384;   // plain: latent dims 256-511 of the Q tile as a TMEM A operand (both lane halves hold the rows)
constexpr uint32_t kColOr = 384;  // output-phase: the 64 rope dims of O (N = 64 folds onto 32 columns)
constexpr uint32_t kColQp = 416;  // output-phase: latent dims 320-511 of the Q tile (96 columns)

constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 256, 0, 0);
constexpr uint32_t kIdescPV = umma_idesc_bf16(128, 256, 0, 1);
constexpr uint32_t kIdescPVr = umma_idesc_bf16(128, 64, 0, 1);  // rope part of the value: 32 dims per CTA

// wait tags reported on timeout
enum { W_QFULL = 1, W_QFREE, W_QRREADY, W_QRFREE, W_RINGFULL, W_RINGEMPTY, W_SFULL, W_PREADY, W_PVDONE, W_DRAIN, W_SFREE, W_QHFULL, W_QHDONE };

struct SegIter {
  // Iterates the segments a row tile can see; kmax = number of canonical keys of the segment that
  // any row of the tile may see.  Online mode: everything at request positions <= the tile's
  // largest position.  Isolated mode (offline artifact build): only the segments the tile's own
  // packed rows [prow0, prow1] lie in, each up to the tile's last row in it.
  const AttnParams& p;
  int maxpos, prow0, prow1;
  int seg;
  int kmax;
  __device__ SegIter(const AttnParams& p_, const AttnWorkItem& item) : p(p_), maxpos(item.maxpos), seg(-1), kmax(0) {
    const int r0 = item.tile * kAttnRowsPerPair;
    int r1 = r0 + kAttnRowsPerPair - 1;
    if (r1 > p.n_flat - 1) r1 = p.n_flat - 1;
    prow0 = p.row_base + r0 / p.hpt;
    prow1 = p.row_base + r1 / p.hpt;
    if (p.isolated) {
      // start at the segment that holds the tile's first packed row (binary search) instead of walking
      // the table from the top: a row tile of a document build sees a handful of key tiles only, and
      // every role walks the table a few times per row tile
      int lo = 0, hi = p.n_segs - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (p.seg_off[mid] <= prow0) lo = mid; else hi = mid - 1;
      }
      seg = lo - 1;
    }
  }
  __device__ bool next() {
    while (++seg < p.n_segs) {
      const int lo = p.seg_off[seg], hi = p.seg_off[seg + 1];
      if (p.isolated) {
        if (lo > prow1) { seg = p.n_segs; return false; }  // past the tile's last row: nothing further overlaps
        if (prow1 < lo || prow0 >= hi) { kmax = 0; continue; }
        kmax = (prow1 < hi ? prow1 : hi - 1) - lo + 1;
      } else {
        const int lim = maxpos - p.seg_delta[seg] + 1;
        kmax = lim < hi - lo ? lim : hi - lo;
      }
      if (kmax > 0) return true;
    }
    return false;
  }
};

__device__ __forceinline__ AttnWorkItem get_work(const AttnParams& p, int w) {
  if (p.work != nullptr) return p.work[w];
  AttnWorkItem it;  // natural order (isolated mode has no host-built list)
  it.tile = w;
  it.maxpos = 0;
  return it;
}

// Ring bookkeeping shared by the producer and the UMMA issuer: both walk the same stage
// sequence.  A stage holds two 16 KB boxes: two 64-dim K chunks (QK^T), the single rope chunk,
// or the two 64-dim halves of this CTA's 128 output dims (PV; 16 KB apart = the descriptor's
// leading byte offset).
template <int kStages>
struct RingPos {
  uint32_t it = 0;  // stages used so far
  __device__ uint32_t stage() const { return it % kStages; }
  __device__ uint32_t parity() const { return (it / kStages) & 1u; }
  __device__ void advance() { ++it; }
};

// number of key tiles a row tile walks through (all visible segments)
__device__ __forceinline__ int count_key_tiles(const AttnParams& p, const AttnWorkItem& item) {
  SegIter it(p, item);
  int n = 0;
  while (it.next()) n += (it.kmax + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
  return n;
}

// The four threads that share one query row (TMEM lanes m and m + 64, two column halves each,
// all in different warps) combine one float through shared memory.  Sequence-tagged and
// double-buffered by sequence parity; the poll is bounded like every other wait here.
template <bool kMax>
__device__ __forceinline__ bool quad_exchange(volatile unsigned long long* xbuf, int part, int m, uint32_t seq,
                                              float mine, float& combined, uint64_t limit_ns,
                                              volatile int* abort_flag, DeviceStatus* st, int aux) {
  volatile unsigned long long* base = xbuf + (seq & 1u) * 256;
  base[part * 64 + m] = ((unsigned long long)seq << 32) | (unsigned long long)__float_as_uint(mine);
  float acc = mine;
#pragma unroll
  for (int o = 1; o < 4; ++o) {
    volatile unsigned long long* theirs = base + ((part + o) & 3) * 64 + m;
    uint64_t t0 = 0;
    uint32_t spins = 0;
    while (true) {
      const unsigned long long v = *theirs;
      if ((uint32_t)(v >> 32) == seq) {
        const float x = __uint_as_float((uint32_t)v);
        acc = kMax ? fmaxf(acc, x) : acc + x;
        break;
      }
      if ((++spins & 0xff) == 0) {
        if (*abort_flag != 0) return false;
        if (t0 == 0) t0 = globaltimer_ns();
        if (globaltimer_ns() - t0 > limit_ns) {
          *abort_flag = 1;
          report_timeout(st, 20, aux);
          return false;
        }
      }
    }
  }
  combined = acc;
  return true;
}
#define quad_exchange_max quad_exchange<true>
#define quad_exchange_sum quad_exchange<false>

// (cos, sin) of d * theta_j for an integer position difference d (any sign, up to 2^30): the angle is
// reduced in double precision in units of turns (theta_j / 2 pi is a host-computed double), so that the
// float sincospi sees an argument in [-1, 1] whatever the size of d
__device__ __forceinline__ void rope_cs(const AttnParams& p, int d, int j, float& c, float& s) {
  const double t = (double)d * p.rope_turns[j];
  const float f = (float)(t - rint(t));
  sincospif(2.f * f, &s, &c);
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace

// kStarve: test instantiation whose load warp leaves every ring stage empty, so that the consumers'
// bounded waits expire and the kernel returns with RK_ERR_TIMEOUT in the status word (the test of the
// timeout path launches it; the production instantiation carries no such switch in its loops).
// kPhase: the output-phase instantiation (see Cfg).
template <bool kPhase, bool kStarve>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kAttnThreads, 1)
    rk_mla_attn_kernel(const __grid_constant__ AttnParams p) {
  using C = Cfg<kPhase>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t crank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const bool leader = (crank == 0);

  auto bar = [&](int i) -> uint32_t { return smem_base + C::kOffBars + 8u * i; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + C::kOffTmemPtr);
  const uint64_t limit = p.wait_ns;

  for (int i = threadIdx.x; i < 512; i += kAttnThreads) reinterpret_cast<volatile unsigned long long*>(smem + C::kOffXchg)[i] = 0ull;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(C::kBarQFull), 1);
    mbar_init(bar(C::kBarQFree), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(C::kBarQrReady + b), 2);
      mbar_init(bar(C::kBarQrFree + b), 1);
    }
    mbar_init(bar(C::kBarSFull), 1);
    mbar_init(bar(C::kBarSFree), 16);   // every softmax warp of the pair has read the score buffer
    mbar_init(bar(C::kBarQhFull), 1);   // this CTA's upper Q half has landed in its ring stage
    mbar_init(bar(C::kBarQhDone), 16);  // every softmax warp of the pair has moved its part into TMEM
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar(C::kBarRingFull + s), 1);
      mbar_init(bar(C::kBarRingEmpty + s), 1);
    }
    mbar_init(bar(C::kBarPReady), 16);
    mbar_init(bar(C::kBarPvDone), 1);
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<2>(smem_base + C::kOffTmemPtr, 512);
    tmem_relinquish<2>();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_ptr_smem;

  // =====================================================================================
  if (warp == 0) {
    // ------------------------------ TMA producer (whole warp loops; one elected lane issues) ------
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_q);
      tma_prefetch_desc(&p.tm_kv);
    }
    RingPos<kStages> rp;
    uint32_t qfree_phase = 0;
    bool ok = true;
    int n_done = 0;
    const uint64_t pol_kv = l2_policy_evict_last(), pol_q = l2_policy_evict_first();
    // fills one stage with one or two boxes; every lane waits, one lane issues
    auto fill = [&](int col0, int col1, int row, int w) -> bool {
      const uint32_t s = rp.stage();
      if (rp.it >= (uint32_t)kStages) {
        if (!mbar_wait_bounded<false>(bar(C::kBarRingEmpty + s), rp.parity() ^ 1u, limit, abort_flag, p.status,
                                      W_RINGEMPTY, w))
          return false;
      }
      if constexpr (kStarve) {  // leave the stage empty: the consumer's bounded wait expires
        rp.advance();
        return true;
      }
      if (elect_one()) {
        const uint32_t full_local = bar(C::kBarRingFull + s);
        const uint32_t nbox = (col1 >= 0) ? 2u : 1u;
        if (leader) mbar_arrive_expect_tx(full_local, 2 * nbox * kChunkBytes);
        const uint32_t full_remote = mapa_shared(full_local, 0);
        const uint32_t dst = smem_base + C::kOffRing + s * kStageBytes;
        tma_load_2d_pair_hint(dst, &p.tm_kv, full_remote, col0, row, pol_kv);
        if (col1 >= 0) tma_load_2d_pair_hint(dst + kChunkBytes, &p.tm_kv, full_remote, col1, row, pol_kv);
      }
      __syncwarp();
      rp.advance();
      return true;
    };
    auto fill2 = [&](int col, int row_a, int row_b, int w) -> bool {  // one stage: the same columns of two row blocks
      const uint32_t s = rp.stage();
      if (rp.it >= (uint32_t)kStages) {
        if (!mbar_wait_bounded<false>(bar(C::kBarRingEmpty + s), rp.parity() ^ 1u, limit, abort_flag, p.status,
                                      W_RINGEMPTY, w))
          return false;
      }
      if constexpr (kStarve) {
        rp.advance();
        return true;
      }
      if (elect_one()) {
        const uint32_t full_local = bar(C::kBarRingFull + s);
        if (leader) mbar_arrive_expect_tx(full_local, 4 * kChunkBytes);
        const uint32_t full_remote = mapa_shared(full_local, 0);
        const uint32_t dst = smem_base + C::kOffRing + s * kStageBytes;
        tma_load_2d_pair_hint(dst, &p.tm_kv, full_remote, col, row_a, pol_kv);
        tma_load_2d_pair_hint(dst + kChunkBytes, &p.tm_kv, full_remote, col, row_b, pol_kv);
      }
      __syncwarp();
      rp.advance();
      return true;
    };
    auto load_k = [&](int seg_row0, int kb, int w) -> bool {  // this CTA's 128 keys: 4 dim pairs + rope
      const int row = seg_row0 + kb + (int)crank * 128;
      for (int d = 0; d < 4; ++d)
        if (!fill(128 * d, 128 * d + 64, row, w)) return false;
      return fill(kDLatent, -1, row, w);
    };
    auto load_v = [&](int seg_row0, int kb, int w) -> bool {  // (key half, output half): this CTA's 128 dims
      for (int kh = 0; kh < 2; ++kh)
        for (int h = 0; h < 2; ++h) {
          const int col = 256 * h + 128 * (int)crank;
          if (!fill(col, col + 64, seg_row0 + kb + kh * 128, w)) return false;
        }
      if constexpr (kPhase) {
        // rope part of the value: this CTA's 32 of the 64 rope dims for all 256 keys of the tile.  The box is
        // the usual 64 columns wide and starts at this CTA's first dim (544 for the second CTA: the columns
        // beyond the row's 576 are zero-filled and never read), so both CTAs find their dims at the same
        // shared-memory offset, which the single MMA descriptor of the pair requires.
        const int col = kDLatent + 32 * (int)crank;
        if (!fill2(col, seg_row0 + kb, seg_row0 + kb + 128, w)) return false;
      }
      return true;
    };
    for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs, ++n_done) {
      const AttnWorkItem item = get_work(p, w);
      // Q tile: wait until the previous tile's QK^T MMAs have finished reading it
      if (n_done > 0) {
        ok = mbar_wait_bounded<false>(bar(C::kBarQFree), qfree_phase, limit, abort_flag, p.status, W_QFREE, w);
        qfree_phase ^= 1;
        if (!ok) break;
      }
      const int qrow = item.tile * kAttnRowsPerPair + (int)crank * kAttnRowsPerCta;
      if (elect_one()) {  // latent chunks kept in shared memory and the rope chunk stay for the whole row tile
        mbar_arrive_expect_tx(bar(C::kBarQFull), (C::kQSmemChunks + 1) * kQChunkBytes);
        for (int d = 0; d < C::kQSmemChunks; ++d)
          tma_load_2d_hint(smem_base + C::kOffQLat + d * kQChunkBytes, &p.tm_q, bar(C::kBarQFull), d * 64, qrow, pol_q);
        tma_load_2d_hint(smem_base + C::kOffQPristine, &p.tm_q, bar(C::kBarQFull), kDLatent, qrow, pol_q);
        // The next row tile's queries can only be loaded once this tile's QK^T products are done (one Q buffer);
        // asking for them now puts them into L2, so that load pays the L2 latency instead of the DRAM one.  It
        // matters where a row tile sees few key tiles (documents built alone: 16 at most).
        if (w + p.n_pairs < p.n_tiles) {
          const int qnext = get_work(p, w + p.n_pairs).tile * kAttnRowsPerPair + (int)crank * kAttnRowsPerCta;
#pragma unroll
          for (int d = 0; d < 9; ++d) tma_prefetch_2d(&p.tm_q, d * 64, qnext);
        }
      }
      __syncwarp();
      // Upper latent part (dims 256-511, or 320-511): staged through one ring stage, from where the softmax
      // warps move it into tensor memory.  Each CTA loads its own rows and signals its own barrier; the issuer
      // lets go of the ring position once both CTAs have finished the move.
      {
        const uint32_t s = rp.stage();
        if (rp.it >= (uint32_t)kStages) {
          ok = mbar_wait_bounded<false>(bar(C::kBarRingEmpty + s), rp.parity() ^ 1u, limit, abort_flag, p.status,
                                        W_RINGEMPTY, w);
          if (!ok) break;
        }
        if (!kStarve && elect_one()) {
          if (leader) mbar_arrive(bar(C::kBarRingFull + s));  // keeps the ring's phases in step; no bytes land here
          mbar_arrive_expect_tx(bar(C::kBarQhFull), C::kQTmemChunks * kQChunkBytes);
          for (int d = 0; d < C::kQTmemChunks; ++d)
            tma_load_2d_hint(smem_base + C::kOffRing + s * kStageBytes + d * kQChunkBytes, &p.tm_q, bar(C::kBarQhFull),
                             (C::kQSmemChunks + d) * 64, qrow, pol_q);
        }
        __syncwarp();
        rp.advance();
      }
      // order of consumption: K(0), K(1), V(0), K(2), V(1), ..., V(last)
      SegIter it(p, item);
      int prev_row0 = -1, prev_kb = 0;
      while (ok && it.next()) {
        const int row0 = p.seg_off[it.seg];
        for (int kb = 0; kb < it.kmax && ok; kb += kAttnKeysPerTile) {
          ok = load_k(row0, kb, w);
          if (ok && prev_row0 >= 0) ok = load_v(prev_row0, prev_kb, w);
          prev_row0 = row0;
          prev_kb = kb;
        }
      }
      if (ok && prev_row0 >= 0) ok = load_v(prev_row0, prev_kb, w);
    }
    // drain: every stage this CTA filled must have been released by the tensor core, and the
    // last Q tile must be free, before the CTA may exit
    if (ok && n_done > 0)
      ok = mbar_wait_bounded<false>(bar(C::kBarQFree), qfree_phase, limit, abort_flag, p.status, W_DRAIN, -1);
    for (uint32_t back = 1; back <= (uint32_t)kStages && ok; ++back) {
      if (rp.it >= back) {
        const uint32_t u = rp.it - back;  // a fill that has not been waited for yet
        ok = mbar_wait_bounded<false>(bar(C::kBarRingEmpty + u % kStages), (u / kStages) & 1u, limit, abort_flag,
                                      p.status, W_DRAIN, (int)u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ UMMA issuer (leader CTA; whole warp loops, elected lane issues) --
    if (leader) {
      RingPos<kStages> rp;
      uint32_t qr_ready_phases = 0;  // bit rb = parity to wait for
      uint32_t p_ready_phase = 0;
      uint32_t qh_done_phase = 0;
      uint32_t s_writes = 0;  // how often the score buffer has been written (gives the s_free phase)
      uint32_t qr_use = 0;  // counts rope-buffer uses across tiles
      bool ok = true;
      const uint32_t q_base = smem_base + C::kOffQLat;
      const uint32_t p_base = smem_base + C::kOffP;

      for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
        const AttnWorkItem item = get_work(p, w);
        const int n_kt = count_key_tiles(p, item);
        int kt_issued = 0;  // key tiles whose QK^T has been issued
        int kt_pv = 0;      // key tiles whose PV has been issued
        {  // ring position of the staged upper Q part: wait for both CTAs' move into TMEM, then let go of it
          const uint32_t s = rp.stage();
          ok = mbar_wait_bounded<false>(bar(C::kBarRingFull + s), rp.parity(), limit, abort_flag, p.status, W_RINGFULL, w) &&
               mbar_wait_bounded<true>(bar(C::kBarQhDone), qh_done_phase, limit, abort_flag, p.status, W_QHDONE, w);
          qh_done_phase ^= 1;
          if (!ok) break;
          tc_fence_after_sync();
          if (elect_one()) umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
          __syncwarp();
          rp.advance();
        }

        auto issue_qk = [&](bool first_of_seg, bool last_of_seg, uint32_t rb) -> bool {
          if (first_of_seg) {
            if (!mbar_wait_bounded<true>(bar(C::kBarQrReady + rb), (qr_ready_phases >> rb) & 1u, limit, abort_flag,
                                         p.status, W_QRREADY, w))
              return false;
            qr_ready_phases ^= (1u << rb);
          }
          if (s_writes > 0) {  // one score buffer: the softmax warps must have read the previous key tile's scores
            if (!mbar_wait_bounded<true>(bar(C::kBarSFree), (s_writes - 1) & 1u, limit, abort_flag, p.status, W_SFREE, w))
              return false;
            tc_fence_after_sync();
          }
          ++s_writes;
          const uint32_t tmem_s = tmem_base + kColS;
#pragma unroll 1
          for (int st = 0; st < 5; ++st) {
            const uint32_t s = rp.stage();
            {
              if (!mbar_wait_bounded<false>(bar(C::kBarRingFull + s), rp.parity(), limit, abort_flag, p.status, W_RINGFULL, w))
                return false;
            }
            const uint32_t b_addr = smem_base + C::kOffRing + s * kStageBytes;
            if (elect_one()) {
              if (kPhase && st == 2) {  // output-phase: dims 256-319 from shared memory, 320-383 from tensor memory
                const uint64_t da = umma_desc_sw128(q_base + 4 * kQChunkBytes, 16, 1024), db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_f16<2>(tmem_s, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kIdescQK, 1u);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_f16_ts<2>(tmem_s, tmem_base + kColQp + 8u * k, db + (uint64_t)((kChunkBytes + k * 32) >> 4), kIdescQK, 1u);
                umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              } else if (kPhase && st == 3) {  // output-phase: dims 384-511 from tensor memory
                const uint64_t db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                  umma_f16_ts<2>(tmem_s, tmem_base + kColQp + 32u + 8u * k,
                                 db + (uint64_t)(((k >> 2) * kChunkBytes + (k & 3) * 32) >> 4), kIdescQK, 1u);
                umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              } else if (!kPhase && st >= 2 && st < 4) {  // latent dims 256-511: A from tensor memory, 8 columns per K = 16 step
                const uint32_t a_tmem = tmem_base + kColQ + (uint32_t)(st - 2) * 64u;
                const uint64_t db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                  umma_f16_ts<2>(tmem_s, a_tmem + 8u * k, db + (uint64_t)(((k >> 2) * kChunkBytes + (k & 3) * 32) >> 4),
                                 kIdescQK, 1u);
                }
                umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              } else if (st < 2) {  // latent dims 0-255: A from shared memory
                const uint32_t a_addr = q_base + 2 * st * kQChunkBytes;
                // descriptors differ only in the start-address field (16-byte units): add constants
                const uint64_t da = umma_desc_sw128(a_addr, 16, 1024), db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                  umma_f16<2>(tmem_s, da + (uint64_t)(((k >> 2) * kQChunkBytes + (k & 3) * 32) >> 4),
                              db + (uint64_t)(((k >> 2) * kChunkBytes + (k & 3) * 32) >> 4), kIdescQK,
                              (st > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              } else {
                const uint32_t a_addr = smem_base + C::kOffQRot + rb * kQChunkBytes;
                const uint64_t da = umma_desc_sw128(a_addr, 16, 1024), db = umma_desc_sw128(b_addr, 16, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_f16<2>(tmem_s, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), kIdescQK, 1u);
                umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
                umma_commit_2_mc(bar(C::kBarSFull), 3);
                if (last_of_seg) umma_commit_2_mc(bar(C::kBarQrFree + rb), 3);
                // all QK^T of this row tile issued: the Q tile is free once they complete
                if (kt_issued + 1 == n_kt) umma_commit_2_mc(bar(C::kBarQFree), 3);
              }
            }
            __syncwarp();
            rp.advance();
          }
          ++kt_issued;
          return true;
        };
        auto issue_pv = [&]() -> bool {
          {
            if (!mbar_wait_bounded<true>(bar(C::kBarPReady), p_ready_phase, limit, abort_flag, p.status, W_PREADY, w))
              return false;
          }
          p_ready_phase ^= 1;
          tc_fence_after_sync();
#pragma unroll 1
          for (int q = 0; q < 4; ++q) {
            const int kh = q >> 1, h = q & 1;
            const uint32_t s = rp.stage();
            {
              if (!mbar_wait_bounded<false>(bar(C::kBarRingFull + s), rp.parity(), limit, abort_flag, p.status, W_RINGFULL, w))
                return false;
            }
            const uint32_t b_addr = smem_base + C::kOffRing + s * kStageBytes;
            const uint32_t tmem_o = tmem_base + kColO + (uint32_t)h * 128u;
            if (elect_one()) {
              const uint64_t da = umma_desc_sw128(p_base + 2 * kh * kQChunkBytes, 16, 1024);
              const uint64_t db = umma_desc_sw128(b_addr, kChunkBytes, 1024);
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                umma_f16<2>(tmem_o, da + (uint64_t)(((k >> 2) * kQChunkBytes + (k & 3) * 32) >> 4),
                            db + (uint64_t)((k * 2048) >> 4), kIdescPV, (kt_pv > 0 || kh > 0 || k > 0) ? 1u : 0u);
              }
              umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              if (!kPhase && q == 3) umma_commit_2_mc(bar(C::kBarPvDone), 3);
            }
            __syncwarp();
            rp.advance();
          }
          if constexpr (kPhase) {  // rope part of the value: O_rope[64 x 64] += P[64 x 256] V_rope[256 x 64]
            const uint32_t s = rp.stage();
            if (!mbar_wait_bounded<false>(bar(C::kBarRingFull + s), rp.parity(), limit, abort_flag, p.status, W_RINGFULL, w))
              return false;
            const uint32_t b_addr = smem_base + C::kOffRing + s * kStageBytes;
            if (elect_one()) {
              const uint64_t da = umma_desc_sw128(p_base, 16, 1024);
              const uint64_t db = umma_desc_sw128(b_addr, kChunkBytes, 1024);
#pragma unroll
              for (int k = 0; k < 16; ++k) {  // 16 keys per step; the two 128-key boxes are contiguous
                umma_f16<2>(tmem_base + kColOr, da + (uint64_t)(((k >> 2) * kQChunkBytes + (k & 3) * 32) >> 4),
                            db + (uint64_t)((k * 2048) >> 4), kIdescPVr, (kt_pv > 0 || k > 0) ? 1u : 0u);
              }
              umma_commit_2_mc(bar(C::kBarRingEmpty + s), 3);
              umma_commit_2_mc(bar(C::kBarPvDone), 3);
            }
            __syncwarp();
            rp.advance();
          }
          ++kt_pv;
          return true;
        };

        SegIter it(p, item);
        while (ok && it.next()) {
          const uint32_t rb = qr_use & 1u;
          ++qr_use;
          for (int kb = 0; kb < it.kmax && ok; kb += kAttnKeysPerTile) {
            const bool first = (kb == 0);
            const bool last = (kb + kAttnKeysPerTile >= it.kmax);
            ok = issue_qk(first, last, rb);
            if (ok && kt_issued >= 2) ok = issue_pv();
          }
        }
        while (ok && kt_pv < kt_issued) ok = issue_pv();
      }
    }
  } else if (warp == 2) {
    // ------------------------------ query relocation ----------------------------------------
    uint32_t qfull_phase = 0;
    uint32_t qr_free_phases = 0;  // bit rb = parity to wait for
    uint32_t qr_use = 0;
    bool ok = true;
    for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
      const AttnWorkItem item = get_work(p, w);
      ok = mbar_wait_bounded<false>(bar(C::kBarQFull), qfull_phase, limit, abort_flag, p.status, W_QFULL, w);
      qfull_phase ^= 1;
      uint4 pr[16];  // output-phase: the rope chunk as loaded, this lane's 16 pieces (it landed in a rotated buffer)
      if constexpr (kPhase) {
        if (ok) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int idx = lane + 32 * i;
            pr[i] = *reinterpret_cast<const uint4*>(smem + C::kOffQPristine + sw128_offset((uint32_t)(idx >> 3), (uint32_t)(idx & 7)));
          }
        }
        __syncwarp();  // every lane has its pieces before any lane overwrites the buffer
      }
      SegIter it(p, item);
      while (ok && it.next()) {
        const uint32_t rb = qr_use & 1u;
        if (qr_use >= 2) {
          ok = mbar_wait_bounded<true>(bar(C::kBarQrFree + rb), (qr_free_phases >> rb) & 1u, limit, abort_flag, p.status,
                                       W_QRFREE, w);
          qr_free_phases ^= (1u << rb);
          if (!ok) break;
        }
        ++qr_use;
        const float2* cs = p.seg_cs + (size_t)it.seg * 32;
        const uint8_t* src = smem + C::kOffQPristine;
        uint8_t* dst = smem + C::kOffQRot + rb * kQChunkBytes;
#pragma unroll(kPhase ? 16 : 4)
        for (int i = 0; i < 16; ++i) {
          const int idx = lane + 32 * i;
          const uint32_t row = idx >> 3, c = idx & 7;
          const uint32_t off = sw128_offset(row, c);
          uint4 v;
          if constexpr (kPhase) v = pr[i]; else v = *reinterpret_cast<const uint4*>(src + off);
          uint32_t in[4] = {v.x, v.y, v.z, v.w};
          uint32_t outv[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 t = __ldg(cs + 4 * c + e);
            __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&in[e]);
            const float x0 = __bfloat162float(x.x), x1 = __bfloat162float(x.y);
            // R(-delta): rotate by the negative angle
            outv[e] = pack_bf16(x0 * t.x + x1 * t.y, x1 * t.x - x0 * t.y);
          }
          *reinterpret_cast<uint4*>(dst + off) = make_uint4(outv[0], outv[1], outv[2], outv[3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(mapa_shared(bar(C::kBarQrReady + rb), 0));
      }
    }
    // drain the last releases so that no commit targets this CTA after it exits
    if (lane == 0) {
      for (uint32_t u = (qr_use >= 2 ? qr_use - 2 : 0); u < qr_use && ok; ++u) {
        const uint32_t rb = u & 1u;
        ok = mbar_wait_bounded<true>(bar(C::kBarQrFree + rb), (qr_free_phases >> rb) & 1u, limit, abort_flag, p.status,
                                     W_DRAIN, 100 + (int)rb);
        qr_free_phases ^= (1u << rb);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------ softmax / correction / epilogue ----------------------------
    // 8 warps.  Warp sw = warp - 4 reads TMEM lanes [32 (sw % 4), +32) and the column half
    // ch = sw / 4 of every 128-column buffer, so one query row (TMEM lanes m and m + 64) is
    // shared by four threads: (kh, ch) = (key half of the tile, 64-key quarter within it).
    const int sw = warp - 4;
    const int ch = sw >> 2;
    const int L = (sw & 3) * 32 + lane;  // TMEM lane
    const int m = L & 63;                // row within this CTA
    const int kh = L >> 6;               // which 128-key half of the tile (and which dims half of O)
    const int part = kh * 2 + ch;        // which 64-key quarter of the tile
    const uint32_t lane_base = ((uint32_t)((sw & 3) * 32)) << 16;
    volatile unsigned long long* xbuf = reinterpret_cast<volatile unsigned long long*>(smem + C::kOffXchg);
    uint32_t xseq = 0;  // exchange sequence number
    uint32_t ring_it = 0;  // ring position of the current row tile's staged Q half
    uint32_t s_full_phase = 0;
    uint32_t qh_full_phase = 0;
    uint32_t pv_done_phase = 0;
    bool ok = true;
    const float scale = p.scale_log2;
    const uint32_t p_ready_remote = mapa_shared(bar(C::kBarPReady), 0);
    const uint32_t s_free_remote = mapa_shared(bar(C::kBarSFree), 0);
    const uint32_t qh_done_remote = mapa_shared(bar(C::kBarQhDone), 0);

    for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
      const AttnWorkItem item = get_work(p, w);
      const int r = item.tile * kAttnRowsPerPair + (int)crank * kAttnRowsPerCta + m;
      bool valid = rk_index_ok(item.tile >= 0 && (long long)item.tile * kAttnRowsPerPair < p.n_flat, p.status,
                               RK_CHK_WORK_TILE, item.tile) && r < p.n_flat;
      int pos = -1, prow = -1;
      if (valid) {
        const int tok = r / p.hpt;
        prow = p.rowmap ? p.rowmap[tok] : p.row_base + tok;
        if (rk_index_ok(prow >= 0 && prow < p.n_rows_total, p.status, RK_CHK_PROT_ROW, prow))
          pos = p.row_pos[prow];
        else
          valid = false;  // bounds-checked build: the row is skipped, nothing is read or written for it
      }
      float m_run = -INFINITY, l_run = 0.f;
      int kt = 0;
      {  // move this thread's share of the upper Q part (row m) from its ring stage into TMEM
        ok = mbar_wait_bounded<false>(bar(C::kBarQhFull), qh_full_phase, limit, abort_flag, p.status, W_QHFULL, w);
        qh_full_phase ^= 1;
        if (!ok) break;
        // every role counts ring positions alike: one staged half per row tile, nine stages per key tile
        const uint8_t* stage = smem + C::kOffRing + (ring_it % kStages) * kStageBytes;
        ring_it += 1u + (uint32_t)C::kStagesPerKeyTile * (uint32_t)count_key_tiles(p, item);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (2 * ch + half >= C::kQTmemChunks) continue;  // output-phase: three chunks only (warp-uniform)
          uint32_t qv[32];
          const uint8_t* chunk = stage + (2 * ch + half) * kQChunkBytes;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 v = *reinterpret_cast<const uint4*>(chunk + sw128_offset((uint32_t)m, (uint32_t)c));
            qv[4 * c] = v.x; qv[4 * c + 1] = v.y; qv[4 * c + 2] = v.z; qv[4 * c + 3] = v.w;
          }
          tmem_st_x32(tmem_base + lane_base + (kPhase ? kColQp : kColQ) + (uint32_t)(ch * 64 + half * 32), qv);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(qh_done_remote);
      }

      // output-phase instantiation: the rope part of O is accumulated in the frame of the segment being
      // walked (its stored rope dims are in that document's position-zero frame); seg_frame is that segment
      int seg_frame = -1;
      const int jr = 16 * kh + 8 * ch;  // first of this thread's 8 rotation pairs (16 rope dims) of the row
      SegIter it(p, item);
      while (ok && it.next()) {
        const int n_seg = p.seg_off[it.seg + 1] - p.seg_off[it.seg];
        int lim = pos - p.seg_delta[it.seg];  // last visible canonical index
        if (lim > n_seg - 1) lim = n_seg - 1;
        if (pos < 0) lim = -1;
        if (p.isolated) {  // only the row's own segment, causal in its canonical frame
          const int lo = p.seg_off[it.seg];
          lim = (prow >= lo && prow < lo + n_seg) ? prow - lo : -1;
        }
        for (int kb = 0; kb < it.kmax && ok; kb += kAttnKeysPerTile, ++kt) {
          int nv = lim - (kb + part * 64) + 1;
          nv = nv < 0 ? 0 : (nv > 64 ? 64 : nv);
          {
            ok = mbar_wait_bounded<false>(bar(C::kBarSFull), s_full_phase, limit, abort_flag, p.status, W_SFULL, w);
          }
          s_full_phase ^= 1;
          if (!ok) break;
          tc_fence_after_sync();
          uint32_t s[64];
          const uint32_t taddr = tmem_base + lane_base + kColS + (uint32_t)ch * 64u;
          tmem_ld_x32(taddr + 0, s + 0);
          tmem_ld_x32(taddr + 32, s + 32);
          tmem_wait_ld();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(s_free_remote);  // the issuer may overwrite the score buffer
          const bool full = __all_sync(0xffffffffu, nv == 64);  // no masking needed anywhere in this warp
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          if (full) {
#pragma unroll
            for (int c = 0; c < 64; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], __uint_as_float(s[c]));
          } else {
#pragma unroll
            for (int c = 0; c < 64; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], (c < nv) ? __uint_as_float(s[c]) : -INFINITY);
          }
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          float mxo = mx;
          ok = quad_exchange_max(xbuf, part, m, ++xseq, mx, mxo, limit, abort_flag, p.status, w);
          if (!ok) break;
          const float mt = mxo * scale;
          // lazy rescale: only when the running maximum grows by more than 2^8
          float alpha = 1.f;
          bool need = false;
          if (mt > m_run + 8.f) {  // also true for the first finite maximum (m_run = -inf)
            alpha = (m_run == -INFINITY) ? 0.f : fast_exp2(m_run - mt);
            need = (m_run != -INFINITY);
            m_run = mt;
            l_run *= alpha;
          }
          const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
          uint32_t pk[32];
          float ls4[4] = {0.f, 0.f, 0.f, 0.f};
          if (full) {
#pragma unroll
            for (int c = 0; c < 64; c += 2) {
              const float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), scale, -m_use));
              const float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale, -m_use));
              ls4[(c >> 1) & 3] += p0 + p1;
              pk[c >> 1] = pack_bf16(p0, p1);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 64; c += 2) {
              const float p0 = (c < nv) ? fast_exp2(fmaf(__uint_as_float(s[c]), scale, -m_use)) : 0.f;
              const float p1 = (c + 1 < nv) ? fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale, -m_use)) : 0.f;
              ls4[(c >> 1) & 3] += p0 + p1;
              pk[c >> 1] = pack_bf16(p0, p1);
            }
          }
          l_run += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
          // P buffer and O are free once the previous PV has completed
          if (kt > 0) {
            {
              ok = mbar_wait_bounded<false>(bar(C::kBarPvDone), pv_done_phase, limit, abort_flag, p.status, W_PVDONE, w);
            }
            pv_done_phase ^= 1;
            if (!ok) break;
            tc_fence_after_sync();
            const bool any_need = __any_sync(0xffffffffu, need);
            if (any_need) {
#pragma unroll 1
              for (int cc = 0; cc < 128; cc += 32) {  // this thread's 2 x 64 columns of O
                uint32_t o[32];
                const uint32_t oaddr = tmem_base + lane_base + kColO + (uint32_t)((cc >> 6) * 128 + ch * 64 + (cc & 63));
                tmem_ld_x32(oaddr, o);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                tmem_st_x32(oaddr, o);
              }
              tmem_wait_st();
            }
            if constexpr (kPhase) {
              // Segment switch (Algorithm 2, RestorePhase folded into the running merge): what has been
              // accumulated so far is in the previous segment's frame; turning it by
              // R(delta_prev - delta_this) moves it into the frame of the segment whose keys come next, so
              // that the PV products of both can share one accumulator.  The lazy rescale rides along.
              const bool turn = (kb == 0 && seg_frame >= 0);
              if (turn || any_need) {
                uint32_t o[16];
                const uint32_t oaddr = tmem_base + lane_base + kColOr + (uint32_t)(ch * 16);
                tmem_ld_x16(oaddr, o);
                tmem_wait_ld();
                if (turn) {
                  const int d = p.seg_delta[seg_frame] - p.seg_delta[it.seg];
#pragma unroll
                  for (int i = 0; i < 8; ++i) {
                    float c, sn;
                    rope_cs(p, d, jr + i, c, sn);
                    const float x0 = __uint_as_float(o[2 * i]) * alpha, x1 = __uint_as_float(o[2 * i + 1]) * alpha;
                    o[2 * i] = __float_as_uint(x0 * c - x1 * sn);
                    o[2 * i + 1] = __float_as_uint(x0 * sn + x1 * c);
                  }
                } else {
#pragma unroll
                  for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                }
                tmem_st_x16(oaddr, o);
                tmem_wait_st();
              }
            }
          }
          if constexpr (kPhase) seg_frame = it.seg;
          // write P (bf16, K-major 128B swizzle): row m of sub-chunk `part` (64 keys = 128 bytes)
          uint8_t* pbase = smem + C::kOffP + part * kQChunkBytes;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            uint8_t* dstp = pbase + sw128_offset((uint32_t)m, (uint32_t)c);
            *reinterpret_cast<uint4*>(dstp) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          }
          fence_proxy_async_smem();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_remote(p_ready_remote);
        }
      }
      if (!ok) break;
      // ---- epilogue: wait for the last PV, normalise, store ----
      ok = mbar_wait_bounded<false>(bar(C::kBarPvDone), pv_done_phase, limit, abort_flag, p.status, W_PVDONE, w);
      pv_done_phase ^= 1;
      if (!ok) break;
      tc_fence_after_sync();
      float l_tot = l_run;
      ok = quad_exchange_sum(xbuf, part, m, ++xseq, l_run, l_tot, limit, abort_flag, p.status, w);
      if (!ok) break;
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      __nv_bfloat16* Orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)(valid ? r : 0) * C::kOW;
#pragma unroll 1
      for (int cc = 0; cc < 128; cc += 32) {
        const int h = cc >> 6, c0 = cc & 63;
        uint32_t o[32];
        tmem_ld_x32(tmem_base + lane_base + kColO + (uint32_t)(h * 128 + ch * 64 + c0), o);
        tmem_wait_ld();
        if (valid) {
          uint4* dstg = reinterpret_cast<uint4*>(Orow + 256 * h + 128 * kh + 64 * ch + c0);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(o[8 * e + 0]) * inv, __uint_as_float(o[8 * e + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(o[8 * e + 2]) * inv, __uint_as_float(o[8 * e + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(o[8 * e + 4]) * inv, __uint_as_float(o[8 * e + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(o[8 * e + 6]) * inv, __uint_as_float(o[8 * e + 7]) * inv);
            __stcs(dstg + e, v);
          }
        }
      }
      if constexpr (kPhase) {
        // rope part of the output: normalise, then RestorePhase of the last frame and the inverse output
        // RoPE of the row in one turn, R(-pos) R(delta_frame) = R(delta_frame - pos)  (Eq. offonline)
        uint32_t o[16];
        tmem_ld_x16(tmem_base + lane_base + kColOr + (uint32_t)(ch * 16), o);
        tmem_wait_ld();
        if (valid) {
          const int d = (seg_frame >= 0 ? p.seg_delta[seg_frame] : 0) - pos;
          uint32_t v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float c, sn;
            rope_cs(p, d, jr + i, c, sn);
            const float x0 = __uint_as_float(o[2 * i]) * inv, x1 = __uint_as_float(o[2 * i + 1]) * inv;
            v[i] = pack_bf16(x0 * c - x1 * sn, x0 * sn + x1 * c);
          }
          uint4* dstg = reinterpret_cast<uint4*>(Orow + kDLatent + 32 * kh + 16 * ch);
          __stcs(dstg, make_uint4(v[0], v[1], v[2], v[3]));
          __stcs(dstg + 1, make_uint4(v[4], v[5], v[6], v[7]));
        }
      }
      if (valid && part == 0)
        p.lse[r] = (l_tot > 0.f) ? (m_run + log2f(l_tot)) * 0.69314718055994530942f : -INFINITY;
      tc_fence_before_sync();
    }
  }

  // ------------------------------ teardown ---------------------------------------------------
  // after a wait has expired: give this CTA's bulk copies that may still be in flight a bounded time
  // to land before its shared memory goes away
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


cudaError_t attention_setup() {
  cudaError_t e = cudaFuncSetAttribute(rk_mla_attn_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)Cfg<false>::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(rk_mla_attn_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg<false>::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(rk_mla_attn_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg<true>::kSmemBytes);
  return e;
}

int attention_max_pairs(int sm_count) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (sm_count / 2), 1, 1);
  cfg.blockDim = dim3(kAttnThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg<false>::kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, rk_mla_attn_kernel<false, false>, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = sm_count / 2;
  }
  return n < sm_count / 2 ? n : sm_count / 2;
}

cudaError_t launch_attention(const AttnParams& p, int n_pairs, bool value_phase, bool starve_loads, cudaStream_t stream) {
  const dim3 grid(2 * n_pairs, 1, 1), block(kAttnThreads, 1, 1);
  if (value_phase)
    rk_mla_attn_kernel<true, false><<<grid, block, Cfg<true>::kSmemBytes, stream>>>(p);
  else if (starve_loads)
    rk_mla_attn_kernel<false, true><<<grid, block, Cfg<false>::kSmemBytes, stream>>>(p);
  else
    rk_mla_attn_kernel<false, false><<<grid, block, Cfg<false>::kSmemBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rk
