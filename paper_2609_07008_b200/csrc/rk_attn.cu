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
// columns [0,N/2), lanes 64-127: columns [N/2,N)), so O takes 256 columns and two S buffers
// 2 x 128: exactly the 512 columns of TMEM.  The B operand is split across the pair: for QK^T
// each CTA streams its 128 keys of the tile, for PV its 128 of each 256 output dims.  The same
// [128 keys x 64 dims] 128B-swizzled TMA box serves as K-major B (QK^T) and MN-major B (PV).
//
// Warp roles per CTA (256 threads): warp 0 TMA producer, warp 1 UMMA issuer (leader CTA only),
// warp 2 query relocation, warps 4-7 softmax / correction / epilogue (thread <-> TMEM lane).
#include <cuda_bf16.h>

#include "rk_internal.h"

namespace rk {
namespace {

constexpr int kRing = 6;
constexpr uint32_t kChunkBytes = 16384;  // 128 keys x 64 dims bf16
constexpr uint32_t kQChunkBytes = 8192;  // 64 rows x 64 dims bf16

// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQLat = 0;                                // 8 chunks
constexpr uint32_t kOffQPristine = kOffQLat + 8 * kQChunkBytes;  // rope chunk as loaded
constexpr uint32_t kOffQRot = kOffQPristine + kQChunkBytes;      // 2 rotated rope chunks
constexpr uint32_t kOffP = kOffQRot + 2 * kQChunkBytes;          // 4 sub-chunks [64 x 64 keys]
constexpr uint32_t kOffRing = kOffP + 4 * kQChunkBytes;
constexpr uint32_t kOffBars = kOffRing + kRing * kChunkBytes;
// barrier indices (8 bytes each)
constexpr int kBarQFull = 0, kBarQFree = 1, kBarQrReady = 2 /*2*/, kBarQrFree = 4 /*2*/, kBarRingFull = 6,
              kBarRingEmpty = kBarRingFull + kRing, kBarSFull = kBarRingEmpty + kRing /*2*/,
              kBarPReady = kBarSFull + 2, kBarPvDone = kBarPReady + 1, kNumBars = kBarPvDone + 1;
constexpr uint32_t kOffTmemPtr = kOffBars + kNumBars * 8;
constexpr uint32_t kOffAbort = kOffTmemPtr + 8;
constexpr uint32_t kOffXchg = kOffAbort + 8;                 // u64 [2 parity][2 halves][64]: (seq << 32) | value
constexpr uint32_t kSmemUsed = kOffXchg + 2 * 2 * 64 * 8;
constexpr uint32_t kSmemBytes = kSmemUsed + 1024;            // + alignment slack

// TMEM columns
constexpr uint32_t kColO = 0;    // two halves of 128 columns
constexpr uint32_t kColS = 256;  // two buffers of 128 columns

constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 256, 0, 0);
constexpr uint32_t kIdescPV = umma_idesc_bf16(128, 256, 0, 1);

// wait tags reported on timeout
enum { W_QFULL = 1, W_QFREE, W_QRREADY, W_QRFREE, W_RINGFULL, W_RINGEMPTY, W_SFULL, W_PREADY, W_PVDONE, W_DRAIN };

struct SegIter {
  // iterates the segments a row tile can see; kmax = number of canonical keys any row may see
  const AttnParams& p;
  int maxpos;
  int seg;
  int kmax;
  __device__ SegIter(const AttnParams& p_, int maxpos_) : p(p_), maxpos(maxpos_), seg(-1), kmax(0) {}
  __device__ bool next() {
    while (++seg < p.n_segs) {
      int n = p.seg_off[seg + 1] - p.seg_off[seg];
      int lim = maxpos - p.seg_delta[seg] + 1;
      kmax = lim < n ? lim : n;
      if (kmax > 0) return true;
    }
    return false;
  }
};

// Ring bookkeeping shared by the producer and the UMMA issuer: both walk the same slot
// sequence.  A V stage needs two consecutive slots (fixed 16 KB apart for the descriptor's
// leading byte offset), so a pair never starts on the last slot: that slot is skipped.
struct RingPos {
  uint32_t slot = 0;
  uint32_t phases = 0;  // bit s = parity to wait for on slot s
  __device__ void advance() { phases ^= (1u << slot); slot = (slot + 1 == kRing) ? 0 : slot + 1; }
  __device__ void skip() { slot = (slot + 1 == kRing) ? 0 : slot + 1; }
  __device__ uint32_t parity() const { return (phases >> slot) & 1u; }
};

// The two threads that hold the two halves of one query row (lanes m and m + 64 of TMEM, in
// different warps) swap one float through shared memory.  Sequence-tagged and double-buffered
// by sequence parity; the poll is bounded like every other wait in this kernel.
__device__ __forceinline__ bool pair_exchange(volatile unsigned long long* xbuf, int kh, int m, uint32_t seq,
                                              float mine, float& other, uint64_t limit_ns,
                                              volatile int* abort_flag, DeviceStatus* st, int aux) {
  volatile unsigned long long* base = xbuf + (seq & 1u) * 128;
  base[kh * 64 + m] = ((unsigned long long)seq << 32) | (unsigned long long)__float_as_uint(mine);
  volatile unsigned long long* theirs = base + (kh ^ 1) * 64 + m;
  uint64_t t0 = 0;
  uint32_t spins = 0;
  while (true) {
    const unsigned long long v = *theirs;
    if ((uint32_t)(v >> 32) == seq) {
      other = __uint_as_float((uint32_t)v);
      return true;
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

}  // namespace

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(256, 1)
    rk_mla_attn_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t crank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  const bool leader = (crank == 0);

  auto bar = [&](int i) -> uint32_t { return smem_base + kOffBars + 8u * i; };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffAbort);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + kOffTmemPtr);
  const uint64_t limit = p.wait_ns;

  if (threadIdx.x < 256) reinterpret_cast<volatile unsigned long long*>(smem + kOffXchg)[threadIdx.x] = 0ull;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(kBarQFull), 1);
    mbar_init(bar(kBarQFree), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(kBarQrReady + b), 2);
      mbar_init(bar(kBarQrFree + b), 1);
      mbar_init(bar(kBarSFull + b), 1);
    }
    for (int s = 0; s < kRing; ++s) {
      mbar_init(bar(kBarRingFull + s), 1);
      mbar_init(bar(kBarRingEmpty + s), 1);
    }
    mbar_init(bar(kBarPReady), 8);
    mbar_init(bar(kBarPvDone), 1);
    fence_mbar_init_cluster();
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc<2>(smem_base + kOffTmemPtr, 512);
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
    // ------------------------------ TMA producer -----------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&p.tm_q);
      tma_prefetch_desc(&p.tm_kv);
      RingPos rp;
      uint32_t qfree_phase = 0;
      uint32_t used_slots = 0;  // bit s set once slot s has been filled at least once
      bool ok = true;
      int n_done = 0;
      for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs, ++n_done) {
        const AttnWorkItem item = p.work[w];
        // Q tile: wait until the previous tile's QK^T MMAs have finished reading it
        if (n_done > 0) {
          ok = mbar_wait_bounded<true>(bar(kBarQFree), qfree_phase, limit, abort_flag, p.status, W_QFREE, w);
          qfree_phase ^= 1;
          if (!ok) break;
        }
        mbar_arrive_expect_tx(bar(kBarQFull), 9 * kQChunkBytes);
        const int qrow = item.tile * kAttnRowsPerPair + (int)crank * kAttnRowsPerCta;
        for (int d = 0; d < 9; ++d)
          tma_load_2d(smem_base + kOffQLat + d * kQChunkBytes, &p.tm_q, bar(kBarQFull), d * 64, qrow);

        auto load_slot = [&](int col, int row) -> bool {
          if (used_slots & (1u << rp.slot)) {
            if (!mbar_wait_bounded<true>(bar(kBarRingEmpty + rp.slot), rp.parity() ^ 1u, limit, abort_flag,
                                         p.status, W_RINGEMPTY, w))
              return false;
          }
          used_slots |= (1u << rp.slot);
          const uint32_t full_local = bar(kBarRingFull + rp.slot);
          if (leader) mbar_arrive_expect_tx(full_local, 2 * kChunkBytes);
          tma_load_2d_pair(smem_base + kOffRing + rp.slot * kChunkBytes, &p.tm_kv, mapa_shared(full_local, 0), col,
                           row);
          rp.advance();
          return true;
        };
        auto load_k = [&](int seg_row0, int kb) -> bool {  // 9 single slots: this CTA's 128 keys
          const int row = seg_row0 + kb + (int)crank * 128;
          for (int d = 0; d < 9; ++d)
            if (!load_slot(d * 64, row)) return false;
          return true;
        };
        auto load_v = [&](int seg_row0, int kb) -> bool {  // 4 pairs: (key half, output half)
          for (int kh = 0; kh < 2; ++kh)
            for (int h = 0; h < 2; ++h) {
              if (rp.slot == kRing - 1) rp.skip();
              const int row = seg_row0 + kb + kh * 128;
              const int col = 256 * h + 128 * (int)crank;
              if (!load_slot(col, row)) return false;
              if (!load_slot(col + 64, row)) return false;
            }
          return true;
        };

        // order of consumption: K(0), K(1), V(0), K(2), V(1), ..., V(last)
        SegIter it(p, item.maxpos);
        int prev_row0 = -1, prev_kb = 0;
        while (ok && it.next()) {
          const int row0 = p.seg_off[it.seg];
          for (int kb = 0; kb < it.kmax && ok; kb += kAttnKeysPerTile) {
            ok = load_k(row0, kb);
            if (ok && prev_row0 >= 0) ok = load_v(prev_row0, prev_kb);
            prev_row0 = row0;
            prev_kb = kb;
          }
        }
        if (ok && prev_row0 >= 0) ok = load_v(prev_row0, prev_kb);
      }
      // drain: every slot this CTA filled must have been released by the tensor core, and the
      // last Q tile must be free, before the CTA may exit
      if (ok && n_done > 0)
        ok = mbar_wait_bounded<true>(bar(kBarQFree), qfree_phase, limit, abort_flag, p.status, W_DRAIN, -1);
      for (int s = 0; s < kRing && ok; ++s) {
        if (used_slots & (1u << s))
          ok = mbar_wait_bounded<true>(bar(kBarRingEmpty + s), ((rp.phases >> s) & 1u) ^ 1u, limit, abort_flag,
                                       p.status, W_DRAIN, s);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ UMMA issuer (leader CTA) --------------------------------
    if (leader && lane == 0) {
      RingPos rp;
      uint32_t qr_ready_phase[2] = {0, 0};
      uint32_t p_ready_phase = 0;
      uint32_t qr_use = 0;  // counts rope-buffer uses across tiles
      bool ok = true;
      const uint32_t q_base = smem_base + kOffQLat;
      const uint32_t p_base = smem_base + kOffP;

      for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
        const AttnWorkItem item = p.work[w];
        int kt_issued = 0;   // key tiles whose QK^T has been issued
        int kt_pv = 0;       // key tiles whose PV has been issued

        auto issue_qk = [&](bool first_of_seg, bool last_of_seg, uint32_t rb) -> bool {
          if (first_of_seg) {
            if (!mbar_wait_bounded<true>(bar(kBarQrReady + rb), qr_ready_phase[rb], limit, abort_flag, p.status,
                                         W_QRREADY, w))
              return false;
            qr_ready_phase[rb] ^= 1;
          }
          const uint32_t tmem_s = tmem_base + kColS + (uint32_t)(kt_issued & 1) * 128u;
          for (int d = 0; d < 9; ++d) {
            if (!mbar_wait_bounded<true>(bar(kBarRingFull + rp.slot), rp.parity(), limit, abort_flag, p.status,
                                         W_RINGFULL, w))
              return false;
            tc_fence_after_sync();
            const uint32_t a_addr = (d < 8) ? (q_base + d * kQChunkBytes) : (smem_base + kOffQRot + rb * kQChunkBytes);
            const uint32_t b_addr = smem_base + kOffRing + rp.slot * kChunkBytes;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_f16<2>(tmem_s, umma_desc_sw128(a_addr + k * 32, 16, 1024), umma_desc_sw128(b_addr + k * 32, 16, 1024),
                          kIdescQK, (d > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_2_mc(bar(kBarRingEmpty + rp.slot), 3);
            rp.advance();
          }
          umma_commit_2_mc(bar(kBarSFull + (kt_issued & 1)), 3);
          if (last_of_seg) umma_commit_2_mc(bar(kBarQrFree + rb), 3);
          ++kt_issued;
          return true;
        };
        auto issue_pv = [&]() -> bool {
          if (!mbar_wait_bounded<true>(bar(kBarPReady), p_ready_phase, limit, abort_flag, p.status, W_PREADY, w))
            return false;
          p_ready_phase ^= 1;
          tc_fence_after_sync();
          for (int kh = 0; kh < 2; ++kh)
            for (int h = 0; h < 2; ++h) {
              if (rp.slot == kRing - 1) rp.skip();
              const uint32_t s0 = rp.slot;
              if (!mbar_wait_bounded<true>(bar(kBarRingFull + s0), rp.parity(), limit, abort_flag, p.status,
                                           W_RINGFULL, w))
                return false;
              rp.advance();
              if (!mbar_wait_bounded<true>(bar(kBarRingFull + s0 + 1), rp.parity(), limit, abort_flag, p.status,
                                           W_RINGFULL, w))
                return false;
              rp.advance();
              tc_fence_after_sync();
              const uint32_t b_addr = smem_base + kOffRing + s0 * kChunkBytes;
              const uint32_t tmem_o = tmem_base + kColO + (uint32_t)h * 128u;
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const uint32_t a_addr = p_base + (2 * kh + (k >> 2)) * kQChunkBytes + (k & 3) * 32;
                umma_f16<2>(tmem_o, umma_desc_sw128(a_addr, 16, 1024),
                            umma_desc_sw128(b_addr + k * 2048, kChunkBytes, 1024), kIdescPV,
                            (kt_pv > 0 || kh > 0 || k > 0) ? 1u : 0u);
              }
              umma_commit_2_mc(bar(kBarRingEmpty + s0), 3);
              umma_commit_2_mc(bar(kBarRingEmpty + s0 + 1), 3);
            }
          umma_commit_2_mc(bar(kBarPvDone), 3);
          ++kt_pv;
          return true;
        };

        SegIter it(p, item.maxpos);
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
        // all QK^T of this row tile issued: the Q tile is free once they complete
        if (ok) umma_commit_2_mc(bar(kBarQFree), 3);
        while (ok && kt_pv < kt_issued) ok = issue_pv();
      }
    }
  } else if (warp == 2) {
    // ------------------------------ query relocation ----------------------------------------
    uint32_t qfull_phase = 0;
    uint32_t qr_free_phase[2] = {0, 0};
    uint32_t qr_use = 0;
    bool ok = true;
    for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
      const AttnWorkItem item = p.work[w];
      ok = mbar_wait_bounded<false>(bar(kBarQFull), qfull_phase, limit, abort_flag, p.status, W_QFULL, w);
      qfull_phase ^= 1;
      SegIter it(p, item.maxpos);
      while (ok && it.next()) {
        const uint32_t rb = qr_use & 1u;
        if (qr_use >= 2) {
          ok = mbar_wait_bounded<true>(bar(kBarQrFree + rb), qr_free_phase[rb], limit, abort_flag, p.status,
                                       W_QRFREE, w);
          qr_free_phase[rb] ^= 1;
          if (!ok) break;
        }
        ++qr_use;
        const float2* cs = p.seg_cs + (size_t)it.seg * 32;
        const uint8_t* src = smem + kOffQPristine;
        uint8_t* dst = smem + kOffQRot + rb * kQChunkBytes;
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int idx = lane + 32 * i;
          const uint32_t row = idx >> 3, c = idx & 7;
          const uint32_t off = sw128_offset(row, c);
          uint4 v = *reinterpret_cast<const uint4*>(src + off);
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
        if (lane == 0) mbar_arrive_cluster(mapa_shared(bar(kBarQrReady + rb), 0));
      }
    }
    // drain the last releases so that no commit targets this CTA after it exits
    if (lane == 0) {
      for (uint32_t u = (qr_use >= 2 ? qr_use - 2 : 0); u < qr_use && ok; ++u) {
        const uint32_t rb = u & 1u;
        ok = mbar_wait_bounded<true>(bar(kBarQrFree + rb), qr_free_phase[rb], limit, abort_flag, p.status, W_DRAIN,
                                     100 + (int)rb);
        qr_free_phase[rb] ^= 1;
      }
    }
  } else if (warp >= 4) {
    // ------------------------------ softmax / correction / epilogue ----------------------------
    const int L = threadIdx.x - 128;  // TMEM lane
    const int m = L & 63;             // row within this CTA
    const int kh = L >> 6;            // which 128-key half of the tile (and which dims half of O)
    const uint32_t lane_base = ((uint32_t)((warp & 3) * 32)) << 16;
    volatile unsigned long long* xbuf = reinterpret_cast<volatile unsigned long long*>(smem + kOffXchg);
    uint32_t xseq = 0;  // exchange sequence number (warps {4,6} and {5,7} hold the halves of the same rows)
    uint32_t s_full_phase[2] = {0, 0};
    uint32_t pv_done_phase = 0;
    bool ok = true;
    const float scale = p.scale_log2;
    const uint32_t p_ready_remote = mapa_shared(bar(kBarPReady), 0);

    for (int w = pair; w < p.n_tiles && ok; w += p.n_pairs) {
      const AttnWorkItem item = p.work[w];
      const int r = item.tile * kAttnRowsPerPair + (int)crank * kAttnRowsPerCta + m;
      const bool valid = r < p.n_flat;
      int pos = -1;
      if (valid) {
        const int tok = r / p.hpt;
        const int prow = p.rowmap ? p.rowmap[tok] : tok;
        pos = p.row_pos[prow];
      }
      float m_run = -INFINITY, l_run = 0.f;
      int kt = 0;

      SegIter it(p, item.maxpos);
      while (ok && it.next()) {
        const int n_seg = p.seg_off[it.seg + 1] - p.seg_off[it.seg];
        int lim = pos - p.seg_delta[it.seg];           // last visible canonical index
        if (lim > n_seg - 1) lim = n_seg - 1;
        if (pos < 0) lim = -1;
        for (int kb = 0; kb < it.kmax && ok; kb += kAttnKeysPerTile, ++kt) {
          int nv = lim - (kb + kh * 128) + 1;
          nv = nv < 0 ? 0 : (nv > 128 ? 128 : nv);
          const int b = kt & 1;
          ok = mbar_wait_bounded<true>(bar(kBarSFull + b), s_full_phase[b], limit, abort_flag, p.status, W_SFULL, w);
          s_full_phase[b] ^= 1;
          if (!ok) break;
          tc_fence_after_sync();
          uint32_t s[128];
          const uint32_t taddr = tmem_base + lane_base + kColS + (uint32_t)b * 128u;
          tmem_ld_x32(taddr + 0, s + 0);
          tmem_ld_x32(taddr + 32, s + 32);
          tmem_ld_x32(taddr + 64, s + 64);
          tmem_ld_x32(taddr + 96, s + 96);
          tmem_wait_ld();
          float mx = -INFINITY;
#pragma unroll
          for (int c = 0; c < 128; ++c) {
            const float v = (c < nv) ? __uint_as_float(s[c]) : -INFINITY;
            mx = fmaxf(mx, v);
          }
          float mx_other;
          ok = pair_exchange(xbuf, kh, m, ++xseq, mx, mx_other, limit, abort_flag, p.status, w);
          if (!ok) break;
          const float mt = fmaxf(mx, mx_other) * scale;
          // lazy rescale: only when the running maximum grows by more than 2^8
          float alpha = 1.f;
          bool need = false;
          if (mt > m_run + 8.f) {  // also true for the first finite maximum (m_run = -inf)
            alpha = (m_run == -INFINITY) ? 0.f : exp2f(m_run - mt);
            need = (m_run != -INFINITY);
            m_run = mt;
            l_run *= alpha;
          }
          const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
          uint32_t pk[64];
          float lsum = 0.f;
#pragma unroll
          for (int c = 0; c < 128; c += 2) {
            float p0 = (c < nv) ? exp2f(fmaf(__uint_as_float(s[c]), scale, -m_use)) : 0.f;
            float p1 = (c + 1 < nv) ? exp2f(fmaf(__uint_as_float(s[c + 1]), scale, -m_use)) : 0.f;
            lsum += p0 + p1;
            pk[c >> 1] = pack_bf16(p0, p1);
          }
          l_run += lsum;
          // P buffer and O are free once the previous PV has completed
          if (kt > 0) {
            ok = mbar_wait_bounded<true>(bar(kBarPvDone), pv_done_phase, limit, abort_flag, p.status, W_PVDONE, w);
            pv_done_phase ^= 1;
            if (!ok) break;
            tc_fence_after_sync();
            if (__any_sync(0xffffffffu, need)) {
#pragma unroll 1
              for (int cc = 0; cc < 256; cc += 32) {
                uint32_t o[32];
                tmem_ld_x32(tmem_base + lane_base + kColO + cc, o);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                tmem_st_x32(tmem_base + lane_base + kColO + cc, o);
              }
              tmem_wait_st();
            }
          }
          // write P (bf16, K-major 128B swizzle): row m, sub-chunks 2kh and 2kh+1
          uint8_t* pbase = smem + kOffP + (2 * kh) * kQChunkBytes;
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            uint8_t* dstp = pbase + (c >> 3) * kQChunkBytes + sw128_offset((uint32_t)m, (uint32_t)(c & 7));
            *reinterpret_cast<uint4*>(dstp) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          }
          fence_proxy_async_smem();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(p_ready_remote);
        }
      }
      if (!ok) break;
      // ---- epilogue: wait for the last PV, normalise, store ----
      ok = mbar_wait_bounded<true>(bar(kBarPvDone), pv_done_phase, limit, abort_flag, p.status, W_PVDONE, w);
      pv_done_phase ^= 1;
      if (!ok) break;
      tc_fence_after_sync();
      float l_other;
      ok = pair_exchange(xbuf, kh, m, ++xseq, l_run, l_other, limit, abort_flag, p.status, w);
      if (!ok) break;
      const float l_tot = l_run + l_other;
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      __nv_bfloat16* Orow = reinterpret_cast<__nv_bfloat16*>(p.O) + (size_t)(valid ? r : 0) * kDLatent;
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
#pragma unroll 1
        for (int cc = 0; cc < 128; cc += 32) {
          uint32_t o[32];
          tmem_ld_x32(tmem_base + lane_base + kColO + h * 128 + cc, o);
          tmem_wait_ld();
          if (valid) {
            uint4* dstg = reinterpret_cast<uint4*>(Orow + 256 * h + 128 * kh + cc);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint4 v;
              v.x = pack_bf16(__uint_as_float(o[8 * e + 0]) * inv, __uint_as_float(o[8 * e + 1]) * inv);
              v.y = pack_bf16(__uint_as_float(o[8 * e + 2]) * inv, __uint_as_float(o[8 * e + 3]) * inv);
              v.z = pack_bf16(__uint_as_float(o[8 * e + 4]) * inv, __uint_as_float(o[8 * e + 5]) * inv);
              v.w = pack_bf16(__uint_as_float(o[8 * e + 6]) * inv, __uint_as_float(o[8 * e + 7]) * inv);
              dstg[e] = v;
            }
          }
        }
      }
      if (valid && kh == 0)
        p.lse[r] = (l_tot > 0.f) ? (m_run + log2f(l_tot)) * 0.69314718055994530942f : -INFINITY;
      tc_fence_before_sync();
    }
  }

  // ------------------------------ teardown ---------------------------------------------------
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
  return cudaFuncSetAttribute(rk_mla_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

int attention_max_pairs(int sm_count) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (sm_count / 2), 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, rk_mla_attn_kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = sm_count / 2;
  }
  return n < sm_count / 2 ? n : sm_count / 2;
}

cudaError_t launch_attention(const AttnParams& p, int n_pairs, cudaStream_t stream) {
  rk_mla_attn_kernel<<<dim3(2 * n_pairs, 1, 1), dim3(256, 1, 1), kSmemBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rk
