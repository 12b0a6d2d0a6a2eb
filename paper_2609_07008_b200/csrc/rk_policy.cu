// Selection rules beside the MLA-Online step, as device-side integer work:
//
//  * the protected token-row set of Eq. (protected): Q u N u D u B_edge u T_tail by a per-row
//    predicate over the segment geometry, then the controller's budget (a share of the candidate
//    rows) filled with the rows of largest Indexer score by an exact radix select over 64-bit keys
//    (score, row), and an order-preserving compaction into the ascending row list;
//  * the retained expert fan-out K_t of Eq. (moe) from the Top-6 router weights.
//
// Everything here is a few bytes per row: the kernels are short streaming passes whose cost is the
// launch, not the traffic.  No kernel waits on another; ordering is stream order.
#include <cuda_runtime.h>

#include <cstdint>

#include "rk_internal.h"

namespace rk {
namespace {

constexpr int kPolicyThreads = 1024;  // rows per block in every per-row pass

__device__ __forceinline__ int find_segment(const int32_t* seg_off, int n_segs, int t) {
  int lo = 0, hi = n_segs - 1;  // largest i with seg_off[i] <= t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (seg_off[mid] <= t) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Order-preserving key of (score, row): larger score first, then lower row.  -0.0 counts as +0.0.
__device__ __forceinline__ unsigned long long select_key(float score, int row) {
  uint32_t u = __float_as_uint(score + 0.0f);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - (uint32_t)row);
}

__global__ void policy_dirty_kernel(const int32_t* dirty, int64_t n_dirty, int64_t T, uint8_t* flags) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_dirty) return;
  const int32_t t = dirty[i];
  if (t >= 0 && t < T) flags[t] = kPolicyDirty;  // same value from every writer of a duplicate
}

// flags[t]: bit 0 structural (Q u N u D u B_edge u T_tail), bit 1 candidate (row of a segment with artifact)
__global__ void __launch_bounds__(kPolicyThreads) policy_flags_kernel(PolicyParams p) {
  const int t = blockIdx.x * kPolicyThreads + threadIdx.x;
  bool cand = false, structural = false;
  if (t < p.T) {
    const int i = find_segment(p.seg_off, p.n_segs, t);
    const int lo = p.seg_off[i], n_i = p.seg_off[i + 1] - lo, j = t - lo;
    const int delta = p.seg_delta[i];
    cand = p.seg_has_artifact[i] != 0;
    structural = !cand || (p.flags[t] & kPolicyDirty) != 0 ||
                 (delta != 0 && (j < p.edge_rows || j >= n_i - p.edge_rows)) ||
                 ((long long)delta + j >= p.req_end - p.tail_rows);
    p.flags[t] = (structural ? kPolicyStructural : 0) | (cand ? kPolicyCandidate : 0);
  }
  const int n_c = __syncthreads_count(cand);
  const int n_sc = __syncthreads_count(cand && structural);
  __shared__ bool last;
  if (threadIdx.x == 0) {
    atomicAdd(&p.state->n_cand, (unsigned)n_c);
    atomicAdd(&p.state->n_struct_cand, (unsigned)n_sc);
    __threadfence();
    last = atomicAdd(&p.state->blocks_done, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {  // the controller's top-up count
    __threadfence();
    const unsigned n_cand = *(volatile unsigned*)&p.state->n_cand;
    const unsigned n_sc_all = *(volatile unsigned*)&p.state->n_struct_cand;
    const unsigned long long budget = (unsigned long long)p.budget_bp * n_cand / 10000ull;
    unsigned n_top = 0;
    if (p.scores != nullptr && budget > n_sc_all) {
      n_top = (unsigned)(budget - n_sc_all);
      if (n_top > n_cand - n_sc_all) n_top = n_cand - n_sc_all;
    }
    p.state->n_top = n_top;
    p.state->k_rem = n_top;
    p.state->prefix = 0ull;
    p.state->blocks_done = 0u;
  }
}

// One digit of the radix select, most significant first: histogram of digit `d` over the eligible
// rows whose higher digits equal the prefix found so far; the last block to finish picks the digit
// that holds the k_rem-th largest key and leaves the histogram clean for the next pass.
__global__ void __launch_bounds__(kPolicyThreads) policy_select_kernel(PolicyParams p, int d) {
  // nothing to pick, or an earlier digit already ended the search (its whole bin was needed, so the
  // prefix with zeros below it is the threshold)
  if (*(volatile unsigned*)&p.state->n_top == 0u || *(volatile unsigned*)&p.state->done != 0u) return;
  __shared__ unsigned hist[256];
  __shared__ bool last;
  if (threadIdx.x < 256) hist[threadIdx.x] = 0u;
  __syncthreads();
  const int t = blockIdx.x * kPolicyThreads + threadIdx.x;
  unsigned bin = 0xffffffffu;  // not counted
  if (t < p.T && (p.flags[t] & (kPolicyStructural | kPolicyCandidate)) == kPolicyCandidate) {
    const unsigned long long key = select_key(p.scores[t], t);
    const unsigned long long prefix = p.state->prefix;
    const bool match = (d == 7) || ((key >> (8 * (d + 1))) == (prefix >> (8 * (d + 1))));
    if (match) bin = (unsigned)(key >> (8 * d)) & 255u;
  }
  // scores cluster in a few exponent bins: one shared-memory atomic per distinct bin of a warp
  const unsigned peers = __match_any_sync(0xffffffffu, bin);
  if (bin != 0xffffffffu && (threadIdx.x & 31) == (unsigned)(__ffs(peers) - 1)) atomicAdd(&hist[bin], (unsigned)__popc(peers));
  __syncthreads();
  if (threadIdx.x < 256 && hist[threadIdx.x] != 0u) atomicAdd(&p.state->hist[threadIdx.x], hist[threadIdx.x]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(&p.state->blocks_done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    volatile unsigned* gh = p.state->hist;
    unsigned k = p.state->k_rem, above = 0u;
    int digit = 0;
    for (int b = 255; b >= 0; --b) {
      const unsigned h = gh[b];
      if (above + h >= k) { digit = b; break; }
      above += h;
    }
    p.state->k_rem = k - above;
    p.state->prefix |= (unsigned long long)digit << (8 * d);
    if (above + gh[digit] == k) p.state->done = 1u;
    for (int b = 0; b < 256; ++b) gh[b] = 0u;
    p.state->blocks_done = 0u;
  }
}

__device__ __forceinline__ bool row_selected(const PolicyParams& p, int t, unsigned n_top, unsigned long long thr) {
  if (t >= p.T) return false;
  const uint8_t f = p.flags[t];
  if (f & kPolicyStructural) return true;
  return n_top != 0u && (f & kPolicyCandidate) && select_key(p.scores[t], t) >= thr;
}

__global__ void __launch_bounds__(kPolicyThreads) policy_count_kernel(PolicyParams p) {
  const unsigned n_top = p.state->n_top;
  const unsigned long long thr = p.state->prefix;  // after the last pass: the n_top-th largest key itself
  const int t = blockIdx.x * kPolicyThreads + threadIdx.x;
  const int n = __syncthreads_count(row_selected(p, t, n_top, thr));
  if (threadIdx.x == 0) p.block_counts[blockIdx.x] = (unsigned)n;
}

// exclusive scan of the block counts by one block; also writes the total
__global__ void __launch_bounds__(kPolicyThreads) policy_scan_kernel(PolicyParams p, int n_blocks) {
  __shared__ unsigned warp_sums[32];
  __shared__ unsigned carry;
  if (threadIdx.x == 0) carry = 0u;
  __syncthreads();
  for (int base = 0; base < n_blocks; base += kPolicyThreads) {
    const int i = base + threadIdx.x;
    const unsigned v = i < n_blocks ? p.block_counts[i] : 0u;
    unsigned x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, x, o);
      if ((threadIdx.x & 31) >= o) x += y;
    }
    if ((threadIdx.x & 31) == 31) warp_sums[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x < 32) {
      unsigned w = warp_sums[threadIdx.x];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned y = __shfl_up_sync(0xffffffffu, w, o);
        if (threadIdx.x >= o) w += y;
      }
      warp_sums[threadIdx.x] = w;
    }
    __syncthreads();
    const unsigned before = carry + (threadIdx.x >= 32 ? warp_sums[(threadIdx.x >> 5) - 1] : 0u) + x - v;
    if (i < n_blocks) p.block_counts[i] = before;
    __syncthreads();
    if (threadIdx.x == kPolicyThreads - 1) carry = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) *p.count_out = (long long)carry;
}

__global__ void __launch_bounds__(kPolicyThreads) policy_scatter_kernel(PolicyParams p) {
  __shared__ unsigned warp_sums[32];
  const unsigned n_top = p.state->n_top;
  const unsigned long long thr = p.state->prefix;
  const int t = blockIdx.x * kPolicyThreads + threadIdx.x;
  const bool sel = row_selected(p, t, n_top, thr);
  const unsigned ballot = __ballot_sync(0xffffffffu, sel);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) warp_sums[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    const unsigned v = warp_sums[lane];
    unsigned x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    warp_sums[lane] = x - v;
  }
  __syncthreads();
  if (sel) {
    const unsigned at = p.block_counts[blockIdx.x] + warp_sums[warp] + __popc(ballot & ((1u << lane) - 1u));
    if (rk_index_ok(at < (unsigned)p.T, p.status, RK_CHK_COMPACT, at)) p.rows_out[at] = t;
  }
}

// Eq. (moe) for one token.  The six weights are sorted by a 12-exchange min/max network (values only:
// equal weights are interchangeable in the sums); the sums run in sorted order in float32.  Which slots
// stay: every slot above the K_t-th largest value, and of the slots equal to it as many of the lowest as
// are still needed (equal weights: lower slot first).  Returns K_t | keep << 8.
__device__ __forceinline__ unsigned moe_fanout_token(const float (&w)[6], float tau, int fence) {
  float s[6] = {w[0], w[1], w[2], w[3], w[4], w[5]};
#define RK_CE(i, j) { const float hi = fmaxf(s[i], s[j]), lo = fminf(s[i], s[j]); s[i] = hi; s[j] = lo; }
  RK_CE(0, 5) RK_CE(1, 3) RK_CE(2, 4)
  RK_CE(1, 2) RK_CE(3, 4)
  RK_CE(0, 3) RK_CE(2, 5)
  RK_CE(0, 1) RK_CE(2, 3) RK_CE(4, 5)
  RK_CE(1, 2) RK_CE(3, 4)
#undef RK_CE
  const float c3 = __fadd_rn(__fadd_rn(s[0], s[1]), s[2]);
  const float c4 = __fadd_rn(c3, s[3]);
  const float c5 = __fadd_rn(c4, s[4]);
  const float c6 = __fadd_rn(c5, s[5]);
  int k = 6;
  float v = s[5];  // the K_t-th largest value
  if (!fence) {
    const float thr = __fmul_rn(tau, c6);
    if (c3 >= thr) { k = 3; v = s[2]; }
    else if (c4 >= thr) { k = 4; v = s[3]; }
    else if (c5 >= thr) { k = 5; v = s[4]; }
  }
  unsigned gt = 0u, eq = 0u;
#pragma unroll
  for (int q = 0; q < 6; ++q) {
    gt |= (w[q] > v ? 1u : 0u) << q;
    eq |= (w[q] == v ? 1u : 0u) << q;
  }
  int need = k - __popc(gt);       // slots still to take among those equal to v (at least one)
  unsigned keep = gt | eq;
  if (__popc(eq) != need) {        // more equal slots than places: the lowest slots win
    keep = gt;
    for (unsigned m = eq; need > 0; --need) {
      const unsigned low = m & (0u - m);
      keep |= low;
      m ^= low;
    }
  }
  return (unsigned)k | (keep << 8);
}

// One token per thread (any alignment; also the tail of the four-token kernel).
__global__ void __launch_bounds__(256) moe_fanout_kernel(const float* __restrict__ p, long long n, float tau, int fence,
                                                         uint8_t* __restrict__ k_out, uint8_t* __restrict__ keep_out) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const float2* src = reinterpret_cast<const float2*>(p + 6 * t);
  const float2 a = __ldcs(src), b = __ldcs(src + 1), c = __ldcs(src + 2);
  const float w[6] = {a.x, a.y, b.x, b.y, c.x, c.y};
  const unsigned r = moe_fanout_token(w, tau, fence);
  k_out[t] = (uint8_t)(r & 0xffu);
  keep_out[t] = (uint8_t)(r >> 8);
}

// Four consecutive tokens per thread: 96 contiguous bytes in as six 16-byte loads, the four K_t and the
// four masks out as one 32-bit store each.  Against one token per thread that removes most of the load,
// store and address instructions (about a tenth of the work per token) and gives every thread four
// independent chains, which is what an issue-bound streaming kernel needs.  n4 = number of token quads.
__global__ void __launch_bounds__(256) moe_fanout4_kernel(const float4* __restrict__ p, long long n4, float tau, int fence,
                                                          uint32_t* __restrict__ k_out, uint32_t* __restrict__ keep_out) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n4) return;
  const float4* src = p + 6 * t;
  float4 v[6];
#pragma unroll
  for (int i = 0; i < 6; ++i) v[i] = __ldcs(src + i);
  const float f[24] = {v[0].x, v[0].y, v[0].z, v[0].w, v[1].x, v[1].y, v[1].z, v[1].w, v[2].x, v[2].y, v[2].z, v[2].w,
                       v[3].x, v[3].y, v[3].z, v[3].w, v[4].x, v[4].y, v[4].z, v[4].w, v[5].x, v[5].y, v[5].z, v[5].w};
  uint32_t kk = 0u, mm = 0u;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const float w[6] = {f[6 * u], f[6 * u + 1], f[6 * u + 2], f[6 * u + 3], f[6 * u + 4], f[6 * u + 5]};
    const unsigned r = moe_fanout_token(w, tau, fence);
    kk |= (r & 0xffu) << (8 * u);
    mm |= (r >> 8) << (8 * u);
  }
  __stcs(k_out + t, kk);
  __stcs(keep_out + t, mm);
}

}  // namespace

size_t policy_workspace_bytes(int64_t T, int32_t n_segs) {
  const size_t n_blocks = (size_t)((T + kPolicyThreads - 1) / kPolicyThreads);
  size_t b = 0;
  b += ((sizeof(PolicyState) + 255) / 256) * 256;
  b += (((size_t)(2 * n_segs + 1) * 4 + 255) / 256) * 256;  // seg_off, seg_delta
  b += (((size_t)n_segs + 255) / 256) * 256;                // seg_has_artifact
  b += (((size_t)T + 255) / 256) * 256;                     // flags
  b += ((n_blocks * 4 + 255) / 256) * 256;                  // block counts / offsets
  return b;
}

cudaError_t launch_protected_rows(const PolicyHost& h, cudaStream_t stream) {
  // carve the workspace
  uint8_t* w = static_cast<uint8_t*>(h.workspace);
  auto take = [&](size_t bytes) { uint8_t* r = w; w += ((bytes + 255) / 256) * 256; return r; };
  PolicyParams p = {};
  p.state = reinterpret_cast<PolicyState*>(take(sizeof(PolicyState)));
  int32_t* seg_tab = reinterpret_cast<int32_t*>(take((size_t)(2 * h.n_segs + 1) * 4));
  uint8_t* has = take((size_t)h.n_segs);
  p.flags = take((size_t)h.T);
  const int n_blocks = (int)((h.T + kPolicyThreads - 1) / kPolicyThreads);
  p.block_counts = reinterpret_cast<unsigned*>(take((size_t)n_blocks * 4));
  p.seg_off = seg_tab;
  p.seg_delta = seg_tab + h.n_segs + 1;
  p.seg_has_artifact = has;
  p.n_segs = h.n_segs;
  p.T = (int)h.T;
  p.edge_rows = h.edge_rows;
  p.tail_rows = h.tail_rows;
  p.req_end = h.req_end;
  p.budget_bp = h.budget_bp;
  p.scores = h.scores;
  p.rows_out = h.rows_out;
  p.count_out = h.count_out;
  p.status = h.status;

  cudaError_t e;
  // h.seg_tab_host: [seg_off (S+1) | seg_delta (S)] as int32, h.has_host: [S]; both stay alive in the
  // caller until the copies are done (pageable memory: the copy is staged before the call returns)
  if ((e = cudaMemcpyAsync(seg_tab, h.seg_tab_host, (size_t)(2 * h.n_segs + 1) * 4, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return e;
  if ((e = cudaMemcpyAsync(has, h.has_host, (size_t)h.n_segs, cudaMemcpyHostToDevice, stream)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(p.state, 0, sizeof(PolicyState), stream)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(p.flags, 0, (size_t)h.T, stream)) != cudaSuccess) return e;
  if (h.n_dirty > 0) {
    const int64_t nb = (h.n_dirty + 255) / 256;
    policy_dirty_kernel<<<(unsigned)nb, 256, 0, stream>>>(h.dirty, h.n_dirty, h.T, p.flags);
  }
  policy_flags_kernel<<<n_blocks, kPolicyThreads, 0, stream>>>(p);
  if (h.scores != nullptr && h.budget_bp > 0)
    for (int d = 7; d >= 0; --d) policy_select_kernel<<<n_blocks, kPolicyThreads, 0, stream>>>(p, d);
  policy_count_kernel<<<n_blocks, kPolicyThreads, 0, stream>>>(p);
  policy_scan_kernel<<<1, kPolicyThreads, 0, stream>>>(p, n_blocks);
  policy_scatter_kernel<<<n_blocks, kPolicyThreads, 0, stream>>>(p);
  return cudaGetLastError();
}

int protected_rows_launches(bool with_scores, bool with_dirty) { return 4 + (with_dirty ? 1 : 0) + (with_scores ? 8 : 0); }

cudaError_t launch_moe_fanout(const float* p, int64_t n, float tau, int fence, uint8_t* k_out, uint8_t* keep_out,
                              cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  int64_t done = 0;
  const bool vec = (reinterpret_cast<uintptr_t>(p) & 15u) == 0 && (reinterpret_cast<uintptr_t>(k_out) & 3u) == 0 &&
                   (reinterpret_cast<uintptr_t>(keep_out) & 3u) == 0;
  if (vec && n >= 4) {
    const int64_t n4 = n / 4;
    moe_fanout4_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, stream>>>(reinterpret_cast<const float4*>(p), (long long)n4, tau,
                                                                         fence, reinterpret_cast<uint32_t*>(k_out),
                                                                         reinterpret_cast<uint32_t*>(keep_out));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    done = 4 * n4;
  }
  if (done < n) {
    const int64_t rest = n - done;
    moe_fanout_kernel<<<(unsigned)((rest + 255) / 256), 256, 0, stream>>>(p + 6 * done, (long long)rest, tau, fence,
                                                                          k_out + done, keep_out + done);
  }
  return cudaGetLastError();
}

}  // namespace rk
