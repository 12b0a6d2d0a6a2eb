// HBM-bound steps of the MLA-Online layer: standalone query relocation (Algorithm 2,
// q_i = R(-delta_i) q), standalone segmented log-sum-exp merge (SegmentedLSEMerge) and
// restore-and-replace (z = z_on_g + (row in A ? z_on_l : z_off)).  16-byte vector accesses,
// consecutive threads on consecutive addresses, grids sized in multiples of the SM count.
#include <cuda_bf16.h>
#include <math.h>

#include "rk_internal.h"

namespace rk {
namespace {

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162*>(&w[e]);
    f[2 * e] = __bfloat162float(x.x);
    f[2 * e + 1] = __bfloat162float(x.y);
  }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}

// A thread owns kRelU 16-byte chunks (4 rotation pairs each) of the input, 256 chunks apart, so all of them
// use the same four (cos, sin) pairs of a frame; it keeps them unpacked in registers and writes one rotated
// copy per segment frame.  Per 16 bytes written that leaves the arithmetic, one pack and one store.
// Measured on B200 (6.2 GB written, 0.27 GB read): write-through-L2 plain stores beat st.cs (5.58 against
// 5.20 TB/s), and one block per group of chunks, scheduled in order, beats a persistent grid-stride loop
// (5.89 against 5.58 TB/s): blocks that are handed out in order keep the GPU's writes inside a compact
// moving window of every frame, persistent blocks drift apart.  A plain fill shows the same (one block
// per 16 KB: 7.4 TB/s; persistent, 8 blocks per SM: 5.9 TB/s).
constexpr int kRelU = 4;
__global__ void __launch_bounds__(256) rk_relocate_kernel(const __nv_bfloat16* __restrict__ q, int64_t n_rows,
                                                          int32_t n_heads, int64_t row_stride, int64_t head_stride,
                                                          const float2* __restrict__ seg_cs, int32_t seg_begin,
                                                          int32_t n_frames, __nv_bfloat16* __restrict__ out) {
  const int64_t n_items = n_rows * n_heads * 8;
  const int64_t frame_elems = n_rows * n_heads * 64;
  const int c = (int)(threadIdx.x & 7);
  const int64_t n_groups = (n_items + 256 * kRelU - 1) / (256 * kRelU);
  for (int64_t grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
    const int64_t it0 = grp * (256 * kRelU) + threadIdx.x;
    float x[kRelU][8];
#pragma unroll
    for (int u = 0; u < kRelU; ++u) {
      const int64_t it = it0 + u * 256;
      if (it < n_items) {
        const int64_t rh = it >> 3;
        const int64_t r = (rh < (int64_t)0x7fffffff) ? (int64_t)((uint32_t)rh / (uint32_t)n_heads) : rh / n_heads;
        const int h = (int)(rh - r * n_heads);
        unpack8(__ldcs(reinterpret_cast<const uint4*>(q + r * row_stride + h * head_stride + c * 8)), x[u]);
      }
    }
    // Frames are whole multiples of a megabyte apart, so writing frame i from every block at the same
    // time would hit the same memory channels; each group of chunks starts at a different frame instead.
    int i = (int)(grp % (int64_t)n_frames);
#pragma unroll 2
    for (int n = 0; n < n_frames; ++n) {
      const float4* cs = reinterpret_cast<const float4*>(seg_cs + (size_t)(seg_begin + i) * 32 + 4 * c);
      const float4 t01 = __ldg(cs), t23 = __ldg(cs + 1);
      __nv_bfloat16* dst = out + (int64_t)i * frame_elems + it0 * 8;
#pragma unroll
      for (int u = 0; u < kRelU; ++u) {
        if (it0 + u * 256 < n_items) {
          float y[8];
          // R(-delta): (x0, x1) -> (x0 cos + x1 sin, x1 cos - x0 sin)
          y[0] = x[u][0] * t01.x + x[u][1] * t01.y;  y[1] = x[u][1] * t01.x - x[u][0] * t01.y;
          y[2] = x[u][2] * t01.z + x[u][3] * t01.w;  y[3] = x[u][3] * t01.z - x[u][2] * t01.w;
          y[4] = x[u][4] * t23.x + x[u][5] * t23.y;  y[5] = x[u][5] * t23.x - x[u][4] * t23.y;
          y[6] = x[u][6] * t23.z + x[u][7] * t23.w;  y[7] = x[u][7] * t23.z - x[u][6] * t23.w;
          *reinterpret_cast<uint4*>(dst + u * 2048) = pack8(y);
        }
      }
      i = (i + 1 == n_frames) ? 0 : i + 1;
    }
  }
}

// One warp per (row, head): weights from the per-part LSE (max-subtracted), then the weighted
// sum of the 512-wide partial outputs; lane l owns dims [8l, 8l+8) and [256+8l, 256+8l+8).
template <bool kF32>
__global__ void __launch_bounds__(256) rk_merge_kernel(int32_t n_parts, int64_t n_rh, const void* __restrict__ O_part,
                                                       const float* __restrict__ lse_part,
                                                       __nv_bfloat16* __restrict__ O, float* __restrict__ lse) {
  extern __shared__ float wsm[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* w = wsm + (size_t)warp * n_parts;
  const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t rh = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp; rh < n_rh; rh += n_warps) {
    float mx = -INFINITY;
    for (int j = lane; j < n_parts; j += 32) {
      const float l = __ldg(lse_part + (int64_t)j * n_rh + rh);
      w[j] = l;
      mx = fmaxf(mx, l);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float m_safe = (mx == -INFINITY) ? 0.f : mx;
    float tot = 0.f;
    __syncwarp();
    for (int j = lane; j < n_parts; j += 32) {
      const float e = __expf(w[j] - m_safe);  // exp(-inf) = 0 for empty parts
      w[j] = e;
      tot += e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
    __syncwarp();
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
    float acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.f;
    // The loads of kMergeU parts are issued together and without looking at the weights (an empty part's
    // rows are valid memory; what they hold is never used), so that a warp keeps kMergeU KB in flight
    // instead of one; only the arithmetic is skipped for a part of weight zero.
    constexpr int kMergeU = 4;
    const int64_t part_stride = n_rh * 512;
    for (int j0 = 0; j0 < n_parts; j0 += kMergeU) {
      float wj[kMergeU];
#pragma unroll
      for (int u = 0; u < kMergeU; ++u) wj[u] = (j0 + u < n_parts) ? w[j0 + u] * inv : 0.f;
      if (kF32) {
        float4 v[kMergeU][4];
        const float* src = reinterpret_cast<const float*>(O_part) + ((int64_t)j0 * n_rh + rh) * 512 + 8 * lane;
#pragma unroll
        for (int u = 0; u < kMergeU; ++u)
          if (j0 + u < n_parts) {
            v[u][0] = __ldcs(reinterpret_cast<const float4*>(src + u * part_stride));
            v[u][1] = __ldcs(reinterpret_cast<const float4*>(src + u * part_stride + 4));
            v[u][2] = __ldcs(reinterpret_cast<const float4*>(src + u * part_stride + 256));
            v[u][3] = __ldcs(reinterpret_cast<const float4*>(src + u * part_stride + 260));
          }
#pragma unroll
        for (int u = 0; u < kMergeU; ++u)
          if (wj[u] > 0.f) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              acc[4 * q + 0] += wj[u] * v[u][q].x; acc[4 * q + 1] += wj[u] * v[u][q].y;
              acc[4 * q + 2] += wj[u] * v[u][q].z; acc[4 * q + 3] += wj[u] * v[u][q].w;
            }
          }
      } else {
        uint4 v[kMergeU][2];
        const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(O_part) + ((int64_t)j0 * n_rh + rh) * 512 + 8 * lane;
#pragma unroll
        for (int u = 0; u < kMergeU; ++u)
          if (j0 + u < n_parts) {
            v[u][0] = __ldcs(reinterpret_cast<const uint4*>(src + u * part_stride));
            v[u][1] = __ldcs(reinterpret_cast<const uint4*>(src + u * part_stride + 256));
          }
#pragma unroll
        for (int u = 0; u < kMergeU; ++u)
          if (wj[u] > 0.f) {
            float f[16];
            unpack8(v[u][0], f);
            unpack8(v[u][1], f + 8);
#pragma unroll
            for (int e = 0; e < 16; ++e) acc[e] += wj[u] * f[e];
          }
      }
    }
    __nv_bfloat16* dst = O + rh * 512;
    *reinterpret_cast<uint4*>(dst + 8 * lane) = pack8(acc);
    *reinterpret_cast<uint4*>(dst + 256 + 8 * lane) = pack8(acc + 8);
    if (lane == 0) lse[rh] = tot > 0.f ? m_safe + logf(tot) : -INFINITY;
    __syncwarp();
  }
}

// The merge for per-segment partial results of the output-phase variant (Algorithm 2: RestorePhase, then
// SegmentedLSEMerge, then the inverse output RoPE of Eq. offonline).  Rows are 576 wide; the 512 latent dims
// merge as above, the 64 rope dims (lanes 0-7, 8 dims = 4 rotation pairs each) are turned by
// R(+delta of the part's segment) before they are added and by R(-row position) at the end.
struct MergePhaseArgs {
  const float2* seg_cs;    // [S][32] (cos, sin)(delta_i theta_j), first part's segment first
  const int32_t* row_pos;  // [n_rows] or nullptr
  int32_t n_heads;
  double rope_turns[32];   // theta_j / (2 pi)
};

template <bool kF32>
__global__ void __launch_bounds__(256) rk_merge_phase_kernel(int32_t n_parts, int64_t n_rh, const void* __restrict__ O_part,
                                                             const float* __restrict__ lse_part, const MergePhaseArgs a,
                                                             __nv_bfloat16* __restrict__ O, float* __restrict__ lse) {
  extern __shared__ float wsm[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* w = wsm + (size_t)warp * n_parts;
  const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t rh = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp; rh < n_rh; rh += n_warps) {
    float mx = -INFINITY;
    for (int j = lane; j < n_parts; j += 32) {
      const float l = __ldg(lse_part + (int64_t)j * n_rh + rh);
      w[j] = l;
      mx = fmaxf(mx, l);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float m_safe = (mx == -INFINITY) ? 0.f : mx;
    float tot = 0.f;
    __syncwarp();
    for (int j = lane; j < n_parts; j += 32) {
      const float e = __expf(w[j] - m_safe);
      w[j] = e;
      tot += e;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
    __syncwarp();
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
    float acc[16], accr[8];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) accr[e] = 0.f;
    for (int j = 0; j < n_parts; ++j) {
      const float wj = w[j] * inv;
      if (wj > 0.f) {
        float f[24];
        if (kF32) {
          const float* src = reinterpret_cast<const float*>(O_part) + ((int64_t)j * n_rh + rh) * 576;
#pragma unroll
          for (int hlf = 0; hlf < 2; ++hlf) {
            const float4 x = __ldcs(reinterpret_cast<const float4*>(src + 256 * hlf + 8 * lane));
            const float4 y = __ldcs(reinterpret_cast<const float4*>(src + 256 * hlf + 8 * lane + 4));
            f[8 * hlf + 0] = x.x; f[8 * hlf + 1] = x.y; f[8 * hlf + 2] = x.z; f[8 * hlf + 3] = x.w;
            f[8 * hlf + 4] = y.x; f[8 * hlf + 5] = y.y; f[8 * hlf + 6] = y.z; f[8 * hlf + 7] = y.w;
          }
          if (lane < 8) {
            const float4 x = __ldcs(reinterpret_cast<const float4*>(src + 512 + 8 * lane));
            const float4 y = __ldcs(reinterpret_cast<const float4*>(src + 512 + 8 * lane + 4));
            f[16] = x.x; f[17] = x.y; f[18] = x.z; f[19] = x.w; f[20] = y.x; f[21] = y.y; f[22] = y.z; f[23] = y.w;
          }
        } else {
          const __nv_bfloat16* src = reinterpret_cast<const __nv_bfloat16*>(O_part) + ((int64_t)j * n_rh + rh) * 576;
          unpack8(__ldcs(reinterpret_cast<const uint4*>(src + 8 * lane)), f);
          unpack8(__ldcs(reinterpret_cast<const uint4*>(src + 256 + 8 * lane)), f + 8);
          if (lane < 8) unpack8(__ldcs(reinterpret_cast<const uint4*>(src + 512 + 8 * lane)), f + 16);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] += wj * f[e];
        if (lane < 8) {  // RestorePhase: R(+delta): (x0, x1) -> (x0 cos - x1 sin, x0 sin + x1 cos)
          const float4* cs = reinterpret_cast<const float4*>(a.seg_cs + (size_t)j * 32 + 4 * lane);
          const float4 t01 = __ldg(cs), t23 = __ldg(cs + 1);
          accr[0] += wj * (f[16] * t01.x - f[17] * t01.y);  accr[1] += wj * (f[16] * t01.y + f[17] * t01.x);
          accr[2] += wj * (f[18] * t01.z - f[19] * t01.w);  accr[3] += wj * (f[18] * t01.w + f[19] * t01.z);
          accr[4] += wj * (f[20] * t23.x - f[21] * t23.y);  accr[5] += wj * (f[20] * t23.y + f[21] * t23.x);
          accr[6] += wj * (f[22] * t23.z - f[23] * t23.w);  accr[7] += wj * (f[22] * t23.w + f[23] * t23.z);
        }
      }
    }
    __nv_bfloat16* dst = O + rh * 576;
    *reinterpret_cast<uint4*>(dst + 8 * lane) = pack8(acc);
    *reinterpret_cast<uint4*>(dst + 256 + 8 * lane) = pack8(acc + 8);
    if (lane < 8) {
      if (a.row_pos != nullptr) {  // inverse output RoPE at the row's request position
        const int pos = a.row_pos[rh / a.n_heads];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const double t = -(double)pos * a.rope_turns[4 * lane + i];
          float sn, c;
          sincospif(2.f * (float)(t - rint(t)), &sn, &c);
          const float x0 = accr[2 * i], x1 = accr[2 * i + 1];
          accr[2 * i] = x0 * c - x1 * sn;
          accr[2 * i + 1] = x0 * sn + x1 * c;
        }
      }
      *reinterpret_cast<uint4*>(dst + 512 + 8 * lane) = pack8(accr);
    }
    if (lane == 0) lse[rh] = tot > 0.f ? m_safe + logf(tot) : -INFINITY;
    __syncwarp();
  }
}

// z = z_on_g + (protected ? z_on_l[slot] : z_off[row]): a per-row select, never an add of both.
__global__ void __launch_bounds__(256) rk_combine_kernel(const __nv_bfloat16* __restrict__ z_on_g,
                                                         const __nv_bfloat16* __restrict__ z_on_l,
                                                         const __nv_bfloat16* __restrict__ z_off,
                                                         const int32_t* __restrict__ inv_map, int64_t T, int64_t width,
                                                         __nv_bfloat16* __restrict__ z, int64_t n_prot, DeviceStatus* status) {
  const int64_t cpr = width >> 3;  // 16-byte chunks per row
  const int64_t n_items = T * cpr;
  for (int64_t it = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; it < n_items;
       it += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = it / cpr;
    const int64_t c = it - t * cpr;
    const int32_t slot = __ldg(inv_map + t);
    if (!rk_index_ok(slot < n_prot, status, RK_CHK_INV_MAP, slot)) continue;
    const uint4 a = __ldcs(reinterpret_cast<const uint4*>(z_on_g + t * width) + c);
    const uint4 b = slot >= 0 ? __ldcs(reinterpret_cast<const uint4*>(z_on_l + (int64_t)slot * width) + c)
                              : __ldcs(reinterpret_cast<const uint4*>(z_off + t * width) + c);
    float fa[8], fb[8];
    unpack8(a, fa);
    unpack8(b, fb);
#pragma unroll
    for (int e = 0; e < 8; ++e) fa[e] += fb[e];
    *(reinterpret_cast<uint4*>(z + t * width) + c) = pack8(fa);
  }
}

inline int grid_for(int64_t n_threads_needed, int sm_count, int per_sm) {
  int64_t blocks = (n_threads_needed + 255) / 256;
  int64_t cap = (int64_t)sm_count * per_sm;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace

cudaError_t stream_setup() {
  const int bytes = 8 * kMergeMaxParts * (int)sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(rk_merge_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(rk_merge_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(rk_merge_phase_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(rk_merge_phase_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  return e;
}

cudaError_t launch_merge_phase(int32_t n_parts, int64_t n_rows, int32_t n_heads, const void* O_part, int32_t part_dtype,
                               const float* lse_part, const float2* seg_cs, const int32_t* row_pos, const double* rope_turns,
                               void* O, float* lse, int sm_count, cudaStream_t stream) {
  const int64_t n_rh = n_rows * n_heads;
  if (n_rh == 0) return cudaSuccess;
  MergePhaseArgs a;
  a.seg_cs = seg_cs;
  a.row_pos = row_pos;
  a.n_heads = n_heads;
  for (int j = 0; j < 32; ++j) a.rope_turns[j] = rope_turns[j];
  const size_t smem = (size_t)8 * n_parts * sizeof(float);
  const int grid = grid_for(n_rh * 32, sm_count, 8);
  if (part_dtype == 1)
    rk_merge_phase_kernel<true><<<grid, 256, smem, stream>>>(n_parts, n_rh, O_part, lse_part, a,
                                                              reinterpret_cast<__nv_bfloat16*>(O), lse);
  else
    rk_merge_phase_kernel<false><<<grid, 256, smem, stream>>>(n_parts, n_rh, O_part, lse_part, a,
                                                               reinterpret_cast<__nv_bfloat16*>(O), lse);
  return cudaGetLastError();
}

cudaError_t launch_relocate(const void* q_rope, int64_t n_rows, int32_t n_heads, int64_t row_stride,
                            int64_t head_stride, const float2* seg_cs, int32_t seg_begin, int32_t seg_end, void* out,
                            int sm_count, cudaStream_t stream) {
  const int64_t items = n_rows * n_heads * 8;
  if (items == 0 || seg_end <= seg_begin) return cudaSuccess;
  const int64_t n_groups = (items + 256 * kRelU - 1) / (256 * kRelU);  // one block each, handed out in order
  const int64_t cap = (int64_t)sm_count * 4096;                        // far above what is resident; keeps gridDim.x in range
  rk_relocate_kernel<<<(unsigned)(n_groups < cap ? n_groups : cap), 256, 0, stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(q_rope), n_rows, n_heads, row_stride, head_stride, seg_cs, seg_begin,
      seg_end - seg_begin, reinterpret_cast<__nv_bfloat16*>(out));
  return cudaGetLastError();
}

cudaError_t launch_merge(int32_t n_parts, int64_t n_rh, const void* O_part, int32_t part_dtype, const float* lse_part,
                         void* O, float* lse, int sm_count, cudaStream_t stream) {
  if (n_rh == 0) return cudaSuccess;
  const size_t smem = (size_t)8 * n_parts * sizeof(float);
  // persistent warps: as many blocks as stay resident with four parts' loads in registers (80 / 123 registers)
  const int grid = grid_for(n_rh * 32, sm_count, part_dtype == 1 ? 2 : 3);
  if (part_dtype == 1)
    rk_merge_kernel<true><<<grid, 256, smem, stream>>>(n_parts, n_rh, O_part, lse_part,
                                                        reinterpret_cast<__nv_bfloat16*>(O), lse);
  else
    rk_merge_kernel<false><<<grid, 256, smem, stream>>>(n_parts, n_rh, O_part, lse_part,
                                                         reinterpret_cast<__nv_bfloat16*>(O), lse);
  return cudaGetLastError();
}

__global__ void rk_check_selftest_kernel(DeviceStatus* status) {
  // a deliberately bad index through the checking function: the bounds-checked build records it, nothing is accessed
  rk_index_ok(false, status, RK_CHK_SELFTEST, 12345);
}

cudaError_t launch_check_selftest(DeviceStatus* status, cudaStream_t stream) {
#ifdef RK_CHECK
  rk_check_selftest_kernel<<<1, 32, 0, stream>>>(status);
  return cudaGetLastError();
#else
  (void)status;
  (void)stream;
  return cudaErrorNotSupported;
#endif
}

cudaError_t launch_combine(const void* z_on_g, const void* z_on_l, const void* z_off, const int32_t* inv_map, int64_t T,
                           int64_t width, void* z, int64_t n_prot, DeviceStatus* status, int sm_count, cudaStream_t stream) {
  const int64_t items = T * (width >> 3);
  if (items == 0) return cudaSuccess;
  rk_combine_kernel<<<grid_for(items, sm_count, 8), 256, 0, stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(z_on_g), reinterpret_cast<const __nv_bfloat16*>(z_on_l),
      reinterpret_cast<const __nv_bfloat16*>(z_off), inv_map, T, width, reinterpret_cast<__nv_bfloat16*>(z), n_prot, status);
  return cudaGetLastError();
}

}  // namespace rk
