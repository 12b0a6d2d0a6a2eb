// Internal declarations shared by the host layer and the kernel launchers (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rk_ptx.cuh"

namespace rk {

constexpr int kDLatent = 512;
constexpr int kDRope = 64;
constexpr int kDQK = 576;
constexpr int kDV = 128;
constexpr int kGroup = 8;

// ---- attention -----------------------------------------------------------------------
constexpr int kAttnRowsPerCta = 64;    // query rows (token x head pairs) per CTA
constexpr int kAttnRowsPerPair = 128;  // per CTA pair (one UMMA M=128 across two SMs)
constexpr int kAttnKeysPerTile = 256;  // keys per UMMA N

struct AttnWorkItem {
  int32_t tile;    // flattened-row tile index (128 rows each)
  int32_t maxpos;  // largest request position among the tile's rows
};

struct AttnParams {
  CUtensorMap tm_q;   // [n_flat][576] bf16, box 64 cols x 64 rows, 128B swizzle
  CUtensorMap tm_kv;  // [T][576] bf16, box 64 cols x 128 rows, 128B swizzle
  const int32_t* row_pos;    // [T] request position of each packed row
  const int32_t* rowmap;     // [n_tok] token slot -> packed row, or nullptr (identity)
  const int32_t* seg_off;    // [S+1]
  const int32_t* seg_delta;  // [S]
  const float2* seg_cs;      // [S][32] (cos, sin)(delta_i * theta_j)
  const AttnWorkItem* work;  // [n_tiles] cost-descending
  void* O;                   // bf16 [n_flat][512] (output-phase instantiation: [n_flat][576])
  float* lse;                // [n_flat]
  DeviceStatus* status;
  unsigned long long wait_ns;
  int32_t n_segs;
  int32_t n_tiles;
  int32_t n_flat;  // tokens * heads_per_token
  int32_t hpt;     // heads per token in this pass (G or L)
  int32_t n_pairs;
  float scale_log2;  // sm_scale * log2(e)
  int32_t isolated;  // 1: a row sees only its own segment (documents built alone, Algorithm 1)
  int32_t row_base;  // packed row of token slot 0 when rowmap is null
  int32_t n_rows_total;  // T: bound of every packed-row index (read by the bounds-checked build)
  double rope_turns[32];  // theta_j / (2 pi), j = 0..31 (used by the output-phase instantiation only)
};

cudaError_t launch_attention(const AttnParams& p, int n_pairs, bool value_phase, bool starve_loads, cudaStream_t stream);
cudaError_t attention_setup();  // sets the dynamic shared memory attribute once
int attention_max_pairs(int sm_count);

// ---- batched GEMM  C[M,N] = A[M,K] * B[N,K]^T  (bf16 in, fp32 accumulate, bf16 out) ----------
struct GemmBatch {
  int32_t a_col0;   // column offset of this batch's A block
  int32_t b_row0;   // row offset of this batch's B block
  int32_t b_col0;   // column offset of this batch's B block
  int32_t b_skip;   // K index at which a 128-column hole starts in B (or a huge value)
  int32_t c_col0;   // column offset of this batch's C block
  int32_t pad[3];
};

struct GemmParams {
  CUtensorMap tm_a;  // [M rows][a_cols] box 64 x 128
  CUtensorMap tm_b;  // [b_rows][b_cols] box 64 x BN (64 x 128 for the CTA-pair kernel)
  CUtensorMap tm_c;  // [M rows][ldc] box 64 x 128 (epilogue stores)
  void* C;
  const GemmBatch* batches;
  DeviceStatus* status;
  unsigned long long wait_ns;
  int64_t ldc;  // elements
  int32_t M, N, K;
  int32_t n_batches;
};

cudaError_t launch_gemm(const GemmParams& p, int bn, int sm_count, cudaStream_t stream);
cudaError_t gemm_setup();
// single-batch launches with N a multiple of 256 run on CTA pairs; their B tensor map needs a 128-row box
bool gemm_uses_pairs(int M, int N, int n_batches);

// fused sliced first projection of the Global heads: o = O_g W_uv^T stays on chip, z_on_g = o W_a[slice]^T
struct FusedProjParams {
  CUtensorMap tm_a;   // O_g  [M][G * ow]      box 64 x 128
  CUtensorMap tm_b1;  // W_uv [H * 128][ow]    box 64 x 128
  CUtensorMap tm_b2;  // W_a  [G * r_o][1024]  box 64 x 128
  CUtensorMap tm_c;   // z_on_g [M][G * r_o]   box 64 x 128 (stores)
  const GemmBatch* batches_uv;  // per group: a_col0 = g * ow, b_row0 = Global head * 128
  const GemmBatch* batches_wa;  // per group: b_row0 = g * r_o, b_col0 = 128 * slot of the Global head, c_col0 = g * r_o
  DeviceStatus* status;
  unsigned long long wait_ns;
  int32_t M, n_groups, K1, o_rank;
};
cudaError_t launch_proj_fused(const FusedProjParams& p, int sm_count, cudaStream_t stream);
cudaError_t proj_fused_setup();

// ---- streaming kernels -----------------------------------------------------------------------
constexpr int kMergeMaxParts = 4096;  // the merge keeps 8 warps x n_parts weights in shared memory (128 KB at most)
cudaError_t stream_setup();          // raises the merge kernels' dynamic shared memory limit once
cudaError_t launch_relocate(const void* q_rope, int64_t n_rows, int32_t n_heads, int64_t row_stride,
                            int64_t head_stride, const float2* seg_cs, int32_t seg_begin, int32_t seg_end,
                            void* out, int sm_count, cudaStream_t stream);
cudaError_t launch_merge(int32_t n_parts, int64_t n_rh, const void* O_part, int32_t part_dtype,
                         const float* lse_part, void* O, float* lse, int sm_count, cudaStream_t stream);
cudaError_t launch_merge_phase(int32_t n_parts, int64_t n_rows, int32_t n_heads, const void* O_part, int32_t part_dtype,
                               const float* lse_part, const float2* seg_cs, const int32_t* row_pos, const double* rope_turns,
                               void* O, float* lse, int sm_count, cudaStream_t stream);
cudaError_t launch_combine(const void* z_on_g, const void* z_on_l, const void* z_off, const int32_t* inv_map, int64_t T,
                           int64_t width, void* z, int64_t n_prot, DeviceStatus* status, int sm_count, cudaStream_t stream);
cudaError_t launch_check_selftest(DeviceStatus* status, cudaStream_t stream);  // does something in the bounds-checked build only

// ---- selection rules (Eq. protected, Eq. moe) --------------------------------------------------
constexpr uint8_t kPolicyStructural = 1, kPolicyCandidate = 2, kPolicyDirty = 4;

struct PolicyState {
  unsigned n_cand, n_struct_cand, blocks_done, n_top, k_rem, done;
  unsigned long long prefix;  // digits of the n_top-th largest (score,row) key found so far
  unsigned hist[256];
};

struct PolicyParams {
  const int32_t* seg_off;
  const int32_t* seg_delta;
  const uint8_t* seg_has_artifact;
  const float* scores;
  uint8_t* flags;
  PolicyState* state;
  unsigned* block_counts;
  int32_t* rows_out;
  long long* count_out;
  DeviceStatus* status;
  long long req_end, tail_rows;
  int32_t n_segs, T, edge_rows, budget_bp;
};

struct PolicyHost {
  const int32_t* seg_tab_host;  // [seg_off (S+1) | seg_delta (S)]
  const uint8_t* has_host;      // [S]
  int32_t n_segs;
  int64_t T, req_end, tail_rows;
  int32_t edge_rows, budget_bp;
  const int32_t* dirty;
  int64_t n_dirty;
  const float* scores;
  int32_t* rows_out;
  long long* count_out;
  void* workspace;
  DeviceStatus* status;
};

size_t policy_workspace_bytes(int64_t T, int32_t n_segs);
cudaError_t launch_protected_rows(const PolicyHost& h, cudaStream_t stream);
cudaError_t launch_moe_fanout(const float* p, int64_t n, float tau, int fence, uint8_t* k_out, uint8_t* keep_out,
                              cudaStream_t stream);

}  // namespace rk
