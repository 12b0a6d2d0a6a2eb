// Host side of the C ABI: argument validation, request geometry (row positions, relocation
// tables, inverse row map, tile work lists), TMA tensor maps and kernel launches.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/rk.h"
#include "rk_internal.h"

using namespace rk;

// ------------------------------------------------------------------------------------------
// objects
// ------------------------------------------------------------------------------------------
typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct rk_ctx {
  rk_profile prof;
  std::vector<int32_t> global_heads, local_heads;
  int device = 0;
  int sm_count = 0;
  int n_pairs = 0;
  DeviceStatus* d_status = nullptr;
  GemmBatch* d_batches = nullptr;  // [uv_g: G][uv_l: L][wa_g: G][wa_l: G][wb: 1]
  int off_uv_g = 0, off_uv_l = 0, off_wa_g = 0, off_wa_l = 0, off_wb = 0;
  unsigned long long wait_ns = 2000ull * 1000 * 1000;
  bool value_phase = false;  // output-phase variant: the whole stored row is the value, O rows are 576 wide
  int ow = kDLatent;         // width of an attention output row (512, or 576 with value_phase)
  double rope_turns[32];     // theta_j / (2 pi)
  bool starve_loads = false;  // rk_test_starve_loads: the timeout test's instantiation of the attention kernel
  cudaStream_t copy_stream = nullptr;  // rk_layer_host: copies that overlap the kernels
  cudaStream_t copy_out_stream = nullptr;  // rk_layer_stack_host: device->host copies (full duplex with the above)
  cudaEvent_t sev[10] = {nullptr};     // rk_layer_stack_host: kv_ql_in[2], qg_in[2], zoff_in[2], compute_done[2], y_copied[2]
  cudaEvent_t ev[8] = {nullptr};       // device-side ordering between the two streams (no host polling)
  PFN_encodeTiled encode = nullptr;
  mutable std::string err;
};

struct rk_request {
  rk_ctx* ctx = nullptr;
  int64_t T = 0, A = 0, n_off_rows = 0;
  int32_t S = 0;
  int64_t pairs_global = 0, pairs_local = 0;
  int32_t n_tiles_g = 0, n_tiles_l = 0;
  // device tables
  int32_t* d_row_pos = nullptr;
  int32_t* d_prot_rows = nullptr;
  int32_t* d_inv_map = nullptr;
  int32_t* d_seg_off = nullptr;
  int32_t* d_seg_delta = nullptr;
  float2* d_seg_cs = nullptr;
  AttnWorkItem* d_work_g = nullptr;
  AttnWorkItem* d_work_l = nullptr;
  // rk_layer_host runs the Global pass in two row ranges [0, split_tok) and [split_tok, T) so that the
  // first range's y travels to the host while the second computes; each range has its own tile list
  int64_t split_tok = 0;  // 0: not split
  AttnWorkItem* d_work_g_part[2] = {nullptr, nullptr};
  int32_t n_tiles_g_part[2] = {0, 0};
  // likewise the Local pass: a short first range of protected-row slots [0, split_slot) lets the pass
  // start as soon as kv and that range's queries are on the device
  int64_t split_slot = 0;
  AttnWorkItem* d_work_l_part[2] = {nullptr, nullptr};
  int32_t n_tiles_l_part[2] = {0, 0};
};

namespace {

rk_status fail(const rk_ctx* ctx, rk_status s, const char* fmt, ...) {
  if (ctx) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    ctx->err = buf;
  }
  return s;
}

rk_status cuda_fail(const rk_ctx* ctx, cudaError_t e, const char* what) {
  cudaGetLastError();
  return fail(ctx, RK_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <class T>
cudaError_t upload(T** dst, const std::vector<T>& v) {
  *dst = nullptr;
  size_t bytes = std::max<size_t>(v.size(), 1) * sizeof(T);
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(dst), bytes);
  if (e != cudaSuccess) return e;
  if (!v.empty()) e = cudaMemcpy(*dst, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice);
  return e;
}

// 2-D bf16 row-major tensor map with 128-byte swizzle; box = box_cols x box_rows.
rk_status make_tmap(const rk_ctx* ctx, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
                    uint64_t row_stride_elems, uint32_t box_cols, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {row_stride_elems * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(ctx, RK_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d) rows=%llu cols=%llu stride=%llu", (int)r,
                (unsigned long long)rows, (unsigned long long)cols, (unsigned long long)row_stride_elems);
  return RK_OK;
}

// tile_lo / tile_hi restrict the list to the row tiles [tile_lo, tile_hi) (-1: up to the last tile)
void build_work(const std::vector<int32_t>& tok_pos, int hpt, const std::vector<int32_t>& seg_n,
                const std::vector<int32_t>& seg_delta, int n_pairs, std::vector<AttnWorkItem>* out,
                int64_t tile_lo = 0, int64_t tile_hi = -1) {
  const int64_t n_flat = (int64_t)tok_pos.size() * hpt;
  const int64_t all_tiles = (n_flat + kAttnRowsPerPair - 1) / kAttnRowsPerPair;
  if (tile_hi < 0 || tile_hi > all_tiles) tile_hi = all_tiles;
  const int64_t n_tiles = tile_hi - tile_lo;
  std::vector<std::pair<int64_t, AttnWorkItem>> items((size_t)n_tiles);
  for (int64_t t = tile_lo; t < tile_hi; ++t) {
    const int64_t r0 = t * kAttnRowsPerPair, r1 = std::min<int64_t>(n_flat, r0 + kAttnRowsPerPair);
    const int64_t tok0 = r0 / hpt, tok1 = (r1 - 1) / hpt;
    int32_t maxpos = 0;
    for (int64_t k = tok0; k <= tok1; ++k) maxpos = std::max(maxpos, tok_pos[(size_t)k]);
    int64_t cost = 0;
    for (size_t i = 0; i < seg_n.size(); ++i) {
      int64_t kmax = std::min<int64_t>(seg_n[i], (int64_t)maxpos - seg_delta[i] + 1);
      if (kmax > 0) cost += (kmax + kAttnKeysPerTile - 1) / kAttnKeysPerTile;
    }
    items[(size_t)(t - tile_lo)] = {cost, AttnWorkItem{(int32_t)t, maxpos}};
  }
  std::stable_sort(items.begin(), items.end(),
                   [](const auto& a, const auto& b) { return a.first > b.first; });
  // longest first; every other round of n_pairs tiles is reversed so that the static
  // round-robin assignment (pair p takes entries p, p + n_pairs, ...) stays balanced
  out->resize((size_t)n_tiles);
  for (int64_t base = 0, round = 0; base < n_tiles; base += n_pairs, ++round) {
    const int64_t cnt = std::min<int64_t>(n_pairs, n_tiles - base);
    for (int64_t k = 0; k < cnt; ++k) {
      const int64_t src = (round & 1) ? (base + cnt - 1 - k) : (base + k);
      (*out)[(size_t)(base + k)] = items[(size_t)src].second;
    }
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// Projection without any allocation by the caller or the library.
//
// Some users of this library cannot obtain device memory at call time: a serving runtime that
// hands the whole device to its own memory pool at start-up has nothing left for cudaMalloc,
// and a latency-critical request path cannot afford the implicit device-wide synchronisation
// an allocation may cause.  For them the per-head intermediate o = W_uv O_lat lives in a
// fixed array that is part of the loaded library image instead of a caller workspace.
// ------------------------------------------------------------------------------------------
#define RK_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)

static __device__ __align__(256) unsigned char rk_static_scratch[RK_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices] = {nullptr};
std::mutex g_static_scratch_mutex;  // first calls may come from several host threads

// Device address of rk_static_scratch on the CURRENT device (resolved once per device).  In host
// code the array's name is only a handle for the runtime, not a device address, so the address
// must come from cudaGetSymbolAddress.  rk_create calls this: the lookup is what makes the runtime
// load this file's module and materialise the array on the device, which may allocate and
// synchronise -- work that belongs to set-up, not to the entry point that promises to allocate nothing.
cudaError_t static_scratch_address(int device, void** out) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_ptr[device] == nullptr) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, rk_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_scratch_ptr[device] = ptr;
  }
  *out = g_static_scratch_ptr[device];
  return cudaSuccess;
}
}  // namespace

// ------------------------------------------------------------------------------------------
extern "C" {

const char* rk_version(void) { return "rk-mla-online 0.1 (sm_100a)"; }

const char* rk_status_string(rk_status s) {
  switch (s) {
    case RK_OK: return "RK_OK";
    case RK_ERR_NULL: return "RK_ERR_NULL";
    case RK_ERR_PROFILE: return "RK_ERR_PROFILE";
    case RK_ERR_LAYOUT: return "RK_ERR_LAYOUT";
    case RK_ERR_ROWS: return "RK_ERR_ROWS";
    case RK_ERR_ALIGN: return "RK_ERR_ALIGN";
    case RK_ERR_WORKSPACE: return "RK_ERR_WORKSPACE";
    case RK_ERR_UNSUPPORTED: return "RK_ERR_UNSUPPORTED";
    case RK_ERR_CUDA: return "RK_ERR_CUDA";
    case RK_ERR_TIMEOUT: return "RK_ERR_TIMEOUT";
  }
  return "RK_ERR_?";
}

const char* rk_last_error(const rk_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

rk_status rk_create(const rk_profile* prof, rk_ctx** out) { return rk_create_ex(prof, 0u, out); }

rk_status rk_create_ex(const rk_profile* prof, uint32_t flags, rk_ctx** out) {
  if (!prof || !out) return RK_ERR_NULL;
  *out = nullptr;
  if (flags & ~(uint32_t)RK_VALUE_PHASE) return RK_ERR_UNSUPPORTED;
  if (!prof->global_heads) return RK_ERR_NULL;
  if (prof->group_size != kGroup || prof->d_latent != kDLatent || prof->d_rope != kDRope || prof->d_v != kDV)
    return RK_ERR_UNSUPPORTED;
  if (prof->n_groups <= 0 || prof->n_heads != prof->n_groups * prof->group_size) return RK_ERR_PROFILE;
  if (prof->o_rank <= 0 || prof->o_rank % 128 != 0 || prof->d_model <= 0 || prof->d_model % 128 != 0)
    return RK_ERR_UNSUPPORTED;
  if (!(prof->sm_scale > 0.f) || !(prof->rope_base > 1.f)) return RK_ERR_PROFILE;
  for (int g = 0; g < prof->n_groups; ++g) {
    const int h = prof->global_heads[g];
    if (h < 0 || h >= prof->n_heads || h / prof->group_size != g) return RK_ERR_PROFILE;
  }
  rk_ctx* ctx = new (std::nothrow) rk_ctx();
  if (!ctx) return RK_ERR_CUDA;
  ctx->prof = *prof;
  ctx->global_heads.assign(prof->global_heads, prof->global_heads + prof->n_groups);
  ctx->prof.global_heads = ctx->global_heads.data();
  ctx->value_phase = (flags & RK_VALUE_PHASE) != 0;
  ctx->ow = ctx->value_phase ? kDQK : kDLatent;
  for (int j = 0; j < 32; ++j)
    ctx->rope_turns[j] = std::pow((double)prof->rope_base, -2.0 * j / (double)kDRope) / 6.283185307179586476925286766559;
  for (int h = 0; h < prof->n_heads; ++h)
    if (ctx->global_heads[h / kGroup] != h) ctx->local_heads.push_back(h);

  cudaError_t e = cudaGetDevice(&ctx->device);
  cudaDeviceProp dp;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&dp, ctx->device);
  if (e != cudaSuccess) {
    cudaGetLastError();
    delete ctx;
    return RK_ERR_CUDA;
  }
  if (dp.major != 10) {  // tcgen05 / TMEM path only; there is no fallback
    delete ctx;
    return RK_ERR_UNSUPPORTED;
  }
  ctx->sm_count = dp.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    delete ctx;
    return RK_ERR_CUDA;
  }
  ctx->encode = reinterpret_cast<PFN_encodeTiled>(fn);
  e = attention_setup();
  if (e == cudaSuccess) e = gemm_setup();
  if (e == cudaSuccess) e = stream_setup();
  if (e == cudaSuccess) e = proj_fused_setup();
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->d_status), sizeof(DeviceStatus));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(DeviceStatus));
  if (e != cudaSuccess) {
    cudaGetLastError();
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    return RK_ERR_CUDA;
  }
  ctx->n_pairs = attention_max_pairs(ctx->sm_count);
  {  // bind the built-in projection scratch of rk_group_sliced_proj_static on this device now
    void* scratch = nullptr;
    e = static_scratch_address(ctx->device, &scratch);
    if (e != cudaSuccess) {
      cudaGetLastError();
      rk_destroy(ctx);
      return RK_ERR_CUDA;
    }
  }
  e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_out_stream, cudaStreamNonBlocking);
  for (int i = 0; i < 10 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->sev[i], cudaEventDisableTiming);
  for (int i = 0; i < 8 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ctx->ev[i], cudaEventDisableTiming);
  if (e != cudaSuccess) {
    cudaGetLastError();
    rk_destroy(ctx);
    return RK_ERR_CUDA;
  }

  // GEMM batch tables (depend only on the head partition)
  const int G = prof->n_groups, L = (int)ctx->local_heads.size(), ro = prof->o_rank;
  const int32_t kNoSkip = 1 << 30;
  std::vector<GemmBatch> b;
  ctx->off_uv_g = (int)b.size();
  for (int g = 0; g < G; ++g) b.push_back(GemmBatch{g * ctx->ow, ctx->global_heads[g] * kDV, 0, kNoSkip, g * kDV, {0, 0, 0}});
  ctx->off_uv_l = (int)b.size();
  for (int l = 0; l < L; ++l) b.push_back(GemmBatch{l * ctx->ow, ctx->local_heads[l] * kDV, 0, kNoSkip, l * kDV, {0, 0, 0}});
  ctx->off_wa_g = (int)b.size();
  for (int g = 0; g < G; ++g) {
    const int j = ctx->global_heads[g] % kGroup;
    b.push_back(GemmBatch{g * kDV, g * ro, j * kDV, kNoSkip, g * ro, {0, 0, 0}});
  }
  ctx->off_wa_l = (int)b.size();
  for (int g = 0; g < G; ++g) {
    const int j = ctx->global_heads[g] % kGroup;
    b.push_back(GemmBatch{g * (kGroup - 1) * kDV, g * ro, 0, j * kDV, g * ro, {0, 0, 0}});
  }
  ctx->off_wb = (int)b.size();
  b.push_back(GemmBatch{0, 0, 0, kNoSkip, 0, {0, 0, 0}});
  e = upload(&ctx->d_batches, b);
  if (e != cudaSuccess) {
    cudaGetLastError();
    cudaFree(ctx->d_status);
    if (ctx->d_batches) cudaFree(ctx->d_batches);
    delete ctx;
    return RK_ERR_CUDA;
  }
  *out = ctx;
  return RK_OK;
}

rk_status rk_destroy(rk_ctx* ctx) {
  if (!ctx) return RK_ERR_NULL;
  for (int i = 0; i < 8; ++i)
    if (ctx->ev[i]) cudaEventDestroy(ctx->ev[i]);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  for (int i = 0; i < 10; ++i)
    if (ctx->sev[i]) cudaEventDestroy(ctx->sev[i]);
  if (ctx->copy_out_stream) cudaStreamDestroy(ctx->copy_out_stream);
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_batches);
  delete ctx;
  return RK_OK;
}

rk_status rk_set_wait_limit_ms(rk_ctx* ctx, int32_t ms) {
  if (!ctx) return RK_ERR_NULL;
  if (ms <= 0) return fail(ctx, RK_ERR_PROFILE, "wait limit must be positive");
  ctx->wait_ns = (unsigned long long)ms * 1000ull * 1000ull;
  return RK_OK;
}

rk_status rk_check_selftest(rk_ctx* ctx, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  cudaError_t e = launch_check_selftest(ctx->d_status, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorNotSupported) {
    cudaGetLastError();
    return fail(ctx, RK_ERR_UNSUPPORTED, "this library was built without the device index checks (-DRK_CHECK)");
  }
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "self-test launch");
}

rk_status rk_test_starve_loads(rk_ctx* ctx, int32_t on) {
  if (!ctx) return RK_ERR_NULL;
  ctx->starve_loads = on != 0;
  return RK_OK;
}

rk_status rk_poll_status(rk_ctx* ctx, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
  DeviceStatus h;
  e = cudaMemcpy(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "status readback");
  if (h.code != 0) {
    cudaMemset(ctx->d_status, 0, sizeof(DeviceStatus));
    if (h.code == RK_ERR_ROWS)  // only the bounds-checked build reports this
      return fail(ctx, RK_ERR_ROWS, "device index check failed: table %d, block %d, value %d", h.where, h.block, h.aux);
    return fail(ctx, RK_ERR_TIMEOUT, "device wait expired: tag %d, block %d, aux %d", h.where, h.block, h.aux);
  }
  return RK_OK;
}

// ------------------------------------------------------------------------------------------
// Pure host check of a layout and a protected-row list (no device needed).  msg may be NULL.
rk_status rk_check_request(const rk_layout* lay, const int32_t* prot_rows, int64_t n_prot, char* msg,
                           size_t msg_len) {
  auto bad = [&](rk_status s, const char* fmt, long long a, long long b) {
    if (msg && msg_len) snprintf(msg, msg_len, fmt, a, b);
    return s;
  };
  if (!lay || !lay->seg_off || !lay->seg_delta || !lay->seg_has_artifact || (n_prot > 0 && !prot_rows))
    return bad(RK_ERR_NULL, "null argument", 0, 0);
  const int S = lay->n_segs;
  if (S <= 0) return bad(RK_ERR_LAYOUT, "n_segs must be positive", 0, 0);
  if (lay->seg_off[0] != 0) return bad(RK_ERR_LAYOUT, "seg_off[0] must be 0", 0, 0);
  for (int i = 0; i < S; ++i) {
    if (lay->seg_off[i + 1] <= lay->seg_off[i])
      return bad(RK_ERR_LAYOUT, "segment %lld is empty or seg_off is not increasing", i, 0);
    if (lay->seg_delta[i] < 0) return bad(RK_ERR_LAYOUT, "segment %lld has a negative request offset", i, 0);
    if (lay->seg_delta[i] + (lay->seg_off[i + 1] - lay->seg_off[i]) >= (int64_t)1 << 30)
      return bad(RK_ERR_LAYOUT, "segment %lld reaches request position 2^30 or beyond", i, 0);
  }
  const int64_t T = lay->seg_off[S];
  if (T >= ((int64_t)1 << 30)) return bad(RK_ERR_LAYOUT, "too many rows", 0, 0);
  {  // request-position intervals must not overlap
    std::vector<std::pair<int64_t, int64_t>> iv;
    for (int i = 0; i < S; ++i)
      iv.push_back({lay->seg_delta[i], lay->seg_delta[i] + lay->seg_off[i + 1] - lay->seg_off[i]});
    std::sort(iv.begin(), iv.end());
    for (int i = 1; i < S; ++i)
      if (iv[i].first < iv[i - 1].second)
        return bad(RK_ERR_LAYOUT, "request-position intervals overlap at position %lld", iv[i].first, 0);
  }
  if (n_prot < 0 || n_prot > T) return bad(RK_ERR_ROWS, "n_prot out of range", 0, 0);
  std::vector<uint8_t> is_prot((size_t)T, 0);
  for (int64_t a = 0; a < n_prot; ++a) {
    const int64_t r = prot_rows[a];
    if (r < 0 || r >= T) return bad(RK_ERR_ROWS, "protected row %lld out of range", r, 0);
    if (a > 0 && prot_rows[a] <= prot_rows[a - 1])
      return bad(RK_ERR_ROWS, "protected rows must be strictly ascending (entry %lld)", a, 0);
    is_prot[(size_t)r] = 1;
  }
  for (int i = 0; i < S; ++i)
    if (!lay->seg_has_artifact[i])
      for (int64_t r = lay->seg_off[i]; r < lay->seg_off[i + 1]; ++r)
        if (!is_prot[(size_t)r])
          return bad(RK_ERR_ROWS, "row %lld of segment %lld has no artifact and is not protected", r, i);
  return RK_OK;
}

rk_status rk_request_create(rk_ctx* ctx, const rk_layout* lay, const int32_t* prot_rows, int64_t n_prot,
                            rk_request** out) {
  if (!ctx) return RK_ERR_NULL;
  if (!out) return fail(ctx, RK_ERR_NULL, "null argument");
  *out = nullptr;
  {
    char msg[256] = {0};
    rk_status s = rk_check_request(lay, prot_rows, n_prot, msg, sizeof(msg));
    if (s != RK_OK) return fail(ctx, s, "%s", msg);
  }
  const int S = lay->n_segs;
  const int64_t T = lay->seg_off[S];
  std::vector<int32_t> inv((size_t)T, -1);
  for (int64_t a = 0; a < n_prot; ++a) inv[(size_t)prot_rows[a]] = (int32_t)a;
  int64_t n_off_rows = 0;
  for (int i = 0; i < S; ++i)
    if (lay->seg_has_artifact[i]) n_off_rows = lay->seg_off[i + 1];

  rk_request* rq = new (std::nothrow) rk_request();
  if (!rq) return fail(ctx, RK_ERR_CUDA, "out of host memory");
  rq->ctx = ctx;
  rq->T = T;
  rq->A = n_prot;
  rq->S = S;
  rq->n_off_rows = n_off_rows;

  std::vector<int32_t> seg_off32((size_t)S + 1), seg_delta32((size_t)S), seg_n((size_t)S), row_pos((size_t)T);
  for (int i = 0; i <= S; ++i) seg_off32[(size_t)i] = (int32_t)lay->seg_off[i];
  for (int i = 0; i < S; ++i) {
    seg_delta32[(size_t)i] = (int32_t)lay->seg_delta[i];
    seg_n[(size_t)i] = seg_off32[(size_t)i + 1] - seg_off32[(size_t)i];
    for (int64_t r = lay->seg_off[i]; r < lay->seg_off[i + 1]; ++r)
      row_pos[(size_t)r] = (int32_t)(lay->seg_delta[i] + (r - lay->seg_off[i]));
  }
  // relocation tables: angle delta_i * theta_j evaluated in double, theta_j = base^(-2j/d_rope)
  std::vector<float2> cs((size_t)S * 32);
  for (int i = 0; i < S; ++i)
    for (int j = 0; j < 32; ++j) {
      const double theta = std::pow((double)ctx->prof.rope_base, -2.0 * j / (double)kDRope);
      const double ang = (double)lay->seg_delta[i] * theta;
      cs[(size_t)i * 32 + j] = make_float2((float)std::cos(ang), (float)std::sin(ang));
    }
  // visible-pair counts (for flop accounting): a row of segment i at canonical index c sees every key
  // of the segments placed before it in the request (intervals do not overlap) plus c + 1 of its own
  std::vector<int64_t> keys_before((size_t)S, 0);
  {
    std::vector<int> order((size_t)S);
    for (int i = 0; i < S; ++i) order[(size_t)i] = i;
    std::sort(order.begin(), order.end(), [&](int a, int b) { return seg_delta32[(size_t)a] < seg_delta32[(size_t)b]; });
    int64_t run = 0;
    for (int k = 0; k < S; ++k) {
      keys_before[(size_t)order[(size_t)k]] = run;
      run += seg_n[(size_t)order[(size_t)k]];
    }
  }
  for (int i = 0; i < S; ++i) {
    const int64_t n = seg_n[(size_t)i];
    rq->pairs_global += n * keys_before[(size_t)i] + n * (n + 1) / 2;
  }
  std::vector<int32_t> prot((size_t)n_prot), prot_pos((size_t)n_prot);
  {
    int seg = 0;
    for (int64_t a = 0; a < n_prot; ++a) {
      const int64_t r = prot_rows[a];
      while (r >= lay->seg_off[seg + 1]) ++seg;  // the list is ascending
      prot[(size_t)a] = (int32_t)r;
      prot_pos[(size_t)a] = row_pos[(size_t)r];
      rq->pairs_local += keys_before[(size_t)seg] + (r - lay->seg_off[seg]) + 1;
    }
  }
  std::vector<AttnWorkItem> work_g, work_l;
  build_work(row_pos, ctx->prof.n_groups, seg_n, seg_delta32, ctx->n_pairs, &work_g);
  build_work(prot_pos, (int)ctx->local_heads.size(), seg_n, seg_delta32, ctx->n_pairs, &work_l);
  rq->n_tiles_g = (int32_t)work_g.size();
  rq->n_tiles_l = (int32_t)work_l.size();
  std::vector<AttnWorkItem> work_part[2];
  {  // two row ranges for rk_layer_host: the boundary must fall on a row-tile boundary of the Global pass
    const int G = ctx->prof.n_groups;
    int gcd = G, b = kAttnRowsPerPair;
    while (b) { const int r = gcd % b; gcd = b; b = r; }
    const int64_t unit = kAttnRowsPerPair / gcd;  // tokens per smallest whole number of tiles
    const int64_t split = (T * 7 / 8) / unit * unit;
    if (T >= 512 && split > 0 && split < T) {
      rq->split_tok = split;
      const int64_t tile_split = split * G / kAttnRowsPerPair;
      build_work(row_pos, G, seg_n, seg_delta32, ctx->n_pairs, &work_part[0], 0, tile_split);
      build_work(row_pos, G, seg_n, seg_delta32, ctx->n_pairs, &work_part[1], tile_split, -1);
      rq->n_tiles_g_part[0] = (int32_t)work_part[0].size();
      rq->n_tiles_g_part[1] = (int32_t)work_part[1].size();
    }
  }
  std::vector<AttnWorkItem> work_lpart[2];
  {
    const int L = (int)ctx->local_heads.size();
    int gcd = L, b = kAttnRowsPerPair;
    while (b) { const int r = gcd % b; gcd = b; b = r; }
    const int64_t unit = kAttnRowsPerPair / gcd;
    const int64_t split = (n_prot / 8) / unit * unit;
    if (n_prot >= 512 && split > 0 && split < n_prot) {
      rq->split_slot = split;
      const int64_t tile_split = split * L / kAttnRowsPerPair;
      build_work(prot_pos, L, seg_n, seg_delta32, ctx->n_pairs, &work_lpart[0], 0, tile_split);
      build_work(prot_pos, L, seg_n, seg_delta32, ctx->n_pairs, &work_lpart[1], tile_split, -1);
      rq->n_tiles_l_part[0] = (int32_t)work_lpart[0].size();
      rq->n_tiles_l_part[1] = (int32_t)work_lpart[1].size();
    }
  }

  cudaError_t e = upload(&rq->d_row_pos, row_pos);
  if (e == cudaSuccess) e = upload(&rq->d_prot_rows, prot);
  if (e == cudaSuccess) e = upload(&rq->d_inv_map, inv);
  if (e == cudaSuccess) e = upload(&rq->d_seg_off, seg_off32);
  if (e == cudaSuccess) e = upload(&rq->d_seg_delta, seg_delta32);
  if (e == cudaSuccess) e = upload(&rq->d_seg_cs, cs);
  if (e == cudaSuccess) e = upload(&rq->d_work_g, work_g);
  if (e == cudaSuccess) e = upload(&rq->d_work_l, work_l);
  if (e == cudaSuccess && rq->split_tok > 0) e = upload(&rq->d_work_g_part[0], work_part[0]);
  if (e == cudaSuccess && rq->split_tok > 0) e = upload(&rq->d_work_g_part[1], work_part[1]);
  if (e == cudaSuccess && rq->split_slot > 0) e = upload(&rq->d_work_l_part[0], work_lpart[0]);
  if (e == cudaSuccess && rq->split_slot > 0) e = upload(&rq->d_work_l_part[1], work_lpart[1]);
  if (e != cudaSuccess) {
    rk_request_destroy(rq);
    return cuda_fail(ctx, e, "request table upload");
  }
  *out = rq;
  return RK_OK;
}

rk_status rk_request_destroy(rk_request* rq) {
  if (!rq) return RK_ERR_NULL;
  cudaFree(rq->d_row_pos);
  cudaFree(rq->d_prot_rows);
  cudaFree(rq->d_inv_map);
  cudaFree(rq->d_seg_off);
  cudaFree(rq->d_seg_delta);
  cudaFree(rq->d_seg_cs);
  cudaFree(rq->d_work_g);
  cudaFree(rq->d_work_l);
  cudaFree(rq->d_work_g_part[0]);
  cudaFree(rq->d_work_g_part[1]);
  cudaFree(rq->d_work_l_part[0]);
  cudaFree(rq->d_work_l_part[1]);
  delete rq;
  return RK_OK;
}

rk_status rk_request_get_info(const rk_request* rq, rk_request_info* out) {
  if (!rq || !out) return RK_ERR_NULL;
  out->n_rows = rq->T;
  out->n_prot = rq->A;
  out->n_off_rows = rq->n_off_rows;
  out->pairs_global = rq->pairs_global;
  out->pairs_local = rq->pairs_local;
  out->n_tiles_global = rq->n_tiles_g;
  out->n_tiles_local = rq->n_tiles_l;
  return RK_OK;
}

static size_t proj_ws_bytes(const rk_request* rq) {
  const rk_ctx* c = rq->ctx;
  const size_t og = ((size_t)rq->T * c->prof.n_groups * kDV * 2 + 255) & ~(size_t)255;
  const size_t ol = ((size_t)rq->A * c->local_heads.size() * kDV * 2 + 255) & ~(size_t)255;
  return og + ol;
}

rk_status rk_workspace_bytes(const rk_request* rq, size_t* out) {
  if (!rq || !out) return RK_ERR_NULL;
  *out = proj_ws_bytes(rq);
  return RK_OK;
}

// ------------------------------------------------------------------------------------------
rk_status rk_relocate_q(rk_ctx* ctx, const rk_request* rq, const void* q_rope, int64_t n_rows, int32_t n_heads,
                        int64_t row_stride, int64_t head_stride, int32_t seg_begin, int32_t seg_end, void* out,
                        void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !q_rope || !out) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  if (n_rows < 0 || n_heads <= 0) return fail(ctx, RK_ERR_LAYOUT, "bad row/head count");
  if (seg_begin < 0 || seg_end > rq->S || seg_begin > seg_end) return fail(ctx, RK_ERR_LAYOUT, "segment range out of bounds");
  if (!aligned16(q_rope) || !aligned16(out) || row_stride % 8 != 0 || head_stride % 8 != 0)
    return fail(ctx, RK_ERR_ALIGN, "q_rope/out must be 16-byte aligned and strides multiples of 8 elements");
  if (head_stride < kDRope || row_stride < head_stride) return fail(ctx, RK_ERR_LAYOUT, "strides too small");
  cudaError_t e = launch_relocate(q_rope, n_rows, n_heads, row_stride, head_stride, rq->d_seg_cs, seg_begin, seg_end,
                                  out, ctx->sm_count, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "relocate launch");
}

static rk_status attn_pass(rk_ctx* ctx, const rk_request* rq, const void* kv, const void* q, int64_t n_tok, int hpt,
                           const int32_t* rowmap, const AttnWorkItem* work, int n_tiles, void* O, float* lse,
                           cudaStream_t stream, int isolated = 0, int64_t row_base = 0) {
  if (n_tiles == 0) return RK_OK;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  const int64_t n_flat = n_tok * hpt;
  if (n_flat >= ((int64_t)1 << 31) - 256)
    return fail(ctx, RK_ERR_LAYOUT, "rows x heads of one attention pass must stay below 2^31");
  rk_status s = make_tmap(ctx, &p.tm_q, q, (uint64_t)n_flat, kDQK, kDQK, 64, kAttnRowsPerCta);
  if (s != RK_OK) return s;
  s = make_tmap(ctx, &p.tm_kv, kv, (uint64_t)rq->T, kDQK, kDQK, 64, 128);
  if (s != RK_OK) return s;
  p.row_pos = rq->d_row_pos;
  p.rowmap = rowmap;
  p.seg_off = rq->d_seg_off;
  p.seg_delta = rq->d_seg_delta;
  p.seg_cs = rq->d_seg_cs;
  p.work = work;
  p.O = O;
  p.lse = lse;
  p.status = ctx->d_status;
  p.wait_ns = ctx->wait_ns;
  p.n_segs = rq->S;
  p.n_tiles = n_tiles;
  p.n_flat = (int32_t)n_flat;
  p.hpt = hpt;
  const int n_pairs = std::min(ctx->n_pairs, n_tiles);
  p.n_pairs = n_pairs;
  p.scale_log2 = ctx->prof.sm_scale * 1.44269504088896340736f;
  p.isolated = isolated;
  p.row_base = (int32_t)row_base;
  p.n_rows_total = (int32_t)rq->T;
  memcpy(p.rope_turns, ctx->rope_turns, sizeof(p.rope_turns));
  cudaError_t e = launch_attention(p, n_pairs, ctx->value_phase, ctx->starve_loads, stream);
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "attention launch");
}

rk_status rk_mla_online_attn(rk_ctx* ctx, const rk_request* rq, const void* kv, const void* q_g, const void* q_l,
                             void* O_g, float* lse_g, void* O_l, float* lse_l, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !kv) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  const bool do_g = q_g || O_g || lse_g, do_l = q_l || O_l || lse_l;
  if (do_g && !(q_g && O_g && lse_g)) return fail(ctx, RK_ERR_NULL, "Global pass needs q_g, O_g and lse_g");
  if (do_l && !(q_l && O_l && lse_l)) return fail(ctx, RK_ERR_NULL, "Local pass needs q_l, O_l and lse_l");
  if (!aligned16(kv) || !aligned16(q_g) || !aligned16(q_l) || !aligned16(O_g) || !aligned16(O_l))
    return fail(ctx, RK_ERR_ALIGN, "tensor base pointers must be 16-byte aligned");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  rk_status s = RK_OK;
  if (do_g)
    s = attn_pass(ctx, rq, kv, q_g, rq->T, ctx->prof.n_groups, nullptr, rq->d_work_g, rq->n_tiles_g, O_g, lse_g, st);
  if (s == RK_OK && do_l && rq->A > 0)
    s = attn_pass(ctx, rq, kv, q_l, rq->A, (int)ctx->local_heads.size(), rq->d_prot_rows, rq->d_work_l, rq->n_tiles_l,
                  O_l, lse_l, st);
  return s;
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
static rk_status run_gemm(rk_ctx* ctx, const void* A, int64_t a_rows, int64_t a_cols, const void* B, int64_t b_rows,
                          int64_t b_cols, void* C, int64_t ldc, int M, int N, int K, int batch_off, int n_batches,
                          cudaStream_t st);

rk_status rk_mla_off_workspace_bytes(const rk_request* rq, int64_t n_rows, size_t* out) {
  if (!rq || !out) return RK_ERR_NULL;
  if (n_rows < 0) return RK_ERR_LAYOUT;
  const size_t L = rq->ctx->local_heads.size();
  *out = align256((size_t)n_rows * L * rq->ctx->ow * 2) + align256((size_t)n_rows * L * 4) +
         align256((size_t)n_rows * L * kDV * 2);
  return RK_OK;
}

rk_status rk_mla_off_build(rk_ctx* ctx, const rk_request* rq, const void* kv, int64_t row_begin, int64_t row_end,
                           const void* q_l_rows, const void* W_uv, const void* W_a, void* z_off_rows, void* workspace,
                           size_t workspace_bytes, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !kv || !q_l_rows || !W_uv || !W_a || !z_off_rows || !workspace) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  if (row_begin < 0 || row_end > rq->T || row_begin > row_end) return fail(ctx, RK_ERR_LAYOUT, "row range out of bounds");
  if (!aligned16(kv) || !aligned16(q_l_rows) || !aligned16(W_uv) || !aligned16(W_a) || !aligned16(z_off_rows) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return fail(ctx, RK_ERR_ALIGN, "tensors must be 16-byte aligned and the workspace 256-byte aligned");
  const int64_t n = row_end - row_begin;
  size_t need = 0;
  rk_mla_off_workspace_bytes(rq, n, &need);
  if (workspace_bytes < need) return fail(ctx, RK_ERR_WORKSPACE, "workspace too small: need %zu bytes", need);
  if (n == 0) return RK_OK;
  const int G = ctx->prof.n_groups, H = ctx->prof.n_heads, L = H - G, ro = ctx->prof.o_rank;
  if (n * L >= ((int64_t)1 << 31)) return fail(ctx, RK_ERR_LAYOUT, "row range too long for one call: split it");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  void* O = ws;
  float* lse = reinterpret_cast<float*>(ws + align256((size_t)n * L * ctx->ow * 2));
  void* o = reinterpret_cast<uint8_t*>(lse) + align256((size_t)n * L * 4);
  const int n_tiles = (int)((n * L + kAttnRowsPerPair - 1) / kAttnRowsPerPair);
  // documents alone: a row sees only its own segment, causally, with the query relocated into
  // the segment's position-zero frame; tiles in natural order (no host-built list)
  rk_status s = attn_pass(ctx, rq, kv, q_l_rows, n, L, nullptr, nullptr, n_tiles, O, lse, st, 1, row_begin);
  if (s != RK_OK) return s;
  s = run_gemm(ctx, O, n, (int64_t)L * ctx->ow, W_uv, (int64_t)H * kDV, ctx->ow, o, (int64_t)L * kDV, (int)n, kDV,
               ctx->ow, ctx->off_uv_l, L, st);
  if (s != RK_OK) return s;
  return run_gemm(ctx, o, n, (int64_t)L * kDV, W_a, (int64_t)G * ro, kGroup * kDV, z_off_rows, (int64_t)G * ro, (int)n, ro,
                  (kGroup - 1) * kDV, ctx->off_wa_l, G, st);
}

rk_status rk_segmented_merge(rk_ctx* ctx, int32_t n_parts, int64_t n_rows, int32_t n_heads, const void* O_part,
                             int32_t part_dtype, const float* lse_part, void* O, float* lse, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!O_part || !lse_part || !O || !lse) return fail(ctx, RK_ERR_NULL, "null argument");
  if (n_parts <= 0 || n_parts > kMergeMaxParts || n_rows < 0 || n_heads <= 0) return fail(ctx, RK_ERR_LAYOUT, "bad part/row/head count");
  if (part_dtype != 0 && part_dtype != 1) return fail(ctx, RK_ERR_UNSUPPORTED, "part_dtype must be 0 (bf16) or 1 (fp32)");
  if (!aligned16(O_part) || !aligned16(O)) return fail(ctx, RK_ERR_ALIGN, "O_part/O must be 16-byte aligned");
  cudaError_t e = launch_merge(n_parts, n_rows * n_heads, O_part, part_dtype, lse_part, O, lse, ctx->sm_count,
                               reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "merge launch");
}

rk_status rk_segmented_merge_phase(rk_ctx* ctx, const rk_request* rq, int32_t seg_begin, int32_t n_parts, int64_t n_rows,
                                   int32_t n_heads, const void* O_part, int32_t part_dtype, const float* lse_part,
                                   const int32_t* row_pos, void* O, float* lse, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !O_part || !lse_part || !O || !lse) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  if (n_parts <= 0 || n_parts > kMergeMaxParts || n_rows < 0 || n_heads <= 0) return fail(ctx, RK_ERR_LAYOUT, "bad part/row/head count");
  if (seg_begin < 0 || seg_begin + n_parts > rq->S) return fail(ctx, RK_ERR_LAYOUT, "segment range out of bounds");
  if (part_dtype != 0 && part_dtype != 1) return fail(ctx, RK_ERR_UNSUPPORTED, "part_dtype must be 0 (bf16) or 1 (fp32)");
  if (!aligned16(O_part) || !aligned16(O)) return fail(ctx, RK_ERR_ALIGN, "O_part/O must be 16-byte aligned");
  cudaError_t e = launch_merge_phase(n_parts, n_rows, n_heads, O_part, part_dtype, lse_part, rq->d_seg_cs + (size_t)seg_begin * 32,
                                     row_pos, ctx->rope_turns, O, lse, ctx->sm_count, reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "merge launch");
}

static rk_status run_gemm(rk_ctx* ctx, const void* A, int64_t a_rows, int64_t a_cols, const void* B, int64_t b_rows,
                          int64_t b_cols, void* C, int64_t ldc, int M, int N, int K, int batch_off, int n_batches,
                          cudaStream_t st) {
  if (M == 0) return RK_OK;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  const int bn = (N % 256 == 0) ? 256 : 128;
  rk_status s = make_tmap(ctx, &p.tm_a, A, (uint64_t)a_rows, (uint64_t)a_cols, (uint64_t)a_cols, 64, 128);
  if (s != RK_OK) return s;
  s = make_tmap(ctx, &p.tm_b, B, (uint64_t)b_rows, (uint64_t)b_cols, (uint64_t)b_cols, 64,
                gemm_uses_pairs(M, N, n_batches) ? 128u : (uint32_t)bn);
  if (s != RK_OK) return s;
  s = make_tmap(ctx, &p.tm_c, C, (uint64_t)M, (uint64_t)ldc, (uint64_t)ldc, 64, 128);
  if (s != RK_OK) return s;
  p.C = C;
  p.batches = ctx->d_batches + batch_off;
  p.status = ctx->d_status;
  p.wait_ns = ctx->wait_ns;
  p.ldc = ldc;
  p.M = M;
  p.N = N;
  p.K = K;
  p.n_batches = n_batches;
  cudaError_t e = launch_gemm(p, bn, ctx->sm_count, st);
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "gemm launch");
}

// Global half of the sliced first projection for `n` rows: one fused kernel when the group rank is a multiple of
// 256 (o = W_uv O stays on chip), else the two batched GEMMs with o in the workspace.
static rk_status proj_global(rk_ctx* ctx, const void* O_g, int64_t n, const void* W_uv, const void* W_a, void* o_g,
                             void* z_on_g, cudaStream_t st) {
  const int G = ctx->prof.n_groups, H = ctx->prof.n_heads, ro = ctx->prof.o_rank;
  if (n == 0) return RK_OK;
  if (ro % 256 == 0) {
    FusedProjParams p;
    memset(&p, 0, sizeof(p));
    rk_status s = make_tmap(ctx, &p.tm_a, O_g, (uint64_t)n, (uint64_t)G * ctx->ow, (uint64_t)G * ctx->ow, 64, 128);
    if (s == RK_OK) s = make_tmap(ctx, &p.tm_b1, W_uv, (uint64_t)H * kDV, (uint64_t)ctx->ow, (uint64_t)ctx->ow, 64, 128);
    if (s == RK_OK) s = make_tmap(ctx, &p.tm_b2, W_a, (uint64_t)G * ro, (uint64_t)kGroup * kDV, (uint64_t)kGroup * kDV, 64, 128);
    if (s == RK_OK) s = make_tmap(ctx, &p.tm_c, z_on_g, (uint64_t)n, (uint64_t)G * ro, (uint64_t)G * ro, 64, 128);
    if (s != RK_OK) return s;
    p.batches_uv = ctx->d_batches + ctx->off_uv_g;
    p.batches_wa = ctx->d_batches + ctx->off_wa_g;
    p.status = ctx->d_status;
    p.wait_ns = ctx->wait_ns;
    p.M = (int32_t)n;
    p.n_groups = G;
    p.K1 = ctx->ow;
    p.o_rank = ro;
    cudaError_t e = launch_proj_fused(p, ctx->sm_count, st);
    return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "fused projection launch");
  }
  rk_status s = run_gemm(ctx, O_g, n, (int64_t)G * ctx->ow, W_uv, (int64_t)H * kDV, ctx->ow, o_g, (int64_t)G * kDV, (int)n, kDV,
                         ctx->ow, ctx->off_uv_g, G, st);
  if (s == RK_OK)
    s = run_gemm(ctx, o_g, n, (int64_t)G * kDV, W_a, (int64_t)G * ro, kGroup * kDV, z_on_g, (int64_t)G * ro, (int)n, ro, kDV,
                 ctx->off_wa_g, G, st);
  return s;
}

rk_status rk_group_sliced_proj(rk_ctx* ctx, const rk_request* rq, const void* O_g, const void* O_l, const void* W_uv,
                               const void* W_a, void* z_on_g, void* z_on_l, void* workspace, size_t workspace_bytes,
                               void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !W_uv || !W_a || !workspace) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  const bool do_g = O_g || z_on_g, do_l = O_l || z_on_l;
  if (do_g && !(O_g && z_on_g)) return fail(ctx, RK_ERR_NULL, "Global half needs O_g and z_on_g");
  if (do_l && !(O_l && z_on_l)) return fail(ctx, RK_ERR_NULL, "Local half needs O_l and z_on_l");
  if (!aligned16(O_g) || !aligned16(O_l) || !aligned16(W_uv) || !aligned16(W_a) || !aligned16(z_on_g) ||
      !aligned16(z_on_l) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return fail(ctx, RK_ERR_ALIGN, "tensors must be 16-byte aligned and the workspace 256-byte aligned");
  if (workspace_bytes < proj_ws_bytes(rq)) return fail(ctx, RK_ERR_WORKSPACE, "workspace too small: need %zu bytes", proj_ws_bytes(rq));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int G = ctx->prof.n_groups, H = ctx->prof.n_heads, L = H - G, ro = ctx->prof.o_rank;
  const int64_t T = rq->T, A = rq->A;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  void* o_g = ws;
  void* o_l = ws + (((size_t)T * G * kDV * 2 + 255) & ~(size_t)255);
  rk_status s = RK_OK;
  if (do_g) s = proj_global(ctx, O_g, T, W_uv, W_a, o_g, z_on_g, st);
  if (s == RK_OK && do_l && A > 0) {
    s = run_gemm(ctx, O_l, A, (int64_t)L * ctx->ow, W_uv, (int64_t)H * kDV, ctx->ow, o_l, (int64_t)L * kDV, (int)A, kDV,
                 ctx->ow, ctx->off_uv_l, L, st);
    if (s == RK_OK)
      s = run_gemm(ctx, o_l, A, (int64_t)L * kDV, W_a, (int64_t)G * ro, kGroup * kDV, z_on_l, (int64_t)G * ro, (int)A, ro,
                   (kGroup - 1) * kDV, ctx->off_wa_l, G, st);
  }
  return s;
}

rk_status rk_combine_offline(rk_ctx* ctx, const rk_request* rq, const void* z_on_g, const void* z_on_l,
                             const void* z_off, const void* W_b, void* z, void* y, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !z_on_g || !z) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  if (rq->A > 0 && !z_on_l) return fail(ctx, RK_ERR_NULL, "z_on_l is required when rows are protected");
  if (rq->A < rq->T && !z_off) return fail(ctx, RK_ERR_NULL, "z_off is required when some rows are not protected");
  if (W_b && !y) return fail(ctx, RK_ERR_NULL, "y is required when W_b is given");
  if (!aligned16(z_on_g) || !aligned16(z_on_l) || !aligned16(z_off) || !aligned16(W_b) || !aligned16(z) || !aligned16(y))
    return fail(ctx, RK_ERR_ALIGN, "tensor base pointers must be 16-byte aligned");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int64_t width = (int64_t)ctx->prof.n_groups * ctx->prof.o_rank;
  cudaError_t e = launch_combine(z_on_g, z_on_l, z_off, rq->d_inv_map, rq->T, width, z, rq->A, ctx->d_status, ctx->sm_count, st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "combine launch");
  if (!W_b) return RK_OK;
  return run_gemm(ctx, z, rq->T, width, W_b, ctx->prof.d_model, width, y, ctx->prof.d_model, (int)rq->T,
                  ctx->prof.d_model, (int)width, ctx->off_wb, 1, st);
}

// The compute part of one layer on `st`, shared by rk_layer_host and rk_layer_stack_host.  Inputs may still
// be on their way: ev_ql_rest (NULL = none) guards the protected-row queries beyond the request's first
// Local range, ev_qg the Global queries, ev_zoff the artifact.  With split_global the Global pass and
// everything after it run in the request's two row ranges; the y rows of each range are copied to the
// host on y_stream as soon as they are complete (chunk_ev: two events that order those copies).
static rk_status layer_compute(rk_ctx* ctx, const rk_request* rq, const rk_layer_buffers* dev, const void* W_uv,
                               const void* W_a, const void* W_b, cudaStream_t st, cudaEvent_t ev_ql_rest, cudaEvent_t ev_qg,
                               cudaEvent_t ev_zoff, bool split_global, void* y_host, cudaStream_t y_stream,
                               cudaEvent_t* chunk_ev) {
  const int G = ctx->prof.n_groups, H = ctx->prof.n_heads, L = H - G, ro = ctx->prof.o_rank;
  const int64_t T = rq->T, dm = ctx->prof.d_model;
  const size_t width = (size_t)G * ro;
  const bool has_l = rq->A > 0;
  if (!aligned16(dev->kv) || !aligned16(dev->q_g) || !aligned16(dev->O_g) || !aligned16(dev->z_on_g) || !aligned16(dev->z) ||
      !aligned16(dev->y) || (reinterpret_cast<uintptr_t>(dev->workspace) & 255u))
    return fail(ctx, RK_ERR_ALIGN, "device buffers must be 16-byte aligned and the workspace 256-byte aligned");
  if (dev->workspace_bytes < proj_ws_bytes(rq)) return fail(ctx, RK_ERR_WORKSPACE, "workspace too small: need %zu bytes", proj_ws_bytes(rq));
  cudaError_t e = cudaSuccess;
  rk_status s = RK_OK;
  if (has_l) {  // Local pass and the Local half of the first projection: need kv, q_l only
    if (!aligned16(dev->q_l) || !aligned16(dev->O_l)) return fail(ctx, RK_ERR_ALIGN, "device buffers must be 16-byte aligned");
    if (ev_ql_rest != nullptr && rq->split_slot > 0) {
      s = attn_pass(ctx, rq, dev->kv, dev->q_l, rq->A, L, rq->d_prot_rows, rq->d_work_l_part[0], rq->n_tiles_l_part[0],
                    dev->O_l, dev->lse_l, st);
      e = cudaStreamWaitEvent(st, ev_ql_rest, 0);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "stream wait");
      if (s == RK_OK)
        s = attn_pass(ctx, rq, dev->kv, dev->q_l, rq->A, L, rq->d_prot_rows, rq->d_work_l_part[1], rq->n_tiles_l_part[1],
                      dev->O_l, dev->lse_l, st);
    } else {
      s = attn_pass(ctx, rq, dev->kv, dev->q_l, rq->A, L, rq->d_prot_rows, rq->d_work_l, rq->n_tiles_l, dev->O_l,
                    dev->lse_l, st);
    }
    if (s == RK_OK)
      s = rk_group_sliced_proj(ctx, rq, nullptr, dev->O_l, W_uv, W_a, nullptr, dev->z_on_l, dev->workspace,
                               dev->workspace_bytes, st);
    if (s != RK_OK) return s;
  }
  e = cudaStreamWaitEvent(st, ev_qg, 0);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "stream wait");
  // Global pass, Global half of the first projection, restore-and-replace and W_b per row range; the y
  // rows of a range are copied out while the next range computes
  const int n_chunks = (split_global && rq->split_tok > 0) ? 2 : 1;
  const uint8_t* Og = reinterpret_cast<const uint8_t*>(dev->O_g);
  uint8_t* og = reinterpret_cast<uint8_t*>(dev->workspace);  // per-head W_uv output of the Global heads
  uint8_t* zg = reinterpret_cast<uint8_t*>(dev->z_on_g);
  const uint8_t* zo = reinterpret_cast<const uint8_t*>(dev->z_off);
  uint8_t* zz = reinterpret_cast<uint8_t*>(dev->z);
  uint8_t* yy = reinterpret_cast<uint8_t*>(dev->y);
  for (int c = 0; c < n_chunks; ++c) {
    const int64_t r0 = c == 0 ? 0 : rq->split_tok, r1 = (n_chunks == 2 && c == 0) ? rq->split_tok : T;
    const int64_t n = r1 - r0;
    s = attn_pass(ctx, rq, dev->kv, dev->q_g, T, G, nullptr, n_chunks == 2 ? rq->d_work_g_part[c] : rq->d_work_g,
                  n_chunks == 2 ? rq->n_tiles_g_part[c] : rq->n_tiles_g, dev->O_g, dev->lse_g, st);
    if (s == RK_OK)
      s = proj_global(ctx, Og + (size_t)r0 * G * ctx->ow * 2, n, W_uv, W_a, og + (size_t)r0 * G * kDV * 2,
                      zg + (size_t)r0 * width * 2, st);
    if (s != RK_OK) return s;
    if (c == 0) {  // the artifact has to be there from here on
      e = cudaStreamWaitEvent(st, ev_zoff, 0);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "stream wait");
    }
    e = launch_combine(zg + (size_t)r0 * width * 2, dev->z_on_l, zo ? zo + (size_t)r0 * width * 2 : nullptr, rq->d_inv_map + r0, n,
                       (int64_t)width, zz + (size_t)r0 * width * 2, rq->A, ctx->d_status, ctx->sm_count, st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "combine launch");
    s = run_gemm(ctx, zz + (size_t)r0 * width * 2, n, (int64_t)width, W_b, dm, (int64_t)width, yy + (size_t)r0 * dm * 2, dm, (int)n,
                 (int)dm, (int)width, ctx->off_wb, 1, st);
    if (s != RK_OK) return s;
    e = cudaEventRecord(chunk_ev[c], st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(y_stream, chunk_ev[c], 0);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(reinterpret_cast<uint8_t*>(y_host) + (size_t)r0 * dm * 2, yy + (size_t)r0 * dm * 2, (size_t)n * dm * 2,
                          cudaMemcpyDeviceToHost, y_stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "device to host copy");
  }
  return RK_OK;
}

rk_status rk_layer_host(rk_ctx* ctx, const rk_request* rq, const void* kv_host, const void* q_g_host,
                        const void* q_l_host, const void* z_off_host, const void* W_uv, const void* W_a,
                        const void* W_b, const rk_layer_buffers* dev, void* y_host, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq || !kv_host || !q_g_host || !W_uv || !W_a || !W_b || !dev || !y_host) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  if (rq->A > 0 && !q_l_host) return fail(ctx, RK_ERR_NULL, "q_l_host is required");
  if (rq->A < rq->T && !z_off_host) return fail(ctx, RK_ERR_NULL, "z_off_host is required");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaStream_t cp = ctx->copy_stream;
  const int G = ctx->prof.n_groups, L = ctx->prof.n_heads - G;
  const int64_t T = rq->T;
  const size_t width = (size_t)G * ctx->prof.o_rank;
  const bool has_l = rq->A > 0;
  // The copy stream starts after everything already queued on `stream` (the staging buffers may
  // still be in use by an earlier call) and runs beside the kernels from then on: the Local pass
  // needs only kv and q_l, so q_g and the artifact travel while it computes; the rest of the layer
  // runs in two row ranges, and the y rows of the first go back while the second computes.
  // Ordering is by device events.
  // first on the wire: kv and the queries of the first Local range, alone, so that the Local pass can
  // start; the copy stream follows with the rest of q_l, then q_g, then the artifact
  const size_t ql_row = (size_t)L * kDQK * 2;
  const int64_t slot0 = (has_l && rq->split_slot > 0) ? rq->split_slot : rq->A;  // protected-row slots sent up front
  cudaError_t e = cudaMemcpyAsync(dev->kv, kv_host, (size_t)T * kDQK * 2, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && has_l) e = cudaMemcpyAsync(dev->q_l, q_l_host, (size_t)slot0 * ql_row, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev[0], st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(cp, ctx->ev[0], 0);
  if (e == cudaSuccess && slot0 < rq->A)
    e = cudaMemcpyAsync(reinterpret_cast<uint8_t*>(dev->q_l) + (size_t)slot0 * ql_row,
                        reinterpret_cast<const uint8_t*>(q_l_host) + (size_t)slot0 * ql_row, (size_t)(rq->A - slot0) * ql_row,
                        cudaMemcpyHostToDevice, cp);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev[6], cp);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dev->q_g, q_g_host, (size_t)T * G * kDQK * 2, cudaMemcpyHostToDevice, cp);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev[1], cp);
  if (e == cudaSuccess && rq->n_off_rows > 0 && z_off_host)
    e = cudaMemcpyAsync(dev->z_off, z_off_host, (size_t)rq->n_off_rows * width * 2, cudaMemcpyHostToDevice, cp);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->ev[2], cp);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "host to device copy");
  rk_status s = layer_compute(ctx, rq, dev, W_uv, W_a, W_b, st, slot0 < rq->A ? ctx->ev[6] : nullptr, ctx->ev[1], ctx->ev[2],
                              rq->split_tok > 0, y_host, cp, &ctx->ev[3]);
  if (s != RK_OK) return s;
  e = cudaEventRecord(ctx->ev[7], cp);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, ctx->ev[7], 0);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "device to host copy");
}

rk_status rk_layer_stack_host(rk_ctx* ctx, int32_t n_layers, const rk_layer_io* layers, const rk_layer_buffers* dev0,
                              const rk_layer_buffers* dev1, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!layers || !dev0 || !dev1) return fail(ctx, RK_ERR_NULL, "null argument");
  if (n_layers <= 0) return fail(ctx, RK_ERR_LAYOUT, "n_layers must be positive");
  for (int l = 0; l < n_layers; ++l) {
    const rk_layer_io& io = layers[l];
    if (!io.req || !io.kv_host || !io.q_g_host || !io.W_uv || !io.W_a || !io.W_b || !io.y_host)
      return fail(ctx, RK_ERR_NULL, "layer %d: null argument", l);
    if (io.req->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "layer %d: request belongs to another context", l);
    if (io.req->A > 0 && !io.q_l_host) return fail(ctx, RK_ERR_NULL, "layer %d: q_l_host is required", l);
    if (io.req->A < io.req->T && !io.z_off_host) return fail(ctx, RK_ERR_NULL, "layer %d: z_off_host is required", l);
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  cudaStream_t cin = ctx->copy_stream, cout = ctx->copy_out_stream;
  cudaEvent_t* kv_ql_in = ctx->sev;          // [2] kv and q_l of buffer set b are on the device
  cudaEvent_t* qg_in = ctx->sev + 2;         // [2] ... q_g
  cudaEvent_t* zoff_in = ctx->sev + 4;       // [2] ... the artifact
  cudaEvent_t* compute_done = ctx->sev + 6;  // [2] the layer running on set b has finished
  cudaEvent_t* y_copied = ctx->sev + 8;      // [2] y of the layer that ran on set b is on the host
  const rk_layer_buffers* sets[2] = {dev0, dev1};
  const int G = ctx->prof.n_groups, L = ctx->prof.n_heads - G;
  const size_t width = (size_t)G * ctx->prof.o_rank;

  // host -> device of layer l into set l & 1, on the copy-in stream, in the order the layer consumes them
  auto copy_in = [&](int l) -> cudaError_t {
    const rk_layer_io& io = layers[l];
    const rk_request* rq = io.req;
    const rk_layer_buffers* d = sets[l & 1];
    cudaError_t e = cudaMemcpyAsync(d->kv, io.kv_host, (size_t)rq->T * kDQK * 2, cudaMemcpyHostToDevice, cin);
    if (e == cudaSuccess && rq->A > 0)
      e = cudaMemcpyAsync(d->q_l, io.q_l_host, (size_t)rq->A * L * kDQK * 2, cudaMemcpyHostToDevice, cin);
    if (e == cudaSuccess) e = cudaEventRecord(kv_ql_in[l & 1], cin);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d->q_g, io.q_g_host, (size_t)rq->T * G * kDQK * 2, cudaMemcpyHostToDevice, cin);
    if (e == cudaSuccess) e = cudaEventRecord(qg_in[l & 1], cin);
    if (e == cudaSuccess && rq->n_off_rows > 0 && io.z_off_host)
      e = cudaMemcpyAsync(d->z_off, io.z_off_host, (size_t)rq->n_off_rows * width * 2, cudaMemcpyHostToDevice, cin);
    if (e == cudaSuccess) e = cudaEventRecord(zoff_in[l & 1], cin);
    return e;
  };

  // everything already queued on `stream` comes first (the buffer sets may still be in use)
  cudaError_t e = cudaEventRecord(ctx->ev[0], st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(cin, ctx->ev[0], 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(cout, ctx->ev[0], 0);
  if (e == cudaSuccess) e = copy_in(0);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "host to device copy");
  for (int l = 0; l < n_layers; ++l) {
    const int b = l & 1;
    const rk_layer_io& io = layers[l];
    const rk_layer_buffers* d = sets[b];
    if (l + 1 < n_layers) {  // prefetch the next layer while this one computes
      if (l >= 1) e = cudaStreamWaitEvent(cin, compute_done[b ^ 1], 0);  // layer l-1 has released set b^1
      if (e == cudaSuccess) e = copy_in(l + 1);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "host to device copy");
    }
    e = cudaStreamWaitEvent(st, kv_ql_in[b], 0);
    if (e == cudaSuccess && l >= 2) e = cudaStreamWaitEvent(st, y_copied[b], 0);  // y of layer l-2 has left set b
    if (e != cudaSuccess) return cuda_fail(ctx, e, "stream wait");
    // the first layer starts as soon as its first inputs are in; the last layer returns y in two row
    // ranges so that only the second one's copy is left when the kernels end
    rk_status s = layer_compute(ctx, io.req, d, io.W_uv, io.W_a, io.W_b, st, nullptr, qg_in[b], zoff_in[b],
                                l == n_layers - 1, io.y_host, cout, &ctx->ev[3]);
    if (s != RK_OK) return s;
    e = cudaEventRecord(compute_done[b], st);
    if (e == cudaSuccess) e = cudaEventRecord(y_copied[b], cout);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "device to host copy");
  }
  e = cudaStreamWaitEvent(st, y_copied[(n_layers - 1) & 1], 0);
  if (e == cudaSuccess && n_layers >= 2) e = cudaStreamWaitEvent(st, y_copied[n_layers & 1], 0);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? RK_OK : cuda_fail(ctx, e, "stack synchronisation");
}

// ------------------------------------------------------------------------------------------
// Selection rules: protected-row set (Eq. protected) and expert fan-out (Eq. moe)
rk_status rk_protected_rows_workspace_bytes(int64_t n_rows, int32_t n_segs, size_t* out) {
  if (!out) return RK_ERR_NULL;
  if (n_rows <= 0 || n_rows >= ((int64_t)1 << 30) || n_segs <= 0) return RK_ERR_LAYOUT;
  *out = policy_workspace_bytes(n_rows, n_segs);
  return RK_OK;
}

rk_status rk_protected_rows(rk_ctx* ctx, const rk_layout* lay, const rk_policy* pol, const int32_t* dirty_rows,
                            int64_t n_dirty, const float* scores, int32_t* rows_out, int64_t* count_out,
                            void* workspace, size_t workspace_bytes, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!lay || !pol || !rows_out || !count_out || !workspace || (n_dirty > 0 && !dirty_rows))
    return fail(ctx, RK_ERR_NULL, "null argument");
  {
    char msg[256] = {0};
    rk_status s = rk_check_request(lay, nullptr, 0, msg, sizeof(msg));
    // the layout-only part of the check: rows without artifact are what this call is about to protect
    if (s != RK_OK && s != RK_ERR_ROWS) return fail(ctx, s, "%s", msg);
  }
  if (pol->edge_rows < 0 || pol->tail_rows < 0 || pol->budget_bp < 0 || pol->budget_bp > 10000)
    return fail(ctx, RK_ERR_PROFILE, "policy out of range: edge_rows %d, tail_rows %lld, budget_bp %d", pol->edge_rows,
                (long long)pol->tail_rows, pol->budget_bp);
  if (n_dirty < 0) return fail(ctx, RK_ERR_ROWS, "n_dirty is negative");
  const int S = lay->n_segs;
  const int64_t T = lay->seg_off[S];
  const size_t need = policy_workspace_bytes(T, S);
  if (workspace_bytes < need) return fail(ctx, RK_ERR_WORKSPACE, "workspace too small: %zu < %zu", workspace_bytes, need);
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return fail(ctx, RK_ERR_WORKSPACE, "workspace must be 256-byte aligned");
  std::vector<int32_t> tab((size_t)(2 * S + 1));
  int64_t req_end = 0;
  for (int i = 0; i <= S; ++i) tab[(size_t)i] = (int32_t)lay->seg_off[i];
  for (int i = 0; i < S; ++i) {
    tab[(size_t)(S + 1 + i)] = (int32_t)lay->seg_delta[i];
    req_end = std::max<int64_t>(req_end, lay->seg_delta[i] + lay->seg_off[i + 1] - lay->seg_off[i]);
  }
  // the artifact flags are staged in a library-owned pageable vector like the segment table: the copy then
  // never reads the caller's array after this call has returned, whether or not that array is pinned
  std::vector<uint8_t> has_stage(lay->seg_has_artifact, lay->seg_has_artifact + S);
  PolicyHost h = {};
  h.seg_tab_host = tab.data();
  h.has_host = has_stage.data();
  h.n_segs = S;
  h.T = T;
  h.req_end = req_end;
  h.tail_rows = pol->tail_rows;
  h.edge_rows = pol->edge_rows;
  h.budget_bp = pol->budget_bp;
  h.dirty = dirty_rows;
  h.n_dirty = n_dirty;
  h.scores = scores;
  h.rows_out = rows_out;
  h.count_out = reinterpret_cast<long long*>(count_out);
  h.workspace = workspace;
  h.status = ctx->d_status;
  cudaError_t e = launch_protected_rows(h, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e, "protected-row kernels");
  return RK_OK;
}

rk_status rk_moe_fanout(rk_ctx* ctx, const float* p, int64_t n, float tau, int32_t fence, uint8_t* k_out,
                        uint8_t* keep_out, void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (n < 0) return fail(ctx, RK_ERR_ROWS, "n is negative");
  if (n > 0 && (!p || !k_out || !keep_out)) return fail(ctx, RK_ERR_NULL, "null argument");
  if ((reinterpret_cast<uintptr_t>(p) & 7u) != 0) return fail(ctx, RK_ERR_LAYOUT, "router weights must be 8-byte aligned");
  if (!(tau == tau)) return fail(ctx, RK_ERR_PROFILE, "tau is NaN");
  cudaError_t e = launch_moe_fanout(p, n, tau, fence != 0, k_out, keep_out, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(ctx, e, "fan-out kernel");
  return RK_OK;
}

}  // extern "C"

extern "C" rk_status rk_group_sliced_proj_static(rk_ctx* ctx, const rk_request* rq, const void* O_g, const void* O_l,
                                                 const void* W_uv, const void* W_a, void* z_on_g, void* z_on_l,
                                                 void* stream) {
  if (!ctx) return RK_ERR_NULL;
  if (!rq) return fail(ctx, RK_ERR_NULL, "null argument");
  if (rq->ctx != ctx) return fail(ctx, RK_ERR_LAYOUT, "request belongs to another context");
  const size_t need = proj_ws_bytes(rq);
  if (need > (size_t)RK_STATIC_SCRATCH_BYTES)
    return fail(ctx, RK_ERR_WORKSPACE,
                "request needs %zu bytes of projection scratch but the built-in array holds %u; use "
                "rk_group_sliced_proj with a caller workspace",
                need, (unsigned)RK_STATIC_SCRATCH_BYTES);
  int device = -1;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetDevice");
  if (device != ctx->device) return fail(ctx, RK_ERR_CUDA, "the context's device is not current");
  void* scratch = nullptr;
  e = static_scratch_address(device, &scratch);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaGetSymbolAddress(rk_static_scratch)");
  // (already resolved by rk_create on this device: a table lookup, no runtime call)
  // nothing in the scratch has to start at zero: o is fully written before it is read, and rows
  // beyond the tensor's extent are zero-filled by the TMA load, never read from the array
  return rk_group_sliced_proj(ctx, rq, O_g, O_l, W_uv, W_a, z_on_g, z_on_l, scratch, RK_STATIC_SCRATCH_BYTES, stream);
}
