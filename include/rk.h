/* rk.h -- C ABI of the B200 (sm_100a) MLA-Online step of RedKnot-MLA.
 *
 * One online layer (Algorithm 2 "Relocate, recompute, and merge one online layer"):
 *   for every document segment i:  q_i = R(-delta_i) q;  SelectiveMLA(q_i, C_i, A)
 *   SegmentedLSEMerge over segments;  z_online = W_{a,G} O_G + W_{a,L} O_{L,A};
 *   z = RestoreAndReplace(z_off, z_online, A);  y = W_b z.
 *
 * Conventions
 *  - Every function returns an rk_status (0 = RK_OK) and never throws.  All argument errors
 *    are found on the host before anything is enqueued.  rk_last_error() gives a message.
 *  - "device" pointers are CUDA device memory owned by the caller; "host" pointers are
 *    ordinary host memory that is copied during the call and not retained.
 *  - bf16 tensors are passed as `const void*` holding 16-bit bfloat16 (the bits of
 *    torch.bfloat16 / __nv_bfloat16); all tensors are dense row-major, innermost dimension
 *    contiguous, base pointers 16-byte aligned.
 *  - Rows are in PACKED order: document 0, 1, ..., then the query suffix -- the order of the
 *    packed latent stream.  Packed row r of segment i sits at request position
 *    pos[r] = seg_delta[i] + (r - seg_off[i]).  Row t sees key k iff pos[k] <= pos[t].
 *  - `stream` is a cudaStream_t (0 = default stream).  Calls enqueue work and return; the
 *    only blocking calls are rk_create / rk_request_create / rk_poll_status / *_destroy and
 *    rk_layer_host.
 *  - The library allocates device memory only inside rk_create and rk_request_create (small
 *    tables) and frees it in the matching destroy.  kv, weights and z_off are never written.
 *  - No kernel traps: a device-side wait that expires records RK_ERR_TIMEOUT in a status
 *    word, the kernel drains and returns; rk_poll_status() reads (and clears) that word.
 *  - There is no fallback: rk_create fails with RK_ERR_UNSUPPORTED on a device that is not
 *    compute capability 10.x.
 */
#ifndef RK_H_
#define RK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum rk_status {
  RK_OK = 0,
  RK_ERR_NULL = 1,        /* a required pointer is NULL */
  RK_ERR_PROFILE = 2,     /* head/group geometry inconsistent */
  RK_ERR_LAYOUT = 3,      /* segment table invalid */
  RK_ERR_ROWS = 4,        /* protected-row list invalid */
  RK_ERR_ALIGN = 5,       /* pointer or stride not 16-byte aligned */
  RK_ERR_WORKSPACE = 6,   /* workspace too small */
  RK_ERR_UNSUPPORTED = 7, /* dims / device not supported */
  RK_ERR_CUDA = 8,        /* a CUDA call failed */
  RK_ERR_TIMEOUT = 9      /* a bounded device-side wait expired */
} rk_status;

/* Head partition and projection geometry (Eq. partition; Section "DeepSeek-V4 Flash and Pro
 * profiles": one Global head per native group of eight).  Supported: group_size 8,
 * d_latent 512, d_rope 64, d_v 128; o_rank and d_model multiples of 128. */
typedef struct rk_profile {
  int32_t n_heads;              /* H */
  int32_t n_groups;             /* G = H / group_size */
  int32_t group_size;           /* 8 */
  int32_t d_latent;             /* 512: width of the shared latent c (also the value width) */
  int32_t d_rope;               /* 64 */
  int32_t d_v;                  /* 128: per-head width after W_uv */
  int32_t o_rank;               /* r_o: rows of each group's block of W_a */
  int32_t d_model;              /* rows of W_b */
  float sm_scale;               /* softmax scale applied to q.k */
  float rope_base;              /* theta_j = rope_base^(-2j/d_rope), interleaved pairs */
  const int32_t* global_heads;  /* host [n_groups]: absolute index of each group's Global head,
                                   global_heads[g] / group_size == g */
} rk_profile;

/* Segment geometry of one request (Section "Online position restoration and segmented
 * merge"): document i was built at positions 0..n_i-1 and appears at request offset
 * seg_delta[i].  Request-position intervals must not overlap; gaps are legal. */
typedef struct rk_layout {
  int32_t n_segs;
  const int64_t* seg_off;          /* host [n_segs+1], packed-row prefix sums, seg_off[0] = 0 */
  const int64_t* seg_delta;        /* host [n_segs], >= 0 */
  const uint8_t* seg_has_artifact; /* host [n_segs]; 0 = no offline artifact (all its rows must be protected) */
} rk_layout;

typedef struct rk_request_info {
  int64_t n_rows;        /* T */
  int64_t n_prot;        /* A */
  int64_t n_off_rows;    /* rows the z_off tensor must have (end of the last segment with artifact) */
  int64_t pairs_global;  /* visible (row,key) pairs summed over rows: T(T+1)/2 for gap-free layouts */
  int64_t pairs_local;   /* visible pairs summed over protected rows */
  int32_t n_tiles_global;
  int32_t n_tiles_local;
} rk_request_info;

typedef struct rk_ctx rk_ctx;
typedef struct rk_request rk_request;

const char* rk_version(void);
const char* rk_status_string(rk_status s);

/* Creates a context on the CURRENT CUDA device.  Copies the profile (including global_heads). */
rk_status rk_create(const rk_profile* profile, rk_ctx** out);
/* Output-phase variant (Eq. offonline: z = W_a R^{-1}(O); Algorithm 2: RestorePhase(O_i, delta_i) per
 * segment before SegmentedLSEMerge and R^{-1} in the z_online statement).  With RK_VALUE_PHASE the
 * value of a key is its whole stored row [c | k_rope] (576 wide), not the latent alone, so an
 * attention output carries 64 rotated dims.  Inside a segment they accumulate in the document's
 * position-zero frame; RestorePhase turns them by R(+seg_delta[i]) into the request frame, where
 * segments may be merged; R^{-1} turns row t's merged rope dims by R(-pos[t]), after which they
 * depend on relative positions only.  The attention kernel does all three inside its running merge.
 * What changes at the interface, and nothing else:
 *   O_g / O_l (and O_part / O of rk_segmented_merge_phase) rows are 576 wide, rope dims last;
 *   W_uv is [H][128][576];  rk_mla_off_build applies R^{-1} at the row's canonical position.
 * The plain context (flags = 0) treats both maps as the identity: its values carry no rotated dims. */
#define RK_VALUE_PHASE 1u
rk_status rk_create_ex(const rk_profile* profile, uint32_t flags, rk_ctx** out);
rk_status rk_destroy(rk_ctx* ctx);
/* Message of the last failing call on this context (valid until the next call). */
const char* rk_last_error(const rk_ctx* ctx);
/* Synchronises `stream`, returns the device status word (RK_OK, RK_ERR_TIMEOUT, or RK_ERR_ROWS from the
 * bounds-checked build) and clears it. */
rk_status rk_poll_status(rk_ctx* ctx, void* stream);
/* Per-wait time limit of device-side waits, in milliseconds (default 2000). */
rk_status rk_set_wait_limit_ms(rk_ctx* ctx, int32_t ms);
/* Test hook for the timeout path (failure detection without a GPU fault): while `on` is non-zero the
 * attention launches of this context use an instantiation whose load warp leaves every ring stage
 * empty, so the consumers' bounded waits expire, the kernel drains and returns, and
 * rk_poll_status() reports RK_ERR_TIMEOUT.  Results are not produced while it is on.  Use it
 * together with a short rk_set_wait_limit_ms. */
rk_status rk_test_starve_loads(rk_ctx* ctx, int32_t on);
/* The library can be built with -DRK_CHECK (paper_2609_07008_b200/build.py, check=True): its kernels then
 * test every index they derive from a request table (protected-row list, inverse row map, work list,
 * compaction offsets) before using it, skip the access when it is out of range and record RK_ERR_ROWS in
 * the status word that rk_poll_status reads.  It is a debugging aid for small cases, not the production
 * build.  rk_check_selftest pushes one deliberately bad index through that check (nothing is accessed):
 * on the checking build the next rk_poll_status returns RK_ERR_ROWS; the ordinary build returns
 * RK_ERR_UNSUPPORTED here. */
rk_status rk_check_selftest(rk_ctx* ctx, void* stream);

/* Request geometry object: validates the layout and the protected-row list (Eq. protected;
 * the list is data here), builds row positions, per-segment relocation tables
 * cos/sin(delta_i * theta_j) in double precision, the inverse row map and the tile work
 * lists, and uploads them.  prot_rows: host [n_prot], strictly ascending packed rows; must
 * contain every row of every segment without artifact.  Reusable across layers and calls. */
rk_status rk_request_create(rk_ctx* ctx, const rk_layout* layout, const int32_t* prot_rows, int64_t n_prot,
                            rk_request** out);
rk_status rk_request_destroy(rk_request* req);
/* The same validation as rk_request_create, on the host only (no device, no context): returns the
 * status rk_request_create would return for this layout / row list and writes a message into msg
 * (may be NULL). */
rk_status rk_check_request(const rk_layout* layout, const int32_t* prot_rows, int64_t n_prot, char* msg,
                           size_t msg_len);
rk_status rk_request_get_info(const rk_request* req, rk_request_info* out);
/* Bytes of device scratch that rk_group_sliced_proj needs (per-head o = W_uv O_lat in bf16). */
rk_status rk_workspace_bytes(const rk_request* req, size_t* out);

/* (1) Query-side RoPE relocation, standalone form (Algorithm 2: q_i <- R(-delta_i) q; Eq. rope).
 * q_rope: device bf16, rope sub-vectors (64 wide) of n_rows x n_heads queries already rotated at
 * their request positions; element (r, h, e) at q_rope[r*row_stride + h*head_stride + e]
 * (strides in elements, multiples of 8).  out: device bf16 [seg_end-seg_begin][n_rows][n_heads][64],
 * out[i] = R(-seg_delta[seg_begin+i]) q.  The same rotation is fused into rk_mla_online_attn. */
rk_status rk_relocate_q(rk_ctx* ctx, const rk_request* req, const void* q_rope, int64_t n_rows, int32_t n_heads,
                        int64_t row_stride, int64_t head_stride, int32_t seg_begin, int32_t seg_end, void* out,
                        void* stream);

/* (2) Absorbed-MLA attention over the packed latent (Algorithm 2: SelectiveMLA for every
 * segment + running SegmentedLSEMerge inside the kernel; relocation fused into the Q load).
 *   kv   device bf16 [T][576] = [c (512) | k_rope at the document's canonical position (64)]
 *   q_g  device bf16 [T][G][576]  queries of the Global heads (group order), request position
 *   q_l  device bf16 [A][L][576]  queries of the Local heads (ascending head index) on the
 *        protected rows in list order
 *   O_g  device bf16 [T][G][512], lse_g device fp32 [T][G]   (natural-log LSE of scaled scores)
 *   O_l  device bf16 [A][L][512], lse_l device fp32 [A][L]
 * Either pass may be skipped by passing NULL for its q, O and lse. */
rk_status rk_mla_online_attn(rk_ctx* ctx, const rk_request* req, const void* kv, const void* q_g, const void* q_l,
                             void* O_g, float* lse_g, void* O_l, float* lse_l, void* stream);

/* (3) Stable segmented log-sum-exp merge, standalone form (Algorithm 2: SegmentedLSEMerge):
 * lse = log sum_j exp(lse_j), O = sum_j exp(lse_j - lse) O_j over n_parts partial results.
 *   O_part   device [n_parts][n_rows][n_heads][512], bf16 (part_dtype 0) or fp32 (part_dtype 1)
 *   lse_part device fp32 [n_parts][n_rows][n_heads]; -inf marks an empty part (its O is ignored)
 *   O device bf16 [n_rows][n_heads][512], lse device fp32 [n_rows][n_heads]
 * All parts empty gives O = 0, lse = -inf.  n_parts <= 4096. */
rk_status rk_segmented_merge(rk_ctx* ctx, int32_t n_parts, int64_t n_rows, int32_t n_heads, const void* O_part,
                             int32_t part_dtype, const float* lse_part, void* O, float* lse, void* stream);

/* The same merge for per-segment partial results of the output-phase variant (Algorithm 2:
 * RestorePhase, then SegmentedLSEMerge, then R^{-1}).  Part j is the partial result against the
 * canonical rows of segment seg_begin + j: its 64 rope dims (the last of 576) are in that document's
 * frame and are turned by R(+seg_delta[seg_begin + j]) before they are added.
 *   O_part   device [n_parts][n_rows][n_heads][576], bf16 (part_dtype 0) or fp32 (part_dtype 1)
 *   lse_part device fp32 [n_parts][n_rows][n_heads]; -inf marks an empty part (its O is ignored)
 *   row_pos  device int32 [n_rows]: request position of each row, whose merged rope dims are turned by
 *            R(-row_pos[r]); NULL leaves the result in the request frame
 *   O device bf16 [n_rows][n_heads][576], lse device fp32 [n_rows][n_heads]
 * seg_begin + n_parts <= number of segments of `req`; n_parts <= 4096. */
rk_status rk_segmented_merge_phase(rk_ctx* ctx, const rk_request* req, int32_t seg_begin, int32_t n_parts, int64_t n_rows,
                                   int32_t n_heads, const void* O_part, int32_t part_dtype, const float* lse_part,
                                   const int32_t* row_pos, void* O, float* lse, void* stream);

/* (4) Group-aligned sliced first output projection (Eq. offonline; Algorithm 2: z_online):
 * per head o = W_uv[h] O_lat (512 -> 128), then the head's 128-column slice of its group's W_a:
 *   z_on_g[t][g] = W_a[g][:, 128 j_g : 128 j_g + 128] o[t][global head of g]         (all T rows)
 *   z_on_l[a][g] = sum over the 7 Local heads j of group g of W_a[g][:, 128 j : ..] o[a][8g+j]
 *   W_uv device bf16 [H][128][512];  W_a device bf16 [G][r_o][1024]
 *   z_on_g device bf16 [T][G*r_o];   z_on_l device bf16 [A][G*r_o]
 * workspace: device scratch of at least rk_workspace_bytes().  Either half may be skipped by
 * passing NULL for its O and z. */
rk_status rk_group_sliced_proj(rk_ctx* ctx, const rk_request* req, const void* O_g, const void* O_l,
                               const void* W_uv, const void* W_a, void* z_on_g, void* z_on_l, void* workspace,
                               size_t workspace_bytes, void* stream);

/* The same projection for callers that cannot allocate device memory (the paper has no
 * counterpart; it is a property of this library's interface only).  A serving process that has
 * given the whole device to its own memory pool, or a request path that must not pay the
 * device-wide synchronisation an allocation can trigger, has no workspace to pass to
 * rk_group_sliced_proj.  Here the per-head intermediate lives in a fixed 32 MiB
 * (33 554 432 bytes) array inside the loaded library image; every device that loads the library
 * holds that array until the process exits.  The call allocates and frees nothing.
 *  - Requests whose scratch need (rk_workspace_bytes) exceeds 32 MiB are rejected with
 *    RK_ERR_WORKSPACE and a message; use rk_group_sliced_proj with your own workspace then.
 *  - rk_create looks up the array's device address on the context's device (the lookup makes the
 *    runtime place the array on that device, which may allocate and synchronise once); the entry
 *    point itself only reads the cached address, so create the context before any stream capture.
 *    The context's device must be current when the entry point is called.
 *  - All calls, from all contexts and streams of a process, share the one array, and it keeps
 *    whatever the previous call left in it.  Nothing in it needs to start at zero.  Two calls
 *    whose kernels overlap on the GPU (different streams) race on it: serialise them.
 * Arguments and results are exactly those of rk_group_sliced_proj, minus the workspace. */
rk_status rk_group_sliced_proj_static(rk_ctx* ctx, const rk_request* req, const void* O_g, const void* O_l,
                                      const void* W_uv, const void* W_a, void* z_on_g, void* z_on_l, void* stream);

/* (5) Add the offline MLA-Off artifact and run the shared second projection (Algorithm 2:
 * RestoreAndReplace, then W_b z; the paragraph after Eq. protected: a row in A takes the online Local
 * value in place of the artifact's, the two are never added):
 *   z[t] = z_on_g[t] + (t in A ? z_on_l[slot(t)] : z_off[t]);  y = W_b z.
 *   z_off device bf16 [n_off_rows][G*r_o] (packed rows; rows in A are never read)
 *   W_b   device bf16 [d_model][G*r_o], may be NULL to stop at z
 *   z     device bf16 [T][G*r_o] (required);  y device bf16 [T][d_model] (required iff W_b) */
rk_status rk_combine_offline(rk_ctx* ctx, const rk_request* req, const void* z_on_g, const void* z_on_l,
                             const void* z_off, const void* W_b, void* z, void* y, void* stream);

/* Offline side (Algorithm 1 "Build one canonical MLA-Off document artifact"): for packed rows
 * [row_begin, row_end) each row attends only the keys of its own segment, causally in the
 * segment's position-zero frame, with the Local heads; then z_off = W_{a,L} (W_uv O_L) summed over
 * each group's seven Local heads.  Queries are given at their REQUEST positions (like q_l); the
 * kernel rotates them by -seg_delta into the document's frame, which is the query the document had
 * when it was processed alone at position zero.
 *   q_l_rows   device bf16 [row_end-row_begin][L][576]
 *   z_off_rows device bf16 [row_end-row_begin][G*r_o]  (row row_begin of the artifact tensor)
 *   workspace  device scratch of at least rk_mla_off_workspace_bytes(req, row_end-row_begin)
 * Long requests are built in several calls over row ranges (the scratch holds the Local-head
 * attention output of the range). */
rk_status rk_mla_off_workspace_bytes(const rk_request* req, int64_t n_rows, size_t* out);
rk_status rk_mla_off_build(rk_ctx* ctx, const rk_request* req, const void* kv, int64_t row_begin, int64_t row_end,
                           const void* q_l_rows, const void* W_uv, const void* W_a, void* z_off_rows, void* workspace,
                           size_t workspace_bytes, void* stream);

/* Controller of the protected-row set (Eq. protected).  The paper's values: edge_rows 128,
 * tail_rows 32768, budget_bp 0 (no expansion), 1000, 2000 or 2500. */
typedef struct rk_policy {
  int32_t edge_rows;  /* B_edge: first and last rows of every relocated segment; >= 0 */
  int64_t tail_rows;  /* T_tail: the last request positions; >= 0 */
  int32_t budget_bp;  /* active budget in basis points of the candidate rows; 0..10000 */
} rk_policy;

/* Builds the protected token-row set A = Q u N u D u B_edge u I_top u T_tail (Eq. protected;
 * `ProtectedRows` of Algorithm 2) on the device, as the strictly ascending packed-row list that
 * rk_request_create takes.  Packed row t of segment i has canonical index j = t - seg_off[i] and
 * request position seg_delta[i] + j.
 *   Q u N   every row of a segment without artifact
 *   D       dirty_rows: device int32 [n_dirty], any order, duplicates allowed, entries outside
 *           [0,T) ignored; may be NULL iff n_dirty == 0
 *   B_edge  rows with j < edge_rows or j >= n_i - edge_rows of every segment that has an artifact
 *           and seg_delta[i] != 0 (artifacts are built at offset 0; any other offset relocates)
 *   T_tail  rows at request positions >= end - tail_rows, end = largest position + 1
 *   I_top   candidate rows = rows of segments with artifact.  If the sets above hold fewer than
 *           floor(budget_bp * candidates / 10000) candidate rows, the candidate rows outside them
 *           with the largest scores are added until that number is reached (equal scores: lower
 *           packed row first; -0.0 equals +0.0).  The sets above are never cut.
 *           scores: device float32 [T] (the Indexer's row scores, recomputed by the caller for
 *           this request; entries of non-candidate rows are not read), no NaN; NULL = no top-up.
 *   rows_out  device int32 [T] (capacity); the first *count_out entries are the result
 *   count_out device int64 [1]
 *   workspace device scratch of at least rk_protected_rows_workspace_bytes(T, n_segs), 256-byte aligned
 * The layout is host data and is validated like in rk_request_create (RK_ERR_LAYOUT).  The call
 * enqueues on `stream` and does not synchronise; read rows_out / count_out after the stream has
 * passed it.  The selection is exact (integer work; the scores are only compared), so the list is
 * bit-identical to the definition. */
rk_status rk_protected_rows_workspace_bytes(int64_t n_rows, int32_t n_segs, size_t* out);
rk_status rk_protected_rows(rk_ctx* ctx, const rk_layout* layout, const rk_policy* policy, const int32_t* dirty_rows,
                            int64_t n_dirty, const float* scores, int32_t* rows_out, int64_t* count_out,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Retained expert fan-out of the adaptive sparse-MoE path (Eq. moe) for n tokens.
 *   p        device float32 [n][6]: the router weights of the token's Top-6 experts, any slot
 *            order, positive, no NaN; 8-byte aligned
 *   tau      the cumulative-share threshold
 *   fence    non-zero: a full-recompute fence layer, every token keeps all six (K_t = 6)
 *   k_out    device uint8 [n]: K_t in {3,4,5,6}
 *   keep_out device uint8 [n]: bit s set = the expert in slot s stays (the K_t largest weights;
 *            equal weights: lower slot first)
 * The weights are not renormalised and not written.  Decision arithmetic (float32, fixed order):
 * weights sorted descending, c_1 = p_(1), c_k = c_(k-1) + p_(k); K_t = the smallest k in {3,4,5}
 * with c_k >= tau * c_6, else 6 -- the paper's condition with both sides multiplied by the sum. */
rk_status rk_moe_fanout(rk_ctx* ctx, const float* p, int64_t n, float tau, int32_t fence, uint8_t* k_out,
                        uint8_t* keep_out, void* stream);

/* Device buffers that rk_layer_host stages through; all owned by the caller. */
typedef struct rk_layer_buffers {
  void *kv, *q_g, *q_l, *z_off;            /* device copies of the per-request inputs */
  void *O_g, *O_l, *z_on_g, *z_on_l, *z, *y;
  float *lse_g, *lse_l;
  void* workspace;
  size_t workspace_bytes;
} rk_layer_buffers;

/* rk_layer_host and rk_layer_stack_host use one set of internal copy streams and events per
 * context: at most one of them may be running on a context at any time (two host threads must not
 * call them concurrently on the same rk_ctx; use one context per thread).
 *
 * One whole layer from HOST inputs: copies kv, q_g, q_l, z_off host->device (use pinned host
 * memory; pageable memory works but serialises), runs (2), (4), (5), copies y device->host and
 * synchronises `stream`.  Weights stay resident on the device.  Copies that the running kernel
 * does not need yet travel on an internal second stream beside it (the Local pass needs only kv
 * and q_l; q_g and the artifact arrive meanwhile; the Global pass and everything after it run in
 * two row ranges, and the y rows of the first range return while the second computes) and are
 * ordered by device events, not by host polling (Section "Turning omitted
 * work into latency reduction": prefetch stream guarded by device events). */
rk_status rk_layer_host(rk_ctx* ctx, const rk_request* req, const void* kv_host, const void* q_g_host,
                        const void* q_l_host, const void* z_off_host, const void* W_uv, const void* W_a,
                        const void* W_b, const rk_layer_buffers* dev, void* y_host, void* stream);

/* One layer of a stack for rk_layer_stack_host. */
typedef struct rk_layer_io {
  const rk_request* req;                                    /* geometry + protected rows of this layer */
  const void *kv_host, *q_g_host, *q_l_host, *z_off_host;   /* pinned host inputs (shapes as in rk_layer_host) */
  const void *W_uv, *W_a, *W_b;                             /* device weights of this layer */
  void* y_host;                                             /* pinned host output [T][d_model] */
} rk_layer_io;

/* A stack of layers from HOST inputs with cross-layer prefetch (Section "Turning omitted work into
 * latency reduction": while layer l runs, a dedicated stream brings in the inputs of layer l+1;
 * device events, not host polling, guard consumption).  Two complete buffer sets are used in turn:
 * the inputs of layer l+1 are copied into the other set while layer l computes, and y of layer l
 * is copied out on a third stream while layer l+1 computes.  Synchronises `stream` before it
 * returns.  Every request must belong to `ctx`; the sets must be large enough for every layer. */
rk_status rk_layer_stack_host(rk_ctx* ctx, int32_t n_layers, const rk_layer_io* layers, const rk_layer_buffers* dev0,
                              const rk_layer_buffers* dev1, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RK_H_ */
