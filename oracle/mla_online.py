"""Plain float64 definition of what one MLA-Online layer computes (numpy only).

Test infrastructure: slow on purpose, no blocking / fusion / reordering beyond what each
cited passage states.  All tensors are float64 arrays holding the (bf16-rounded) values
that the CUDA path receives.

Notation follows the paper: H logical heads split into Local and Global sets
(Eq. partition); one Global head per native group of eight (Section "DeepSeek-V4 Flash
and Pro profiles"); packed latent stream C shared by every head; document i built at
positions 0..n_i-1 and placed at request offset delta_i (Eq. rope); protected token-row
set A (Eq. protected); z = z_off + z_online, y = W_b z (Eq. factorization).
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "rope_theta", "rope_rotate", "request_positions", "segment_of_rows",
    "keys_in_request_frame", "attend_rows", "head_contributions",
    "mla_online_rows", "full_recompute_rows", "mla_off_artifact", "segmented_merge",
    "relocate_query", "attend_rows_segmentwise", "head_row_ceiling", "cold_speed_ratio",
    "reuse_error_report", "inverse_row_map",
]


# ---------------------------------------------------------------------------------
# RoPE.  The paper only uses R(.) and its orthogonality (Eq. rope).  Convention taken
# here: interleaved pairs (2j, 2j+1), theta_j = base^(-2j/d_r), and
#   R(p): (x_2j, x_2j+1) -> (x_2j cos(p theta_j) - x_2j+1 sin(p theta_j),
#                            x_2j sin(p theta_j) + x_2j+1 cos(p theta_j)).
# ---------------------------------------------------------------------------------

def rope_theta(d_rope: int, base: float) -> np.ndarray:
    j = np.arange(d_rope // 2, dtype=np.float64)
    return np.power(np.float64(base), -2.0 * j / np.float64(d_rope))


def rope_rotate(x: np.ndarray, pos, base: float) -> np.ndarray:
    """R(pos) applied to the last axis of x (width d_r).  pos broadcasts against x's
    leading axes (a scalar, or an array shaped like x.shape[:-1] or broadcastable)."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    theta = rope_theta(d, base)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta       # [..., d/2]
    c, s = np.cos(ang), np.sin(ang)
    xe, xo = x[..., 0::2], x[..., 1::2]
    out = np.empty(np.broadcast_shapes(x.shape, c.shape[:-1] + (d,)), dtype=np.float64)
    out[..., 0::2] = xe * c - xo * s
    out[..., 1::2] = xe * s + xo * c
    return out


def relocate_query(q_rope: np.ndarray, delta, base: float) -> np.ndarray:
    """q_i = R(-delta_i) q  (Algorithm 2, the first statement of the segment loop)."""
    return rope_rotate(q_rope, -np.asarray(delta, dtype=np.float64), base)


# ---------------------------------------------------------------------------------
# geometry
# ---------------------------------------------------------------------------------

def segment_of_rows(seg_off: np.ndarray) -> np.ndarray:
    seg_off = np.asarray(seg_off, dtype=np.int64)
    T = int(seg_off[-1])
    seg = np.empty(T, dtype=np.int64)
    for i in range(len(seg_off) - 1):
        seg[seg_off[i]:seg_off[i + 1]] = i
    return seg


def request_positions(seg_off: np.ndarray, seg_delta: np.ndarray) -> np.ndarray:
    """pos[r] = delta_i + (r - off_i) for packed row r in segment i."""
    seg_off = np.asarray(seg_off, dtype=np.int64)
    T = int(seg_off[-1])
    pos = np.empty(T, dtype=np.int64)
    for i in range(len(seg_off) - 1):
        n = int(seg_off[i + 1] - seg_off[i])
        pos[seg_off[i]:seg_off[i + 1]] = int(seg_delta[i]) + np.arange(n, dtype=np.int64)
    return pos


def inverse_row_map(prot_rows: np.ndarray, T: int) -> np.ndarray:
    """slot of each packed row in the protected list, -1 when the row is not protected."""
    inv = np.full(T, -1, dtype=np.int64)
    inv[np.asarray(prot_rows, dtype=np.int64)] = np.arange(len(prot_rows), dtype=np.int64)
    return inv


def keys_in_request_frame(kv: np.ndarray, seg_off, seg_delta, d_latent: int, base: float) -> np.ndarray:
    """Left side of Eq. rope: the stored key of canonical position p_k in document i is
    re-rotated to its request position, K_req[k] = [c_k | R(+delta_i) k_rope[k]]
    (the stored rope part already carries R(p_k), so one more R(delta_i) gives
    R(p_k + delta_i))."""
    kv = np.asarray(kv, dtype=np.float64)
    seg = segment_of_rows(seg_off)
    d = np.asarray(seg_delta, dtype=np.float64)[seg]
    out = kv.copy()
    out[:, d_latent:] = rope_rotate(kv[:, d_latent:], d, base)
    return out


# ---------------------------------------------------------------------------------
# attention: one softmax per (row, head) over everything the row may see
# ---------------------------------------------------------------------------------

def attend_rows(q: np.ndarray, row_pos: np.ndarray, k_req: np.ndarray, v: np.ndarray,
                key_pos: np.ndarray, sm_scale: float, key_subset: np.ndarray | None = None):
    """q [n, h, d_qk] (already at request position), row_pos [n]; k_req [T, d_qk];
    v [T, d_c]; key_pos [T].  Row t sees key k iff key_pos[k] <= row_pos[t] (causal in
    request-position space; documents placed earlier are seen in full, later ones not at
    all).  Returns O_lat [n, h, d_c] and the natural-log LSE of the scaled scores [n, h].
    key_subset (optional index array) restricts the keys -- used to form partial results.
    A row with no visible key gets O = 0, lse = -inf."""
    q = np.asarray(q, dtype=np.float64)
    n, h, _ = q.shape
    dc = v.shape[1]
    O = np.zeros((n, h, dc), dtype=np.float64)
    lse = np.full((n, h), -np.inf, dtype=np.float64)
    for i in range(n):
        vis = key_pos <= row_pos[i]
        if key_subset is not None:
            m2 = np.zeros_like(vis)
            m2[key_subset] = True
            vis &= m2
        idx = np.nonzero(vis)[0]
        if len(idx) == 0:
            continue
        s = (q[i] @ k_req[idx].T) * sm_scale            # [h, nvis]
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        l = p.sum(axis=1, keepdims=True)
        O[i] = (p @ v[idx]) / l
        lse[i] = (m + np.log(l))[:, 0]
    return O, lse


def segmented_merge(O_parts: np.ndarray, lse_parts: np.ndarray):
    """Stable log-sum-exp merge of partial attention results (Algorithm 2,
    SegmentedLSEMerge): lse = log sum_j exp(lse_j), O = sum_j exp(lse_j - lse) O_j.
    O_parts [P, ..., d], lse_parts [P, ...].  A part with lse_j = -inf contributes nothing
    (its O_j is ignored even if it is not finite); if every part is empty the result is
    O = 0, lse = -inf."""
    O_parts = np.asarray(O_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    m_safe = np.where(np.isfinite(m), m, 0.0)
    w = np.exp(lse_parts - m_safe)                      # exp(-inf) = 0 for empty parts
    tot = w.sum(axis=0)
    with np.errstate(divide="ignore"):
        lse = np.where(tot > 0, m_safe + np.log(np.where(tot > 0, tot, 1.0)), -np.inf)
    wn = np.where(tot > 0, w / np.where(tot > 0, tot, 1.0), 0.0)
    Oc = np.where(wn[..., None] > 0, O_parts, 0.0)
    O = (wn[..., None] * Oc).sum(axis=0)
    return O, lse


def attend_rows_segmentwise(q: np.ndarray, row_pos: np.ndarray, kv: np.ndarray, seg_off, seg_delta,
                            d_latent: int, base: float, sm_scale: float):
    """The paper's own order of evaluation (Algorithm 2): for every document segment i
    rotate the query by -delta_i, attend the *canonical* stored keys of that segment with
    the causal limit expressed in the canonical frame, then LSE-merge the per-segment
    partials.  Used to pin the plain definition above (relocation + merge are exact
    re-associations)."""
    q = np.asarray(q, dtype=np.float64)
    kv = np.asarray(kv, dtype=np.float64)
    S = len(seg_delta)
    Op, Lp = [], []
    for i in range(S):
        lo, hi = int(seg_off[i]), int(seg_off[i + 1])
        qi = q.copy()
        qi[..., d_latent:] = relocate_query(q[..., d_latent:], float(seg_delta[i]), base)
        canon = np.arange(hi - lo, dtype=np.int64)
        # key at canonical index c is visible iff delta_i + c <= row_pos
        O_i, l_i = attend_rows(qi, np.asarray(row_pos) - int(seg_delta[i]), kv[lo:hi],
                               kv[lo:hi, :d_latent], canon, sm_scale)
        Op.append(O_i)
        Lp.append(l_i)
    return segmented_merge(np.stack(Op), np.stack(Lp))


# ---------------------------------------------------------------------------------
# output projections (Eq. offonline / Eq. factorization)
# ---------------------------------------------------------------------------------

def head_contributions(O_lat: np.ndarray, head_ids: np.ndarray, w_uv: np.ndarray, w_a: np.ndarray,
                       group_size: int = 8) -> np.ndarray:
    """O_lat [n, h, d_c] for absolute heads head_ids [h].  Per head: o = W_uv[head] O_lat
    (d_c -> d_v), then its slice of the group's first output projection:
    contribution = W_a[g][:, d_v*j : d_v*(j+1)] o with g = head // 8, j = head % 8.
    Returns [n, h, r_o].  Inverse output RoPE is the identity because the value stream is
    the non-rotated latent."""
    n, h, _ = O_lat.shape
    dv = w_uv.shape[1]
    ro = w_a.shape[1]
    out = np.empty((n, h, ro), dtype=np.float64)
    for a, head in enumerate(np.asarray(head_ids)):
        g, j = int(head) // group_size, int(head) % group_size
        o = O_lat[:, a, :] @ w_uv[head].T                       # [n, d_v]
        out[:, a, :] = o @ w_a[g][:, dv * j: dv * (j + 1)].T     # [n, r_o]
    return out


def _group_sum(contrib: np.ndarray, head_ids: np.ndarray, n_groups: int, group_size: int = 8):
    n, _, ro = contrib.shape
    z = np.zeros((n, n_groups, ro), dtype=np.float64)
    for a, head in enumerate(np.asarray(head_ids)):
        z[:, int(head) // group_size, :] += contrib[:, a, :]
    return z


def mla_online_rows(rows: np.ndarray, q_g_rows: np.ndarray, q_l_rows, kv: np.ndarray, seg_off, seg_delta,
                    prot_rows: np.ndarray, global_heads: np.ndarray, local_heads: np.ndarray,
                    w_uv: np.ndarray, w_a: np.ndarray, w_b: np.ndarray | None, z_off: np.ndarray,
                    sm_scale: float, base: float, d_latent: int, group_size: int = 8):
    """Expected MLA-Online result on the packed rows `rows` (any subset, ascending or not).

    q_g_rows [n, G, d_qk]: Global-head queries of those rows.
    q_l_rows: dict {packed row -> [L, d_qk]} (or array aligned with the protected ones among
    `rows`, in the order they appear) with the Local-head queries of the protected rows.
    Steps (Algorithm 2 after the merge; Eq. offonline; RestoreAndReplace: a protected row takes the
    online Local value in place of the artifact, the two are never added):
      O_G   = attention of the Global heads, every row
      O_L,A = attention of the Local heads, protected rows only
      z_on_g[t, g] = contribution of group g's Global head
      z_on_l[t, g] = sum of the contributions of group g's seven Local heads   (t in A)
      z[t] = z_on_g[t] + (z_on_l[t] if t in A else z_off[t]);  y[t] = W_b z[t]
    Returns a dict with O_g, lse_g, O_l, lse_l (protected rows of `rows`, in order), z_on_g,
    z_on_l, z, y, is_prot."""
    rows = np.asarray(rows, dtype=np.int64)
    T = int(np.asarray(seg_off)[-1])
    pos = request_positions(seg_off, seg_delta)
    k_req = keys_in_request_frame(kv, seg_off, seg_delta, d_latent, base)
    v = np.asarray(kv, dtype=np.float64)[:, :d_latent]
    G = len(global_heads)
    inv = inverse_row_map(prot_rows, T)
    is_prot = inv[rows] >= 0

    O_g, lse_g = attend_rows(q_g_rows, pos[rows], k_req, v, pos, sm_scale)
    c_g = head_contributions(O_g, global_heads, w_uv, w_a, group_size)
    z_on_g = _group_sum(c_g, global_heads, G, group_size)

    prot_sel = np.nonzero(is_prot)[0]
    if isinstance(q_l_rows, dict):
        ql = np.stack([q_l_rows[int(rows[i])] for i in prot_sel]) if len(prot_sel) else \
            np.zeros((0, len(local_heads), kv.shape[1]))
    else:
        ql = np.asarray(q_l_rows, dtype=np.float64)
    O_l, lse_l = attend_rows(ql, pos[rows[prot_sel]], k_req, v, pos, sm_scale)
    c_l = head_contributions(O_l, local_heads, w_uv, w_a, group_size)
    z_on_l = _group_sum(c_l, local_heads, G, group_size)

    ro = w_a.shape[1]
    z = z_on_g.copy()
    k = 0
    for i in range(len(rows)):
        if is_prot[i]:
            z[i] += z_on_l[k]
            k += 1
        else:
            z[i] += np.asarray(z_off[int(rows[i])], dtype=np.float64).reshape(G, ro)
    zf = z.reshape(len(rows), G * ro)
    y = zf @ np.asarray(w_b, dtype=np.float64).T if w_b is not None else None
    return dict(O_g=O_g, lse_g=lse_g, O_l=O_l, lse_l=lse_l, z_on_g=z_on_g, z_on_l=z_on_l,
                z=zf, y=y, is_prot=is_prot)


def full_recompute_rows(rows: np.ndarray, q_all_rows: np.ndarray, kv: np.ndarray, seg_off, seg_delta,
                        w_uv: np.ndarray, w_a: np.ndarray, w_b: np.ndarray, sm_scale: float, base: float,
                        d_latent: int, group_size: int = 8, heads: np.ndarray | None = None):
    """Full-head recomputation in the request context: every head (or the subset `heads`,
    absolute indices, with q_all_rows holding exactly those heads), one softmax per row,
    all eight slices of each group's W_a summed, then W_b.  Returns (z [n, G*r_o], y)."""
    rows = np.asarray(rows, dtype=np.int64)
    pos = request_positions(seg_off, seg_delta)
    k_req = keys_in_request_frame(kv, seg_off, seg_delta, d_latent, base)
    v = np.asarray(kv, dtype=np.float64)[:, :d_latent]
    H = w_uv.shape[0]
    heads = np.arange(H) if heads is None else np.asarray(heads)
    O, _ = attend_rows(q_all_rows, pos[rows], k_req, v, pos, sm_scale)
    c = head_contributions(O, heads, w_uv, w_a, group_size)
    G = w_a.shape[0]
    z = _group_sum(c, heads, G, group_size).reshape(len(rows), -1)
    y = z @ np.asarray(w_b, dtype=np.float64).T if w_b is not None else None
    return z, y


def mla_off_artifact(seg: int, q_local_doc: np.ndarray, kv: np.ndarray, seg_off, seg_delta,
                     local_heads: np.ndarray, w_uv: np.ndarray, w_a: np.ndarray, sm_scale: float,
                     base: float, d_latent: int, group_size: int = 8, rows: np.ndarray | None = None) -> np.ndarray:
    """Algorithm 1 for one document: the document alone at positions 0..n-1, causal over its
    own keys only, Local heads only, z_off = W_{a,L} O_L.  q_local_doc [n, L, d_qk] are the
    request-position queries of the document's rows; the query the document had at
    position zero is R(-delta_i) of that.  Returns [n, G*r_o].  With `rows` (canonical indices
    inside the document) only those rows are evaluated and q_local_doc holds just their queries."""
    lo, hi = int(seg_off[seg]), int(seg_off[seg + 1])
    n = hi - lo
    q0 = np.asarray(q_local_doc, dtype=np.float64).copy()
    q0[..., d_latent:] = relocate_query(q0[..., d_latent:], float(seg_delta[seg]), base)
    kd = np.asarray(kv, dtype=np.float64)[lo:hi]
    canon = np.arange(n, dtype=np.int64)
    row_canon = canon if rows is None else np.asarray(rows, dtype=np.int64)
    O, _ = attend_rows(q0, row_canon, kd, kd[:, :d_latent], canon, sm_scale)
    c = head_contributions(O, local_heads, w_uv, w_a, group_size)
    return _group_sum(c, local_heads, w_a.shape[0], group_size).reshape(len(row_canon), -1)


# ---------------------------------------------------------------------------------
# profile arithmetic the paper prints
# ---------------------------------------------------------------------------------

def head_row_ceiling(n_reusable_layers: int, n_layers: int, n_local: int, n_heads: int) -> float:
    """Eq. ceiling: S = (N_R / N) (|L| / H)."""
    return (n_reusable_layers / n_layers) * (n_local / n_heads)


def cold_speed_ratio(s_hot: float, build_units: float = 0.75) -> float:
    """Planning model of the cold-artifact panel: S_cold = 1 / (0.75 + 1 / S_hot)."""
    return 1.0 / (build_units + 1.0 / s_hot)


def reuse_error_report(y_online: np.ndarray, y_full: np.ndarray, is_prot: np.ndarray) -> dict:
    """Relative L2 distance between MLA-Online and full recomputation, split by protected /
    unprotected rows (a report, not a check).  The arithmetic is pinned by a closed form on hand-made
    vectors; the quantity it reports on random data has no counterpart in the paper (which measures
    reuse quality through model-level F1 / EM only), so no expected value exists for it."""
    def rel(a, b):
        d = np.linalg.norm(b)
        return float(np.linalg.norm(a - b) / d) if d > 0 else 0.0
    return dict(protected=rel(y_online[is_prot], y_full[is_prot]) if is_prot.any() else 0.0,
                unprotected=rel(y_online[~is_prot], y_full[~is_prot]) if (~is_prot).any() else 0.0)
