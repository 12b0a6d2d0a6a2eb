"""Plain float64 definition of the output-phase variant of one MLA-Online layer (numpy only).

Test infrastructure, not product code: slow on purpose, no blocking / fusion / reordering
beyond what each cited passage states.  Shares no code with the CUDA library.

The variant.  Section "Logical heads, one physical latent" writes both projected states with
an inverse output RoPE, z = W_a R^{-1}(O) (Eq. offonline), and Algorithm 2 restores the output
phase of every segment's partial result (RestorePhase(O_i, delta_i)) before SegmentedLSEMerge
and applies R^{-1} once more in its z_online statement.  Those maps act on something only when
the value stream itself carries rotated dimensions.  Reading taken here (the paper gives no
tensor widths): the packed row [c | r] is key AND value -- the 64 rope dims r_k, stored rotated
at the document's canonical position p_k like the key's, are part of the value -- so

    O[t, h]   = sum_k softmax_k( sm_scale <q[t,h], K_req[k]> )  V_req[k],   V_req = K_req
    K_req[k]  = [ c_k | R(delta_seg(k)) r_k ]                        (request frame, Eq. rope)
    R^{-1}    : rope dims of O[t, h] turned by R(-pos[t])            (before W_uv / W_a)

After R^{-1} the rope dims of the output are sum_k p_k R(pos[k] - pos[t]) r_k^raw: they depend on
relative positions only, which is what lets a document built at position zero be reused
elsewhere.  W_uv[h] is [d_v x (d_c + d_r)] here (it takes the wider value).

Algorithm 2's own order of evaluation (`attend_rows_segmentwise_phase`): per segment rotate the
query by -delta_i, attend the canonical stored rows (their rope dims in the document's frame),
RestorePhase = turn the partial output's rope dims by R(+delta_i) into the request frame, merge
the partials with the stable log-sum-exp rule, then R^{-1} per row.  The pins
(tests/test_oracle_phase_pins.py) tie the plain definition to that order, to a scalar brute
force, to the relative-position closed form built from raw (unrotated) vectors, to the
existing path when r = 0, to shift invariance and to the exact factorization.
"""
from __future__ import annotations

import numpy as np

from .mla_online import (attend_rows, inverse_row_map, keys_in_request_frame, relocate_query,
                         request_positions, rope_rotate, segmented_merge)

__all__ = [
    "inverse_output_rope", "restore_phase", "attend_rows_phase", "attend_rows_segmentwise_phase",
    "head_contributions_phase", "mla_online_rows_phase", "full_recompute_rows_phase",
    "mla_off_artifact_phase", "segmented_merge_phase",
]


def inverse_output_rope(O: np.ndarray, row_pos: np.ndarray, d_latent: int, base: float) -> np.ndarray:
    """R^{-1} of Eq. offonline: the rope dims of every row's output turned by R(-pos[row]).
    O [n, h, d_c + d_r], row_pos [n]."""
    O = np.asarray(O, dtype=np.float64)
    out = O.copy()
    p = -np.asarray(row_pos, dtype=np.float64)[:, None]          # broadcast over heads
    out[..., d_latent:] = rope_rotate(O[..., d_latent:], p, base)
    return out


def restore_phase(O_part: np.ndarray, delta, d_latent: int, base: float) -> np.ndarray:
    """RestorePhase(O_i, delta_i) of Algorithm 2: a partial output computed against the canonical
    rows of document i has its rope dims in the document's position-zero frame; turning them by
    R(+delta_i) puts them into the request frame, where partial results of different segments
    may be added."""
    O_part = np.asarray(O_part, dtype=np.float64)
    out = O_part.copy()
    out[..., d_latent:] = rope_rotate(O_part[..., d_latent:], float(delta), base)
    return out


def attend_rows_phase(q: np.ndarray, row_pos: np.ndarray, kv: np.ndarray, seg_off, seg_delta, d_latent: int,
                      base: float, sm_scale: float):
    """Plain definition: keys and values both turned to request positions, one softmax per
    (row, head), then R^{-1}.  q [n, h, d_qk] at request positions, row_pos [n].
    Returns O [n, h, d_qk] (rope dims already passed through R^{-1}) and lse [n, h]."""
    pos = request_positions(seg_off, seg_delta)
    kv_req = keys_in_request_frame(kv, seg_off, seg_delta, d_latent, base)
    O, lse = attend_rows(q, row_pos, kv_req, kv_req, pos, sm_scale)
    return inverse_output_rope(O, row_pos, d_latent, base), lse


def attend_rows_segmentwise_phase(q: np.ndarray, row_pos: np.ndarray, kv: np.ndarray, seg_off, seg_delta,
                                  d_latent: int, base: float, sm_scale: float):
    """Algorithm 2's order: for each segment q_i = R(-delta_i) q, SelectiveMLA against the
    canonical rows (value = the stored row, rope dims in the document's frame),
    RestorePhase(+delta_i), SegmentedLSEMerge, and R^{-1} before the projection."""
    q = np.asarray(q, dtype=np.float64)
    kv = np.asarray(kv, dtype=np.float64)
    Op, Lp = [], []
    for i in range(len(seg_delta)):
        lo, hi = int(seg_off[i]), int(seg_off[i + 1])
        qi = q.copy()
        qi[..., d_latent:] = relocate_query(q[..., d_latent:], float(seg_delta[i]), base)
        canon = np.arange(hi - lo, dtype=np.int64)
        O_i, l_i = attend_rows(qi, np.asarray(row_pos) - int(seg_delta[i]), kv[lo:hi], kv[lo:hi], canon, sm_scale)
        Op.append(restore_phase(O_i, seg_delta[i], d_latent, base))
        Lp.append(l_i)
    O, lse = segmented_merge(np.stack(Op), np.stack(Lp))
    return inverse_output_rope(O, row_pos, d_latent, base), lse


def segmented_merge_phase(O_parts: np.ndarray, lse_parts: np.ndarray, part_delta, row_pos, d_latent: int,
                          base: float):
    """Standalone form: parts j are per-segment partial results with rope dims in their own
    document frames; RestorePhase(+part_delta[j]) on each, the stable merge, then (row_pos given)
    R^{-1} per row.  O_parts [P, n, h, d_c + d_r], lse_parts [P, n, h].  A part with lse = -inf is
    ignored even when its O is not finite."""
    O_parts = np.asarray(O_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    safe = np.where(np.isfinite(lse_parts)[..., None], O_parts, 0.0)
    restored = np.stack([restore_phase(safe[j], part_delta[j], d_latent, base) for j in range(len(part_delta))])
    O, lse = segmented_merge(restored, lse_parts)
    if row_pos is not None:
        O = inverse_output_rope(O, row_pos, d_latent, base)
    return O, lse


def head_contributions_phase(O: np.ndarray, head_ids: np.ndarray, w_uv: np.ndarray, w_a: np.ndarray,
                             group_size: int = 8) -> np.ndarray:
    """O [n, h, d_c + d_r] AFTER R^{-1}, for absolute heads head_ids.  Per head o = W_uv[head] O
    (W_uv[head] is [d_v, d_c + d_r]), then the head's d_v-column slice of its group's W_a
    (Eq. offonline).  Returns [n, h, r_o]."""
    n, h, _ = O.shape
    dv = w_uv.shape[1]
    out = np.empty((n, h, w_a.shape[1]), dtype=np.float64)
    for a, head in enumerate(np.asarray(head_ids)):
        g, j = int(head) // group_size, int(head) % group_size
        o = O[:, a, :] @ w_uv[head].T
        out[:, a, :] = o @ w_a[g][:, dv * j: dv * (j + 1)].T
    return out


def _group_sum(contrib, head_ids, n_groups, group_size=8):
    n, _, ro = contrib.shape
    z = np.zeros((n, n_groups, ro), dtype=np.float64)
    for a, head in enumerate(np.asarray(head_ids)):
        z[:, int(head) // group_size, :] += contrib[:, a, :]
    return z


def mla_online_rows_phase(rows, q_g_rows, q_l_rows, kv, seg_off, seg_delta, prot_rows, global_heads, local_heads,
                          w_uv, w_a, w_b, z_off, sm_scale: float, base: float, d_latent: int, group_size: int = 8):
    """Expected MLA-Online result of the variant on packed rows `rows` (arguments as in
    `mla_online_rows`; W_uv is [H, d_v, d_c + d_r]).  Steps (Algorithm 2 after the merge):
    Global heads on every row, Local heads on protected rows, R^{-1}, sliced W_a, select
    z_on_l on protected rows / z_off elsewhere (never both), W_b."""
    rows = np.asarray(rows, dtype=np.int64)
    T = int(np.asarray(seg_off)[-1])
    pos = request_positions(seg_off, seg_delta)
    G = len(global_heads)
    inv = inverse_row_map(prot_rows, T)
    is_prot = inv[rows] >= 0

    O_g, lse_g = attend_rows_phase(q_g_rows, pos[rows], kv, seg_off, seg_delta, d_latent, base, sm_scale)
    z_on_g = _group_sum(head_contributions_phase(O_g, global_heads, w_uv, w_a, group_size), global_heads, G, group_size)

    prot_sel = np.nonzero(is_prot)[0]
    if isinstance(q_l_rows, dict):
        ql = np.stack([q_l_rows[int(rows[i])] for i in prot_sel]) if len(prot_sel) else \
            np.zeros((0, len(local_heads), np.asarray(kv).shape[1]))
    else:
        ql = np.asarray(q_l_rows, dtype=np.float64)
    O_l, lse_l = attend_rows_phase(ql, pos[rows[prot_sel]], kv, seg_off, seg_delta, d_latent, base, sm_scale)
    z_on_l = _group_sum(head_contributions_phase(O_l, local_heads, w_uv, w_a, group_size), local_heads, G, group_size)

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
    return dict(O_g=O_g, lse_g=lse_g, O_l=O_l, lse_l=lse_l, z_on_g=z_on_g, z_on_l=z_on_l, z=zf, y=y,
                is_prot=is_prot)


def full_recompute_rows_phase(rows, q_all_rows, kv, seg_off, seg_delta, w_uv, w_a, w_b, sm_scale: float, base: float,
                              d_latent: int, group_size: int = 8, heads=None):
    """Every head (or the subset `heads`) recomputed in the request context, all slices of each
    group's W_a summed, then W_b.  Returns (z [n, G*r_o], y)."""
    rows = np.asarray(rows, dtype=np.int64)
    pos = request_positions(seg_off, seg_delta)
    heads = np.arange(w_uv.shape[0]) if heads is None else np.asarray(heads)
    O, _ = attend_rows_phase(q_all_rows, pos[rows], kv, seg_off, seg_delta, d_latent, base, sm_scale)
    c = head_contributions_phase(O, heads, w_uv, w_a, group_size)
    z = _group_sum(c, heads, w_a.shape[0], group_size).reshape(len(rows), -1)
    y = z @ np.asarray(w_b, dtype=np.float64).T if w_b is not None else None
    return z, y


def mla_off_artifact_phase(seg: int, q_local_doc, kv, seg_off, seg_delta, local_heads, w_uv, w_a, sm_scale: float,
                           base: float, d_latent: int, group_size: int = 8, rows=None) -> np.ndarray:
    """Algorithm 1 in the variant: the document alone at positions 0..n-1 (keys and values as
    stored), Local heads, z_off = W_{a,L} R^{-1}(O_L) with R^{-1} at the canonical position.
    q_local_doc holds the request-position queries of the document's rows (or of `rows`,
    canonical indices); the query the document had at position zero is R(-delta_i) of that."""
    lo, hi = int(seg_off[seg]), int(seg_off[seg + 1])
    q0 = np.asarray(q_local_doc, dtype=np.float64).copy()
    q0[..., d_latent:] = relocate_query(q0[..., d_latent:], float(seg_delta[seg]), base)
    kd = np.asarray(kv, dtype=np.float64)[lo:hi]
    canon = np.arange(hi - lo, dtype=np.int64)
    row_canon = canon if rows is None else np.asarray(rows, dtype=np.int64)
    O, _ = attend_rows(q0, row_canon, kd, kd, canon, sm_scale)
    O = inverse_output_rope(O, row_canon, d_latent, base)
    c = head_contributions_phase(O, local_heads, w_uv, w_a, group_size)
    return _group_sum(c, local_heads, w_a.shape[0], group_size).reshape(len(row_canon), -1)
