"""Pins for the output-phase variant of the float64 checker (oracle/phase.py): RestorePhase per
segment and the inverse output RoPE R^{-1} before the first projection (Eq. offonline;
Algorithm 2).  Each test ties the plain definition to something other than itself: Algorithm 2's
own order of evaluation, a relative-position closed form built from raw vectors with complex
arithmetic, a scalar brute force, the existing path when the value's rope dims are zero,
invariances, the exact factorization, and a library routine.  CPU only."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import brute, phase

from test_oracle_pins import rel, small_problem


def phase_problem(seed, **kw):
    """The toy of the other pins with W_uv widened to take the whole stored row as the value."""
    p = small_problem(seed, **kw)
    rng = np.random.default_rng(1000 + seed)
    p["w_uv"] = rng.normal(size=(p["H"], p["d_v"], p["d_c"] + p["d_r"])) * 0.3
    return p


def online(p, rows=None, z_off=None, prot=None):
    rows = np.arange(p["T"]) if rows is None else np.asarray(rows)
    prot = p["prot"] if prot is None else prot
    z_off = p["z_off"] if z_off is None else z_off
    ql = {int(r): p["q_all"][r][p["lh"]] for r in prot}
    return phase.mla_online_rows_phase(rows, p["q_all"][rows][:, p["gh"]], ql, p["kv"], p["seg_off"], p["seg_delta"],
                                       prot, p["gh"], p["lh"], p["w_uv"], p["w_a"], p["w_b"], z_off, p["sm_scale"],
                                       p["base"], p["d_c"])


def full(p, rows=None):
    rows = np.arange(p["T"]) if rows is None else np.asarray(rows)
    return phase.full_recompute_rows_phase(rows, p["q_all"][rows], p["kv"], p["seg_off"], p["seg_delta"], p["w_uv"],
                                           p["w_a"], p["w_b"], p["sm_scale"], p["base"], p["d_c"])


# -- Algorithm 2's order == plain definition --------------------------------------------------------

@pytest.mark.parametrize("seed", [0, 3, 8])
def test_segmentwise_restore_phase_then_merge_equals_plain_definition(seed):
    """q_i = R(-delta_i) q, canonical rows as keys and values, RestorePhase(+delta_i), merge, R^{-1}
    gives the one-softmax result with keys and values at request positions."""
    p = phase_problem(seed)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    O1, l1 = phase.attend_rows_phase(p["q_all"], pos, p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"],
                                     p["sm_scale"])
    O2, l2 = phase.attend_rows_segmentwise_phase(p["q_all"], pos, p["kv"], p["seg_off"], p["seg_delta"], p["d_c"],
                                                 p["base"], p["sm_scale"])
    assert rel(O2, O1) < 1e-12
    assert np.max(np.abs(l2 - l1)) < 1e-12
    # the phase matters: leaving RestorePhase out changes the rope dims of the result
    Op, Lp = [], []
    for i in range(len(p["seg_delta"])):
        lo, hi = int(p["seg_off"][i]), int(p["seg_off"][i + 1])
        qi = p["q_all"].copy()
        qi[..., p["d_c"]:] = oracle.relocate_query(qi[..., p["d_c"]:], float(p["seg_delta"][i]), p["base"])
        a, b = oracle.attend_rows(qi, pos - int(p["seg_delta"][i]), p["kv"][lo:hi], p["kv"][lo:hi],
                                  np.arange(hi - lo), p["sm_scale"])
        Op.append(a)
        Lp.append(b)
    O3, _ = oracle.segmented_merge(np.stack(Op), np.stack(Lp))
    O3 = phase.inverse_output_rope(O3, pos, p["d_c"], p["base"])
    assert rel(O3[..., :p["d_c"]], O1[..., :p["d_c"]]) < 1e-12           # latent dims carry no phase
    assert rel(O3[..., p["d_c"]:], O1[..., p["d_c"]:]) > 1e-2


def test_standalone_merge_with_part_phases():
    """segmented_merge_phase on per-segment partials (rope dims in each document's frame) equals
    the plain definition; an empty part with garbage O is ignored."""
    p = phase_problem(5)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    O1, l1 = phase.attend_rows_phase(p["q_all"], pos, p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"],
                                     p["sm_scale"])
    Op, Lp = [], []
    for i in range(len(p["seg_delta"])):
        lo, hi = int(p["seg_off"][i]), int(p["seg_off"][i + 1])
        qi = p["q_all"].copy()
        qi[..., p["d_c"]:] = oracle.relocate_query(qi[..., p["d_c"]:], float(p["seg_delta"][i]), p["base"])
        a, b = oracle.attend_rows(qi, pos - int(p["seg_delta"][i]), p["kv"][lo:hi], p["kv"][lo:hi],
                                  np.arange(hi - lo), p["sm_scale"])
        a[np.isneginf(b)] = np.nan
        Op.append(a)
        Lp.append(b)
    assert np.isnan(np.stack(Op)).any()                                   # some rows see nothing of some segment
    O2, l2 = phase.segmented_merge_phase(np.stack(Op), np.stack(Lp), p["seg_delta"], pos, p["d_c"], p["base"])
    assert rel(O2, O1) < 1e-12 and np.max(np.abs(l2 - l1)) < 1e-12
    # without row positions the result stays in the request frame
    O3, _ = phase.segmented_merge_phase(np.stack(Op), np.stack(Lp), p["seg_delta"], None, p["d_c"], p["base"])
    assert rel(phase.inverse_output_rope(O3, pos, p["d_c"], p["base"]), O1) < 1e-12


# -- relative-position closed form from raw vectors (complex arithmetic) ------------------------------

def test_restored_output_depends_on_relative_positions_only():
    """With raw (unrotated) rope vectors r_k and q_t, stored r = R(p_k) r_k and given q = R(pos_t) q_t:
    score = sm_scale (q_c.c_k + Re sum_j conj(.)...) is a function of pos_t - pos_k, and the restored
    rope dims are sum_k p_k R(pos_k - pos_t) r_k.  Evaluated here with complex numbers."""
    rng = np.random.default_rng(21)
    d_c, d_r, base = 6, 8, 10000.0
    seg_off = np.array([0, 4, 9, 12])
    seg_delta = np.array([5, 0, 9])                                       # document 1 is first, then 0, then the suffix
    T = 12
    pos = oracle.request_positions(seg_off, seg_delta)
    canon = np.concatenate([np.arange(4), np.arange(5), np.arange(3)])
    theta = base ** (-2.0 * np.arange(d_r // 2) / d_r)
    c = rng.normal(size=(T, d_c))
    r_raw = rng.normal(size=(T, d_r // 2)) + 1j * rng.normal(size=(T, d_r // 2))
    q_c = rng.normal(size=(T, 1, d_c))
    q_raw = rng.normal(size=(T, d_r // 2)) + 1j * rng.normal(size=(T, d_r // 2))
    # what the library is given: keys rotated at canonical positions, queries at request positions
    r_st = r_raw * np.exp(1j * canon[:, None] * theta)
    q_st = q_raw * np.exp(1j * pos[:, None] * theta)
    kv = np.concatenate([c, np.stack([r_st.real, r_st.imag], -1).reshape(T, d_r)], axis=1)
    q = np.concatenate([q_c, np.stack([q_st.real, q_st.imag], -1).reshape(T, 1, d_r)], axis=2)
    sm = 0.37
    O, lse = phase.attend_rows_phase(q, pos, kv, seg_off, seg_delta, d_c, base, sm)
    for t in range(T):
        vis = np.nonzero(pos <= pos[t])[0]
        rel_rot = np.exp(1j * (pos[vis] - pos[t])[:, None] * theta)         # R(pos_k - pos_t)
        s = sm * (c[vis] @ q_c[t, 0] + np.real(np.conj(q_raw[t])[None, :] * r_raw[vis] * rel_rot).sum(axis=1))
        w = np.exp(s - s.max())
        w /= w.sum()
        want_c = w @ c[vis]
        want_r = (w[:, None] * r_raw[vis] * rel_rot).sum(axis=0)
        assert np.allclose(O[t, 0, :d_c], want_c, atol=1e-12)
        assert np.allclose(O[t, 0, d_c::2], want_r.real, atol=1e-12)
        assert np.allclose(O[t, 0, d_c + 1::2], want_r.imag, atol=1e-12)
        assert abs(lse[t, 0] - (s.max() + math.log(np.exp(s - s.max()).sum()))) < 1e-12


# -- scalar brute force -------------------------------------------------------------------------------

def test_scalar_brute_force_phase():
    p = phase_problem(11, doc_lens=(5, 6), n_q=3, d_c=8, d_r=4, d_v=4, r_o=3, d_model=5)
    b = brute.brute_layer_phase(p["q_all"].tolist(), p["kv"].tolist(), p["seg_off"], p["seg_delta"], p["prot"], p["gh"],
                                p["w_uv"].tolist(), p["w_a"].tolist(), p["w_b"].tolist(), p["z_off"].tolist(),
                                p["sm_scale"], p["base"], p["d_c"])
    out = online(p)
    _, y_full = full(p)
    assert rel(out["z"], np.array(b["z"])) < 1e-12
    assert rel(out["y"], np.array(b["y"])) < 1e-12
    assert rel(y_full, np.array(b["y_full"])) < 1e-12
    for t in range(p["T"]):
        for a, h in enumerate(p["gh"]):
            assert abs(out["lse_g"][t, a] - b["lse"][t][h]) < 1e-12
            assert np.allclose(out["O_g"][t, a, p["d_c"]:], b["o_rope"][t][h], atol=1e-12)
    for k, t in enumerate(p["prot"]):
        for a, h in enumerate(p["lh"]):
            assert np.allclose(out["O_l"][k, a, p["d_c"]:], b["o_rope"][t][h], atol=1e-12)


# -- reduces to the existing path -----------------------------------------------------------------------

def test_zero_value_columns_reduce_to_latent_only_path():
    """When W_uv ignores the rope dims (their columns are zero) the variant's z and y equal those of
    the latent-only path with the 512-wide W_uv: the phase maps then act on nothing that is used."""
    p = phase_problem(12)
    w_narrow = p["w_uv"][:, :, :p["d_c"]].copy()
    p["w_uv"][:, :, p["d_c"]:] = 0.0
    out = online(p)
    ql = {int(r): p["q_all"][r][p["lh"]] for r in p["prot"]}
    ref = oracle.mla_online_rows(np.arange(p["T"]), p["q_all"][:, p["gh"]], ql, p["kv"], p["seg_off"], p["seg_delta"],
                                 p["prot"], p["gh"], p["lh"], w_narrow, p["w_a"], p["w_b"], p["z_off"], p["sm_scale"],
                                 p["base"], p["d_c"])
    assert rel(out["y"], ref["y"]) < 1e-12
    assert rel(out["O_g"][..., :p["d_c"]], ref["O_g"]) < 1e-12 and np.max(np.abs(out["lse_g"] - ref["lse_g"])) < 1e-12


# -- invariances ----------------------------------------------------------------------------------------

def test_global_shift_invariance_of_restored_output():
    """Adding a constant to every delta_i (and re-rotating the given queries) changes nothing:
    after R^{-1} only relative positions are left."""
    p = phase_problem(16)
    out = online(p)
    shift = 977
    p2 = dict(p)
    p2["seg_delta"] = p["seg_delta"] + shift
    q2 = p["q_all"].copy()
    q2[..., p["d_c"]:] = oracle.rope_rotate(p["q_all"][..., p["d_c"]:], shift, p["base"])
    p2["q_all"] = q2
    out2 = online(p2)
    assert rel(out2["y"], out["y"]) < 1e-10
    assert rel(out2["O_g"], out["O_g"]) < 1e-10
    # without R^{-1} the rope dims would move with the shift
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    kvr = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    kvr2 = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p2["seg_delta"], p["d_c"], p["base"])
    A, _ = oracle.attend_rows(p["q_all"][:, p["gh"]], pos, kvr, kvr, pos, p["sm_scale"])
    B, _ = oracle.attend_rows(q2[:, p["gh"]], pos + shift, kvr2, kvr2, pos + shift, p["sm_scale"])
    assert rel(B[..., p["d_c"]:], A[..., p["d_c"]:]) > 1e-2


def test_factorization_and_prefix_exactness():
    """Eq. factorization in the variant: Local contribution computed in the request context +
    Global online = full recomputation; and the honest position-zero artifact of the document placed
    first equals its request-context Local contribution (its rows are exact without protection)."""
    p = phase_problem(2)
    rows = np.arange(p["T"])
    z_loc, _ = phase.full_recompute_rows_phase(rows, p["q_all"][:, p["lh"]], p["kv"], p["seg_off"], p["seg_delta"],
                                               p["w_uv"], p["w_a"], None, p["sm_scale"], p["base"], p["d_c"],
                                               heads=p["lh"])
    out = online(p, z_off=z_loc[:p["N_doc"]])
    z_full, y_full = full(p)
    assert rel(out["z"], z_full) < 1e-12 and rel(out["y"], y_full) < 1e-12
    D = len(p["seg_delta"]) - 1
    z_off = np.zeros_like(p["z_off"])
    for i in range(D):
        lo, hi = p["seg_off"][i], p["seg_off"][i + 1]
        z_off[lo:hi] = phase.mla_off_artifact_phase(i, p["q_all"][lo:hi][:, p["lh"]], p["kv"], p["seg_off"],
                                                    p["seg_delta"], p["lh"], p["w_uv"], p["w_a"], p["sm_scale"],
                                                    p["base"], p["d_c"])
    out = online(p, z_off=z_off)
    first = int(np.argmin(p["seg_delta"][:D]))
    lo, hi = p["seg_off"][first], p["seg_off"][first + 1]
    assert rel(out["y"][lo:hi], y_full[lo:hi]) < 1e-12
    assert rel(out["y"][out["is_prot"]], y_full[out["is_prot"]]) < 1e-12
    # a document that is NOT first but has no visible predecessor's influence removed would differ
    others = np.ones(p["T"], bool)
    others[lo:hi] = False
    others &= ~out["is_prot"]
    assert rel(out["y"][others], y_full[others]) > 1e-3
    # the rows= form of the artifact equals the same rows of the whole-document call
    i = (first + 1) % D
    lo, hi = p["seg_off"][i], p["seg_off"][i + 1]
    pick = np.array([0, 2, hi - lo - 1])
    part = phase.mla_off_artifact_phase(i, p["q_all"][lo:hi][pick][:, p["lh"]], p["kv"], p["seg_off"], p["seg_delta"],
                                        p["lh"], p["w_uv"], p["w_a"], p["sm_scale"], p["base"], p["d_c"], rows=pick)
    assert np.allclose(part, z_off[lo:hi][pick], atol=1e-13)


# -- closed form and library routine ---------------------------------------------------------------------

def test_zero_query_running_mean_of_request_frame_values():
    """q = 0: every visible key has weight 1/(pos+1), so the output before R^{-1} is the running mean
    of the request-frame rows in position order; R^{-1} then turns its rope dims by -pos."""
    p = phase_problem(13)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    q0 = np.zeros((p["T"], 1, p["d_c"] + p["d_r"]))
    O, lse = phase.attend_rows_phase(q0, pos, p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"], p["sm_scale"])
    order = np.argsort(pos)
    theta = p["base"] ** (-2.0 * np.arange(p["d_r"] // 2) / p["d_r"])
    seg = oracle.segment_of_rows(p["seg_off"])
    z = (p["kv"][:, p["d_c"]::2] + 1j * p["kv"][:, p["d_c"] + 1::2]) * np.exp(1j * p["seg_delta"][seg][:, None] * theta)
    cm_c = np.cumsum(p["kv"][order, :p["d_c"]], axis=0) / (np.arange(p["T"]) + 1)[:, None]
    cm_r = np.cumsum(z[order], axis=0) / (np.arange(p["T"]) + 1)[:, None]
    for t in range(p["T"]):
        want = cm_r[pos[t]] * np.exp(-1j * pos[t] * theta)
        assert np.allclose(O[t, 0, :p["d_c"]], cm_c[pos[t]], atol=1e-13)
        assert np.allclose(O[t, 0, p["d_c"]::2], want.real, atol=1e-13)
        assert np.allclose(O[t, 0, p["d_c"] + 1::2], want.imag, atol=1e-13)
        assert abs(lse[t, 0] - math.log(pos[t] + 1)) < 1e-13


def test_torch_sdpa_float64_with_shared_key_value():
    p = phase_problem(17)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    kvr = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    O, _ = phase.attend_rows_phase(p["q_all"], pos, p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"],
                                   p["sm_scale"])
    q_t = torch.from_numpy(p["q_all"]).permute(1, 0, 2)[None]
    kv_t = torch.from_numpy(kvr)[None, None].expand(1, p["H"], -1, -1)
    mask = torch.from_numpy(pos[None, :] <= pos[:, None])
    ref = torch.nn.functional.scaled_dot_product_attention(q_t, kv_t, kv_t, attn_mask=mask, scale=p["sm_scale"])
    ref = ref[0].permute(1, 0, 2).numpy().copy()
    # R^{-1} by complex multiplication
    theta = p["base"] ** (-2.0 * np.arange(p["d_r"] // 2) / p["d_r"])
    zr = (ref[..., p["d_c"]::2] + 1j * ref[..., p["d_c"] + 1::2]) * np.exp(-1j * pos[:, None, None] * theta)
    ref[..., p["d_c"]::2], ref[..., p["d_c"] + 1::2] = zr.real, zr.imag
    assert rel(O, ref) < 1e-12


# -- the rows= branch of the latent-only artifact builder (Algorithm 1) -----------------------------------

def test_mla_off_artifact_rows_branch_equals_whole_document_and_brute_force():
    p = small_problem(23, doc_lens=(6, 5), n_q=2, d_c=8, d_r=4, d_v=4, r_o=3, d_model=5)
    for i in range(2):
        lo, hi = int(p["seg_off"][i]), int(p["seg_off"][i + 1])
        whole = oracle.mla_off_artifact(i, p["q_all"][lo:hi][:, p["lh"]], p["kv"], p["seg_off"], p["seg_delta"],
                                        p["lh"], p["w_uv"], p["w_a"], p["sm_scale"], p["base"], p["d_c"])
        pick = np.array([hi - lo - 1, 0, 3])                              # any order
        part = oracle.mla_off_artifact(i, p["q_all"][lo:hi][pick][:, p["lh"]], p["kv"], p["seg_off"], p["seg_delta"],
                                       p["lh"], p["w_uv"], p["w_a"], p["sm_scale"], p["base"], p["d_c"], rows=pick)
        assert np.allclose(part, whole[pick], atol=1e-13)
        # brute force: the document alone as a one-segment request at offset 0, nothing protected, z_off = 0:
        # the Local part of its full recomputation is the artifact
        n = hi - lo
        q0 = p["q_all"][lo:hi].copy()
        q0[..., p["d_c"]:] = oracle.rope_rotate(q0[..., p["d_c"]:], -float(p["seg_delta"][i]), p["base"])
        w_a_loc = p["w_a"].copy()
        for g, h in enumerate(p["gh"]):
            j = int(h) % 8
            w_a_loc[g][:, p["d_v"] * j: p["d_v"] * (j + 1)] = 0.0          # drop the Global slices
        b = brute.brute_layer(q0.tolist(), p["kv"][lo:hi].tolist(), np.array([0, n]), np.array([0]), np.arange(n),
                              p["gh"], p["w_uv"].tolist(), w_a_loc.tolist(), np.eye(p["G"] * p["r_o"]).tolist(),
                              np.zeros((n, p["G"] * p["r_o"])).tolist(), p["sm_scale"], p["base"], p["d_c"])
        assert rel(whole, np.array(b["y_full"])) < 1e-12
