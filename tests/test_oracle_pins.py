"""Pins for the float64 checker: each test ties it to something other than itself --
an identity the paper states, a closed form, a brute force, a library routine, or a value
the paper prints.  A dropped term, wrong sign, wrong index or transposed operand in
oracle/ fails at least one of these.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import brute


def small_problem(seed, doc_lens=(5, 7, 6), n_q=3, H=16, G=2, d_c=16, d_r=8, d_v=4, r_o=6, d_model=10,
                  shuffle=True, prot_extra=4, base=10000.0):
    """float64 toy with the paper's structure (several documents at shuffled request
    offsets, a query suffix, one Global head per group of eight at a random slot)."""
    rng = np.random.default_rng(seed)
    D = len(doc_lens)
    order = rng.permutation(D) if shuffle else np.arange(D)
    delta = np.zeros(D + 1, dtype=np.int64)
    run = 0
    for d in order:
        delta[d] = run
        run += doc_lens[d]
    delta[D] = run
    seg_off = np.concatenate([[0], np.cumsum(list(doc_lens) + [n_q])]).astype(np.int64)
    T = int(seg_off[-1])
    N_doc = int(seg_off[D])
    gh = (8 * np.arange(G) + rng.integers(0, 8, size=G)).astype(np.int64)
    lh = np.array([h for h in range(H) if h not in set(gh.tolist())], dtype=np.int64)
    prot = np.unique(np.concatenate([rng.choice(N_doc, size=prot_extra, replace=False),
                                     np.arange(N_doc, T)])).astype(np.int64)
    p = dict(
        seg_off=seg_off, seg_delta=delta, T=T, N_doc=N_doc, gh=gh, lh=lh, prot=prot, H=H, G=G,
        d_c=d_c, d_r=d_r, d_v=d_v, r_o=r_o, d_model=d_model, base=base,
        sm_scale=1.0 / math.sqrt(d_v + d_r),
        kv=rng.normal(size=(T, d_c + d_r)),
        q_all=rng.normal(size=(T, H, d_c + d_r)) * 1.3,
        w_uv=rng.normal(size=(H, d_v, d_c)) * 0.3,
        w_a=rng.normal(size=(G, r_o, 8 * d_v)) * 0.3,
        w_b=rng.normal(size=(d_model, G * r_o)) * 0.3,
        z_off=rng.normal(size=(N_doc, G * r_o)),
    )
    return p


def online(p, rows=None, z_off=None, prot=None):
    rows = np.arange(p["T"]) if rows is None else np.asarray(rows)
    prot = p["prot"] if prot is None else prot
    z_off = p["z_off"] if z_off is None else z_off
    ql = {int(r): p["q_all"][r][p["lh"]] for r in prot}
    return oracle.mla_online_rows(rows, p["q_all"][rows][:, p["gh"]], ql, p["kv"], p["seg_off"], p["seg_delta"],
                                  prot, p["gh"], p["lh"], p["w_uv"], p["w_a"], p["w_b"], z_off,
                                  p["sm_scale"], p["base"], p["d_c"])


def full(p, rows=None):
    rows = np.arange(p["T"]) if rows is None else np.asarray(rows)
    return oracle.full_recompute_rows(rows, p["q_all"][rows], p["kv"], p["seg_off"], p["seg_delta"],
                                      p["w_uv"], p["w_a"], p["w_b"], p["sm_scale"], p["base"], p["d_c"])


def rel(a, b):
    return float(np.linalg.norm(np.asarray(a) - np.asarray(b)) / max(np.linalg.norm(np.asarray(b)), 1e-300))


# -- P1: Eq. factorization ---------------------------------------------------------

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_p1_factorization_exact_with_request_context_local(seed):
    """z_off := Local contribution computed in the full request context => z_off + z_on_g
    equals the full-head projected state on every row, whatever the protected set."""
    p = small_problem(seed)
    rows = np.arange(p["T"])
    z_loc, _ = oracle.full_recompute_rows(rows, p["q_all"][:, p["lh"]], p["kv"], p["seg_off"], p["seg_delta"],
                                          p["w_uv"], p["w_a"], None, p["sm_scale"], p["base"], p["d_c"],
                                          heads=p["lh"])
    out = online(p, z_off=z_loc[:p["N_doc"]])
    z_full, y_full = full(p)
    assert rel(out["z"], z_full) < 1e-12
    assert rel(out["y"], y_full) < 1e-12


def test_p1_all_rows_protected_equals_full():
    p = small_problem(3)
    out = online(p, prot=np.arange(p["T"]), z_off=np.full_like(p["z_off"], np.nan))
    _, y_full = full(p)
    assert np.isfinite(out["y"]).all()
    assert rel(out["y"], y_full) < 1e-12


# -- P2: Eq. rope -------------------------------------------------------------------

def test_p2_relocation_identity_raw_vectors():
    rng = np.random.default_rng(5)
    for _ in range(200):
        q, k = rng.normal(size=64), rng.normal(size=64)
        pq, pk, d = (int(x) for x in rng.integers(0, 2 ** 19, size=3))
        lhs = oracle.rope_rotate(q, pq, 10000.0) @ oracle.rope_rotate(k, pk + d, 10000.0)
        rhs = oracle.rope_rotate(q, pq - d, 10000.0) @ oracle.rope_rotate(k, pk, 10000.0)
        assert abs(lhs - rhs) < 1e-9 * (1 + abs(lhs))


def test_p2_rope_textbook_properties():
    """R(p) is orthogonal, R(a)R(b) = R(a+b), R(0) = I, and pair j turns by p*theta_j in the
    positive sense (checked against complex multiplication)."""
    rng = np.random.default_rng(6)
    x = rng.normal(size=(7, 64))
    assert np.allclose(oracle.rope_rotate(x, 0, 10000.0), x, atol=0)
    a, b = 12345, 678
    assert np.allclose(oracle.rope_rotate(oracle.rope_rotate(x, a, 10000.0), b, 10000.0),
                       oracle.rope_rotate(x, a + b, 10000.0), atol=1e-10)
    assert np.allclose(np.linalg.norm(oracle.rope_rotate(x, 999, 10000.0), axis=-1), np.linalg.norm(x, axis=-1))
    theta = 10000.0 ** (-2.0 * np.arange(32) / 64.0)
    assert np.allclose(oracle.rope_theta(64, 10000.0), theta)
    z = (x[:, 0::2] + 1j * x[:, 1::2]) * np.exp(1j * 17 * theta)
    r = oracle.rope_rotate(x, 17, 10000.0)
    assert np.allclose(r[:, 0::2], z.real) and np.allclose(r[:, 1::2], z.imag)
    # per-row positions broadcast
    pos = np.arange(7)
    r2 = oracle.rope_rotate(x, pos, 10000.0)
    for i in range(7):
        assert np.allclose(r2[i], oracle.rope_rotate(x[i], int(pos[i]), 10000.0))


@pytest.mark.parametrize("seed", [0, 4])
def test_p2_p3_segmentwise_query_side_equals_key_side_single_softmax(seed):
    """Algorithm 2's order (rotate query by -delta_i, attend canonical keys per segment,
    LSE-merge) equals the plain definition (keys at request positions, one softmax)."""
    p = small_problem(seed)
    rows = np.arange(p["T"])
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    O1, l1 = oracle.attend_rows(p["q_all"], pos[rows], k_req, p["kv"][:, :p["d_c"]], pos, p["sm_scale"])
    O2, l2 = oracle.attend_rows_segmentwise(p["q_all"], pos[rows], p["kv"], p["seg_off"], p["seg_delta"],
                                            p["d_c"], p["base"], p["sm_scale"])
    assert rel(O2, O1) < 1e-12
    assert np.max(np.abs(l2 - l1)) < 1e-12


# -- P3: merge over any partition == one softmax ----------------------------------------

def test_p3_merge_any_partition_with_empty_parts():
    p = small_problem(7)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    v = p["kv"][:, :p["d_c"]]
    rows = np.arange(p["T"])
    O1, l1 = oracle.attend_rows(p["q_all"], pos, k_req, v, pos, p["sm_scale"])
    rng = np.random.default_rng(0)
    label = rng.integers(0, 4, size=p["T"])
    label[label == 2] = 3                    # part 2 is empty for everybody
    parts = [oracle.attend_rows(p["q_all"], pos, k_req, v, pos, p["sm_scale"],
                                key_subset=np.nonzero(label == j)[0]) for j in range(4)]
    Op = np.stack([a for a, _ in parts])
    Lp = np.stack([b for _, b in parts])
    assert np.isinf(Lp[2]).all()
    Op[2] = np.nan                           # ignored because its lse is -inf
    O2, l2 = oracle.segmented_merge(Op, Lp)
    assert rel(O2, O1) < 1e-12 and np.max(np.abs(l2 - l1)) < 1e-12
    # one part is the identity; all-empty gives O = 0, lse = -inf, no NaN
    O3, l3 = oracle.segmented_merge(Op[:1], Lp[:1])
    assert np.array_equal(O3[np.isfinite(Lp[0])], Op[0][np.isfinite(Lp[0])])
    O4, l4 = oracle.segmented_merge(Op[2:3], Lp[2:3])
    assert np.all(O4 == 0) and np.all(np.isneginf(l4))


def test_p3_merge_closed_form_two_parts():
    """Two parts with lse a, b: weights are the logistic function of (a - b)."""
    a, b = 1.7, -0.4
    Oa, Ob = np.array([[1.0, 2.0]]), np.array([[-3.0, 5.0]])
    O, l = oracle.segmented_merge(np.stack([Oa, Ob]), np.array([[a], [b]]))
    wa = 1.0 / (1.0 + math.exp(b - a))
    assert np.allclose(O, wa * Oa + (1 - wa) * Ob, atol=1e-15)
    assert abs(l[0] - math.log(math.exp(a) + math.exp(b))) < 1e-15
    # huge magnitudes do not overflow
    O, l = oracle.segmented_merge(np.stack([Oa, Ob]), np.array([[5000.0], [4999.0]]))
    assert np.isfinite(O).all() and abs(l[0] - (5000.0 + math.log1p(math.exp(-1.0)))) < 1e-9


# -- P4: scalar brute force ------------------------------------------------------------------

def test_p4_scalar_brute_force():
    p = small_problem(11, doc_lens=(5, 6), n_q=3, d_c=8, d_r=4, d_v=4, r_o=3, d_model=5)
    b = brute.brute_layer(p["q_all"].tolist(), p["kv"].tolist(), p["seg_off"], p["seg_delta"], p["prot"], p["gh"],
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
    for k, t in enumerate(p["prot"]):
        for a, h in enumerate(p["lh"]):
            assert abs(out["lse_l"][k, a] - b["lse"][t][h]) < 1e-12
    # heads that are neither Global nor on a protected row are not computed
    unprot = [t for t in range(p["T"]) if t not in set(p["prot"].tolist())]
    assert all(b["lse"][unprot[0]][h] is None for h in p["lh"])


# -- P5: prefix exactness ----------------------------------------------------------------------

@pytest.mark.parametrize("seed", [0, 9])
def test_p5_first_document_reuses_exactly(seed):
    """The document placed first in the request (delta = 0) was built in exactly the
    context it is used in, so its honest position-zero artifact makes MLA-Online equal to
    full recomputation on its rows, protected or not; other documents' rows do not."""
    p = small_problem(seed)
    D = len(p["seg_delta"]) - 1
    z_off = np.zeros_like(p["z_off"])
    for i in range(D):
        lo, hi = p["seg_off"][i], p["seg_off"][i + 1]
        z_off[lo:hi] = oracle.mla_off_artifact(i, p["q_all"][lo:hi][:, p["lh"]], p["kv"], p["seg_off"],
                                               p["seg_delta"], p["lh"], p["w_uv"], p["w_a"], p["sm_scale"],
                                               p["base"], p["d_c"])
    out = online(p, z_off=z_off)
    _, y_full = full(p)
    first = int(np.argmin(p["seg_delta"][:D]))
    lo, hi = p["seg_off"][first], p["seg_off"][first + 1]
    assert rel(out["y"][lo:hi], y_full[lo:hi]) < 1e-12
    isp = out["is_prot"]
    assert rel(out["y"][isp], y_full[isp]) < 1e-12          # protected rows are recomputed
    others = np.ones(p["T"], bool)
    others[lo:hi] = False
    others &= ~isp
    assert rel(out["y"][others], y_full[others]) > 1e-3     # reuse elsewhere is an approximation
    rep = oracle.reuse_error_report(out["y"], y_full, isp)
    assert rep["protected"] < 1e-12 and rep["unprotected"] > 0


# -- P6 / P7: closed forms -----------------------------------------------------------------------

def test_p6_zero_query_running_mean_and_count():
    p = small_problem(13)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    v = p["kv"][:, :p["d_c"]]
    q0 = np.zeros((p["T"], 2, p["d_c"] + p["d_r"]))
    O, lse = oracle.attend_rows(q0, pos, k_req, v, pos, p["sm_scale"])
    order = np.argsort(pos)
    assert np.array_equal(pos[order], np.arange(p["T"]))          # gap-free layout
    cm = np.cumsum(v[order], axis=0) / (np.arange(p["T"]) + 1)[:, None]
    for t in range(p["T"]):
        assert np.allclose(O[t, 0], cm[pos[t]], atol=1e-13)
        assert abs(lse[t, 1] - math.log(pos[t] + 1)) < 1e-13


def test_p7_one_hot_limit():
    """q = lambda K_req[k*] with k* the visible key of largest norm: its own score lambda |K*|^2 exceeds every other
    score lambda <K*, K_k> (Cauchy-Schwarz, strict for non-parallel keys), so for large lambda the softmax puts all
    weight on k* and the output is its latent c_{k*}; lse tends to the top score."""
    p = small_problem(14)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    v = p["kv"][:, :p["d_c"]]
    t = int(np.argmax(pos))                                          # sees everything
    kstar = int(np.argmax(np.linalg.norm(k_req, axis=1)))
    lam = 4000.0 / p["sm_scale"]
    q = (k_req[kstar] * lam)[None, None, :]
    s_all = (k_req @ q[0, 0]) * p["sm_scale"]
    assert int(np.argmax(s_all)) == kstar and np.sort(s_all)[-1] - np.sort(s_all)[-2] > 50.0
    O, lse = oracle.attend_rows(q, pos[[t]], k_req, v, pos, p["sm_scale"])
    assert np.allclose(O[0, 0], v[kstar], atol=1e-12)
    assert abs(lse[0, 0] - s_all[kstar]) < 1e-9 * abs(s_all[kstar])
    # a row that cannot see k* does not get its latent
    hidden = np.nonzero(pos < pos[kstar])[0]
    if len(hidden):
        O2, _ = oracle.attend_rows(q, pos[hidden[:1]], k_req, v, pos, p["sm_scale"])
        assert not np.allclose(O2[0, 0], v[kstar], atol=1e-3)


# -- P8 / P9: invariances -----------------------------------------------------------------------

def test_p8_packed_order_permutation_invariance():
    """Moving documents around in the packed stream while every token keeps its request
    position changes no token's output."""
    p = small_problem(15, doc_lens=(5, 7, 6))
    out = online(p)
    D = 3
    perm = [2, 0, 1]                                             # new packed order of the documents
    lens = [int(p["seg_off"][i + 1] - p["seg_off"][i]) for i in range(D + 1)]
    new_rows = np.concatenate([np.arange(p["seg_off"][i], p["seg_off"][i + 1]) for i in perm] +
                              [np.arange(p["seg_off"][D], p["T"])])
    p2 = dict(p)
    p2["seg_off"] = np.concatenate([[0], np.cumsum([lens[i] for i in perm] + [lens[D]])]).astype(np.int64)
    p2["seg_delta"] = np.concatenate([p["seg_delta"][perm], p["seg_delta"][D:]])
    p2["kv"] = p["kv"][new_rows]
    p2["q_all"] = p["q_all"][new_rows]
    inv_new = np.empty(p["T"], dtype=np.int64)
    inv_new[new_rows] = np.arange(p["T"])
    p2["prot"] = np.sort(inv_new[p["prot"]])
    p2["z_off"] = p["z_off"][new_rows[:p["N_doc"]]]
    out2 = online(p2)
    assert rel(out2["y"], out["y"][new_rows]) < 1e-12


def test_p9_global_shift_invariance():
    p = small_problem(16)
    out = online(p)
    shift = 977
    p2 = dict(p)
    p2["seg_delta"] = p["seg_delta"] + shift
    q2 = p["q_all"].copy()
    q2[..., p["d_c"]:] = oracle.rope_rotate(p["q_all"][..., p["d_c"]:], shift, p["base"])
    p2["q_all"] = q2
    out2 = online(p2)
    assert rel(out2["y"], out["y"]) < 1e-10
    assert np.max(np.abs(out2["lse_g"] - out["lse_g"])) < 1e-10


# -- P10: printed constants (fixtures under tests/golden) ------------------------------------------

def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "profile_constants.txt")
    rows = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, inputs, printed, _cite = [s.strip() for s in line.split("|")]
        rows[name] = ([float(x) for x in inputs.split()], [float(x) for x in printed.split()])
    return rows


def test_p10_printed_profile_ceilings_and_cold_model():
    g = _golden()
    for name in ("ceiling_flash", "ceiling_pro"):
        (nr, n, l, h), (printed,) = g[name]
        assert round(100 * oracle.head_row_ceiling(int(nr), int(n), int(l), int(h)), 2) == printed
    hot, (lo, hi) = g["cold_range"]
    vals = [oracle.cold_speed_ratio(s) for s in hot]
    assert round(min(vals), 2) == lo and round(max(vals), 2) == hi


# -- P11: library special case -------------------------------------------------------------------

def test_p11_torch_sdpa_float64():
    p = small_problem(17)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    v = p["kv"][:, :p["d_c"]]
    O, _ = oracle.attend_rows(p["q_all"], pos, k_req, v, pos, p["sm_scale"])
    q_t = torch.from_numpy(p["q_all"]).permute(1, 0, 2)[None]               # [1, H, T, dqk]
    k_t = torch.from_numpy(k_req)[None, None].expand(1, p["H"], -1, -1)
    v_t = torch.from_numpy(v)[None, None].expand(1, p["H"], -1, -1)
    mask = torch.from_numpy(pos[None, :] <= pos[:, None])                    # [T(row), T(key)]
    ref = torch.nn.functional.scaled_dot_product_attention(q_t, k_t, v_t, attn_mask=mask, scale=p["sm_scale"])
    assert rel(O, ref[0].permute(1, 0, 2).numpy()) < 1e-12


# -- replace semantics and selection -------------------------------------------------------------------

def test_replace_never_double_counted():
    p = small_problem(18)
    out = online(p)
    z_poison = p["z_off"].copy()
    doc_prot = p["prot"][p["prot"] < p["N_doc"]]
    z_poison[doc_prot] = np.nan
    out2 = online(p, z_off=z_poison)
    assert np.array_equal(out["y"], out2["y"]) and np.isfinite(out2["y"]).all()
    # unprotected rows take z_off verbatim on top of the Global contribution
    un = ~out["is_prot"]
    zg = out["z_on_g"].reshape(p["T"], -1)
    assert np.allclose(out["z"][un], zg[un] + p["z_off"][np.nonzero(un)[0]], atol=0)


def test_geometry_helpers():
    seg_off = np.array([0, 3, 5, 9])
    delta = np.array([4, 0, 7])
    assert oracle.request_positions(seg_off, delta).tolist() == [4, 5, 6, 0, 1, 7, 8, 9, 10]
    assert oracle.segment_of_rows(seg_off).tolist() == [0, 0, 0, 1, 1, 2, 2, 2, 2]
    assert oracle.inverse_row_map(np.array([1, 4, 8]), 9).tolist() == [-1, 0, -1, -1, 1, -1, -1, -1, 2]


def test_wrong_slice_detector():
    """Zeroing one head's slice of W_a removes exactly that head's contribution."""
    p = small_problem(19)
    rows = np.arange(p["T"])
    z0, _ = full(p)
    h = int(p["lh"][3])
    g, j = h // 8, h % 8
    p2 = dict(p)
    w = p["w_a"].copy()
    w[g][:, p["d_v"] * j: p["d_v"] * (j + 1)] = 0
    p2["w_a"] = w
    z1, _ = full(p2)
    pos = oracle.request_positions(p["seg_off"], p["seg_delta"])
    k_req = oracle.keys_in_request_frame(p["kv"], p["seg_off"], p["seg_delta"], p["d_c"], p["base"])
    O, _ = oracle.attend_rows(p["q_all"][:, [h]], pos, k_req, p["kv"][:, :p["d_c"]], pos, p["sm_scale"])
    c = oracle.head_contributions(O, np.array([h]), p["w_uv"], p["w_a"])[:, 0]
    d = (z0 - z1).reshape(p["T"], p["G"], p["r_o"])
    assert np.allclose(d[:, g], c, atol=1e-12)
    assert np.allclose(np.delete(d, g, axis=1), 0, atol=1e-13)


def test_reuse_error_report_closed_form():
    """The report is a relative L2 distance on two row subsets: hand-made vectors with known norms."""
    y_full = np.array([[3.0, 4.0], [0.0, 5.0], [6.0, 8.0], [1.0, 0.0]])          # row norms 5, 5, 10, 1
    y_on = y_full.copy()
    y_on[1] += [3.0, 4.0]                                                         # unprotected row off by norm 5
    y_on[2] += [0.0, 1.0]                                                         # protected row off by norm 1
    is_prot = np.array([True, False, True, False])
    rep = oracle.reuse_error_report(y_on, y_full, is_prot)
    assert abs(rep["protected"] - 1.0 / math.sqrt(25.0 + 100.0)) < 1e-15          # ||(0,0),(0,1)|| / ||rows 0, 2||
    assert abs(rep["unprotected"] - 5.0 / math.sqrt(25.0 + 1.0)) < 1e-15          # ||(3,4),(0,0)|| / ||rows 1, 3||
    assert oracle.reuse_error_report(y_full, y_full, is_prot) == dict(protected=0.0, unprotected=0.0)
    none = oracle.reuse_error_report(y_on, y_full, np.zeros(4, bool))
    assert none["protected"] == 0.0 and none["unprotected"] > 0
