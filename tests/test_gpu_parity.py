"""GPU parity: every C-ABI call against the float64 checker on identical seeded inputs
(bf16 storage, fp32 accumulate).  Tolerances: max-abs <= 1e-2 and relative L2 <= 5e-3 per
tensor; one-rounding steps (relocation) are held to one bf16 ulp; selections are bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_07008_b200 import synth
from tests.helpers import assert_close, f64, max_abs, oracle_online, rel_l2, to_device

# guard zones around every buffer the binding allocates are checked after every library call here
pytestmark = [pytest.mark.gpu, pytest.mark.guard_each_call]


@pytest.fixture(scope="module")
def rk():
    from paper_2609_07008_b200 import binding
    return binding


def make(rk, w):
    ctx = rk.Context.from_profile(w.profile)
    req = ctx.rk_request_create(w.layout.seg_off, w.layout.seg_delta, w.layout.seg_has_artifact, w.prot_rows)
    return ctx, req


def small_ragged(regime="sharp", seed=5):
    return synth.make_custom([300, 77, 513], 50, n_heads=16, n_groups=2, o_rank=256, d_model=512, pct_bp=700,
                             seed=seed, regime=regime)


# -- (1) relocation ---------------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["tiny", "ragged"])
def test_relocate_q(rk, name):
    w = synth.make_workload("tiny") if name == "tiny" else small_ragged()
    ctx, req = make(rk, w)
    to_device(w)
    S = w.layout.n_segs
    view = w.q_g[:, :, 512:]                       # strided view of the rope sub-vectors
    out = ctx.rk_relocate_q(req, view, 0, S)
    ctx.rk_poll_status()
    x = f64(view)
    for i in range(S):
        want = oracle.relocate_query(x, float(w.layout.seg_delta[i]), w.profile.rope_base)
        got = f64(out[i])
        err = np.abs(got - want)
        assert (err <= 2.0 ** -8 * np.abs(want) + 1e-6 * np.abs(x).max()).all(), f"segment {i}: {err.max()}"
    # a sub-range of segments lands in the right frames
    out2 = ctx.rk_relocate_q(req, view, 1, S)
    assert torch.equal(out2, out[1:])


# -- (3) standalone merge ---------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("P", [1, 3, 65, 4096])        # 4096 = the largest part count the call accepts
def test_segmented_merge(rk, dtype, P):
    w = synth.make_workload("tiny")
    ctx, _ = make(rk, w)
    g = torch.Generator().manual_seed(P)
    n_rows, n_heads = (37, 5) if P <= 65 else (3, 2)
    O_part = torch.randn((P, n_rows, n_heads, 512), generator=g).to(dtype)
    lse_part = torch.randn((P, n_rows, n_heads), generator=g) * 3
    if P > 1:
        lse_part[torch.rand((P, n_rows, n_heads), generator=g) < 0.3] = -float("inf")
        lse_part[:, 0, 0] = -float("inf")                      # a (row, head) whose parts are all empty
        O_part[1, 1, 1] = float("nan")                         # ignored: its part is empty
        lse_part[1, 1, 1] = -float("inf")
    O, lse = ctx.rk_segmented_merge(O_part.cuda(), lse_part.cuda())
    ctx.rk_poll_status()
    want_O, want_lse = oracle.segmented_merge(f64(O_part), f64(lse_part))
    got_lse = f64(lse)
    fin = np.isfinite(want_lse)
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(want_lse))
    assert max_abs(got_lse[fin], want_lse[fin]) <= 1e-3
    assert_close(f64(O), want_O, "merged O", unit_scale=True)
    if P == 1:
        assert torch.equal(O.cpu(), O_part[0].to(torch.bfloat16))    # one part is the identity


# -- (2) attention -----------------------------------------------------------------------------------

# lse tolerance: the rotated rope sub-vector is rounded to bf16 once more before QK^T, which moves a
# logit by about |q_rope| |k_rope| sm_scale 2^-9 ~ 1e-3 when q, k are O(1) ("sharp" values) and by
# far less for the benchmark's N(0, 0.02) latents; lse is a convex combination of logits.
LSE_TOL = {"mandated": 1e-3, "sharp": 5e-3}


def check_attention(rk, w, rows=None, lse_tol=LSE_TOL["sharp"]):
    ctx, req = make(rk, w)
    T = w.layout.n_rows
    rows = np.arange(T) if rows is None else rows
    exp = oracle_online(w, rows)
    to_device(w)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    ctx.rk_poll_status()
    r1 = assert_close(f64(O_g)[rows], exp["O_g"], "O_g", unit_scale=w.regime == "sharp")
    assert max_abs(f64(lse_g)[rows], exp["lse_g"]) <= lse_tol
    inv = oracle.inverse_row_map(w.prot_rows, T)
    slots = inv[rows][inv[rows] >= 0]
    r2 = assert_close(f64(O_l)[slots], exp["O_l"], "O_l", unit_scale=w.regime == "sharp")
    assert max_abs(f64(lse_l)[slots], exp["lse_l"]) <= lse_tol
    return r1, r2


@pytest.mark.parametrize("regime", ["mandated", "sharp"])
def test_attention_tiny(rk, regime):
    check_attention(rk, synth.make_workload("tiny", regime=regime), lse_tol=LSE_TOL[regime])


@pytest.mark.parametrize("seed", [5, 6])
def test_attention_ragged(rk, seed):
    check_attention(rk, small_ragged(seed=seed))


def test_attention_single_pass_and_shift(rk):
    """Each pass can run alone; adding a constant to every request offset (and re-rotating q)
    leaves the outputs unchanged within rounding."""
    w = small_ragged(seed=7)
    ctx, req = make(rk, w)
    to_device(w)
    O_g, lse_g, _, _ = ctx.rk_mla_online_attn(req, w.kv, w.q_g, None)
    _, _, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, None, w.q_l)
    O_g2, lse_g2, O_l2, lse_l2 = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    ctx.rk_poll_status()
    assert torch.equal(O_g, O_g2) and torch.equal(O_l, O_l2) and torch.equal(lse_g, lse_g2)


# -- (4) sliced projection ------------------------------------------------------------------------------

def test_group_sliced_proj(rk):
    w = small_ragged(seed=8)
    ctx, req = make(rk, w)
    p = w.profile
    T, A = w.layout.n_rows, len(w.prot_rows)
    g = torch.Generator().manual_seed(1)
    O_g = (torch.randn((T, p.n_groups, 512), generator=g) * 0.5).to(torch.bfloat16)
    O_l = (torch.randn((A, p.n_local, 512), generator=g) * 0.5).to(torch.bfloat16)
    to_device(w)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g.cuda(), O_l.cuda(), w.w_uv, w.w_a)
    ctx.rk_poll_status()
    wuv, wa = f64(w.w_uv), f64(w.w_a)
    cg = oracle.head_contributions(f64(O_g), p.global_heads, wuv, wa)
    want_g = cg.reshape(T, -1)                                  # one Global head per group, group order
    cl = oracle.head_contributions(f64(O_l), p.local_heads, wuv, wa)
    want_l = np.zeros((A, p.n_groups, p.o_rank))
    for a, h in enumerate(p.local_heads):
        want_l[:, h // 8] += cl[:, a]
    assert_close(f64(z_on_g), want_g, "z_on_g", unit_scale=w.regime == "sharp")
    assert_close(f64(z_on_l), want_l.reshape(A, -1), "z_on_l", unit_scale=w.regime == "sharp")
    # wrong-slice detector: zero one Local head's slice of W_a -> exactly that head's contribution goes
    h = int(p.local_heads[4])
    wa2 = w.w_a.clone()
    wa2[h // 8, :, 128 * (h % 8):128 * (h % 8 + 1)] = 0
    _, z2 = ctx.rk_group_sliced_proj(req, None, O_l.cuda(), w.w_uv, wa2)
    ctx.rk_poll_status()
    want2 = want_l.copy()
    want2[:, h // 8] -= cl[:, 4]
    assert_close(f64(z2), want2.reshape(A, -1), "z_on_l with one slice zeroed", unit_scale=w.regime == "sharp")


@pytest.mark.parametrize("H, G, ro, lens, nq", [
    (16, 2, 512, [513, 255, 64], 128),     # fused Global kernel, four column tiles
    (32, 4, 1024, [130, 77], 31),          # eight column tiles, ragged last row block
    (16, 2, 768, [1000], 5),               # six column tiles
    (8, 1, 256, [64], 64),                 # one group, exactly one row block
    (16, 2, 128, [300, 200], 40),          # r_o not a multiple of 256: the two-GEMM path
])
def test_group_sliced_proj_shapes(rk, H, G, ro, lens, nq):
    """The sliced first projection over group ranks and row counts that take every path of its kernels (the Global
    half is one fused kernel when r_o is a multiple of 256), each against the checker."""
    w = synth.make_custom(lens, nq, n_heads=H, n_groups=G, o_rank=ro, d_model=256, pct_bp=1500, seed=90 + ro // 128)
    ctx, req = make(rk, w)
    p, T, A = w.profile, w.layout.n_rows, len(w.prot_rows)
    g = torch.Generator().manual_seed(ro)
    O_g = (torch.randn((T, G, 512), generator=g) * 0.5).to(torch.bfloat16)
    O_l = (torch.randn((A, H - G, 512), generator=g) * 0.5).to(torch.bfloat16)
    to_device(w)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g.cuda(), O_l.cuda(), w.w_uv, w.w_a)
    ctx.rk_poll_status()
    wuv, wa = f64(w.w_uv), f64(w.w_a)
    want_g = oracle.head_contributions(f64(O_g), p.global_heads, wuv, wa).reshape(T, -1)
    cl = oracle.head_contributions(f64(O_l), p.local_heads, wuv, wa)
    want_l = np.zeros((A, G, ro))
    for a, h in enumerate(p.local_heads):
        want_l[:, h // 8] += cl[:, a]
    assert_close(f64(z_on_g), want_g, "z_on_g", unit_scale=True)
    assert_close(f64(z_on_l), want_l.reshape(A, -1), "z_on_l", unit_scale=True)


# -- (5) combine + W_b -----------------------------------------------------------------------------------

def test_combine_offline(rk):
    w = small_ragged(seed=9)
    ctx, req = make(rk, w)
    p = w.profile
    T, A = w.layout.n_rows, len(w.prot_rows)
    width = p.n_groups * p.o_rank
    g = torch.Generator().manual_seed(2)
    z_on_g = (torch.randn((T, width), generator=g) * 0.3).to(torch.bfloat16)
    z_on_l = (torch.randn((A, width), generator=g) * 0.3).to(torch.bfloat16)
    z_off = (torch.randn((w.layout.n_doc_rows, width), generator=g) * 0.3).to(torch.bfloat16)
    to_device(w)
    z, y = ctx.rk_combine_offline(req, z_on_g.cuda(), z_on_l.cuda(), z_off.cuda(), w.w_b)
    ctx.rk_poll_status()
    inv = oracle.inverse_row_map(w.prot_rows, T)
    want_z = f64(z_on_g).copy()
    for t in range(T):
        want_z[t] += f64(z_on_l[inv[t]]) if inv[t] >= 0 else f64(z_off[t])
    assert_close(f64(z), want_z, "z", unit_scale=w.regime == "sharp")
    assert_close(f64(y), f64(z) @ f64(w.w_b).T, "y from the library's own z", unit_scale=w.regime == "sharp")
    assert_close(f64(y), want_z @ f64(w.w_b).T, "y", unit_scale=w.regime == "sharp")
    # a protected row takes z_on_l in place of the artifact, never both: poisoning z_off on protected rows changes nothing
    z_poison = z_off.clone()
    doc_prot = torch.as_tensor(w.prot_rows[w.prot_rows < w.layout.n_doc_rows].astype(np.int64))
    z_poison[doc_prot] = float("nan")
    zp = z_poison.cuda()
    before = zp.clone()
    z2, y2 = ctx.rk_combine_offline(req, z_on_g.cuda(), z_on_l.cuda(), zp, w.w_b)
    ctx.rk_poll_status()
    assert torch.equal(z2, z) and torch.equal(y2, y)
    assert torch.equal(zp.view(torch.int16), before.view(torch.int16))     # the artifact is never written


# -- end to end ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("regime", ["mandated", "sharp"])
def test_end_to_end_tiny_honest_artifact(rk, regime):
    w = synth.make_workload("tiny", regime=regime, with_q_all=True)
    p, lay = w.profile, w.layout
    # honest MLA-Off artifact from the checker (each document alone at position zero)
    z_off = np.zeros((lay.n_doc_rows, p.n_groups * p.o_rank))
    q_all = f64(w.q_all)
    for i in range(lay.n_segs):
        if lay.seg_has_artifact[i]:
            lo, hi = int(lay.seg_off[i]), int(lay.seg_off[i + 1])
            z_off[lo:hi] = oracle.mla_off_artifact(i, q_all[lo:hi][:, p.local_heads], f64(w.kv), lay.seg_off,
                                                   lay.seg_delta, p.local_heads, f64(w.w_uv), f64(w.w_a), p.sm_scale,
                                                   p.rope_base, p.d_latent)
    w.z_off = torch.from_numpy(z_off).to(torch.bfloat16)
    rows = np.arange(lay.n_rows)
    exp = oracle_online(w, rows)
    ctx, req = make(rk, w)
    to_device(w)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
    ctx.rk_poll_status()
    assert_close(f64(z), exp["z"], "z", unit_scale=w.regime == "sharp")
    assert_close(f64(y), exp["y"], "y", unit_scale=w.regime == "sharp")
    # the same through the host-buffer entry point
    bufs = ctx.alloc_layer_buffers(req, "cuda")
    pin = lambda t: t.cpu().pin_memory()
    y_h = torch.empty((lay.n_rows, p.d_model), dtype=torch.bfloat16).pin_memory()
    ctx.rk_layer_host(req, pin(w.kv), pin(w.q_g), pin(w.q_l), pin(w.z_off), w.w_uv, w.w_a, w.w_b, bufs, y_h)
    ctx.rk_poll_status()
    assert torch.equal(y_h, y.cpu())


def test_layer_host_row_ranges_equal_device_path(rk):
    """rk_layer_host runs the Local pass and everything from the Global pass on in two row ranges each
    (so that copies overlap kernels); the result is bit-identical to the call-by-call device path."""
    w = synth.make_custom([1500, 900, 700], 200, n_heads=16, n_groups=2, o_rank=256, d_model=512, pct_bp=3000, seed=9)
    ctx, req = make(rk, w)
    assert req.A >= 512 and w.layout.n_rows >= 512          # both passes are split at these sizes
    to_device(w)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
    ctx.rk_poll_status()
    bufs = ctx.alloc_layer_buffers(req, "cuda")
    pin = lambda t: t.cpu().pin_memory()
    y_h = torch.empty((w.layout.n_rows, w.profile.d_model), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):                                       # a second call reuses the staging buffers
        y_h.zero_()
        ctx.rk_layer_host(req, pin(w.kv), pin(w.q_g), pin(w.q_l), pin(w.z_off), w.w_uv, w.w_a, w.w_b, bufs, y_h)
        ctx.rk_poll_status()
        assert torch.equal(y_h, y.cpu())
    rows = synth.sample_rows(w.layout, w.prot_rows, 16, seed=1)
    exp = oracle_online(w, rows)
    assert_close(f64(y_h[rows]), exp["y"], "y (host path, sampled rows)", unit_scale=w.regime == "sharp")


@pytest.mark.parametrize("seed", range(10))
def test_irregular_requests_every_row(rk, seed):
    """Seeded irregular requests (segment lengths on and around tile boundaries, length-1 segments, gaps,
    shuffled request order, uncached segments in the middle): every row of every stage against the checker."""
    w = synth.make_random_request(seed)
    lay = w.layout
    rows = np.arange(lay.n_rows)
    exp = oracle_online(w, rows)
    ctx, req = make(rk, w)
    to_device(w)
    inputs = dict(kv=w.kv, q_g=w.q_g, q_l=w.q_l, W_uv=w.w_uv, W_a=w.w_a, W_b=w.w_b, z_off=w.z_off)
    before = {k: t.clone() for k, t in inputs.items()}
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
    ctx.rk_poll_status()
    assert_close(f64(O_g), exp["O_g"], "O_g", unit_scale=w.regime == "sharp")
    assert np.abs(f64(lse_g) - exp["lse_g"]).max() <= 5e-3
    assert_close(f64(O_l), exp["O_l"], "O_l", unit_scale=w.regime == "sharp")
    assert_close(f64(z), exp["z"], "z", unit_scale=w.regime == "sharp")
    assert_close(f64(y), exp["y"], "y", unit_scale=w.regime == "sharp")
    # the same request through the host-buffer entry point gives the same bits
    bufs = ctx.alloc_layer_buffers(req, "cuda")
    pin = lambda t: t.cpu().pin_memory()
    y_h = torch.empty((lay.n_rows, w.profile.d_model), dtype=torch.bfloat16).pin_memory()
    ctx.rk_layer_host(req, pin(w.kv), pin(w.q_g), pin(w.q_l), pin(w.z_off), w.w_uv, w.w_a, w.w_b, bufs, y_h)
    ctx.rk_poll_status()
    assert torch.equal(y_h, y.cpu())
    # the latent stream, the queries, the weights and the artifact are read-only for the library: byte-equal after
    for k, t in inputs.items():
        assert torch.equal(t.view(torch.int16), before[k].view(torch.int16)), f"{k} was written"


# -- edge cases -------------------------------------------------------------------------------------------

def _layer(rk, w):
    ctx, req = make(rk, w)
    to_device(w)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l if req.A else None)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off if w.layout.n_doc_rows else None, w.w_b)
    ctx.rk_poll_status()
    return y


def test_query_only_request(rk):
    """No documents: one segment without artifact, every row protected, z_off never touched."""
    w = synth.make_custom([], 37, n_heads=16, n_groups=2, o_rank=128, d_model=256, pct_bp=0, seed=41)
    assert w.layout.n_segs == 1 and len(w.prot_rows) == 37 and w.layout.n_doc_rows == 0
    exp = oracle_online(w, np.arange(37), z_off=np.zeros((0, 256)))
    y = _layer(rk, w)
    assert_close(f64(y), exp["y"], "y", unit_scale=w.regime == "sharp")


def test_no_protected_rows(rk):
    """Every segment has an artifact and nothing is protected: the Local pass is skipped and every row
    takes z_off."""
    rng = np.random.default_rng(42)
    lay = synth.make_layout([130, 200], 0, rng, shuffle=True)
    lay = synth.Layout(seg_off=lay.seg_off[:-1], seg_delta=lay.seg_delta[:-1], seg_has_artifact=lay.seg_has_artifact[:-1])
    prof = synth.Profile(n_heads=16, n_groups=2, o_rank=128, d_model=256, global_heads=synth.draw_global_heads(2, rng),
                         sm_scale=float(1 / np.sqrt(192)))
    w = synth.make_tensors("custom", prof, lay, np.zeros(0, np.int32), 42, regime="sharp")
    exp = oracle_online(w, np.arange(lay.n_rows))
    y = _layer(rk, w)
    assert_close(f64(y), exp["y"], "y", unit_scale=w.regime == "sharp")
    # the host-buffer entry point without any Local work (no q_l at all)
    ctx, req = make(rk, w)
    bufs = ctx.alloc_layer_buffers(req, "cuda")
    pin = lambda t: t.cpu().pin_memory()
    y_h = torch.empty((lay.n_rows, prof.d_model), dtype=torch.bfloat16).pin_memory()
    ctx.rk_layer_host(req, pin(w.kv), pin(w.q_g), None, pin(w.z_off), w.w_uv, w.w_a, w.w_b, bufs, y_h)
    ctx.rk_poll_status()
    assert torch.equal(y_h, y.cpu())


def test_gaps_between_segments_and_large_offsets(rk):
    """Request-position intervals need not be contiguous: offsets with gaps (and beyond 2^20, where the
    relocation angles are large) leave the result equal to the checker's."""
    w = synth.make_custom([100, 260, 31], 20, n_heads=16, n_groups=2, o_rank=128, d_model=256, pct_bp=1000, seed=43)
    lay = w.layout
    lay.seg_delta = lay.seg_delta * 3 + np.array([7, 1 << 20, 12345, 5 << 20])[: lay.n_segs]
    # keep intervals disjoint
    order = np.argsort(lay.seg_delta)
    ends = lay.seg_delta[order] + (lay.seg_off[1:] - lay.seg_off[:-1])[order]
    assert (lay.seg_delta[order][1:] >= ends[:-1]).all()
    exp = oracle_online(w, np.arange(lay.n_rows))
    ctx, req = make(rk, w)
    to_device(w)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    ctx.rk_poll_status()
    assert_close(f64(O_g), exp["O_g"], "O_g", unit_scale=w.regime == "sharp")
    assert_close(f64(O_l), exp["O_l"], "O_l", unit_scale=w.regime == "sharp")
    assert max_abs(f64(lse_g), exp["lse_g"]) <= LSE_TOL["sharp"]


def test_argument_errors_on_device(rk):
    """Errors that need a context: misaligned pointers, short workspace, half-specified passes, a
    request from another context.  All are reported before anything is enqueued."""
    w = small_ragged(seed=12)
    ctx, req = make(rk, w)
    ctx2, _ = make(rk, w)
    to_device(w)
    T, A, p = w.layout.n_rows, len(w.prot_rows), w.profile
    O_g = torch.empty((T, p.n_groups, 512), dtype=torch.bfloat16, device="cuda")
    lse_g = torch.empty((T, p.n_groups), dtype=torch.float32, device="cuda")
    L = rk.lib
    s = torch.cuda.current_stream().cuda_stream
    # misaligned kv (2-byte offset)
    kv_pad = torch.empty(T * 576 + 8, dtype=torch.bfloat16, device="cuda")
    assert L.rk_mla_online_attn(ctx.handle, req.handle, kv_pad.data_ptr() + 2, w.q_g.data_ptr(), None, O_g.data_ptr(),
                                lse_g.data_ptr(), None, None, s) == 5
    # Global pass half specified
    assert L.rk_mla_online_attn(ctx.handle, req.handle, w.kv.data_ptr(), w.q_g.data_ptr(), None, None, None, None,
                                None, s) == 1
    # request created by another context
    assert L.rk_mla_online_attn(ctx2.handle, req.handle, w.kv.data_ptr(), w.q_g.data_ptr(), None, O_g.data_ptr(),
                                lse_g.data_ptr(), None, None, s) == 3
    # workspace one byte short
    ws = torch.empty(req.workspace_bytes, dtype=torch.uint8, device="cuda")
    z = torch.empty((T, p.n_groups * p.o_rank), dtype=torch.bfloat16, device="cuda")
    assert L.rk_group_sliced_proj(ctx.handle, req.handle, O_g.data_ptr(), None, w.w_uv.data_ptr(), w.w_a.data_ptr(),
                                  z.data_ptr(), None, ws.data_ptr(), req.workspace_bytes - 1, s) == 6
    assert b"workspace" in L.rk_last_error(ctx.handle)
    # relocation: segment range out of bounds, stride not a multiple of 8
    out = torch.empty((1, T, p.n_groups, 64), dtype=torch.bfloat16, device="cuda")
    assert L.rk_relocate_q(ctx.handle, req.handle, w.q_g.data_ptr(), T, p.n_groups, 576 * p.n_groups, 576, 0,
                           w.layout.n_segs + 1, out.data_ptr(), s) == 3
    assert L.rk_relocate_q(ctx.handle, req.handle, w.q_g.data_ptr(), T, p.n_groups, 577 * p.n_groups, 577, 0, 1,
                           out.data_ptr(), s) == 5
    # merge: unknown part dtype
    assert L.rk_segmented_merge(ctx.handle, 2, 4, 2, O_g.data_ptr(), 7, lse_g.data_ptr(), O_g.data_ptr(),
                                lse_g.data_ptr(), s) == 7
    # merge with part phases: segment range beyond the request, too many parts, unknown dtype
    S = w.layout.n_segs
    assert L.rk_segmented_merge_phase(ctx.handle, req.handle, 1, S, 4, 2, O_g.data_ptr(), 0, lse_g.data_ptr(), None,
                                      O_g.data_ptr(), lse_g.data_ptr(), s) == 3
    assert L.rk_segmented_merge_phase(ctx.handle, req.handle, 0, 4097, 4, 2, O_g.data_ptr(), 0, lse_g.data_ptr(), None,
                                      O_g.data_ptr(), lse_g.data_ptr(), s) == 3
    assert L.rk_segmented_merge_phase(ctx.handle, req.handle, 0, 1, 4, 2, O_g.data_ptr(), 5, lse_g.data_ptr(), None,
                                      O_g.data_ptr(), lse_g.data_ptr(), s) == 7
    # combine: W_b given without y
    assert L.rk_combine_offline(ctx.handle, req.handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), w.w_b.data_ptr(),
                                z.data_ptr(), None, s) == 1
    ctx.rk_poll_status()          # nothing was enqueued, nothing timed out


def test_bounded_wait_reports_timeout_and_context_stays_usable(rk):
    """A device-side wait that nothing satisfies (the load warp is told to leave the ring stages empty)
    expires after the configured limit: the kernel drains and returns, rk_poll_status reports
    RK_ERR_TIMEOUT once, and the next call on the same context works."""
    w = synth.make_workload("tiny")
    ctx, req = make(rk, w)
    to_device(w)
    ctx.rk_set_wait_limit_ms(20)
    ctx.rk_test_starve_loads(True)
    ctx.rk_mla_online_attn(req, w.kv, w.q_g, None)
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_poll_status()
    assert ei.value.status == 9 and "wait expired" in str(ei.value)
    ctx.rk_poll_status()                                   # the status word was cleared
    ctx.rk_test_starve_loads(False)
    ctx.rk_set_wait_limit_ms(2000)
    exp = oracle_online(w, np.arange(w.layout.n_rows))
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    ctx.rk_poll_status()
    assert_close(f64(O_g), exp["O_g"], "O_g after a timed-out launch", unit_scale=w.regime == "sharp")


# -- offline side: MLA-Off artifact build (Algorithm 1) ----------------------------------------------------

def _honest_artifact_oracle(w):
    p, lay = w.profile, w.layout
    z = np.zeros((lay.n_doc_rows, p.n_groups * p.o_rank))
    q_all = f64(w.q_all)
    for i in range(lay.n_segs):
        if lay.seg_has_artifact[i]:
            lo, hi = int(lay.seg_off[i]), int(lay.seg_off[i + 1])
            z[lo:hi] = oracle.mla_off_artifact(i, q_all[lo:hi][:, p.local_heads], f64(w.kv), lay.seg_off, lay.seg_delta,
                                               p.local_heads, f64(w.w_uv), f64(w.w_a), p.sm_scale, p.rope_base, p.d_latent)
    return z


@pytest.mark.parametrize("name", ["tiny", "ragged"])
def test_mla_off_build_matches_checker(rk, name):
    w = synth.make_workload("tiny", regime="sharp", with_q_all=True) if name == "tiny" else \
        synth.make_custom([300, 77, 513], 50, n_heads=16, n_groups=2, o_rank=256, d_model=512, pct_bp=700, seed=15,
                          with_q_all=True)
    p, lay = w.profile, w.layout
    want = _honest_artifact_oracle(w)
    ctx, req = make(rk, w)
    to_device(w)
    n = lay.n_doc_rows
    q_l_doc = w.q_all[:n][:, torch.as_tensor(p.local_heads.astype(np.int64), device="cuda")].contiguous()
    z_off = ctx.rk_mla_off_build(req, w.kv, 0, n, q_l_doc, w.w_uv, w.w_a)
    ctx.rk_poll_status()
    assert_close(f64(z_off), want, "z_off", unit_scale=w.regime == "sharp")
    # built in two row ranges that cut a document in the middle: same rows, same values
    cut = n // 2 + 3
    za = ctx.rk_mla_off_build(req, w.kv, 0, cut, q_l_doc[:cut].contiguous(), w.w_uv, w.w_a)
    zb = ctx.rk_mla_off_build(req, w.kv, cut, n, q_l_doc[cut:].contiguous(), w.w_uv, w.w_a)
    ctx.rk_poll_status()
    assert_close(f64(torch.cat([za, zb])), want, "z_off in two ranges", unit_scale=w.regime == "sharp")


def test_offline_then_online_chain_reuses_first_document_exactly(rk):
    """GPU-built artifact -> GPU online layer.  Against the checker's expected MLA-Online output, and:
    the document placed first in the request (delta = 0) was built in the very context it is used in,
    so its rows equal full recomputation (all heads on all rows) even where they are not protected."""
    w = synth.make_workload("tiny", regime="sharp", with_q_all=True)
    p, lay = w.profile, w.layout
    want_off = _honest_artifact_oracle(w)
    exp = oracle_online(w, np.arange(lay.n_rows), z_off=want_off)
    _, y_full = oracle.full_recompute_rows(np.arange(lay.n_rows), f64(w.q_all), f64(w.kv), lay.seg_off, lay.seg_delta,
                                           f64(w.w_uv), f64(w.w_a), f64(w.w_b), p.sm_scale, p.rope_base, p.d_latent)
    ctx, req = make(rk, w)
    to_device(w)
    n = lay.n_doc_rows
    q_l_doc = w.q_all[:n][:, torch.as_tensor(p.local_heads.astype(np.int64), device="cuda")].contiguous()
    z_off = ctx.rk_mla_off_build(req, w.kv, 0, n, q_l_doc, w.w_uv, w.w_a)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, z_off, w.w_b)
    ctx.rk_poll_status()
    assert_close(f64(y), exp["y"], "y with the GPU-built artifact", unit_scale=w.regime == "sharp")
    first = int(np.argmin(lay.seg_delta[:-1]))
    lo, hi = int(lay.seg_off[first]), int(lay.seg_off[first + 1])
    assert_close(f64(y[lo:hi]), y_full[lo:hi], "first document rows vs full recomputation", unit_scale=w.regime == "sharp")
    inv = oracle.inverse_row_map(w.prot_rows, lay.n_rows)
    assert_close(f64(y)[inv >= 0], y_full[inv >= 0], "protected rows vs full recomputation", unit_scale=w.regime == "sharp")


def test_request_info_pair_counts(rk):
    """pairs_global / pairs_local (used for flop accounting) equal a brute-force count of visible keys."""
    w = synth.make_custom([100, 260, 31], 20, n_heads=16, n_groups=2, o_rank=128, d_model=256, pct_bp=1000, seed=44)
    lay = w.layout
    lay.seg_delta = lay.seg_delta * 2 + 5             # gaps between segments
    ctx, req = make(rk, w)
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    vis = (pos[None, :] <= pos[:, None]).sum(axis=1)
    assert req.pairs_global == int(vis.sum())
    assert req.pairs_local == int(vis[w.prot_rows].sum())
    assert (req.T, req.A, req.n_off_rows) == (lay.n_rows, len(w.prot_rows), lay.n_doc_rows)


def test_layer_stack_host_matches_device_path(rk):
    """Five independent layers (own values, own protected rows, shared layout) through the stack entry
    point with cross-layer prefetch: every layer's y is bit-identical to the device-buffer path."""
    layers, want = [], []
    ctx = None
    for l in range(5):
        prof, lay, prot = synth.make_geometry("tiny", layer=l)
        rng = np.random.default_rng(100 + l)
        prot = synth.draw_protected_rows(lay, 300 + 200 * l, rng)            # a different row set per layer
        w = synth.make_tensors("tiny", prof, lay, prot, 500 + l, regime="sharp")
        if ctx is None:
            ctx = rk.Context.from_profile(prof)
        req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)
        pin = lambda t: t.cpu().pin_memory()
        host = dict(req=req, kv=pin(w.kv), q_g=pin(w.q_g), q_l=pin(w.q_l), z_off=pin(w.z_off))
        to_device(w)
        O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
        z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
        _, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
        want.append(y.cpu())
        host.update(W_uv=w.w_uv, W_a=w.w_a, W_b=w.w_b,
                    y=torch.full((lay.n_rows, prof.d_model), float("nan"), dtype=torch.bfloat16).pin_memory())
        layers.append(host)
    ctx.rk_poll_status()
    big = max(layers, key=lambda l: l["req"].A)["req"]
    b0, b1 = ctx.alloc_layer_buffers(big, "cuda"), ctx.alloc_layer_buffers(big, "cuda")
    for _ in range(2):                                     # twice: events and buffer sets are reused
        rk.rk_layer_stack_host(ctx, layers, b0, b1)
        ctx.rk_poll_status()
        for l in range(5):
            assert torch.equal(layers[l]["y"], want[l]), f"layer {l}"
    rk.rk_layer_stack_host(ctx, layers[:1], b0, b1)         # a stack of one
    assert torch.equal(layers[0]["y"], want[0])
