"""GPU parity of the output-phase variant (RK_VALUE_PHASE; Eq. offonline's inverse output RoPE and
Algorithm 2's RestorePhase): the value of a key is its whole stored row, attention outputs are 576 wide,
W_uv is [H, 128, 576].  Every stage against the float64 checker in oracle/phase.py on identical seeded
inputs; the stated tolerances (max-abs <= 1e-2, relative L2 <= 5e-3)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import phase
from paper_2609_07008_b200 import synth
from tests.helpers import assert_close, f64, max_abs, oracle_online, to_device

pytestmark = [pytest.mark.gpu, pytest.mark.guard_each_call]

LSE_TOL = {"mandated": 1e-3, "sharp": 5e-3}


@pytest.fixture(scope="module")
def rk():
    from paper_2609_07008_b200 import binding
    return binding


def make(rk, w):
    ctx = rk.Context.from_profile(w.profile, value_phase=True)
    req = ctx.rk_request_create(w.layout.seg_off, w.layout.seg_delta, w.layout.seg_has_artifact, w.prot_rows)
    return ctx, req


def layer(ctx, req, w):
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
    ctx.rk_poll_status()
    return O_g, lse_g, O_l, lse_l, z, y


def check_every_row(rk, w):
    us = w.regime == "sharp"
    rows = np.arange(w.layout.n_rows)
    exp = oracle_online(w, rows, value_phase=True)
    ctx, req = make(rk, w)
    to_device(w)
    O_g, lse_g, O_l, lse_l, z, y = layer(ctx, req, w)
    assert O_g.shape[-1] == 576 and O_l.shape[-1] == 576
    assert_close(f64(O_g)[..., :512], exp["O_g"][..., :512], "O_g latent dims", unit_scale=us)
    assert_close(f64(O_g)[..., 512:], exp["O_g"][..., 512:], "O_g rope dims (RestorePhase and R^-1 applied)", unit_scale=us)
    assert max_abs(f64(lse_g), exp["lse_g"]) <= LSE_TOL[w.regime]
    assert_close(f64(O_l)[..., :512], exp["O_l"][..., :512], "O_l latent dims", unit_scale=us)
    assert_close(f64(O_l)[..., 512:], exp["O_l"][..., 512:], "O_l rope dims", unit_scale=us)
    assert max_abs(f64(lse_l), exp["lse_l"]) <= LSE_TOL[w.regime]
    assert_close(f64(z), exp["z"], "z", unit_scale=us)
    assert_close(f64(y), exp["y"], "y", unit_scale=us)
    return ctx, req, y


@pytest.mark.parametrize("regime", ["mandated", "sharp"])
def test_phase_layer_tiny(rk, regime):
    check_every_row(rk, synth.make_workload("tiny", regime=regime, value_phase=True))


@pytest.mark.parametrize("seed", range(10))
def test_phase_irregular_requests_every_row(rk, seed):
    """Segment lengths on and around tile boundaries, length-1 segments, gaps, shuffled order, uncached
    segments in the middle: many segment switches per row tile, each of which turns the rope accumulator."""
    w = synth.make_random_request(seed, value_phase=True)
    ctx, req, y = check_every_row(rk, w)
    # the host-buffer entry point gives the same bits
    bufs = ctx.alloc_layer_buffers(req, "cuda")
    pin = lambda t: t.cpu().pin_memory()
    y_h = torch.empty((w.layout.n_rows, w.profile.d_model), dtype=torch.bfloat16).pin_memory()
    ctx.rk_layer_host(req, pin(w.kv), pin(w.q_g), pin(w.q_l), pin(w.z_off), w.w_uv, w.w_a, w.w_b, bufs, y_h)
    ctx.rk_poll_status()
    assert torch.equal(y_h, y.cpu())


def test_phase_large_offsets_and_gaps(rk):
    """Offsets beyond 2^20 and gaps between segments: the angle (delta - pos) theta is reduced in double."""
    w = synth.make_custom([300, 200], 40, n_heads=16, n_groups=2, o_rank=128, d_model=256, pct_bp=1000, seed=31,
                          base_delta=(1 << 20) + 12345, value_phase=True)
    check_every_row(rk, w)


@pytest.mark.parametrize("name, regime", [("flash1", "mandated"), ("flash1", "sharp"), ("flash256k", "sharp")])
def test_phase_full_size_sampled_rows(rk, name, regime):
    """Full-size layers of the variant in the launch configuration `bench.py --value-phase` times (flash256k is its
    workload); sampled rows against the checker."""
    prof, lay, prot = synth.make_geometry(name)
    w = synth.make_tensors(name, prof, lay, prot, synth.CONFIGS[name]["seed"] * 1000, device="cuda", regime=regime,
                           value_phase=True)
    ctx, req = make(rk, w)
    O_g, lse_g, O_l, lse_l, z, y = layer(ctx, req, w)
    cand = synth.sample_rows(lay, prot, 16, w.seed, max_docs=3)
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    inv = oracle.inverse_row_map(prot, lay.n_rows)
    rows, used = [], 0
    for r in np.random.default_rng(3).permutation(cand):
        c = (int(pos[r]) + 1) * (prof.n_heads if inv[r] >= 0 else prof.n_groups)
        if used + c > (3e7 if name == "flash1" else 6e7) and len(rows) >= 4:
            continue
        rows.append(int(r))
        used += c
    rows = np.sort(np.asarray(rows, dtype=np.int64))
    ridx = torch.as_tensor(rows, device="cuda")
    ql = {int(r): f64(w.q_l[int(inv[r])]) for r in rows if inv[r] >= 0}
    zo = {int(r): f64(w.z_off[int(r)]) for r in rows if inv[r] < 0}
    exp = phase.mla_online_rows_phase(rows, f64(w.q_g[ridx]), ql, f64(w.kv), lay.seg_off, lay.seg_delta, prot,
                                      prof.global_heads, prof.local_heads, f64(w.w_uv), f64(w.w_a), f64(w.w_b), zo,
                                      prof.sm_scale, prof.rope_base, prof.d_latent)
    us = regime == "sharp"
    assert_close(f64(O_g[ridx]), exp["O_g"], "O_g", unit_scale=us)
    assert_close(f64(O_g[ridx])[..., 512:], exp["O_g"][..., 512:], "O_g rope dims", unit_scale=us)
    assert max_abs(f64(lse_g[ridx]), exp["lse_g"]) <= LSE_TOL[regime]
    slots = torch.as_tensor(inv[rows][inv[rows] >= 0], device="cuda")
    assert_close(f64(O_l[slots]), exp["O_l"], "O_l", unit_scale=us)
    assert_close(f64(z[ridx]), exp["z"], "z", unit_scale=us)
    assert_close(f64(y[ridx]), exp["y"], "y", unit_scale=us)
    assert torch.isfinite(y.float()).all()


def test_phase_offline_build_then_online_chain(rk):
    """rk_mla_off_build in the variant (documents alone, R^-1 at the canonical position) against the checker,
    then the GPU-built artifact through the online layer: the document placed first is reused exactly."""
    w = synth.make_workload("tiny", regime="sharp", with_q_all=True, value_phase=True)
    p, lay = w.profile, w.layout
    ctx, req = make(rk, w)
    n = lay.n_doc_rows
    q_all = f64(w.q_all)
    want = np.zeros((n, p.n_groups * p.o_rank))
    for i in range(lay.n_segs):
        if lay.seg_has_artifact[i]:
            lo, hi = int(lay.seg_off[i]), int(lay.seg_off[i + 1])
            want[lo:hi] = phase.mla_off_artifact_phase(i, q_all[lo:hi][:, p.local_heads], f64(w.kv), lay.seg_off,
                                                       lay.seg_delta, p.local_heads, f64(w.w_uv), f64(w.w_a),
                                                       p.sm_scale, p.rope_base, p.d_latent)
    lh = torch.as_tensor(p.local_heads.astype(np.int64))
    q_l_doc = w.q_all[:n][:, lh].contiguous().cuda()
    to_device(w)
    z_off = ctx.rk_mla_off_build(req, w.kv, 0, n, q_l_doc, w.w_uv, w.w_a)
    ctx.rk_poll_status()
    assert_close(f64(z_off), want, "z_off (variant)", unit_scale=True)
    w.z_off = z_off
    _, _, _, _, z, y = layer(ctx, req, w)
    rows = np.arange(lay.n_rows)
    _, y_full = phase.full_recompute_rows_phase(rows, q_all, f64(w.kv), lay.seg_off, lay.seg_delta, f64(w.w_uv),
                                                f64(w.w_a), f64(w.w_b), p.sm_scale, p.rope_base, p.d_latent)
    first = int(np.argmin(lay.seg_delta[:lay.n_segs - 1]))
    lo, hi = int(lay.seg_off[first]), int(lay.seg_off[first + 1])
    assert_close(f64(y[lo:hi]), y_full[lo:hi], "first document rows vs full recomputation", unit_scale=True)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_segmented_merge_phase(rk, dtype):
    """Standalone merge with RestorePhase per part and R^-1 per row against the checker; empty parts with
    garbage O are ignored; without row positions the result stays in the request frame."""
    w = synth.make_random_request(4, value_phase=True)
    ctx, req = make(rk, w)
    lay = w.layout
    S = lay.n_segs
    g = torch.Generator().manual_seed(7)
    n_rows, n_heads = 29, 3
    seg_begin, P = 1, S - 1
    O_part = torch.randn((P, n_rows, n_heads, 576), generator=g).to(dtype)
    lse_part = torch.randn((P, n_rows, n_heads), generator=g) * 2
    lse_part[torch.rand((P, n_rows, n_heads), generator=g) < 0.25] = -float("inf")
    lse_part[:, 0, 0] = -float("inf")
    O_part[0, 1, 1] = float("nan")
    lse_part[0, 1, 1] = -float("inf")
    row_pos = torch.randint(0, 1 << 21, (n_rows,), generator=g, dtype=torch.int32)
    O, lse = ctx.rk_segmented_merge_phase(req, seg_begin, O_part.cuda(), lse_part.cuda(), row_pos.cuda())
    O2, _ = ctx.rk_segmented_merge_phase(req, seg_begin, O_part.cuda(), lse_part.cuda(), None)
    ctx.rk_poll_status()
    deltas = lay.seg_delta[seg_begin:seg_begin + P]
    want_O, want_lse = phase.segmented_merge_phase(f64(O_part), f64(lse_part), deltas, row_pos.numpy(), 512,
                                                   w.profile.rope_base)
    want_O2, _ = phase.segmented_merge_phase(f64(O_part), f64(lse_part), deltas, None, 512, w.profile.rope_base)
    fin = np.isfinite(want_lse)
    assert np.array_equal(np.isneginf(f64(lse)), np.isneginf(want_lse))
    assert max_abs(f64(lse)[fin], want_lse[fin]) <= 1e-3
    assert_close(f64(O), want_O, "merged O with part phases and R^-1", unit_scale=True)
    assert_close(f64(O2), want_O2, "merged O in the request frame", unit_scale=True)


def test_phase_layer_stack_host_matches_device_path(rk):
    """Three independent layers of the variant through the stack entry point with cross-layer prefetch:
    bit-identical to the call-by-call device path."""
    layers, want = [], []
    ctx = None
    for l in range(3):
        prof, lay, prot = synth.make_geometry("tiny", layer=l)
        prot = synth.draw_protected_rows(lay, 300 + 300 * l, np.random.default_rng(200 + l))
        w = synth.make_tensors("tiny", prof, lay, prot, 700 + l, regime="sharp", value_phase=True)
        if ctx is None:
            ctx = rk.Context.from_profile(prof, value_phase=True)
        req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)
        pin = lambda t: t.cpu().pin_memory()
        host = dict(req=req, kv=pin(w.kv), q_g=pin(w.q_g), q_l=pin(w.q_l), z_off=pin(w.z_off))
        to_device(w)
        _, _, _, _, _, y = layer(ctx, req, w)
        want.append(y.cpu())
        host.update(W_uv=w.w_uv, W_a=w.w_a, W_b=w.w_b,
                    y=torch.full((lay.n_rows, prof.d_model), float("nan"), dtype=torch.bfloat16).pin_memory())
        layers.append(host)
    big = max(layers, key=lambda l: l["req"].A)["req"]
    b0, b1 = ctx.alloc_layer_buffers(big, "cuda"), ctx.alloc_layer_buffers(big, "cuda")
    rk.rk_layer_stack_host(ctx, layers, b0, b1)
    ctx.rk_poll_status()
    for l in range(3):
        assert torch.equal(layers[l]["y"], want[l]), f"layer {l}"
