"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The float64 checker cannot evaluate O(T^2) work at these sizes, so the tests use (a) a seeded
sample of rows that it computes one by one, and (b) properties that hold at any size and cost
O(T) on the CPU: the zero-query closed form (lse = log(#visible keys), O = running mean of the
latent in request order), the rope-only Toeplitz closed form for relocation, and metamorphic
relations between two GPU runs (packed-order permutation, document split)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_07008_b200 import synth
from tests.helpers import assert_close, f64, max_abs, oracle_online, rel_l2, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rk():
    from paper_2609_07008_b200 import binding
    return binding


def make(rk, prof, lay, prot):
    ctx = rk.Context.from_profile(prof)
    req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)
    return ctx, req


def sample_within_budget(w, budget_pairs, n_random=24):
    """Segment-edge rows + seeded random rows whose visible-pair total fits the checker's budget."""
    lay, p = w.layout, w.profile
    cand = synth.sample_rows(lay, w.prot_rows, n_random, w.seed, max_docs=3)
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    inv = oracle.inverse_row_map(w.prot_rows, lay.n_rows)
    order = np.random.default_rng(w.seed).permutation(len(cand))
    rows, used = [], 0
    for r in cand[order]:
        c = (int(pos[r]) + 1) * (p.n_heads if inv[r] >= 0 else p.n_groups)
        if used + c > budget_pairs and len(rows) >= 4:
            continue
        rows.append(int(r))
        used += c
    return np.sort(np.asarray(rows, dtype=np.int64))


# flash32k draws its own protected rows per layer: layer 0 (2.7 % of the document rows), layer 1 (2.06 %, the
# smallest share of the 37) and layer 9 (4.72 %, the largest)
@pytest.mark.parametrize("name, regime, budget, layer", [
    ("flash1", "mandated", 4e7, 0), ("flash1", "sharp", 4e7, 0),
    ("flash32k", "mandated", 4e7, 0), ("flash32k", "sharp", 4e7, 0), ("flash32k", "mandated", 4e7, 1),
    ("flash32k", "sharp", 4e7, 9),
    ("flash256k", "mandated", 6e7, 0), ("flash256k", "sharp", 6e7, 0),
    ("pro128k", "mandated", 6e7, 0), ("pro128k", "sharp", 6e7, 0), ("flash440k", "mandated", 8e7, 0),
])
def test_full_size_layer_on_sampled_rows(rk, name, regime, budget, layer):
    """Whole layer (the three calls bench.py times) at full size; sampled rows against the checker."""
    prof, lay, prot = synth.make_geometry(name, layer=layer)
    w = synth.make_tensors(name, prof, lay, prot, synth.CONFIGS[name]["seed"] * 1000 + layer, device="cuda", regime=regime)
    ctx, req = make(rk, prof, lay, prot)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
    z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
    z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
    ctx.rk_poll_status()
    rows = sample_within_budget(w, budget)
    ridx = torch.as_tensor(rows, device="cuda")
    inv = oracle.inverse_row_map(prot, lay.n_rows)
    # the checker gets only what it needs of the big tensors
    ql = {int(r): f64(w.q_l[int(inv[r])]) for r in rows if inv[r] >= 0}
    zo = {int(r): f64(w.z_off[int(r)]) for r in rows if inv[r] < 0}
    exp = oracle.mla_online_rows(rows, f64(w.q_g[ridx]), ql, f64(w.kv), lay.seg_off, lay.seg_delta, prot,
                                 prof.global_heads, prof.local_heads, f64(w.w_uv), f64(w.w_a), f64(w.w_b), zo,
                                 prof.sm_scale, prof.rope_base, prof.d_latent)
    lse_tol = 1e-3 if regime == "mandated" else 5e-3
    assert_close(f64(O_g[ridx]), exp["O_g"], "O_g", unit_scale=w.regime == "sharp")
    assert max_abs(f64(lse_g[ridx]), exp["lse_g"]) <= lse_tol
    slots = torch.as_tensor(inv[rows][inv[rows] >= 0], device="cuda")
    if len(slots):
        assert_close(f64(O_l[slots]), exp["O_l"], "O_l", unit_scale=w.regime == "sharp")
        assert max_abs(f64(lse_l[slots]), exp["lse_l"]) <= lse_tol
    assert_close(f64(z[ridx]), exp["z"], "z", unit_scale=w.regime == "sharp")
    assert_close(f64(y[ridx]), exp["y"], "y", unit_scale=w.regime == "sharp")
    # rows outside the sample: finite, and O inside the convex hull of the latent values
    assert torch.isfinite(y.float()).all() and torch.isfinite(lse_g).all() and torch.isfinite(lse_l).all()
    cmax = w.kv[:, :512].float().abs().max().item()
    assert O_g.float().abs().max().item() <= cmax * 1.01 and O_l.float().abs().max().item() <= cmax * 1.01
    # selection is bit-exact: unprotected rows take z_off, protected rows take z_on_l
    un = torch.as_tensor(np.nonzero(inv < 0)[0][:: max(1, lay.n_rows // 4096)], device="cuda")
    want = (z_on_g[un].float() + w.z_off[un].float()).to(torch.bfloat16)
    assert torch.equal(z[un], want)
    pr = torch.as_tensor(prot.astype(np.int64), device="cuda")
    want = (z_on_g[pr].float() + z_on_l.float()).to(torch.bfloat16)
    assert torch.equal(z[pr], want)


@pytest.mark.parametrize("name", ["flash1", "flash32k", "flash256k"])
def test_zero_query_closed_form_every_row(rk, name):
    """q = 0: every visible key gets the same weight, so lse = log(pos + 1) for a gap-free layout and
    O is the running mean of the latent in request order.  Any masking, segment-visibility, tile-edge
    or row-map error changes an integer count and shows in lse."""
    prof, lay, prot = synth.make_geometry(name)
    T, A = lay.n_rows, len(prot)
    g = torch.Generator(device="cuda").manual_seed(11)
    kv = (torch.randn((T, 576), generator=g, device="cuda")).to(torch.bfloat16)
    q_g = torch.zeros((T, prof.n_groups, 576), dtype=torch.bfloat16, device="cuda")
    q_l = torch.zeros((A, prof.n_local, 576), dtype=torch.bfloat16, device="cuda")
    ctx, req = make(rk, prof, lay, prot)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, kv, q_g, q_l)
    ctx.rk_poll_status()
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    order = np.argsort(pos, kind="stable")
    assert np.array_equal(pos[order], np.arange(T))                     # gap-free
    c = f64(kv[:, :512])
    run_mean = np.cumsum(c[order], axis=0) / (np.arange(T) + 1.0)[:, None]   # indexed by position
    want_lse = np.log(pos + 1.0)
    got = f64(lse_g)
    assert np.max(np.abs(got - want_lse[:, None])) <= 2e-4
    got_l = f64(lse_l)
    assert np.max(np.abs(got_l - want_lse[prot][:, None])) <= 2e-4
    # O on a strided subset of rows (all heads are identical here)
    sel = np.arange(0, T, max(1, T // 2048))
    Og = f64(O_g[torch.as_tensor(sel, device="cuda")])
    for h in range(prof.n_groups):
        assert rel_l2(Og[:, h], run_mean[pos[sel]]) <= 5e-3
    Ol = f64(O_l)
    assert rel_l2(Ol[:, 0], run_mean[pos[prot]]) <= 5e-3 and rel_l2(Ol[:, -1], run_mean[pos[prot]]) <= 5e-3


def test_rope_only_toeplitz_closed_form(rk):
    """Relocation at full scale (ragged 32K layout): q carries only a rope part R(pos) a_h and every key
    only R(canonical index) b, so a score depends on the request-position distance alone,
    s = sm_scale f_h(pos_t - pos_k) with f_h(d) = <R(d) a_h, b>, and lse[t, h] =
    log cumsum_d exp(sm_scale f_h(d)) at d = pos[t].  A wrong delta, sign, pairing or a stale rotated
    tile after a segment switch changes lse by about the logit spread (0.6 here).  Tolerance 1e-2: the
    test's own bf16 rounding of the rotated q and k moves a logit by about 1e-3 rms (64 terms of
    magnitude 1 x 2^-9 x sm_scale), a few times that at the maximum over 3e5 entries."""
    prof, lay, prot = synth.make_geometry("flash32k")
    T, A, G, L = lay.n_rows, len(prot), prof.n_groups, prof.n_local
    rng = np.random.default_rng(3)
    a = rng.normal(size=(prof.n_heads, 64))
    b = rng.normal(size=64)
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    canon = np.concatenate([np.arange(lay.seg_off[i + 1] - lay.seg_off[i]) for i in range(lay.n_segs)])
    kv = np.zeros((T, 576))
    kv[:, :512] = rng.normal(size=(T, 512))
    kv[:, 512:] = oracle.rope_rotate(np.broadcast_to(b, (T, 64)), canon, prof.rope_base)
    kv_t = torch.from_numpy(kv).to(torch.bfloat16).cuda()

    def rotated(heads, positions):            # [len(positions), len(heads), 576] with only the rope part set
        out = np.zeros((len(positions), len(heads), 576), dtype=np.float32)
        for j, h in enumerate(heads):
            out[:, j, 512:] = oracle.rope_rotate(np.broadcast_to(a[h], (len(positions), 64)), positions,
                                                 prof.rope_base)
        return torch.from_numpy(out).to(torch.bfloat16).cuda()

    q_g = rotated(prof.global_heads, pos)
    q_l = rotated(prof.local_heads, pos[prot])
    ctx, req = make(rk, prof, lay, prot)
    O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, kv_t, q_g, q_l)
    ctx.rk_poll_status()
    d = np.arange(T)
    f = np.stack([oracle.rope_rotate(np.broadcast_to(a[h], (T, 64)), d, prof.rope_base) @ b
                  for h in range(prof.n_heads)], axis=1)                             # f_h(d), [d, h]
    cum = np.log(np.cumsum(np.exp(prof.sm_scale * f), axis=0))                       # [d, h]
    want_g = cum[pos][:, prof.global_heads]
    want_l = cum[pos[prot]][:, prof.local_heads]
    assert np.max(np.abs(f64(lse_g) - want_g)) <= 1e-2
    assert np.max(np.abs(f64(lse_l) - want_l)) <= 1e-2


def _mid_workload(seed=31):
    return synth.make_custom([1500, 700, 2300, 1111], 300, n_heads=16, n_groups=2, o_rank=256, d_model=512,
                             pct_bp=400, seed=seed, regime="sharp", device="cuda")


def test_packed_order_permutation_gpu_vs_gpu(rk):
    """Moving documents inside the packed stream while each keeps its request offset leaves every
    token's output unchanged (within twice the rounding tolerance)."""
    w = _mid_workload()
    lay = w.layout
    ctx, req = make(rk, w.profile, lay, w.prot_rows)
    O1, l1, _, _ = ctx.rk_mla_online_attn(req, w.kv, w.q_g, None)
    D = lay.n_segs - 1
    perm = [2, 0, 3, 1]
    lens = [int(lay.seg_off[i + 1] - lay.seg_off[i]) for i in range(D + 1)]
    new_rows = np.concatenate([np.arange(lay.seg_off[i], lay.seg_off[i + 1]) for i in perm] +
                              [np.arange(lay.seg_off[D], lay.n_rows)])
    lay2 = synth.Layout(seg_off=np.concatenate([[0], np.cumsum([lens[i] for i in perm] + [lens[D]])]).astype(np.int64),
                        seg_delta=np.concatenate([lay.seg_delta[perm], lay.seg_delta[D:]]),
                        seg_has_artifact=lay.seg_has_artifact.copy())
    inv_new = np.empty(lay.n_rows, dtype=np.int64)
    inv_new[new_rows] = np.arange(lay.n_rows)
    prot2 = np.sort(inv_new[w.prot_rows]).astype(np.int32)
    idx = torch.as_tensor(new_rows, device="cuda")
    ctx2, req2 = make(rk, w.profile, lay2, prot2)
    O2, l2, _, _ = ctx2.rk_mla_online_attn(req2, w.kv[idx].contiguous(), w.q_g[idx].contiguous(), None)
    ctx2.rk_poll_status()
    assert rel_l2(f64(O2), f64(O1[idx])) <= 1e-2
    assert max_abs(f64(l2), f64(l1[idx])) <= 1e-2


def test_document_split_gpu_vs_gpu(rk):
    """A document cut into two adjacent segments (second half re-based to canonical positions and
    offset by the first half's length) gives the same result as the unsplit document: exercises
    relocation + merge."""
    w = _mid_workload(seed=32)
    lay, p = w.layout, w.profile
    ctx, req = make(rk, p, lay, w.prot_rows)
    O1, l1, _, _ = ctx.rk_mla_online_attn(req, w.kv, w.q_g, None)
    cut_seg, cut = 2, 1000                        # split document 2 after 1000 tokens
    lo = int(lay.seg_off[cut_seg])
    seg_off = np.insert(lay.seg_off, cut_seg + 1, lo + cut)
    seg_delta = np.insert(lay.seg_delta, cut_seg + 1, lay.seg_delta[cut_seg] + cut)
    has = np.insert(lay.seg_has_artifact, cut_seg + 1, 1)
    kv2 = w.kv.clone()
    hi = int(lay.seg_off[cut_seg + 1])
    k_r = f64(w.kv[lo + cut:hi, 512:])
    kv2[lo + cut:hi, 512:] = torch.from_numpy(oracle.rope_rotate(k_r, -float(cut), p.rope_base)).to(torch.bfloat16).cuda()
    lay2 = synth.Layout(seg_off=seg_off.astype(np.int64), seg_delta=seg_delta.astype(np.int64),
                        seg_has_artifact=has.astype(np.uint8))
    ctx2, req2 = make(rk, p, lay2, w.prot_rows)
    O2, l2, _, _ = ctx2.rk_mla_online_attn(req2, kv2, w.q_g, None)
    ctx2.rk_poll_status()
    assert rel_l2(f64(O2), f64(O1)) <= 1e-2
    assert max_abs(f64(l2), f64(l1)) <= 1e-2


def test_offline_artifact_build_full_size_sampled_rows(rk):
    """rk_mla_off_build over all 32 768 document rows of the flash1 layout (built in two row ranges);
    sampled rows of three documents against the checker's position-zero artifact."""
    prof, lay, prot = synth.make_geometry("flash1")
    n, L = lay.n_doc_rows, prof.n_local
    g = torch.Generator(device="cuda").manual_seed(77)
    kv = torch.randn((lay.n_rows, 576), generator=g, device="cuda").to(torch.bfloat16)
    q_l_doc = (torch.randn((n, L, 576), generator=g, device="cuda") * 1.2).to(torch.bfloat16)
    w_uv = (torch.randn((prof.n_heads, 128, 512), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    w_a = (torch.randn((prof.n_groups, prof.o_rank, 1024), generator=g, device="cuda") * 0.02).to(torch.bfloat16)
    ctx, req = make(rk, prof, lay, prot)
    half = 5 * 4096 + 1234
    z_off = torch.cat([ctx.rk_mla_off_build(req, kv, 0, half, q_l_doc[:half].contiguous(), w_uv, w_a),
                       ctx.rk_mla_off_build(req, kv, half, n, q_l_doc[half:].contiguous(), w_uv, w_a)])
    ctx.rk_poll_status()
    assert torch.isfinite(z_off.float()).all()
    kv64, wuv, wa = f64(kv), f64(w_uv), f64(w_a)
    for seg in (0, 5, 7):                      # document 5 is the one cut by the two row ranges
        lo = int(lay.seg_off[seg])
        canon = np.array([0, 1, 127, 128, 129, 255, 256, 257, 1233, 1234, 1235, 2047, 4094, 4095])
        want = oracle.mla_off_artifact(seg, f64(q_l_doc[torch.as_tensor(lo + canon, device="cuda")]), kv64, lay.seg_off,
                                       lay.seg_delta, prof.local_heads, wuv, wa, prof.sm_scale, prof.rope_base,
                                       prof.d_latent, rows=canon)
        assert_close(f64(z_off[torch.as_tensor(lo + canon, device="cuda")]), want, f"z_off rows of document {seg}", unit_scale=True)



def test_full_size_layer_pair_through_the_stack_entry_point(rk):
    """Two flash32k layers with different protected sets (layers 1 and 9: the smallest and the largest share)
    through rk_layer_stack_host from pinned host buffers; sampled rows of both against the checker."""
    layers, ws = [], []
    ctx = None
    for l in (1, 9):
        prof, lay, prot = synth.make_geometry("flash32k", layer=l)
        w = synth.make_tensors("flash32k", prof, lay, prot, 2000 + l, device="cuda", regime="sharp")
        if ctx is None:
            ctx = rk.Context.from_profile(prof)
        req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)
        pin = lambda t: t.cpu().pin_memory()
        layers.append(dict(req=req, kv=pin(w.kv), q_g=pin(w.q_g), q_l=pin(w.q_l), z_off=pin(w.z_off), W_uv=w.w_uv,
                           W_a=w.w_a, W_b=w.w_b,
                           y=torch.full((lay.n_rows, prof.d_model), float("nan"), dtype=torch.bfloat16).pin_memory()))
        ws.append(w)
    big = max(layers, key=lambda l: l["req"].A)["req"]
    b0, b1 = ctx.alloc_layer_buffers(big, "cuda"), ctx.alloc_layer_buffers(big, "cuda")
    rk.rk_layer_stack_host(ctx, layers, b0, b1)
    ctx.rk_poll_status()
    for w, l in zip(ws, layers):
        assert torch.isfinite(l["y"].float()).all()
        rows = sample_within_budget(w, 3e7)
        exp = oracle_online(w, rows)
        assert_close(f64(l["y"][torch.as_tensor(rows)]), exp["y"], "y of a stacked layer", unit_scale=True)
