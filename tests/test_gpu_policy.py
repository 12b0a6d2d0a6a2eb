"""GPU parity of the selection rules: the protected-row set (Eq. protected) and the expert fan-out
(Eq. moe) through the C ABI against the CPU checker on identical seeded inputs.  Both end in
integers: the comparison is bit-exact."""
import os

import numpy as np
import pytest
import torch

from oracle import policy
from paper_2609_07008_b200 import synth
from tests.test_oracle_policy_pins import read_example, read_moe_examples

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rk():
    from paper_2609_07008_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(rk):
    return rk.Context.from_profile(synth.make_workload("tiny").profile)


def run_rows(ctx, lay, dirty, scores, **kw):
    d = None if dirty is None else torch.from_numpy(np.ascontiguousarray(dirty, dtype=np.int32)).cuda()
    s = None if scores is None else torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).cuda()
    out = ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, d, s, **kw)
    got = ctx.protected_rows_to_host(out)
    ctx.rk_poll_status()
    return got


class Lay:
    def __init__(self, seg_off, seg_delta, has):
        self.seg_off, self.seg_delta, self.seg_has_artifact = seg_off, seg_delta, has


def test_hand_worked_request(ctx):
    seg_off, seg_delta, has, edge, tail, dirty, cases = read_example()
    scores = np.array([(7 * t) % 11 for t in range(seg_off[-1])], dtype=np.float32)
    for bp, want in cases.items():
        got = run_rows(ctx, Lay(seg_off, seg_delta, has), dirty, scores, edge_rows=edge, tail_rows=tail, budget_bp=bp)
        assert got.tolist() == want, bp


@pytest.mark.parametrize("bp", [0, 1000, 2000, 2500])
@pytest.mark.parametrize("name", ["tiny", "ragged", "flash1"])
def test_protected_rows_match_checker(ctx, name, bp):
    if name == "ragged":
        lay = synth.make_custom([300, 77, 513, 1500, 41], 50, n_heads=16, n_groups=2, o_rank=256, d_model=512,
                                pct_bp=700, seed=3).layout
    else:
        lay = synth.make_geometry(name, 0)[1] if name == "flash1" else synth.make_workload("tiny").layout
    edge, tail = (128, 2048) if name == "flash1" else (16, 100)
    dirty, scores = synth.draw_policy_inputs(lay, seed=bp + 7)
    want = policy.protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, dirty, scores, edge_rows=edge,
                                 tail_rows=tail, budget_bp=bp)
    got = run_rows(ctx, lay, dirty, scores, edge_rows=edge, tail_rows=tail, budget_bp=bp)
    assert got.dtype == np.int32 and np.array_equal(got, want)
    # the list is what the request object takes
    req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, got)
    assert req.A == len(want)


def test_protected_rows_edge_cases(ctx):
    lay = Lay([0, 40, 90, 100], [60, 0, 110], [1, 1, 0])            # a gap between position 100 and 110
    dirty = np.array([5, 5, 99, -3, 1000], dtype=np.int32)          # duplicates and out-of-range entries
    for kw in [dict(edge_rows=0, tail_rows=0, budget_bp=0), dict(edge_rows=1000, tail_rows=0, budget_bp=0),
               dict(edge_rows=3, tail_rows=10 ** 9, budget_bp=0), dict(edge_rows=3, tail_rows=25, budget_bp=10000)]:
        ok_dirty = dirty[(dirty >= 0) & (dirty < 100)]
        scores = np.linspace(-1, 1, 100).astype(np.float32)
        want = policy.protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, ok_dirty, scores, **kw)
        got = run_rows(ctx, lay, dirty, scores, **kw)
        assert np.array_equal(got, want), kw
    # no dirty rows, no scores: the budget cannot be filled and is ignored
    got = run_rows(ctx, lay, None, None, edge_rows=2, tail_rows=0, budget_bp=2500)
    assert np.array_equal(got, policy.protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, edge_rows=2, tail_rows=0))
    # a request that is one segment without artifact: every row
    got = run_rows(ctx, Lay([0, 77], [0], [0]), None, None)
    assert np.array_equal(got, np.arange(77))
    # all scores equal: the top-up takes the lowest rows; signed zeros are one value
    z = np.zeros(100, dtype=np.float32)
    z[::2] = -0.0
    got = run_rows(ctx, lay, None, z, edge_rows=0, tail_rows=0, budget_bp=2000)
    assert np.array_equal(got, np.concatenate([np.arange(18), np.arange(90, 100)]))


def test_protected_rows_argument_errors(rk, ctx):
    lay = Lay([0, 40, 90, 100], [60, 0, 110], [1, 1, 0])
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, budget_bp=10001)
    assert ei.value.status == 2
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_protected_rows(lay.seg_off, [60, 0, 80], lay.seg_has_artifact)       # overlapping positions
    assert ei.value.status == 3
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact,
                              workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert ei.value.status == 6


def test_protected_rows_full_size_paper_policy(ctx):
    """The 256K request with the paper's constants (edge 128, tail 32K) and each controller budget."""
    lay = synth.make_geometry("flash256k", 0)[1]
    dirty, scores = synth.draw_policy_inputs(lay, seed=99, n_dirty=500)
    d = torch.from_numpy(dirty).cuda()
    s = torch.from_numpy(scores).cuda()
    for bp in (0, 1000, 2000, 2500):
        want = policy.protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, dirty, scores, budget_bp=bp)
        out = ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, d, s, budget_bp=bp)
        got = ctx.protected_rows_to_host(out)
        assert np.array_equal(got, want), bp
    # at 25 % the budget exceeds what the structural sets protect here, so it is met exactly
    n_cand = int(sum(lay.seg_off[i + 1] - lay.seg_off[i] for i in range(lay.n_segs) if lay.seg_has_artifact[i]))
    assert len(got) - (lay.n_rows - n_cand) == 2500 * n_cand // 10000


@pytest.mark.parametrize("tau", [0.5, 0.7, 0.85, 0.95, 1.0])
def test_moe_fanout_matches_checker(ctx, tau):
    p = synth.draw_router_weights(20011, seed=int(tau * 100))
    k_want, keep_want = policy.moe_fanout(p, tau)
    k, keep = ctx.rk_moe_fanout(torch.from_numpy(p).cuda(), tau)
    ctx.rk_poll_status()
    assert np.array_equal(k.cpu().numpy(), k_want)
    assert np.array_equal(keep.cpu().numpy(), keep_want)


def test_moe_hand_worked_examples(ctx):
    for w, tau, k_want, kept in read_moe_examples():
        k, keep = ctx.rk_moe_fanout(torch.tensor([w], dtype=torch.float32, device="cuda"), tau)
        assert int(k[0]) == k_want and [s for s in range(6) if (int(keep[0]) >> s) & 1] == kept, (w, tau)


def test_moe_fanout_edge_cases(ctx):
    p = synth.draw_router_weights(1000, seed=1)
    dev = torch.from_numpy(p).cuda()
    k, keep = ctx.rk_moe_fanout(dev, 0.8, fence=True)
    assert (k == 6).all() and (keep == 63).all()
    before = dev.clone()
    k, keep = ctx.rk_moe_fanout(dev, 0.0)                      # any three experts reach a zero threshold
    assert (k == 3).all() and torch.equal(dev, before)          # the weights are not touched
    # weights that start 24 bytes into an allocation (8-byte aligned only) and a token count of 4n + 3
    k_all, keep_all = ctx.rk_moe_fanout(dev, 0.8)
    k_off, keep_off = ctx.rk_moe_fanout(dev[1:], 0.8)
    assert torch.equal(k_off, k_all[1:]) and torch.equal(keep_off, keep_all[1:])
    kw, keepw = policy.moe_fanout(p, 0.8)
    assert np.array_equal(k_all.cpu().numpy(), kw) and np.array_equal(keep_all.cpu().numpy(), keepw)
    k0, keep0 = ctx.rk_moe_fanout(torch.empty((0, 6), dtype=torch.float32, device="cuda"), 0.8)
    assert k0.numel() == 0
    geo = torch.tensor([[4, 32, 1, 8, 16, 2]], dtype=torch.float32, device="cuda")
    for tau, k_want in [(0.85, 3), (0.9, 4), (0.96, 5), (0.99, 6)]:
        k, keep = ctx.rk_moe_fanout(geo, tau)
        assert int(k[0]) == k_want and int(keep[0]) == sum(1 << s for s in [1, 4, 3, 0, 5, 2][:k_want])
