"""The allocation-free projection entry point, checked against the ordinary one.

Some users of the library cannot allocate device memory when a request arrives -- their
process gave the whole device to its own pool at start-up, or the request path must not pay
for the device-wide synchronisation an allocation can cause -- so rk_group_sliced_proj_static
keeps its intermediate in a fixed 32 MiB array inside the library instead of a caller
workspace.  This file is collected last on purpose (a run that stops at the first failure has
then already run every other test) and passes both alone in a fresh process and after the
other tests: it depends on nothing they leave behind, and the array it uses keeps stale
contents between calls by design."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_07008_b200 import synth
from tests.helpers import assert_close, f64, to_device

pytestmark = pytest.mark.gpu


def test_static_scratch_projection_matches_workspace_projection_twice():
    from paper_2609_07008_b200 import binding as rk
    w = synth.make_custom([300, 77, 513], 50, n_heads=16, n_groups=2, o_rank=256, d_model=512, pct_bp=700, seed=21)
    ctx = rk.Context.from_profile(w.profile)
    req = ctx.rk_request_create(w.layout.seg_off, w.layout.seg_delta, w.layout.seg_has_artifact, w.prot_rows)
    assert req.workspace_bytes <= 32 * 1024 * 1024
    p, T, A = w.profile, w.layout.n_rows, len(w.prot_rows)
    width = p.n_groups * p.o_rank
    to_device(w)
    for call in range(2):                      # two calls in a row share the built-in array
        g = torch.Generator().manual_seed(100 + call)
        O_g = (torch.randn((T, p.n_groups, 512), generator=g) * 0.5).to(torch.bfloat16).cuda()
        O_l = (torch.randn((A, p.n_local, 512), generator=g) * 0.5).to(torch.bfloat16).cuda()
        want_g, want_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
        z_g = torch.full((T, width), float("nan"), dtype=torch.bfloat16, device="cuda")
        z_l = torch.full((A, width), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        ctx.rk_group_sliced_proj_static(req, O_g, O_l, w.w_uv, w.w_a, z_g, z_l)
        ctx.rk_poll_status()
        assert torch.cuda.mem_get_info()[0] == free_before       # the call took no device memory
        assert_close(f64(z_g), f64(want_g), f"z_on_g, call {call}", unit_scale=True)
        assert_close(f64(z_l), f64(want_l), f"z_on_l, call {call}", unit_scale=True)
        assert torch.equal(z_g, want_g) and torch.equal(z_l, want_l)
        # and against the float64 checker (Eq. offonline: per-head W_uv, then the head's slice of W_a)
        cg = oracle.head_contributions(f64(O_g), p.global_heads, f64(w.w_uv), f64(w.w_a))
        assert_close(f64(z_g), cg.reshape(T, -1), f"z_on_g vs checker, call {call}", unit_scale=True)
        cl = oracle.head_contributions(f64(O_l), p.local_heads, f64(w.w_uv), f64(w.w_a))
        want = np.zeros((A, p.n_groups, p.o_rank))
        for a, h in enumerate(p.local_heads):
            want[:, h // 8] += cl[:, a]
        assert_close(f64(z_l), want.reshape(A, -1), f"z_on_l vs checker, call {call}", unit_scale=True)


def test_static_scratch_rejects_requests_beyond_its_size():
    from paper_2609_07008_b200 import binding as rk
    prof, lay, prot = synth.make_geometry("flash1")       # needs about 100 MB of scratch
    ctx = rk.Context.from_profile(prof)
    req = ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)
    assert req.workspace_bytes > 32 * 1024 * 1024
    dummy = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_group_sliced_proj_static(req, dummy, dummy, dummy, dummy, dummy, dummy)
    assert ei.value.status == 6 and "33554432" in str(ei.value)
