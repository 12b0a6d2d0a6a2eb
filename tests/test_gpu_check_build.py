"""The bounds-checked build of the library (-DRK_CHECK: every index derived from a request table is tested on
the device and reported through the status word instead of being used) on the small parity cases: the same
results as the ordinary build, no index report -- and its self-test, which pushes one bad index through the
check and must see RK_ERR_ROWS.  A stand-in for a memory checker; runs in a child process because a process
loads one build of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import numpy as np, torch, sys
sys.path.insert(0, %(root)r)
from paper_2609_07008_b200 import binding as rk, synth
from oracle import policy
from tests.helpers import assert_close, f64, oracle_online, to_device
assert rk.lib._name.endswith("librk_check.so")
ctx = None
for seed in (0, 3, 7):
    for phase in (False, True):
        w = synth.make_random_request(seed, value_phase=phase)
        exp = oracle_online(w, np.arange(w.layout.n_rows), value_phase=phase)
        ctx = rk.Context.from_profile(w.profile, value_phase=phase)
        req = ctx.rk_request_create(w.layout.seg_off, w.layout.seg_delta, w.layout.seg_has_artifact, w.prot_rows)
        to_device(w)
        O_g, lse_g, O_l, lse_l = ctx.rk_mla_online_attn(req, w.kv, w.q_g, w.q_l)
        z_on_g, z_on_l = ctx.rk_group_sliced_proj(req, O_g, O_l, w.w_uv, w.w_a)
        z, y = ctx.rk_combine_offline(req, z_on_g, z_on_l, w.z_off, w.w_b)
        ctx.rk_poll_status()                      # raises on an index report (RK_ERR_ROWS) or a timeout
        assert_close(f64(y), exp["y"], "y", unit_scale=True)
lay = w.layout
dirty, scores = synth.draw_policy_inputs(lay, seed=1, n_dirty=8)
out = ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, torch.from_numpy(dirty).cuda(),
                            torch.from_numpy(scores).cuda(), edge_rows=16, tail_rows=100, budget_bp=2500)
ctx.rk_poll_status()
want = policy.protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, dirty, scores, edge_rows=16, tail_rows=100,
                             budget_bp=2500)
assert np.array_equal(ctx.protected_rows_to_host(out), want)
ctx.rk_check_selftest()
try:
    ctx.rk_poll_status()
    raise SystemExit("the self-test's bad index was not reported")
except rk.RKError as e:
    assert e.status == 4 and "index check failed" in str(e), str(e)
ctx.rk_poll_status()                              # cleared; the context stays usable
print("check build ok")
'''


def test_small_cases_on_the_bounds_checked_build():
    from paper_2609_07008_b200 import build
    path = build.build_library(check=True)
    env = dict(os.environ, RK_LIBRARY_PATH=path)
    r = subprocess.run([sys.executable, "-c", CHILD % dict(root=ROOT)], capture_output=True, text=True, timeout=900,
                       env=env, cwd=ROOT)
    assert r.returncode == 0 and "check build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_ordinary_build_has_no_index_checks():
    from paper_2609_07008_b200 import binding as rk, synth
    prof, lay, prot = synth.make_geometry("tiny")
    ctx = rk.Context.from_profile(prof)
    with pytest.raises(rk.RKError) as ei:
        ctx.rk_check_selftest()
    assert ei.value.status == 7
