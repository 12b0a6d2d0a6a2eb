"""CPU-side checks of the C ABI: the shared library loads and exports every symbol that
include/rk.h declares, and the host-side validation returns the documented status codes
without touching a device.  No compute call is made here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rk():
    from paper_2609_07008_b200 import build
    build.build_library()
    from paper_2609_07008_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rk_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(rk):
    syms = declared_symbols()
    assert len(syms) >= 18 and "rk_mla_online_attn" in syms
    for s in syms:
        assert hasattr(rk.lib, s), f"librk.so does not export {s}"
    assert sorted(rk.EXPORTS) == syms
    assert b"sm_100a" in rk.lib.rk_version()
    assert rk.lib.rk_status_string(9) == b"RK_ERR_TIMEOUT"


def good_layout():
    return dict(seg_off=[0, 5, 12, 15], seg_delta=[7, 0, 12], seg_has_artifact=[1, 1, 0], prot_rows=[3, 12, 13, 14])


@pytest.mark.parametrize("change, status", [
    ({}, 0),
    (dict(seg_off=[1, 5, 12, 15]), 3),                      # seg_off[0] != 0
    (dict(seg_off=[0, 5, 5, 15]), 3),                       # empty segment
    (dict(seg_delta=[7, 0, 10]), 3),                        # request intervals overlap
    (dict(seg_delta=[7, -1, 12]), 3),                       # negative offset
    (dict(seg_delta=[7, 0, 1 << 31]), 3),                   # position overflow
    (dict(prot_rows=[3, 12, 13]), 4),                       # query-suffix row 14 unprotected
    (dict(prot_rows=[12, 3, 13, 14]), 4),                   # not ascending
    (dict(prot_rows=[3, 3, 12, 13, 14]), 4),                # duplicate
    (dict(prot_rows=[3, 12, 13, 14, 15]), 4),               # out of range
    (dict(seg_delta=[20, 0, 12]), 0),                       # gaps between segments are legal
])
def test_check_request_status_codes(rk, change, status):
    a = good_layout()
    a.update(change)
    s, msg = rk.rk_check_request(a["seg_off"], a["seg_delta"], a["seg_has_artifact"], a["prot_rows"])
    assert s == status, msg
    assert (msg == "") == (status == 0)


def test_check_request_null_arguments(rk):
    assert rk.lib.rk_check_request(None, None, 0, None, 0) == 1


def profile_struct(rk, **kw):
    base = dict(n_heads=16, n_groups=2, group_size=8, d_latent=512, d_rope=64, d_v=128, o_rank=256, d_model=1024,
                sm_scale=0.07, rope_base=10000.0)
    gh = np.asarray(kw.pop("global_heads", [3, 9]), dtype=np.int32)
    base.update(kw)
    p = rk.rk_profile(base["n_heads"], base["n_groups"], base["group_size"], base["d_latent"], base["d_rope"],
                      base["d_v"], base["o_rank"], base["d_model"], base["sm_scale"], base["rope_base"],
                      gh.ctypes.data_as(C.POINTER(C.c_int32)))
    return p, gh


@pytest.mark.parametrize("kw, status", [
    (dict(n_heads=17), 2),                    # H != 8 G
    (dict(global_heads=[3, 4]), 2),           # two Global heads in group 0, none in group 1
    (dict(global_heads=[3, 16]), 2),          # out of range
    (dict(sm_scale=0.0), 2),
    (dict(d_latent=256), 7),                  # unsupported dims
    (dict(group_size=4, n_heads=8), 7),
    (dict(o_rank=100), 7),
])
def test_create_rejects_bad_profiles_before_touching_the_device(rk, kw, status):
    p, keep = profile_struct(rk, **kw)
    h = C.c_void_p()
    assert rk.lib.rk_create(C.byref(p), C.byref(h)) == status
    assert not h.value


def test_create_null(rk):
    h = C.c_void_p()
    assert rk.lib.rk_create(None, C.byref(h)) == 1
    assert rk.lib.rk_destroy(None) == 1
    assert rk.lib.rk_request_destroy(None) == 1
    assert rk.lib.rk_last_error(None) == b"null context"


def test_create_ex_rejects_unknown_flags_and_null_calls_of_the_variant(rk):
    p, keep = profile_struct(rk)
    h = C.c_void_p()
    assert rk.lib.rk_create_ex(C.byref(p), 2, C.byref(h)) == 7          # only RK_VALUE_PHASE (1) is defined
    assert rk.lib.rk_create_ex(C.byref(p), 0xFFFFFFFE, C.byref(h)) == 7
    assert not h.value
    assert rk.lib.rk_create_ex(None, 1, C.byref(h)) == 1
    assert rk.lib.rk_segmented_merge_phase(None, None, 0, 1, 1, 1, None, 0, None, None, None, None, None) == 1
    assert rk.lib.rk_check_selftest(None, None) == 1
    assert rk.lib.rk_test_starve_loads(None, 1) == 1
