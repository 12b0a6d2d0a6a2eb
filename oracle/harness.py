"""Bridge between torch tensors of a synthetic workload and the float64 checker's arguments, plus
the two error measures the parity criteria are stated in.  Test infrastructure like the rest of
this package: used by tests/, by the smoke check and by the benchmark's cpu_baseline / reference
legs, never by the CUDA library (which this package does not import either: workloads are read
through their attributes only)."""
from __future__ import annotations

import numpy as np
import torch

from . import mla_online as _m
from . import phase as _ph


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def rel_l2(a, b) -> float:
    """||a - b||_2 / ||b||_2 over the whole tensor."""
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def max_abs(a, b) -> float:
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.max(np.abs(a - b))) if a.size else 0.0


def oracle_online(w, rows, z_off=None, value_phase=False):
    """float64 expected MLA-Online result of workload `w` on packed rows `rows`.  `w` needs the
    attributes profile, layout, prot_rows, kv, q_g, q_l, w_uv, w_a, w_b, z_off.  value_phase: the
    output-phase variant (whole stored row as the value, W_uv [H, 128, 576])."""
    p, lay = w.profile, w.layout
    rows = np.asarray(rows, dtype=np.int64)
    inv = _m.inverse_row_map(w.prot_rows, lay.n_rows)
    ql = {int(r): f64(w.q_l[int(inv[r])]) for r in rows if inv[r] >= 0}
    z_off = f64(w.z_off) if z_off is None else z_off
    fn = _ph.mla_online_rows_phase if value_phase else _m.mla_online_rows
    return fn(rows, f64(w.q_g[torch.as_tensor(rows)]), ql, f64(w.kv), lay.seg_off, lay.seg_delta, w.prot_rows,
              p.global_heads, p.local_heads, f64(w.w_uv), f64(w.w_a), f64(w.w_b), z_off, p.sm_scale, p.rope_base,
              p.d_latent)
