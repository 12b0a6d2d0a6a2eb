"""ctypes binding of librk.so with the same names as the C ABI (argument marshalling only).

Every step of the path runs in the library's CUDA kernels; torch is used for device
memory and streams.  Importing this module fails loudly if the shared library has not been
built (`python paper_2609_07008_b200/build.py`): there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

RK_OK = 0
STATUS_NAMES = {0: "RK_OK", 1: "RK_ERR_NULL", 2: "RK_ERR_PROFILE", 3: "RK_ERR_LAYOUT", 4: "RK_ERR_ROWS",
                5: "RK_ERR_ALIGN", 6: "RK_ERR_WORKSPACE", 7: "RK_ERR_UNSUPPORTED", 8: "RK_ERR_CUDA",
                9: "RK_ERR_TIMEOUT"}


class rk_profile(C.Structure):
    _fields_ = [("n_heads", C.c_int32), ("n_groups", C.c_int32), ("group_size", C.c_int32),
                ("d_latent", C.c_int32), ("d_rope", C.c_int32), ("d_v", C.c_int32), ("o_rank", C.c_int32),
                ("d_model", C.c_int32), ("sm_scale", C.c_float), ("rope_base", C.c_float),
                ("global_heads", C.POINTER(C.c_int32))]


class rk_layout(C.Structure):
    _fields_ = [("n_segs", C.c_int32), ("seg_off", C.POINTER(C.c_int64)), ("seg_delta", C.POINTER(C.c_int64)),
                ("seg_has_artifact", C.POINTER(C.c_uint8))]


class rk_policy(C.Structure):
    _fields_ = [("edge_rows", C.c_int32), ("tail_rows", C.c_int64), ("budget_bp", C.c_int32)]


class rk_request_info(C.Structure):
    _fields_ = [("n_rows", C.c_int64), ("n_prot", C.c_int64), ("n_off_rows", C.c_int64),
                ("pairs_global", C.c_int64), ("pairs_local", C.c_int64), ("n_tiles_global", C.c_int32),
                ("n_tiles_local", C.c_int32)]


class rk_layer_buffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("kv", "q_g", "q_l", "z_off", "O_g", "O_l", "z_on_g", "z_on_l", "z", "y",
                                          "lse_g", "lse_l", "workspace")] + [("workspace_bytes", C.c_size_t)]


class rk_layer_io(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("req", "kv_host", "q_g_host", "q_l_host", "z_off_host", "W_uv", "W_a", "W_b",
                                          "y_host")]


EXPORTS = ["rk_version", "rk_status_string", "rk_create", "rk_destroy", "rk_last_error", "rk_poll_status",
           "rk_create_ex", "rk_segmented_merge_phase", "rk_check_selftest", "rk_set_wait_limit_ms", "rk_test_starve_loads", "rk_request_create", "rk_request_destroy", "rk_check_request",
           "rk_request_get_info", "rk_workspace_bytes", "rk_relocate_q", "rk_mla_online_attn",
           "rk_segmented_merge", "rk_group_sliced_proj", "rk_group_sliced_proj_static", "rk_combine_offline",
           "rk_layer_host", "rk_layer_stack_host", "rk_mla_off_workspace_bytes", "rk_mla_off_build",
           "rk_protected_rows_workspace_bytes", "rk_protected_rows", "rk_moe_fanout"]


def _load() -> C.CDLL:
    # RK_LIBRARY_PATH selects another build of the same library (the bounds-checked one, librk_check.so)
    path = os.environ.get("RK_LIBRARY_PATH") or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python paper_2609_07008_b200/build.py` "
                           "(there is no fallback path)")
    lib = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.rk_version.restype = C.c_char_p
    lib.rk_status_string.restype = C.c_char_p
    lib.rk_status_string.argtypes = [C.c_int]
    lib.rk_last_error.restype = C.c_char_p
    lib.rk_last_error.argtypes = [vp]
    lib.rk_create.argtypes = [C.POINTER(rk_profile), C.POINTER(vp)]
    lib.rk_destroy.argtypes = [vp]
    lib.rk_poll_status.argtypes = [vp, vp]
    lib.rk_set_wait_limit_ms.argtypes = [vp, i32]
    lib.rk_test_starve_loads.argtypes = [vp, i32]
    lib.rk_check_selftest.argtypes = [vp, vp]
    lib.rk_create_ex.argtypes = [C.POINTER(rk_profile), C.c_uint32, C.POINTER(vp)]
    lib.rk_segmented_merge_phase.argtypes = [vp, vp, i32, i32, i64, i32, vp, i32, vp, vp, vp, vp, vp]
    lib.rk_request_create.argtypes = [vp, C.POINTER(rk_layout), C.POINTER(i32), i64, C.POINTER(vp)]
    lib.rk_request_destroy.argtypes = [vp]
    lib.rk_check_request.argtypes = [C.POINTER(rk_layout), C.POINTER(i32), i64, C.c_char_p, C.c_size_t]
    lib.rk_request_get_info.argtypes = [vp, C.POINTER(rk_request_info)]
    lib.rk_workspace_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
    lib.rk_relocate_q.argtypes = [vp, vp, vp, i64, i32, i64, i64, i32, i32, vp, vp]
    lib.rk_mla_online_attn.argtypes = [vp] * 10
    lib.rk_segmented_merge.argtypes = [vp, i32, i64, i32, vp, i32, vp, vp, vp, vp]
    lib.rk_group_sliced_proj.argtypes = [vp] * 9 + [C.c_size_t, vp]
    lib.rk_group_sliced_proj_static.argtypes = [vp] * 9
    lib.rk_combine_offline.argtypes = [vp] * 9
    lib.rk_layer_host.argtypes = [vp] * 9 + [C.POINTER(rk_layer_buffers), vp, vp]
    lib.rk_layer_stack_host.argtypes = [vp, i32, C.POINTER(rk_layer_io), C.POINTER(rk_layer_buffers),
                                        C.POINTER(rk_layer_buffers), vp]
    lib.rk_mla_off_workspace_bytes.argtypes = [vp, i64, C.POINTER(C.c_size_t)]
    lib.rk_mla_off_build.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp, vp, vp, C.c_size_t, vp]
    lib.rk_protected_rows_workspace_bytes.argtypes = [i64, i32, C.POINTER(C.c_size_t)]
    lib.rk_protected_rows.argtypes = [vp, C.POINTER(rk_layout), C.POINTER(rk_policy), vp, i64, vp, vp, vp, vp,
                                      C.c_size_t, vp]
    lib.rk_moe_fanout.argtypes = [vp, vp, i64, C.c_float, i32, vp, vp, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int:  # default restype: rk_status
            fn.restype = C.c_int
    return lib


lib = _load()


class RKError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _empty(shape, dtype, device):
    """Every buffer the binding allocates on behalf of the caller (outputs, scratch) comes from here, so a
    caller with its own memory pool -- or a test that wants guard zones around the outputs -- can replace it."""
    return torch.empty(shape, dtype=dtype, device=device)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_layout_struct(seg_off, seg_delta, seg_has_artifact):
    so = np.ascontiguousarray(seg_off, dtype=np.int64)
    sd = np.ascontiguousarray(seg_delta, dtype=np.int64)
    sh = np.ascontiguousarray(seg_has_artifact, dtype=np.uint8)
    lay = rk_layout(len(sd), so.ctypes.data_as(C.POINTER(C.c_int64)), sd.ctypes.data_as(C.POINTER(C.c_int64)),
                    sh.ctypes.data_as(C.POINTER(C.c_uint8)))
    return lay, (so, sd, sh)


def rk_check_request(seg_off, seg_delta, seg_has_artifact, prot_rows):
    """Host-only validation; returns (status, message)."""
    lay, keep = make_layout_struct(seg_off, seg_delta, seg_has_artifact)
    pr = np.ascontiguousarray(prot_rows, dtype=np.int32)
    msg = C.create_string_buffer(256)
    s = lib.rk_check_request(C.byref(lay), pr.ctypes.data_as(C.POINTER(C.c_int32)), len(pr), msg, 256)
    return s, msg.value.decode()


class Context:
    """rk_ctx: one per (device, head profile)."""

    def __init__(self, n_heads, n_groups, o_rank, d_model, global_heads, sm_scale, rope_base=10000.0,
                 group_size=8, d_latent=512, d_rope=64, d_v=128, value_phase=False):
        gh = np.ascontiguousarray(global_heads, dtype=np.int32)
        self._gh = gh
        self.profile = rk_profile(n_heads, n_groups, group_size, d_latent, d_rope, d_v, o_rank, d_model,
                                  float(sm_scale), float(rope_base), gh.ctypes.data_as(C.POINTER(C.c_int32)))
        self.handle = C.c_void_p()
        # value_phase: the output-phase variant (RK_VALUE_PHASE): attention outputs are 576 wide, W_uv [H,128,576]
        s = lib.rk_create_ex(C.byref(self.profile), 1 if value_phase else 0, C.byref(self.handle))
        if s != RK_OK:
            raise RKError(s, "rk_create failed")
        self.value_phase = bool(value_phase)
        self.ow = 576 if value_phase else 512
        self.n_heads, self.n_groups, self.n_local = n_heads, n_groups, n_heads - n_groups
        self.o_rank, self.d_model = o_rank, d_model

    @classmethod
    def from_profile(cls, p, value_phase=False):
        return cls(p.n_heads, p.n_groups, p.o_rank, p.d_model, p.global_heads, p.sm_scale, p.rope_base,
                   value_phase=value_phase)

    def check(self, s: int):
        if s != RK_OK:
            raise RKError(s, lib.rk_last_error(self.handle).decode())

    def close(self):
        if self.handle:
            lib.rk_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def rk_poll_status(self):
        self.check(lib.rk_poll_status(self.handle, _stream()))

    def rk_set_wait_limit_ms(self, ms: int):
        self.check(lib.rk_set_wait_limit_ms(self.handle, ms))

    def rk_check_selftest(self):
        self.check(lib.rk_check_selftest(self.handle, _stream()))

    def rk_test_starve_loads(self, on: bool):
        self.check(lib.rk_test_starve_loads(self.handle, 1 if on else 0))

    def rk_request_create(self, seg_off, seg_delta, seg_has_artifact, prot_rows) -> "Request":
        return Request(self, seg_off, seg_delta, seg_has_artifact, prot_rows)

    # -- the five calls ---------------------------------------------------------------------
    def rk_relocate_q(self, req, q_rope_view: torch.Tensor, seg_begin: int, seg_end: int,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q_rope_view: [n_rows, n_heads, 64] bf16 view (may be a strided slice of a wider tensor)."""
        n_rows, n_heads, w = q_rope_view.shape
        assert w == 64 and q_rope_view.stride(2) == 1 and q_rope_view.dtype == torch.bfloat16
        if out is None:
            out = _empty((seg_end - seg_begin, n_rows, n_heads, 64), dtype=torch.bfloat16,
                              device=q_rope_view.device)
        self.check(lib.rk_relocate_q(self.handle, req.handle, q_rope_view.data_ptr(), n_rows, n_heads,
                                     q_rope_view.stride(0), q_rope_view.stride(1), seg_begin, seg_end,
                                     out.data_ptr(), _stream()))
        return out

    def rk_mla_online_attn(self, req, kv, q_g, q_l, O_g=None, lse_g=None, O_l=None, lse_l=None):
        dev = kv.device
        if q_g is not None and O_g is None:
            O_g = _empty((req.T, self.n_groups, self.ow), dtype=torch.bfloat16, device=dev)
            lse_g = _empty((req.T, self.n_groups), dtype=torch.float32, device=dev)
        if q_l is not None and O_l is None:
            O_l = _empty((req.A, self.n_local, self.ow), dtype=torch.bfloat16, device=dev)
            lse_l = _empty((req.A, self.n_local), dtype=torch.float32, device=dev)
        self.check(lib.rk_mla_online_attn(self.handle, req.handle, _ptr(kv), _ptr(q_g), _ptr(q_l), _ptr(O_g),
                                          _ptr(lse_g), _ptr(O_l), _ptr(lse_l), _stream()))
        return O_g, lse_g, O_l, lse_l

    def rk_segmented_merge(self, O_part: torch.Tensor, lse_part: torch.Tensor, O=None, lse=None):
        P, n_rows, n_heads, d = O_part.shape
        assert d == 512 and lse_part.shape == (P, n_rows, n_heads) and lse_part.dtype == torch.float32
        dt = {torch.bfloat16: 0, torch.float32: 1}[O_part.dtype]
        if O is None:
            O = _empty((n_rows, n_heads, 512), dtype=torch.bfloat16, device=O_part.device)
            lse = _empty((n_rows, n_heads), dtype=torch.float32, device=O_part.device)
        self.check(lib.rk_segmented_merge(self.handle, P, n_rows, n_heads, _ptr(O_part), dt, _ptr(lse_part),
                                          _ptr(O), _ptr(lse), _stream()))
        return O, lse

    def rk_segmented_merge_phase(self, req, seg_begin: int, O_part: torch.Tensor, lse_part: torch.Tensor,
                                 row_pos: Optional[torch.Tensor] = None, O=None, lse=None):
        """Output-phase merge: part j belongs to segment seg_begin + j; O_part [P, n_rows, n_heads, 576]."""
        P, n_rows, n_heads, d = O_part.shape
        assert d == 576 and lse_part.shape == (P, n_rows, n_heads) and lse_part.dtype == torch.float32
        assert row_pos is None or (row_pos.dtype == torch.int32 and row_pos.shape == (n_rows,))
        dt = {torch.bfloat16: 0, torch.float32: 1}[O_part.dtype]
        if O is None:
            O = _empty((n_rows, n_heads, 576), dtype=torch.bfloat16, device=O_part.device)
            lse = _empty((n_rows, n_heads), dtype=torch.float32, device=O_part.device)
        self.check(lib.rk_segmented_merge_phase(self.handle, req.handle, seg_begin, P, n_rows, n_heads, _ptr(O_part), dt,
                                                _ptr(lse_part), _ptr(row_pos), _ptr(O), _ptr(lse), _stream()))
        return O, lse

    def rk_group_sliced_proj(self, req, O_g, O_l, W_uv, W_a, z_on_g=None, z_on_l=None, workspace=None):
        dev = W_uv.device
        width = self.n_groups * self.o_rank
        if O_g is not None and z_on_g is None:
            z_on_g = _empty((req.T, width), dtype=torch.bfloat16, device=dev)
        if O_l is not None and z_on_l is None:
            z_on_l = _empty((req.A, width), dtype=torch.bfloat16, device=dev)
        if workspace is None:
            workspace = _empty(max(req.workspace_bytes, 256), dtype=torch.uint8, device=dev)
        self.check(lib.rk_group_sliced_proj(self.handle, req.handle, _ptr(O_g), _ptr(O_l), _ptr(W_uv), _ptr(W_a),
                                            _ptr(z_on_g), _ptr(z_on_l), _ptr(workspace), workspace.numel(),
                                            _stream()))
        return z_on_g, z_on_l

    def rk_group_sliced_proj_static(self, req, O_g, O_l, W_uv, W_a, z_on_g, z_on_l):
        """Projection for callers that cannot allocate: outputs are passed in, the intermediate
        lives in the library's built-in 32 MiB array (shared by all calls; see include/rk.h)."""
        self.check(lib.rk_group_sliced_proj_static(self.handle, req.handle, _ptr(O_g), _ptr(O_l), _ptr(W_uv),
                                                   _ptr(W_a), _ptr(z_on_g), _ptr(z_on_l), _stream()))
        return z_on_g, z_on_l

    def rk_protected_rows(self, seg_off, seg_delta, seg_has_artifact, dirty_rows=None, scores=None, *, edge_rows=128,
                          tail_rows=32768, budget_bp=0, device="cuda", out=None, workspace=None):
        """Eq. (protected) on the device.  Returns (rows_out, count_out): a device int32 buffer of capacity T
        whose first count_out[0] entries are the ascending protected rows, and the device int64 count.
        Nothing is synchronised; `protected_rows_to_host` reads the list back."""
        lay, keep = make_layout_struct(seg_off, seg_delta, seg_has_artifact)
        pol = rk_policy(int(edge_rows), int(tail_rows), int(budget_bp))
        T, S = int(keep[0][-1]), len(keep[1])
        if workspace is None:
            need = C.c_size_t(0)
            s = lib.rk_protected_rows_workspace_bytes(T, S, C.byref(need))
            if s != 0:
                raise RKError(s, "rk_protected_rows_workspace_bytes")
            workspace = _empty(need.value, dtype=torch.uint8, device=device)
        if out is None:
            out = (_empty(T, dtype=torch.int32, device=device), _empty(1, dtype=torch.int64, device=device))
        n_dirty = 0 if dirty_rows is None else dirty_rows.numel()
        self.check(lib.rk_protected_rows(self.handle, C.byref(lay), C.byref(pol), _ptr(dirty_rows), n_dirty, _ptr(scores),
                                         _ptr(out[0]), _ptr(out[1]), _ptr(workspace), workspace.numel(), _stream()))
        return out

    @staticmethod
    def protected_rows_to_host(out) -> np.ndarray:
        n = int(out[1].item())
        return out[0][:n].cpu().numpy()

    def rk_moe_fanout(self, p: torch.Tensor, tau: float, fence: bool = False, k_out=None, keep_out=None):
        """Eq. (moe): p [n, 6] float32 Top-6 router weights -> (K_t [n] uint8, keep mask [n] uint8)."""
        assert p.dtype == torch.float32 and p.dim() == 2 and p.shape[1] == 6 and p.is_contiguous()
        n = p.shape[0]
        if k_out is None:
            k_out = _empty(n, dtype=torch.uint8, device=p.device)
            keep_out = _empty(n, dtype=torch.uint8, device=p.device)
        self.check(lib.rk_moe_fanout(self.handle, _ptr(p), n, float(tau), int(bool(fence)), _ptr(k_out), _ptr(keep_out),
                                     _stream()))
        return k_out, keep_out

    def rk_combine_offline(self, req, z_on_g, z_on_l, z_off, W_b, z=None, y=None):
        dev = z_on_g.device
        if z is None:
            z = _empty((req.T, self.n_groups * self.o_rank), dtype=torch.bfloat16, device=dev)
        if W_b is not None and y is None:
            y = _empty((req.T, self.d_model), dtype=torch.bfloat16, device=dev)
        self.check(lib.rk_combine_offline(self.handle, req.handle, _ptr(z_on_g), _ptr(z_on_l), _ptr(z_off),
                                          _ptr(W_b), _ptr(z), _ptr(y), _stream()))
        return z, y

    def rk_mla_off_build(self, req, kv, row_begin, row_end, q_l_rows, W_uv, W_a, z_off_rows=None, workspace=None):
        """Offline artifact rows [row_begin, row_end): documents alone at position zero, Local heads."""
        n = row_end - row_begin
        if z_off_rows is None:
            z_off_rows = _empty((n, self.n_groups * self.o_rank), dtype=torch.bfloat16, device=kv.device)
        ws = C.c_size_t()
        self.check(lib.rk_mla_off_workspace_bytes(req.handle, n, C.byref(ws)))
        if workspace is None:
            workspace = _empty(max(ws.value, 256), dtype=torch.uint8, device=kv.device)
        self.check(lib.rk_mla_off_build(self.handle, req.handle, _ptr(kv), row_begin, row_end, _ptr(q_l_rows),
                                        _ptr(W_uv), _ptr(W_a), _ptr(z_off_rows), _ptr(workspace), workspace.numel(),
                                        _stream()))
        return z_off_rows

    def alloc_layer_buffers(self, req, device) -> dict:
        G, L, T, A = self.n_groups, self.n_local, req.T, req.A
        width = G * self.o_rank
        bf, f32 = torch.bfloat16, torch.float32
        e = lambda shape, dt=bf: _empty(shape, dtype=dt, device=device)
        return dict(kv=e((T, 576)), q_g=e((T, G, 576)), q_l=e((max(A, 1), L, 576)),
                    z_off=e((max(req.n_off_rows, 1), width)), O_g=e((T, G, self.ow)), O_l=e((max(A, 1), L, self.ow)),
                    z_on_g=e((T, width)), z_on_l=e((max(A, 1), width)), z=e((T, width)), y=e((T, self.d_model)),
                    lse_g=e((T, G), f32), lse_l=e((max(A, 1), L), f32),
                    workspace=_empty(max(req.workspace_bytes, 256), dtype=torch.uint8, device=device))

    def rk_layer_host(self, req, kv_h, q_g_h, q_l_h, z_off_h, W_uv, W_a, W_b, bufs: dict, y_h: torch.Tensor):
        """Whole layer from pinned host tensors: H2D copies, the three device calls, D2H of y, sync."""
        b = rk_layer_buffers(*[bufs[n].data_ptr() for n in ("kv", "q_g", "q_l", "z_off", "O_g", "O_l", "z_on_g",
                                                            "z_on_l", "z", "y", "lse_g", "lse_l", "workspace")],
                             bufs["workspace"].numel())
        self.check(lib.rk_layer_host(self.handle, req.handle, _ptr(kv_h), _ptr(q_g_h), _ptr(q_l_h), _ptr(z_off_h),
                                     _ptr(W_uv), _ptr(W_a), _ptr(W_b), C.byref(b), _ptr(y_h), _stream()))
        return y_h


def _buffers_struct(bufs: dict) -> rk_layer_buffers:
    return rk_layer_buffers(*[bufs[n].data_ptr() for n in ("kv", "q_g", "q_l", "z_off", "O_g", "O_l", "z_on_g", "z_on_l",
                                                           "z", "y", "lse_g", "lse_l", "workspace")],
                            bufs["workspace"].numel())


def rk_layer_stack_host(ctx: "Context", layers, bufs0: dict, bufs1: dict):
    """layers: list of dicts with keys req, kv, q_g, q_l, z_off (pinned host tensors), W_uv, W_a, W_b (device
    tensors) and y (pinned host output).  Runs the stack with cross-layer prefetch."""
    arr = (rk_layer_io * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = rk_layer_io(l["req"].handle.value, _ptr(l["kv"]), _ptr(l["q_g"]), _ptr(l["q_l"]), _ptr(l["z_off"]),
                             _ptr(l["W_uv"]), _ptr(l["W_a"]), _ptr(l["W_b"]), _ptr(l["y"]))
    b0, b1 = _buffers_struct(bufs0), _buffers_struct(bufs1)
    ctx.check(lib.rk_layer_stack_host(ctx.handle, len(layers), arr, C.byref(b0), C.byref(b1), _stream()))


class Request:
    """rk_request: validated geometry of one request + protected-row list."""

    def __init__(self, ctx: Context, seg_off, seg_delta, seg_has_artifact, prot_rows):
        self.ctx = ctx
        lay, keep = make_layout_struct(seg_off, seg_delta, seg_has_artifact)
        pr = np.ascontiguousarray(prot_rows, dtype=np.int32)
        self.handle = C.c_void_p()
        ctx.check(lib.rk_request_create(ctx.handle, C.byref(lay), pr.ctypes.data_as(C.POINTER(C.c_int32)), len(pr),
                                        C.byref(self.handle)))
        info = rk_request_info()
        ctx.check(lib.rk_request_get_info(self.handle, C.byref(info)))
        self.T, self.A, self.n_off_rows = info.n_rows, info.n_prot, info.n_off_rows
        self.pairs_global, self.pairs_local = info.pairs_global, info.pairs_local
        self.n_tiles_global, self.n_tiles_local = info.n_tiles_global, info.n_tiles_local
        ws = C.c_size_t()
        ctx.check(lib.rk_workspace_bytes(self.handle, C.byref(ws)))
        self.workspace_bytes = ws.value

    def close(self):
        if self.handle:
            lib.rk_request_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
