"""ctypes binding of libmohge.so: same names and argument order as include/mohge.h.

Only argument marshalling happens here (tensor -> device pointer); every step
of the layer runs in the CUDA library.  There is no fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

MAX_GROUPS = 8
BF16, F32 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmohge.so")


class MohgeError(RuntimeError):
    pass


class mohge_config(C.Structure):
    _fields_ = [
        ("d_model", C.c_int32), ("n_groups", C.c_int32), ("experts_per_group", C.c_int32),
        ("k_groups", C.c_int32), ("k_experts", C.c_int32),
        ("group_width", C.c_int32 * MAX_GROUPS), ("dtype", C.c_int32),
        ("alpha_g", C.c_float), ("alpha_e", C.c_float), ("eps", C.c_float),
        ("f_norm_by_T", C.c_int32), ("fe_mode", C.c_int32), ("row_align", C.c_int32),
    ]


_lib = None

_P = C.c_void_p
_SIGS = {
    "mohge_launch_count": (C.c_int64, []),
    "mohge_workspace_bytes": (C.c_int64, [C.POINTER(mohge_config), C.c_int64]),
    "mohge_perm_rows": (C.c_int64, [C.POINTER(mohge_config), C.c_int64]),
    "mohge_workspace_init": (C.c_int32, [C.POINTER(mohge_config), C.c_int64, _P, C.c_int64, _P]),
    "mohge_get_switch": (C.c_int32, [C.c_char_p]),
    "mohge_set_switch": (C.c_int32, [C.c_char_p, C.c_int32]),
    "mohge_map_cache_stats": (None, [C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "mohge_get_device_status": (C.c_int32, [_P, C.POINTER(C.c_int32), _P]),
    "mohge_route": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 12),
    "mohge_aux_stats": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 12),
    "mohge_aux_stats_static": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 11),
    "mohge_dispatch": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 11),
    "mohge_expert_fwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 10),
    "mohge_combine": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 6),
    "mohge_combine_bwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 9),
    "mohge_expert_bwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 12
                         + [C.c_int32, _P, _P]),
    "mohge_expert_bwd_dgate": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 12
                               + [C.c_int32] + [_P] * 7),
    "mohge_dispatch_indices": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 10),
    "mohge_expert_fwd_gather": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 11),
    "mohge_expert_bwd_gather": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 13
                                + [C.c_int32] + [_P] * 7),
    "mohge_row_tokens": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 6),
    "mohge_expert_bwd_dy": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 13
                            + [C.c_int32] + [_P] * 8),
    "mohge_dispatch_bwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 5),
    "mohge_shared_fwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64, C.c_int32] + [_P] * 8),
    "mohge_shared_bwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64, C.c_int32] + [_P] * 10
                         + [C.c_int32, _P, _P]),
    "mohge_route_bwd": (C.c_int32, [C.POINTER(mohge_config), C.c_int64] + [_P] * 14),
}


def lib():
    """Loads libmohge.so (built by paper_2604_23108_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MohgeError("libmohge.so is not built: run `python -m paper_2604_23108_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.mohge_last_error.restype = C.c_char_p
        L.mohge_last_error.argtypes = []
        for name, (res, args) in _SIGS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def exported_symbols() -> List[str]:
    return ["mohge_last_error"] + list(_SIGS)


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise MohgeError("%s failed (%d): %s" % (what, rc, lib().mohge_last_error().decode()))


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return t.data_ptr()          # an int: ctypes converts it for a c_void_p parameter


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream():
    """The caller's current stream as a raw handle (every call is enqueued on it)."""
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _ptr_array(ts: Sequence[torch.Tensor]):
    arr = (C.c_void_p * len(ts))()
    for i, t in enumerate(ts):
        assert t.is_cuda and t.is_contiguous()
        arr[i] = t.data_ptr()
    return arr


@dataclass
class Config:
    d_model: int
    n_groups: int
    experts_per_group: int
    k_groups: int
    k_experts: int
    group_width: Sequence[int]
    dtype: str = "bf16"
    alpha_g: float = 1e-4
    alpha_e: float = 2.5e-3
    eps: float = 1e-20
    f_norm_by_T: int = 1
    fe_mode: int = 0
    row_align: int = 128

    def c(self) -> mohge_config:
        """The POD of the C ABI; rebuilt only when a field has changed since the last call."""
        key = (self.d_model, self.n_groups, self.experts_per_group, self.k_groups, self.k_experts,
               tuple(self.group_width), self.dtype, self.alpha_g, self.alpha_e, self.eps,
               self.f_norm_by_T, self.fe_mode, self.row_align)
        cached = self.__dict__.get("_c_cache")
        if cached is not None and cached[0] == key:
            return cached[1]
        s = mohge_config()
        s.d_model, s.n_groups, s.experts_per_group = self.d_model, self.n_groups, self.experts_per_group
        s.k_groups, s.k_experts = self.k_groups, self.k_experts
        for g in range(MAX_GROUPS):
            s.group_width[g] = self.group_width[g] if g < len(self.group_width) else 0
        s.dtype = BF16 if self.dtype == "bf16" else F32
        s.alpha_g, s.alpha_e, s.eps = self.alpha_g, self.alpha_e, self.eps
        s.f_norm_by_T, s.fe_mode, s.row_align = self.f_norm_by_T, self.fe_mode, self.row_align
        self.__dict__["_c_cache"] = (key, s)
        return s

    @property
    def n_experts(self):
        return self.n_groups * self.experts_per_group

    @property
    def n_logits(self):
        return self.n_groups + self.n_experts

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


def mohge_launch_count() -> int:
    return int(lib().mohge_launch_count())


def mohge_workspace_bytes(cfg: Config, T: int) -> int:
    n = lib().mohge_workspace_bytes(C.byref(cfg.c()), T)
    if n <= 0:
        raise MohgeError("mohge_workspace_bytes: %s" % lib().mohge_last_error().decode())
    return n


def mohge_perm_rows(cfg: Config, T: int) -> int:
    n = lib().mohge_perm_rows(C.byref(cfg.c()), T)
    if n <= 0 and T > 0:
        raise MohgeError("mohge_perm_rows: %s" % lib().mohge_last_error().decode())
    return n


def mohge_workspace_init(cfg, T, ws):
    _check(lib().mohge_workspace_init(C.byref(cfg.c()), T, _ptr(ws), ws.numel() * ws.element_size(),
                                      _stream()), "mohge_workspace_init")


MOHGE_ERR_TIMEOUT, MOHGE_ERR_DEVICE_CHECK = -5, -6


def mohge_get_device_status_rc(ws):
    """(return code, status word): the code is 0, MOHGE_ERR_TIMEOUT or MOHGE_ERR_DEVICE_CHECK as
    decoded from the word by the library."""
    out = C.c_int32(0)
    rc = lib().mohge_get_device_status(_ptr(ws), C.byref(out), _stream())
    if rc not in (0, MOHGE_ERR_TIMEOUT, MOHGE_ERR_DEVICE_CHECK):
        _check(rc, "mohge_get_device_status")
    return rc, out.value


def mohge_get_device_status(ws) -> int:
    """The device status word (0 = nothing reported)."""
    return mohge_get_device_status_rc(ws)[1]


def mohge_get_switch(name: str) -> int:
    return int(lib().mohge_get_switch(name.encode()))


def mohge_set_switch(name: str, value: int) -> None:
    _check(lib().mohge_set_switch(name.encode(), int(value)), "mohge_set_switch")


def mohge_map_cache_stats():
    h, m = C.c_int64(0), C.c_int64(0)
    lib().mohge_map_cache_stats(C.byref(h), C.byref(m))
    return h.value, m.value


def mohge_route(cfg, T, x, w_router, logit_bias, logits_in, logits_out, group_idx, expert_idx,
                gate_w, gs_saved, esp_saved, ws):
    _check(lib().mohge_route(C.byref(cfg.c()), T, _ptr(x), _ptr(w_router), _ptr(logit_bias),
                             _ptr(logits_in), _ptr(logits_out), _ptr(group_idx), _ptr(expert_idx),
                             _ptr(gate_w), _ptr(gs_saved), _ptr(esp_saved), _ptr(ws), _stream()),
           "mohge_route")


def mohge_aux_stats(cfg, T, gs_saved, esp_saved, group_idx, expert_idx, group_count, group_psum,
                    expert_count_routed, expert_count_lit, expert_psum, loss_out, ws):
    _check(lib().mohge_aux_stats(C.byref(cfg.c()), T, _ptr(gs_saved), _ptr(esp_saved),
                                 _ptr(group_idx), _ptr(expert_idx), _ptr(group_count),
                                 _ptr(group_psum), _ptr(expert_count_routed),
                                 _ptr(expert_count_lit), _ptr(expert_psum), _ptr(loss_out),
                                 _ptr(ws), _stream()), "mohge_aux_stats")


def mohge_aux_stats_static(cfg, T, gs_saved, esp_saved, group_idx, expert_idx, group_count,
                           group_psum, expert_count_routed, expert_count_lit, expert_psum, loss_out):
    """mohge_aux_stats without a workspace: for callers that cannot allocate one (see mohge.h)."""
    _check(lib().mohge_aux_stats_static(C.byref(cfg.c()), T, _ptr(gs_saved), _ptr(esp_saved),
                                        _ptr(group_idx), _ptr(expert_idx), _ptr(group_count),
                                        _ptr(group_psum), _ptr(expert_count_routed),
                                        _ptr(expert_count_lit), _ptr(expert_psum), _ptr(loss_out),
                                        _stream()), "mohge_aux_stats_static")


def mohge_dispatch(cfg, T, x, expert_idx, counts, offsets, aligned_offsets, row_of, prow_of,
                   src_of, x_perm, ws):
    _check(lib().mohge_dispatch(C.byref(cfg.c()), T, _ptr(x), _ptr(expert_idx), _ptr(counts),
                                _ptr(offsets), _ptr(aligned_offsets), _ptr(row_of), _ptr(prow_of),
                                _ptr(src_of), _ptr(x_perm), _ptr(ws), _stream()), "mohge_dispatch")


def mohge_expert_fwd(cfg, T, x_perm, counts, aligned_offsets, w13, w2, au_saved, h_saved, y_perm, ws):
    a13, a2 = _ptr_array(w13), _ptr_array(w2)
    _check(lib().mohge_expert_fwd(C.byref(cfg.c()), T, _ptr(x_perm), _ptr(counts),
                                  _ptr(aligned_offsets), C.cast(a13, _P), C.cast(a2, _P),
                                  _ptr(au_saved), _ptr(h_saved), _ptr(y_perm), _ptr(ws), _stream()),
           "mohge_expert_fwd")


def mohge_combine(cfg, T, y_perm, prow_of, gate_w, y, y_add=None):
    _check(lib().mohge_combine(C.byref(cfg.c()), T, _ptr(y_perm), _ptr(prow_of), _ptr(gate_w),
                               _ptr(y_add), _ptr(y), _stream()), "mohge_combine")


def mohge_combine_bwd(cfg, T, dy, y_perm, prow_of, gate_w, counts, aligned_offsets, dy_perm, dgate_w):
    _check(lib().mohge_combine_bwd(C.byref(cfg.c()), T, _ptr(dy), _ptr(y_perm), _ptr(prow_of),
                                   _ptr(gate_w), _ptr(counts), _ptr(aligned_offsets), _ptr(dy_perm),
                                   _ptr(dgate_w), _stream()), "mohge_combine_bwd")


def mohge_expert_bwd(cfg, T, dy_perm, x_perm, au_saved, h_saved, counts, aligned_offsets, w13, w2,
                     dau, dx_perm, dw13, dw2, accumulate, ws):
    a13, a2, d13, d2 = _ptr_array(w13), _ptr_array(w2), _ptr_array(dw13), _ptr_array(dw2)
    _check(lib().mohge_expert_bwd(C.byref(cfg.c()), T, _ptr(dy_perm), _ptr(x_perm), _ptr(au_saved),
                                  _ptr(h_saved), _ptr(counts), _ptr(aligned_offsets),
                                  C.cast(a13, _P), C.cast(a2, _P), _ptr(dau), _ptr(dx_perm),
                                  C.cast(d13, _P), C.cast(d2, _P), int(accumulate), _ptr(ws),
                                  _stream()), "mohge_expert_bwd")


def mohge_expert_bwd_dgate(cfg, T, dy_perm, x_perm, au_saved, h_saved, counts, aligned_offsets, w13, w2,
                           dau, dx_perm, dw13, dw2, accumulate, dy, y_perm, prow_of, gate_w, dgate_w, ws):
    a13, a2, d13, d2 = _ptr_array(w13), _ptr_array(w2), _ptr_array(dw13), _ptr_array(dw2)
    _check(lib().mohge_expert_bwd_dgate(C.byref(cfg.c()), T, _ptr(dy_perm), _ptr(x_perm), _ptr(au_saved),
                                        _ptr(h_saved), _ptr(counts), _ptr(aligned_offsets),
                                        C.cast(a13, _P), C.cast(a2, _P), _ptr(dau), _ptr(dx_perm),
                                        C.cast(d13, _P), C.cast(d2, _P), int(accumulate), _ptr(dy),
                                        _ptr(y_perm), _ptr(prow_of), _ptr(gate_w), _ptr(dgate_w),
                                        _ptr(ws), _stream()), "mohge_expert_bwd_dgate")


def mohge_dispatch_indices(cfg, T, expert_idx, counts, offsets, aligned_offsets, row_of, prow_of,
                           src_of, tok_of_prow, ws):
    _check(lib().mohge_dispatch_indices(C.byref(cfg.c()), T, _ptr(expert_idx), _ptr(counts),
                                        _ptr(offsets), _ptr(aligned_offsets), _ptr(row_of),
                                        _ptr(prow_of), _ptr(src_of), _ptr(tok_of_prow), _ptr(ws),
                                        _stream()), "mohge_dispatch_indices")


def mohge_expert_fwd_gather(cfg, T, x, tok_of_prow, counts, aligned_offsets, w13, w2, au_saved, h_saved,
                            y_perm, ws):
    a13, a2 = _ptr_array(w13), _ptr_array(w2)
    _check(lib().mohge_expert_fwd_gather(C.byref(cfg.c()), T, _ptr(x), _ptr(tok_of_prow), _ptr(counts),
                                         _ptr(aligned_offsets), C.cast(a13, _P), C.cast(a2, _P),
                                         _ptr(au_saved), _ptr(h_saved), _ptr(y_perm), _ptr(ws), _stream()),
           "mohge_expert_fwd_gather")


def mohge_expert_bwd_gather(cfg, T, dy_perm, x, tok_of_prow, au_saved, h_saved, counts, aligned_offsets,
                            w13, w2, dau, dx_perm, dw13, dw2, accumulate, dy, y_perm, prow_of, gate_w,
                            dgate_w, ws):
    a13, a2, d13, d2 = _ptr_array(w13), _ptr_array(w2), _ptr_array(dw13), _ptr_array(dw2)
    _check(lib().mohge_expert_bwd_gather(C.byref(cfg.c()), T, _ptr(dy_perm), _ptr(x), _ptr(tok_of_prow),
                                         _ptr(au_saved), _ptr(h_saved), _ptr(counts),
                                         _ptr(aligned_offsets), C.cast(a13, _P), C.cast(a2, _P),
                                         _ptr(dau), _ptr(dx_perm), C.cast(d13, _P), C.cast(d2, _P),
                                         int(accumulate), _ptr(dy), _ptr(y_perm), _ptr(prow_of),
                                         _ptr(gate_w), _ptr(dgate_w), _ptr(ws), _stream()),
           "mohge_expert_bwd_gather")


def mohge_row_tokens(cfg, T, counts, offsets, aligned_offsets, src_of, tok_of_prow):
    _check(lib().mohge_row_tokens(C.byref(cfg.c()), T, _ptr(counts), _ptr(offsets), _ptr(aligned_offsets),
                                  _ptr(src_of), _ptr(tok_of_prow), _stream()), "mohge_row_tokens")


def mohge_expert_bwd_dy(cfg, T, dy, tok_of_prow, x_perm, au_saved, h_saved, counts, aligned_offsets, w13, w2,
                        dau, dx_perm, dw13, dw2, accumulate, y_perm, prow_of, gate_w, dgate_w, hs, row_gate,
                        ws):
    a13, a2, d13, d2 = _ptr_array(w13), _ptr_array(w2), _ptr_array(dw13), _ptr_array(dw2)
    _check(lib().mohge_expert_bwd_dy(C.byref(cfg.c()), T, _ptr(dy), _ptr(tok_of_prow), _ptr(x_perm),
                                     _ptr(au_saved), _ptr(h_saved), _ptr(counts), _ptr(aligned_offsets),
                                     C.cast(a13, _P), C.cast(a2, _P), _ptr(dau), _ptr(dx_perm),
                                     C.cast(d13, _P), C.cast(d2, _P), int(accumulate), _ptr(y_perm),
                                     _ptr(prow_of), _ptr(gate_w), _ptr(dgate_w), _ptr(hs), _ptr(row_gate),
                                     _ptr(ws), _stream()), "mohge_expert_bwd_dy")


def mohge_dispatch_bwd(cfg, T, dx_perm, prow_of, dx, dx_add=None):
    _check(lib().mohge_dispatch_bwd(C.byref(cfg.c()), T, _ptr(dx_perm), _ptr(prow_of),
                                    _ptr(dx_add), _ptr(dx), _stream()), "mohge_dispatch_bwd")


def mohge_shared_fwd(cfg, T, shared_width, x, w13_shared, w2_shared, au_shared, h_shared, y_shared, ws):
    _check(lib().mohge_shared_fwd(C.byref(cfg.c()), T, int(shared_width), _ptr(x), _ptr(w13_shared),
                                  _ptr(w2_shared), _ptr(au_shared), _ptr(h_shared), _ptr(y_shared),
                                  _ptr(ws), _stream()), "mohge_shared_fwd")


def mohge_shared_bwd(cfg, T, shared_width, dy, x, au_shared, h_shared, w13_shared, w2_shared,
                     dau_shared, dx_shared, dw13_shared, dw2_shared, accumulate, ws):
    _check(lib().mohge_shared_bwd(C.byref(cfg.c()), T, int(shared_width), _ptr(dy), _ptr(x),
                                  _ptr(au_shared), _ptr(h_shared), _ptr(w13_shared),
                                  _ptr(w2_shared), _ptr(dau_shared), _ptr(dx_shared),
                                  _ptr(dw13_shared), _ptr(dw2_shared), int(accumulate), _ptr(ws),
                                  _stream()), "mohge_shared_bwd")


def mohge_route_bwd(cfg, T, x, w_router, dgate_w, gs_saved, esp_saved, group_idx, expert_idx,
                    group_count, expert_count, dlogits, dx, dw_router, ws):
    _check(lib().mohge_route_bwd(C.byref(cfg.c()), T, _ptr(x), _ptr(w_router), _ptr(dgate_w),
                                 _ptr(gs_saved), _ptr(esp_saved), _ptr(group_idx), _ptr(expert_idx),
                                 _ptr(group_count), _ptr(expert_count), _ptr(dlogits), _ptr(dx),
                                 _ptr(dw_router), _ptr(ws), _stream()), "mohge_route_bwd")


class LayerBuffers:
    """Device allocations for one layer step (torch is used for memory only)."""

    def __init__(self, cfg: Config, T: int, device="cuda", shared_width: int = 0):
        self.cfg, self.T, self.shared_width = cfg, T, shared_width
        dt, dev = cfg.torch_dtype, device
        Ne, NL, Ke, Kg, d = cfg.n_experts, cfg.n_logits, cfg.k_experts, cfg.k_groups, cfg.d_model
        Wmax = max(cfg.group_width)
        rows = max(1, mohge_perm_rows(cfg, T))
        self.rows = rows
        Tn = max(1, T)
        e = lambda *shape, dtype=dt: torch.empty(*shape, dtype=dtype, device=dev)
        i32, f32 = torch.int32, torch.float32
        self.ws = torch.empty(mohge_workspace_bytes(cfg, T), dtype=torch.uint8, device=dev)
        self.logits = e(Tn, NL, dtype=f32)
        self.group_idx, self.expert_idx = e(Tn, Kg, dtype=i32), e(Tn, Ke, dtype=i32)
        self.gate_w, self.gs, self.esp = e(Tn, Ke, dtype=f32), e(Tn, cfg.n_groups, dtype=f32), e(Tn, Ne, dtype=f32)
        self.group_count, self.group_psum = e(cfg.n_groups, dtype=i32), e(cfg.n_groups, dtype=f32)
        self.cnt_routed, self.cnt_lit, self.expert_psum = e(Ne, dtype=i32), e(Ne, dtype=i32), e(Ne, dtype=f32)
        self.loss = e(4, dtype=f32)
        self.counts, self.offsets, self.aligned = e(Ne, dtype=i32), e(Ne + 4, dtype=i32), e(Ne + 4, dtype=i32)
        self.row_of, self.prow_of, self.src_of = e(Tn, Ke, dtype=i32), e(Tn, Ke, dtype=i32), e(Tn * Ke, dtype=i32)
        self.x_perm, self.y_perm = e(rows, d), e(rows, d)
        self.tok_of_prow = e(rows + 128, dtype=i32)        # row map of the gathering entry points
        self.au, self.h = e(rows, 2 * Wmax), e(rows, Wmax)
        self.y = e(Tn, d)
        # backward
        self.dy_perm, self.dx_perm, self.dau = e(rows, d), e(rows, d), e(rows, 2 * Wmax)
        self.dgate, self.dlogits = e(Tn, Ke, dtype=f32), e(Tn, NL, dtype=f32)
        self.dx = e(Tn, d)
        self.dw_router = e(NL, d, dtype=f32)
        self.dw13 = [e(cfg.experts_per_group, 2 * w, d, dtype=f32) for w in cfg.group_width]
        self.dw2 = [e(cfg.experts_per_group, d, w, dtype=f32) for w in cfg.group_width]
        if shared_width:
            Ws = shared_width
            self.au_sh, self.h_sh, self.y_sh = e(Tn, 2 * Ws), e(Tn, Ws), e(Tn, d)
            self.dau_sh, self.dx_sh = e(Tn, 2 * Ws), e(Tn, d)
            self.dw13_sh, self.dw2_sh = e(2 * Ws, d, dtype=f32), e(d, Ws, dtype=f32)
        mohge_workspace_init(cfg, T, self.ws)


def layer_forward(cfg: Config, b: LayerBuffers, x, w_router, w13, w2, logit_bias=None,
                  logits_in=None, aux=True, shared=None, gather=False):
    """route -> aux_stats -> dispatch -> expert_fwd (-> shared_fwd) -> combine; results stay in
    `b`.  shared = (w13_shared, w2_shared) adds the shared experts (b.shared_width wide).
    gather: no x_perm is written; the GEMMs gather the rows of x (mohge_dispatch_indices,
    mohge_expert_fwd_gather)."""
    T = b.T
    mohge_route(cfg, T, x, w_router, logit_bias, logits_in, b.logits, b.group_idx, b.expert_idx,
                b.gate_w, b.gs, b.esp, b.ws)
    if aux:
        mohge_aux_stats(cfg, T, b.gs, b.esp, b.group_idx, b.expert_idx, b.group_count, b.group_psum,
                        b.cnt_routed, b.cnt_lit, b.expert_psum, b.loss, b.ws)
    if gather:
        mohge_dispatch_indices(cfg, T, b.expert_idx, b.counts, b.offsets, b.aligned, b.row_of, b.prow_of,
                               b.src_of, b.tok_of_prow, b.ws)
        mohge_expert_fwd_gather(cfg, T, x, b.tok_of_prow, b.counts, b.aligned, w13, w2, b.au, b.h,
                                b.y_perm, b.ws)
    else:
        mohge_dispatch(cfg, T, x, b.expert_idx, b.counts, b.offsets, b.aligned, b.row_of, b.prow_of,
                       b.src_of, b.x_perm, b.ws)
        mohge_expert_fwd(cfg, T, b.x_perm, b.counts, b.aligned, w13, w2, b.au, b.h, b.y_perm, b.ws)
    if shared is not None:
        mohge_shared_fwd(cfg, T, b.shared_width, x, shared[0], shared[1], b.au_sh, b.h_sh, b.y_sh, b.ws)
    mohge_combine(cfg, T, b.y_perm, b.prow_of, b.gate_w, b.y,
                  y_add=b.y_sh if shared is not None else None)
    return b.y


def layer_backward(cfg: Config, b: LayerBuffers, x, w_router, w13, w2, dy, aux=True, accumulate=False,
                   shared=None, fused_dgate=True, gather=False, dy_fused=False):
    """combine_bwd -> expert_bwd (-> shared_bwd) -> dispatch_bwd -> route_bwd; results stay in `b`.
    fused_dgate: the gate gradient comes out of the experts' backward (mohge_expert_bwd_dgate) and
    combine_bwd does not read y_perm; otherwise combine_bwd computes it from y_perm.
    dy_fused: no combine_bwd and no dy_perm at all (mohge_expert_bwd_dy gathers the rows of dy)."""
    T = b.T
    assert not (gather and dy_fused), "the backward without dy_perm reads x_perm: not with gather=True"
    if dy_fused:    # after a forward through x_perm
        if getattr(b, "hs", None) is None:
            b.hs = torch.empty_like(b.h)
            b.row_gate = torch.empty(b.h.shape[0], dtype=torch.float32, device=b.h.device)
        mohge_row_tokens(cfg, T, b.counts, b.offsets, b.aligned, b.src_of, b.tok_of_prow)
        mohge_expert_bwd_dy(cfg, T, dy, b.tok_of_prow, b.x_perm, b.au, b.h, b.counts, b.aligned, w13, w2,
                            b.dau, b.dx_perm, b.dw13, b.dw2, accumulate, b.y_perm, b.prow_of, b.gate_w,
                            b.dgate, b.hs, b.row_gate, b.ws)
    elif gather:    # after a forward with gather=True: x_perm was never written
        mohge_combine_bwd(cfg, T, dy, None, b.prow_of, b.gate_w, b.counts, b.aligned, b.dy_perm, None)
        mohge_expert_bwd_gather(cfg, T, b.dy_perm, x, b.tok_of_prow, b.au, b.h, b.counts, b.aligned, w13,
                                w2, b.dau, b.dx_perm, b.dw13, b.dw2, accumulate, dy, b.y_perm, b.prow_of,
                                b.gate_w, b.dgate, b.ws)
    elif fused_dgate:
        mohge_combine_bwd(cfg, T, dy, None, b.prow_of, b.gate_w, b.counts, b.aligned, b.dy_perm, None)
        mohge_expert_bwd_dgate(cfg, T, b.dy_perm, b.x_perm, b.au, b.h, b.counts, b.aligned, w13, w2,
                               b.dau, b.dx_perm, b.dw13, b.dw2, accumulate, dy, b.y_perm, b.prow_of,
                               b.gate_w, b.dgate, b.ws)
    else:
        mohge_combine_bwd(cfg, T, dy, b.y_perm, b.prow_of, b.gate_w, b.counts, b.aligned, b.dy_perm,
                          b.dgate)
        mohge_expert_bwd(cfg, T, b.dy_perm, b.x_perm, b.au, b.h, b.counts, b.aligned, w13, w2, b.dau,
                         b.dx_perm, b.dw13, b.dw2, accumulate, b.ws)
    if shared is not None:
        mohge_shared_bwd(cfg, T, b.shared_width, dy, x, b.au_sh, b.h_sh, shared[0], shared[1],
                         b.dau_sh, b.dx_sh, b.dw13_sh, b.dw2_sh, accumulate, b.ws)
    mohge_dispatch_bwd(cfg, T, b.dx_perm, b.prow_of, b.dx,
                       dx_add=b.dx_sh if shared is not None else None)
    cnt_e = b.cnt_lit if cfg.fe_mode == 0 else b.cnt_routed
    mohge_route_bwd(cfg, T, x, w_router, b.dgate, b.gs, b.esp, b.group_idx, b.expert_idx,
                    b.group_count if aux else None, cnt_e if aux else None, b.dlogits, b.dx,
                    b.dw_router, b.ws)
    return b.dx
