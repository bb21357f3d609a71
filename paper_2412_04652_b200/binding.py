"""Thin ctypes binding of libcsp.so: same names as the C interface, argument marshalling only.

Every step of the path runs inside the CUDA library; PyTorch is used for device memory and for
the current stream.  There is no CPU fallback: if the library is missing, import of the symbols
fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcsp.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(7)
F32, BF16 = 0, 1
COMBINE_OR, COMBINE_AND = 0, 1
SELECT_SEGMENTED, SELECT_GLOBAL, SELECT_OVERALL = 0, 1, 2
HEADS_PER_KV, HEADS_MEAN_ALL = 0, 1
DEV_K_CLAMPED, DEV_CAPACITY, DEV_TIMEOUT, DEV_BAD_LEN = 1, 2, 4, 8

EXPORTS = ("csp_workspace_bytes", "csp_workspace_reset", "csp_score", "csp_select", "csp_compact",
           "csp_prune_layer", "csp_host_staging_bytes", "csp_prune_layer_host", "csp_device_status",
           "csp_status_string", "csp_prune_layer_static", "csp_static_workspace_limit",
           "csp_decode_workspace_bytes", "csp_decode_attn", "csp_decode_step_workspace_bytes", "csp_decode_step",
           "csp_weight_histogram", "csp_probe_ex2_rate", "csp_prune_layer_paged",
           "csp_decode_attn_paged", "csp_select_compact")
HIST_BINS, HIST_LO, HIST_WIDTH = 64, -32.0, 0.5


class CspError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (csp_status {code})")


class CTensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_t", C.c_int64)]


class CPages(C.Structure):
    _fields_ = [("page_table", C.c_void_p), ("max_pages", C.c_int32), ("page_rows", C.c_int32), ("n_pages", C.c_int32)]


class CParams(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("window", C.c_int32), ("recent", C.c_int32),
                ("max_len", C.c_int32), ("out_capacity", C.c_int32), ("dtype", C.c_int32),
                ("n", C.c_float), ("scale", C.c_float), ("combine", C.c_int32),
                ("select_mode", C.c_int32), ("head_reduce", C.c_int32)]


@dataclass
class Params:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int
    recent: int
    max_len: int
    out_capacity: int
    dtype: int = BF16
    n: float = 1.0
    scale: float = 0.0
    combine: int = COMBINE_OR
    select_mode: int = SELECT_SEGMENTED
    head_reduce: int = HEADS_PER_KV

    def c(self) -> CParams:
        return CParams(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.window,
                       self.recent, self.max_len, self.out_capacity, self.dtype, self.n, self.scale,
                       self.combine, self.select_mode, self.head_reduce)


_lib = None


def lib() -> C.CDLL:
    """Loads libcsp.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # not built yet (fresh checkout): compile in-tree now; there is no other implementation to fall
            # back to, so a failed build is an import error
            try:
                from . import build as _build
                _build.build()
            except Exception as exc:  # noqa: BLE001
                raise ImportError(f"{LIB_PATH} is missing and could not be built with nvcc: {exc}") from exc
        l = C.CDLL(LIB_PATH)
        P = C.POINTER(CParams)
        vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
        l.csp_workspace_bytes.restype = sz
        l.csp_workspace_bytes.argtypes = [P]
        l.csp_workspace_reset.restype = C.c_int
        l.csp_workspace_reset.argtypes = [vp, vp]
        l.csp_score.restype = C.c_int
        l.csp_score.argtypes = [P, CTensor, CTensor, vp, i64, i64, vp, vp, vp, vp, vp, sz, vp]
        l.csp_select.restype = C.c_int
        l.csp_select.argtypes = [P, vp, vp, vp, i64, i64, vp, vp, vp, vp, vp, vp, sz, vp]
        l.csp_compact.restype = C.c_int
        l.csp_compact.argtypes = [P, CTensor, CTensor, vp, i64, i64, vp, vp, CTensor, CTensor, vp, vp]
        l.csp_select_compact.restype = C.c_int
        l.csp_select_compact.argtypes = [P, vp, vp, CTensor, CTensor, vp, i64, i64, vp, vp, vp, CTensor, CTensor, vp, vp,
                                         vp, vp, sz, vp]
        l.csp_prune_layer.restype = C.c_int
        l.csp_prune_layer.argtypes = [P, CTensor, CTensor, CTensor, vp, i64, i64, vp, vp, vp, vp,
                                      CTensor, CTensor, vp, vp, vp, vp, vp, vp, sz, vp]
        l.csp_host_staging_bytes.restype = sz
        l.csp_host_staging_bytes.argtypes = [P]
        l.csp_prune_layer_host.restype = C.c_int
        l.csp_prune_layer_host.argtypes = [P, vp, vp, vp, vp, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp,
                                           vp, sz, vp]
        l.csp_prune_layer_static.restype = C.c_int
        l.csp_prune_layer_static.argtypes = [P, CTensor, CTensor, CTensor, vp, i64, i64, vp, vp, vp, vp,
                                             CTensor, CTensor, vp, vp, vp, vp]
        l.csp_static_workspace_limit.restype = sz
        l.csp_static_workspace_limit.argtypes = []
        l.csp_decode_workspace_bytes.restype = sz
        l.csp_decode_workspace_bytes.argtypes = [P]
        l.csp_decode_attn.restype = C.c_int
        l.csp_decode_attn.argtypes = [P, CTensor, CTensor, CTensor, vp, vp, vp, sz, vp]
        l.csp_decode_step_workspace_bytes.restype = sz
        l.csp_decode_step_workspace_bytes.argtypes = [P]
        l.csp_decode_step.restype = C.c_int
        l.csp_decode_step.argtypes = [P, CTensor, CTensor, CTensor, vp, vp, i64, i64, vp, C.c_int32, vp, vp, vp, vp, sz, vp]
        l.csp_prune_layer_paged.restype = C.c_int
        l.csp_prune_layer_paged.argtypes = [P, CTensor, CTensor, CTensor, C.POINTER(CPages), vp, i64, i64, vp, vp, vp, vp,
                                            CTensor, CTensor, vp, vp, vp, vp, vp, vp, sz, vp]
        l.csp_decode_attn_paged.restype = C.c_int
        l.csp_decode_attn_paged.argtypes = [P, CTensor, CTensor, CTensor, C.POINTER(CPages), vp, vp, vp, sz, vp]
        l.csp_probe_ex2_rate.restype = C.c_int
        l.csp_probe_ex2_rate.argtypes = [C.c_int32, C.c_int32, vp, sz, C.POINTER(C.c_int64), vp]
        l.csp_weight_histogram.restype = C.c_int
        l.csp_weight_histogram.argtypes = [P, CTensor, CTensor, vp, i64, i64, vp, vp, vp, vp, vp, vp, sz, vp]
        l.csp_device_status.restype = C.c_int
        l.csp_device_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
        l.csp_status_string.restype = C.c_char_p
        l.csp_status_string.argtypes = [C.c_int]
        _lib = l
    return _lib


def status_string(code: int) -> str:
    return lib().csp_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != OK:
        raise CspError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def tensor4(t: torch.Tensor) -> CTensor:
    """[B, H, T, d] tensor -> (pointer, element strides); the last axis must be contiguous."""
    assert t.dim() == 4 and (t.stride(3) == 1 or t.shape[3] == 1), "head_dim axis must be contiguous"
    return CTensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


def _mod_strides(modality: torch.Tensor):
    """[B, L] (shared by the heads) or [B, H, L] labels -> (stride_b, stride_h)."""
    assert modality.dtype == torch.uint8 and modality.stride(-1) == 1
    if modality.dim() == 2:
        return modality.stride(0), 0
    return modality.stride(0), modality.stride(1)


def workspace_bytes(p: Params) -> int:
    cp = p.c()
    return int(lib().csp_workspace_bytes(C.byref(cp)))


def new_workspace(p: Params, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and zeroes a workspace for these parameters."""
    n = workspace_bytes(p)
    if n == 0:
        raise CspError(ERR_UNSUPPORTED, "csp_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def workspace_reset(ws: torch.Tensor):
    _check(lib().csp_workspace_reset(_ptr(ws), _stream()), "csp_workspace_reset")


def decode_workspace_bytes(p: Params) -> int:
    cp = p.c()
    return int(lib().csp_decode_workspace_bytes(C.byref(cp)))


def new_decode_workspace(p: Params, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and zeroes a workspace for csp_decode_attn."""
    n = decode_workspace_bytes(p)
    if n == 0:
        raise CspError(ERR_UNSUPPORTED, "csp_decode_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def decode_attn(p: Params, q, k, v, n_rows, out, ws):
    """q [B, Hq, d]; k, v [B, Hkv, out_capacity, d]; n_rows int32 [B, Hkv]; out fp32 [B, Hq, d] (dense)."""
    cp = p.c()
    assert q.dim() == 3 and q.stride(2) == 1 and out.is_contiguous() and out.dtype == torch.float32
    qt = CTensor(q.data_ptr(), q.stride(0), q.stride(1), q.shape[2])
    _check(lib().csp_decode_attn(C.byref(cp), qt, tensor4(k), tensor4(v), _ptr(n_rows), _ptr(out), _ptr(ws),
                                 ws.numel(), _stream()), "csp_decode_attn")


def new_decode_step_workspace(p: Params, device="cuda") -> torch.Tensor:
    """Allocates (with torch) and zeroes a workspace for csp_decode_step."""
    cp = p.c()
    n = int(lib().csp_decode_step_workspace_bytes(C.byref(cp)))
    if n == 0:
        raise CspError(ERR_UNSUPPORTED, "csp_decode_step_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def decode_step(p: Params, q, k, v, n_rows, modality, query_label, first_step, out, acc_self, acc_cross, ws):
    """csp_decode_attn plus the running intra / inter sums: modality uint8 [B, Hkv, cap] (or [B, cap]), query_label
    uint8 [B], acc_self / acc_cross fp32 [B, Hkv, cap] (dense)."""
    cp = p.c()
    assert q.dim() == 3 and q.stride(2) == 1 and out.is_contiguous() and out.dtype == torch.float32
    assert acc_self.is_contiguous() and acc_cross.is_contiguous() and acc_self.dtype == torch.float32
    assert query_label.dtype == torch.uint8 and query_label.is_contiguous()
    qt = CTensor(q.data_ptr(), q.stride(0), q.stride(1), q.shape[2])
    sb, sh = _mod_strides(modality)
    _check(lib().csp_decode_step(C.byref(cp), qt, tensor4(k), tensor4(v), _ptr(n_rows), _ptr(modality), sb, sh,
                                 _ptr(query_label), int(bool(first_step)), _ptr(out), _ptr(acc_self), _ptr(acc_cross),
                                 _ptr(ws), ws.numel(), _stream()), "csp_decode_step")


def score(p: Params, q_win, k, modality, seq_lens, score_self, score_cross, ws, lse=None):
    cp = p.c()
    sb, sh = _mod_strides(modality)
    _check(lib().csp_score(C.byref(cp), tensor4(q_win), tensor4(k), _ptr(modality), sb, sh, _ptr(seq_lens),
                           _ptr(lse), _ptr(score_self), _ptr(score_cross), _ptr(ws), ws.numel(), _stream()),
           "csp_score")


def weight_histogram(p: Params, q_win, k, modality, seq_lens, hist, ws, js=None, js_all=None, lse=None):
    """hist uint32-as-int32 [B, Hkv, 2, HIST_BINS]; js fp32 [B, Hkv]; js_all fp32 [1]."""
    cp = p.c()
    sb, sh = _mod_strides(modality)
    assert hist.is_contiguous() and hist.element_size() == 4
    _check(lib().csp_weight_histogram(C.byref(cp), tensor4(q_win), tensor4(k), _ptr(modality), sb, sh, _ptr(seq_lens),
                                      _ptr(lse), _ptr(hist), _ptr(js), _ptr(js_all), _ptr(ws), ws.numel(), _stream()),
           "csp_weight_histogram")


def probe_ex2_rate(fma_pipe: bool, iterations: int, sink: Optional[torch.Tensor] = None) -> int:
    """Enqueues the exponential-throughput probe on the current stream; returns how many exponentials it evaluates."""
    n = C.c_int64(0)
    _check(lib().csp_probe_ex2_rate(int(fma_pipe), int(iterations), _ptr(sink), 0 if sink is None else sink.numel(),
                                    C.byref(n), _stream()), "csp_probe_ex2_rate")
    return int(n.value)


def select(p: Params, score_self, score_cross, modality, seq_lens, budgets, keep_idx, n_out, ws,
           total_budget=None):
    cp = p.c()
    sb, sh = _mod_strides(modality)
    _check(lib().csp_select(C.byref(cp), _ptr(score_self), _ptr(score_cross), _ptr(modality), sb, sh,
                            _ptr(seq_lens), _ptr(budgets), _ptr(total_budget), _ptr(keep_idx), _ptr(n_out),
                            _ptr(ws), ws.numel(), _stream()), "csp_select")


def compact(p: Params, k, v, modality, keep_idx, n_out, k_out, v_out, mod_out=None):
    cp = p.c()
    sb, sh = _mod_strides(modality) if modality is not None else (0, 0)
    _check(lib().csp_compact(C.byref(cp), tensor4(k), tensor4(v), _ptr(modality), sb, sh, _ptr(keep_idx),
                             _ptr(n_out), tensor4(k_out), tensor4(v_out), _ptr(mod_out), _stream()),
           "csp_compact")


def select_compact(p: Params, score_self, score_cross, k, v, modality, seq_lens, budgets, k_out, v_out, mod_out, n_out,
                   ws, total_budget=None, keep_idx=None):
    cp = p.c()
    sb, sh = _mod_strides(modality)
    _check(lib().csp_select_compact(C.byref(cp), _ptr(score_self), _ptr(score_cross), tensor4(k), tensor4(v),
                                    _ptr(modality), sb, sh, _ptr(seq_lens), _ptr(budgets), _ptr(total_budget),
                                    tensor4(k_out), tensor4(v_out), _ptr(mod_out), _ptr(n_out), _ptr(keep_idx),
                                    _ptr(ws), ws.numel(), _stream()), "csp_select_compact")


def prune_layer(p: Params, q_win, k, v, modality, seq_lens, budgets, k_out, v_out, mod_out, n_out, ws,
                total_budget=None, lse=None, score_self=None, score_cross=None, keep_idx=None):
    cp = p.c()
    sb, sh = _mod_strides(modality)
    _check(lib().csp_prune_layer(C.byref(cp), tensor4(q_win), tensor4(k), tensor4(v), _ptr(modality), sb, sh,
                                 _ptr(seq_lens), _ptr(budgets), _ptr(total_budget), _ptr(lse),
                                 tensor4(k_out), tensor4(v_out), _ptr(mod_out), _ptr(n_out),
                                 _ptr(score_self), _ptr(score_cross), _ptr(keep_idx),
                                 _ptr(ws), ws.numel(), _stream()), "csp_prune_layer")


def prune_layer_paged(p: Params, q_win, k_pool, v_pool, page_table, modality, seq_lens, budgets, k_out, v_out, mod_out,
                      n_out, ws, total_budget=None, lse=None, score_self=None, score_cross=None, keep_idx=None):
    """k_pool, v_pool [n_pages, Hkv, page_rows, d]; page_table int32 [B, max_pages] (dense).  k_out / v_out dense
    [B, Hkv, cap, d], or the pools themselves for pruning in place."""
    cp = p.c()
    sb, sh = _mod_strides(modality)
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and page_table.dim() == 2
    pg = CPages(page_table.data_ptr(), page_table.shape[1], k_pool.shape[2], k_pool.shape[0])
    _check(lib().csp_prune_layer_paged(C.byref(cp), tensor4(q_win), tensor4(k_pool), tensor4(v_pool), C.byref(pg),
                                       _ptr(modality), sb, sh, _ptr(seq_lens), _ptr(budgets), _ptr(total_budget),
                                       _ptr(lse), tensor4(k_out), tensor4(v_out), _ptr(mod_out), _ptr(n_out),
                                       _ptr(score_self), _ptr(score_cross), _ptr(keep_idx), _ptr(ws), ws.numel(),
                                       _stream()), "csp_prune_layer_paged")


def decode_attn_paged(p: Params, q, k_pool, v_pool, page_table, n_rows, out, ws):
    """csp_decode_attn over pools [n_pages, Hkv, page_rows, d] addressed through page_table int32 [B, max_pages]."""
    cp = p.c()
    assert q.dim() == 3 and q.stride(2) == 1 and out.is_contiguous() and out.dtype == torch.float32
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and page_table.dim() == 2
    qt = CTensor(q.data_ptr(), q.stride(0), q.stride(1), q.shape[2])
    pg = CPages(page_table.data_ptr(), page_table.shape[1], k_pool.shape[2], k_pool.shape[0])
    _check(lib().csp_decode_attn_paged(C.byref(cp), qt, tensor4(k_pool), tensor4(v_pool), C.byref(pg), _ptr(n_rows),
                                       _ptr(out), _ptr(ws), ws.numel(), _stream()), "csp_decode_attn_paged")


def static_workspace_limit() -> int:
    return int(lib().csp_static_workspace_limit())


def prune_layer_static(p: Params, q_win, k, v, modality, seq_lens, budgets, k_out, v_out, mod_out, n_out,
                       total_budget=None, lse=None, dev_status_out=None):
    """csp_prune_layer without a caller workspace: the library's built-in scratch array is used, so
    nothing is allocated.  Raises CspError(ERR_WORKSPACE) for shapes beyond static_workspace_limit()."""
    cp = p.c()
    sb, sh = _mod_strides(modality)
    _check(lib().csp_prune_layer_static(C.byref(cp), tensor4(q_win), tensor4(k), tensor4(v), _ptr(modality), sb, sh,
                                        _ptr(seq_lens), _ptr(budgets), _ptr(total_budget), _ptr(lse),
                                        tensor4(k_out), tensor4(v_out), _ptr(mod_out), _ptr(n_out),
                                        _ptr(dev_status_out), _stream()), "csp_prune_layer_static")


def host_staging_bytes(p: Params) -> int:
    cp = p.c()
    return int(lib().csp_host_staging_bytes(C.byref(cp)))


def prune_layer_host(p: Params, q, k, v, modality, seq_lens, budgets, k_out, v_out, mod_out, n_out,
                     staging: torch.Tensor, total_budget=None) -> int:
    """All tensors but `staging` are dense CPU tensors (pinned for asynchronous copies).
    Returns the device status word."""
    cp = p.c()
    for t in (q, k, v, modality, seq_lens, budgets, k_out, v_out, n_out):
        assert t.device.type == "cpu" and t.is_contiguous()
    word = C.c_int32(0)
    _check(lib().csp_prune_layer_host(C.byref(cp), _ptr(q), _ptr(k), _ptr(v), _ptr(modality),
                                      int(modality.dim() == 3), _ptr(seq_lens), _ptr(budgets),
                                      _ptr(total_budget), _ptr(k_out), _ptr(v_out), _ptr(mod_out),
                                      _ptr(n_out), C.addressof(word), _ptr(staging), staging.numel(),
                                      _stream()), "csp_prune_layer_host")
    return int(word.value)


def device_status(ws: torch.Tensor) -> int:
    """Waits for the current stream, returns the status word (CSP_DEV_* bits) and clears it."""
    word = C.c_int32(0)
    rc = lib().csp_device_status(_ptr(ws), _stream(), C.byref(word))
    if rc not in (OK, ERR_TIMEOUT):
        raise CspError(rc, "csp_device_status")
    return int(word.value)
