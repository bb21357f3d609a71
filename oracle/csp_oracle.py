"""ctypes front-end of the CPU oracle (``csp_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the bench may import this
module.  It shares nothing with the CUDA library.  Arguments are numpy arrays (bf16 data is
passed as ``uint16`` bit patterns); torch CPU tensors are converted on the way in.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csp_oracle.c")
_HDR = os.path.join(_HERE, "csp_oracle.h")
_LIB = os.path.join(_HERE, "libcsp_oracle.so")

F32, BF16 = 0, 1
COMBINE_OR, COMBINE_AND = 0, 1
SELECT_SEGMENTED, SELECT_GLOBAL, SELECT_OVERALL = 0, 1, 2
HEADS_PER_KV, HEADS_MEAN_ALL = 0, 1
FLAG_K_CLAMPED, FLAG_CAPACITY, FLAG_IDENTITY = 1, 2, 4
HIST_BINS, HIST_LO, HIST_WIDTH = 64, -32.0, 0.5


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) next to its source."""
    stale = (not os.path.exists(_LIB)) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB) for s in (_SRC, _HDR))
    if force or stale:
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "n_q_heads", "n_kv_heads", "head_dim", "window",
                                          "recent", "max_len", "out_capacity", "dtype", "combine",
                                          "select_mode", "head_reduce")] + \
               [("n", C.c_double), ("scale", C.c_double)]


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
    combine: int = COMBINE_OR
    select_mode: int = SELECT_SEGMENTED
    head_reduce: int = HEADS_PER_KV
    n: float = 1.0
    scale: float = 0.0

    def c(self) -> _Params:
        return _Params(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.window,
                       self.recent, self.max_len, self.out_capacity, self.dtype, self.combine,
                       self.select_mode, self.head_reduce, float(self.n), float(self.scale))


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_topk.restype = C.c_int
        _lib.orc_num_threads.restype = C.c_int
        _lib.orc_js_divergence.restype = C.c_double
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _np(x, dtype=None):
    """numpy view/copy of a numpy array or torch CPU tensor (bf16 -> uint16 bits)."""
    if x is None:
        return None
    if not isinstance(x, np.ndarray):
        import torch
        t = x.detach().cpu().contiguous()
        if t.dtype == torch.bfloat16:
            t = t.view(torch.int16)
            x = t.numpy().view(np.uint16)
        else:
            x = t.numpy()
    if dtype is not None and x.dtype != dtype:
        x = x.astype(dtype)
    return np.ascontiguousarray(x)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _elem(p: Params):
    return np.float32 if p.dtype == F32 else np.uint16


def nsoftmax(o, n: float):
    o = _np(o, np.float64)
    a = np.empty_like(o)
    lib().orc_nsoftmax(_ptr(o), C.c_int64(o.size), C.c_double(n), _ptr(a))
    return a


def score(p: Params, q, k, modality, seq_lens, lse=None, want_row_mass=False):
    q, k = _np(q, _elem(p)), _np(k, _elem(p))
    modality = _np(modality, np.uint8)
    seq_lens = _np(seq_lens, np.int32)
    lse = _np(lse, np.float64)
    per_head = int(modality.ndim == 3)
    shape = (p.batch, p.n_kv_heads, p.max_len)
    s = np.zeros(shape, np.float64)
    c = np.zeros(shape, np.float64)
    mass = np.zeros((p.batch, p.n_q_heads, p.window), np.float64) if want_row_mass else None
    cp = p.c()
    rc = lib().orc_score(C.byref(cp), _ptr(q), _ptr(k), _ptr(modality), per_head, _ptr(seq_lens),
                         _ptr(lse), _ptr(s), _ptr(c), _ptr(mass))
    if rc:
        raise ValueError("orc_score: bad argument")
    return (s, c, mass) if want_row_mass else (s, c)


def topk(score_vec, cand, k: int):
    score_vec = _np(score_vec, np.float32)
    cand = _np(cand, np.uint8)
    mask = np.zeros(score_vec.shape, np.uint8)
    kth, knext = C.c_float(), C.c_float()
    n_sel = lib().orc_topk(_ptr(score_vec), _ptr(cand), C.c_int64(score_vec.size), C.c_int64(k),
                           _ptr(mask), C.byref(kth), C.byref(knext))
    return mask, n_sel, kth.value, knext.value


def select(p: Params, score_self, score_cross, modality, seq_lens, budgets, total_budget=None):
    s, c = _np(score_self, np.float32), _np(score_cross, np.float32)
    modality = _np(modality, np.uint8)
    seq_lens = _np(seq_lens, np.int32)
    budgets = _np(budgets, np.int32)
    total_budget = _np(total_budget, np.int32)
    per_head = int(modality.ndim == 3)
    idx = np.full((p.batch, p.n_kv_heads, p.out_capacity), -1, np.int32)
    n_out = np.zeros((p.batch, p.n_kv_heads), np.int32)
    flags = np.zeros((p.batch, p.n_kv_heads), np.int32)
    margins = np.zeros((p.batch, p.n_kv_heads, 4, 2), np.float32)
    cp = p.c()
    rc = lib().orc_select(C.byref(cp), _ptr(s), _ptr(c), _ptr(modality), per_head, _ptr(seq_lens),
                          _ptr(budgets), _ptr(total_budget), _ptr(idx), _ptr(n_out), _ptr(flags),
                          _ptr(margins))
    if rc:
        raise ValueError("orc_select: bad argument")
    return idx, n_out, flags, margins


def compact(p: Params, k, v, modality, keep_idx, n_out):
    k, v = _np(k, _elem(p)), _np(v, _elem(p))
    modality = _np(modality, np.uint8)
    keep_idx, n_out = _np(keep_idx, np.int32), _np(n_out, np.int32)
    per_head = int(modality.ndim == 3)
    oshape = (p.batch, p.n_kv_heads, p.out_capacity, p.head_dim)
    k_out = np.zeros(oshape, k.dtype)
    v_out = np.zeros(oshape, v.dtype)
    mod_out = np.zeros(oshape[:3], np.uint8)
    cp = p.c()
    rc = lib().orc_compact(C.byref(cp), _ptr(k), _ptr(v), _ptr(modality), per_head, _ptr(keep_idx),
                           _ptr(n_out), _ptr(k_out), _ptr(v_out), _ptr(mod_out))
    if rc:
        raise ValueError("orc_compact: bad index")
    return k_out, v_out, mod_out


def prune_layer(p: Params, q, k, v, modality, seq_lens, budgets, total_budget=None, lse=None):
    q, k, v = _np(q, _elem(p)), _np(k, _elem(p)), _np(v, _elem(p))
    modality = _np(modality, np.uint8)
    seq_lens = _np(seq_lens, np.int32)
    budgets = _np(budgets, np.int32)
    total_budget = _np(total_budget, np.int32)
    lse = _np(lse, np.float64)
    per_head = int(modality.ndim == 3)
    sshape = (p.batch, p.n_kv_heads, p.max_len)
    oshape = (p.batch, p.n_kv_heads, p.out_capacity, p.head_dim)
    out = dict(
        score_self=np.zeros(sshape, np.float32), score_cross=np.zeros(sshape, np.float32),
        keep_idx=np.full(oshape[:3], -1, np.int32), n_out=np.zeros(oshape[:2], np.int32),
        flags=np.zeros(oshape[:2], np.int32), margins=np.zeros(oshape[:2] + (4, 2), np.float32),
        k_out=np.zeros(oshape, k.dtype), v_out=np.zeros(oshape, v.dtype),
        mod_out=np.zeros(oshape[:3], np.uint8))
    cp = p.c()
    rc = lib().orc_prune_layer(C.byref(cp), _ptr(q), _ptr(k), _ptr(v), _ptr(modality), per_head,
                               _ptr(seq_lens), _ptr(budgets), _ptr(total_budget), _ptr(lse),
                               _ptr(out["score_self"]), _ptr(out["score_cross"]),
                               _ptr(out["keep_idx"]), _ptr(out["n_out"]), _ptr(out["flags"]),
                               _ptr(out["margins"]), _ptr(out["k_out"]), _ptr(out["v_out"]),
                               _ptr(out["mod_out"]))
    if rc:
        raise ValueError("orc_prune_layer: bad argument")
    return out


def decode_attn(p: Params, q, k, v, n_rows):
    """Section 3.3: one query per head over the pruned cache with the n-softmax normaliser.
    q [B, Hq, d]; k, v [B, Hkv, out_capacity, d]; n_rows [B, Hkv] -> float64 [B, Hq, d]."""
    q, k, v = _np(q, _elem(p)), _np(k, _elem(p)), _np(v, _elem(p))
    n_rows = _np(n_rows, np.int32)
    out = np.zeros((p.batch, p.n_q_heads, p.head_dim), np.float64)
    cp = p.c()
    if lib().orc_decode_attn(C.byref(cp), _ptr(q), _ptr(k), _ptr(v), _ptr(n_rows), _ptr(out)):
        raise ValueError("orc_decode_attn: bad argument")
    return out


def decode_step(p: Params, q, k, v, n_rows, modality, query_label, acc_self, acc_cross, first: bool):
    """One appended token of the iteration loop: decode attention plus the running sums of Eq. 1.
    modality uint8 [B, Hkv, out_capacity]; query_label uint8 [B]; acc_self / acc_cross float64
    [B, Hkv, out_capacity], updated in place (overwritten when `first`).  Returns out float64 [B, Hq, d]."""
    q, k, v = _np(q, _elem(p)), _np(k, _elem(p)), _np(v, _elem(p))
    n_rows = _np(n_rows, np.int32)
    modality, query_label = _np(modality, np.uint8), _np(query_label, np.uint8)
    assert modality.shape == (p.batch, p.n_kv_heads, p.out_capacity) and query_label.shape == (p.batch,)
    assert acc_self.dtype == np.float64 and acc_self.flags.c_contiguous and acc_cross.flags.c_contiguous
    out = np.zeros((p.batch, p.n_q_heads, p.head_dim), np.float64)
    cp = p.c()
    if lib().orc_decode_step(C.byref(cp), _ptr(q), _ptr(k), _ptr(v), _ptr(n_rows), _ptr(modality),
                             _ptr(query_label), int(bool(first)), _ptr(out), _ptr(acc_self), _ptr(acc_cross)):
        raise ValueError("orc_decode_step: bad argument")
    return out


def js_divergence(hist_p, hist_q) -> float:
    hp, hq = _np(hist_p, np.int64), _np(hist_q, np.int64)
    assert hp.shape == hq.shape and hp.ndim == 1
    return float(lib().orc_js_divergence(_ptr(hp), _ptr(hq), C.c_int(hp.size)))


def weight_histogram(p: Params, q, k, modality, seq_lens, near_eps: float = 0.0):
    """Histograms of log2(attention weight) of the window, intra- and inter-modality, and their JS divergence.
    Returns (hist int64 [B,Hkv,2,HIST_BINS], near int64 (same shape), js float64 [B,Hkv], js_all float)."""
    q, k = _np(q, _elem(p)), _np(k, _elem(p))
    modality = _np(modality, np.uint8)
    seq_lens = _np(seq_lens, np.int32)
    per_head = int(modality.ndim == 3)
    hist = np.zeros((p.batch, p.n_kv_heads, 2, HIST_BINS), np.int64)
    near = np.zeros_like(hist)
    js = np.zeros((p.batch, p.n_kv_heads), np.float64)
    js_all = C.c_double(0.0)
    cp = p.c()
    if lib().orc_weight_histogram(C.byref(cp), _ptr(q), _ptr(k), _ptr(modality), per_head, _ptr(seq_lens),
                                  _ptr(hist), _ptr(near), C.c_double(near_eps), _ptr(js), C.byref(js_all)):
        raise ValueError("orc_weight_histogram: bad argument")
    return hist, near, js, float(js_all.value)
