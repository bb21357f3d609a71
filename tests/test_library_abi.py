"""CPU-side checks of the C interface: the library loads, exports every declared symbol, and
rejects bad arguments on the host before anything is enqueued.  No kernel runs here."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def csp():
    from paper_2412_04652_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def test_every_declared_symbol_is_exported(csp):
    header = open(os.path.join(ROOT, "include", "csp.h")).read()
    declared = set(re.findall(r"\b(csp_[a-z0-9_]+)\s*\(", header))
    assert declared == set(csp.EXPORTS)
    for name in declared:
        assert hasattr(csp.lib(), name), name


def test_struct_layout_matches_header(csp):
    assert C.sizeof(csp.CParams) == 14 * 4
    assert C.sizeof(csp.CTensor) == 32


def test_status_strings(csp):
    assert csp.status_string(csp.OK) == "ok"
    assert len({csp.status_string(i) for i in range(7)}) == 7


def test_workspace_size_formula(csp):
    p = csp.Params(2, 8, 4, 128, 32, 32, 1000, 300)
    scores = ((2 * 4 * 1000 * 4 + 255) // 256) * 256
    idx = ((2 * 4 * 300 * 4 + 255) // 256) * 256
    order = 256                  # one int32 per sequence, rounded up
    assert csp.workspace_bytes(p) == 256 + 4 * scores + idx + order
    assert csp.host_staging_bytes(p) > csp.workspace_bytes(p)


@pytest.mark.parametrize("field,value,code", [
    ("n_q_heads", 7, 1),        # not a multiple of the KV heads
    ("head_dim", 96, 2),        # row bytes not 128/256/512
    ("window", 33, 2),
    ("n_q_heads", 64, 2),       # group of 16
    ("dtype", 5, 2),
    ("combine", 3, 1),
    ("n", -1.0, 1),
    ("recent", -1, 1),
])
def test_bad_parameters_are_rejected_on_the_host(csp, field, value, code):
    p = csp.Params(1, 8, 4, 128, 32, 32, 512, 128)
    setattr(p, field, value)
    assert csp.workspace_bytes(p) == 0
    cp = p.c()
    t = csp.CTensor(256, 1, 1, 128)
    rc = csp.lib().csp_score(C.byref(cp), t, t, 256, 0, 0, 256, None, 256, 256, 256, 1 << 30, None)
    assert rc == code


def test_null_misaligned_and_small_workspace(csp):
    p = csp.Params(1, 8, 4, 128, 32, 32, 512, 128)
    cp = p.c()
    good = csp.CTensor(4096, 4 * 512 * 128, 512 * 128, 128)
    l = csp.lib()
    assert l.csp_score(C.byref(cp), good, good, None, 0, 0, 256, None, 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    odd = csp.CTensor(4096 + 2, 4 * 512 * 128, 512 * 128, 128)
    assert l.csp_score(C.byref(cp), good, odd, 256, 0, 0, 256, None, 256, 256, 256, 1 << 30, None) == csp.ERR_UNSUPPORTED
    bad_stride = csp.CTensor(4096, 4 * 512 * 128, 512 * 128, 129)
    assert l.csp_score(C.byref(cp), good, bad_stride, 256, 0, 0, 256, None, 256, 256, 256, 1 << 30, None) == csp.ERR_UNSUPPORTED
    assert l.csp_score(C.byref(cp), good, good, 256, 0, 0, 256, None, 256, 256, 256, 16, None) == csp.ERR_WORKSPACE
    assert l.csp_score(C.byref(cp), good, good, 256, 0, 0, 256, None, 256, 256, None, 1 << 30, None) == csp.ERR_WORKSPACE
    assert l.csp_select(C.byref(cp), 256, 256, 256, 0, 0, 256, None, None, 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    assert l.csp_compact(C.byref(cp), good, good, None, 0, 0, 256, 256, good, good, 256, None) == csp.ERR_INVALID_ARG
    assert l.csp_prune_layer(C.byref(cp), good, good, good, 256, 0, 0, 256, 256, None, None, good, good, None,
                             None, None, None, None, 256, 1 << 30, None) == csp.ERR_INVALID_ARG


def test_later_entry_points_reject_bad_arguments_on_the_host(csp):
    """The decode step, the histogram diagnostic, the paged decode call and the probe check their arguments before
    any CUDA call, so the refusals are the same with and without a device."""
    p = csp.Params(1, 8, 4, 128, 1, 0, 512, 512)
    cp = p.c()
    good = csp.CTensor(4096, 4 * 512 * 128, 512 * 128, 128)
    l = csp.lib()
    # csp_decode_step: a missing label array, then a workspace that is too small
    assert l.csp_decode_step(C.byref(cp), good, good, good, 256, None, 0, 0, 256, 1, 256, 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    assert l.csp_decode_step(C.byref(cp), good, good, good, 256, 256, 0, 0, 256, 1, 256, 256, 256, 256, 64, None) == csp.ERR_WORKSPACE
    n = csp.lib().csp_decode_step_workspace_bytes(C.byref(cp))
    assert n > csp.decode_workspace_bytes(p) > 0
    # csp_weight_histogram: no histogram array; fp32 caches are not supported
    ps = csp.Params(1, 8, 4, 128, 32, 32, 512, 128)
    cps = ps.c()
    assert l.csp_weight_histogram(C.byref(cps), good, good, 256, 0, 0, 256, None, None, None, None, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    pf = csp.Params(1, 8, 4, 64, 32, 32, 512, 128, dtype=csp.F32)
    cpf = pf.c()
    assert l.csp_weight_histogram(C.byref(cpf), good, good, 256, 0, 0, 256, None, 256, None, None, 256, 1 << 30, None) == csp.ERR_UNSUPPORTED
    # csp_decode_attn_paged: pages that do not hold whole 128-key tiles, a table that does not cover the capacity
    bad_rows = csp.CPages(256, 8, 64, 16)
    assert l.csp_decode_attn_paged(C.byref(cp), good, good, good, C.byref(bad_rows), 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    short_table = csp.CPages(256, 2, 128, 16)
    assert l.csp_decode_attn_paged(C.byref(cp), good, good, good, C.byref(short_table), 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    assert l.csp_decode_attn_paged(C.byref(cp), good, good, good, None, 256, 256, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    # csp_select_compact: no row-count array, a misaligned output, a workspace that is too small
    odd = csp.CTensor(4096 + 2, 4 * 512 * 128, 512 * 128, 128)
    assert l.csp_select_compact(C.byref(cps), 256, 256, good, good, 256, 0, 0, 256, 256, None, good, good, None, None,
                                None, 256, 1 << 30, None) == csp.ERR_INVALID_ARG
    assert l.csp_select_compact(C.byref(cps), 256, 256, good, good, 256, 0, 0, 256, 256, None, good, odd, None, 256,
                                None, 256, 1 << 30, None) == csp.ERR_UNSUPPORTED
    assert l.csp_select_compact(C.byref(cps), 256, 256, good, good, 256, 0, 0, 256, 256, None, good, good, None, 256,
                                None, 256, 64, None) == csp.ERR_WORKSPACE
    # csp_probe_ex2_rate: iteration count out of range
    out = C.c_int64(0)
    assert l.csp_probe_ex2_rate(0, 0, None, 0, C.byref(out), None) == csp.ERR_INVALID_ARG
    assert l.csp_probe_ex2_rate(0, 1 << 21, None, 0, C.byref(out), None) == csp.ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_without_a_gpu_the_path_fails_loudly(csp):
    """There is no CPU fallback: with valid arguments and no device the call reports an error."""
    p = csp.Params(1, 8, 4, 128, 32, 32, 512, 128)
    cp = p.c()
    good = csp.CTensor(4096, 4 * 512 * 128, 512 * 128, 128)
    rc = csp.lib().csp_score(C.byref(cp), good, good, 256, 0, 0, 256, None, 256, 256, 256, 1 << 30, None)
    assert rc in (csp.ERR_CUDA, csp.ERR_ARCH)
