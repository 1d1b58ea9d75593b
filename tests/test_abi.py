"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2609_39813_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "bsp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bsp_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(built):
    lib = ctypes.CDLL(built)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_header(built):
    from paper_2609_39813_b200 import binding
    assert binding.exported_names() == _declared()
    l = binding.lib()
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(binding.ERR_WORKSPACE)
    # workspace queries are pure host arithmetic
    assert l.bsp_norm_bwd_workspace_bytes(4096, 1024) > 0
    assert l.bsp_linear_wgrad_workspace_bytes(4096, 4096, 1024, binding.READ_FORWARD) == 256
    assert l.bsp_mc_stats_workspace_bytes(10) % 256 == 0


def test_struct_layouts_match_header(built):
    from paper_2609_39813_b200 import binding as b
    assert ctypes.sizeof(b.Key) == 24 and ctypes.sizeof(b.Quant) == 24
    assert ctypes.sizeof(b.Diag) == 24 and ctypes.sizeof(b.UseResult) == 88
    assert ctypes.sizeof(b.VerdictRule) == 48 and ctypes.sizeof(b.AttnFp8) == 72
    assert ctypes.sizeof(b.NormLinearDesc) == 120 and ctypes.sizeof(b.AttnDesc) == 104
    assert ctypes.sizeof(b.McLayout) == 15 * ctypes.sizeof(ctypes.c_size_t)
    d = b.NormLinearDesc()
    d.T, d.C, d.O = 64, 128, 128
    full = b.bsp_mc_check_workspace_bytes(d, 16)
    assert full > 64 * 128
    # the layout query is host arithmetic: offsets are distinct, aligned and inside the workspace
    lay = b.bsp_mc_check_layout(d, 16)
    offs = [getattr(lay, n) for n, _ in b.McLayout._fields_]
    assert len(set(offs)) == len(offs) and all(o % 256 == 0 and o < full for o in offs)
    # a smaller code buffer makes a smaller workspace
    d.draw_buffer_bytes = 2 * 128 * 64
    assert b.bsp_mc_check_workspace_bytes(d, 16) < full


def test_check_argument_errors_need_no_gpu(built):
    from paper_2609_39813_b200 import binding as b
    import ctypes as C
    l = b.lib()
    d = b.NormLinearDesc()
    d.T, d.C, d.O = 64, 128, 128
    d.x = d.gamma = d.W = d.dY = 4096
    res = (b.UseResult * 12)()
    n = C.c_int(0)
    # fewer than four draws, and a rule whose hold threshold lies above its fail threshold
    assert l.bsp_mc_check(C.byref(d), 3, None, res, C.byref(n), 4096, 1 << 30, None, None) == b.ERR_ARG
    bad = b.rule(qprime_hold=5.0, qprime_fail=4.0)
    assert l.bsp_mc_check(C.byref(d), 8, C.byref(bad), res, C.byref(n), 4096, 1 << 30, None, None) == b.ERR_ARG
    assert l.bsp_mc_check(C.byref(d), 8, None, res, C.byref(n), None, 0, None, None) == b.ERR_WORKSPACE
    a = b.AttnDesc()
    a.B, a.H, a.S, a.Dh, a.dtype = 1, 1, 64, 64, b.BF16
    a.q = a.k = a.v = a.dO = 4096
    a.fp8_operands = 1                       # the FP8-operand mode needs its two scales
    assert l.bsp_mc_check_attn(C.byref(a), 8, None, res, C.byref(n), 4096, 1 << 30, None, None) == b.ERR_ARG
    a.fp8_operands, a.Dh = 0, 128
    assert l.bsp_mc_check_attn(C.byref(a), 8, None, res, C.byref(n), 4096, 1 << 30, None, None) == b.ERR_UNSUPPORTED
    assert l.bsp_selftest_bounded_wait(0, 4096, None) == b.ERR_ARG


def test_host_side_argument_errors_need_no_gpu(built):
    from paper_2609_39813_b200 import binding as b
    l = b.lib()
    k = b.key(0, 1, 0)
    q = b.quant(b.E4M3, b.ROUND_NEAREST, 1.0)
    assert l.bsp_round(None, b.F32, 16, q, k, 0, None, None, None) == b.ERR_ARG
    assert l.bsp_round(16, b.F32, 16, q, k, 0, 24, None, None) == b.ERR_ALIGN       # misaligned codes
    assert l.bsp_round(16, 7, 16, q, k, 0, 32, None, None) == b.ERR_ARG             # bad dtype
    bad = b.key(0, 1 << 24, 0)
    assert l.bsp_philox_fill(bad, 4, 16, None) == b.ERR_ARG
    assert l.bsp_round_2d(16, b.F32, 8, 24, q, k, 32, None, 0, None, None) == b.ERR_UNSUPPORTED
    assert l.bsp_norm_bwd(0, 16, 0, 8, 16, 16, None, 16, None, 16, 0, 0, 0, None, q, k, 16, None, None,
                          None, 0, None, None) == b.ERR_WORKSPACE
    assert l.bsp_norm_bwd(0, 16, 0, 8, 16, 16, None, 16, None, 16, 0, 0, 5, None, q, k, 16, None, None,
                          None, 0, None, None) == b.ERR_ARG                          # dx_read out of range
    assert l.bsp_linear_wgrad(8, 16, 16, 16, q, b.READ_FORWARD, 16, q, 8, 16, None, None, None, None, 0,
                              None, None) == b.ERR_ALIGN                             # ld_t not a multiple of 16
    # the one-kernel attention backward: head width, missing gradient, misaligned operand (in that order)
    args = lambda Dh, q_, dq_: (1, 1, 128, Dh, 1, 0.125, q_, 32, 48, 64, b.BF16, 80, 96, dq_, 112, 128, None, None)
    assert l.bsp_attn_bwd_dterm_fused(*args(128, 16, 144)) == b.ERR_UNSUPPORTED
    assert l.bsp_attn_bwd_dterm_fused(*args(64, 16, None)) == b.ERR_ARG
    assert l.bsp_attn_bwd_dterm_fused(*args(64, 24, 144)) == b.ERR_ALIGN
