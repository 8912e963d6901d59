"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "mp.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(mp_[a-z_0-9]+)\s*\(", src)))


def test_header_declares_the_five_calls():
    names = _declared()
    for n in ("mp_linear_fwd", "mp_linear_bwd_dgrad", "mp_linear_bwd_wgrad", "mp_master_update",
              "mp_loss_scale_update"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_1805_10387_b200 import build, mp
    path = build.build()
    L = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(L, name), name
    assert set(mp.SIGNATURES) == set(_declared())


def test_workspace_query_is_pure_host_logic():
    from paper_1805_10387_b200 import mp
    assert mp.mp_gemm_workspace_bytes(6400, 2048, 4096, mp.MP_OP_FWD) == 0
    assert mp.mp_gemm_workspace_bytes(8192, 1024, 1024, mp.MP_OP_WGRAD) > 0
    assert mp.mp_gemm_workspace_bytes(0, 8, 8, mp.MP_OP_FWD) == 0
    assert mp.mp_gemm_workspace_bytes(8, 8, 8, 7) == 0


def test_argument_errors_need_no_gpu():
    """Null pointers and bad sizes are rejected on the host before any CUDA call."""
    from paper_1805_10387_b200 import mp
    L = mp.lib()
    assert L.mp_linear_fwd(None, 8, None, 8, None, 8, 8, 8, 8, None, 0, None) == mp.MP_ERR_INVALID_ARG
    assert b"null" in L.mp_last_error()
    assert L.mp_loss_scale_update(None, None) == mp.MP_ERR_INVALID_ARG
    assert L.mp_master_update(None, None, None, 0, None) == mp.MP_ERR_INVALID_ARG
    assert L.mp_state_destroy(None) == mp.MP_OK and L.mp_update_plan_destroy(None) == mp.MP_OK
    buf = (ctypes.c_uint16 * 64)()
    p = ctypes.addressof(buf)
    p16 = (p + 15) // 16 * 16
    assert L.mp_linear_fwd(p16, 8, p16, 8, p16, 8, 0, 8, 8, None, 0, None) == mp.MP_ERR_INVALID_ARG
    assert L.mp_linear_fwd(p16, 4, p16, 8, p16, 8, 8, 8, 8, None, 0, None) == mp.MP_ERR_INVALID_ARG
    assert L.mp_linear_fwd(p16, 12, p16, 8, p16, 8, 8, 8, 8, None, 0, None) == mp.MP_ERR_ALIGNMENT
    assert L.mp_linear_fwd(p16 + 2, 8, p16, 8, p16, 8, 8, 8, 8, None, 0, None) == mp.MP_ERR_ALIGNMENT
    # the masked data gradient reads the layer input with 128-bit loads: checked on the host too
    args = lambda a16, lda: (p16, 8, p16, 8, a16, lda, p16, 8, 8, 8, 8, mp.MP_ACT_RELU, ctypes.c_float(0.0),
                             None, 0, None)
    assert L.mp_linear_bwd_dgrad_act(*args(p16 + 2, 8)) == mp.MP_ERR_ALIGNMENT
    assert L.mp_linear_bwd_dgrad_act(*args(p16, 12)) == mp.MP_ERR_ALIGNMENT
    assert L.mp_linear_bwd_dgrad_act(*args(p16, 4)) == mp.MP_ERR_INVALID_ARG
    assert L.mp_linear_bwd_dgrad_act(*args(None, 8)) == mp.MP_ERR_INVALID_ARG
    # the error-path self-test refuses more than one tile and limits outside 1 us .. 2 s
    st = lambda M, N, us: L.mp_selftest_wait_timeout(p16, 8, p16, 8, p16, 8, M, 8, N, us, None, None)
    assert st(8, 8, 0) == mp.MP_ERR_INVALID_ARG and st(8, 8, 3_000_000) == mp.MP_ERR_INVALID_ARG
    assert st(129, 8, 100) == mp.MP_ERR_INVALID_ARG and st(8, 257, 100) == mp.MP_ERR_INVALID_ARG
