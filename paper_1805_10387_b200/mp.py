"""Python binding of the C-ABI library (include/mp.h): argument marshalling only.

Every function below has the name of the C entry point it calls and does nothing but turn
torch tensors (device memory), Python numbers and the current torch stream into the plain
pointers and sizes of the C signature.  All arithmetic runs in the CUDA kernels of the
library.  There is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

MP_OK = 0
MP_ERR_INVALID_ARG, MP_ERR_ALIGNMENT, MP_ERR_UNSUPPORTED_ARCH = -1, -2, -3
MP_ERR_CUDA, MP_ERR_TIMEOUT, MP_ERR_NOMEM, MP_ERR_TOO_LARGE = -4, -5, -6, -7
MP_OPT_ADAM, MP_OPT_MOMENTUM = 0, 1
MP_OP_FWD, MP_OP_DGRAD, MP_OP_WGRAD = 0, 1, 2
MP_LOG_CAPACITY = 4096
MP_ACT_NONE, MP_ACT_RELU, MP_ACT_CLIPPED_RELU = 0, 1, 2


class MpError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"mp error {code}: {msg}")
        self.code = code


class ScalerConfig(C.Structure):
    _fields_ = [("init_scale", C.c_float), ("min_scale", C.c_float), ("max_scale", C.c_float),
                ("growth_interval", C.c_int32), ("dynamic", C.c_int32),
                ("overflow_tolerance", C.c_int32)]


class OptimConfig(C.Structure):
    _fields_ = [("kind", C.c_int32), ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float),
                ("eps", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float)]


class StateHost(C.Structure):
    _fields_ = [("scale", C.c_float), ("min_scale", C.c_float), ("max_scale", C.c_float),
                ("growth_interval", C.c_int32), ("dynamic", C.c_int32), ("good_steps", C.c_int32),
                ("found_inf", C.c_int32), ("status", C.c_int32),
                ("overflow_tolerance", C.c_int32), ("strikes", C.c_int32), ("t", C.c_int64),
                ("step", C.c_int64), ("skipped", C.c_int64)]


class LogRecord(C.Structure):
    _fields_ = [("step", C.c_int64), ("t", C.c_int64), ("scale_before", C.c_float),
                ("scale_after", C.c_float), ("found_inf", C.c_int32), ("good_steps", C.c_int32)]


# name -> (restype, argtypes): the declarations of include/mp.h
_p, _i64, _i32, _sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
SIGNATURES = {
    "mp_linear_fwd": (_i32, [_p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _sz, _p]),
    "mp_linear_bwd_dgrad": (_i32, [_p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _sz, _p]),
    "mp_linear_bwd_wgrad": (_i32, [_p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _p, _sz, _p]),
    "mp_linear_bwd_wgrad_static": (_i32, [_p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _p]),
    "mp_static_scratch_bytes": (_sz, []),
    "mp_linear_fwd_grouped": (_i32, [_i32, _p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _sz, _p]),
    "mp_linear_bwd_dgrad_grouped": (_i32, [_i32, _p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _sz, _p]),
    "mp_linear_bwd_wgrad_grouped": (_i32, [_i32, _p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _p, _p, _sz, _p]),
    "mp_linear_fwd_act_grouped": (_i32, [_i32, _p, _i64, _p, _i64, _p, _p, _i64, _i64, _i64, _i64, _i32,
                                         C.c_float, _p, _sz, _p]),
    "mp_max_group": (_i32, []),
    "mp_gemm_workspace_bytes_grouped": (_sz, [_i32, _i64, _i64, _i64, _i32]),
    "mp_linear_fwd_act": (_i32, [_p, _i64, _p, _i64, _p, _p, _i64, _i64, _i64, _i64, _i32, C.c_float, _p, _sz, _p]),
    "mp_linear_bwd_dgrad_act": (_i32, [_p, _i64, _p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _i32,
                                       C.c_float, _p, _sz, _p]),
    "mp_bias_grad": (_i32, [_p, _i64, _p, _i64, _i64, _p, _p, _sz, _p]),
    "mp_bias_grad_workspace_bytes": (_sz, [_i64, _i64]),
    "mp_bias_grad_grouped": (_i32, [_i32, _p, _i64, _p, _i64, _i64, _p, _p, _sz, _p]),
    "mp_lstm_cell_fwd": (_i32, [_p, _i64, _p, _p, _p, _i64, _i64, _p]),
    "mp_lstm_cell_bwd": (_i32, [_p, _i64, _p, _p, _p, _p, _p, _i64, _p, _i64, _i64, _p]),
    "mp_master_update": (_i32, [_p, _p, C.POINTER(OptimConfig), _i32, _p]),
    "mp_loss_scale_update": (_i32, [_p, _p]),
    "mp_gemm_workspace_bytes": (_sz, [_i64, _i64, _i64, _i32]),
    "mp_scale_upstream": (_i32, [_p, _p, _i64, _p, _p]),
    "mp_check_finite": (_i32, [_p, _i64, _p, _p]),
    "mp_state_create": (_i32, [C.POINTER(ScalerConfig), C.POINTER(_p)]),
    "mp_state_destroy": (_i32, [_p]),
    "mp_state_read": (_i32, [_p, C.POINTER(StateHost), _p]),
    "mp_state_write": (_i32, [_p, C.POINTER(StateHost), _p]),
    "mp_state_export_flag": (_i32, [_p, _p, _p]),
    "mp_state_import_flag": (_i32, [_p, _p, _p]),
    "mp_state_read_log": (_i32, [_p, C.POINTER(LogRecord), _i32, C.POINTER(_i32), _p]),
    "mp_update_plan_create": (_i32, [_i32, C.POINTER(_p), C.POINTER(_p), C.POINTER(_p),
                                     C.POINTER(_p), C.POINTER(_p), C.POINTER(_i64), C.POINTER(_p)]),
    "mp_update_plan_destroy": (_i32, [_p]),
    "mp_selftest_wait_timeout": (_i32, [_p, _i64, _p, _i64, _p, _i64, _i64, _i64, _i64, _i64, _p, _p]),
    "mp_gemm_device_status": (_i32, [C.POINTER(_i32)]),
    "mp_last_error": (C.c_char_p, []),
    "mp_kernel_launch_count": (_i64, []),
}

_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Loads the shared library (building it first if the sources are newer)."""
    global _lib
    if _lib is None:
        path = _build.build()
        if not os.path.exists(path):
            raise ImportError(f"CUDA library {path} is missing and could not be built")
        L = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(rc: int):
    if rc != MP_OK:
        raise MpError(rc, lib().mp_last_error().decode())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype) -> int:
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"expected a CUDA tensor of {dtype}, got {t.device} {t.dtype}")
    return t.data_ptr()


def _mat(t: torch.Tensor):
    """(pointer, leading dimension) of a row-major 2-D FP16 CUDA tensor."""
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("expected a 2-D tensor with unit column stride")
    return _dev(t, torch.float16), t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def last_error() -> str:
    return lib().mp_last_error().decode()


def mp_kernel_launch_count() -> int:
    return int(lib().mp_kernel_launch_count())


def mp_gemm_workspace_bytes(M: int, K: int, N: int, op: int) -> int:
    return int(lib().mp_gemm_workspace_bytes(M, K, N, op))


def _ws(workspace):
    if workspace is None:
        return None, 0
    return workspace.data_ptr(), workspace.numel() * workspace.element_size()


def mp_linear_fwd(X16, W16, Y16, workspace=None):
    (x, ldx), (w, ldw), (y, ldy) = _mat(X16), _mat(W16), _mat(Y16)
    M, K = X16.shape
    N = W16.shape[1]
    assert W16.shape[0] == K and tuple(Y16.shape) == (M, N)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_fwd(x, ldx, w, ldw, y, ldy, M, K, N, ws, nb, _stream()))


def mp_linear_bwd_dgrad(dY16, W16, dX16, workspace=None):
    (dy, lddy), (w, ldw), (dx, lddx) = _mat(dY16), _mat(W16), _mat(dX16)
    M, N = dY16.shape
    K = W16.shape[0]
    assert W16.shape[1] == N and tuple(dX16.shape) == (M, K)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_bwd_dgrad(dy, lddy, w, ldw, dx, lddx, M, K, N, ws, nb, _stream()))


def mp_linear_bwd_wgrad(X16, dY16, dW16, state=None, workspace=None):
    (x, ldx), (dy, lddy), (dw, lddw) = _mat(X16), _mat(dY16), _mat(dW16)
    M, K = X16.shape
    N = dY16.shape[1]
    assert dY16.shape[0] == M and tuple(dW16.shape) == (K, N)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_bwd_wgrad(x, ldx, dy, lddy, dw, lddw, M, K, N,
                                     state.handle if state is not None else None, ws, nb, _stream()))


def mp_linear_bwd_wgrad_static(X16, dY16, dW16, state=None):
    """Weight gradient with the library's built-in scratch: for callers that cannot allocate
    device memory or lend a workspace.  Same result as mp_linear_bwd_wgrad."""
    (x, ldx), (dy, lddy), (dw, lddw) = _mat(X16), _mat(dY16), _mat(dW16)
    M, K = X16.shape
    N = dY16.shape[1]
    assert dY16.shape[0] == M and tuple(dW16.shape) == (K, N)
    _check(lib().mp_linear_bwd_wgrad_static(x, ldx, dy, lddy, dw, lddw, M, K, N,
                                            state.handle if state is not None else None, _stream()))


def mp_max_group() -> int:
    return int(lib().mp_max_group())


def mp_gemm_workspace_bytes_grouped(count: int, M: int, K: int, N: int, op: int) -> int:
    return int(lib().mp_gemm_workspace_bytes_grouped(count, M, K, N, op))


def _mats(ts):
    """(array of pointers, common leading dimension, common shape) of same-shaped 2-D FP16 tensors."""
    pl = [_mat(t) for t in ts]
    assert len({ld for _, ld in pl}) == 1 and len({tuple(t.shape) for t in ts}) == 1, \
        "grouped problems share one shape and one leading dimension"
    return (C.c_void_p * len(ts))(*[p for p, _ in pl]), pl[0][1], tuple(ts[0].shape)


def mp_linear_fwd_grouped(X16s, W16s, Y16s, workspace=None):
    (x, ldx, (M, K)), (w, ldw, (K2, N)), (y, ldy, ys) = _mats(X16s), _mats(W16s), _mats(Y16s)
    assert K2 == K and ys == (M, N) and len(X16s) == len(W16s) == len(Y16s)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_fwd_grouped(len(X16s), x, ldx, w, ldw, y, ldy, M, K, N, ws, nb, _stream()))


def mp_linear_fwd_act_grouped(X16s, W16s, bias16s, Y16s, act=MP_ACT_NONE, clip=20.0, workspace=None):
    (x, ldx, (M, K)), (w, ldw, (K2, N)), (y, ldy, ys) = _mats(X16s), _mats(W16s), _mats(Y16s)
    assert K2 == K and ys == (M, N) and len(X16s) == len(W16s) == len(Y16s)
    b = None
    if bias16s is not None:
        assert len(bias16s) == len(X16s) and all(t.numel() == N and t.is_contiguous() for t in bias16s)
        b = (C.c_void_p * len(bias16s))(*[_dev(t, torch.float16) for t in bias16s])
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_fwd_act_grouped(len(X16s), x, ldx, w, ldw, b, y, ldy, M, K, N, act, clip, ws, nb,
                                           _stream()))


def mp_linear_bwd_dgrad_grouped(dY16s, W16s, dX16s, workspace=None):
    (dy, lddy, (M, N)), (w, ldw, (K, N2)), (dx, lddx, xs) = _mats(dY16s), _mats(W16s), _mats(dX16s)
    assert N2 == N and xs == (M, K) and len(dY16s) == len(W16s) == len(dX16s)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_bwd_dgrad_grouped(len(dY16s), dy, lddy, w, ldw, dx, lddx, M, K, N, ws, nb, _stream()))


def mp_linear_bwd_wgrad_grouped(X16s, dY16s, dW16s, state=None, workspace=None):
    (x, ldx, (M, K)), (dy, lddy, (M2, N)), (dw, lddw, ws_) = _mats(X16s), _mats(dY16s), _mats(dW16s)
    assert M2 == M and ws_ == (K, N) and len(X16s) == len(dY16s) == len(dW16s)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_bwd_wgrad_grouped(len(X16s), x, ldx, dy, lddy, dw, lddw, M, K, N,
                                             state.handle if state is not None else None, ws, nb, _stream()))


def mp_static_scratch_bytes() -> int:
    return int(lib().mp_static_scratch_bytes())


def mp_linear_fwd_act(X16, W16, bias16, Y16, act=MP_ACT_NONE, clip=20.0, workspace=None):
    (x, ldx), (w, ldw), (y, ldy) = _mat(X16), _mat(W16), _mat(Y16)
    M, K = X16.shape
    N = W16.shape[1]
    assert W16.shape[0] == K and tuple(Y16.shape) == (M, N)
    b = None
    if bias16 is not None:
        assert bias16.numel() == N and bias16.is_contiguous()
        b = _dev(bias16, torch.float16)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_fwd_act(x, ldx, w, ldw, b, y, ldy, M, K, N, act, clip, ws, nb, _stream()))


def mp_linear_bwd_dgrad_act(dY16, W16, A16, dX16, act=MP_ACT_NONE, clip=20.0, workspace=None):
    (dy, lddy), (w, ldw), (dx, lddx) = _mat(dY16), _mat(W16), _mat(dX16)
    M, N = dY16.shape
    K = W16.shape[0]
    assert W16.shape[1] == N and tuple(dX16.shape) == (M, K)
    a, lda = (None, 0) if A16 is None else _mat(A16)
    ws, nb = _ws(workspace)
    _check(lib().mp_linear_bwd_dgrad_act(dy, lddy, w, ldw, a, lda, dx, lddx, M, K, N, act, clip, ws, nb,
                                         _stream()))


def mp_bias_grad_workspace_bytes(M: int, N: int) -> int:
    return int(lib().mp_bias_grad_workspace_bytes(M, N))


def mp_bias_grad(dY16, db16, state=None, workspace=None):
    dy, lddy = _mat(dY16)
    M, N = dY16.shape
    assert db16.numel() == N and db16.is_contiguous()
    ws, nb = _ws(workspace)
    _check(lib().mp_bias_grad(dy, lddy, _dev(db16, torch.float16), M, N,
                              state.handle if state is not None else None, ws, nb, _stream()))


def mp_bias_grad_grouped(dY16s, db16s, state=None, workspace=None):
    dy, lddy, (M, N) = _mats(dY16s)
    assert len(db16s) == len(dY16s) and all(t.numel() == N and t.is_contiguous() for t in db16s)
    db = (C.c_void_p * len(db16s))(*[_dev(t, torch.float16) for t in db16s])
    ws, nb = _ws(workspace)
    _check(lib().mp_bias_grad_grouped(len(dY16s), dy, lddy, db, M, N,
                                      state.handle if state is not None else None, ws, nb, _stream()))


def mp_lstm_cell_fwd(G16, c_prev16, c_new16, h16):
    g, ldg = _mat(G16)
    M, H = c_prev16.shape
    assert G16.shape == (M, 4 * H) and c_prev16.is_contiguous() and c_new16.is_contiguous() and h16.is_contiguous()
    _check(lib().mp_lstm_cell_fwd(g, ldg, _dev(c_prev16, torch.float16), _dev(c_new16, torch.float16),
                                  _dev(h16, torch.float16), M, H, _stream()))


def mp_lstm_cell_bwd(G16, c_prev16, c_new16, dh16, dc_in16, dG16, dc_prev16):
    g, ldg = _mat(G16)
    dg, lddg = _mat(dG16)
    M, H = c_prev16.shape
    for t in (c_prev16, c_new16, dh16, dc_prev16):
        assert t.is_contiguous() and tuple(t.shape) == (M, H)
    _check(lib().mp_lstm_cell_bwd(g, ldg, _dev(c_prev16, torch.float16), _dev(c_new16, torch.float16),
                                  _dev(dh16, torch.float16),
                                  _dev(dc_in16, torch.float16) if dc_in16 is not None else None,
                                  dg, lddg, _dev(dc_prev16, torch.float16), M, H, _stream()))


def mp_master_update(plan, state, opt: OptimConfig, check_mode: int = 0):
    _check(lib().mp_master_update(plan.handle, state.handle, C.byref(opt), check_mode, _stream()))


def mp_loss_scale_update(state):
    _check(lib().mp_loss_scale_update(state.handle, _stream()))


def mp_scale_upstream(g32, dY16, state):
    assert g32.numel() == dY16.numel() and g32.is_contiguous() and dY16.is_contiguous()
    _check(lib().mp_scale_upstream(_dev(g32, torch.float32), _dev(dY16, torch.float16),
                                   g32.numel(), state.handle, _stream()))


def mp_check_finite(g16, state):
    assert g16.is_contiguous()
    _check(lib().mp_check_finite(_dev(g16, torch.float16), g16.numel(), state.handle, _stream()))


def mp_state_export_flag(state, word):
    """word[0] (int32 CUDA tensor) = the state's overflow flag, on the stream."""
    _check(lib().mp_state_export_flag(state.handle, _dev(word, torch.int32), _stream()))


def mp_state_import_flag(state, word):
    """ORs word[0] != 0 (int32 CUDA tensor) into the state's overflow flag, on the stream."""
    _check(lib().mp_state_import_flag(state.handle, _dev(word, torch.int32), _stream()))


def mp_selftest_wait_timeout(X16, W16, Y16, wait_us: int, state=None):
    """Error-path self-test: one tile of the forward kernel whose loader fetches nothing, so its
    bounded waits run out after wait_us microseconds and it reports MP_ERR_TIMEOUT."""
    (x, ldx), (w, ldw), (y, ldy) = _mat(X16), _mat(W16), _mat(Y16)
    M, K = X16.shape
    N = W16.shape[1]
    _check(lib().mp_selftest_wait_timeout(x, ldx, w, ldw, y, ldy, M, K, N, int(wait_us),
                                          state.handle if state is not None else None, _stream()))


def mp_gemm_device_status() -> int:
    out = C.c_int(0)
    _check(lib().mp_gemm_device_status(C.byref(out)))
    return out.value


class State:
    """Owner of an mp_state handle (device-resident loss-scale state)."""

    def __init__(self, init_scale=65536.0, growth_interval=1000, min_scale=1.0,
                 max_scale=2.0 ** 24, dynamic=True, overflow_tolerance=1):
        cfg = ScalerConfig(init_scale, min_scale, max_scale, growth_interval, 1 if dynamic else 0,
                           overflow_tolerance)
        h = C.c_void_p()
        _check(lib().mp_state_create(C.byref(cfg), C.byref(h)))
        self.handle = h

    def read(self) -> StateHost:
        out = StateHost()
        _check(lib().mp_state_read(self.handle, C.byref(out), _stream()))
        return out

    def write(self, host: StateHost):
        _check(lib().mp_state_write(self.handle, C.byref(host), _stream()))

    def read_log(self, max_records=MP_LOG_CAPACITY):
        buf = (LogRecord * max_records)()
        n = C.c_int(0)
        _check(lib().mp_state_read_log(self.handle, buf, max_records, C.byref(n), _stream()))
        return [buf[i] for i in range(n.value)]

    def close(self):
        if self.handle is not None and _lib is not None:
            _lib.mp_state_destroy(self.handle)
        self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class UpdatePlan:
    """Owner of an mp_update_plan handle over lists of per-tensor CUDA buffers."""

    def __init__(self, g16, w32, m, v, w16):
        n = len(g16)
        self._keep = (g16, w32, m, v, w16)
        arr = lambda ts, dt: (C.c_void_p * n)(*[_dev(t, dt) if t.numel() else None for t in ts])
        counts = (C.c_int64 * n)(*[t.numel() for t in g16])
        for ts in (w32, m, w16) + ((v,) if v is not None else ()):
            assert [t.numel() for t in ts] == [t.numel() for t in g16]
        h = C.c_void_p()
        _check(lib().mp_update_plan_create(
            n, arr(g16, torch.float16), arr(w32, torch.float32), arr(m, torch.float32),
            arr(v, torch.float32) if v is not None else None, arr(w16, torch.float16), counts,
            C.byref(h)))
        self.handle = h
        self.total = sum(t.numel() for t in g16)

    def close(self):
        if self.handle is not None and _lib is not None:
            _lib.mp_update_plan_destroy(self.handle)
        self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
