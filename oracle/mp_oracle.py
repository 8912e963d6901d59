"""ctypes front end of the CPU oracle (mp_oracle.cpp) plus the step driver.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA path never imports this module and this
module never imports the CUDA package.

All FP16 data are numpy uint16 arrays of bit patterns; FP32 data are float32.
The step driver follows the paper's Sections 3.1-3.3 in their order: forward in
FP16 with FP32 accumulation, scale the upstream gradient by S, backward in FP16,
inspect the FP16 weight gradients, convert to FP32 and unscale, optimizer on the
FP32 master (skipped as a whole when any gradient is non-finite), FP16 working
copy rewritten, scale for the next iteration chosen.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mp_oracle.cpp")
_LIB = os.path.join(_HERE, "libmp_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA, no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
               "-shared", "-pthread", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


class _Scaler(C.Structure):
    _fields_ = [("S", C.c_float), ("s_min", C.c_float), ("s_max", C.c_float),
                ("interval", C.c_int32), ("dynamic", C.c_int32), ("good", C.c_int32),
                ("t", C.c_int64), ("step", C.c_int64), ("skipped", C.c_int64),
                ("tolerance", C.c_int32), ("strikes", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        p, i64, i32, f32 = C.c_void_p, C.c_int64, C.c_int, C.c_float
        L.orc_h2f.restype = f32; L.orc_h2f.argtypes = [C.c_uint16]
        L.orc_f2h.restype = C.c_uint16; L.orc_f2h.argtypes = [f32]
        L.orc_h2f_array.argtypes = [p, p, i64]
        L.orc_f2h_array.argtypes = [p, p, i64]
        for name in ("orc_linear_fwd", "orc_linear_bwd_dgrad", "orc_linear_bwd_wgrad"):
            getattr(L, name).argtypes = [p, i64, p, i64, p, i64, i64, i64, i64, i32]
            getattr(L, name).restype = None
        L.orc_linear_sampled.argtypes = [i32, p, i64, p, i64, i64, i64, i64, p, p, i64, p, p, p]
        L.orc_linear_exact.argtypes = [i32, p, i64, p, i64, i64, i64, i64, p, p, i32]
        L.orc_linear_fwd_act.argtypes = [p, i64, p, i64, p, p, i64, i64, i64, i64, i32, f32, i32]
        L.orc_linear_bwd_dgrad_act.argtypes = [p, i64, p, i64, p, i64, p, i64, i64, i64, i64, i32, f32, i32]
        L.orc_bias_grad.argtypes = [p, i64, p, i64, i64]
        L.orc_lstm_cell_fwd.argtypes = [p, i64, p, p, p, i64, i64]
        L.orc_lstm_cell_bwd.argtypes = [p, i64, p, p, p, p, p, i64, p, i64, i64]
        L.orc_scale_upstream.argtypes = [p, f32, p, i64]
        L.orc_found_inf.restype = i32; L.orc_found_inf.argtypes = [p, i64]
        L.orc_adam_update.argtypes = [p, p, p, p, p, i64, f32, f32, f32, f32, f32, f32, i64]
        L.orc_momentum_update.argtypes = [p, p, p, p, i64, f32, f32, f32, f32]
        L.orc_scaler_update.argtypes = [C.POINTER(_Scaler), i32]
        L.orc_hardware_threads.restype = i32
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _chk(a: np.ndarray, dtype) -> np.ndarray:
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a


def hardware_threads() -> int:
    return int(lib().orc_hardware_threads())


# ------------------------------------------------------------------ FP16
def h2f(h) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, np.float32)
    lib().orc_h2f_array(_ptr(h), _ptr(out), h.size)
    return out


def f2h(x) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, np.uint16)
    lib().orc_f2h_array(_ptr(x), _ptr(out), x.size)
    return out


# --------------------------------------------------------------- matmuls
def linear_fwd(X16, W16, nthreads=0) -> np.ndarray:
    """Y[M,N] = rn16(sum_k X[m,k] W[k,n]), FP32 running sum (Section 3.1)."""
    _chk(X16, np.uint16); _chk(W16, np.uint16)
    M, K = X16.shape; K2, N = W16.shape; assert K == K2
    Y = np.empty((M, N), np.uint16)
    lib().orc_linear_fwd(_ptr(X16), K, _ptr(W16), N, _ptr(Y), N, M, K, N,
                         nthreads or hardware_threads())
    return Y


def linear_bwd_dgrad(dY16, W16, nthreads=0) -> np.ndarray:
    """dX[M,K] = rn16(sum_n dY[m,n] W[k,n])."""
    _chk(dY16, np.uint16); _chk(W16, np.uint16)
    M, N = dY16.shape; K, N2 = W16.shape; assert N == N2
    dX = np.empty((M, K), np.uint16)
    lib().orc_linear_bwd_dgrad(_ptr(dY16), N, _ptr(W16), N, _ptr(dX), K, M, K, N,
                               nthreads or hardware_threads())
    return dX


def linear_bwd_wgrad(X16, dY16, nthreads=0) -> np.ndarray:
    """dW[K,N] = rn16(sum_m X[m,k] dY[m,n])."""
    _chk(X16, np.uint16); _chk(dY16, np.uint16)
    M, K = X16.shape; M2, N = dY16.shape; assert M == M2
    dW = np.empty((K, N), np.uint16)
    lib().orc_linear_bwd_wgrad(_ptr(X16), K, _ptr(dY16), N, _ptr(dW), N, M, K, N,
                               nthreads or hardware_threads())
    return dW


ACT = {"none": 0, "relu": 1, "clipped_relu": 2}


def linear_fwd_act(X16, W16, b16=None, act="none", clip=20.0, nthreads=0) -> np.ndarray:
    """Y = rn16(act(X W + b)): bias added to the FP32 sum, activation on the FP32 value."""
    _chk(X16, np.uint16); _chk(W16, np.uint16)
    M, K = X16.shape; K2, N = W16.shape; assert K == K2
    if b16 is not None:
        _chk(b16, np.uint16); assert b16.shape == (N,)
    Y = np.empty((M, N), np.uint16)
    lib().orc_linear_fwd_act(_ptr(X16), K, _ptr(W16), N, _ptr(b16) if b16 is not None else None,
                             _ptr(Y), N, M, K, N, ACT[act], clip, nthreads or hardware_threads())
    return Y


def linear_bwd_dgrad_act(dY16, W16, A16, act="none", clip=20.0, nthreads=0) -> np.ndarray:
    """dX = rn16(dY W^T) masked by the derivative of `act` at the layer input A (FP16 [M,K])."""
    _chk(dY16, np.uint16); _chk(W16, np.uint16); _chk(A16, np.uint16)
    M, N = dY16.shape; K, N2 = W16.shape; assert N == N2 and A16.shape == (M, K)
    dX = np.empty((M, K), np.uint16)
    lib().orc_linear_bwd_dgrad_act(_ptr(dY16), N, _ptr(W16), N, _ptr(A16), K, _ptr(dX), K, M, K, N,
                                   ACT[act], clip, nthreads or hardware_threads())
    return dX


def bias_grad(dY16) -> np.ndarray:
    """db[n] = rn16(sum_m dY[m,n]), FP32 running sum."""
    _chk(dY16, np.uint16)
    M, N = dY16.shape
    db = np.empty(N, np.uint16)
    lib().orc_bias_grad(_ptr(dY16), N, _ptr(db), M, N)
    return db


def lstm_cell_fwd(G16, c_prev16):
    """(c_new, h) of an LSTM cell from the FP16 gate pre-activations [M,4H] (order i,f,g,o)."""
    _chk(G16, np.uint16); _chk(c_prev16, np.uint16)
    M, H4 = G16.shape; H = H4 // 4; assert c_prev16.shape == (M, H)
    c = np.empty((M, H), np.uint16); h = np.empty((M, H), np.uint16)
    lib().orc_lstm_cell_fwd(_ptr(G16), H4, _ptr(c_prev16), _ptr(c), _ptr(h), M, H)
    return c, h


def lstm_cell_bwd(G16, c_prev16, c_new16, dh16, dc_in16=None):
    """(dG [M,4H], dc_prev [M,H]) from the stored gates and states."""
    for a in (G16, c_prev16, c_new16, dh16):
        _chk(a, np.uint16)
    M, H4 = G16.shape; H = H4 // 4
    dG = np.empty((M, H4), np.uint16); dcp = np.empty((M, H), np.uint16)
    lib().orc_lstm_cell_bwd(_ptr(G16), H4, _ptr(c_prev16), _ptr(c_new16), _ptr(dh16),
                            _ptr(dc_in16) if dc_in16 is not None else None, _ptr(dG), H4, _ptr(dcp), M, H)
    return dG, dcp


_OPS = {"fwd": 0, "dgrad": 1, "wgrad": 2}


def _dims(op, A, B):
    if op == "fwd":
        (M, K), (_, N) = A.shape, B.shape
    elif op == "dgrad":
        (M, N), (K, _) = A.shape, B.shape
    else:
        (M, K), (_, N) = A.shape, B.shape
    return M, K, N


def linear_sampled(op: str, A16, B16, rows, cols):
    """Selected outputs of one of the three products.

    Returns (fp16 bits, the sum carried in double, sum of |a||b|)."""
    _chk(A16, np.uint16); _chk(B16, np.uint16)
    M, K, N = _dims(op, A16, B16)
    rows = np.ascontiguousarray(rows, np.int64); cols = np.ascontiguousarray(cols, np.int64)
    n = rows.size
    o16 = np.empty(n, np.uint16); ex = np.empty(n, np.float64); ab = np.empty(n, np.float64)
    lib().orc_linear_sampled(_OPS[op], _ptr(A16), A16.shape[1], _ptr(B16), B16.shape[1],
                             M, K, N, _ptr(rows), _ptr(cols), n, _ptr(o16), _ptr(ex), _ptr(ab))
    return o16, ex, ab


def linear_exact(op: str, A16, B16, nthreads=0):
    """Every output of one product with the sum carried in double; also sum |a||b|."""
    _chk(A16, np.uint16); _chk(B16, np.uint16)
    M, K, N = _dims(op, A16, B16)
    R, Cc = (K if op == "wgrad" else M), (K if op == "dgrad" else N)
    ex = np.empty((R, Cc), np.float64); ab = np.empty((R, Cc), np.float64)
    lib().orc_linear_exact(_OPS[op], _ptr(A16), A16.shape[1], _ptr(B16), B16.shape[1],
                           M, K, N, _ptr(ex), _ptr(ab), nthreads or hardware_threads())
    return ex, ab


# ------------------------------------------------- scale, flag, optimizers
def scale_upstream(g32, S: float) -> np.ndarray:
    _chk(g32, np.float32)
    out = np.empty(g32.shape, np.uint16)
    lib().orc_scale_upstream(_ptr(g32), S, _ptr(out), g32.size)
    return out


def found_inf(g16) -> int:
    _chk(g16, np.uint16)
    return int(lib().orc_found_inf(_ptr(g16), g16.size))


def adam_update(g16, w32, m, v, w16, S, lr, b1, b2, eps, t, weight_decay=0.0):
    """In place on w32, m, v, w16.  t = applied-step count including this step."""
    for a, d in ((g16, np.uint16), (w32, np.float32), (m, np.float32), (v, np.float32),
                 (w16, np.uint16)):
        _chk(a, d)
    lib().orc_adam_update(_ptr(g16), _ptr(w32), _ptr(m), _ptr(v), _ptr(w16), g16.size,
                          S, lr, b1, b2, eps, weight_decay, t)


def momentum_update(g16, w32, u, w16, S, lr, mu, weight_decay=0.0):
    for a, d in ((g16, np.uint16), (w32, np.float32), (u, np.float32), (w16, np.uint16)):
        _chk(a, d)
    lib().orc_momentum_update(_ptr(g16), _ptr(w32), _ptr(u), _ptr(w16), g16.size,
                              S, lr, mu, weight_decay)


class Scaler:
    """Loss-scale state machine: halve at the `tolerance`-th overflow since S last changed
    (1: at every overflow), double after `interval` clean steps in a row."""

    def __init__(self, init_scale=65536.0, interval=1000, s_min=1.0, s_max=2.0 ** 24,
                 dynamic=True, tolerance=1):
        self.c = _Scaler(init_scale, s_min, s_max, interval, 1 if dynamic else 0, 0, 0, 0, 0,
                         tolerance, 0)

    def update(self, flag: int):
        lib().orc_scaler_update(C.byref(self.c), int(flag))

    S = property(lambda self: float(self.c.S))
    good = property(lambda self: int(self.c.good))
    t = property(lambda self: int(self.c.t))
    step = property(lambda self: int(self.c.step))
    skipped = property(lambda self: int(self.c.skipped))
    strikes = property(lambda self: int(self.c.strikes))


# ------------------------------------------------------------ step driver
@dataclass
class Optim:
    kind: str = "adam"          # "adam" | "momentum"
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    momentum: float = 0.9
    weight_decay: float = 0.0


@dataclass
class Layer:
    w32: np.ndarray             # [K,N] float32 master
    w16: np.ndarray             # [K,N] uint16 working copy
    m: np.ndarray               # Adam first moment, or the momentum buffer
    v: np.ndarray | None        # Adam second moment
    chained: bool = False       # input is the previous layer's output
    act: str = "none"           # activation after this layer's product ("none" for a top layer)
    clip: float = 20.0
    b32: np.ndarray | None = None   # FP32 master bias [N] (None: no bias)
    b16: np.ndarray | None = None
    bm: np.ndarray | None = None
    bv: np.ndarray | None = None
    db: np.ndarray | None = None
    X: np.ndarray | None = None
    Y: np.ndarray | None = None
    dY: np.ndarray | None = None
    dX: np.ndarray | None = None
    dW: np.ndarray | None = None


def make_layer(w32: np.ndarray, kind: str, chained: bool, act: str = "none", clip: float = 20.0,
               b32: np.ndarray | None = None) -> Layer:
    w32 = np.ascontiguousarray(w32, np.float32).copy()
    ly = Layer(w32=w32, w16=f2h(w32), m=np.zeros_like(w32),
               v=np.zeros_like(w32) if kind == "adam" else None, chained=chained, act=act, clip=clip)
    if b32 is not None:
        ly.b32 = np.ascontiguousarray(b32, np.float32).copy()
        ly.b16 = f2h(ly.b32)
        ly.bm = np.zeros_like(ly.b32)
        ly.bv = np.zeros_like(ly.b32) if kind == "adam" else None
    return ly


@dataclass
class StepRecord:
    found_inf: int
    S_before: float
    S_after: float
    good: int
    t: int


def train_step(layers: list[Layer], xs: list, gs: list, scaler: Scaler, opt: Optim,
               nthreads=0) -> StepRecord:
    """One mixed-precision step of the stack.

    xs[l]: FP16 bits [M,K_l] for a layer that is not chained (None otherwise).
    gs[l]: FP32 upstream gradient [M,N_l] for a layer whose output feeds no chained
    layer (None otherwise); it is multiplied by S and rounded to FP16 there.
    A chained layer takes X_l = Y_{l-1} and hands dY_{l-1} = dX_l back.
    """
    L = len(layers)
    S = scaler.S
    for l, ly in enumerate(layers):                       # forward, Section 3.1
        ly.X = layers[l - 1].Y if ly.chained else xs[l]
        if ly.act == "none" and ly.b16 is None:
            ly.Y = linear_fwd(ly.X, ly.w16, nthreads)
        else:
            ly.Y = linear_fwd_act(ly.X, ly.w16, ly.b16, ly.act, ly.clip, nthreads)
    flag = 0
    for l in range(L - 1, -1, -1):                        # backward in FP16
        ly = layers[l]
        feeds_next = l + 1 < L and layers[l + 1].chained
        assert feeds_next or ly.act == "none", "a top layer has no activation"
        # dY is the gradient at this layer's pre-activation: the layer above has already
        # masked it with this layer's activation derivative (taken from this layer's output)
        ly.dY = layers[l + 1].dX if feeds_next else scale_upstream(gs[l], S)
        ly.dW = linear_bwd_wgrad(ly.X, ly.dY, nthreads)
        below = layers[l - 1] if ly.chained else None
        if below is not None and below.act != "none":
            ly.dX = linear_bwd_dgrad_act(ly.dY, ly.w16, ly.X, below.act, below.clip, nthreads)
        else:
            ly.dX = linear_bwd_dgrad(ly.dY, ly.w16, nthreads)
        flag |= found_inf(ly.dW)                          # inspection, Section 3.1 item 1
        if ly.b16 is not None:
            ly.db = bias_grad(ly.dY)
            flag |= found_inf(ly.db)
    if not flag:                                          # Section 3.2
        t = scaler.t + 1
        for ly in layers:
            pairs = [(ly.dW, ly.w32, ly.m, ly.v, ly.w16)]
            if ly.b16 is not None:
                pairs.append((ly.db, ly.b32, ly.bm, ly.bv, ly.b16))
            for g16, w32, m, v, w16 in pairs:
                if opt.kind == "adam":
                    adam_update(g16, w32, m, v, w16, S, opt.lr, opt.beta1, opt.beta2, opt.eps, t,
                                opt.weight_decay)
                else:
                    momentum_update(g16, w32, m, w16, S, opt.lr, opt.momentum, opt.weight_decay)
    scaler.update(flag)                                   # scale for the next iteration
    return StepRecord(flag, S, scaler.S, scaler.good, scaler.t)
