"""Pins for the oracle's three FP16-in / FP32-accumulate products (Section 3.1)."""
import numpy as np
import pytest


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _f(h):
    return h.view(np.float16).astype(np.float64)


def _brute(op, A, B):
    """Pure-Python definition in double: one loop nest per operation, indices written out."""
    A, B = _f(A), _f(B)
    if op == "fwd":
        M, K = A.shape; N = B.shape[1]
        out = [[sum(A[m][k] * B[k][n] for k in range(K)) for n in range(N)] for m in range(M)]
    elif op == "dgrad":
        M, N = A.shape; K = B.shape[0]
        out = [[sum(A[m][n] * B[k][n] for n in range(N)) for k in range(K)] for m in range(M)]
    else:
        M, K = A.shape; N = B.shape[1]
        out = [[sum(A[m][k] * B[m][n] for m in range(M)) for n in range(N)] for k in range(K)]
    return np.array(out, np.float64)


def _call(orc, op, A, B):
    return {"fwd": orc.linear_fwd, "dgrad": orc.linear_bwd_dgrad, "wgrad": orc.linear_bwd_wgrad}[op](A, B)


SHAPES = [(1, 1, 1), (2, 3, 5), (5, 8, 3), (8, 8, 8), (7, 1, 4), (3, 6, 2)]


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_brute_force_small(orc, op, M, K, N):
    rng = np.random.default_rng(M * 100 + K * 10 + N)
    A = _h(rng.standard_normal((M, N) if op == "dgrad" else (M, K)))
    B = _h(rng.standard_normal((M, N) if op == "wgrad" else (K, N)))
    want = _brute(op, A, B)
    got = _f(_call(orc, op, A, B))
    assert got.shape == want.shape
    red = {"fwd": K, "dgrad": N, "wgrad": M}[op]
    # one FP16 rounding (2^-11 relative) + FP32 running-sum error
    tol = 2.0 ** -11 * np.abs(want) + red * 2.0 ** -24 * 16.0 + 2.0 ** -25
    assert (np.abs(got - want) <= tol).all()
    ex, ab = orc.linear_exact(op, A, B)
    assert np.allclose(ex, want, rtol=1e-14, atol=1e-14)
    assert (ab >= np.abs(ex) - 1e-12).all()


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
def test_integer_exact_family(orc, op):
    """Entries in {-2..2}, reduction <= 64: every partial sum is an integer below 2^24 and
    the result is below 2048, so it is exact in FP16 whatever the summation order."""
    rng = np.random.default_rng(11)
    M, K, N = 37, 64, 29
    if op == "dgrad":
        K, N = 29, 64
    elif op == "wgrad":
        M, K = 64, 37
    Ai = rng.integers(-2, 3, (M, N) if op == "dgrad" else (M, K))
    Bi = rng.integers(-2, 3, (M, N) if op == "wgrad" else (K, N))
    want = {"fwd": lambda: Ai @ Bi, "dgrad": lambda: Ai @ Bi.T, "wgrad": lambda: Ai.T @ Bi}[op]()
    got = _call(orc, op, _h(Ai), _h(Bi))
    assert np.abs(want).max() < 2048
    assert (got == _h(want)).all()


def test_permutation_and_identity_reproduce_bits(orc):
    rng = np.random.default_rng(3)
    X = _h(rng.standard_normal((9, 16)) * 50)
    perm = rng.permutation(16)
    P = np.zeros((16, 16)); P[np.arange(16), perm] = 1.0        # Y[:, perm[k]] = X[:, k]
    Y = orc.linear_fwd(X, _h(P))
    assert (Y[:, perm] == X).all()
    # dgrad with the same W undoes the permutation: dX[m,k] = dY[m, perm[k]]
    dX = orc.linear_bwd_dgrad(Y, _h(P))
    assert (dX == X).all()
    # wgrad with X = identity rows returns dY
    I = _h(np.eye(9))
    dY = _h(rng.standard_normal((9, 5)))
    assert (orc.linear_bwd_wgrad(I, dY) == dY).all()


def test_dgrad_wgrad_are_fwd_on_transposed_copies(orc):
    rng = np.random.default_rng(5)
    M, K, N = 13, 24, 17
    X = _h(rng.standard_normal((M, K))); W = _h(rng.standard_normal((K, N)) / 5)
    dY = _h(rng.standard_normal((M, N)))
    dX = orc.linear_bwd_dgrad(dY, W)
    assert (dX == orc.linear_fwd(dY, np.ascontiguousarray(W.T))).all()
    dW = orc.linear_bwd_wgrad(X, dY)
    assert (dW == orc.linear_fwd(np.ascontiguousarray(X.T), dY)).all()


def test_accumulation_is_fp32_and_ascending(orc):
    """Sums whose value shows that the running sum is FP32 and taken in ascending order."""
    K = 8192 + 1
    a = np.ones((1, K), np.float32); b = np.full((K, 1), 2.0 ** -13, np.float32)
    a[0, 0] = 1.0; b[0, 0] = 1024.0
    # ascending FP32: 1024 then 8192 additions of 2^-13 (ulp of 1024 in FP32 is 2^-13) -> exact
    got = _f(orc.linear_fwd(_h(a), _h(b)))[0, 0]
    assert got == 1025.0                         # an FP16 running sum would stay at 1024
    # order matters: the same data reversed accumulates exactly as well, but a huge value
    # added first in FP32 absorbs smaller ones below half an ulp
    a2 = np.ones((1, 3), np.float32); b2 = np.array([[2.0 ** 15], [2.0 ** -10], [-2.0 ** 15]], np.float32)
    assert _f(orc.linear_fwd(_h(a2), _h(b2)))[0, 0] == 0.0     # 2^15 + 2^-10 rounds to 2^15 in FP32
    b3 = np.array([[2.0 ** 15], [-2.0 ** 15], [2.0 ** -10]], np.float32)
    assert _f(orc.linear_fwd(_h(a2), _h(b3)))[0, 0] == 2.0 ** -10


def test_overflow_rounds_to_inf_and_nan_propagates(orc):
    X = _h(np.full((1, 4), 200.0)); W = _h(np.full((4, 1), 200.0))
    assert orc.linear_fwd(X, W)[0, 0] == 0x7C00               # 160000 > 65520
    X2 = X.copy(); X2[0, 1] = 0x7C00; W2 = W.copy(); W2[2, 0] = 0xFC00
    out = orc.linear_fwd(X2, W2)[0, 0]
    assert (out & 0x7C00) == 0x7C00 and (out & 0x3FF) != 0    # inf - inf = NaN


def test_sampled_matches_full(orc):
    rng = np.random.default_rng(9)
    M, K, N = 20, 33, 12
    X = _h(rng.standard_normal((M, K))); W = _h(rng.standard_normal((K, N))); dY = _h(rng.standard_normal((M, N)))
    for op, A, B, R, Cn in (("fwd", X, W, M, N), ("dgrad", dY, W, M, K), ("wgrad", X, dY, K, N)):
        full = _call(orc, op, A, B)
        r = rng.integers(0, R, 50); c = rng.integers(0, Cn, 50)
        s16, ex, ab = orc.linear_sampled(op, A, B, r, c)
        assert (s16 == full[r, c]).all()
        assert np.allclose(ex, _brute(op, A, B)[r, c], rtol=1e-13, atol=1e-13)
