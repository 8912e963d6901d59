"""Pins for the oracle's bias / activation / bias-gradient pieces."""
import numpy as np
import pytest


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _f(h):
    return h.view(np.float16).astype(np.float64)


@pytest.mark.parametrize("act", ["none", "relu", "clipped_relu"])
def test_fwd_act_brute_force(orc, act):
    rng = np.random.default_rng(3)
    M, K, N = 6, 9, 5
    X = _h(rng.standard_normal((M, K)) * 3); W = _h(rng.standard_normal((K, N)) * 3)
    b = _h(rng.standard_normal(N) * 4)
    got = _f(orc.linear_fwd_act(X, W, b, act, clip=6.0))
    z = np.array([[sum(_f(X)[m][k] * _f(W)[k][n] for k in range(K)) + _f(b)[n] for n in range(N)]
                  for m in range(M)])
    want = {"none": z, "relu": np.maximum(z, 0), "clipped_relu": np.minimum(np.maximum(z, 0), 6.0)}[act]
    assert (np.abs(got - want) <= 2.0 ** -11 * np.abs(want) + 1e-5).all()
    if act != "none":
        assert (got >= 0).all() and (got[z < -1e-3] == 0).all()
    if act == "clipped_relu":
        assert got.max() == 6.0 and (got[z > 6.01] == 6.0).all()


def test_fwd_act_reduces_to_plain_product_and_to_bias(orc):
    rng = np.random.default_rng(4)
    X = _h(rng.standard_normal((7, 12))); W = _h(rng.standard_normal((12, 10)))
    assert (orc.linear_fwd_act(X, W, None, "none") == orc.linear_fwd(X, W)).all()
    zero_b = np.zeros(10, np.uint16)
    assert (orc.linear_fwd_act(X, W, zero_b, "none") == orc.linear_fwd(X, W)).all()
    b = _h(rng.standard_normal(10))
    Y = orc.linear_fwd_act(np.zeros((7, 12), np.uint16), W, b, "relu")
    assert (Y == _h(np.maximum(_f(b), 0))[None, :]).all()          # X = 0: the activated bias, exactly
    # the bias joins the FP32 sum before the single rounding: 2048 + 1 is not an FP16 number,
    # 2048 + 1 + 1 (= 2050) is
    X1 = _h(np.array([[2048.0, 1.0]])); W1 = _h(np.array([[1.0], [1.0]]))
    assert _f(orc.linear_fwd_act(X1, W1, _h(np.array([1.0])), "none"))[0, 0] == 2050.0


def test_dgrad_act_masks_by_the_stored_output(orc):
    rng = np.random.default_rng(5)
    M, K, N = 8, 11, 6
    dY = _h(rng.standard_normal((M, N))); W = _h(rng.standard_normal((K, N)))
    A = _h(np.maximum(rng.standard_normal((M, K)) * 10, 0))        # an activated layer output
    A[0, 0] = _h(np.array([20.0]))[0]; A[0, 1] = _h(np.array([25.0]))[0]; A[0, 2] = 0x8000   # -0
    plain = orc.linear_bwd_dgrad(dY, W)
    assert (orc.linear_bwd_dgrad_act(dY, W, A, "none") == plain).all()
    relu = orc.linear_bwd_dgrad_act(dY, W, A, "relu")
    pos = _f(A) > 0
    assert (relu[pos] == plain[pos]).all() and (relu[~pos] == 0).all()
    clip = orc.linear_bwd_dgrad_act(dY, W, A, "clipped_relu", clip=20.0)
    inside = (_f(A) > 0) & (_f(A) < 20.0)
    assert (clip[inside] == plain[inside]).all() and (clip[~inside] == 0).all()
    assert clip[0, 0] == 0 and clip[0, 1] == 0 and relu[0, 0] == plain[0, 0]


def test_bias_grad_is_the_weight_gradient_of_a_column_of_ones(orc):
    rng = np.random.default_rng(6)
    M, N = 257, 13
    dY = _h(rng.standard_normal((M, N)) * 3)
    ones = _h(np.ones((M, 1)))
    assert (orc.bias_grad(dY) == orc.linear_bwd_wgrad(ones, dY)[0]).all()
    want = _f(dY).sum(axis=0)
    assert (np.abs(_f(orc.bias_grad(dY)) - want) <= 2.0 ** -10 * np.abs(want) + 1e-3).all()
    dY[5, 2] = 0x7C00
    assert orc.bias_grad(dY)[2] == 0x7C00
