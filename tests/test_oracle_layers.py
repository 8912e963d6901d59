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


# ------------------------------------------------------------------ LSTM cell
def _cell_double(G, c):
    """The cell in double precision, gate order i, f, g, o."""
    H = c.shape[1]
    sg = lambda x: 1.0 / (1.0 + np.exp(-x))
    i, f, g, o = sg(G[:, :H]), sg(G[:, H:2 * H]), np.tanh(G[:, 2 * H:3 * H]), sg(G[:, 3 * H:])
    cn = f * c + i * g
    return cn, o * np.tanh(cn)


def test_lstm_cell_forward_special_cases_and_double_reference(orc):
    M, H = 5, 7
    zeros = np.zeros((M, 4 * H), np.uint16)
    c = _h(np.linspace(-2, 2, M * H).reshape(M, H))
    cn, h = orc.lstm_cell_fwd(zeros, c)                      # all gates 0: i=f=o=1/2, g=0
    assert (cn == _h(0.5 * _f(c))).all()
    assert np.abs(_f(h) - 0.5 * np.tanh(_f(cn))).max() <= 2.0 ** -11
    big = _h(np.full((M, 4 * H), 30.0))                      # saturated: c' = c + 1, h = tanh(c')
    cn, h = orc.lstm_cell_fwd(big, c)
    assert (cn == _h(_f(c) + 1.0)).all()
    rng = np.random.default_rng(7)
    G = _h(rng.standard_normal((M, 4 * H)) * 2)
    cn, h = orc.lstm_cell_fwd(G, c)
    wc, wh = _cell_double(_f(G), _f(c))
    assert np.abs(_f(cn) - wc).max() <= 2.0 ** -10 * np.abs(wc).max() + 1e-6
    assert np.abs(_f(h) - wh).max() <= 2.0 ** -10


def test_lstm_cell_backward_matches_finite_differences(orc):
    """Gradients of L = sum(a*h) + sum(b*c_new) with respect to the gate pre-activations and
    c_prev, by central differences on the double-precision cell."""
    rng = np.random.default_rng(8)
    M, H = 3, 4
    G = rng.standard_normal((M, 4 * H)); c = rng.standard_normal((M, H))
    a = rng.standard_normal((M, H)); b = rng.standard_normal((M, H))
    G16, c16, a16, b16 = _h(G), _h(c), _h(a), _h(b)
    Gq, cq, aq, bq = _f(G16), _f(c16), _f(a16), _f(b16)

    def loss(Gv, cv):
        cn, h = _cell_double(Gv, cv)
        return (aq * h).sum() + (bq * cn).sum()
    eps = 1e-6
    dG_fd = np.zeros_like(Gq); dc_fd = np.zeros_like(cq)
    for idx in np.ndindex(*Gq.shape):
        d = np.zeros_like(Gq); d[idx] = eps
        dG_fd[idx] = (loss(Gq + d, cq) - loss(Gq - d, cq)) / (2 * eps)
    for idx in np.ndindex(*cq.shape):
        d = np.zeros_like(cq); d[idx] = eps
        dc_fd[idx] = (loss(Gq, cq + d) - loss(Gq, cq - d)) / (2 * eps)
    cn16, _ = orc.lstm_cell_fwd(G16, c16)
    dG, dcp = orc.lstm_cell_bwd(G16, c16, cn16, a16, b16)
    # the oracle takes tanh of the FP16-rounded c_new and rounds its outputs to FP16
    assert np.abs(_f(dG) - dG_fd).max() <= 4e-3 and np.abs(_f(dcp) - dc_fd).max() <= 4e-3
    assert np.abs(_f(dG) - dG_fd).mean() <= 5e-4
    # no incoming cell gradient = a zero one
    z = np.zeros((M, H), np.uint16)
    d1, c1 = orc.lstm_cell_bwd(G16, c16, cn16, a16, None)
    d2, c2 = orc.lstm_cell_bwd(G16, c16, cn16, a16, z)
    assert (d1 == d2).all() and (c1 == c2).all()
