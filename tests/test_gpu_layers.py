"""Parity of the bias / activation epilogues and of the bias gradient against the oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ACTS = {"none": 0, "relu": 1, "clipped_relu": 2}


def _pad8(n):
    return (n + 7) // 8 * 8


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _dev(bits):
    if bits.ndim == 1:
        return torch.from_numpy(bits.view(np.float16).copy()).cuda()
    r, c = bits.shape
    buf = torch.zeros(r, _pad8(c), dtype=torch.float16, device="cuda")
    buf[:, :c] = torch.from_numpy(bits.view(np.float16)).cuda()
    return buf[:, :c]


def _out(r, c):
    return torch.full((r, _pad8(c)), 7.0, dtype=torch.float16, device="cuda")[:, :c]


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


SHAPES = [(37, 64, 29), (300, 200, 520), (128, 72, 257), (129, 328, 264), (1, 8, 8)]


@pytest.mark.parametrize("act", ["none", "relu", "clipped_relu"])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_fwd_bias_activation_integer_exact(orc, mp, act, M, K, N):
    """Small-integer operands and bias: the FP32 value before the activation is exact, so the
    GPU must match the oracle bit for bit."""
    rng = np.random.default_rng(M + K + N)
    X, W = _h(rng.integers(-2, 3, (M, K))), _h(rng.integers(-2, 3, (K, N)))
    b = _h(rng.integers(-30, 31, N))
    Y = _out(M, N)
    ws = torch.empty(max(mp.mp_gemm_workspace_bytes(M, K, N, 0), 16), dtype=torch.uint8, device="cuda")
    mp.mp_linear_fwd_act(_dev(X), _dev(W), _dev(b), Y, ACTS[act], 20.0, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    want = orc.linear_fwd_act(X, W, b, act, clip=20.0)
    assert (_bits(Y) == want).all()
    if act == "clipped_relu" and M * N > 1000:
        f = want.view(np.float16).astype(np.float32)
        assert f.max() <= 20.0 and (f == 20.0).any() and (f == 0).any()
    # no bias: same call with NULL
    mp.mp_linear_fwd_act(_dev(X), _dev(W), None, Y, ACTS[act], 20.0, ws)
    assert (_bits(Y) == orc.linear_fwd_act(X, W, None, act, clip=20.0)).all()


@pytest.mark.parametrize("act", ["none", "relu", "clipped_relu"])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_dgrad_activation_mask_integer_exact(orc, mp, act, M, K, N):
    rng = np.random.default_rng(M * 3 + K + N)
    dY, W = _h(rng.integers(-2, 3, (M, N))), _h(rng.integers(-2, 3, (K, N)))
    A = _h(np.clip(rng.integers(-15, 30, (M, K)), 0, 20))           # an activated output: 0 .. 20
    A[0, 0] = 0x8000                                                # -0 does not pass
    dX = _out(M, K)
    ws = torch.empty(max(mp.mp_gemm_workspace_bytes(M, K, N, 1), 16), dtype=torch.uint8, device="cuda")
    mp.mp_linear_bwd_dgrad_act(_dev(dY), _dev(W), _dev(A), dX, ACTS[act], 20.0, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    want = orc.linear_bwd_dgrad_act(dY, W, A, act, clip=20.0)
    assert (_bits(dX) == want).all()
    if act != "none":
        assert (want == 0).mean() > 0.3


@pytest.mark.parametrize("act", ["none", "relu"])
def test_grouped_fwd_bias_activation_integer_exact(orc, mp, act):
    """Three problems with their own biases in one launch: integer operands, bit-exact against the
    oracle's forward product with bias and activation."""
    M, K, N = 300, 72, 264
    rng = np.random.default_rng(31)
    Xs = [_h(rng.integers(-2, 3, (M, K))) for _ in range(3)]
    Ws = [_h(rng.integers(-2, 3, (K, N))) for _ in range(3)]
    bs = [_h(rng.integers(-3, 4, (N,))) for _ in range(3)]
    Ys = [_out(M, N) for _ in range(3)]
    bd = [torch.from_numpy(b.view(np.float16).copy()).cuda() for b in bs]
    mp.mp_linear_fwd_act_grouped([_dev(x) for x in Xs], [_dev(w) for w in Ws], bd, Ys,
                                 {"none": mp.MP_ACT_NONE, "relu": mp.MP_ACT_RELU}[act], 20.0)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    for i in range(3):
        assert (_bits(Ys[i]) == orc.linear_fwd_act(Xs[i], Ws[i], bs[i], act)).all(), i


def test_fwd_act_random_values_within_tolerance(orc, mp):
    rng = np.random.default_rng(1)
    M, K, N = 384, 520, 264
    X, W = _h(rng.standard_normal((M, K))), _h(rng.standard_normal((K, N)) / 8)
    b = _h(rng.standard_normal(N))
    Y = _out(M, N)
    ws = torch.empty(max(mp.mp_gemm_workspace_bytes(M, K, N, 0), 16), dtype=torch.uint8, device="cuda")
    mp.mp_linear_fwd_act(_dev(X), _dev(W), _dev(b), Y, ACTS["relu"], 20.0, ws)
    got = _bits(Y).view(np.float16).astype(np.float64)
    ex, ab = orc.linear_exact("fwd", X, W)
    z = ex + b.view(np.float16).astype(np.float64)[None, :]
    want = np.maximum(z, 0)
    tol = 2.0 ** -10 * np.abs(z) + K * 2.0 ** -24 * (ab + 4.0) + 2.0 ** -24
    assert (np.abs(got - want) <= tol).all()
    assert (_bits(Y) == orc.linear_fwd_act(X, W, b, "relu")).mean() > 0.98


@pytest.mark.parametrize("M,N", [(1, 8), (257, 13), (5000, 1000), (8192, 4096), (25600, 29)])
def test_bias_grad(orc, mp, M, N):
    rng = np.random.default_rng(M + N)
    dYi = rng.integers(-3, 4, (M, N))
    dY = _h(dYi)
    db = torch.zeros(_pad8(N), dtype=torch.float16, device="cuda")
    ws = torch.empty(max(mp.mp_bias_grad_workspace_bytes(M, N), 16), dtype=torch.uint8, device="cuda")
    st = mp.State()
    mp.mp_bias_grad(_dev(dY), db[:N], st, ws)
    got = _bits(db)
    assert (got[:N] == _h(dYi.sum(axis=0))).all() and (got[N:] == 0).all()   # integer sums: bit exact
    if M * N <= 5_000_000:
        assert (got[:N] == orc.bias_grad(dY)).all()
    assert st.read().found_inf == 0
    # random values: FP32 sums in another order, one FP16 rounding
    if M * N <= 5_000_000:
        dYr = _h(rng.standard_normal((M, N)) * 4)
        mp.mp_bias_grad(_dev(dYr), db[:N], st, ws)
        g = _bits(db)[:N].view(np.float16).astype(np.float64)
        f = dYr.view(np.float16).astype(np.float64)
        want, ab = f.sum(axis=0), np.abs(f).sum(axis=0)
        assert (np.abs(g - want) <= 2.0 ** -10 * np.abs(want) + M * 2.0 ** -24 * ab + 2.0 ** -24).all()
        assert (_bits(db)[:N] == orc.bias_grad(dYr)).mean() > 0.97
    # an inf in the column sum raises the flag
    dY2 = dY.copy(); dY2[M - 1, N - 1] = 0x7C00
    mp.mp_bias_grad(_dev(dY2), db[:N], st, ws)
    assert _bits(db)[N - 1] == 0x7C00 and st.read().found_inf == 1
    st.close()


def test_bias_grad_grouped_equals_single_calls(orc, mp):
    """Four gradients of one shape in one pair of launches: every result is the single call's,
    bit for bit, and the oracle's on integer values; a non-finite sum in one of them raises the flag."""
    M, N = 777, 520
    rng = np.random.default_rng(9)
    dYs = [_h(rng.standard_normal((M, N)) * 3) for _ in range(3)] + [_h(rng.integers(-3, 4, (M, N)))]
    devs = [_dev(d) for d in dYs]
    single = [torch.zeros(N, dtype=torch.float16, device="cuda") for _ in dYs]
    grouped = [torch.full((N,), 7.0, dtype=torch.float16, device="cuda") for _ in dYs]
    ws = torch.empty(4 * mp.mp_bias_grad_workspace_bytes(M, N), dtype=torch.uint8, device="cuda")
    st = mp.State()
    for d, o in zip(devs, single):
        mp.mp_bias_grad(d, o, st, ws)
    mp.mp_bias_grad_grouped(devs, grouped, st, ws)
    for a, b in zip(single, grouped):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert (_bits(grouped[3]) == orc.bias_grad(dYs[3])).all()
    assert st.read().found_inf == 0
    dYs[1][5, 17] = 0x7C00
    mp.mp_bias_grad_grouped([_dev(d) for d in dYs], grouped, st, ws)
    assert _bits(grouped[1])[17] == 0x7C00 and st.read().found_inf == 1
    assert torch.equal(grouped[0].view(torch.int16), single[0].view(torch.int16))
    with pytest.raises(mp.MpError):
        mp.mp_bias_grad_grouped(devs, grouped, st, ws[:16])
    st.close()


# ------------------------------------------------------------------ LSTM cell
@pytest.mark.parametrize("M,H", [(1, 8), (37, 64), (640, 1024)])
def test_lstm_cell_forward_and_backward(orc, mp, M, H):
    """Elementwise cell kernels against the oracle: both evaluate sigma and tanh in FP32 from the
    same FP16 inputs, with different exp/tanh routines, so results agree to one FP16 unit in
    the last place and nearly all outputs are identical bits."""
    rng = np.random.default_rng(M + H)
    G = _h(rng.standard_normal((M, 4 * H)) * 2.5)
    c = _h(rng.standard_normal((M, H)))
    Gd = _dev(G)
    cd = torch.from_numpy(c.view(np.float16).copy()).cuda()
    cn = torch.empty(M, H, dtype=torch.float16, device="cuda"); h = torch.empty_like(cn)
    mp.mp_lstm_cell_fwd(Gd, cd, cn, h)
    wc, wh = orc.lstm_cell_fwd(G, c)

    def close(got_bits, want_bits, frac=0.995, scale=None, extra=None):
        g = got_bits.view(np.float16).astype(np.float64); w = want_bits.view(np.float16).astype(np.float64)
        fin = np.isfinite(w)
        assert (np.isfinite(g) == fin).all()
        tol = 2.0 ** -10 * np.abs(w) + 2.0 ** -24                                 # one FP16 ulp
        if scale is not None:
            # factors like 1 - sigma(x) cancel: an FP32 ulp of sigma is an absolute, not a
            # relative, error of the factor, so allow 1e-5 of the incoming gradient's size
            tol = tol + 1e-5 * np.tile(scale, (1, w.shape[1] // scale.shape[1]))
        if extra is not None:
            tol = tol + extra
        assert (np.abs(g - w)[fin] <= tol[fin]).all()
        # share of identical bits; on a handful of outputs one differing rounding must not decide
        assert (got_bits == want_bits).mean() >= frac - 2.0 / got_bits.size
    # c = f c_prev + i g can cancel: the two sides' sigma and tanh differ by a few FP32 units in
    # the last place (different exponential and division routines), an absolute error of up to
    # 4e-6 (|c_prev| + 1) in c and, through tanh' <= 1, in h
    slack = 4e-6 * (np.abs(c.view(np.float16).astype(np.float64)) + 1.0)
    close(_bits(cn), wc, extra=slack); close(_bits(h), wh, extra=slack)
    # backward, fed with the oracle's stored c_new so that both sides see identical inputs
    dh = _h(rng.standard_normal((M, H)) * 64); dci = _h(rng.standard_normal((M, H)) * 64)
    dG = _out(M, 4 * H); dcp = torch.empty(M, H, dtype=torch.float16, device="cuda")
    t16 = lambda b: torch.from_numpy(b.view(np.float16).copy()).cuda()
    for dc_bits in (dci, None):
        mp.mp_lstm_cell_bwd(Gd, cd, t16(wc), t16(dh), None if dc_bits is None else t16(dc_bits), dG, dcp)
        wG, wcp = orc.lstm_cell_bwd(G, c, wc, dh, dc_bits)
        sc = np.abs(dh.view(np.float16).astype(np.float64)) + \
            (0 if dc_bits is None else np.abs(dc_bits.view(np.float16).astype(np.float64)))
        close(_bits(dG), wG, 0.98, sc); close(_bits(dcp), wcp, 0.98, sc)
    # saturated gates and an overflowing gradient behave like the oracle's (inf stays inf)
    Gs = _h(np.full((M, 4 * H), 30.0)); dh2 = dh.copy(); dh2[0, 0] = 0x7C00
    mp.mp_lstm_cell_bwd(_dev(Gs), cd, t16(wc), t16(dh2), None, dG, dcp)
    wG, wcp = orc.lstm_cell_bwd(Gs, c, wc, dh2, None)
    assert ((_bits(dG) & 0x7C00) == 0x7C00).sum() == ((wG & 0x7C00) == 0x7C00).sum()
