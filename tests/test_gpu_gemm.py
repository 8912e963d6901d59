"""Parity of the tcgen05 GEMMs (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _pad8(n):
    return (n + 7) // 8 * 8


def _to_dev(bits: np.ndarray):
    """uint16 bit patterns [R,C] -> CUDA FP16 view [R,C] inside a buffer whose row pitch is a
    multiple of 8 elements (the library's alignment rule).  The padding columns hold NaN: an
    operand element read from beyond the view would poison the result."""
    r, c = bits.shape
    buf = torch.full((r, _pad8(c)), float("nan"), dtype=torch.float16, device="cuda")
    buf[:, :c] = torch.from_numpy(bits.view(np.float16)).cuda()
    return buf[:, :c]


GUARD_ROWS = 3


def _out(r, c, fill=0x5A5A):
    """Output view [r, c] inside a pattern-filled buffer with padding columns and guard rows
    before and after: whatever the kernel writes outside the view shows up."""
    buf = torch.full((r + 2 * GUARD_ROWS, _pad8(c) + 8), 0, dtype=torch.int16, device="cuda")
    buf.fill_(fill if fill < 0x8000 else fill - 0x10000)
    return buf.view(torch.float16)[GUARD_ROWS:GUARD_ROWS + r, :c], buf


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _run(mp, op, A, B, state=None):
    ws_bytes = 0
    if op == "fwd":
        (M, K), N = A.shape, B.shape[1]
        out, raw = _out(M, N)
    elif op == "dgrad":
        (M, N), K = A.shape, B.shape[0]
        out, raw = _out(M, K)
    else:
        (M, K), N = A.shape, B.shape[1]
        out, raw = _out(K, N)
    ws_bytes = mp.mp_gemm_workspace_bytes(M, K, N, {"fwd": 0, "dgrad": 1, "wgrad": 2}[op])
    ws = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device="cuda")
    dA, dB = _to_dev(A), _to_dev(B)
    if op == "fwd":
        mp.mp_linear_fwd(dA, dB, out, ws)
    elif op == "dgrad":
        mp.mp_linear_bwd_dgrad(dA, dB, out, ws)
    else:
        mp.mp_linear_bwd_wgrad(dA, dB, out, state, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    # padding columns and guard rows of the output buffer must be untouched
    assert bool((raw[:, out.shape[1]:] == 0x5A5A).all())
    assert bool((raw[:GUARD_ROWS] == 0x5A5A).all()) and bool((raw[-GUARD_ROWS:] == 0x5A5A).all())
    return _bits(out), ws_bytes


def _shapes_for(op, M, K, N):
    """operand shapes (A, B) of each op for the layer (M rows, K in, N out)"""
    return {"fwd": ((M, K), (K, N)), "dgrad": ((M, N), (K, N)), "wgrad": ((M, K), (M, N))}[op]


def _oracle(orc, op, A, B):
    return {"fwd": orc.linear_fwd, "dgrad": orc.linear_bwd_dgrad, "wgrad": orc.linear_bwd_wgrad}[op](A, B)


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


INT_CASES = [
    (128, 64, 256),     # exactly one tile, one k-block
    (128, 256, 256),    # one tile, the ring wraps once
    (1, 8, 8),          # smallest legal sizes
    (37, 64, 29),       # ragged everywhere, narrow output (the 1600->29 layer's shape class)
    (300, 200, 520),    # several tiles in both directions, ragged tails
    (260, 1000, 130),   # long reduction, many ring wraps
    (129, 72, 257),     # one past a tile edge
    (8, 20000, 8),      # very long reduction on a sliver of output (split paths, 313 k-blocks)
    (5000, 8, 8),       # many row tiles, one partial k-block
    (16, 8, 3000),      # many column tiles
]


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
@pytest.mark.parametrize("M,K,N", INT_CASES)
def test_integer_exact_bitwise(orc, mp, op, M, K, N):
    """Small-integer entries: every partial sum is an exact FP32 integer whatever the order,
    so the result must equal the oracle bit for bit."""
    rng = np.random.default_rng(M * 7 + K * 3 + N)
    sa, sb = _shapes_for(op, M, K, N)
    A, B = _h(rng.integers(-2, 3, sa)), _h(rng.integers(-2, 3, sb))
    got, _ = _run(mp, op, A, B)
    want = _oracle(orc, op, A, B)
    assert got.shape == want.shape
    bad = np.argwhere(got != want)
    assert bad.size == 0, (bad[:5], got[tuple(bad[0])], want[tuple(bad[0])])


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
@pytest.mark.parametrize("width", [8, 40, 72, 96, 136, 168, 200, 232, 256 + 24, 256 + 104])
def test_every_width_of_the_last_column_tile(orc, mp, op, width):
    """The last column tile is multiplied only as wide as it is (rounded up to 32 columns):
    every such width, for each operand layout, on the CTA-pair kernel (more than 128 output
    rows) and on the one-CTA kernel."""
    rng = np.random.default_rng(width)
    for rows in (300, 70):
        M, K, N = {"fwd": (rows, 136, width), "dgrad": (rows, width, 136), "wgrad": (136, rows, width)}[op]
        sa, sb = _shapes_for(op, M, K, N)
        A, B = _h(rng.integers(-2, 3, sa)), _h(rng.integers(-2, 3, sb))
        got, _ = _run(mp, op, A, B)
        want = _oracle(orc, op, A, B)
        assert got.shape == want.shape and (got == want).all(), (op, rows, width)


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
@pytest.mark.parametrize("M,K,N,count", [(300, 200, 264, 3), (70, 136, 40, 4), (4096, 128, 256, 2),
                                         (1024, 512, 512, 4), (520, 72, 29, 2)])
def test_grouped_call_equals_single_calls(orc, mp, op, M, K, N, count):
    """Several independent products of one shape in one launch: with integer operands (sums exact
    in any order, so a different reduction split cannot show) every problem's output is bit for
    bit the oracle's and the single call's; nothing is written outside any output."""
    rng = np.random.default_rng(M + K + N + count)
    sa, sb = _shapes_for(op, M, K, N)
    As = [_h(rng.integers(-2, 3, sa)) for _ in range(count)]
    Bs = [_h(rng.integers(-2, 3, sb)) for _ in range(count)]
    oshape = {"fwd": (M, N), "dgrad": (M, K), "wgrad": (K, N)}[op]
    outs = [_out(*oshape) for _ in range(count)]
    opi = {"fwd": 0, "dgrad": 1, "wgrad": 2}[op]
    ws = torch.empty(max(mp.mp_gemm_workspace_bytes_grouped(count, M, K, N, opi), 16), dtype=torch.uint8, device="cuda")
    ws.fill_(0x7F)                                      # stale scratch must not matter
    dA, dB = [_to_dev(a) for a in As], [_to_dev(b) for b in Bs]
    st = mp.State()
    if op == "fwd":
        mp.mp_linear_fwd_grouped(dA, dB, [o for o, _ in outs], ws)
    elif op == "dgrad":
        mp.mp_linear_bwd_dgrad_grouped(dA, dB, [o for o, _ in outs], ws)
    else:
        mp.mp_linear_bwd_wgrad_grouped(dA, dB, [o for o, _ in outs], st, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0 and st.read().found_inf == 0
    for i in range(count):
        out, raw = outs[i]
        assert bool((raw[:, out.shape[1]:] == 0x5A5A).all())
        assert bool((raw[:GUARD_ROWS] == 0x5A5A).all()) and bool((raw[-GUARD_ROWS:] == 0x5A5A).all())
        want = _oracle(orc, op, As[i], Bs[i])
        assert (_bits(out) == want).all(), (op, i)
        single, _ = _run(mp, op, As[i], Bs[i])
        assert (single == want).all()
    st.close()


@pytest.mark.parametrize("M,K,N,count", [(520, 200, 264, 3), (2048, 512, 1024, 4)])
def test_grouped_call_is_bitwise_the_single_call_on_random_values(mp, M, K, N, count):
    """A tile is accumulated in the same order whether its problem is launched alone or in a
    group, so with random operands the grouped outputs equal the single calls' bit for bit
    wherever both split the reduction the same way (always for these forward and data-gradient
    products; for the weight gradient when the scratch sizes say the split counts agree)."""
    g = torch.Generator(device="cuda"); g.manual_seed(M + count)
    X = [torch.randn(M, K, generator=g, device="cuda").half() for _ in range(count)]
    W = [(torch.randn(K, N, generator=g, device="cuda") / 16).half() for _ in range(count)]
    dY = [(torch.randn(M, N, generator=g, device="cuda") * 4).half() for _ in range(count)]
    z = lambda r, c: [torch.zeros(r, c, dtype=torch.float16, device="cuda") for _ in range(count)]
    need = max(max(mp.mp_gemm_workspace_bytes_grouped(count, M, K, N, op), mp.mp_gemm_workspace_bytes(M, K, N, op))
               for op in range(3))
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    Yg, dXg, dWg, Ys, dXs, dWs = z(M, N), z(M, K), z(K, N), z(M, N), z(M, K), z(K, N)
    mp.mp_linear_fwd_grouped(X, W, Yg, ws)
    mp.mp_linear_bwd_dgrad_grouped(dY, W, dXg, ws)
    mp.mp_linear_bwd_wgrad_grouped(X, dY, dWg, None, ws)
    for i in range(count):
        mp.mp_linear_fwd(X[i], W[i], Ys[i], ws)
        mp.mp_linear_bwd_dgrad(dY[i], W[i], dXs[i], ws)
        mp.mp_linear_bwd_wgrad(X[i], dY[i], dWs[i], None, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    same_split = {op: mp.mp_gemm_workspace_bytes_grouped(count, M, K, N, op) == count * mp.mp_gemm_workspace_bytes(M, K, N, op)
                  for op in range(3)}
    for i in range(count):
        if same_split[0]:
            assert torch.equal(Yg[i].view(torch.int16), Ys[i].view(torch.int16))
        if same_split[1]:
            assert torch.equal(dXg[i].view(torch.int16), dXs[i].view(torch.int16))
        if same_split[2]:
            assert torch.equal(dWg[i].view(torch.int16), dWs[i].view(torch.int16))
        else:   # another fixed order of FP32 partial sums: equal to within an FP16 rounding
            a, b = dWg[i].float(), dWs[i].float()
            assert (a - b).abs().max() <= 2.0 ** -9 * b.abs().max()
    assert same_split[0] and same_split[1]


def test_grouped_call_rejects_bad_counts(mp):
    a = torch.zeros(16, 16, dtype=torch.float16, device="cuda")
    n = mp.mp_max_group()
    assert n >= 2 and mp.mp_gemm_workspace_bytes_grouped(n + 1, 64, 64, 64, mp.MP_OP_FWD) == 0
    with pytest.raises(mp.MpError) as e:
        mp.mp_linear_fwd_grouped([a] * (n + 1), [a] * (n + 1), [a.clone() for _ in range(n + 1)])
    assert e.value.code == mp.MP_ERR_INVALID_ARG


@pytest.mark.parametrize("op,M,K,N", [("wgrad", 4096, 128, 256), ("wgrad", 3000, 200, 300),
                                      ("fwd", 2048, 2048, 512), ("dgrad", 1500, 640, 2048)])
def test_integer_exact_large_and_split(orc, mp, op, M, K, N):
    """Sizes that take the split-reduction path (few tiles, long reduction) and multi-wave
    persistent scheduling; expected values from an integer matrix product."""
    rng = np.random.default_rng(5)
    sa, sb = _shapes_for(op, M, K, N)
    Ai, Bi = rng.integers(-2, 3, sa), rng.integers(-2, 3, sb)
    got, ws_bytes = _run(mp, op, _h(Ai), _h(Bi))
    exact = {"fwd": lambda: Ai @ Bi, "dgrad": lambda: Ai @ Bi.T, "wgrad": lambda: Ai.T @ Bi}[op]()
    assert np.abs(exact).max() < 2 ** 24
    assert (got == _h(exact.astype(np.float32))).all()
    if op == "wgrad":
        assert ws_bytes > 0                      # the split path was the one exercised
    r = rng.integers(0, exact.shape[0], 200); c = rng.integers(0, exact.shape[1], 200)
    s16, _, _ = orc.linear_sampled(op, _h(Ai), _h(Bi), r, c)
    assert (got[r, c] == s16).all()


@pytest.mark.parametrize("op", ["fwd", "dgrad", "wgrad"])
@pytest.mark.parametrize("M,K,N", [(200, 328, 264), (640, 96, 40)])
def test_random_values_within_tolerance(orc, mp, op, M, K, N):
    rng = np.random.default_rng(17)
    sa, sb = _shapes_for(op, M, K, N)
    A, B = _h(rng.standard_normal(sa)), _h(rng.standard_normal(sb) / 4)
    got, _ = _run(mp, op, A, B)
    want = _oracle(orc, op, A, B)
    ex, ab = orc.linear_exact(op, A, B)
    red = {"fwd": K, "dgrad": N, "wgrad": M}[op]
    g = got.view(np.float16).astype(np.float64)
    # one FP16 rounding of the sum + FP32 accumulation in a different order
    tol = 2.0 ** -10 * np.abs(ex) + red * 2.0 ** -24 * ab + 2.0 ** -24
    assert (np.abs(g - ex) <= tol).all()
    w = want.view(np.float16).astype(np.float64)
    big = np.abs(w) >= 1e-3 * np.sqrt((w * w).mean())
    rel = np.abs(g[big] - w[big]) / np.abs(w[big])
    assert rel.max() <= 1e-2
    assert (got == want).mean() > 0.98           # nearly all outputs round identically


def test_overflow_and_nan_propagate_and_set_the_flag(orc, mp):
    """Outputs beyond FP16's range become inf (no saturation), inf - inf becomes NaN, and the
    weight-gradient kernel raises the device flag exactly when it stored such a value."""
    M, K, N = 64, 40, 48
    rng = np.random.default_rng(2)
    X = _h(rng.integers(-2, 3, (M, K))); dY = _h(rng.integers(-2, 3, (M, N)))
    st = mp.State()
    got, _ = _run(mp, "wgrad", X, dY, st)
    assert st.read().found_inf == 0 and (got == orc.linear_bwd_wgrad(X, dY)).all()
    X2 = X.copy(); X2[:, 3] = _h(np.full(M, 300.0)); dY2 = dY.copy(); dY2[:, 5] = _h(np.full(M, 300.0))
    got, _ = _run(mp, "wgrad", X2, dY2, st)
    want = orc.linear_bwd_wgrad(X2, dY2)
    assert want[3, 5] == 0x7C00 and (got == want).all()
    assert st.read().found_inf == 1
    mp.mp_loss_scale_update(st)
    assert st.read().found_inf == 0
    dY3 = dY.copy(); dY3[0, 7] = 0x7C00; dY3[1, 7] = 0xFC00
    X3 = X.copy(); X3[0, :] = _h(np.ones(K)); X3[1, :] = _h(np.ones(K))
    got, _ = _run(mp, "wgrad", X3, dY3, st)
    col = got[:, 7]
    assert ((col & 0x7C00) == 0x7C00).all() and ((col & 0x3FF) != 0).all()      # NaN column
    assert st.read().found_inf == 1
    st.close()


def test_argument_errors(mp):
    a = torch.zeros(16, 16, dtype=torch.float16, device="cuda")
    odd = torch.zeros(16, 20, dtype=torch.float16, device="cuda")       # pitch 20: not a multiple of 8
    with pytest.raises(mp.MpError) as e:
        mp.mp_linear_fwd(odd[:, :16], a, torch.zeros(16, 16, dtype=torch.float16, device="cuda"))
    assert e.value.code == mp.MP_ERR_ALIGNMENT
    big = torch.zeros(4096, 128, dtype=torch.float16, device="cuda")
    dy = torch.zeros(4096, 256, dtype=torch.float16, device="cuda")
    dw = torch.zeros(128, 256, dtype=torch.float16, device="cuda")
    assert mp.mp_gemm_workspace_bytes(4096, 128, 256, mp.MP_OP_WGRAD) > 0
    with pytest.raises(mp.MpError) as e:
        mp.mp_linear_bwd_wgrad(big, dy, dw, None, None)                   # workspace missing
    assert e.value.code == mp.MP_ERR_NOMEM


def test_results_do_not_depend_on_timing(mp):
    """Split reductions add their partial sums in a fixed order and nothing uses atomics on
    values, so repeated launches on the same inputs give identical bits (a race in the pipeline
    or in the split path would show up here as a difference)."""
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    for (M, K, N) in [(3000, 200, 296), (8192, 1024, 1024), (4096, 128, 256)]:
        X = (torch.randn(M, K, generator=g, device="cuda")).half()
        dY = (torch.randn(M, N, generator=g, device="cuda") * 8).half()
        W = (torch.randn(K, N, generator=g, device="cuda") / 16).half()
        ws = torch.empty(max(max(mp.mp_gemm_workspace_bytes(M, K, N, o) for o in range(3)), 16),
                         dtype=torch.uint8, device="cuda")
        ref = None
        for rep in range(4):
            dW = torch.zeros(K, N, dtype=torch.float16, device="cuda")
            dX = torch.zeros(M, K, dtype=torch.float16, device="cuda")
            Y = torch.zeros(M, N, dtype=torch.float16, device="cuda")
            ws.fill_(rep)                                   # stale scratch contents must not matter
            mp.mp_linear_bwd_wgrad(X, dY, dW, None, ws)
            mp.mp_linear_bwd_dgrad(dY, W, dX, ws)
            mp.mp_linear_fwd(X, W, Y, ws)
            out = [t.view(torch.int16).clone() for t in (dW, dX, Y)]
            if ref is None:
                ref = out
            else:
                assert all(torch.equal(a, b) for a, b in zip(ref, out))
    assert mp.mp_gemm_device_status() == 0
