"""Pins for the oracle's flag, unscale + optimizer update and loss-scale state machine.

Expected values are closed forms of Adam / momentum for special inputs, a library
optimizer run in float64 (torch.optim, an implementation independent of the oracle),
and the hand-derived scale trajectory in tests/golden/.
"""
import os

import numpy as np
import pytest
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _f(h):
    return h.view(np.float16).astype(np.float64)


# ------------------------------------------------------------------ flag
def test_flag_exhaustive_single_element(orc):
    for h in range(65536):
        want = 1 if ((h >> 10) & 0x1F) == 0x1F else 0
        assert orc.found_inf(np.array([h], np.uint16)) == want


def test_flag_position_sweep(orc):
    n = 1003
    base = _h(np.random.default_rng(0).standard_normal(n))
    assert orc.found_inf(base) == 0
    for pos in (0, 1, 7, 8, 500, n - 9, n - 2, n - 1):
        for bad in (0x7C00, 0xFC00, 0x7E00, 0xFFFF):
            g = base.copy(); g[pos] = bad
            assert orc.found_inf(g) == 1
    g = base.copy(); g[5] = 0x7BFF; g[6] = 0xFBFF                  # largest finite values
    assert orc.found_inf(g) == 0
    assert orc.found_inf(np.empty(0, np.uint16)) == 0


# ------------------------------------------------------- upstream scaling
def _hx(h):
    return np.array([h], np.uint16)


def test_scale_upstream_scales_in_fp32_before_the_one_rounding(orc):
    """rn16(S * g32): the product is formed in FP32 and rounded to FP16 once.

    Each case has a value fixed by the binary16 format; rounding g to FP16 first, or
    multiplying in FP16, gives a different one."""
    one = lambda g, S: int(orc.scale_upstream(np.array([g], np.float32), S)[0])
    # 2^-26 is below half the smallest subnormal: FP16 holds it as 0, yet 2^16 * 2^-26 = 2^-10 is a normal
    assert one(2.0 ** -26, 2.0 ** 16) == 0x1400
    assert one(-(2.0 ** -26), 2.0 ** 16) == 0x9400
    # g = 1 + 2^-11 is a tie that FP16 rounds to 1.0; with S = 3 the FP32 product 3 + 1.5 * 2^-10 lies above
    # the midpoint between 3 and 3 + 2^-9, so the result is 3 + 2^-9; rounding g first would give 3.0 = 0x4200
    assert one(1.0 + 2.0 ** -11, 3.0) == 0x4201
    # S = 1 reduces to the plain conversion: the fixture's ties and thresholds
    for line in open(os.path.join(GOLD, "fp16_thresholds.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        g = np.array([int(line[0], 16)], np.uint32).view(np.float32)
        assert int(orc.scale_upstream(g, 1.0)[0]) == int(line[1], 16), line
    # overflow of the scaled value: 65520 is the first value that becomes inf
    assert one(65519.0 / 1024.0, 1024.0) == 0x7BFF          # 65519 < 65520 -> 65504
    assert one(65520.0 / 1024.0, 1024.0) == 0x7C00
    assert one(-64.0, 1024.0) == 0xFC00                     # -65536 -> -inf
    assert one(1.0, 2.0 ** 16) == 0x7C00
    assert one(np.inf, 2.0) == 0x7C00 and one(-np.inf, 2.0) == 0xFC00
    nan = one(np.nan, 2.0)
    assert (nan & 0x7C00) == 0x7C00 and (nan & 0x03FF) != 0
    assert one(0.0, 2.0 ** 16) == 0x0000 and one(-0.0, 2.0 ** 16) == 0x8000
    assert orc.scale_upstream(np.empty(0, np.float32), 4.0).size == 0


def test_scale_upstream_against_library_product(orc):
    """10^6 seeded floats, S = 10 (not a power of two) and S = 2^15: numpy's float32 product cast to
    float16 is the same definition in an independent implementation."""
    rng = np.random.default_rng(77)
    g = (rng.standard_normal(1_000_000) * np.exp(rng.uniform(-18, 9, 1_000_000))).astype(np.float32)
    g[:8] = [0.0, -0.0, np.inf, -np.inf, 6552.0, 6551.9, 2.0 ** -27, -(2.0 ** -24)]
    for S in (10.0, 2.0 ** 15, 3.0, 1.0):
        with np.errstate(over="ignore"):
            want = (np.float32(S) * g).astype(np.float16).view(np.uint16)
        got = orc.scale_upstream(g, S)
        assert (got == want).all(), S
        assert ((got & 0x7C00) == 0x7C00).any() and (got == 0).any()       # both ends exercised
    # and not the result of rounding first: on this sample the two differ somewhere
    with np.errstate(over="ignore"):
        first = (g.astype(np.float16).astype(np.float32) * np.float32(10.0)).astype(np.float16).view(np.uint16)
    assert (first != orc.scale_upstream(g, 10.0)).any()


# ------------------------------------------------------------------ Adam
ADAM = dict(lr=1e-3, b1=0.9, b2=0.999, eps=1e-8)


def _state(n, w=None):
    w32 = np.zeros(n, np.float32) if w is None else np.asarray(w, np.float32).copy()
    return w32, np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.uint16)


def test_adam_first_step_closed_form(orc):
    """From zero moments: m/c1 = g, v/c2 = g^2, so dw = -lr * g / (|g| + eps)."""
    g = np.array([0.5, -0.25, 3.0, -1e-3, 2.0 ** -14, 0.0], np.float32)
    w32, m, v, w16 = _state(g.size, np.linspace(-1, 1, g.size))
    w0 = w32.astype(np.float64)
    orc.adam_update(_h(g), w32, m, v, w16, 1.0, t=1, **ADAM)
    gd = _f(_h(g))                                   # the gradient as FP16 holds it
    want = w0 - 1e-3 * gd / (np.abs(gd) + 1e-8)
    assert np.abs(w32 - want).max() <= 2e-7
    # 1-b1 and 1-b2 are formed in FP32: relative error up to 2.4e-7 and 1.3e-5
    assert np.allclose(m, 0.1 * gd, rtol=1e-6) and np.allclose(v, 0.001 * gd * gd, rtol=5e-5)
    assert w32[-1] == np.float32(w0[-1]) and m[-1] == 0 and v[-1] == 0     # g = 0 moves nothing
    assert (w16 == _h(w32)).all()


def test_adam_constant_gradient_closed_form(orc):
    """Constant g: m_t = g(1-b1^t), v_t = g^2(1-b2^t), every step moves by -lr*g/(|g|+eps)."""
    g = np.array([0.125, -2.0, 0.03125], np.float32)
    w32, m, v, w16 = _state(3)
    gd = g.astype(np.float64)
    for t in range(1, 41):
        orc.adam_update(_h(g), w32, m, v, w16, 1.0, t=t, **ADAM)
        assert np.allclose(m, gd * (1 - 0.9 ** t), rtol=2e-6)
        assert np.allclose(v, gd * gd * (1 - 0.999 ** t), rtol=5e-5)
        assert np.allclose(w32, -t * 1e-3 * gd / (np.abs(gd) + 1e-8), rtol=5e-6)


def test_adam_epsilon_sits_outside_the_root_of_corrected_v(orc):
    """With |g| = eps the step is lr/2: only 'sqrt(v/c2) + eps' gives that."""
    g16 = np.array([0x0001], np.uint16)                     # 2^-24, exact in FP16
    eps = 2.0 ** -24
    w32, m, v, w16 = _state(1)
    orc.adam_update(g16, w32, m, v, w16, 1.0, 1e-3, 0.9, 0.999, eps, t=1)
    assert abs(w32[0] + 0.5e-3) < 1e-9


def test_adam_unscale_and_step_count(orc):
    g = np.array([0.75, -0.5], np.float32)
    a = _state(2, [1.0, 2.0]); b = _state(2, [1.0, 2.0])
    orc.adam_update(_h(g * 1024), *a, 1024.0, t=3, **ADAM)
    orc.adam_update(_h(g), *b, 1.0, t=3, **ADAM)
    for x, y in zip(a, b):
        assert (x.view(np.uint8) == y.view(np.uint8)).all()          # power-of-two S: bitwise
    c = _state(2, [1.0, 2.0])
    orc.adam_update(_h(g), *c, 1.0, t=4, **ADAM)
    assert (c[0] != b[0]).any()                                      # bias correction uses t


@pytest.mark.parametrize("wd", [0.0, 1e-2])
def test_adam_against_library_float64(orc, wd):
    rng = np.random.default_rng(21)
    n, steps, S = 257, 25, 512.0
    w0 = rng.standard_normal(n).astype(np.float32) * 0.1
    w32, m, v, w16 = _state(n, w0)
    p = torch.tensor(w0.astype(np.float64), requires_grad=True)
    opt = torch.optim.Adam([p], lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    for t in range(1, steps + 1):
        g16 = _h(rng.standard_normal(n) * 0.01 * S)
        orc.adam_update(g16, w32, m, v, w16, S, t=t, weight_decay=wd, **ADAM)
        p.grad = torch.tensor(_f(g16) / S)
        opt.step()
        ref = p.detach().numpy()
        assert np.abs(w32 - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())
    assert (w16 == _h(w32)).all()


def test_weight_decay_is_formed_from_the_fp32_master(orc):
    """Section 3.3: the decay term uses the FP32 master, not the FP16 working copy.  With a zero
    gradient the only input of the step is wd * w, for weights that FP16 cannot hold exactly."""
    w0 = np.array([1.0 + 2.0 ** -12, 3.0001, -0.3333333, 1e-9, 70000.0], np.float32)   # none is an FP16 value
    assert (_h(w0).view(np.float16).astype(np.float32) != w0).all()
    g0 = np.zeros(w0.size, np.uint16)
    # momentum SGD with mu = 0, lr * wd = 1/2: every step halves the master exactly
    w32 = w0.copy(); u = np.zeros_like(w0); w16 = np.zeros(w0.size, np.uint16)
    for step in range(1, 4):
        orc.momentum_update(g0, w32, u, w16, 1.0, 0.5, 0.0, 1.0)
        assert (w32 == w0 * np.float32(0.5 ** step)).all()
        assert (u == w0 * np.float32(0.5 ** (step - 1))).all()              # u = wd * w of the step
    # Adam: the first moment is (1 - b1) * wd * w32 to FP32 rounding; from the FP16 copy it would be off by 2^-11
    w32, m, v, w16 = _state(w0.size, w0)
    orc.adam_update(g0, w32, m, v, w16, 1.0, t=1, weight_decay=0.5, **ADAM)
    want = (1.0 - np.float64(np.float32(0.9))) * 0.5 * w0.astype(np.float64)
    assert np.allclose(m, want, rtol=1e-6, atol=0)


# -------------------------------------------------------------- momentum
def test_momentum_constant_gradient_closed_form(orc):
    g = np.array([0.5, -0.125], np.float32)
    w32 = np.zeros(2, np.float32); u = np.zeros(2, np.float32); w16 = np.zeros(2, np.uint16)
    gd = g.astype(np.float64); acc = np.zeros(2)
    for t in range(1, 31):
        orc.momentum_update(_h(g * 4), w32, u, w16, 4.0, 1e-2, 0.9)
        ut = gd * (1 - 0.9 ** t) / (1 - 0.9)
        acc -= 1e-2 * ut
        assert np.allclose(u, ut, rtol=2e-6)
        assert np.allclose(w32, acc, rtol=5e-6)
    assert (w16 == _h(w32)).all()


def test_momentum_against_library_float64(orc):
    rng = np.random.default_rng(22)
    n = 130
    w0 = rng.standard_normal(n).astype(np.float32)
    w32 = w0.copy(); u = np.zeros(n, np.float32); w16 = np.zeros(n, np.uint16)
    p = torch.tensor(w0.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=1e-3, momentum=0.9, weight_decay=1e-3)
    for _ in range(20):
        g16 = _h(rng.standard_normal(n) * 64.0)
        orc.momentum_update(g16, w32, u, w16, 64.0, 1e-3, 0.9, 1e-3)
        p.grad = torch.tensor(_f(g16) / 64.0)
        opt.step()
        assert np.abs(w32 - p.detach().numpy()).max() <= 2e-6


# ---------------------------------------------------------------- scaler
def _golden_trajectory():
    rows = [l.split() for l in open(os.path.join(GOLD, "scaler_c1_trajectory.txt"))
            if l.strip() and not l.startswith("#")]
    return [(int(a), int(b), int(c)) for a, b, c in rows]


def test_scaler_golden_trajectory(orc):
    s = orc.Scaler(init_scale=2.0 ** 16, interval=4)
    for step, flag, log2s in _golden_trajectory():
        s.update(flag)
        assert s.S == 2.0 ** log2s, step
    assert s.t == 9 and s.skipped == 1 and s.step == 10


def test_scaler_clamps_and_static_mode(orc):
    s = orc.Scaler(init_scale=2.0, interval=1, s_min=1.0, s_max=8.0)
    for want in (4.0, 8.0, 8.0, 8.0):
        s.update(0); assert s.S == want
    for want in (4.0, 2.0, 1.0, 1.0):
        s.update(1); assert s.S == want
    assert s.t == 4 and s.skipped == 4
    st = orc.Scaler(init_scale=10.0, interval=2, dynamic=False)
    for flag in (0, 0, 1, 0, 0, 0):
        st.update(flag); assert st.S == 10.0
    assert st.t == 5 and st.skipped == 1


def test_scaler_closed_form_from_flag_sequence(orc):
    """log2 S follows a counter walk: -1 on a flagged step, +1 on each N-th clean step in a row."""
    rng = np.random.default_rng(5)
    flags = (rng.uniform(size=400) < 0.07).astype(int)
    N, log2s, run = 5, 10, 0
    s = orc.Scaler(init_scale=2.0 ** 10, interval=N)
    for f in flags:
        if f:
            log2s, run = max(log2s - 1, 0), 0
        else:
            run += 1
            if run == N:
                log2s, run = min(log2s + 1, 24), 0
        s.update(int(f))
        assert s.S == 2.0 ** log2s and s.good == run


def test_scaler_overflow_tolerance_golden_and_invariants(orc):
    """Second policy: halve at the H-th overflow since S last changed."""
    rows = [tuple(int(x) for x in l.split()) for l in open(os.path.join(GOLD, "scaler_tolerance2_trajectory.txt"))
            if l.strip() and not l.startswith("#")]
    s = orc.Scaler(init_scale=2.0 ** 10, interval=3, tolerance=2)
    for step, flag, log2s in rows:
        s.update(flag)
        assert s.S == 2.0 ** log2s, step
    assert s.skipped == sum(f for _, f, _ in rows) and s.t == len(rows) - s.skipped
    # n overflows in a row from a fresh state halve floor(n / H) times; every one is skipped
    for H in (1, 2, 3, 5):
        for n in range(0, 12):
            s = orc.Scaler(init_scale=2.0 ** 20, interval=1000, tolerance=H)
            for _ in range(n):
                s.update(1)
            assert s.S == 2.0 ** (20 - n // H) and s.skipped == n and s.t == 0 and s.strikes == n % H
    # isolated overflows, each followed by a doubling, never halve when H >= 2
    s = orc.Scaler(init_scale=2.0 ** 10, interval=2, tolerance=2)
    for rep in range(5):
        s.update(1); assert s.S == 2.0 ** (10 + rep)
        s.update(0); s.update(0); assert s.S == 2.0 ** (11 + rep) and s.strikes == 0
    # static mode: nothing moves S, counters still advance
    s = orc.Scaler(init_scale=10.0, interval=2, dynamic=False, tolerance=2)
    for f in (1, 1, 1, 0, 0):
        s.update(f); assert s.S == 10.0
    assert s.skipped == 3 and s.t == 2
