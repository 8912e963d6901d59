"""Parity of the streaming kernels (scale, inspect, fused master update, loss-scale state
machine) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1805_10387_b200 import synth  # noqa: E402


def _h(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _dev16(bits):
    return torch.from_numpy(bits.view(np.float16).copy()).cuda()


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _f32bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


class Tensors:
    """n tensors carved out of flat buffers at 16-byte-aligned offsets (ragged sizes)."""

    def __init__(self, counts, adam=True):
        offs, tot = [], 0
        for c in counts:
            offs.append(tot)
            tot += (c + 7) // 8 * 8
        self.counts, self.offs = counts, offs
        mk = lambda dt: torch.zeros(max(tot, 8), dtype=dt, device="cuda")
        self.g16, self.w16 = mk(torch.float16), mk(torch.float16)
        self.w32, self.m = mk(torch.float32), mk(torch.float32)
        self.v = mk(torch.float32) if adam else None
        self.views = lambda flat: [flat[o:o + c] for o, c in zip(offs, counts)]

    def plan(self, mp):
        return mp.UpdatePlan(self.views(self.g16), self.views(self.w32), self.views(self.m),
                             self.views(self.v) if self.v is not None else None, self.views(self.w16))


def test_scale_upstream_bitwise(orc, mp):
    rng = np.random.default_rng(0)
    for n, S in ((1, 65536.0), (7, 10.0), (4099, 2.0 ** 15), (100003, 3.0)):
        g = (rng.standard_normal(n) * np.exp(rng.uniform(-12, 3, n))).astype(np.float32)
        g[0] = np.inf if n > 1 else g[0]
        st = mp.State(init_scale=S)
        out = torch.zeros(n + 8, dtype=torch.float16, device="cuda")
        mp.mp_scale_upstream(torch.from_numpy(g).cuda(), out[:n], st)
        got = _bits(out)
        assert (got[:n] == orc.scale_upstream(g, S)).all()
        assert (got[n:] == 0).all()
        st.close()


def test_check_finite_positions_and_patterns(orc, mp):
    n = 10007
    base = _h(np.random.default_rng(1).standard_normal(n))
    st = mp.State()
    mp.mp_check_finite(_dev16(base), st)
    assert st.read().found_inf == 0
    for pos in (0, 7, 8, 4096, n - 8, n - 7, n - 1):
        for bad in (0x7C00, 0xFC00, 0x7E00, 0xFFFF, 0x7C01):
            g = base.copy(); g[pos] = bad
            mp.mp_check_finite(_dev16(g), st)
            assert st.read().found_inf == orc.found_inf(g) == 1
            mp.mp_loss_scale_update(st)                      # clears the flag
            assert st.read().found_inf == 0
    g = base.copy(); g[3] = 0x7BFF; g[n - 1] = 0xFBFF         # largest finite magnitudes
    mp.mp_check_finite(_dev16(g), st)
    assert st.read().found_inf == 0
    st.close()


def test_check_finite_exhaustive_patterns(orc, mp):
    """Every one of the 65536 patterns, each alone in a one-element tensor of a plan."""
    allbits = np.arange(65536, dtype=np.uint16)
    want = np.array([orc.found_inf(allbits[i:i + 1]) for i in range(65536)])
    st = mp.State()
    # finite ones together must not raise the flag; each non-finite one alone must
    fin = allbits[want == 0]
    mp.mp_check_finite(_dev16(fin), st)
    assert st.read().found_inf == 0
    bad = allbits[want == 1]
    assert bad.size == 2048                              # 2 infinities + 2046 NaNs
    buf = torch.from_numpy(fin[:100].view(np.int16).copy()).cuda()
    for h in bad:                                        # all of them, one at a time
        buf[50] = int(np.int16(np.uint16(h).view(np.int16)))
        mp.mp_check_finite(buf.view(torch.float16), st)
        assert st.read().found_inf == 1, hex(int(h))
        mp.mp_loss_scale_update(st)
    st.close()


@pytest.mark.parametrize("kind", ["adam", "momentum"])
@pytest.mark.parametrize("counts", [[1], [5, 0, 13, 4096, 4097, 8191, 8192, 8193, 3, 100000], [1 << 20]])
def test_master_update_matches_oracle(orc, mp, kind, counts):
    rng = np.random.default_rng(len(counts))
    adam = kind == "adam"
    T = Tensors(counts, adam)
    S = 1024.0
    st = mp.State(init_scale=S, growth_interval=3)
    opt = mp.OptimConfig(mp.MP_OPT_ADAM if adam else mp.MP_OPT_MOMENTUM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
    host = []
    for c, o in zip(counts, T.offs):
        w = (rng.standard_normal(c) / 16).astype(np.float32)
        T.w32[o:o + c] = torch.from_numpy(w).cuda()
        host.append(dict(w32=w.copy(), m=np.zeros(c, np.float32), v=np.zeros(c, np.float32),
                         w16=np.zeros(c, np.uint16)))
    plan = T.plan(mp)
    sc = orc.Scaler(S, 3)
    for step in range(5):
        flag_want = 0
        gs = []
        for i, (c, o) in enumerate(zip(counts, T.offs)):
            g = _h(rng.standard_normal(c) * 0.02 * sc.S)
            if step == 2 and i == len(counts) - 1 and c:
                g[c - 1] = 0x7E00                              # NaN in the very last element
            gs.append(g)
            if c:
                T.g16[o:o + c] = _dev16(g)
            flag_want |= orc.found_inf(g)
        mp.mp_master_update(plan, st, opt, 1)                 # check_mode 1: inspect in the call
        assert st.read().found_inf == flag_want
        if not flag_want:
            for g, hs in zip(gs, host):
                if adam:
                    orc.adam_update(g, hs["w32"], hs["m"], hs["v"], hs["w16"], sc.S, 1e-3, 0.9, 0.999,
                                    1e-8, sc.t + 1)
                else:
                    orc.momentum_update(g, hs["w32"], hs["m"], hs["w16"], sc.S, 1e-3, 0.9)
        sc.update(flag_want)
        mp.mp_loss_scale_update(st)
        h = st.read()
        assert (h.scale, h.good_steps, h.t, h.skipped, h.step) == (sc.S, sc.good, sc.t, sc.skipped, sc.step)
        for (c, o), hs in zip(zip(counts, T.offs), host):
            if not c:
                continue
            w32 = T.w32[o:o + c].cpu().numpy(); m = T.m[o:o + c].cpu().numpy()
            w16 = _bits(T.w16[o:o + c])
            tol = 1e-6 * np.maximum(np.abs(hs["w32"]), 1e-3)
            assert (np.abs(w32 - hs["w32"]) <= tol).all()
            assert (np.abs(m - hs["m"]) <= 1e-6 * np.maximum(np.abs(hs["m"]), 1e-6)).all()
            if adam:
                v = T.v[o:o + c].cpu().numpy()
                assert (np.abs(v - hs["v"]) <= 1e-6 * np.maximum(np.abs(hs["v"]), 1e-12)).all()
            if step > 0 or not flag_want:
                assert (w16 == orc.f2h(w32)).all()            # working copy = rounded master, bitwise
            # every operation is individually rounded on both sides: expect identical bits
            assert (_f32bits(w32) == _f32bits(hs["w32"])).mean() > 0.999
    # alignment padding between tensors was never written
    pad = torch.ones_like(T.w32, dtype=torch.bool)
    for c, o in zip(counts, T.offs):
        pad[o:o + c] = False
    assert bool((T.w32[pad] == 0).all()) and bool((T.w16[pad] == 0).all())
    st.close(); plan.close()


def test_overflow_step_is_a_bitwise_no_op(orc, mp):
    counts = [777, 8192 * 3 + 5]
    T = Tensors(counts)
    rng = np.random.default_rng(3)
    for flat in (T.w32, T.m, T.v):
        flat.copy_(torch.from_numpy(rng.standard_normal(flat.numel()).astype(np.float32)).cuda())
    T.v.abs_()
    T.w16.copy_(T.w32.half())
    T.g16.copy_(torch.from_numpy(rng.standard_normal(T.g16.numel()).astype(np.float16)).cuda())
    T.g16[T.offs[1] + 8192 * 3 + 4] = float("inf")            # in the ragged tail of the last chunk
    before = [x.clone() for x in (T.w32, T.m, T.v, T.w16)]
    st = mp.State(init_scale=4.0)
    plan = T.plan(mp)
    opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
    mp.mp_master_update(plan, st, opt, 1)
    mp.mp_loss_scale_update(st)
    h = st.read()
    assert (h.scale, h.t, h.skipped, h.step, h.found_inf) == (2.0, 0, 1, 1, 0)
    for a, b in zip(before, (T.w32, T.m, T.v, T.w16)):
        assert torch.equal(a.view(torch.int32) if a.dtype == torch.float32 else a.view(torch.int16),
                           b.view(torch.int32) if b.dtype == torch.float32 else b.view(torch.int16))
    # same flag, trusted (check_mode 0) after a separate inspection
    mp.mp_check_finite(T.g16, st)
    mp.mp_master_update(plan, st, opt, 0)
    for a, b in zip(before, (T.w32, T.m, T.v, T.w16)):
        assert torch.equal(a, b)
    assert st.read().found_inf == 1
    st.close(); plan.close()


def test_power_of_two_scale_invariance_on_device(mp):
    """Same gradients presented at S = 1 and at S = 2^k give bitwise the same updated state."""
    rng = np.random.default_rng(4)
    n = 50000
    g = (rng.standard_normal(n) * 0.05).astype(np.float16)
    g[np.abs(g) < 2.0 ** -10] = 2.0 ** -10                    # stays normal at S = 1
    w0 = rng.standard_normal(n).astype(np.float32)
    ref = None
    for k in (0, 3, 10):
        T = Tensors([n])
        T.w32[:n] = torch.from_numpy(w0).cuda()
        T.g16[:n] = torch.from_numpy((g.astype(np.float32) * 2.0 ** k).astype(np.float16)).cuda()
        st = mp.State(init_scale=2.0 ** k)
        plan = T.plan(mp)
        mp.mp_master_update(plan, st, mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 1e-2), 1)
        snap = [x[:n].cpu() for x in (T.w32, T.m, T.v, T.w16)]
        if ref is None:
            ref = snap
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, snap))
        st.close(); plan.close()


def test_scaler_clamps_static_mode_and_log(orc, mp):
    st = mp.State(init_scale=2.0, growth_interval=1, min_scale=1.0, max_scale=8.0)
    sc = orc.Scaler(2.0, 1, 1.0, 8.0)
    flags = [0, 0, 0, 0, 1, 1, 1, 1, 0]
    one = torch.zeros(8, dtype=torch.float16, device="cuda")
    bad = one.clone(); bad[3] = float("nan")
    for f in flags:
        mp.mp_check_finite(bad if f else one, st)
        mp.mp_loss_scale_update(st)
        sc.update(f)
        assert st.read().scale == sc.S
    log = st.read_log()
    assert [r.found_inf for r in log] == flags and [r.step for r in log] == list(range(len(flags)))
    assert log[-1].scale_after == sc.S and log[4].scale_before == 8.0 and log[4].scale_after == 4.0
    st.close()
    st = mp.State(init_scale=10.0, growth_interval=2, dynamic=False)
    for f in (0, 0, 1, 0):
        mp.mp_check_finite(bad if f else one, st)
        mp.mp_loss_scale_update(st)
        assert st.read().scale == 10.0
    h = st.read()
    assert (h.t, h.skipped) == (3, 1)
    st.close()


def test_sweep_workload_trajectory(orc, mp):
    """Update-only workload at 1e6 parameters in 64 log-uniform tensors: flags, skip decisions
    and the scale sequence must equal the oracle's bit for bit over 40 steps."""
    sw = synth.UpdateSweep(P=1_000_000, n_tensors=64)
    steps = 40
    plant = synth.overflow_steps(sw, steps)
    T = Tensors(sw.counts)
    plan = T.plan(mp)
    st = mp.State(init_scale=sw.init_scale, growth_interval=sw.growth_interval)
    sc = orc.Scaler(sw.init_scale, sw.growth_interval)
    opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
    g32 = torch.empty(T.g16.numel(), dtype=torch.float32, device="cuda")
    w_host = np.zeros(T.g16.numel(), np.float32); m_host = np.zeros_like(w_host); v_host = np.zeros_like(w_host)
    w16_host = np.zeros(T.g16.numel(), np.uint16)
    flags = []
    for s in range(steps):
        z = (synth.normal(sw.seed, 1000 + s, T.g16.numel()) * sw.grad_std).astype(np.float32)
        g32.copy_(torch.from_numpy(z))
        mp.mp_scale_upstream(g32, T.g16, st)                   # S is read on the device
        g_host = orc.scale_upstream(z, sc.S)
        if plant[s]:
            pos = T.offs[s % 64] + (s * 7919) % sw.counts[s % 64]
            bits = 0x7C00 if s % 2 == 0 else 0x7E00
            T.g16.view(torch.int16)[pos] = bits
            g_host[pos] = bits
        mp.mp_master_update(plan, st, opt, 1)
        f = 0
        for c, o in zip(sw.counts, T.offs):
            f |= orc.found_inf(g_host[o:o + c])
        assert st.read().found_inf == f
        if not f:
            for c, o in zip(sw.counts, T.offs):
                orc.adam_update(g_host[o:o + c], w_host[o:o + c], m_host[o:o + c], v_host[o:o + c],
                                w16_host[o:o + c], sc.S, 1e-3, 0.9, 0.999, 1e-8, sc.t + 1)
        sc.update(f)
        mp.mp_loss_scale_update(st)
        flags.append(f)
        assert st.read().scale == sc.S
    assert sum(flags) >= 1 and flags[3] == 1
    log = st.read_log()
    assert [r.found_inf for r in log] == flags
    w = T.w32.cpu().numpy()
    live = np.zeros(w.size, bool)
    for c, o in zip(sw.counts, T.offs):
        live[o:o + c] = True
    assert (np.abs(w - w_host)[live] <= 1e-6 * np.maximum(np.abs(w_host[live]), 1e-3)).all()
    assert (_bits(T.w16)[live] == w16_host[live]).mean() > 0.9999
    st.close(); plan.close()


@pytest.mark.parametrize("kind", ["adam", "momentum"])
def test_weight_decay_on_the_master_copy(orc, mp, kind):
    """Section 3.3: the decay term is formed from the FP32 master and added to the FP32 gradient.
    With a coefficient of 1e-5 and weights near 5e-4 the product is below FP16's smallest
    subnormal, so a decay formed in FP16 would vanish; here it must move the weights."""
    n = 12345
    adam = kind == "adam"
    rng = np.random.default_rng(8)
    T = Tensors([n], adam)
    w0 = (rng.standard_normal(n) * 5e-4).astype(np.float32)
    T.w32[:n] = torch.from_numpy(w0).cuda()
    host = dict(w32=w0.copy(), m=np.zeros(n, np.float32), v=np.zeros(n, np.float32), w16=np.zeros(n, np.uint16))
    plan = T.plan(mp)
    st = mp.State(init_scale=256.0, growth_interval=1000)
    wd = 1e-5
    assert ((orc.f2h((wd * w0).astype(np.float32)) & 0x7FFF) == 0).mean() > 0.99   # lost in FP16
    opt = mp.OptimConfig(mp.MP_OPT_ADAM if adam else mp.MP_OPT_MOMENTUM, 1e-2, 0.9, 0.999, 1e-8, 0.9, wd)
    zero_g = np.zeros(n, np.uint16)                                        # gradient exactly zero
    for step in range(4):
        T.g16[:n] = _dev16(zero_g)
        mp.mp_master_update(plan, st, opt, 1)
        mp.mp_loss_scale_update(st)
        if adam:
            orc.adam_update(zero_g, host["w32"], host["m"], host["v"], host["w16"], 256.0, 1e-2, 0.9, 0.999,
                            1e-8, step + 1, wd)
        else:
            orc.momentum_update(zero_g, host["w32"], host["m"], host["w16"], 256.0, 1e-2, 0.9, wd)
    w = T.w32[:n].cpu().numpy()
    assert (np.abs(w - host["w32"]) <= 1e-6 * np.maximum(np.abs(host["w32"]), 1e-3)).all()
    moved = np.abs(w - w0) > 0
    assert moved.mean() > 0.99                                             # the decay acted
    if not adam:                                                           # plain decay shrinks weights
        assert (np.sign(w0 - w)[moved] == np.sign(w0)[moved]).all() and (np.abs(w) < np.abs(w0))[moved].all()
    assert (_bits(T.w16[:n]) == orc.f2h(w)).all()
    st.close(); plan.close()


def test_state_checkpoint_and_resume(orc, mp):
    """Ten steps in one go equal five steps, a state export / import into fresh objects, and five
    more steps, bit for bit (loss scale, counters, master weights, moments)."""
    rng = np.random.default_rng(9)
    n = 50000
    w0 = rng.standard_normal(n).astype(np.float32)
    grads = [(rng.standard_normal(n) * 300.0).astype(np.float16) for _ in range(10)]
    grads[3][17] = np.inf
    opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)

    def fresh():
        T = Tensors([n])
        T.w32[:n] = torch.from_numpy(w0).cuda()
        return T, T.plan(mp), mp.State(init_scale=1024.0, growth_interval=2)

    def run(T, plan, st, lo, hi):
        for s in range(lo, hi):
            T.g16[:n] = torch.from_numpy(grads[s]).cuda()
            mp.mp_master_update(plan, st, opt, 1)
            mp.mp_loss_scale_update(st)
    Ta, pa, sa = fresh()
    run(Ta, pa, sa, 0, 10)
    Tb, pb, sb = fresh()
    run(Tb, pb, sb, 0, 5)
    snap = sb.read()                                           # export
    saved = [x.clone() for x in (Tb.w32, Tb.m, Tb.v, Tb.w16)]
    Tc, pc, sc2 = fresh()                                      # import into new objects
    for dst, src in zip((Tc.w32, Tc.m, Tc.v, Tc.w16), saved):
        dst.copy_(src)
    sc2.write(snap)
    run(Tc, pc, sc2, 5, 10)
    ha, hc = sa.read(), sc2.read()
    assert (ha.scale, ha.t, ha.step, ha.skipped, ha.good_steps) == (hc.scale, hc.t, hc.step, hc.skipped, hc.good_steps)
    assert ha.skipped == 1
    for x, y in zip((Ta.w32, Ta.m, Ta.v), (Tc.w32, Tc.m, Tc.v)):
        assert torch.equal(x.view(torch.int32), y.view(torch.int32))
    assert torch.equal(Ta.w16.view(torch.int16), Tc.w16.view(torch.int16))
    for s_, p_ in ((sa, pa), (sb, pb), (sc2, pc)):
        s_.close(); p_.close()


def test_log_ring_wraps(mp):
    """More steps than the ring holds: the newest MP_LOG_CAPACITY records come back, oldest first."""
    st = mp.State(init_scale=4.0, growth_interval=1000)
    n = mp.MP_LOG_CAPACITY + 137
    for _ in range(n):
        mp.mp_loss_scale_update(st)
    log = st.read_log()
    assert len(log) == mp.MP_LOG_CAPACITY
    assert [r.step for r in log] == list(range(n - mp.MP_LOG_CAPACITY, n))
    assert st.read().step == n and st.read().t == n
    few = st.read_log(5)
    assert [r.step for r in few] == list(range(n - 5, n))
    st.close()


@pytest.mark.parametrize("H", [1, 2, 3])
def test_scaler_overflow_tolerance(orc, mp, H):
    """Second policy (halve at the H-th overflow since S last changed) against the oracle on a
    seeded flag sequence with bursts, isolated overflows and doublings."""
    rng = np.random.default_rng(40 + H)
    flags = (rng.uniform(size=300) < 0.15).astype(int).tolist() + [1] * 7 + [0] * 9 + [1, 0, 0, 0, 1, 1]
    st = mp.State(init_scale=2.0 ** 12, growth_interval=3, min_scale=2.0 ** 6, max_scale=2.0 ** 15,
                  overflow_tolerance=H)
    sc = orc.Scaler(2.0 ** 12, 3, 2.0 ** 6, 2.0 ** 15, tolerance=H)
    one = torch.zeros(8, dtype=torch.float16, device="cuda")
    bad = one.clone(); bad[5] = float("inf")
    want = []
    for f in flags:
        mp.mp_check_finite(bad if f else one, st)
        mp.mp_loss_scale_update(st)
        sc.update(f)
        want.append(sc.S)
    log = st.read_log()
    assert [r.scale_after for r in log] == want and [r.found_inf for r in log] == flags
    h = st.read()
    assert (h.scale, h.t, h.skipped, h.good_steps, h.strikes, h.overflow_tolerance) == \
        (sc.S, sc.t, sc.skipped, sc.good, sc.strikes, H)
    st.close()
    with pytest.raises(Exception):
        mp.State(overflow_tolerance=0)
