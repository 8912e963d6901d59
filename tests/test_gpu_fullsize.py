"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times:
the GPU result is checked on sampled outputs that the oracle computes one by one."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1805_10387_b200 import synth  # noqa: E402


def _pad8(n):
    return (n + 7) // 8 * 8


def _dev16(bits):
    r, c = bits.shape
    buf = torch.zeros(r, _pad8(c), dtype=torch.float16, device="cuda")
    buf[:, :c] = torch.from_numpy(bits.view(np.float16)).cuda()
    return buf[:, :c]


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _rel_floor(red):
    """The stated bar, max relative error 1e-2 against the FP32-accumulated oracle, is applied to
    outputs of at least this fraction of the tensor's rms.  Both sides add the same exact products
    in FP32 but in different orders; over a reduction of `red` terms that moves a sum by about
    sqrt(red) * 2^-24 times the size of its partial sums (the rms), i.e. by 1e-2 of an output
    that cancelled down to ~1e-4 * sqrt(red) of the rms.  Smaller outputs are covered by the
    absolute bound above, which always holds."""
    return max(1e-3, 1e-4 * float(red) ** 0.5)


def _check_samples(orc, op, A, B, got, n_samples, seed):
    R, Cc = got.shape
    rng = np.random.default_rng(seed)
    rows = np.concatenate([rng.integers(0, R, n_samples), [0, R - 1, 0, R - 1, min(127, R - 1), min(128, R - 1)]])
    cols = np.concatenate([rng.integers(0, Cc, n_samples), [0, Cc - 1, Cc - 1, 0, min(255, Cc - 1), min(256, Cc - 1)]])
    want16, ex, ab = orc.linear_sampled(op, A, B, rows, cols)
    g = got[rows, cols].view(np.float16).astype(np.float64)
    w = want16.view(np.float16).astype(np.float64)
    red = {"fwd": A.shape[1], "dgrad": A.shape[1], "wgrad": A.shape[0]}[op]
    sure = np.abs(ex) < 65520.0 * (1 - 2.0 ** -9)              # clearly below the overflow threshold
    over = np.abs(ex) > 65520.0 * (1 + 2.0 ** -9)              # clearly above it
    # one FP16 rounding of the sum + FP32 accumulation in a different order
    tol = 2.0 ** -10 * np.abs(ex) + red * 2.0 ** -24 * ab + 2.0 ** -24
    assert (np.abs(g - ex)[sure] <= tol[sure]).all()
    assert np.isinf(g[over]).all() and (np.sign(g[over]) == np.sign(ex[over])).all()
    fin = sure & (np.abs(w) > 2.0 ** -14)
    rms = np.sqrt((w[fin] ** 2).mean())
    big = fin & (np.abs(w) >= _rel_floor(red) * rms)
    assert (np.abs(g[big] - w[big]) / np.abs(w[big])).max() <= 1e-2
    return float((got[rows, cols] == want16).mean())


LAYERS = [
    ("c2", 0, 1, 2.0 ** 15),      # 6400 x 2048 -> 4096
    ("c3", 0, 2, 2.0 ** 15),      # 8192 x 1024 -> 4096
    ("c3", 1, 2, 2.0 ** 15),      # 8192 x 4096 -> 1024
    ("c3", 2, 2, 2.0 ** 15),      # 8192 x 1024 -> 1024 (weight gradient takes the split path)
    ("c4", 0, 3, 2.0 ** 10),      # 25600 x 1600 -> 1600, heavy-tailed activations
    ("c4", 5, 3, 2.0 ** 10),      # 25600 x 1600 -> 29
]


@pytest.mark.parametrize("name,layer,seed,S", LAYERS)
def test_layer_products_at_full_size(orc, mp, name, layer, seed, S):
    cfg = synth.config(name)
    M, K, N = cfg.shapes[layer]
    X = synth.activations(cfg, layer, 0)
    W = synth.fp16_bits(synth.weights(cfg, layer)).reshape(K, N)
    g32 = synth.upstream(cfg, layer, 0)
    dXd, dWd, Yd = [torch.zeros(r, _pad8(c), dtype=torch.float16, device="cuda")[:, :c]
                    for r, c in ((M, K), (K, N), (M, N))]
    Xd, Wd = _dev16(X), _dev16(W)
    st = mp.State(init_scale=S)
    dYbuf = torch.zeros(M, _pad8(N), dtype=torch.float16, device="cuda")
    if _pad8(N) == N:
        mp.mp_scale_upstream(torch.from_numpy(g32).cuda(), dYbuf, st)
    else:
        tmp = torch.empty(M, N, dtype=torch.float16, device="cuda")
        mp.mp_scale_upstream(torch.from_numpy(g32).cuda(), tmp, st)
        dYbuf[:, :N] = tmp
    dYd = dYbuf[:, :N]
    need = max(mp.mp_gemm_workspace_bytes(M, K, N, op) for op in (0, 1, 2))
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    mp.mp_linear_fwd(Xd, Wd, Yd, ws)
    mp.mp_linear_bwd_wgrad(Xd, dYd, dWd, st, ws)
    mp.mp_linear_bwd_dgrad(dYd, Wd, dXd, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    dY = _bits(dYd)
    assert (dY == orc.scale_upstream(g32, S)).all()            # bitwise at full size
    same = [_check_samples(orc, "fwd", X, W, _bits(Yd), 1500, seed),
            _check_samples(orc, "wgrad", X, dY, _bits(dWd), 1500, seed + 1),
            _check_samples(orc, "dgrad", dY, W, _bits(dXd), 1500, seed + 2)]
    assert min(same) > 0.9                                      # most sampled outputs have identical bits
    # the flag the weight-gradient kernel raised = an independent scan of what it stored
    dWb = np.ascontiguousarray(_bits(dWd))
    assert st.read().found_inf == int(((dWb & 0x7C00) == 0x7C00).any()) == orc.found_inf(dWb)
    st.close()


@pytest.mark.parametrize("name,first", [("c2", 0), ("c3", 2)])
def test_grouped_layer_products_at_full_size(orc, mp, name, first):
    """The launch configuration the benchmark times for independent layers: four layers of one
    shape per launch (c2: gate products 0..3; c3: the four projections of block 0).  Every
    problem's three products are checked on sampled outputs, and the flag against a scan."""
    cfg = synth.config(name)
    layers = list(range(first, first + 4))
    M, K, N = cfg.shapes[first]
    assert all(cfg.shapes[l] == (M, K, N) for l in layers) and mp.mp_max_group() >= 4
    S = 2.0 ** 15
    st = mp.State(init_scale=S)
    Xs = [synth.activations(cfg, l, 0) for l in layers]
    Ws = [synth.fp16_bits(synth.weights(cfg, l)).reshape(K, N) for l in layers]
    dYs = [orc.scale_upstream(synth.upstream(cfg, l, 0), S) for l in layers]
    Xd, Wd, dYd = [_dev16(x) for x in Xs], [_dev16(w) for w in Ws], [_dev16(d) for d in dYs]
    mk = lambda r, c: [torch.zeros(r, c, dtype=torch.float16, device="cuda") for _ in layers]
    Yd, dWd, dXd = mk(M, N), mk(K, N), mk(M, K)
    need = max(mp.mp_gemm_workspace_bytes_grouped(4, M, K, N, op) for op in (0, 1, 2))
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    mp.mp_linear_fwd_grouped(Xd, Wd, Yd, ws)
    mp.mp_linear_bwd_wgrad_grouped(Xd, dYd, dWd, st, ws)
    mp.mp_linear_bwd_dgrad_grouped(dYd, Wd, dXd, ws)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    any_inf = 0
    for i, l in enumerate(layers):
        same = [_check_samples(orc, "fwd", Xs[i], Ws[i], _bits(Yd[i]), 600, 10 * l),
                _check_samples(orc, "wgrad", Xs[i], dYs[i], _bits(dWd[i]), 600, 10 * l + 1),
                _check_samples(orc, "dgrad", dYs[i], Ws[i], _bits(dXd[i]), 600, 10 * l + 2)]
        assert min(same) > 0.9, (l, same)
        any_inf |= int(((_bits(dWd[i]) & 0x7C00) == 0x7C00).any())
    assert st.read().found_inf == any_inf
    st.close()


@pytest.mark.parametrize("P,n_tensors,steps", [(1_000_000, 1, 8), (10_000_000, 8, 8),
                                               (100_000_000, 64, 5), (1_000_000_000, 500, 3)])
def test_update_sweep_at_full_size(orc, mp, P, n_tensors, steps):
    """Update-only workload (unscale / inspect / Adam / recast) at 1e6 .. 1e9 parameters in
    1 .. 500 tensors of log-uniform sizes.  Flags and the scale sequence are compared bit for
    bit with the oracle; values on sampled chunks (the update is elementwise, so the oracle
    runs on exactly the sampled elements).  The gradient is a 2^24-element seeded block
    repeated across the parameter range (drawing 1e9 normals on the host would dominate
    the test)."""
    sw = synth.UpdateSweep(P=P, n_tensors=n_tensors)
    counts = sw.counts
    offs, tot = [], 0
    for c in counts:
        offs.append(tot)
        tot += _pad8(c)
    mk = lambda dt: torch.zeros(tot, dtype=dt, device="cuda")
    g16, w16, w32, m, v = mk(torch.float16), mk(torch.float16), mk(torch.float32), mk(torch.float32), mk(torch.float32)
    views = lambda flat: [flat[o:o + c] for o, c in zip(offs, counts)]
    plan = mp.UpdatePlan(views(g16), views(w32), views(m), views(v), views(w16))
    st = mp.State(init_scale=sw.init_scale, growth_interval=2)
    sc = orc.Scaler(sw.init_scale, 2)
    opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
    BLK = 1 << 24
    # sampled chunks: start/end of the range, tensor boundaries, random interior places
    rng = np.random.default_rng(P % 1000 + n_tensors)
    picks = []
    for i in set([0, n_tensors - 1] + [int(x) for x in rng.integers(0, n_tensors, 12)]):
        c, o = counts[i], offs[i]
        for lo in {0, max(0, c - 1000), int(rng.integers(0, max(1, c - 1000)))}:
            picks.append((o + lo, min(1000, c - lo)))
    host = {pk: dict(w32=np.zeros(pk[1], np.float32), m=np.zeros(pk[1], np.float32),
                     v=np.zeros(pk[1], np.float32), w16=np.zeros(pk[1], np.uint16)) for pk in picks}
    w0 = (synth.normal(sw.seed, 5, BLK) * 0.05).astype(np.float32)
    w0d = torch.from_numpy(w0).cuda()
    for lo in range(0, tot, BLK):
        n = min(BLK, tot - lo)
        w32[lo:lo + n] = w0d[:n]
    for (lo, n), hs in host.items():
        hs["w32"][:] = w0[(lo + np.arange(n)) % BLK]
    flags = []
    for s in range(steps):
        z = (synth.normal(sw.seed, 2000 + s, BLK) * sw.grad_std).astype(np.float32)
        zd = torch.from_numpy(z).cuda()
        for lo in range(0, tot, BLK):
            n = min(BLK, tot - lo)
            mp.mp_scale_upstream(zd[:n], g16[lo:lo + n], st)    # rn16(S*g32), S read on the device
        plant = (s == 1)
        if plant:
            pos = offs[-1] + counts[-1] - 1                     # very last element of the last tensor
            g16.view(torch.int16)[pos] = 0x7E00
        mp.mp_master_update(plan, st, opt, 1)
        want_flag = int(plant)
        assert st.read().found_inf == want_flag
        gz = orc.scale_upstream(z, sc.S)
        assert orc.found_inf(gz) == 0                            # no natural overflow at these scales
        if not want_flag:
            for (lo, n), hs in host.items():
                gs = np.ascontiguousarray(gz[(lo + np.arange(n)) % BLK])
                orc.adam_update(gs, hs["w32"], hs["m"], hs["v"], hs["w16"], sc.S, 1e-3, 0.9, 0.999, 1e-8, sc.t + 1)
        sc.update(want_flag)
        mp.mp_loss_scale_update(st)
        h = st.read()
        assert (h.scale, h.t, h.skipped, h.good_steps) == (sc.S, sc.t, sc.skipped, sc.good)
        flags.append(want_flag)
    for (lo, n), hs in host.items():
        w = w32[lo:lo + n].cpu().numpy()
        assert (np.abs(w - hs["w32"]) <= 1e-6 * np.maximum(np.abs(hs["w32"]), 1e-3)).all()
        assert (np.abs(m[lo:lo + n].cpu().numpy() - hs["m"]) <= 1e-6 * np.maximum(np.abs(hs["m"]), 1e-7)).all()
        assert (_bits(w16[lo:lo + n]) == orc.f2h(w)).all()
        assert (w.view(np.uint32) == hs["w32"].view(np.uint32)).mean() > 0.99
    assert flags[1] == 1 and sum(flags) == 1
    st.close(); plan.close()


# ---------------------------------------------------------------------------------------------
# The whole step at full size, in the launch configuration the benchmark times: the stack built
# as bench.py builds it (grouped launches for independent layers, one scaling call over a flat
# gradient buffer, one flat update, the step replayed as a CUDA graph), on the workload's seeded
# inputs.  One batch is drawn and every step runs on it, as in the benchmark.
def _threads():
    import os
    return max(1, min(32, os.cpu_count() or 1))


def _sampled(orc, op, A, B, rows, cols):
    """orc.linear_sampled over the host's cores (the call releases the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    n = _threads()
    parts = [(rows[i::n], cols[i::n]) for i in range(n)]
    with ThreadPoolExecutor(n) as ex:
        res = list(ex.map(lambda rc: orc.linear_sampled(op, A, B, rc[0], rc[1]), parts))
    out = [np.empty(rows.size, dt) for dt in (np.uint16, np.float64, np.float64)]
    for i, r in enumerate(res):
        for o, x in zip(out, r):
            o[i::n] = x
    return out


def _check_product_samples(orc, op, A, B, got, n_samples, seed, what):
    """Forced-operand check on sampled outputs: the oracle's product of the very operands the GPU
    kernel read.  Bound: one FP16 rounding of the sum + FP32 summation-order error; and max
    relative error 1e-2 where the value is not tiny.  Returns the fraction of identical bits."""
    R, Cc = got.shape
    rng = np.random.default_rng(seed)
    edge_r = [0, R - 1, 0, R - 1, min(127, R - 1), min(128, R - 1), min(255, R - 1), min(256, R - 1)]
    edge_c = [0, Cc - 1, Cc - 1, 0, min(255, Cc - 1), min(256, Cc - 1), Cc - 1, max(0, Cc - 9)]
    rows = np.concatenate([rng.integers(0, R, n_samples), edge_r]).astype(np.int64)
    cols = np.concatenate([rng.integers(0, Cc, n_samples), edge_c]).astype(np.int64)
    want16, ex, ab = _sampled(orc, op, A, B, rows, cols)
    g = got[rows, cols].view(np.float16).astype(np.float64)
    w = want16.view(np.float16).astype(np.float64)
    red = {"fwd": A.shape[1], "dgrad": A.shape[1], "wgrad": A.shape[0]}[op]
    finite_ops = np.isfinite(ex) & np.isfinite(ab)
    sure = finite_ops & (np.abs(ex) < 65520.0 * (1 - 2.0 ** -9))
    over = finite_ops & (np.abs(ex) > 65520.0 * (1 + 2.0 ** -9))
    tol = 2.0 ** -10 * np.abs(ex) + red * 2.0 ** -24 * ab + 2.0 ** -24
    bad = sure & ~(np.abs(g - ex) <= tol)
    assert not bad.any(), (what, int(bad.sum()))
    assert np.isinf(g[over]).all() and (np.sign(g[over]) == np.sign(ex[over])).all(), what
    # operands that already hold inf/NaN (after an overflow further up): same class of result
    nf = ~finite_ops
    if nf.any():
        assert (np.isfinite(g[nf]) == np.isfinite(w[nf])).all(), what
    fin = sure & (np.abs(w) > 2.0 ** -14)
    if fin.any():
        rms = np.sqrt((w[fin] ** 2).mean())
        big = fin & (np.abs(w) >= _rel_floor(red) * rms)
        assert (np.abs(g[big] - w[big]) / np.abs(w[big])).max() <= 1e-2, what
    return float((got[rows, cols] == want16).mean())


def _build_like_bench(mp, cfg):
    from paper_1805_10387_b200.stack import LinearStack
    L = len(cfg.shapes)
    chained = [cfg.chained(l) for l in range(L)]
    stack = LinearStack(cfg.shapes, chained, optimizer=cfg.optimizer, lr=cfg.lr, beta1=cfg.beta1,
                        beta2=cfg.beta2, eps=cfg.eps, momentum=cfg.momentum, init_scale=cfg.init_scale,
                        growth_interval=cfg.growth_interval)
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(_threads()) as ex:
        ws = list(ex.map(lambda l: synth.weights(cfg, l), range(L)))
        xh = list(ex.map(lambda l: None if chained[l] else synth.activations(cfg, l, 0), range(L)))
        gh = list(ex.map(lambda l: None if cfg.feeds_next(l) else synth.upstream(cfg, l, 0), range(L)))
    for l, w in enumerate(ws):
        stack.load_weights(l, torch.from_numpy(w).cuda(),
                           torch.from_numpy(synth.fp16_bits(w).view(np.float16).reshape(w.shape)).cuda())
    del ws
    xs = []
    for l, x in enumerate(xh):
        if x is None:
            xs.append(None)
            continue
        buf = torch.zeros(x.shape[0], _pad8(x.shape[1]), dtype=torch.float16, device="cuda")
        buf[:, :x.shape[1]] = torch.from_numpy(x.view(np.float16)).cuda()
        xs.append(buf)
    # the FP32 gradients entering the top layers arrive as slices of one flat buffer
    tops = [l for l in range(L) if not cfg.feeds_next(l)]
    g_flat = torch.empty(sum(cfg.shapes[l][0] * cfg.shapes[l][2] for l in tops), device="cuda")
    gs, o = [None] * L, 0
    for l in tops:
        m, _, n = cfg.shapes[l]
        gs[l] = g_flat[o:o + m * n].view(m, n)
        gs[l].copy_(torch.from_numpy(gh[l]))
        o += m * n
    return stack, xs, gs, xh, gh


def _update_check_streamed(orc, cfg, stack, pre, S, t_applied, chunk=1 << 23):
    """The oracle's update fed with the GPU's own FP16 gradient and prior state, chunk by chunk
    over the whole flat range: FP32 master within 1e-6, FP16 copy bitwise rn16 of the GPU master."""
    w_pre, m_pre, v_pre = pre
    total = stack.total
    same = 0
    for lo in range(0, total, chunk):
        hi = min(total, lo + chunk)
        g16 = np.ascontiguousarray(_bits(stack.dw_flat[lo:hi]))
        w = w_pre[lo:hi].cpu().numpy().copy(); m = m_pre[lo:hi].cpu().numpy().copy()
        w16 = np.zeros(hi - lo, np.uint16)
        if cfg.optimizer == "adam":
            v = v_pre[lo:hi].cpu().numpy().copy()
            orc.adam_update(g16, w, m, v, w16, S, cfg.lr, cfg.beta1, cfg.beta2, cfg.eps, t_applied)
            vg = stack.v_flat[lo:hi].cpu().numpy()
            assert (np.abs(vg - v) <= 1e-6 * np.maximum(np.abs(v), 1e-12)).all()
        else:
            orc.momentum_update(g16, w, m, w16, S, cfg.lr, cfg.momentum)
        wg = stack.w32_flat[lo:hi].cpu().numpy()
        mg = stack.m_flat[lo:hi].cpu().numpy()
        assert (np.abs(wg - w) <= 1e-6 * np.maximum(np.abs(w), cfg.lr)).all()
        assert (np.abs(mg - m) <= 1e-6 * np.maximum(np.abs(m), 1e-12)).all()
        assert (_bits(stack.w16_flat[lo:hi]) == orc.f2h(wg)).all()
        same += int((wg.view(np.uint32) == w.view(np.uint32)).sum())
    return same / total


@pytest.mark.parametrize("name,max_steps,want_applied", [("c2", 5, 2), ("c3", 9, 2), ("c4", 11, 2)])
def test_full_step(orc, mp, name, max_steps, want_applied):
    """Steps of the full-size workload, the first launched call by call, the rest replayed from the
    CUDA graph, until `want_applied` steps have been applied (the configured initial loss scale
    overflows at first on c2 and c4, so their first steps are skipped ones; c3 gets a planted inf
    after its applied steps).  Every step: the flag against an
    independent scan of the stored weight gradients, scale and counters bit-exact against the
    scalar oracle, a skipped step leaves everything bitwise unchanged, an applied step's update
    is checked over the whole parameter range.  On the first step and on every applied step all
    products of all layers are checked on >= 10^4 sampled outputs per layer."""
    cfg = synth.config(name)
    L = len(cfg.shapes)
    stack, xs, gs, xh, gh = _build_like_bench(mp, cfg)
    assert any(len(g) > 1 for g in stack.groups) == (name in ("c2", "c3"))     # grouped launches in play
    sc = orc.Scaler(cfg.init_scale, cfg.growth_interval)
    applied = skipped = 0
    identical = []
    planted = None
    for step in range(max_steps + 1):
        if applied >= want_applied:
            if skipped >= 1:
                break
            # no natural overflow at this workload's initial scale: plant one non-finite value in
            # the gradient entering the last top layer, so that the skip runs at full size too
            planted = [l for l in range(L) if not cfg.feeds_next(l)][-1]
            gs[planted][0, 0] = float("inf")
        pre = (stack.w32_flat.clone(), stack.m_flat.clone(),
               stack.v_flat.clone() if stack.v_flat is not None else None)
        w16_pre = stack.w16_flat.clone()
        t_pre = stack.state.read().t
        S = sc.S
        if step == 0:
            stack.step(xs, gs)                              # call by call (also the library's one-time set-up)
        else:
            if stack.graph is None:
                stack.capture(xs, gs, warmup=0)             # recorded, not run
            stack.replay()
        torch.cuda.synchronize()
        assert mp.mp_gemm_device_status() == 0
        log = stack.state.read_log(1)[0]
        h = stack.state.read()
        # (1) the flag = an independent scan of every stored weight gradient
        dw_bits = stack.dw_flat.view(torch.int16)
        scan = int(bool(((dw_bits & 0x7C00) == 0x7C00).any()))
        assert log.found_inf == scan, step
        if step == 0:
            assert orc.found_inf(np.ascontiguousarray(_bits(stack.dw_flat))) == scan
        # (2) scale and counters against the scalar oracle, bit for bit
        sc.update(scan)
        assert (log.scale_before, log.scale_after) == (S, sc.S), step
        assert (h.scale, h.t, h.skipped, h.good_steps, h.status) == (sc.S, sc.t, sc.skipped, sc.good, 0)
        # (3) products on sampled outputs, forced operands
        if step == 0 or not scan:
            w16_host = _bits(w16_pre)
            for l, (M, K, N) in enumerate(cfg.shapes):
                ldw = stack.ldw[l]
                W = w16_host[stack.offsets[l]:stack.offsets[l] + K * ldw].reshape(K, ldw)[:, :N]
                W = np.ascontiguousarray(W)
                Xg, dYg = _bits(stack.X(l)), _bits(stack.dY(l))
                if not cfg.chained(l):
                    assert (Xg == xh[l]).all()
                if not cfg.feeds_next(l) and planted is None:   # upstream scaling: bitwise, whole tensor
                    assert (dYg == orc.scale_upstream(gh[l], S)).all()
                n = 3400
                same = [_check_product_samples(orc, "fwd", Xg, W, _bits(stack.Y(l)), n, 100 * l + step, f"Y{l} step {step}"),
                        _check_product_samples(orc, "wgrad", Xg, dYg, _bits(stack.dW(l)), n, 100 * l + step + 1, f"dW{l} step {step}"),
                        _check_product_samples(orc, "dgrad", dYg, W, _bits(stack.dX(l)), n, 100 * l + step + 2, f"dX{l} step {step}")]
                identical.append(min(same))
        # (4) the update
        if scan:
            skipped += 1
            assert h.t == t_pre
            assert torch.equal(stack.w32_flat.view(torch.int32), pre[0].view(torch.int32))
            assert torch.equal(stack.m_flat.view(torch.int32), pre[1].view(torch.int32))
            if pre[2] is not None:
                assert torch.equal(stack.v_flat.view(torch.int32), pre[2].view(torch.int32))
            assert torch.equal(stack.w16_flat.view(torch.int16), w16_pre.view(torch.int16))
        else:
            applied += 1
            frac = _update_check_streamed(orc, cfg, stack, pre, S, t_pre + 1)
            assert frac > 0.99, frac                        # nearly every FP32 word bitwise equal
        del pre, w16_pre
        if planted is not None:
            assert scan == 1
            break
    assert applied >= want_applied, (applied, skipped)
    assert skipped >= 1                                      # the halving path ran at full size too
    assert min(identical) > 0.9                              # most sampled outputs have identical bits
    stack.close()


def test_c2_long_run_loss_scale_trajectory(orc, mp):
    """2N + 1 = 2001 graph replays of the full-size c2 step (growth interval N = 1000): the flags
    the GPU logged, fed to the scalar oracle, give the scale sequence the GPU logged, bit for bit;
    the flags themselves are confirmed at sampled steps by an independent scan of the weight
    gradients that step stored.  The run crosses a doubling after 1000 clean steps."""
    cfg = synth.config("c2")
    stack, xs, gs, _, _ = _build_like_bench(mp, cfg)
    stack.step(xs, gs)
    stack.capture(xs, gs, warmup=0)
    total = 2 * cfg.growth_interval + 1
    sampled = sorted({1, 2, 3, 500, 999, 1000, 1001, 1002, 1003, 1004, 1005, 1500, total - 1})
    scans = {}
    done = 1
    torch.cuda.synchronize()
    scans[0] = int(bool(((stack.dw_flat.view(torch.int16) & 0x7C00) == 0x7C00).any()))
    for stop in sampled:
        for _ in range(stop + 1 - done):
            stack.replay()
        done = stop + 1
        torch.cuda.synchronize()
        scans[stop] = int(bool(((stack.dw_flat.view(torch.int16) & 0x7C00) == 0x7C00).any()))
    assert done == total and mp.mp_gemm_device_status() == 0
    log = stack.state.read_log()
    assert len(log) == total and [r.step for r in log] == list(range(total))
    sc = orc.Scaler(cfg.init_scale, cfg.growth_interval)
    for r in log:
        assert r.scale_before == sc.S, r.step
        sc.update(r.found_inf)
        assert (r.scale_after, r.t, r.good_steps) == (sc.S, sc.t, sc.good), r.step
    for step, flag in scans.items():
        assert log[step].found_inf == flag, step
    h = stack.state.read()
    assert (h.scale, h.t, h.skipped, h.step) == (sc.S, sc.t, sc.skipped, total)
    scales = [r.scale_after for r in log]
    assert max(scales[1:]) > min(scales) and sc.skipped >= 1            # a halving and a doubling happened
    assert any(b > a for a, b in zip(scales, scales[1:]))
    stack.close()
