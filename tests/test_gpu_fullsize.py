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
    big = fin & (np.abs(w) >= 1e-3 * rms)
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
