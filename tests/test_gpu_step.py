"""The whole step on the GPU (five C-ABI calls per layer stack) against the oracle's step."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1805_10387_b200 import synth  # noqa: E402


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _f(bits):
    return bits.view(np.float16).astype(np.float64)


def _h16(x):
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def _pad_dev(bits):
    r, c = bits.shape
    buf = torch.zeros(r, (c + 7) // 8 * 8, dtype=torch.float16, device="cuda")
    buf[:, :c] = torch.from_numpy(bits.view(np.float16)).cuda()
    return buf


ACT_NAMES = {0: "none", 1: "relu", 2: "clipped_relu"}


def build_both(orc, cfg, dynamic=True, acts=None, bias=False, clip=20.0):
    from paper_1805_10387_b200.stack import LinearStack
    L = len(cfg.shapes)
    chained = [cfg.chained(l) for l in range(L)]
    acts = acts or [0] * L
    gpu = LinearStack(cfg.shapes, chained, optimizer=cfg.optimizer, lr=cfg.lr, beta1=cfg.beta1,
                      beta2=cfg.beta2, eps=cfg.eps, momentum=cfg.momentum,
                      init_scale=cfg.init_scale, growth_interval=cfg.growth_interval, dynamic=dynamic,
                      acts=acts, bias=bias, clip=clip)
    layers = []
    for l in range(L):
        w = synth.weights(cfg, l)
        b = (synth.normal(cfg.seed, 9000 + l, cfg.shapes[l][2]) * 0.1).astype(np.float32) if bias else None
        ly = orc.make_layer(w, cfg.optimizer, chained[l], ACT_NAMES[acts[l]], clip, b)
        layers.append(ly)
        h16 = lambda a: torch.from_numpy(synth.fp16_bits(a).view(np.float16).reshape(a.shape)).cuda()
        gpu.load_weights(l, torch.from_numpy(w).cuda(), h16(w),
                         torch.from_numpy(b).cuda() if bias else None, h16(b) if bias else None)
        assert (synth.fp16_bits(w).reshape(w.shape) == ly.w16).all()
    sc = orc.Scaler(cfg.init_scale, cfg.growth_interval, dynamic=dynamic)
    opt = orc.Optim(kind=cfg.optimizer, lr=cfg.lr, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
                    momentum=cfg.momentum)
    return gpu, layers, sc, opt


def drift_ok(got_bits, want_bits, what, frac=1.0):
    """Free-running comparison: the two sides see inputs that may already differ by an FP16
    rounding (chained layers, updated weights), so the error is measured against the size of
    the tensor, not of each element."""
    g, w = _f(got_bits), _f(want_bits)
    fin = np.isfinite(w) & np.isfinite(g)
    assert (np.isfinite(w) == np.isfinite(g)).mean() > 0.9999, what
    if fin.any():
        rms = np.sqrt((w[fin] ** 2).mean())
        err = np.abs(g[fin] - w[fin])
        ok = err <= 1e-2 * np.abs(w[fin]) + 2e-2 * rms + 2.0 ** -24
        # with activations a value next to zero can fall on either side of the mask in the two
        # free-running copies, which moves a few elements by more than a rounding
        assert ok.mean() >= frac, (what, err.max(), rms, ok.mean())


def forced_ok(orc, op, A_bits, B_bits, got_bits, what):
    """The oracle's product of the very operands the GPU kernel read: bounded by one FP16
    rounding plus FP32 summation-order error, and max relative error 1e-2 where not tiny."""
    A = np.ascontiguousarray(A_bits); B = np.ascontiguousarray(B_bits)
    want = {"fwd": orc.linear_fwd, "dgrad": orc.linear_bwd_dgrad, "wgrad": orc.linear_bwd_wgrad}[op](A, B)
    ex, ab = orc.linear_exact(op, A, B)
    red = {"fwd": A.shape[1], "dgrad": A.shape[1], "wgrad": A.shape[0]}[op]
    g, w = _f(got_bits), _f(want)
    fin = np.isfinite(ex) & (np.abs(ex) < 65000.0)
    tol = 2.0 ** -10 * np.abs(ex) + red * 2.0 ** -24 * ab + 2.0 ** -24
    assert (np.abs(g - ex)[fin] <= tol[fin]).all(), what
    inf_w = ~np.isfinite(w)
    assert (np.isfinite(g) == np.isfinite(w))[~fin | inf_w].mean() > 0.99 if (~fin | inf_w).any() else True
    both = np.isfinite(w) & np.isfinite(g)
    if both.any():
        rms = np.sqrt((w[both] ** 2).mean())
        big = both & (np.abs(w) >= 1e-3 * rms) & (np.abs(w) > 2.0 ** -14)
        if big.any():
            assert (np.abs(g[big] - w[big]) / np.abs(w[big])).max() <= 1e-2, what


def run_config(orc, mp, cfg, steps, dynamic=True, acts=None, bias=False, clip=20.0):
    gpu, layers, sc, opt = build_both(orc, cfg, dynamic, acts, bias, clip)
    acts = acts or [0] * len(cfg.shapes)
    L = len(cfg.shapes)
    records = []
    for step in range(steps):
        xs = [None if cfg.chained(l) else synth.activations(cfg, l, step) for l in range(L)]
        gs = [None if cfg.feeds_next(l) else synth.upstream(cfg, l, step) for l in range(L)]
        dxs = [None if x is None else _pad_dev(x) for x in xs]
        dgs = [None if g is None else torch.from_numpy(g).cuda() for g in gs]
        # state of the GPU before the step, for the checks that reuse the GPU's own operands
        pre = [(gpu.W32(l).cpu().numpy().copy(), gpu.m[l][:, :cfg.shapes[l][2]].cpu().numpy().copy(),
                None if gpu.v is None else gpu.v[l][:, :cfg.shapes[l][2]].cpu().numpy().copy())
               for l in range(L)]
        w16_pre = [_bits(gpu.W16(l)) for l in range(L)]
        b16_pre = [_bits(gpu.b16[l]) if bias else None for l in range(L)]
        t_pre = gpu.state.read().t
        gpu.step(dxs, dgs)
        rec = orc.train_step(layers, xs, gs, sc, opt)
        torch.cuda.synchronize()
        assert mp.mp_gemm_device_status() == 0
        h = gpu.state.read()
        log = gpu.state.read_log(1)[0]
        # flags, skip decision and scale: bit exact
        assert log.found_inf == rec.found_inf, step
        assert (log.scale_before, log.scale_after) == (rec.S_before, rec.S_after), step
        assert (h.t, h.good_steps, h.skipped) == (sc.t, sc.good, sc.skipped)
        records.append(rec)
        for l in range(L):
            Xg, Yg, dYg = _bits(gpu.X(l)), _bits(gpu.Y(l)), _bits(gpu.dY(l))
            dXg, dWg = _bits(gpu.dX(l)), _bits(gpu.dW(l))
            if acts[l] == 0 and not bias:
                forced_ok(orc, "fwd", Xg, w16_pre[l], Yg, f"Y{l} step {step}")
            else:       # the oracle's activated product of the operands the GPU read
                want = orc.linear_fwd_act(np.ascontiguousarray(Xg), np.ascontiguousarray(w16_pre[l]),
                                          np.ascontiguousarray(b16_pre[l]) if bias else None,
                                          ACT_NAMES[acts[l]], clip)
                wf, gf = _f(want), _f(Yg)
                assert (np.abs(gf - wf) <= 2.0 ** -9 * np.abs(wf) + 2e-3 * np.sqrt((wf * wf).mean()) + 1e-6).all()
                assert (Yg == want).mean() > 0.97
            forced_ok(orc, "wgrad", Xg, dYg, dWg, f"dW{l} step {step}")
            below = acts[l - 1] if cfg.chained(l) else 0
            if below == 0:
                forced_ok(orc, "dgrad", dYg, w16_pre[l], dXg, f"dX{l} step {step}")
            else:
                want = orc.linear_bwd_dgrad_act(np.ascontiguousarray(dYg), np.ascontiguousarray(w16_pre[l]),
                                                np.ascontiguousarray(Xg), ACT_NAMES[below], clip)
                assert ((dXg == 0) == (want == 0)).mean() > 0.999          # same mask
                wf, gf = _f(want), _f(dXg)
                fin = np.isfinite(wf) & np.isfinite(gf)
                assert (np.abs(gf - wf)[fin] <= 2.0 ** -9 * np.abs(wf[fin]) + 2e-3 * np.sqrt((wf[fin] ** 2).mean()) + 1e-7).all()
            if bias:
                dbg = _bits(gpu.db[l])
                want = orc.bias_grad(np.ascontiguousarray(dYg))
                wf, gf = _f(want), _f(dbg)
                fin = np.isfinite(wf)
                assert (np.isfinite(gf) == fin).all()
                assert (np.abs(gf - wf)[fin] <= 2.0 ** -9 * np.abs(wf[fin]) + 1e-3 * np.abs(_f(dYg)).sum(axis=0)[fin] * 2.0 ** -10 + 1e-7).all()
            if not cfg.feeds_next(l):              # upstream scaling: bitwise
                assert (dYg == orc.scale_upstream(gs[l], rec.S_before)).all()
            frac = 1.0 if not any(acts) else 0.98
            drift_ok(Yg, layers[l].Y, f"Y{l} step {step}", frac)
            drift_ok(dXg, layers[l].dX, f"dX{l} step {step}", frac)
            drift_ok(dWg, layers[l].dW, f"dW{l} step {step}", frac)
            w_gpu = gpu.W32(l).cpu().numpy()
            if rec.found_inf:                       # skipped: bitwise unchanged
                assert (w_gpu.view(np.uint32) == pre[l][0].view(np.uint32)).all()
                assert (_bits(gpu.W16(l)) == w16_pre[l]).all()
                assert h.t == t_pre
            else:
                # free-running oracle: its gradients may differ by an FP16 rounding, and Adam
                # turns a sign flip of a near-zero gradient into a full step of size lr
                diff = np.abs(w_gpu - layers[l].w32)
                assert diff.max() <= 2.5 * cfg.lr * (h.t if cfg.optimizer == "adam" else 1) + 1e-7
                assert np.median(diff) <= 1e-6
                # the oracle's update fed with the GPU's own FP16 gradient and prior state
                w, m, v = pre[l]
                w16 = np.zeros(w.shape, np.uint16)
                g16 = np.ascontiguousarray(dWg)
                if cfg.optimizer == "adam":
                    orc.adam_update(g16, w, m, v, w16, rec.S_before, cfg.lr, cfg.beta1, cfg.beta2,
                                    cfg.eps, t_pre + 1)
                else:
                    orc.momentum_update(g16, w, m, w16, rec.S_before, cfg.lr, cfg.momentum)
                assert (np.abs(w_gpu - w) <= 1e-6 * np.maximum(np.abs(w), cfg.lr)).all()
                assert (_bits(gpu.W16(l)) == orc.f2h(w_gpu)).all()
    gpu.close()
    return records


def test_c1_ten_steps_with_injected_inf(orc, mp):
    cfg = synth.config("c1")
    recs = run_config(orc, mp, cfg, cfg.steps)
    assert [r.found_inf for r in recs] == [0, 0, 0, 0, 1, 0, 0, 0, 0, 0]
    assert [np.log2(r.S_after) for r in recs] == [16, 16, 16, 17, 16, 16, 16, 16, 17, 17]


def test_static_loss_scale_that_is_not_a_power_of_two(orc, mp):
    """Static loss scaling with the value of the paper's configuration listing (10.0): S never
    changes, the unscale is a multiply by fl32(1/10), the step with the injected inf is still
    skipped, and everything matches the oracle as in the dynamic case."""
    cfg = synth.config("c1")
    cfg.init_scale = 10.0
    recs = run_config(orc, mp, cfg, 7, dynamic=False)
    assert [r.found_inf for r in recs] == [0, 0, 0, 0, 1, 0, 0]
    assert all(r.S_before == 10.0 and r.S_after == 10.0 for r in recs)


@pytest.mark.parametrize("name,rows,shapes", [
    ("c2", 320, [(320, 264, 520)] * 3),                               # unchained gate-GEMM layers
    ("c3", 384, [(384, 136, 520), (384, 520, 136), (384, 136, 136), (384, 136, 136)]),  # FFN pair chained
    ("c4", 512, [(512, 200, 200)] * 2 + [(512, 200, 29)]),            # chained, momentum, narrow top
])
def test_scaled_down_workloads(orc, mp, name, rows, shapes):
    """The c2-c4 recipes with widths shrunk so that the oracle finishes in seconds: same value
    distributions, optimizer and scaler; several tiles and ragged tails per product."""
    cfg = synth.config(name)
    cfg.shapes = shapes
    cfg.chain = cfg.chain[:len(shapes)]
    cfg.growth_interval = 2
    recs = run_config(orc, mp, cfg, 4)
    assert len(recs) == 4


def test_graph_replay_equals_call_by_call(orc, mp):
    """The step captured once as a CUDA graph and replayed must leave bit-for-bit the state that
    the same steps launched call by call leave, including an overflow step (skip + halving),
    because flag, scale and step count never leave the device."""
    from paper_1805_10387_b200.stack import LinearStack
    cfg = synth.config("c1")
    L = len(cfg.shapes)
    chained = [cfg.chained(l) for l in range(L)]

    def make():
        st = LinearStack(cfg.shapes, chained, lr=cfg.lr, init_scale=cfg.init_scale, growth_interval=3)
        for l in range(L):
            w = synth.weights(cfg, l)
            st.load_weights(l, torch.from_numpy(w).cuda(),
                            torch.from_numpy(synth.fp16_bits(w).view(np.float16).reshape(w.shape)).cuda())
        return st
    a, b = make(), make()
    x = _pad_dev(synth.activations(cfg, 0, 0))
    g = torch.from_numpy(synth.upstream(cfg, 1, 0)).cuda()
    xs, gs = [x, None], [None, g]
    steps = 9
    b.capture(xs, gs, warmup=2)                      # two real steps, then the recording
    for _ in range(2):
        a.step(xs, gs)
    for s in range(steps):
        if s == 4:
            g[0, 0] = float("inf")                   # replayed graph reads the tensor as it is now
        if s == 5:
            g[0, 0] = 0.0
        a.step(xs, gs)
        b.replay()
    torch.cuda.synchronize()
    ha, hb = a.state.read(), b.state.read()
    assert (ha.scale, ha.t, ha.skipped, ha.step, ha.good_steps) == (hb.scale, hb.t, hb.skipped, hb.step, hb.good_steps)
    assert ha.skipped >= 1 and ha.step == steps + 2
    assert [r.found_inf for r in a.state.read_log()] == [r.found_inf for r in b.state.read_log()]
    for fa, fb in ((a.w32_flat, b.w32_flat), (a.m_flat, b.m_flat), (a.v_flat, b.v_flat)):
        assert torch.equal(fa.view(torch.int32), fb.view(torch.int32))
    assert torch.equal(a.w16_flat.view(torch.int16), b.w16_flat.view(torch.int16))
    a.close(); b.close()


def test_one_scaling_call_over_a_flat_gradient_buffer(orc, mp):
    """When the FP32 gradients entering the top layers are consecutive slices of one buffer the
    stack scales them with one call; the scaled gradients and the state after the steps are
    bit-for-bit those of one call per layer, with fewer launches."""
    from paper_1805_10387_b200.stack import LinearStack
    shapes = [(96, 64, 40), (96, 40, 72), (96, 64, 72)]      # three independent layers
    chained = [False, False, False]
    rng = np.random.default_rng(11)
    ws = [rng.standard_normal((k, n)).astype(np.float32) / np.sqrt(k) for _, k, n in shapes]

    def make():
        st = LinearStack(shapes, chained, lr=1e-3, init_scale=1024.0, growth_interval=2)
        for l, w in enumerate(ws):
            st.load_weights(l, torch.from_numpy(w).cuda(), torch.from_numpy(w).cuda().half())
        return st
    a, b = make(), make()
    xs = [torch.from_numpy(rng.standard_normal((m, k)).astype(np.float32)).cuda().half() for m, k, _ in shapes]
    g_sep = [torch.from_numpy((rng.standard_normal((m, n)) * 1e-3).astype(np.float32)).cuda() for m, _, n in shapes]
    flat = torch.cat([g.reshape(-1) for g in g_sep])
    g_flat, o = [], 0
    for m, _, n in shapes:
        g_flat.append(flat[o:o + m * n].view(m, n)); o += m * n
    assert a._flat_upstream(g_sep) is None and b._flat_upstream(g_flat) is not None
    n0 = mp.mp_kernel_launch_count()
    for _ in range(3):
        a.step(xs, g_sep)
    n1 = mp.mp_kernel_launch_count()
    for _ in range(3):
        b.step(xs, g_flat)
    n2 = mp.mp_kernel_launch_count()
    torch.cuda.synchronize()
    assert (n1 - n0) - (n2 - n1) == 3 * (len(shapes) - 1)
    for l in range(len(shapes)):
        assert torch.equal(a.dY(l).contiguous().view(torch.int16), b.dY(l).contiguous().view(torch.int16))
    for fa, fb in ((a.w32_flat, b.w32_flat), (a.m_flat, b.m_flat), (a.v_flat, b.v_flat)):
        assert torch.equal(fa.view(torch.int32), fb.view(torch.int32))
    assert a.state.read().scale == b.state.read().scale
    a.close(); b.close()


def test_lstm_gate_layers(orc, mp):
    """Two independent LSTM gate layers (grouped products, cell kernels wired into the step):
    every stage of the step is checked against the oracle applied to the operands the GPU stage
    read -- gate product, cell forward, scaling, cell backward, weight and data gradients."""
    from paper_1805_10387_b200.stack import LinearStack
    M, K, H = 96, 64, 32
    shapes = [(M, K, 4 * H)] * 2
    rng = np.random.default_rng(21)
    ws = [rng.standard_normal((K, 4 * H)).astype(np.float32) / np.sqrt(K) for _ in shapes]
    st = LinearStack(shapes, [False, False], lr=1e-3, init_scale=256.0, growth_interval=1000, lstm=[True, True])
    assert st.groups == [[0, 1]]
    for l, w in enumerate(ws):
        st.load_weights(l, torch.from_numpy(w).cuda(), torch.from_numpy(w).cuda().half())
        st.c_prev[l].copy_(torch.from_numpy(rng.standard_normal((M, H)).astype(np.float32)).cuda().half())
    xs = [torch.from_numpy(rng.standard_normal((M, K)).astype(np.float32)).cuda().half() for _ in shapes]
    gs = [torch.from_numpy((rng.standard_normal((M, H)) * 1e-2).astype(np.float32)).cuda() for _ in shapes]

    def close(got_bits, want_bits, what, scale=None):
        g, w = _f(got_bits), _f(want_bits)
        tol = 2.0 ** -10 * np.abs(w) + 2.0 ** -24
        if scale is not None:
            tol = tol + 1e-5 * np.tile(scale, (1, w.shape[1] // scale.shape[1]))
        assert (np.abs(g - w) <= tol).all(), what
    for step in range(2):
        w16 = [_bits(st.W16(l)) for l in range(2)]        # the weights this step's products read
        st.step(xs, gs)
        torch.cuda.synchronize()
        for l in range(2):
            X = _bits(xs[l]); G = _bits(st.Y(l)); cp = _bits(st.c_prev[l])
            forced_ok(orc, "fwd", X, w16[l], G, ("gates", step, l))
            wc, wh = orc.lstm_cell_fwd(G, cp)
            close(_bits(st.c_new[l]), wc, ("c_new", step, l)); close(_bits(st.h[l]), wh, ("h", step, l))
            dh = _bits(st.dh[l])
            assert (dh == orc.scale_upstream(gs[l].cpu().numpy(), 256.0)).all()
            wG, wcp = orc.lstm_cell_bwd(G, cp, _bits(st.c_new[l]), dh, None)
            sc = np.abs(_f(dh))
            close(_bits(st.dY(l)), wG, ("dG", step, l), sc); close(_bits(st.dc_prev[l]), wcp, ("dc_prev", step, l), sc)
            forced_ok(orc, "wgrad", X, _bits(st.dY(l)), _bits(st.dW(l)), ("dW", step, l))
            forced_ok(orc, "dgrad", _bits(st.dY(l)), w16[l], _bits(st.dX(l)), ("dX", step, l))
    h = st.state.read()
    assert h.step == 2 and h.skipped == 0 and h.t == 2
    st.close()


def test_host_pipeline_equals_serial_host_steps(orc, mp):
    """Batches fed from pinned host memory through the double-buffered pipeline (copy of batch
    i+1 under the step of batch i, one CUDA graph per staging set) leave bit-for-bit the state
    of the same batches copied and stepped one after the other, overflow batch included."""
    from paper_1805_10387_b200.stack import LinearStack, HostPipeline
    cfg = synth.config("c1")
    L = len(cfg.shapes)
    chained = [cfg.chained(l) for l in range(L)]

    def make():
        st = LinearStack(cfg.shapes, chained, lr=cfg.lr, init_scale=cfg.init_scale, growth_interval=3)
        for l in range(L):
            w = synth.weights(cfg, l)
            st.load_weights(l, torch.from_numpy(w).cuda(),
                            torch.from_numpy(synth.fp16_bits(w).view(np.float16).reshape(w.shape)).cuda())
        return st
    a, b = make(), make()
    steps = 9
    batches = []
    for s in range(steps):
        x = torch.from_numpy(synth.activations(cfg, 0, s).view(np.float16)).pin_memory()
        g = synth.upstream(cfg, 1, s).copy()
        if s == 4:
            g[3, 5] = np.inf
        batches.append(([x, None], [None, torch.from_numpy(g).pin_memory()]))
    states_a = [a.step_from_host(xs, gs) for xs, gs in batches]          # serial, call by call
    pipe = HostPipeline(b, use_graph=True)
    states_b = []
    pipe.submit(*batches[0])
    for s in range(steps):
        if s + 1 < steps:
            pipe.submit(*batches[s + 1])
        states_b.append(pipe.run())
    key = lambda h: (h.scale, h.t, h.skipped, h.step, h.good_steps)
    assert [key(h) for h in states_a] == [key(h) for h in states_b]
    assert states_a[-1].skipped == 1 and states_a[-1].step == steps
    for fa, fb in ((a.w32_flat, b.w32_flat), (a.m_flat, b.m_flat), (a.v_flat, b.v_flat)):
        assert torch.equal(fa.view(torch.int32), fb.view(torch.int32))
    assert torch.equal(a.w16_flat.view(torch.int16), b.w16_flat.view(torch.int16))
    with pytest.raises(AssertionError):
        pipe.run()                                   # nothing submitted
    a.close(); b.close()


@pytest.mark.parametrize("name,shapes,acts,clip", [
    ("c3", [(384, 136, 520), (384, 520, 136), (384, 136, 136)], [1, 0, 0], 20.0),       # ReLU inside the FFN pair
    ("c4", [(512, 200, 200)] * 3 + [(512, 200, 29)], [2, 2, 2, 0], 20.0),              # clipped ReLU chain
])
def test_layers_with_bias_and_activation(orc, mp, name, shapes, acts, clip):
    """The scaled-down recipes as real layers: bias on every layer, ReLU between the FFN pair,
    clipped ReLU through the dense chain, bias gradients inspected and updated with the weights."""
    cfg = synth.config(name)
    cfg.shapes = shapes
    cfg.chain = cfg.chain[:len(shapes)]
    cfg.growth_interval = 2
    recs = run_config(orc, mp, cfg, 4, acts=acts, bias=True, clip=clip)
    assert len(recs) == 4


def test_weight_gradients_on_a_second_stream_change_nothing(orc, mp):
    """The stack issues its weight-gradient products on a second stream (beside the data gradients
    of the layers below).  Same kernels on the same operands: gradients, masters, moments, weights
    and the loss-scale state are bit for bit those of the one-stream order, eagerly and replayed
    from a CUDA graph, over steps that include a skipped one."""
    from paper_1805_10387_b200.stack import LinearStack
    shapes = [(384, 136, 520), (384, 520, 136), (384, 136, 136), (384, 136, 136)]   # chained pair + a group of two
    chain = [False, True, False, False]
    rng = np.random.default_rng(5)
    ws = [rng.standard_normal((k, n)).astype(np.float32) / np.sqrt(k) for _, k, n in shapes]

    def make(overlap):
        st = LinearStack(shapes, chain, lr=1e-3, init_scale=2.0 ** 10, growth_interval=2, bias=True,
                         acts=[mp.MP_ACT_RELU, 0, 0, 0], overlap_wgrad=overlap)
        for l, w in enumerate(ws):
            b = np.linspace(-0.1, 0.1, shapes[l][2]).astype(np.float32)
            st.load_weights(l, torch.from_numpy(w).cuda(), torch.from_numpy(w).cuda().half(),
                            torch.from_numpy(b).cuda(), torch.from_numpy(b).cuda().half())
        return st
    a, b, c = make(False), make(True), make(True)
    assert b.side is not None and a.side is None and len(b.groups) == 3
    xs = [_pad_dev(_h16(rng.standard_normal((m, k)))) if not chain[l] else None for l, (m, k, _) in enumerate(shapes)]
    gs = [None] + [torch.from_numpy((rng.standard_normal((m, n)) * 1e-2).astype(np.float32)).cuda()
                   for (m, _, n) in shapes[1:]]
    c.capture(xs, gs, warmup=0)
    for s in range(6):
        if s == 3:
            gs[2][0, 0] = float("inf")
        if s == 4:
            gs[2][0, 0] = 0.0
        a.step(xs, gs); b.step(xs, gs); c.replay()
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    ha = a.state.read()
    assert ha.skipped == 1 and ha.step == 6
    for o in (b, c):
        h = o.state.read()
        assert (h.scale, h.t, h.skipped, h.step, h.good_steps) == (ha.scale, ha.t, ha.skipped, ha.step, ha.good_steps)
        for fa, fo in ((a.w32_flat, o.w32_flat), (a.m_flat, o.m_flat), (a.v_flat, o.v_flat)):
            assert torch.equal(fa.view(torch.int32), fo.view(torch.int32))
        assert torch.equal(a.w16_flat.view(torch.int16), o.w16_flat.view(torch.int16))
        assert torch.equal(a.dw_flat.view(torch.int16), o.dw_flat.view(torch.int16))
    a.close(); b.close(); c.close()
