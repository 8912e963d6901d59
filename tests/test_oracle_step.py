"""Invariants the method fixes, checked on the oracle's whole step (tiny workload)."""
import copy
import os

import numpy as np

from paper_1805_10387_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _build(orc, cfg, init_scale=None, interval=None):
    layers = [orc.make_layer(synth.weights(cfg, l), cfg.optimizer, cfg.chained(l))
              for l in range(len(cfg.shapes))]
    sc = orc.Scaler(init_scale or cfg.init_scale, interval or cfg.growth_interval)
    opt = orc.Optim(kind=cfg.optimizer, lr=cfg.lr, beta1=cfg.beta1, beta2=cfg.beta2, eps=cfg.eps,
                    momentum=cfg.momentum)
    return layers, sc, opt


def _inputs(cfg, step):
    L = len(cfg.shapes)
    xs = [None if cfg.chained(l) else synth.activations(cfg, l, step) for l in range(L)]
    gs = [None if cfg.feeds_next(l) else synth.upstream(cfg, l, step) for l in range(L)]
    return xs, gs


def _snapshot(layers):
    return [(ly.w32.copy(), ly.m.copy(), None if ly.v is None else ly.v.copy(), ly.w16.copy())
            for ly in layers]


def _same(a, b):
    return all((x is None and y is None) or (x.view(np.uint8) == y.view(np.uint8)).all()
               for la, lb in zip(a, b) for x, y in zip(la, lb))


def test_c1_flags_skip_and_scale_trajectory(orc):
    cfg = synth.config("c1")
    layers, sc, opt = _build(orc, cfg)
    gold = [tuple(int(v) for v in l.split()) for l in open(os.path.join(GOLD, "scaler_c1_trajectory.txt"))
            if l.strip() and not l.startswith("#")]
    for step, flag, log2s in gold:
        before = _snapshot(layers)
        t_before = sc.t
        rec = orc.train_step(layers, *_inputs(cfg, step), sc, opt)
        assert rec.found_inf == flag, step
        assert rec.S_after == 2.0 ** log2s, step
        if flag:                                  # overflow step: state bitwise unchanged
            assert _same(before, _snapshot(layers)) and sc.t == t_before
        else:
            assert not _same(before, _snapshot(layers)) and sc.t == t_before + 1
        for ly in layers:                         # working copy is the rounded master
            assert (ly.w16 == orc.f2h(ly.w32)).all()
    assert sc.skipped == 1 and sc.t == 9


def test_master_trajectory_matches_a_library_adam_fed_the_same_gradients(orc):
    """The step driver's bookkeeping around the optimizer: the bias-correction count is the number of
    APPLIED steps including the current one (first applied step: 1) and does not advance on a skipped
    step.  A library Adam in float64 (an independent implementation) is stepped with the gradients the
    oracle's step produced, unscaled, on applied steps only; the masters must follow it."""
    import torch
    cfg = synth.config("c1")
    layers, sc, opt = _build(orc, cfg)
    params = [torch.tensor(ly.w32.astype(np.float64), requires_grad=True) for ly in layers]
    ref = torch.optim.Adam(params, lr=cfg.lr, betas=(cfg.beta1, cfg.beta2), eps=cfg.eps)
    applied = 0
    for step in range(8):                               # the inf arrives at step index 4
        rec = orc.train_step(layers, *_inputs(cfg, step), sc, opt)
        if rec.found_inf:
            continue
        applied += 1
        for p, ly in zip(params, layers):
            p.grad = torch.tensor(orc.h2f(ly.dW).astype(np.float64) / rec.S_before)
        ref.step()
        for p, ly in zip(params, layers):
            want = p.detach().numpy()
            assert np.abs(ly.w32 - want).max() <= 2e-6 * max(1.0, np.abs(want).max()), step
    assert applied == 7 and sc.t == 7 and sc.skipped == 1


def _dyadic_inputs(cfg, step):
    """Inputs on a dyadic grid: X integers in -2..2, upstream gradients multiples of 2^-5 in
    [-1/4, 1/4].  With weights on a 2^-4 grid every product sum is a multiple of 2^-9, so no
    nonzero value of the S = 1 run is subnormal in FP16."""
    rng = np.random.default_rng(100 + step)
    L = len(cfg.shapes)
    xs = [None if cfg.chained(l) else
          synth.fp16_bits(rng.integers(-2, 3, cfg.shapes[l][:2]).astype(np.float32)) for l in range(L)]
    gs = [None if cfg.feeds_next(l) else
          (rng.integers(-8, 9, (cfg.shapes[l][0], cfg.shapes[l][2])) / 32.0).astype(np.float32)
          for l in range(L)]
    return xs, gs


def test_power_of_two_scale_invariance(orc):
    """With S a power of two and no overflow or underflow, the gradients after unscaling, and
    so the whole updated state, are bitwise those of the unscaled loss (S = 1)."""
    cfg = synth.config("c1")
    rng = np.random.default_rng(1)
    w_init = [(rng.integers(-4, 5, (k, n)) / 16.0).astype(np.float32) for _, k, n in cfg.shapes]
    ref = None
    for k in (0, 1, 5, 8):
        layers = [orc.make_layer(w_init[l], "adam", cfg.chained(l)) for l in range(2)]
        sc = orc.Scaler(2.0 ** k, 10 ** 6)
        rec = orc.train_step(layers, *_dyadic_inputs(cfg, 0), sc, orc.Optim(lr=2.0 ** -10))
        assert rec.found_inf == 0
        grads = []
        for ly in layers:
            for arr in (ly.dY, ly.dX, ly.dW):             # the premise, checked
                e = (arr >> 10) & 0x1F
                assert (e[(arr & 0x7FFF) != 0] > 0).all() and (e < 0x1F).all()
            grads.append(orc.h2f(ly.dW) * np.float32(2.0 ** -k))
        snap = _snapshot(layers)
        if ref is None:
            ref = (grads, snap)
        else:
            assert all((a == b).all() for a, b in zip(ref[0], grads)), k
            assert _same(ref[1], snap), k


def test_static_scale_still_skips_overflow(orc):
    cfg = synth.config("c1")
    layers = [orc.make_layer(synth.weights(cfg, l), "adam", cfg.chained(l)) for l in range(2)]
    sc = orc.Scaler(init_scale=10.0, interval=4, dynamic=False)
    opt = orc.Optim()
    for step in range(6):
        before = _snapshot(layers)
        rec = orc.train_step(layers, *_inputs(cfg, step), sc, opt)
        assert rec.S_after == 10.0
        assert _same(before, _snapshot(layers)) == (step == cfg.inject_inf_step)


def test_natural_overflow_halves_until_it_fits(orc):
    """No injected value: a scale far too large overflows the FP16 gradients by itself, each
    such step is skipped and halves S, and the first clean step applies."""
    cfg = synth.config("c1")
    cfg.inject_inf_step = -1
    cfg.grad_std = 1.0
    layers, sc, opt = _build(orc, cfg, init_scale=2.0 ** 16, interval=1000)
    seen_clean = False
    for step in range(12):
        before = _snapshot(layers)
        rec = orc.train_step(layers, *_inputs(cfg, step), sc, opt)
        if rec.found_inf:
            assert not seen_clean and rec.S_after == rec.S_before / 2
            assert _same(before, _snapshot(layers))
        else:
            seen_clean = True
    assert seen_clean and sc.skipped >= 2


def test_relu_stack_equals_plain_stack_when_nothing_is_clipped(orc):
    """If every pre-activation is positive and no bias is present, a ReLU stack is the plain
    stack: outputs, gradients and updated state agree bit for bit; with biases of zero too."""
    rng = np.random.default_rng(12)
    M, K = 16, 24
    w = [np.abs(rng.standard_normal((K, K))).astype(np.float32) / K for _ in range(3)]
    x = synth.fp16_bits(np.abs(rng.standard_normal((M, K))).astype(np.float32))
    g = (rng.standard_normal((M, K)) * 0.01).astype(np.float32)

    def run(acts, bias):
        layers = [orc.make_layer(w[l], "adam", l > 0, acts[l], 20.0,
                                 np.zeros(K, np.float32) if bias else None) for l in range(3)]
        sc = orc.Scaler(256.0, 100)
        rec = orc.train_step(layers, [x, None, None], [None, None, g], sc, orc.Optim())
        return layers, rec
    plain, r0 = run(["none"] * 3, False)
    relu, r1 = run(["relu", "relu", "none"], False)
    relub, r2 = run(["relu", "clipped_relu", "none"], True)
    assert r0.found_inf == r1.found_inf == r2.found_inf == 0
    for a, b, c in zip(plain, relu, relub):
        for name in ("Y", "dY", "dX", "dW", "w32", "w16"):
            assert (getattr(a, name).view(np.uint8) == getattr(b, name).view(np.uint8)).all(), name
            assert (getattr(a, name).view(np.uint8) == getattr(c, name).view(np.uint8)).all(), name
    # the bias gradient is the column sum of the gradient at the pre-activation
    for ly in relub:
        assert (ly.db == orc.bias_grad(ly.dY)).all() and (ly.b16 == orc.f2h(ly.b32)).all()
        assert (ly.b32 != 0).any()                       # Adam moved the biases


def test_activation_gradient_is_taken_from_the_stored_output(orc):
    """Two-layer ReLU stack: rows of the hidden output that are zero get no gradient through
    the first layer, whatever the upstream gradient."""
    rng = np.random.default_rng(13)
    M, K = 12, 16
    w0 = rng.standard_normal((K, K)).astype(np.float32) / 4
    w1 = rng.standard_normal((K, K)).astype(np.float32) / 4
    layers = [orc.make_layer(w0, "adam", False, "relu"), orc.make_layer(w1, "adam", True, "none")]
    x = synth.fp16_bits(rng.standard_normal((M, K)).astype(np.float32))
    g = rng.standard_normal((M, K)).astype(np.float32)
    w1_used = layers[1].w16.copy()                     # the step rewrites the working copy
    orc.train_step(layers, [x, None], [None, g], orc.Scaler(4.0, 100), orc.Optim())
    hidden = layers[0].Y.view(np.float16).astype(np.float32)
    assert (hidden >= 0).all() and (hidden == 0).any() and (hidden > 0).any()
    assert (layers[0].dY[hidden == 0] == 0).all()
    full = orc.linear_bwd_dgrad(layers[1].dY, w1_used)
    assert (layers[0].dY[hidden > 0] == full[hidden > 0]).all()
