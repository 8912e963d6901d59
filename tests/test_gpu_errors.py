"""The library's reaction to a bounded device-side wait that runs out, exercised on a healthy GPU:
the self-test entry point launches one tile of the forward kernel whose loader fetches nothing,
so nothing is in flight, the waits expire after the given limit and the kernel returns."""
import time

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _operands(M, K, N, seed):
    rng = np.random.default_rng(seed)
    X = rng.integers(-2, 3, (M, K)).astype(np.float32).astype(np.float16)
    W = rng.integers(-2, 3, (K, N)).astype(np.float32).astype(np.float16)
    return X, W


def _small_update(mp):
    n = 5000
    g16 = torch.full((n,), 0.5, dtype=torch.float16, device="cuda")
    w32 = torch.linspace(-1, 1, n, device="cuda")
    m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    w16 = w32.half()
    plan = mp.UpdatePlan([g16], [w32], [m], [v], [w16])
    opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
    return plan, opt, (w32, m, v, w16)


@pytest.mark.parametrize("with_state", [True, False])
def test_expired_wait_is_reported_and_freezes_the_training_state(orc, mp, with_state):
    M, K, N = 96, 256, 200
    X, W = _operands(M, K, N, 3)
    Xd, Wd = torch.from_numpy(X).cuda(), torch.from_numpy(W).cuda()
    raw = torch.full((M + 4, N + 8), 0x5A5A, dtype=torch.int16, device="cuda")
    Y = raw.view(torch.float16)[2:2 + M, :N]
    st = mp.State(init_scale=1024.0, growth_interval=2)
    plan, opt, tensors = _small_update(mp)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0

    t0 = time.time()
    mp.mp_selftest_wait_timeout(Xd, Wd, Y, 200, st if with_state else None)     # 200 us limit
    torch.cuda.synchronize()
    assert time.time() - t0 < 2.0                       # the kernel came back by itself
    assert bool((raw == 0x5A5A).all())                  # and wrote nothing
    h = st.read()
    assert h.status == (mp.MP_ERR_TIMEOUT if with_state else 0)

    # frozen: the update writes nothing, the loss-scale call changes nothing but the status
    before = [t.clone() for t in tensors]
    mp.mp_master_update(plan, st, opt, 0)
    mp.mp_loss_scale_update(st)
    torch.cuda.synchronize()
    for a, b in zip(before, tensors):
        assert torch.equal(a.view(torch.int16 if a.dtype == torch.float16 else torch.int32),
                           b.view(torch.int16 if b.dtype == torch.float16 else torch.int32))
    h2 = st.read()
    assert h2.status == mp.MP_ERR_TIMEOUT               # copied from the device-wide word if need be
    assert (h2.step, h2.t, h2.scale, h2.good_steps, h2.skipped) == (h.step, h.t, h.scale, h.good_steps, h.skipped)
    assert len(st.read_log()) == 0

    # the host reads the device-wide word (which clears it) and resets the state's status
    assert mp.mp_gemm_device_status() == mp.MP_ERR_TIMEOUT
    assert mp.mp_gemm_device_status() == 0
    h2.status = 0
    st.write(h2)
    mp.mp_master_update(plan, st, opt, 0)
    mp.mp_loss_scale_update(st)
    h3 = st.read()
    assert (h3.status, h3.step, h3.t) == (0, h.step + 1, h.t + 1)
    assert not torch.equal(before[0], tensors[0])       # this update was applied

    # the context is intact: an ordinary product right after is bit-exact
    mp.mp_linear_fwd(Xd, Wd, Y)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
    want = orc.linear_fwd(X.view(np.uint16), W.view(np.uint16))
    assert (_bits(Y) == want).all()
    raw2 = raw.clone()
    raw2[2:2 + M, :N] = 0x5A5A
    assert bool((raw2 == 0x5A5A).all())                 # only the view was written
    plan.close(); st.close()


def test_self_test_takes_one_tile_only(mp):
    X = torch.zeros(256, 64, dtype=torch.float16, device="cuda")
    W = torch.zeros(64, 64, dtype=torch.float16, device="cuda")
    Y = torch.zeros(256, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(mp.MpError):
        mp.mp_selftest_wait_timeout(X, W, Y, 100)
    with pytest.raises(mp.MpError):
        mp.mp_selftest_wait_timeout(X[:64], W, Y[:64], 0)
    torch.cuda.synchronize()
    assert mp.mp_gemm_device_status() == 0
