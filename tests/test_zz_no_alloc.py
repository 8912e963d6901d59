"""mp_linear_bwd_wgrad_static: the weight gradient for callers that cannot allocate device
memory (a runtime that owns all of it, a step that must not trigger the device-wide stall of an
allocation) and have no buffer to lend.  Its scratch is a fixed array inside the library, so the
only things to prove are that it returns exactly what mp_linear_bwd_wgrad returns -- on a first
call and again on a second call that finds the previous call's partial sums in the array -- and
that it refuses sizes the array cannot hold.

This file is named to be collected last: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _rand16(shape, seed, scale=1.0):
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    return (torch.randn(*shape, generator=g, device="cuda") * scale).half()


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("M,K,N", [(4096, 128, 256), (3000, 200, 296), (640, 64, 64)])
def test_static_scratch_matches_workspace_entry_point_twice(mp, M, K, N):
    need = mp.mp_gemm_workspace_bytes(M, K, N, mp.MP_OP_WGRAD)
    assert need <= mp.mp_static_scratch_bytes() == 32 << 20
    if M >= 3000:
        assert need > 0                           # these sizes really go through the scratch
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    for call in range(2):                         # second call: different data, stale scratch
        X = _rand16((M, K), 10 + call)
        dY = _rand16((M, N), 20 + call, 30.0 if call == 0 else 600.0)   # 2nd call overflows FP16
        want = torch.full((K, N), 7.0, dtype=torch.float16, device="cuda")
        got = torch.full((K, N), 9.0, dtype=torch.float16, device="cuda")
        st_a, st_b = mp.State(), mp.State()
        mp.mp_linear_bwd_wgrad(X, dY, want, st_a, ws)
        mp.mp_linear_bwd_wgrad_static(X, dY, got, st_b)
        torch.cuda.synchronize()
        assert mp.mp_gemm_device_status() == 0
        assert (_bits(got) == _bits(want)).all()            # same arithmetic: identical bits
        fa, fb = st_a.read().found_inf, st_b.read().found_inf
        assert fa == fb
        if M >= 3000:
            assert fa == call                               # overflow exactly on the second call
        st_a.close(); st_b.close()


def test_static_scratch_refuses_what_it_cannot_hold(mp):
    M, K, N = 16384, 2048, 1536                 # 96 tiles, long reduction: split, 36 MiB of partials
    need = mp.mp_gemm_workspace_bytes(M, K, N, mp.MP_OP_WGRAD)
    assert need > mp.mp_static_scratch_bytes()
    X = torch.zeros(M, K, dtype=torch.float16, device="cuda")
    dY = torch.zeros(M, N, dtype=torch.float16, device="cuda")
    dW = torch.full((K, N), 3.0, dtype=torch.float16, device="cuda")
    with pytest.raises(mp.MpError) as e:
        mp.mp_linear_bwd_wgrad_static(X, dY, dW, None)
    assert e.value.code == mp.MP_ERR_TOO_LARGE and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert bool((dW == 3.0).all())              # nothing was launched
