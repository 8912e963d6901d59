"""The data-parallel step on the CUDA path, checked on ONE GPU: G stacks in one process stand for
G ranks (rows split by dp.shard_rows, same weights).  The collectives are test doubles that do
with plain torch operations what the NCCL calls do (a sum over ranks in rank order in FP16, a
slice of it, a concatenation, a max of one word); everything else -- the products, the
inspection of the exchanged gradients, the update over the whole range or over a rank's slice,
the flag exchange, the loss-scale state machine -- is the library's own code, driven through
the same LinearStack methods a real multi-rank run calls, in lockstep.

Checked against the oracle's single-process step on the concatenated rows (paper Section 4:
replicas that exchange gradients compute the gradient of the whole batch)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_1805_10387_b200 import dp, synth  # noqa: E402


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _f(bits):
    return bits.view(np.float16).astype(np.float64)


class Hub:
    """Completes a collective when every rank has posted its buffers (the ranks are driven one
    after the other, phase by phase, on one stream)."""

    def __init__(self, world):
        self.world, self.pending = world, {}

    def post(self, kind, rank, bufs):
        d = self.pending.setdefault(kind, {})
        assert rank not in d
        d[rank] = bufs
        if len(d) == self.world:
            getattr(self, "_" + kind)(self.pending.pop(kind))

    def _sum(self, d):                       # rank order, every partial sum rounded to FP16
        total = d[0][0].clone()
        for r in range(1, self.world):
            total = total + d[r][0]
        return total

    def _ar(self, d):
        self.last_inputs = [d[r][0].clone() for r in range(self.world)]
        total = self._sum(d)
        for r in range(self.world):
            d[r][0].copy_(total)

    def _rs(self, d):
        self.last_inputs = [d[r][0].clone() for r in range(self.world)]
        total = self._sum(d)
        for r in range(self.world):
            lo, hi = dp.shard_params(total.numel(), r, self.world)
            d[r][1].copy_(total[lo:hi])

    def _ag(self, d):
        mine = [d[r][1].clone() for r in range(self.world)]
        n = mine[0].numel()
        for r in range(self.world):
            for q in range(self.world):
                d[r][0][q * n:(q + 1) * n].copy_(mine[q])

    def _max(self, d):
        m = torch.stack([d[r][0] for r in range(self.world)]).max(dim=0).values
        for r in range(self.world):
            d[r][0].copy_(m)


class LockstepComm:
    def __init__(self, hub, rank):
        self.hub, self.rank, self.world = hub, rank, hub.world

    def all_reduce(self, flat): self.hub.post("ar", self.rank, (flat,))
    def reduce_scatter(self, flat, out): self.hub.post("rs", self.rank, (flat, out))
    def all_gather(self, flat, mine): self.hub.post("ag", self.rank, (flat, mine))
    def all_reduce_max(self, word): self.hub.post("max", self.rank, (word,))


SHAPES = [(192, 136, 264), (192, 264, 72), (192, 135, 72)]     # FFN-like chained pair + a free layer
CHAIN = [False, True, False]


def _cfg():
    cfg = synth.config("c3")
    cfg.shapes, cfg.chain = list(SHAPES), list(CHAIN)
    cfg.growth_interval, cfg.init_scale = 2, 2.0 ** 12
    return cfg


def _make_ranks(mp, cfg, world, shard):
    from paper_1805_10387_b200.stack import LinearStack
    hub = Hub(world)
    L = len(cfg.shapes)
    stacks = []
    for r in range(world):
        lo, hi = dp.shard_rows(cfg.shapes[0][0], r, world)
        shapes = [(hi - lo, k, n) for _, k, n in cfg.shapes]
        st = LinearStack(shapes, [cfg.chained(l) for l in range(L)], lr=cfg.lr, init_scale=cfg.init_scale,
                         growth_interval=cfg.growth_interval, comm=LockstepComm(hub, r), shard_update=shard)
        for l in range(L):
            w = synth.weights(cfg, l)
            st.load_weights(l, torch.from_numpy(w).cuda(),
                            torch.from_numpy(synth.fp16_bits(w).view(np.float16).reshape(w.shape)).cuda())
        stacks.append(st)
    return stacks


def _lockstep_step(stacks, xs_r, gs_r):
    for s, xs, gs in zip(stacks, xs_r, gs_r):
        s.products(xs, gs)
    for phase in ("exchange_gradients", "inspect_exchanged", "apply_update", "publish_weights"):
        for s in stacks:
            getattr(s, phase)()
    from paper_1805_10387_b200 import mp
    for s in stacks:
        mp.mp_loss_scale_update(s.state)


def _pad_dev(bits):
    r, c = bits.shape
    buf = torch.zeros(r, (c + 7) // 8 * 8, dtype=torch.float16, device="cuda")
    buf[:, :c] = torch.from_numpy(bits.view(np.float16)).cuda()
    return buf


@pytest.mark.parametrize("world", [2, 3])
def test_data_parallel_step_replicated_and_sharded(orc, mp, world):
    cfg = _cfg()
    L = len(cfg.shapes)
    M = cfg.shapes[0][0]
    rep = _make_ranks(mp, cfg, world, shard=False)
    shd = _make_ranks(mp, cfg, world, shard=True)
    assert shd[0].total % (8 * world) == 0 and shd[0].total >= rep[0].total
    layers = []
    for l in range(L):
        layers.append(orc.make_layer(synth.weights(cfg, l), "adam", cfg.chained(l)))
    sc = orc.Scaler(cfg.init_scale, cfg.growth_interval)
    opt = orc.Optim(lr=cfg.lr)
    n_real = rep[0].total
    flags = []
    for step in range(5):
        xs = [None if cfg.chained(l) else synth.activations(cfg, l, step) for l in range(L)]
        gs = [None if cfg.feeds_next(l) else synth.upstream(cfg, l, step) for l in range(L)]
        if step == 2:                         # a non-finite gradient in the LAST rank's rows only
            gs[1] = gs[1].copy()
            gs[1][M - 1, 5] = np.inf
        xs_r, gs_r = [], []
        for r in range(world):
            lo, hi = dp.shard_rows(M, r, world)
            xs_r.append([None if x is None else _pad_dev(np.ascontiguousarray(x[lo:hi])) for x in xs])
            gs_r.append([None if g is None else torch.from_numpy(np.ascontiguousarray(g[lo:hi])).cuda() for g in gs])
        pre = [(s.w32_flat.clone(), s.m_flat.clone(), s.v_flat.clone(), s.w16_flat.clone()) for s in rep]
        pre_host = (rep[0].w32_flat.cpu().numpy().copy(), rep[0].m_flat.cpu().numpy().copy(),
                    rep[0].v_flat.cpu().numpy().copy())
        t_pre = rep[0].state.read().t
        _lockstep_step(rep, xs_r, gs_r)
        _lockstep_step(shd, xs_r, gs_r)
        rec = orc.train_step(layers, xs, gs, sc, opt)
        torch.cuda.synchronize()
        assert mp.mp_gemm_device_status() == 0
        flags.append(rec.found_inf)

        # every rank of both schedules: same flag, scale and counters as the oracle, bit for bit
        for s in rep + shd:
            h, log = s.state.read(), s.state.read_log(1)[0]
            assert log.found_inf == rec.found_inf, (step, log.found_inf)
            assert (log.scale_before, log.scale_after) == (rec.S_before, rec.S_after)
            assert (h.t, h.good_steps, h.skipped, h.status) == (sc.t, sc.good, sc.skipped, 0)
        if step == 2:                          # only the last rank's own kernels saw the inf
            assert rec.found_inf == 1

        # the ranks of the replicated schedule hold bitwise identical masters, moments and weights
        for s in rep[1:]:
            for a, b in ((s.w32_flat, rep[0].w32_flat), (s.m_flat, rep[0].m_flat), (s.v_flat, rep[0].v_flat)):
                assert torch.equal(a.view(torch.int32), b.view(torch.int32))
            assert torch.equal(s.w16_flat.view(torch.int16), rep[0].w16_flat.view(torch.int16))
        # the sharded schedule: every rank has the full FP16 copy, bitwise the replicated one's;
        # its slice of master and moments is bitwise the replicated run's slice
        for r, s in enumerate(shd):
            assert torch.equal(s.w16_flat[:n_real].view(torch.int16), rep[0].w16_flat.view(torch.int16))
            lo, hi = s.shard
            hi_real = min(hi, n_real)
            for a, b in ((s.w32_flat, rep[0].w32_flat), (s.m_flat, rep[0].m_flat), (s.v_flat, rep[0].v_flat)):
                assert torch.equal(a[:hi_real - lo].view(torch.int32), b[lo:hi_real].view(torch.int32))
                assert bool((a[hi_real - lo:] == 0).all())          # padding past the last tensor stays zero

        if rec.found_inf:                      # skipped everywhere: bitwise unchanged
            for s, p in zip(rep, pre):
                for a, b in zip((s.w32_flat, s.m_flat, s.v_flat), p[:3]):
                    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
                assert torch.equal(s.w16_flat.view(torch.int16), p[3].view(torch.int16))
            continue

        # the exchange: what every rank holds afterwards is the FP16 sum, in rank order, of what the
        # ranks' weight-gradient kernels stored (numpy's float16 addition, correctly rounded)
        hub = rep[0].comm.hub
        parts = [_bits(t).view(np.float16) for t in hub.last_inputs]
        acc = parts[0].copy()
        for r in range(1, world):
            acc = (acc + parts[r]).astype(np.float16)
        assert (_bits(rep[0].dw_flat) == acc.view(np.uint16)).all()
        # each rank's gradient = the oracle's weight gradient of that rank's rows (the operands
        # the rank's kernel read), and their sum = the oracle's gradient over all rows up to the
        # FP16 roundings of the parts and of the running sums
        for l, (_, K, N) in enumerate(cfg.shapes):
            want = _f(layers[l].dW)
            mag = np.zeros_like(want)
            order = np.zeros_like(want)          # FP32 summation-order error of the parts and of the whole
            for r, s in enumerate(rep):
                Xr, dYr = _bits(s.X(l)), _bits(s.dY(l))
                pr = orc.linear_bwd_wgrad(np.ascontiguousarray(Xr), np.ascontiguousarray(dYr))
                off, ld = s.offsets[l], s.ldw[l]
                got_r = parts[r][off:off + K * ld].reshape(K, ld)[:, :N].view(np.uint16)
                assert (got_r == pr).mean() > 0.98
                ex, ab = orc.linear_exact("wgrad", np.ascontiguousarray(Xr), np.ascontiguousarray(dYr))
                assert (np.abs(_f(got_r) - ex) <= 2.0 ** -10 * np.abs(ex) + Xr.shape[0] * 2.0 ** -24 * ab + 2.0 ** -24).all()
                mag += np.abs(_f(pr))
                order += 2 * Xr.shape[0] * world * 2.0 ** -24 * ab
            got = _f(_bits(rep[0].dW(l)))
            # layer 2 reads inputs only, so its operands are the oracle's bit for bit; layers 0
            # and 1 form a chain whose activations already differ by roundings between the sides
            slack = 0.0 if l == 2 else 4e-3 * np.sqrt((want * want).mean())
            assert (np.abs(got - want) <= 2.0 ** -11 * (world + 1) * mag + 2.0 ** -10 * np.abs(want) + order + 2.0 ** -24 + slack).all(), l
        # the update: the oracle fed with the GPU's own reduced gradient and prior state, at 1e-6
        w, m, v = pre_host
        w16 = np.zeros(w.size, np.uint16)
        g16 = np.ascontiguousarray(_bits(rep[0].dw_flat))
        orc.adam_update(g16, w, m, v, w16, rec.S_before, cfg.lr, cfg.beta1, cfg.beta2, cfg.eps, t_pre + 1)
        w_gpu = rep[0].w32_flat.cpu().numpy()
        assert (np.abs(w_gpu - w) <= 1e-6 * np.maximum(np.abs(w), cfg.lr)).all()
        assert (_bits(rep[0].w16_flat) == orc.f2h(w_gpu)).all()
        # free-running oracle on the concatenated rows: bounded drift (Adam turns the sign of a
        # near-zero gradient into a full step of size lr)
        for l in range(L):
            diff = np.abs(rep[0].W32(l).cpu().numpy() - layers[l].w32)
            assert diff.max() <= 2.5 * cfg.lr * (t_pre + 1) + 1e-7 and np.median(diff) <= 2e-6
    assert flags[2] == 1 and sum(flags) >= 1 and flags.count(0) >= 2
    for s in rep + shd:
        s.close()
