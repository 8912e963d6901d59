"""World-size-2 check of the data-parallel path on CPU (gloo): row sharding, one all-reduce of
the FP16 weight gradients, inspection of the reduced gradients, identical updates on all ranks.
The per-rank arithmetic is the oracle's; what is under test is the sharding and exchange logic
that the GPU path uses unchanged (paper_1805_10387_b200/dp.py)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as tmp

from paper_1805_10387_b200 import dp


def test_shard_rows_partitions():
    for M, world in ((6400, 2), (6401, 4), (7, 8), (25600, 3)):
        edges = [dp.shard_rows(M, r, world) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == M
        assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
        sizes = [hi - lo for lo, hi in edges]
        assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, plant_inf, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import mp_oracle as orc
    rng = np.random.default_rng(0)                              # same data drawn on every rank
    M, K, N, S = 96, 40, 24, 64.0
    X = rng.standard_normal((M, K)).astype(np.float16).view(np.uint16)
    g = (rng.standard_normal((M, N)) * 0.05).astype(np.float32)
    w = (rng.standard_normal((K, N)) / 6).astype(np.float32)
    if plant_inf:
        g[M - 1, 3] = np.inf                                    # lives in the LAST rank's shard only
    lo, hi = dp.shard_rows(M, rank, world)
    dY = orc.scale_upstream(np.ascontiguousarray(g[lo:hi]), S)
    dW_local = orc.linear_bwd_wgrad(np.ascontiguousarray(X[lo:hi]), dY, 1)
    local_flag = orc.found_inf(dW_local)
    flat = torch.from_numpy(dW_local.view(np.float16).copy().reshape(-1))
    dp.allreduce_gradients(flat)
    red = flat.numpy().view(np.uint16).reshape(K, N)
    flag = orc.found_inf(red)                                   # inspection of the reduced gradients
    w32 = w.copy().reshape(-1); m = np.zeros_like(w32); v = np.zeros_like(w32)
    w16 = np.zeros(w32.size, np.uint16)
    if not flag:
        orc.adam_update(np.ascontiguousarray(red.reshape(-1)), w32, m, v, w16, S, 1e-3, 0.9, 0.999, 1e-8, 1)
    # single-process result on all rows, for rank 0 to compare with
    if rank == 0:
        full = orc.linear_bwd_wgrad(X, orc.scale_upstream(g, S), 1)
        out.put(("full", full, red.copy(), flag, local_flag))
    out.put(("rank", rank, w32.copy(), flag, local_flag))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("plant_inf", [False, True])
def test_two_ranks_reduce_and_agree(plant_inf):
    ctx = tmp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, plant_inf, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(3)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    full = next(x for x in got if x[0] == "full")
    ranks = sorted((x for x in got if x[0] == "rank"), key=lambda x: x[1])
    # every rank takes the same decision and ends with bitwise identical master weights
    assert ranks[0][3] == ranks[1][3] == int(plant_inf)
    assert (ranks[0][2].view(np.uint32) == ranks[1][2].view(np.uint32)).all()
    if plant_inf:
        assert ranks[0][4] == 0 and ranks[1][4] == 1          # only rank 1 saw it locally
    else:
        # sum of the two shard gradients = gradient over all rows, up to FP16 roundings
        a = full[1].view(np.float16).astype(np.float64); b = full[2].view(np.float16).astype(np.float64)
        assert (np.abs(a - b) <= 2.0 ** -9 * np.abs(a) + 1e-3 * np.sqrt((a * a).mean())).all()


def test_parameter_slices_are_equal_and_aligned():
    for total, world in ((64632, 2), (64632, 3), (1, 8), (75_497_472, 8), (12_846_400 + 29 * 8, 7)):
        padded = dp.padded_total(total, world)
        assert padded >= total and padded % (8 * world) == 0 and padded - total < 8 * world
        edges = [dp.shard_params(padded, r, world) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == padded
        assert all(a[1] == b[0] for a, b in zip(edges, edges[1:]))
        assert len({hi - lo for lo, hi in edges}) == 1
        assert all(lo % 8 == 0 for lo, _ in edges)              # 16-byte boundaries for FP16 and FP32
    with pytest.raises(ValueError):
        dp.shard_params(100, 0, 3)


def _shard_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    comm = dp.Comm()
    total = dp.padded_total(1000 + 13, world)                   # ragged: the last slice holds padding
    rng = np.random.default_rng(100 + rank)
    mine = torch.from_numpy(rng.integers(-8, 9, total).astype(np.float16))   # exact in FP16, any order
    flat = mine.clone()
    lo, hi = dp.shard_params(total, rank, world)
    got = torch.zeros(hi - lo, dtype=torch.float16)
    comm.reduce_scatter(flat, got)
    assert torch.equal(flat, mine)                              # the input is left alone
    # all-gather: every rank contributes (its slice + rank) and ends with the same full buffer
    full = torch.zeros(total, dtype=torch.float16)
    full[lo:hi] = got + rank
    comm.all_gather(full, full[lo:hi])
    word = torch.tensor([1 if rank == world - 1 else 0], dtype=torch.int32)
    comm.all_reduce_max(word)
    out.put((rank, mine.numpy().copy(), got.numpy().copy(), full.numpy().copy(), int(word[0])))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_exchange_bookkeeping(world):
    """reduce-scatter gives each rank the sum of its slice, all-gather rebuilds the full buffer on
    every rank, the flag word takes the max: the exchanges of the sharded-update schedule."""
    ctx = tmp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=120) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    total = got[0][1].size
    want_sum = sum(g[1].astype(np.float32) for g in got)
    want_full = np.empty(total, np.float32)
    for r, g in enumerate(got):
        lo, hi = dp.shard_params(total, r, world)
        assert (g[2].astype(np.float32) == want_sum[lo:hi]).all()
        want_full[lo:hi] = want_sum[lo:hi] + r
    for g in got:
        assert (g[3].astype(np.float32) == want_full).all()
        assert g[4] == 1
