#!/usr/bin/env python
"""Benchmark of the mixed-precision training step of a linear-layer stack on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5] [--impl reference]
  python bench.py --workload c3 --per-shape      (each layer shape's products alone, beside cuBLAS)

Without --workload the line's top-level fields are the GNMT-like stack (c2) and the other
workloads (c3, c4, and the update-only sweep c5 up to 1e9 parameters) are timed after it with
fewer steps and reported under `workloads`, each with its own `roofline`.

One step = forward, weight-gradient and data-gradient products of every layer (FP16 operands,
FP32 accumulation), upstream scaling, the fused unscale / inspect / FP32-master optimizer /
FP16 recast update and the loss-scale state machine, on one batch of seeded synthetic input.
Prints ONE JSON line.  `value` is the whole job's GEMM throughput over the step time (inputs
resident in HBM); `e2e` is the same with pinned host inputs copied in and the loss-scale state
read back every step; `roofline` is for the dominant kernel (the tcgen05 GEMM), timed with CUDA
events around a region that replays the step's product calls alone; `update` gives the fused
update's GB/s.
`--impl reference` times the CPU oracle (the slow, plain restatement of the method) instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MP train step: GEMM TFLOP/s and master-update GB/s, % of B200 peak"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes per launch of the product kernels from one ncu capture per workload (dram__bytes_read.sum
# + dram__bytes_write.sum summed over one step's product launches, split-reduction kernels included,
# divided by their number; on c2 a launch holds four layers' products, 4 x 95.4 MB algorithmic), valid
# only for the kernel source it was taken on.
NCU_TRAFFIC = {"sha": "0874106332883409", "bytes_per_launch": {"c2": 402.4e6, "c3": 176.9e6, "c4": 115.9e6}}
# flop per clock and SM of the FP16 tensor pipe (one 128 x 256 x 16 MMA per SM in 128 clocks)
TENSOR_FLOP_PER_CLK_SM = 8192


# DRAM bytes per parameter of the fused update from one ncu capture at 1e8 parameters in 64 tensors
# (2.7404 GB per launch); a launch over P parameters moves P times this (traffic grows in
# proportion: every parameter is touched once), valid only for the kernel source it was taken on.
NCU_UPDATE_TRAFFIC = {"sha": "77306490e753c3d8", "bytes_per_param": 27.40}


def update_kernel_sha():
    return hashlib.sha256(open(os.path.join(ROOT, "paper_1805_10387_b200", "csrc", "update.cu"), "rb").read()).hexdigest()[:16]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def kernel_sha():
    h = hashlib.sha256()
    for f in ("gemm.cu", "ptx.cuh"):
        h.update(open(os.path.join(ROOT, "paper_1805_10387_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed regions run; every sample
    keeps its arrival time so that a region can ask for the samples that fell inside it."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.rows, self.times, self.proc, self.index = [], [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])
            self.times.append(time.time())

    def stop(self):
        if self.proc:
            self.proc.terminate()
            self.thread.join(timeout=2)

    @staticmethod
    def _num(r, i):
        return float(r[i]) if len(r) > i and r[i].replace(".", "").isdigit() else None

    def summary(self, windows=None):
        """windows: list of (t0, t1) in time.time() seconds; `sm_mhz` is the median over the samples
        inside them (all samples when None or when none fell inside)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = list(zip(self.rows, self.times))
        inside = [r for r, t in rows if windows and any(a <= t <= b + 0.05 for a, b in windows)]
        use = inside if inside else [r for r, _ in rows]
        sm = sorted(x for x in (self._num(r, 0) for r in use) if x is not None)
        mx = [x for x in (self._num(r, 1) for r in use) if x is not None]
        pw = [x for x in (self._num(r, 2) for r in use) if x is not None]
        reasons = [n for i, n in enumerate(self.NAMES) if any(len(r) > 3 + i and r[3 + i] == "Active" for r in use)]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx[0] if mx else None,
                "reasons": reasons, "samples": len(sm), "power_w_max": max(pw) if pw else None,
                "power_w_median": sorted(pw)[len(pw) // 2] if pw else None}


# ------------------------------------------------------------------ reference arm (CPU oracle)
def oracle_sample_step(orc, synth, cfg, rows, upd_params, data=None):
    """One bounded sample of the workload on the CPU oracle: the three products of layer 0 on
    its first `rows` rows and the optimizer update of `upd_params` parameters.  Returns
    (seconds of the products, seconds of the update, gemm_flops, update_bytes, data)."""
    import numpy as np
    M, K, N = cfg.shapes[0]
    if data is None:
        w = synth.weights(cfg, 0)
        X = np.ascontiguousarray(synth.activations(cfg, 0, 0)[:rows])
        g = np.ascontiguousarray(synth.upstream(cfg, 0, 0)[:rows])
        W16 = synth.fp16_bits(w).reshape(K, N)
        n = min(upd_params, K * N)
        st = dict(w32=w.reshape(-1)[:n].copy(), m=np.zeros(n, np.float32), v=np.zeros(n, np.float32),
                  w16=np.zeros(n, np.uint16))
        data = (X, g, W16, st)
    X, g, W16, st = data
    S = 2.0 ** 10
    t0 = time.perf_counter()
    orc.linear_fwd(X, W16)
    dY = orc.scale_upstream(g, S)
    dW = orc.linear_bwd_wgrad(X, dY)
    orc.linear_bwd_dgrad(dY, W16)
    t1 = time.perf_counter()
    n = st["w32"].size
    g16 = np.ascontiguousarray(dW.reshape(-1)[:n])
    if not orc.found_inf(dW):
        if cfg.optimizer == "adam":
            orc.adam_update(g16, st["w32"], st["m"], st["v"], st["w16"], S, cfg.lr, cfg.beta1, cfg.beta2, cfg.eps, 1)
        else:
            orc.momentum_update(g16, st["w32"], st["m"], st["w16"], S, cfg.lr, cfg.momentum)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1, 3 * 2 * rows * K * N, n * (28 if cfg.optimizer == "adam" else 20), data


def workload_config(cfg, world=1, layers_kind="plain linear", sharded=False):
    """The `config` object of the JSON line: the same for the CUDA arm and the reference arm."""
    return {"workload": cfg.name + ": " + cfg.note, "layers": len(cfg.shapes), "params": cfg.n_params(),
            "gemm_gflop_per_step": cfg.gemm_flops() / 1e9, "optimizer": cfg.optimizer,
            "parallelism": (f"dp{world}" + (" sharded update" if sharded else "")) if world > 1 else "single",
            "layers_kind": layers_kind,
            "cache": "per-step working set (weights, moments, activations) far exceeds the 126 MB L2"}


def cpu_baseline_of(orc, synth, cfg, seconds):
    """The oracle as it stands on the host cores, on a bounded sample of the workload: products and
    update timed apart (GFLOP/s, GB/s) and together (`value`, the whole-sample analogue of the
    GPU line's `value`)."""
    rows, upd = 64, 1 << 21
    tg = tu = 0.0
    fl = by = 0
    data = None
    t_budget = time.perf_counter()
    while tg + tu < seconds and time.perf_counter() - t_budget < 3.5 * seconds:
        a, b, f, nb, data = oracle_sample_step(orc, synth, cfg, rows, upd, data)
        tg, tu, fl, by = tg + a, tu + b, fl + f, by + nb
    return {"value": fl / (tg + tu) / 1e12, "unit": "TFLOP/s", "cores": orc.hardware_threads(), "kind": "oracle",
            "gemm_gflops": fl / tg / 1e9, "update_gbs": by / tu / 1e9,
            "update_note": "the oracle's update loop is one thread (a plain loop, as it stands)",
            "sample": f"fwd+wgrad+dgrad of layer 0 of {cfg.name} on its first {rows} rows + update of {upd} params, "
                      f"repeated for {tg + tu:.1f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import mp_oracle as orc
    from paper_1805_10387_b200 import synth
    orc.build()
    wl = args.workload or "c2"
    cfg = synth.config("c2" if wl == "c5" else wl)
    # size the per-step sample so that the whole run (warm-up + steps) takes about two minutes
    upd = 1 << 20
    data = None
    a, b, _, _, data = oracle_sample_step(orc, synth, cfg, 8, upd, data)
    a, b, _, _, data = oracle_sample_step(orc, synth, cfg, 8, upd, data)
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = int(max(4, min(64, 8 * budget / max(a + b, 1e-3))))
    data = None
    for _ in range(args.warmup):
        _, _, _, _, data = oracle_sample_step(orc, synth, cfg, rows, upd, data)
    tg = tu = 0.0
    flops = nbytes = 0
    for _ in range(args.steps):
        a, b, f, nb, data = oracle_sample_step(orc, synth, cfg, rows, upd, data)
        tg, tu, flops, nbytes = tg + a, tu + b, flops + f, nbytes + nb
    tot = tg + tu
    val = flops / tot / 1e12
    cores = orc.hardware_threads()
    sample = f"per step: fwd+wgrad+dgrad of layer 0 on its first {rows} rows + update of {upd} params"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16 in / f32 accumulate",
        "data": "synthetic", "config": workload_config(cfg),
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
                         "gemm_gflops": flops / tg / 1e9, "update_gbs": nbytes / tu / 1e9},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def settle(fn, seconds, sync, dist=None):
    """Runs fn back to back, untimed, for about `seconds` of wall time so that the timed region
    that follows starts in the power and clock state the same work settles into.  With several
    ranks every rank must make the same number of calls (fn holds collectives), so the count is
    fixed from a short calibration and agreed on across the ranks."""
    t0 = time.time()
    if seconds <= 0:
        return 0.0
    if dist is None:
        while time.time() - t0 < seconds:
            for _ in range(8):
                fn()
            sync()
        return time.time() - t0
    import torch
    for _ in range(8):
        fn()
    sync()
    per_call = max((time.time() - t0) / 8, 1e-5)
    n = torch.tensor([int(seconds / per_call) + 1], device="cuda")
    dist.all_reduce(n, op=dist.ReduceOp.MAX)
    for _ in range(int(n.item())):
        fn()
    sync()
    return time.time() - t0


# ------------------------------------------------------------------ update-only sweep
def run_update_sweep(args, sampler=None, steps=None, settle_s=1.0):
    """Update-only workload: unscale / inspect / Adam / FP16 recast over 1e6 .. 1e9 parameters in
    1 .. 500 tensors of log-uniform sizes, gradients rn16(S * N(0, 1e-3)).  Per size: GB/s on the
    algorithmic 28 B/param for applied steps with the flag trusted (check_mode 0) and with the
    in-call inspection (check_mode 1, 30 B/param moved), and the time of a skipped step.  Every
    timed loop follows `settle_s` seconds of the same launches, untimed.  Returns the JSON object."""
    import torch
    from paper_1805_10387_b200 import mp, synth
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    mp.lib()
    steps = steps or args.steps
    pk, pk_src = peaks()
    rows = []
    own_sampler = sampler is None
    if own_sampler:
        sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
        sampler.start()
    windows = []
    timed_launches = 0
    for P, n in ((1_000_000, 1), (10_000_000, 8), (100_000_000, 64), (1_000_000_000, 500)):
        if P > args.max_params:
            break
        counts = synth.tensor_sizes(P, n, 4)
        offs, tot = [], 0
        for c in counts:
            offs.append(tot)
            tot += (c + 7) // 8 * 8
        mk = lambda dt: torch.zeros(tot, dtype=dt, device="cuda")
        g16, w16, w32, m, v = mk(torch.float16), mk(torch.float16), mk(torch.float32), mk(torch.float32), mk(torch.float32)
        views = lambda flat: [flat[o:o + c] for o, c in zip(offs, counts)]
        plan = mp.UpdatePlan(views(g16), views(w32), views(m), views(v), views(w16))
        st = mp.State(init_scale=1024.0, growth_interval=10 ** 6)
        opt = mp.OptimConfig(mp.MP_OPT_ADAM, 1e-3, 0.9, 0.999, 1e-8, 0.9, 0.0)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(5)
        blk = 1 << 24
        z = torch.randn(min(blk, tot), generator=gen, device="cuda") * (0.0316 * 1024.0)
        for lo in range(0, tot, blk):
            k = min(blk, tot - lo)
            g16[lo:lo + k] = z[:k].half()
            w32[lo:lo + k] = z[:k] * 1e-4
        iters = max(3, min(steps, int(2e10 // (P * 30)) + 3))

        def one(mode):
            mp.mp_master_update(plan, st, opt, mode)
            mp.mp_loss_scale_update(st)

        def timed(mode, reps):
            nonlocal timed_launches
            settle(lambda: one(mode), settle_s, torch.cuda.synchronize)
            t0 = time.time()
            n0 = mp.mp_kernel_launch_count()
            ts = []
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                mp.mp_master_update(plan, st, opt, mode)
                b.record()
                mp.mp_loss_scale_update(st)
                ts.append((a, b))
            torch.cuda.synchronize()
            timed_launches += mp.mp_kernel_launch_count() - n0
            if P >= 100_000_000:
                windows.append((t0, time.time()))
            return sum(a.elapsed_time(b) for a, b in ts) / reps
        ms0 = timed(0, iters)
        ms1 = timed(1, iters)
        skipped0 = st.read().skipped
        g16.view(torch.int16)[offs[-1] + counts[-1] - 1] = 0x7C00      # overflow: skipped steps
        ms_skip = timed(1, iters)
        assert st.read().skipped - skipped0 >= iters
        rows.append({"params": P, "tensors": n, "ms_trusted_flag": ms0, "gbs_28B": P * 28 / ms0 / 1e6,
                     "frac_of_peak": P * 28 / ms0 / 1e6 / pk["hbm_gbs"],
                     "ms_with_inspection": ms1, "gbs_28B_with_inspection": P * 28 / ms1 / 1e6,
                     "gbs_30B_moved_with_inspection": P * 30 / ms1 / 1e6, "ms_skipped_step": ms_skip,
                     "timed_launches": iters,
                     "note": "L2-resident / launch-bound" if P * 16 < 126e6 else "HBM-bound"})
        plan.close()
        st.close()
        del g16, w16, w32, m, v, z
        torch.cuda.empty_cache()
    if own_sampler:
        sampler.stop()
    clocks = sampler.summary(windows)
    top = rows[-1]
    return {
        "metric": METRIC, "value": top["gbs_28B"], "unit": "GB/s", "n_gpus": 1, "steps": steps,
        "warmup": 3, "ms_per_step": top["ms_trusted_flag"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 gradients / f32 master", "data": "synthetic",
        "config": {"workload": "c5: update-only sweep, Adam, 1e6..1e9 parameters in 1..500 log-uniform tensors",
                   "cache": "1e8 and 1e9 parameters (1.6 / 16 GB of state) far exceed the 126 MB L2",
                   "settle_s": settle_s},
        "gpu_launches": int(timed_launches),
        "roofline": {"kernel": "mp_master_update_kernel", "bound": "hbm", "achieved": top["gbs_28B"],
                     "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": top["gbs_28B"] / pk["hbm_gbs"],
                     "traffic": (NCU_UPDATE_TRAFFIC["bytes_per_param"] * top["params"]
                                 if NCU_UPDATE_TRAFFIC["sha"] == update_kernel_sha() else None),
                     "traffic_note": "ncu capture at 1e8 parameters scaled by the parameter count",
                     "algorithmic_bytes_per_launch": 28 * top["params"], "avg_launch_ms": top["ms_trusted_flag"],
                     "peak_source": pk_src + " copy", "frac_of_nominal_8000": top["gbs_28B"] / 8000.0},
        "sweep": rows, "clocks": clocks}


# ------------------------------------------------------------------ per-shape timing
def run_per_shape(args):
    """Each distinct layer shape of the workload alone: the three products back to back inside a
    CUDA graph of 24 launches over rotating operand sets (working set above the 126 MB L2), best
    of five replays, with torch.matmul (cuBLAS) on the same operands beside it as a reference
    point.  Prints one JSON line; not the bench value (no power-capped steady state)."""
    import torch
    from paper_1805_10387_b200 import mp, synth
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    mp.lib()
    cfg = synth.config(args.workload)
    reps = 24

    def graph_us(fn, sets):
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            for i in range(3):
                fn(i % sets)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(reps):
                    fn(i % sets)
            g.replay()
            torch.cuda.synchronize()
            best = float("inf")
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                g.replay()
                b.record()
                torch.cuda.synchronize()
                best = min(best, a.elapsed_time(b) / reps)
        return best * 1e3

    rows = []
    for (M, K, N) in sorted(set(cfg.shapes), key=cfg.shapes.index):
        Np = (N + 7) // 8 * 8
        sets = max(2, int(300e6 // (2 * (M * K + K * Np + M * Np))) + 1)
        mk = lambda r, c, scale: [(torch.randn(r, c, device="cuda") * scale).half() for _ in range(sets)]
        X, W, dY = mk(M, K, 1.0), mk(K, Np, K ** -0.5), mk(M, Np, 0.01)
        out = lambda r, c: [torch.empty(r, c, device="cuda", dtype=torch.float16) for _ in range(sets)]
        Y, dX, dW = out(M, Np), out(M, K), out(K, Np)
        ws = torch.empty(max(16, max(mp.mp_gemm_workspace_bytes(M, K, N, op) for op in (0, 1, 2))),
                         dtype=torch.uint8, device="cuda")
        st = mp.State()
        us = {"fwd": graph_us(lambda i: mp.mp_linear_fwd(X[i], W[i][:, :N], Y[i][:, :N], ws), sets),
              "dgrad": graph_us(lambda i: mp.mp_linear_bwd_dgrad(dY[i][:, :N], W[i][:, :N], dX[i], ws), sets),
              "wgrad": graph_us(lambda i: mp.mp_linear_bwd_wgrad(X[i], dY[i][:, :N], dW[i][:, :N], st, ws), sets)}
        if N == Np:
            us["cublas_fwd"] = graph_us(lambda i: torch.matmul(X[i], W[i], out=Y[i]), sets)
            us["cublas_dgrad"] = graph_us(lambda i: torch.matmul(dY[i], W[i].t(), out=dX[i]), sets)
            us["cublas_wgrad"] = graph_us(lambda i: torch.matmul(X[i].t(), dY[i], out=dW[i]), sets)
        rows.append({"M": M, "K": K, "N": N, "operand_sets": sets,
                     "us": {k: round(v, 1) for k, v in us.items()},
                     "tflops": {k: round(2.0 * M * K * N / v / 1e6) for k, v in us.items()}})
        st.close()
        del X, W, dY, Y, dX, dW, ws
        torch.cuda.empty_cache()
    assert mp.mp_gemm_device_status() == 0
    print(json.dumps({"per_shape": rows, "workload": cfg.name, "launches_per_graph": reps}))


# ------------------------------------------------------------------ CUDA arm: one stack workload
def run_stack(args, name, steps, sampler, dist, full):
    """Times one of the GEMM workloads (c2, c3, c4) and returns its JSON object.  `full`: also the
    end-to-end region (host inputs) and the CPU baseline.  Every device-timed region is preceded
    by `--settle` seconds of untimed replays of the same region."""
    import torch
    from paper_1805_10387_b200 import mp, synth
    from paper_1805_10387_b200.stack import HostPipeline, LinearStack

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    cfg = synth.config(name)
    L = len(cfg.shapes)
    chained = [cfg.chained(l) for l in range(L)]
    acts = None
    lstm = None
    if args.real_layers and cfg.name == "c2":      # the gate products feed LSTM cells (no bias, no activation)
        lstm = [True] * L
    elif args.real_layers:
        act = mp.MP_ACT_CLIPPED_RELU if cfg.name == "c4" else mp.MP_ACT_RELU
        acts = [act if (l + 1 < L and chained[l + 1]) else mp.MP_ACT_NONE for l in range(L)]
    comm = None
    if world > 1:      # data parallel over rows: weights replicated, FP16 weight gradients summed
        from paper_1805_10387_b200 import dp
        comm = dp.Comm()
    stack = LinearStack(cfg.shapes, chained, optimizer=cfg.optimizer, lr=cfg.lr, beta1=cfg.beta1,
                        beta2=cfg.beta2, eps=cfg.eps, momentum=cfg.momentum, init_scale=cfg.init_scale,
                        growth_interval=cfg.growth_interval, acts=acts, bias=args.real_layers and lstm is None,
                        lstm=lstm, comm=comm, shard_update=args.shard_update,
                        overlap_wgrad={"auto": None, "on": True, "off": False}[args.overlap_wgrad])
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + cfg.seed)           # same weights on every rank
    for l, (M, K, N) in enumerate(cfg.shapes):
        w = torch.randn(K, N, generator=gen, device="cuda") / K ** 0.5
        if args.real_layers and lstm is None:
            b = torch.randn(N, generator=gen, device="cuda") * 0.1
            stack.load_weights(l, w, w.half(), b, b.half())
        else:
            stack.load_weights(l, w, w.half())
    gen.manual_seed(99 + rank)                 # each rank its own rows
    xs, gs, xs_host, gs_host = [], [], [], []
    # the FP32 gradients entering the top layers arrive as slices of one flat buffer
    tops = [l for l in range(L) if not stack.feeds_next(l)]
    g_flat = torch.empty(sum(cfg.shapes[l][0] * stack.up_width[l] for l in tops), device="cuda")
    g_off = 0
    for l, (M, K, N) in enumerate(cfg.shapes):
        if chained[l]:
            xs.append(None); xs_host.append(None)
        else:
            z = torch.randn(M, K, generator=gen, device="cuda")
            if cfg.x_dist == "lognormal2":
                z = torch.sign(torch.randn(M, K, generator=gen, device="cuda")) * torch.clamp(torch.exp(2 * z), max=6.0e4)
            x = torch.zeros(M, (K + 7) // 8 * 8, dtype=torch.float16, device="cuda")
            x[:, :K] = z.half()
            xs.append(x)
            xs_host.append(x[:, :K].contiguous().cpu().pin_memory() if full else None)
        if stack.feeds_next(l):
            gs.append(None); gs_host.append(None)
        else:
            Ng = stack.up_width[l]                  # N, or H = N / 4 for an LSTM layer (gradient of h)
            g = g_flat[g_off:g_off + M * Ng].view(M, Ng)
            g_off += M * Ng
            g.copy_(torch.randn(M, Ng, generator=gen, device="cuda") * cfg.grad_std)
            gs.append(g)
            gs_host.append(g.cpu().pin_memory() if full else None)
    h2d = sum(t.numel() * t.element_size() for t in xs_host + gs_host if t is not None)
    d2h = 56

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    windows = {}

    def timed(fn, n, key=None, settle_s=None):
        """max over ranks of the device time of n calls, in ms, after the settling replays"""
        t0 = time.time()            # the clock window covers the settling replays too: the same work, the same state
        s = settle(fn, args.settle if settle_s is None else settle_s, torch.cuda.synchronize, dist)
        barrier()
        if s > 0.5:
            t0 += 0.5               # without their first half second, in which the clocks still fall
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n):
            fn()
        b.record()
        barrier()
        if key is not None:
            windows[key] = (t0, time.time())
        ms = torch.tensor([a.elapsed_time(b)], device="cuda")
        if dist is not None:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item()), s

    for _ in range(max(args.warmup, 3)):
        stack.step(xs, gs)
    torch.cuda.synchronize()
    launches0 = mp.mp_kernel_launch_count()
    # (A) the step as one CUDA graph replay per step: `value`
    stack.step(xs, gs)
    launches_per_step = mp.mp_kernel_launch_count() - launches0
    use_graph = world == 1          # the data-parallel step (NCCL collectives inside) is launched call by call
    if use_graph:
        stack.capture(xs, gs)
    run_step = stack.replay if use_graph else (lambda: stack.step(xs, gs))
    st0 = stack.state.read()
    ms_total, settle_step = timed(run_step, steps, "step")
    st1 = stack.state.read()
    launches = launches_per_step * steps
    # (B) the products alone: the step's forward, weight-gradient and data-gradient calls (same
    # order, same buffers) recorded without the other calls and without event nodes, replayed
    # back to back: elapsed device time / launches = the GEMM kernels' average launch duration
    # with their prologue overlap intact and no event between them.  Then per-call device times
    # for the breakdown: the step recorded once more with an event-record node before and after
    # every call, each timed replay followed at once by an untimed one, so that the device never
    # idles while the host reads the events.  Several GPUs: call by call with event pairs.
    per = {}
    gemm_only = None
    upd_only = None
    if use_graph:
        gemm_only = {}
        for key, classes, ss in (("gemm", ("fwd", "dgrad", "wgrad"), None), ("fwd", ("fwd",), args.settle / 4),
                                 ("dgrad", ("dgrad",), args.settle / 4), ("wgrad", ("wgrad",), args.settle / 4)):
            n0 = mp.mp_kernel_launch_count()
            g_sub = stack.capture_only(xs, gs, classes)
            n_launch = mp.mp_kernel_launch_count() - n0
            ms, s = timed(g_sub.replay, steps, key if key == "gemm" else None, ss)
            gemm_only[key] = (ms / steps, n_launch, s)
        g_timed, ev = stack.capture_timed(xs, gs)
        done = torch.cuda.Event()

        def timed_steps():
            for _ in range(steps):
                g_timed.replay()
                done.record()
                stack.replay()
                done.synchronize()
                for nm, a, b in ev:
                    per.setdefault(nm, []).append(a.elapsed_time(b))
        settle(stack.replay, args.settle / 2, torch.cuda.synchronize, dist)
        barrier()
        a_t, b_t = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_t.record(); timed_steps(); b_t.record(); barrier()
        ms_events = a_t.elapsed_time(b_t) / 2.0
        timed_how = ("a further timed region: the step's graph recorded with an event-record node before and "
                     "after every call, each timed replay followed by an untimed one")
    else:
        stack.events = []
        ms_events, _ = timed(lambda: stack.step(xs, gs), steps, None, 0.0)
        events, stack.events = stack.events, None
        for nm, a, b in events:
            per.setdefault(nm, []).append(a.elapsed_time(b))
        timed_how = ("a further timed region of the same steps, launched call by call with a CUDA-event "
                     "pair around every launch")
    # (C) end to end: pinned host inputs in, loss-scale state out, every step, through the
    # double-buffered host pipeline: the copies of batch i+1 run under the kernels of batch i
    ms_e2e = None
    if full:
        pipe = HostPipeline(stack, use_graph=use_graph)

        def e2e_steps(n):
            def go():
                pipe.submit(xs_host, gs_host)
                for i in range(n):
                    if i + 1 < n:
                        pipe.submit(xs_host, gs_host)
                    pipe.run()
            return go
        e2e_steps(3)()
        barrier()
        t0 = time.time()
        a_e, b_e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a_e.record()
        e2e_steps(steps)()
        b_e.record()
        barrier()
        windows["e2e"] = (t0, time.time())
        ms_e2e_t = torch.tensor([a_e.elapsed_time(b_e)], device="cuda")
        if dist is not None:
            dist.all_reduce(ms_e2e_t, op=dist.ReduceOp.MAX)
        ms_e2e = float(ms_e2e_t.item())
    # (D) the fused update alone, replayed back to back (last: it moves the weights without new
    # gradients, which nothing after it reads)
    if use_graph:
        ms, s = timed(lambda: mp.mp_master_update(stack.plan, stack.state, stack.opt, 0), steps, "update",
                      args.settle / 2)
        upd_only = (ms / steps, s)
    assert mp.mp_gemm_device_status() == 0, "a GEMM kernel reported a device-side error"
    assert stack.state.read().status == 0

    flops_step = cfg.gemm_flops()
    ms_step = ms_total / steps
    value = world * flops_step / (ms_step * 1e-3) / 1e12
    pk, pk_src = peaks()
    gemm_calls = sum(len(per.get(k, [])) for k in ("fwd", "dgrad", "wgrad"))
    if gemm_only is not None:
        gemm_ms = gemm_only["gemm"][0] * steps
        gemm_launches = gemm_only["gemm"][1] * steps
        per_op = {k: (flops_step / 3) / (gemm_only[k][0] * 1e-3) / 1e12 for k in ("fwd", "dgrad", "wgrad")}
        gemm_how = ("the step's product calls alone (same order and buffers, no other call, no event between "
                    "them) as a CUDA graph replayed back to back for the same number of steps, after settle_s "
                    "seconds of the same replays untimed; CUDA events around the region; launches include the "
                    "split-reduction kernels of the weight gradients")
        gemm_settle = gemm_only["gemm"][2]
    else:
        gemm_ms = sum(sum(per.get(k, [])) for k in ("fwd", "dgrad", "wgrad"))
        gemm_launches = gemm_calls
        per_op = {k: (flops_step / 3) * steps / (sum(per[k]) * 1e-3) / 1e12
                  for k in ("fwd", "dgrad", "wgrad") if k in per}
        gemm_how = timed_how
        gemm_settle = 0.0
    gemm_tflops = flops_step * steps / (gemm_ms * 1e-3) / 1e12
    skipped = st1.skipped - st0.skipped
    bytes_per_param = 28 if cfg.optimizer == "adam" else 20
    upd_ms = per.get("update", [0.0])
    upd_bytes = cfg.n_params() * bytes_per_param
    # a skipped step's update returns at once (a few microseconds); GB/s is quoted on the
    # applied ones only
    applied_ms = [t for t in upd_ms if t >= 0.25 * max(upd_ms)]
    upd_ms_in_step = sum(applied_ms) / len(applied_ms)
    upd_ms_alone = upd_only[0] if upd_only is not None else upd_ms_in_step
    upd_gbs = upd_bytes / (upd_ms_alone * 1e-3) / 1e9
    sha = kernel_sha()
    traffic = NCU_TRAFFIC["bytes_per_launch"].get(name) if NCU_TRAFFIC["sha"] == sha and not args.real_layers else None
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    clk = {k: (sampler.summary([w]) if sampler is not None else None) for k, w in windows.items()}
    settled = gemm_settle >= 1.5
    peak = pk["bf16_tflops_sustained"] if settled else pk["bf16_tflops"]
    gemm_mhz = clk.get("gemm", {}).get("sm_mhz") if clk.get("gemm") else None
    clock_peak = sms * TENSOR_FLOP_PER_CLK_SM * gemm_mhz * 1e6 / 1e12 if gemm_mhz else None
    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16 in / f32 accumulate", "data": "synthetic",
        "config": workload_config(cfg, world, "LSTM cells on the gate products" if lstm is not None else
                                  "bias + activation (fused epilogues) + bias gradients" if args.real_layers
                                  else "plain linear", stack.shard_update),
        "settle_s": settle_step,
        "settle": "every device-timed region follows that many seconds of untimed replays of itself",
        "gpu_launches": int(launches),
        "launch_mode": "one CUDA graph replay per step (captured from the same C-ABI calls)" if use_graph
                       else "call by call",
        "ms_per_step_in_event_timed_region": ms_events / steps,
        "skipped_steps_in_timed_region": int(skipped),
        "loss_scale": st1.scale,
        "roofline": {"kernel": "mp_gemm_pair_kernel", "bound": "tensor", "achieved": gemm_tflops,
                     "peak": peak, "unit": "TFLOP/s", "frac": gemm_tflops / peak, "traffic": traffic,
                     "peak_source": (f"{pk_src} cuBLAS bf16 sustained (the region is timed after {gemm_settle:.1f} s of "
                                     f"itself; fp16 nominal ratio 1.0)" if settled else
                                     f"{pk_src} cuBLAS bf16 burst (no settling run; fp16 nominal ratio 1.0)"),
                     "settle_s": gemm_settle,
                     "frac_of_burst_peak": gemm_tflops / pk["bf16_tflops"],
                     "frac_of_sustained_peak": gemm_tflops / pk["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": gemm_tflops / 2250.0,
                     "sm_mhz_in_region": gemm_mhz, "clock_peak_tflops": clock_peak,
                     "frac_of_clock_peak": gemm_tflops / clock_peak if clock_peak else None,
                     "clock_peak_how": f"{sms} SMs x {TENSOR_FLOP_PER_CLK_SM} flop/clk x median SM clock sampled inside this "
                                       "region and the settling replays before it (nvidia-smi, every 50 ms)",
                     "launches": gemm_launches, "avg_launch_ms": gemm_ms / max(gemm_launches, 1),
                     "algorithmic_gflop_per_launch": flops_step * steps / max(gemm_launches, 1) / 1e9,
                     "algorithmic_mb_per_launch": cfg_gemm_bytes(cfg) * steps / max(gemm_launches, 1) / 1e6,
                     "grouping": "independent same-shape layers run up to four per launch",
                     "calls": gemm_calls, "timed_in": gemm_how,
                     "per_op_tflops": per_op},
        "update": {"kernel": "mp_master_update_kernel", "bound": "hbm", "achieved": upd_gbs,
                   "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": upd_gbs / pk["hbm_gbs"],
                   "frac_of_nominal_8000": upd_gbs / 8000.0, "bytes_per_param": bytes_per_param,
                   "algorithmic_bytes_per_launch": upd_bytes,
                   "avg_launch_ms": upd_ms_alone, "peak_source": pk_src + " copy",
                   "timed_in": ("the step's update call alone, launched back to back (the kernel outlasts the host's "
                                "call, so the launches queue without gaps) after settling launches"
                                if upd_only is not None else timed_how),
                   "in_step": {"avg_launch_ms": upd_ms_in_step, "achieved": upd_bytes / (upd_ms_in_step * 1e-3) / 1e9,
                               "note": "between event nodes inside the step, right after the products"},
                   "traffic": (NCU_UPDATE_TRAFFIC["bytes_per_param"] * cfg.n_params()
                               if NCU_UPDATE_TRAFFIC["sha"] == update_kernel_sha() and cfg.optimizer == "adam" else None)},
        # device time per call class per step from the event-timed region (sum over the step's
        # calls; every call's interval is stretched by its two event nodes, a few microseconds)
        "breakdown_timed_in": timed_how,
        "breakdown_ms_per_step": {k: sum(v) / steps for k, v in sorted(per.items())},
        "clocks": None,
        "clocks_by_region": clk,
    }
    if ms_e2e is not None:
        out["e2e"] = {"value": world * flops_step / (ms_e2e / steps * 1e-3) / 1e12, "unit": "TFLOP/s",
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps,
                      "feed": "two staging sets: batch i+1 is copied from pinned host memory while batch i runs"}
    if sampler is not None:
        dev_windows = [w for k, w in windows.items() if k != "e2e"]
        c = sampler.summary(dev_windows)
        c["regions"] = "median over the device-timed regions (step, products, update); the PCIe-bound e2e region apart"
        out["clocks"] = c
    if rank == 0 and world == 1 and full and not args.no_cpu_baseline:
        from oracle import mp_oracle as orc
        orc.build()
        out["cpu_baseline"] = cpu_baseline_of(orc, synth, cfg, 12.0)
    stack.close()
    del stack, xs, gs, g_flat
    torch.cuda.empty_cache()
    return out


def cfg_gemm_bytes(cfg):
    """Algorithmic bytes of one step's products: every operand read once, every output written once."""
    return sum(2 * (3 * (m * k + k * n + m * n)) for m, k, n in cfg.shapes)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=None, choices=["c2", "c3", "c4", "c5"],
                    help="time this workload only (default: c2 at the top level, c3, c4 and c5 under `workloads`)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--settle", type=float, default=2.0,
                    help="seconds of untimed replays before each device-timed region (0: none; the roofline "
                         "then divides by the burst peak)")
    ap.add_argument("--real-layers", action="store_true",
                    help="biases on every layer and an activation inside every chain (ReLU; clipped ReLU for c4)")
    ap.add_argument("--per-shape", action="store_true",
                    help="time each distinct layer shape's three products alone, beside torch.matmul")
    ap.add_argument("--shard-update", action="store_true",
                    help="several GPUs: reduce-scatter the gradients, update a 1/N slice of the master per rank, "
                         "all-gather the FP16 weights (default: all-reduce and a replicated update)")
    ap.add_argument("--overlap-wgrad", default="auto", choices=["auto", "on", "off"],
                    help="weight gradients on a second stream beside the data gradients (auto: stacks with chained layers)")
    ap.add_argument("--max-params", type=float, default=1e9, help="c5: largest parameter count of the sweep")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if args.workload == "c5":
        if rank == 0:
            print(json.dumps(run_update_sweep(args, settle_s=min(1.0, args.settle))))
        return
    if args.per_shape:
        args.workload = args.workload or "c2"
        return run_per_shape(args)

    from paper_1805_10387_b200 import mp
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mp.lib()
    sampler = None
    if rank == 0:
        sampler = ClockSampler(local)
        sampler.start()
        time.sleep(0.3)
    main_wl = args.workload or "c2"
    out = run_stack(args, main_wl, args.steps, sampler, dist, full=True)
    if args.workload is None and world == 1:
        # the other workloads, fewer steps, device-timed regions only
        others = {}
        n = max(20, args.steps // 4)
        for wl in ("c3", "c4"):
            o = run_stack(args, wl, n, sampler, dist, full=False)
            others[wl] = {k: o[k] for k in ("value", "unit", "steps", "ms_per_step", "config", "gpu_launches",
                                            "skipped_steps_in_timed_region", "loss_scale", "roofline", "update",
                                            "breakdown_ms_per_step", "clocks")}
        o = run_update_sweep(args, sampler, steps=n, settle_s=min(1.0, args.settle))
        others["c5"] = {k: o[k] for k in ("value", "unit", "ms_per_step", "config", "gpu_launches", "roofline",
                                          "sweep", "clocks")}
        out["workloads"] = others
        out["gpu_launches_all_workloads"] = int(out["gpu_launches"] + sum(w["gpu_launches"] for w in others.values()))
    if sampler is not None:
        sampler.stop()
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
