"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers and names shapes; it holds none of the method's
arithmetic (no matmul, no optimizer, no loss-scale logic) and is the one module
that both the CPU oracle's tests and the CUDA path's tests read.

Generator: counter based.  Element i of stream (seed, stream_id) is
Box-Muller(u1, u2) with u1, u2 taken from splitmix64(key + 2i) and
splitmix64(key + 2i + 1), so any slice can be drawn without drawing the rest.
The paper trains on WMT16 En-De and LibriSpeech (Sections 5.1, 5.2); these inputs
stand in for them and imitate only the dense-layer shapes and value scales.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = x
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _splitmix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], np.uint64))
        k = _splitmix64(k ^ np.array([(stream * 0x632BE59BD9B4E019) & 0xFFFFFFFFFFFFFFFF], np.uint64))
    return k[0]


def uniform01(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in (0,1), elements offset..offset+n-1 of the stream."""
    with np.errstate(over="ignore"):
        idx = np.arange(offset, offset + n, dtype=np.uint64) + _key(seed, stream)
        bits = _splitmix64(idx)
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, stream: int, n: int, offset: int = 0, chunk: int = 1 << 22) -> np.ndarray:
    """n standard normals (float64), elements offset..offset+n-1 of the stream."""
    out = np.empty(n, np.float64)
    for lo in range(0, n, chunk):
        c = min(chunk, n - lo)
        u = uniform01(seed, stream, 2 * c, 2 * (offset + lo))
        r = np.sqrt(-2.0 * np.log(u[0::2]))
        out[lo:lo + c] = r * np.cos(2.0 * np.pi * u[1::2])
    return out


def fp16_bits(x: np.ndarray) -> np.ndarray:
    """Storage format of generated FP16 inputs: IEEE binary16 bit patterns."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


# stream ids: (layer, tensor kind, step) -> one integer
_X, _W, _G, _AUX = 0, 1, 2, 3


def stream_id(layer: int, kind: int, step: int = 0) -> int:
    return (step * 4096 + layer) * 4 + kind


@dataclass
class StackConfig:
    """One of the workload recipes.  Shapes are (M rows, K in, N out) per layer."""
    name: str
    seed: int
    shapes: list                     # [(M,K,N), ...]
    optimizer: str = "adam"
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    momentum: float = 0.9
    grad_std: float = 1e-2           # std of the upstream FP32 gradient
    init_scale: float = 65536.0
    growth_interval: int = 1000
    x_dist: str = "normal"           # "normal" | "lognormal2"
    steps: int = 3
    inject_inf_step: int = -1        # 0-based step whose top gradient gets a +inf
    note: str = ""
    chain: list = field(default_factory=list)   # per layer: reads the previous layer's output

    def chained(self, l: int) -> bool:
        """Layer l reads layer l-1's output (needs matching widths and rows).  Without an
        explicit `chain` list every layer whose input width equals the previous output width
        is chained."""
        fits = l > 0 and self.shapes[l][1] == self.shapes[l - 1][2] and \
            self.shapes[l][0] == self.shapes[l - 1][0]
        return fits and (self.chain[l] if self.chain else True)

    def feeds_next(self, l: int) -> bool:
        return l + 1 < len(self.shapes) and self.chained(l + 1)

    def n_params(self) -> int:
        return sum(k * n for _, k, n in self.shapes)

    def gemm_flops(self) -> int:
        """fwd + dgrad + wgrad, 2MKN each."""
        return sum(3 * 2 * m * k * n for m, k, n in self.shapes)


def config(name: str) -> StackConfig:
    """The four GEMM workloads.  'N(0,x)' in the workload list is read as variance x."""
    if name == "c1":      # tiny chained stack, Adam, inf injected at step index 4
        return StackConfig("c1", 0, [(32, 256, 256)] * 2, grad_std=1e-2, init_scale=2.0 ** 16,
                           growth_interval=4, steps=10, inject_inf_step=4,
                           note="tiny 2-layer stack 256->256->256, 32 rows")
    if name == "c2":      # GNMT-like LSTM gate GEMMs: [x;h] 2048 -> 4 gates x 1024
        return StackConfig("c2", 1, [(6400, 2048, 4096)] * 8, lr=8e-4, grad_std=10 ** -2.5,
                           note="8 layers, 128x50 tokens, 2048->4096; lr from the paper's listing")
    if name == "c3":      # Transformer-big FFN pair + 4 attention projections per block
        blk = [(8192, 1024, 4096), (8192, 4096, 1024)] + [(8192, 1024, 1024)] * 4
        # only the FFN pair is chained; the four attention projections are independent layers
        return StackConfig("c3", 2, blk * 6, grad_std=10 ** -2.5, init_scale=2.0 ** 15,
                           chain=[False, True, False, False, False, False] * 6,
                           note="6 blocks x (FFN 1024->4096->1024 + 4 proj 1024x1024), 8192 tokens")
    if name == "c4":      # DeepSpeech2-like dense stack, momentum SGD, heavy-tailed inputs
        return StackConfig("c4", 3, [(25600, 1600, 1600)] * 5 + [(25600, 1600, 29)],
                           optimizer="momentum", lr=1e-7, grad_std=1e-3, x_dist="lognormal2",
                           note="5 x 1600->1600 over 64x400 frames + 1600->29")
    raise KeyError(name)


def weights(cfg: StackConfig, l: int) -> np.ndarray:
    """FP32 master initialisation, N(0, 1/fan_in)."""
    _, k, n = cfg.shapes[l]
    return (normal(cfg.seed, stream_id(l, _W), k * n) / np.sqrt(k)).astype(np.float32).reshape(k, n)


def activations(cfg: StackConfig, l: int, step: int) -> np.ndarray:
    """FP16 bits [M,K] for a layer that is not chained."""
    m, k, _ = cfg.shapes[l]
    z = normal(cfg.seed, stream_id(l, _X, step), m * k)
    if cfg.x_dist == "lognormal2":
        s = np.where(uniform01(cfg.seed, stream_id(l, _AUX, step), m * k) < 0.5, -1.0, 1.0)
        z = s * np.minimum(np.exp(2.0 * z), 6.0e4)
    return fp16_bits(z.astype(np.float32)).reshape(m, k)


def upstream(cfg: StackConfig, l: int, step: int) -> np.ndarray:
    """FP32 unscaled gradient [M,N] entering layer l from above."""
    m, _, n = cfg.shapes[l]
    g = (normal(cfg.seed, stream_id(l, _G, step), m * n) * cfg.grad_std).astype(np.float32)
    g = g.reshape(m, n)
    if step == cfg.inject_inf_step and not cfg.feeds_next(l) and l == len(cfg.shapes) - 1:
        g[0, 0] = np.inf
    return g


# ------------------------------------------------------- update-only sweep
@dataclass
class UpdateSweep:
    """Update-only workload: P parameters in n tensors of log-uniform sizes."""
    P: int
    n_tensors: int
    seed: int = 4
    grad_std: float = 10 ** -1.5      # N(0, 1e-3) read as variance
    init_scale: float = 65536.0
    growth_interval: int = 10
    p_overflow: float = 0.01
    forced_overflow_step: int = 3
    counts: list = field(default_factory=list)

    def __post_init__(self):
        if not self.counts:
            self.counts = tensor_sizes(self.P, self.n_tensors, self.seed)


def tensor_sizes(P: int, n: int, seed: int) -> list:
    """n sizes, each >= 1, log-uniform over four decades, rescaled to sum to P."""
    if n == 1:
        return [P]
    raw = np.exp(uniform01(seed, 777, n) * np.log(1e4))
    sizes = np.maximum(1, np.floor(raw / raw.sum() * (P - n)).astype(np.int64) + 1)
    sizes[-1] += P - int(sizes.sum())
    assert sizes.min() >= 1 and int(sizes.sum()) == P
    return [int(s) for s in sizes]


def overflow_steps(sw: UpdateSweep, steps: int) -> list:
    """0/1 per step: a non-finite gradient element is planted on these steps."""
    u = uniform01(sw.seed, 778, steps)
    return [int(u[s] < sw.p_overflow or s == sw.forced_overflow_step) for s in range(steps)]
