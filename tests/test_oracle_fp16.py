"""Pins for the oracle's software FP16 (binary16 <-> binary32).

The expected values come from the IEEE 754 format definition evaluated in Python
doubles, from hand-derived thresholds (tests/golden/fp16_thresholds.txt) and from
numpy's independent float16 conversion; none comes from the oracle itself.
"""
import math
import os
import struct

import numpy as np

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _closed_form(h: int) -> float:
    s = -1.0 if h & 0x8000 else 1.0
    e = (h >> 10) & 0x1F
    f = h & 0x3FF
    if e == 0x1F:
        return s * math.inf if f == 0 else math.nan
    if e == 0:
        return s * (f / 1024.0) * 2.0 ** -14
    return s * (1.0 + f / 1024.0) * 2.0 ** (e - 15)


def test_h2f_exhaustive_closed_form(orc):
    h = np.arange(65536, dtype=np.uint16)
    got = orc.h2f(h).astype(np.float64)
    counts = {"zero": 0, "inf": 0, "nan": 0, "sub": 0, "normal": 0}
    for i in range(65536):
        want = _closed_form(i)
        if math.isnan(want):
            assert math.isnan(got[i]), i
            counts["nan"] += 1
            continue
        assert got[i] == want, (hex(i), got[i], want)
        assert math.copysign(1.0, got[i]) == math.copysign(1.0, want), hex(i)
        e, f = (i >> 10) & 0x1F, i & 0x3FF
        if math.isinf(want):
            counts["inf"] += 1
        elif e == 0 and f == 0:
            counts["zero"] += 1
        elif e == 0:
            counts["sub"] += 1
        else:
            counts["normal"] += 1
    assert counts == {"zero": 2, "inf": 2, "nan": 2046, "sub": 2046, "normal": 61440}


def test_h2f_matches_library(orc):
    h = np.arange(65536, dtype=np.uint16)
    got = orc.h2f(h)
    ref = h.view(np.float16).astype(np.float32)
    same = (got.view(np.uint32) == ref.view(np.uint32)) | (np.isnan(got) & np.isnan(ref))
    assert same.all()


def test_f2h_round_trip_exhaustive(orc):
    h = np.arange(65536, dtype=np.uint16)
    f = orc.h2f(h)
    back = orc.f2h(f)
    finite_or_inf = ~np.isnan(f)
    assert (back[finite_or_inf] == h[finite_or_inf]).all()
    nan_back = back[np.isnan(f)]
    assert ((nan_back & 0x7C00) == 0x7C00).all() and ((nan_back & 0x3FF) != 0).all()


def test_f2h_midpoints_and_neighbours(orc):
    """Between every adjacent pair of non-negative finite halves: the midpoint goes to the
    even neighbour, the floats just either side of it to the nearer neighbour."""
    lo_bits = np.arange(0, 0x7BFF, dtype=np.uint16)           # lo .. lo+1 both finite
    lo = _vals(lo_bits)
    hi = _vals(lo_bits + 1)
    mid = ((lo + hi) / 2.0).astype(np.float32)                 # exact: one extra bit
    assert (mid.astype(np.float64) == (lo + hi) / 2.0).all()
    even = np.where(lo_bits % 2 == 0, lo_bits, lo_bits + 1).astype(np.uint16)
    assert (orc.f2h(mid) == even).all()
    below = np.nextafter(mid, np.float32(0))
    above = np.nextafter(mid, np.float32(np.inf))
    assert (orc.f2h(below) == lo_bits).all()
    assert (orc.f2h(above) == lo_bits + 1).all()
    # same on the negative side
    assert (orc.f2h(-mid) == (even | 0x8000)).all()
    assert (orc.f2h(-below) == (lo_bits | 0x8000)).all()


def _vals(bits):
    return np.array([_closed_form(int(b)) for b in bits], np.float64)


def test_f2h_golden_thresholds(orc):
    n = 0
    for line in open(os.path.join(GOLD, "fp16_thresholds.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        x = struct.unpack("<f", struct.pack("<I", int(line[0], 16)))[0]
        got = int(orc.f2h(np.array([x], np.float32))[0])
        assert got == int(line[1], 16), (line, hex(got))
        n += 1
    assert n >= 15


def test_f2h_matches_library_on_random_and_special(orc):
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2 ** 32, size=2_000_000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[~np.isnan(x)]
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    assert (orc.f2h(x) == want).all()
    # dense sweep across the half range, where random bit patterns are sparse
    y = (rng.standard_normal(1_000_000) * np.exp(rng.uniform(-20, 12, 1_000_000))).astype(np.float32)
    with np.errstate(over="ignore"):
        assert (orc.f2h(y) == y.astype(np.float16).view(np.uint16)).all()


def test_f2h_nan_and_overflow_never_saturate(orc):
    out = orc.f2h(np.array([np.nan, 1e30, -1e30, 65519.996, 70000.0], np.float32))
    assert (out[0] & 0x7C00) == 0x7C00 and (out[0] & 0x3FF) != 0
    assert list(out[1:]) == [0x7C00, 0xFC00, 0x7BFF, 0x7C00]


def test_weight_decay_product_underflows_in_fp16_not_fp32(orc):
    """Section 3.3: a decay coefficient of 1e-5 times a small FP16 weight is lost in FP16."""
    w16 = orc.f2h(np.array([1e-3], np.float32))
    w = orc.h2f(w16)[0]
    prod32 = np.float32(1e-5) * w
    assert prod32 != 0.0
    assert int(orc.f2h(np.array([prod32], np.float32))[0]) == 0
