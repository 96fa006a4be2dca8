"""Pins for the oracle's e4m3fn codec: format definition, hand-worked examples,
brute-force nearest-value search, and a third-party cast (torch CPU)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import read_golden_table

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def definition_value(code):
    """e4m3fn value straight from the bit-field definition (test-side copy of the
    format, written independently of the oracle's table)."""
    s = -1.0 if code & 0x80 else 1.0
    e = (code >> 3) & 0xF
    m = code & 7
    if e == 15 and m == 7:
        return math.nan
    if e == 0:
        return s * m * 2.0 ** -9
    return s * (1 + m / 8) * 2.0 ** (e - 7)


def test_decode_matches_definition_and_range():
    tab = oracle.e4m3_decode_table()
    for c in range(256):
        v = definition_value(c)
        if math.isnan(v):
            assert math.isnan(tab[c])
        else:
            assert tab[c] == v
    finite = tab[~np.isnan(tab)]
    assert finite.size == 254
    assert finite.max() == 448.0 and finite.min() == -448.0   # Eq. 2 range
    assert tab[0x7E] == 448.0 and tab[0xFE] == -448.0


def test_decode_matches_torch_cpu_cast():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    tab = oracle.e4m3_decode_table()
    ok = (tab == ref) | (np.isnan(tab) & np.isnan(ref))
    assert ok.all()


def test_round_trip_all_finite_codes():
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue
        assert oracle.e4m3_encode(oracle.e4m3_decode(c)) == c


def test_worked_examples():
    for expr, code in read_golden_table(os.path.join(GOLD, "e4m3_worked_examples.txt")):
        val = eval(expr, {"__builtins__": {}})
        assert oracle.e4m3_encode(val) == int(code, 16), (expr, code)


def test_saturation():
    for y in (448.0, 449.0, 1e30, math.inf):
        assert oracle.e4m3_encode(y) == 0x7E
        assert oracle.e4m3_encode(-y) == 0xFE


def brute_force_encode(y):
    """Nearest finite grid value by exhaustive search; ties -> even mantissa."""
    best = None
    for c in range(127):
        v = definition_value(c)
        dist = abs(abs(y) - v)
        if best is None or dist < best[0] or (dist == best[0] and (c & 1) == 0):
            if best is None or dist < best[0] or (dist == best[0] and (best[1] & 1) == 1):
                best = (dist, c)
    return best[1] | (0x80 if math.copysign(1.0, y) < 0 else 0)


def test_encode_vs_brute_force_on_midpoints_and_neighbours():
    vals = []
    grid = [definition_value(c) for c in range(127)]
    for a, b in zip(grid[:-1], grid[1:]):
        mid = (a + b) / 2
        vals += [a, mid, np.nextafter(np.float32(mid), np.float32(0)).item(),
                 np.nextafter(np.float32(mid), np.float32(1e9)).item(),
                 a + (b - a) * 0.25, a + (b - a) * 0.75]
    vals.append(448.0)
    for v in vals:
        for s in (1.0, -1.0):
            assert oracle.e4m3_encode(s * v) == brute_force_encode(s * v), v


def test_encode_array_vs_torch_cast_random():
    rng = np.random.default_rng(0)
    y = np.concatenate([
        rng.standard_normal(400000).astype(np.float32) * 100,
        rng.standard_normal(400000).astype(np.float32),
        rng.standard_normal(200000).astype(np.float32) * 1e-2,
        (rng.integers(-448 * 16, 448 * 16, 200000) / 16).astype(np.float32),  # many exact ties
    ])
    y = np.clip(y, -448, 448)
    got = oracle.e4m3_encode_array(y)
    ref = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, ref)
    assert not np.any((got & 0x7F) == 0x7F)     # never NaN codes
