"""Pins for the oracle's building blocks: series log2/exp2 and Philox4x32-10."""
import math
import os

import numpy as np
import pytest

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_log2_matches_libm_to_rounding():
    rng = np.random.default_rng(1)
    vals = np.concatenate([
        10.0 ** rng.uniform(-300, 300, 2000),
        rng.uniform(1.0, 2.0, 2000),
        np.array([1.0, 2.0, 4.0, 0.5, 3.0, 1.4142135623730951, 1.4142135623730954, 2.0 ** 31, 1e8 + 1]),
    ])
    for v in vals:
        got, ref = O.log2(float(v)), math.log2(float(v))
        assert abs(got - ref) <= 4e-16 * max(1.0, abs(ref)), (v, got, ref)
    # exact at powers of two (t = 0 exactly): the planner relies on E(0) = 0
    for e in range(-100, 101):
        assert O.log2(2.0 ** e) == float(e)


def test_exp2_matches_pow_to_rounding():
    rng = np.random.default_rng(2)
    for v in np.concatenate([rng.uniform(-1000, 1000, 3000), rng.uniform(-1, 1, 1000)]):
        got, ref = O.exp2(float(v)), 2.0 ** float(v)
        assert abs(got / ref - 1.0) <= 1e-15, (v, got, ref)
    for n in range(-1000, 1001, 7):
        assert O.exp2(float(n)) == 2.0 ** n


def test_powr_inverse_and_identity():
    assert O.powr(1.0, -0.75) == 1.0
    rng = np.random.default_rng(3)
    for _ in range(500):
        a = float(rng.integers(1, 2 ** 31))
        beta = float(rng.uniform(-7, 1))
        ref = a ** beta
        assert abs(O.powr(a, beta) / ref - 1.0) < 1e-13


def _read_kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], tuple(w[6:10])))
    return rows


def test_philox_known_answers():
    rows = _read_kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert O.philox4x32_10(ctr, key) == out


def test_philox_coord_wiring():
    # counter = (coord lo, coord hi, client, round); key = (seed lo, seed hi); word 0
    seed, client, rnd, coord = 0x299F31D0A4093822, 0x13198A2E, 0x03707344, 0x85A308D3243F6A88
    assert O.philox_coord(seed, client, rnd, coord) == 0xD16CFE09
    assert O.philox_coord(0, 0, 0, 0) == 0x6627E8D5


def test_philox_uniformity():
    n = 1 << 16
    u = np.array([O.philox_coord(12345, 3, 1, i) for i in range(n)], dtype=np.float64) / 2.0 ** 32
    assert abs(u.mean() - 0.5) < 4.0 / math.sqrt(12 * n)
    assert abs(u.var() - 1.0 / 12.0) < 0.002
    # different clients / rounds / seeds decorrelate
    v = np.array([O.philox_coord(12345, 4, 1, i) for i in range(4096)], dtype=np.float64) / 2.0 ** 32
    assert abs(np.corrcoef(u[:4096], v)[0, 1]) < 0.06
    bits = np.array([O.philox_coord(7, 0, 0, i) for i in range(4096)], dtype=np.uint64)
    for b in range(32):
        frac = ((bits >> np.uint64(b)) & np.uint64(1)).mean()
        assert 0.45 < frac < 0.55
