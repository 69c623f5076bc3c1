"""Pins of the oracle's stochastic rounding (second rounding mode of the Methodology section)
and of the generator that feeds it."""
import os

import numpy as np
import pytest

import oracle
from oracle.rng import element_uniforms, philox4x32_10

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
FMTS = ["int8", "e4m3", "e5m2"]


def f32(a):
    return np.asarray(a, dtype=np.float32)


def test_philox_known_answers():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for w in rows:
        v = [int(x, 16) for x in w]
        out = philox4x32_10(*[np.array([c], np.uint32) for c in v[:4]], v[4], v[5])
        assert [int(o[0]) for o in out] == v[6:]


def test_uniforms_are_numbered_by_element_and_word():
    u = element_uniforms((2, 5), seed=(7 << 32) | 9, stream=3)
    blk0 = philox4x32_10(*[np.array([c], np.uint32) for c in (0, 0, 3, 0)], 9, 7)
    blk2 = philox4x32_10(*[np.array([c], np.uint32) for c in (2, 0, 3, 0)], 9, 7)
    assert u[0, 1] == (int(blk0[1][0]) >> 8) / 2 ** 24          # element 1 -> block 0, word 1
    assert u[1, 4] == (int(blk2[1][0]) >> 8) / 2 ** 24          # element 9 -> block 2, word 1
    assert u.min() >= 0.0 and u.max() < 1.0
    big = element_uniforms((200_000,), 1, 0)
    assert abs(big.mean() - 0.5) < 0.005 and abs((big < 0.25).mean() - 0.25) < 0.005
    assert not np.array_equal(big, element_uniforms((200_000,), 2, 0))
    assert not np.array_equal(big, element_uniforms((200_000,), 1, 1))


@pytest.mark.parametrize("fmt", FMTS)
def test_grid_values_never_move_and_results_are_neighbours(fmt):
    g = oracle.positive_grid(fmt)
    vals = f32(np.concatenate([g, -g]))[None, :]
    one = f32([1.0])
    assert np.array_equal(oracle.quantize(vals, fmt, one, "stochastic", 5, 0), oracle.quantize(vals, fmt, one))
    rng = np.random.default_rng(3)
    t = f32(rng.uniform(-1.2, 1.2, (40, 500)) * oracle.qmax(fmt))
    q = oracle.dequantize(oracle.quantize(t, fmt, one, "stochastic", 11, 0), fmt)
    a = np.minimum(np.abs(t.astype(np.float64)), g[-1])
    lo = g[np.searchsorted(g, a, side="right") - 1]
    hi = g[np.minimum(np.searchsorted(g, a, side="right"), len(g) - 1)]
    assert np.all((np.abs(q) == lo) | (np.abs(q) == hi))
    assert np.all(np.sign(q) * np.sign(t) >= 0)
    assert np.abs(q).max() == oracle.qmax(fmt)                    # saturation, never beyond


@pytest.mark.parametrize("fmt,t0,lo,hi", [("int8", 2.25, 2.0, 3.0), ("int8", -7.9, 7.0, 8.0),
                                          ("e4m3", 1.03125, 1.0, 1.125), ("e5m2", 2.0 ** -17, 0.0, 2.0 ** -16),
                                          ("e4m3", 300.0, 288.0, 320.0)])
def test_round_up_frequency_is_the_distance_fraction(fmt, t0, lo, hi):
    n = 200_000
    t = f32(np.full((1, n), t0))
    q = np.abs(oracle.dequantize(oracle.quantize(t, fmt, f32([1.0]), "stochastic", 21, 0), fmt))
    p = (abs(t0) - lo) / (hi - lo)
    up = (q == hi).mean()
    assert set(np.unique(q)) <= {lo, hi}
    assert abs(up - p) < 4 * (p * (1 - p) / n) ** 0.5 + 1e-9
    assert abs(q.mean() - abs(t0)) < 4 * (hi - lo) * (p * (1 - p) / n) ** 0.5 + 1e-12   # unbiased


def test_unbiased_where_rtne_is_not():
    # many small equal gradients: RTNE maps all of them to 0, stochastic rounding keeps the mean
    x = f32(np.full((1, 100_000), 0.2))
    x[0, 0] = 127.0                                               # fixes delta = 1
    rt = oracle.dequantize(oracle.quantize(x, "int8", oracle.scale(x, "int8", "tensor")), "int8")
    sr = oracle.dequantize(oracle.quantize(x, "int8", oracle.scale(x, "int8", "tensor"), "stochastic", 1, 0), "int8")
    assert rt[0, 1:].sum() == 0.0
    assert sr[0, 1:].mean() == pytest.approx(0.2, rel=0.03)


def test_sign_symmetry_and_seed_dependence():
    rng = np.random.default_rng(4)
    x = f32(rng.standard_normal((3, 64, 40)))
    d = oracle.scale(x, "e5m2", "channel")
    a = oracle.dequantize(oracle.quantize(x, "e5m2", d, "stochastic", 9, 0), "e5m2")
    b = oracle.dequantize(oracle.quantize(-x, "e5m2", d, "stochastic", 9, 0), "e5m2")
    assert np.array_equal(a, -b)                                  # same draw, mirrored value
    c = oracle.quantize(x, "e5m2", d, "stochastic", 10, 0)
    assert not np.array_equal(oracle.quantize(x, "e5m2", d, "stochastic", 9, 0), c)
    assert not np.array_equal(oracle.quantize(x, "e5m2", d, "stochastic", 9, 1),
                              oracle.quantize(x, "e5m2", d, "stochastic", 9, 0))


def test_probe_with_stochastic_gradient_operand():
    rng = np.random.default_rng(6)
    X = f32(rng.standard_normal((96, 64)))
    dY = f32(np.exp(rng.normal(-9, 2, (64, 48))) * rng.choice([-1, 1], (64, 48)))   # log-normal magnitudes
    rt = oracle.probe(X, dY, "int8", "int8", "tensor", "tensor")
    sr = oracle.probe(X, dY, "int8", "int8", "tensor", "tensor", round_r="stochastic", seed=3)
    full = oracle.probe(X, dY, "int8", "int8", "tensor", "tensor", round_r="stochastic", seed=3, full=True)[1]
    assert np.array_equal(full["codes_r"], oracle.quantize(np.swapaxes(dY, -1, -2), "int8", full["delta_r"], "stochastic", 3, 1))
    assert sr["count"] == rt["count"] and sr["sum_den2"] == rt["sum_den2"] and sr["sum_ref2"] == rt["sum_ref2"]
    assert sr["sum_be"] != rt["sum_be"]
    # row sampling numbers the draws over the whole operand
    rows = np.array([3, 50, 95])
    part = oracle.probe(X, dY, "int8", "int8", "tensor", "tensor", rows=rows, round_l="stochastic", seed=8, full=True)[1]
    whole = oracle.probe(X, dY, "int8", "int8", "tensor", "tensor", round_l="stochastic", seed=8, full=True)[1]
    assert np.array_equal(part["codes_l"], whole["codes_l"][rows])
