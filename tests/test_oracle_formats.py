"""Pins for the oracle's format tables (Methodology section: INT8 / E4M3 / E5M2)."""
import os

import ml_dtypes
import numpy as np
import pytest

from oracle import decode_table, positive_grid, qmax

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_printed_maxima():
    # values printed by the paper, stored with their citation in the fixture
    want = {}
    for line in open(os.path.join(GOLDEN, "format_maxima.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            want[k] = float(v)
    assert set(want) == {"e4m3", "e5m2", "int8"}
    for fmt, v in want.items():
        assert qmax(fmt) == v
        t = decode_table(fmt)
        assert np.nanmax(np.where(np.isfinite(t), t, np.nan)) == v
        assert np.nanmin(np.where(np.isfinite(t), t, np.nan)) == (-v if fmt != "int8" else -128)


def test_cardinalities():
    t = decode_table("e4m3")
    assert np.isfinite(t).sum() == 254 and np.isnan(t).sum() == 2 and np.isinf(t).sum() == 0
    t = decode_table("e5m2")
    assert np.isfinite(t).sum() == 248 and np.isinf(t).sum() == 2 and np.isnan(t).sum() == 6
    t = decode_table("int8")
    assert np.isfinite(t).sum() == 256 and len(np.unique(t)) == 256
    assert len(positive_grid("int8")) == 128
    assert len(positive_grid("e4m3")) == 127     # 0x00..0x7E
    assert len(positive_grid("e5m2")) == 124     # 0x00..0x7B


def test_landmarks():
    # EeMm with bias: smallest subnormal 2^(1-bias-m), smallest normal 2^(1-bias)
    g = positive_grid("e4m3")
    assert g[0] == 0 and g[1] == 2.0 ** -9 and g[8] == 2.0 ** -6 and g[0x38] == 1.0
    assert g[0x7E] == 448.0 and g[0x78] == 256.0
    g = positive_grid("e5m2")
    assert g[0] == 0 and g[1] == 2.0 ** -16 and g[4] == 2.0 ** -14 and g[0x3C] == 1.0
    assert g[0x7B] == 57344.0
    t = decode_table("int8")
    assert t[0x7F] == 127 and t[0x80] == -128 and t[0xFF] == -1 and t[0x81] == -127


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_sign_symmetry_and_spacing(fmt):
    t = decode_table(fmt)
    for c in range(128):
        if np.isfinite(t[c]):
            assert t[c + 128] == -t[c]
    g = positive_grid(fmt)
    m = 3 if fmt == "e4m3" else 2
    # inside a binade spacing is constant, and doubles from one binade to the next
    d = np.diff(g)
    per = 1 << m
    assert np.all(d[:per] == d[0])                      # subnormals and first normals share a step
    for b in range(1, (len(g) - 1) // per - 1):
        assert np.all(d[b * per:(b + 1) * per] == d[b * per])
        if b >= 2:
            assert d[b * per] == 2 * d[(b - 1) * per]


@pytest.mark.parametrize("fmt,dt", [("e4m3", ml_dtypes.float8_e4m3fn), ("e5m2", ml_dtypes.float8_e5m2)])
def test_decode_against_outside_library(fmt, dt):
    # an implementation that is not ours: ml_dtypes' view of the same bytes
    lib = np.arange(256, dtype=np.uint8).view(dt).astype(np.float64)
    ours = decode_table(fmt)
    assert np.array_equal(np.isnan(lib), np.isnan(ours))
    ok = ~np.isnan(lib)
    assert np.array_equal(lib[ok], ours[ok])
