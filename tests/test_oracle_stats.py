"""Pins of oracle/stats.py against things other than itself: closed forms, scipy's routines,
hand-worked examples and identities (Experiments section statistics; Eq. 2 and the clipping /
rounding split of the Results section)."""
import math

import numpy as np
import pytest
from scipy import stats as sps

import oracle


def f32(a):
    return np.asarray(a, dtype=np.float32)


# ------------------------------------------------------------------ tensor statistics
def test_moments_of_one_to_five_by_hand():
    s = oracle.tensor_stats(f32([[1, 2, 3], [4, 5, 3]])[:, :])   # 1,2,3,4,5,3
    # mean 3; deviations -2,-1,0,1,2,0 -> m2 = 10/6, m3 = 0, m4 = 34/6
    assert s["count"] == 6 and s["max_abs"] == 5.0
    assert s["mean"] == pytest.approx(3.0, abs=1e-15)
    assert s["variance"] == pytest.approx(10 / 6, rel=1e-14)
    assert s["skew"] == pytest.approx(0.0, abs=1e-14)
    assert s["kurtosis"] == pytest.approx((34 / 6) / (10 / 6) ** 2, rel=1e-14)
    assert (s["sum1"], s["sum2"], s["sum3"], s["sum4"]) == (18.0, 64.0, 252.0, 1060.0)


def test_skewed_hand_example_sign_and_value():
    # 0,0,0,4: mean 1, deviations -1,-1,-1,3 -> m2 = 3, m3 = 6, m4 = 21
    s = oracle.tensor_stats(f32([0, 0, 0, 4]))
    assert s["variance"] == pytest.approx(3.0) and s["skew"] == pytest.approx(6 / 3 ** 1.5)
    assert s["kurtosis"] == pytest.approx(21 / 9)
    # mirrored data flips the sign of the skew only
    m = oracle.tensor_stats(f32([0, 0, 0, -4]))
    assert m["skew"] == pytest.approx(-s["skew"]) and m["kurtosis"] == pytest.approx(s["kurtosis"])
    assert m["max_abs"] == 4.0


def test_against_scipy_and_closed_form_laws():
    rng = np.random.default_rng(5)
    for x, skew, kurt in ((rng.standard_normal(400_000), 0.0, 3.0),
                          (rng.exponential(2.0, 400_000), 2.0, 9.0),
                          (rng.uniform(-1, 3, 400_000), 0.0, 1.8)):
        x = f32(x).reshape(400, 1000)
        s = oracle.tensor_stats(x)
        v = x.astype(np.float64).ravel()
        assert s["mean"] == pytest.approx(v.mean(), rel=1e-12, abs=1e-15)
        assert s["variance"] == pytest.approx(v.var(), rel=1e-12)
        assert s["skew"] == pytest.approx(sps.skew(v), rel=1e-9, abs=1e-12)
        assert s["kurtosis"] == pytest.approx(sps.kurtosis(v, fisher=False), rel=1e-9)
        assert s["skew"] == pytest.approx(skew, abs=0.1) and s["kurtosis"] == pytest.approx(kurt, rel=0.1)


def test_shift_and_scale_laws():
    rng = np.random.default_rng(6)
    x = f32(rng.gamma(2.0, 1.0, 5000))
    a = oracle.tensor_stats(x)
    b = oracle.tensor_stats(f32(4.0 * x.astype(np.float64)))      # exact in float32
    assert b["mean"] == pytest.approx(4 * a["mean"], rel=1e-12)
    assert b["variance"] == pytest.approx(16 * a["variance"], rel=1e-12)
    assert b["skew"] == pytest.approx(a["skew"], rel=1e-10) and b["kurtosis"] == pytest.approx(a["kurtosis"], rel=1e-10)
    assert b["sum4"] == pytest.approx(256 * a["sum4"], rel=1e-12)


def test_degenerate_tensors():
    assert oracle.tensor_stats(f32(np.zeros((0, 4))))["count"] == 0
    c = oracle.tensor_stats(f32(np.full((3, 4), 2.5)))
    assert c["variance"] == 0.0 and c["skew"] == 0.0 and c["kurtosis"] == 0.0 and c["mean"] == 2.5


# ------------------------------------------------------------------ Eq. 2 and its split
def test_int8_hand_example():
    # amax 127 -> delta 1: codes are the rounded values; 0.4 underflows, 0.5 ties to 0, 1.5 -> 2
    x = f32([[127.0, 0.4, -0.5, 1.5, 0.0, 2.25, -100.0, 64.5]])
    r = oracle.quantize_error(x, "int8", "tensor")
    assert (r["count"], r["n_nonzero"], r["n_overflow"], r["n_underflow"]) == (8, 7, 0, 2)
    # rounding class: 127 (0), 1.5 -> 2 (1/3), 2.25 -> 2 (1/9), -100 (0), 64.5 -> 64 (0.5/64.5)
    want = 1 / 3 + 1 / 9 + 0.5 / 64.5
    assert r["sum_re_round"] == pytest.approx(want, rel=1e-12)
    assert r["sum_re"] == pytest.approx(want + 2.0, rel=1e-12)      # each underflow has RE = 1
    assert r["max_re_round"] == pytest.approx(1 / 3, rel=1e-12)
    assert r["err2_underflow"] == pytest.approx(0.4 ** 2 + 0.25, rel=1e-6)
    assert r["err2_round"] == pytest.approx(0.25 + 0.0625 + 0.25, rel=1e-12)
    assert r["err2_overflow"] == 0.0


def test_overflow_needs_an_outside_scale_and_is_capped():
    x = f32([[1000.0, -3.0, 500.0, 448.0, 449.0]])
    r = oracle.quantize_error(x, "e4m3", "tensor", delta=f32([1.0]))
    # 1000, 500 and 449 exceed 448 and are capped there; -3 and 448 are exact
    assert (r["n_overflow"], r["n_underflow"]) == (3, 0)
    assert r["err2_overflow"] == pytest.approx(552.0 ** 2 + 52.0 ** 2 + 1.0, rel=1e-12)
    assert r["sum_re"] == pytest.approx(552 / 1000 + 52 / 500 + 1 / 449, rel=1e-12)
    assert r["sum_re_round"] == 0.0 and r["err2_round"] == 0.0


def test_e4m3_hand_example_with_subnormals():
    # delta = 1: grid near 1 has spacing 1/8; smallest subnormal 2^-9, half of it underflows
    x = f32([[448.0, 1.0625, 2.0 ** -9, 2.0 ** -10, 2.0 ** -11, -1.1875]])
    r = oracle.quantize_error(x, "e4m3", "tensor")
    # 1.0625 ties between 1.0 and 1.125 -> even mantissa 1.0; 2^-10 ties between 0 and 2^-9 -> 0;
    # 2^-11 -> 0; -1.1875 ties between -1.125 (odd) and -1.25 (even) -> -1.25
    assert (r["n_overflow"], r["n_underflow"]) == (0, 2)
    assert r["sum_re_round"] == pytest.approx(0.0625 / 1.0625 + 0.0625 / 1.1875, rel=1e-12)
    assert r["err2_underflow"] == pytest.approx(2.0 ** -20 + 2.0 ** -22, rel=1e-12)


@pytest.mark.parametrize("fmt,mbits,min_normal", [("e4m3", 3, 2.0 ** -6), ("e5m2", 2, 2.0 ** -14)])
def test_rounding_re_bound_in_the_normal_range(fmt, mbits, min_normal):
    rng = np.random.default_rng(7)
    x = f32(np.exp(rng.uniform(math.log(min_normal), math.log(oracle.qmax(fmt)), 50_000)) * rng.choice([-1, 1], 50_000))
    r = oracle.quantize_error(x[None, :], fmt, "tensor", delta=f32([1.0]))
    assert r["n_overflow"] == 0 and r["n_underflow"] == 0
    # nearest of a grid with relative spacing 2^-m: RE <= 1 / (2^(m+1) + 1)
    assert r["max_re_round"] <= 1.0 / (2 ** (mbits + 1) + 1) + 1e-12
    assert r["max_re_round"] > 0.8 / (2 ** (mbits + 1) + 1)
    # log-uniform input: mean RE of RTNE on a 2^-m grid is about ln2 / 2^(m+2) * (1.5 / 2 ln 2) ~ 2^-m / 5.5
    assert r["sum_re_round"] / r["n_nonzero"] == pytest.approx(2.0 ** -mbits / 5.5, rel=0.1)


@pytest.mark.parametrize("fmt", ["int8", "e4m3", "e5m2"])
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_class_identities(fmt, gran):
    rng = np.random.default_rng(8)
    x = f32(rng.standard_t(3.0, (2, 33, 70)) * 10.0 ** rng.uniform(-4, 2, (2, 33, 1)))
    x[0, 3, :] = 0.0
    r = oracle.quantize_error(x, fmt, gran)
    d = oracle.scale(x, fmt, gran)
    vt = oracle.dequantize(oracle.quantize(x, fmt, d), fmt, d)
    v = x.astype(np.float64)
    assert r["n_nonzero"] == np.count_nonzero(v)
    assert r["err2_round"] + r["err2_overflow"] + r["err2_underflow"] == pytest.approx(((v - vt) ** 2).sum(), rel=1e-12)
    assert r["sum_re"] == pytest.approx(np.nansum(oracle.relative_error(v, vt)), rel=1e-12)
    assert r["sum_re"] >= r["sum_re_round"] + r["n_underflow"] - 1e-9
    assert r["sum_x2"] == pytest.approx((v ** 2).sum(), rel=1e-14)
    # with the scale taken from the data nothing lies beyond the largest value by more than the
    # rounding of delta itself: at most the maxima can be flagged, and their error is tiny
    assert r["err2_overflow"] <= 1e-12 * r["sum_x2"]
    if fmt == "int8":
        assert r["n_underflow"] == np.count_nonzero((np.abs(v) > 0) & (vt == 0))


def test_per_channel_scales_remove_underflow_of_small_channels():
    rng = np.random.default_rng(9)
    x = f32(rng.standard_normal((16, 256)))
    x[:8] *= 1e-4                                       # half the channels are tiny
    t = oracle.quantize_error(x, "int8", "tensor")
    c = oracle.quantize_error(x, "int8", "channel")
    assert t["n_underflow"] > 0.9 * 8 * 256 and c["n_underflow"] < 0.02 * 16 * 256
    assert c["sum_re"] < 0.1 * t["sum_re"]
