"""Pins for the oracle's scale and quantizer (Eq. 1, saturation rule)."""
import ml_dtypes
import numpy as np
import pytest

import oracle
from oracle import positive_grid, qmax

FMTS = ["int8", "e4m3", "e5m2"]


def signed(codes, fmt):
    return oracle.dequantize(codes, fmt)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("p", [-3, 0, 5])
def test_identity_on_grid(fmt, p):
    # inputs already on the grid, absmax = qmax * 2^p  =>  delta = 2^p, zero error
    g = positive_grid(fmt)
    vals = np.concatenate([g, -g[1:]]) * 2.0 ** p
    x = vals.astype(np.float32)[None, :]
    assert np.array_equal(x.astype(np.float64), vals[None, :])       # representable in fp32
    d = oracle.scale(x, fmt, "tensor")
    assert d.shape == (1,) and d[0] == np.float32(2.0 ** p)
    codes = oracle.quantize(x, fmt, d)
    assert np.array_equal(oracle.dequantize(codes, fmt, d), x.astype(np.float64))
    want = np.concatenate([np.arange(len(g)), (np.arange(1, len(g)) + 128) if fmt != "int8"
                           else 256 - np.arange(1, len(g))]).astype(np.uint8)
    assert np.array_equal(codes[0], want)


@pytest.mark.parametrize("fmt", FMTS)
def test_ties_go_to_even_code(fmt):
    g = positive_grid(fmt)
    mid = (g[:-1] + g[1:]) / 2
    x = mid.astype(np.float32)
    assert np.array_equal(x.astype(np.float64), mid)
    one = np.array([1.0], np.float32)
    for s in (1.0, -1.0):
        codes = oracle.quantize((s * x)[None, :], fmt, one)[0]
        mag = np.abs(signed(codes, fmt))
        lo, hi = g[:-1], g[1:]
        even_is_lo = (np.arange(len(g) - 1) % 2) == 0
        assert np.array_equal(mag, np.where(even_is_lo, lo, hi))
    # just off the midpoint goes to the nearer neighbour
    up = np.nextafter(x, np.float32(np.inf)); dn = np.nextafter(x, np.float32(-np.inf))
    assert np.array_equal(np.abs(signed(oracle.quantize(up[None], fmt, one)[0], fmt)), g[1:])
    assert np.array_equal(np.abs(signed(oracle.quantize(dn[None], fmt, one)[0], fmt)), g[:-1])


def test_int8_textbook_ties():
    one = np.array([1.0], np.float32)
    x = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5, 0.49, 0.51]], np.float32)
    got = signed(oracle.quantize(x, "int8", one), "int8")[0]
    assert got.tolist() == [0, 2, 2, 0, -2, -2, 126, 0, 1]


@pytest.mark.parametrize("fmt", FMTS)
def test_saturation_and_underflow(fmt):
    one = np.array([1.0], np.float32)
    big = np.array([[qmax(fmt) * 1.001, qmax(fmt) * 4, 3e38, -qmax(fmt) * 1.5, -3e38]], np.float32)
    v = signed(oracle.quantize(big, fmt, one), fmt)[0]
    assert v.tolist() == [qmax(fmt)] * 3 + [-qmax(fmt)] * 2
    top = {"int8": 0x7F, "e4m3": 0x7E, "e5m2": 0x7B}[fmt]
    codes = oracle.quantize(big, fmt, one)[0]
    assert codes[0] == top and (codes[3] == (0x81 if fmt == "int8" else top + 128))
    s = positive_grid(fmt)[1]          # smallest positive grid value
    tiny = np.array([[s * 0.49, s * 0.5, s * 0.51, s * 0.99, -s * 0.49, -s * 0.5]], np.float32)
    v = signed(oracle.quantize(tiny, fmt, one), fmt)[0]
    assert v.tolist() == [0, 0, s, s, 0, 0]
    # never -128 and never a non-finite pattern, for any finite input
    rng = np.random.default_rng(1)
    x = (rng.standard_cauchy((4, 4096)) * 100).astype(np.float32)
    c = oracle.quantize(x, fmt, oracle.scale(x, fmt, "channel"))
    assert np.all(np.isfinite(signed(c, fmt))) and np.all(np.abs(signed(c, fmt)) <= qmax(fmt))
    if fmt == "int8":
        assert not np.any(c == 0x80)


@pytest.mark.parametrize("fmt", FMTS)
def test_odd_symmetry_and_monotone(fmt):
    rng = np.random.default_rng(2)
    x = np.sort((rng.standard_normal(20000) * qmax(fmt) / 3).astype(np.float32))[None, :]
    one = np.array([1.0], np.float32)
    v = signed(oracle.quantize(x, fmt, one), fmt)[0]
    assert np.all(np.diff(v) >= 0)
    vneg = signed(oracle.quantize(-x, fmt, one), fmt)[0]
    assert np.array_equal(vneg, -v)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_power_of_two_scale_invariance(fmt, gran):
    rng = np.random.default_rng(3)
    x = rng.standard_t(3, (8, 512)).astype(np.float32)
    d0 = oracle.scale(x, fmt, gran); c0 = oracle.quantize(x, fmt, d0)
    for p in (-7, 4):
        xs = (x * np.float32(2.0 ** p)).astype(np.float32)
        d = oracle.scale(xs, fmt, gran)
        assert np.array_equal(d, d0 * np.float32(2.0 ** p))
        assert np.array_equal(oracle.quantize(xs, fmt, d), c0)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_delta_definition_and_absmax_maps_to_qmax(fmt, gran):
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 16, 300)).astype(np.float32)
    d = oracle.scale(x, fmt, gran)
    if gran == "tensor":
        assert d.shape == (1,)
        assert d[0] == np.float32(np.abs(x).max()) / np.float32(qmax(fmt))
    else:
        assert d.shape == (2, 16)
        for b in range(2):
            for i in range(16):
                assert d[b, i] == np.float32(np.abs(x[b, i]).max()) / np.float32(qmax(fmt))
    v = np.abs(signed(oracle.quantize(x, fmt, d), fmt))
    if gran == "tensor":
        assert v.max() == qmax(fmt)
    else:
        assert np.all(v.max(axis=-1) == qmax(fmt))


@pytest.mark.parametrize("fmt", FMTS)
def test_round_trip_reproduces_codes(fmt):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((4, 1000)).astype(np.float32)
    x[:, 0] = qmax(fmt) * 2.0 ** -6           # exact delta = 2^-6 per row
    x = np.clip(x, -x[0, 0], x[0, 0])
    d = oracle.scale(x, fmt, "channel")
    assert np.all(d == np.float32(2.0 ** -6))
    c = oracle.quantize(x, fmt, d)
    y = oracle.dequantize(c, fmt, d).astype(np.float32)
    assert np.array_equal(oracle.scale(y, fmt, "channel"), d)
    assert np.array_equal(oracle.quantize(y, fmt, d), c)


def test_zero_group_and_nonfinite():
    x = np.zeros((3, 8), np.float32); x[1, 2] = -2.0
    d = oracle.scale(x, "e4m3", "channel")
    assert d[0] == 1.0 and d[2] == 1.0 and d[1] == np.float32(2.0) / np.float32(448)
    c = oracle.quantize(x, "e4m3", d)
    assert np.all(c[0] == 0) and np.all(c[2] == 0) and c[1, 2] == 0xFE
    x[0, 0] = np.inf
    with pytest.raises(ValueError):
        oracle.scale(x, "int8", "tensor")
    x[0, 0] = np.nan
    with pytest.raises(ValueError):
        oracle.scale(x, "int8", "tensor")


def test_int8_uniform_closed_form_sqnr():
    # x ~ U(-a, a) in fp32: noise variance delta^2 / 12  =>  SQNR = 4 * 127^2 (48.10 dB)
    rng = np.random.default_rng(6)
    a = 3.7
    x = rng.uniform(-a, a, (1, 1 << 22)).astype(np.float32)
    x[0, 0] = a
    d = oracle.scale(x, "int8", "tensor")
    y = oracle.dequantize(oracle.quantize(x, "int8", d), "int8", d)
    e = y - x.astype(np.float64)
    sqnr_db = 10 * np.log10((x.astype(np.float64) ** 2).mean() / (e ** 2).mean())
    assert abs(sqnr_db - 10 * np.log10(4 * 127 ** 2)) < 0.02
    assert abs((e ** 2).mean() / (float(d[0]) ** 2 / 12) - 1) < 5e-3
    # half a step, plus the fp32 rounding of t = x / delta near |t| = 127
    assert np.abs(e).max() <= float(d[0]) / 2 * (1 + 1e-4)


@pytest.mark.parametrize("fmt,m", [("e4m3", 3), ("e5m2", 2)])
def test_fp8_uniform_binade_closed_form_sqnr(fmt, m):
    # x ~ U[2^e, 2^(e+1)) with delta = 1: SQNR = 28 * 2^(2m); the largest relative error is
    # half a step just above 2^e: 2^-(m+1) / (1 + 2^-(m+1)) = 1 / (2^(m+1) + 1)
    rng = np.random.default_rng(7)
    for e in (-2, 3):
        x = rng.uniform(2.0 ** e, 2.0 ** (e + 1), (1, 1 << 21)).astype(np.float32)
        one = np.array([1.0], np.float32)
        y = oracle.dequantize(oracle.quantize(x, fmt, one), fmt)
        err = y - x.astype(np.float64)
        sqnr = (x.astype(np.float64) ** 2).mean() / (err ** 2).mean()
        assert abs(10 * np.log10(sqnr) - 10 * np.log10(28 * 2 ** (2 * m))) < 0.03
        re = oracle.relative_error(x, y)
        bound = 1.0 / (2 ** (m + 1) + 1)
        assert re.max() <= bound * (1 + 1e-6) and re.max() > 0.999 * bound


@pytest.mark.parametrize("fmt,dt", [("e4m3", ml_dtypes.float8_e4m3fn), ("e5m2", ml_dtypes.float8_e5m2)])
def test_rounding_against_outside_library(fmt, dt):
    # in-range values with delta = 1: a library's float32 -> fp8 RTNE cast must agree
    rng = np.random.default_rng(8)
    mags = np.exp2(rng.uniform(-20, np.log2(qmax(fmt)), 200000))
    t = (mags * rng.choice([-1.0, 1.0], mags.shape)).astype(np.float32)
    t = t[np.abs(t) <= qmax(fmt)]
    lib = t.astype(dt).view(np.uint8)
    ours = oracle.quantize(t[None, :], fmt, np.array([1.0], np.float32))[0]
    assert np.array_equal(lib, ours)             # byte for byte, signed zeros included
    assert (ours == 0x80).any() and (ours == 0x00).any()


def test_fp8_zero_keeps_sign_int8_does_not():
    one = np.array([1.0], np.float32)
    x = np.array([[-1e-30, 1e-30, -0.0, 0.0]], np.float32)
    assert oracle.quantize(x, "e4m3", one)[0].tolist() == [0x80, 0, 0x80, 0]
    assert oracle.quantize(x, "e5m2", one)[0].tolist() == [0x80, 0, 0x80, 0]
    assert oracle.quantize(x, "int8", one)[0].tolist() == [0, 0, 0, 0]


def test_int8_rounding_against_rint():
    rng = np.random.default_rng(9)
    x = rng.uniform(-127.49, 127.49, (1, 100000)).astype(np.float32)
    ours = oracle.dequantize(oracle.quantize(x, "int8", np.array([1.0], np.float32)), "int8")
    assert np.array_equal(ours, np.rint(x.astype(np.float64)))


def test_division_is_fp32_not_reciprocal_multiply():
    # the quantizer divides (Eq. 1); make sure a case where x*(1/d) and x/d differ is a division
    x = np.array([[5.0, 127.0 * 3.0]], np.float32)
    d = oracle.scale(x, "int8", "tensor")
    assert d[0] == np.float32(3.0)
    t = np.float32(5.0) / np.float32(3.0)
    c = oracle.quantize(x, "int8", d)
    assert oracle.dequantize(c, "int8")[0, 0] == np.rint(np.float64(t)) == 2.0
    # a tie produced only by exact division: 7.5 / 3 = 2.5 -> 2
    x = np.array([[7.5, 381.0]], np.float32)
    assert oracle.dequantize(oracle.quantize(x, "int8", d), "int8")[0, 0] == 2.0


# ------------------------------------------------------------------ scales shared along the batch
def test_batch_groups_match_the_granularity_levels_of_the_results_section():
    """'channel' = one scale per non-contracting index shared by the whole matmul batch;
    'fine-grained' = also per head, shared by the examples.  Hand-built case: batch laid out
    [examples = 2][heads = 3], one row, so the maxima can be read off."""
    x = np.zeros((6, 1, 4), np.float32)
    peaks = [1.0, 20.0, 3.0, 40.0, 5.0, 6.0]            # b = e * 3 + h
    for b, p in enumerate(peaks):
        x[b, 0, b % 4] = -p
    own = oracle.scale(x, "int8", "channel")
    assert np.array_equal(own[:, 0] * 127, np.float32(peaks))
    fine = oracle.scale(x, "int8", "channel", batch_groups=3)       # per head: max over the two examples
    assert np.allclose(fine[:, 0] * 127, [40.0, 20.0, 6.0, 40.0, 20.0, 6.0])
    chan = oracle.scale(x, "int8", "channel", batch_groups=1)       # shared by the whole batch
    assert np.allclose(chan[:, 0] * 127, [40.0] * 6)
    assert np.array_equal(oracle.scale(x, "int8", "channel", batch_groups=6), own)
    with pytest.raises(ValueError):
        oracle.scale(x, "int8", "channel", batch_groups=4)


def test_batch_groups_equal_a_per_channel_scale_of_the_regrouped_tensor():
    rng = np.random.default_rng(12)
    E, H, S, D = 3, 4, 10, 16
    x = rng.standard_normal((E * H, S, D)).astype(np.float32) * 10.0 ** rng.uniform(-2, 1, (E * H, 1, 1)).astype(np.float32)
    got = oracle.scale(x, "e4m3", "channel", batch_groups=H)
    # the same numbers from the textbook route: move the examples next to the contraction and take
    # an ordinary per-row absmax
    regrouped = x.reshape(E, H, S, D).transpose(1, 2, 0, 3).reshape(H, S, E * D)
    want = oracle.scale(regrouped, "e4m3", "channel")               # [H, S]
    assert np.array_equal(got.reshape(E, H, S), np.broadcast_to(want, (E, H, S)))
    # coarser sharing never gives a smaller scale, and quantization error cannot shrink with it
    own = oracle.scale(x, "e4m3", "channel")
    assert np.all(got >= own) and np.all(oracle.scale(x, "e4m3", "channel", 1) >= got)


@pytest.mark.parametrize("fmt", FMTS)
def test_quotient_beyond_float32_saturates(fmt):
    """Finite inputs under a much smaller outside scale: x / delta overflows float32, which is a
    magnitude above the largest expressible value and must saturate (Methodology, saturation rule),
    with the sign kept; non-finite inputs or scales remain errors."""
    x = np.array([[3e38, -3e38, 1e30, -0.0, 2e-30]], dtype=np.float32)
    d = np.array([1e-30], dtype=np.float32)
    v = oracle.dequantize(oracle.quantize(x, fmt, d), fmt)
    top = oracle.qmax(fmt)
    assert v[0, 0] == top and v[0, 1] == -top and v[0, 2] == top and v[0, 3] == 0
    assert v[0, 4] == 2.0
    with pytest.raises(ValueError):
        oracle.quantize(np.array([[np.inf]], dtype=np.float32), fmt, d)
    with pytest.raises(ValueError):
        oracle.quantize(x, fmt, np.array([np.nan], dtype=np.float32))
