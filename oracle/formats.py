"""8-bit number formats of the Methodology section, built from first principles.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The paper studies INT8, E4M3 and E5M2 and prints their largest expressible
magnitudes (127, 448, 57344).  An "EeMm" format has one sign bit, e exponent
bits with a bias, and m mantissa bits.  The FP8 rules are those of the FP8
formats paper the Methodology section cites:
  * E4M3: bias 7, subnormals when the exponent field is 0, no infinities, the
    single mantissa pattern 111 under exponent 1111 is NaN, so the largest
    finite value is 1.75 * 2**8 = 448.
  * E5M2: bias 15, IEEE-like: exponent field 31 holds inf (mantissa 0) and NaN,
    so the largest finite value is 1.75 * 2**15 = 57344.
  * INT8: two's complement; symmetric quantization uses -127..127 only
    (Eq. 1 divides by 2**(n-1) - 1), so -128 is never produced.
"""
import numpy as np

FORMATS = ("int8", "e4m3", "e5m2")


def _decode_fp8(code, e_bits, m_bits, bias, ieee_specials):
    sign = -1.0 if (code >> 7) & 1 else 1.0
    e = (code >> m_bits) & ((1 << e_bits) - 1)
    m = code & ((1 << m_bits) - 1)
    e_all_ones = (1 << e_bits) - 1
    if ieee_specials and e == e_all_ones:
        return sign * np.inf if m == 0 else np.nan
    if (not ieee_specials) and e == e_all_ones and m == (1 << m_bits) - 1:
        return np.nan
    if e == 0:  # subnormal: no hidden one, exponent of the smallest normal
        return sign * (m / (1 << m_bits)) * 2.0 ** (1 - bias)
    return sign * (1.0 + m / (1 << m_bits)) * 2.0 ** (e - bias)


def decode_table(fmt):
    """All 256 code -> value entries (float64) of a format, indexed by the
    unsigned byte.  INT8 bytes are two's complement."""
    out = np.empty(256, dtype=np.float64)
    for code in range(256):
        if fmt == "int8":
            out[code] = code - 256 if code >= 128 else code
        elif fmt == "e4m3":
            out[code] = _decode_fp8(code, 4, 3, 7, False)
        elif fmt == "e5m2":
            out[code] = _decode_fp8(code, 5, 2, 15, True)
        else:
            raise ValueError(fmt)
    return out


def positive_grid(fmt):
    """Non-negative finite grid values in ascending order.  For all three
    formats entry c is the value of byte c (positive codes are monotone)."""
    t = decode_table(fmt)
    n = {"int8": 128, "e4m3": 0x7F, "e5m2": 0x7C}[fmt]
    g = t[:n].copy()
    assert np.all(np.isfinite(g)) and np.all(np.diff(g) > 0)
    return g


def qmax(fmt):
    """Largest expressible magnitude: 127 / 448 / 57344 (Methodology, last
    bullet).  Computed from the table, not typed in."""
    return float(positive_grid(fmt)[-1])
