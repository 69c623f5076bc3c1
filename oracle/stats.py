"""Tensor statistics and the per-element quantization error split. TEST INFRASTRUCTURE ONLY.

Two things the paper does to a single tensor, before and beside the matmul probe:

* Experiments section: the inputs of every major matmul of the bf16 baseline are
  sampled "to compute the mean, variance, skew and Kurtosis".  Here: population central
  moments m_k = mean((x - mean)^k) in float64, variance = m2, skew = m3 / m2^1.5,
  kurtosis = m4 / m2^2 (the plain fourth standardised moment: 3 for a normal law).
* Results section, Eq. 2 and the paragraph before it: the error of quantizing one value,
  RE = |v - v~| / |v|, is either clipping error (the value lies outside the format's
  dynamic range: overflow is capped at the largest value, underflow becomes zero) or
  rounding error (the value lies between two expressible numbers).

Everything is written out element by element with numpy in float64; the only steps shared
with the rest of the oracle are its own scale / quantize / dequantize.
"""
import numpy as np

from .formats import qmax
from .probe import _as_f32, _expand, dequantize, quantize, scale


def tensor_stats(x):
    """Mean, variance, skew, kurtosis and max|x| of all elements of x (Experiments section).

    Also returns the raw power sums, which is what a one-pass implementation accumulates.
    An empty or constant tensor has skew = kurtosis = 0 by convention.
    """
    v = _as_f32(x).astype(np.float64).ravel()
    n = v.size
    if n == 0:
        return dict(count=0, max_abs=0.0, mean=0.0, variance=0.0, skew=0.0, kurtosis=0.0,
                    sum1=0.0, sum2=0.0, sum3=0.0, sum4=0.0)
    mean = v.sum() / n
    d = v - mean
    m2 = (d ** 2).sum() / n
    m3 = (d ** 3).sum() / n
    m4 = (d ** 4).sum() / n
    skew = m3 / m2 ** 1.5 if m2 > 0 else 0.0
    kurt = m4 / m2 ** 2 if m2 > 0 else 0.0
    return dict(count=n, max_abs=float(np.abs(v).max()), mean=mean, variance=m2, skew=skew, kurtosis=kurt,
                sum1=v.sum(), sum2=(v ** 2).sum(), sum3=(v ** 3).sum(), sum4=(v ** 4).sum())


def quantize_error(x, fmt, gran, delta=None):
    """Eq. 2 per element of x [.., nc, c] under Eq. 1 with the given format and granularity,
    split the way the Results section splits it.

    t = x / delta is the float32 quotient the quantizer itself uses.  An element is
      overflow   when |t| exceeds the largest expressible magnitude (it is capped),
      underflow  when it is not zero but its code is zero,
      rounding   otherwise (zeros are none of the three and contribute nothing).
    v~ = value(code) * delta in float64.  Returns the counts, the sums of RE over all non-zero
    elements and over the rounding class, the largest rounding RE, the squared absolute error
    of each class and sum x^2 (so that signal-to-noise ratios per class follow).
    """
    x = _as_f32(x)
    if delta is None:
        delta = scale(x, fmt, gran)
    codes = quantize(x, fmt, delta)
    vt = dequantize(codes, fmt, delta)
    v = x.astype(np.float64)
    t = (x / _expand(delta, x)).astype(np.float32)
    nonzero = v != 0
    overflow = nonzero & (np.abs(t.astype(np.float64)) > qmax(fmt))
    underflow = nonzero & ~overflow & (vt == 0)
    rounding = nonzero & ~overflow & ~underflow
    err = np.abs(v - vt)
    with np.errstate(divide="ignore", invalid="ignore"):
        re = np.where(nonzero, err / np.abs(v), 0.0)
    return dict(count=int(v.size), n_nonzero=int(nonzero.sum()), n_overflow=int(overflow.sum()),
                n_underflow=int(underflow.sum()), sum_re=float(re.sum()),
                sum_re_round=float(re[rounding].sum()),
                max_re_round=float(re[rounding].max()) if rounding.any() else 0.0,
                err2_round=float((err[rounding] ** 2).sum()), err2_overflow=float((err[overflow] ** 2).sum()),
                err2_underflow=float((err[underflow] ** 2).sum()), sum_x2=float((v ** 2).sum()))
