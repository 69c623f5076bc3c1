"""The quantized-matmul error probe, step by step, in the paper's order.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Operands are passed in "non-contracting x contracting" orientation: X[..., nc, c]
(an optional leading matmul-batch axis).  For L of a product L.R this is L
itself ([M, K]); for R ([K, N]) it is R transposed ([N, K]).  `probe` takes L
and R in their natural orientation and does that transposition itself.

Values are float32 arrays holding exactly the stored numbers (a bf16 value is
exactly representable in float32).  Everything mathematical is float64; the
two operations the paper writes as arithmetic on the stored tensors (the
division that forms delta and the division x / delta of Eq. 1) are single IEEE
float32 operations, which is the precision decision both sides of a parity
test share.
"""
import numpy as np

from .rng import element_uniforms
from .formats import decode_table, positive_grid, qmax


def _as_f32(x):
    x = np.asarray(x)
    if x.dtype != np.float32:
        raise TypeError("operands are float32 arrays of the stored values")
    return x


def scale(x, fmt, gran, batch_groups=None):
    """Eq. 1, right half: delta = max|X| / qmax, one delta per scaling group.

    gran == "tensor": one number for the whole (batched) tensor, shape [1].
    gran == "channel": one number per index of the non-contracting dimension
    (and per matmul-batch element), shape x.shape[:-1]  ("finer levels of
    granularity on non-contracting dimensions", Methodology 4th bullet).
    An all-zero group gets delta = 1.  Non-finite input is an error.

    batch_groups (channel granularity of a batched [b, nc, c] operand only): the granularity
    levels of the Results section share scales along the matmul-batch axis.  Batch element
    number b belongs to group b mod batch_groups and all elements of a group share their
    per-channel scales: batch_groups = 1 is the paper's "channel" (one scale tensor over the
    non-batch, non-contracting dimension), batch_groups = number of heads with the batch laid
    out [examples][heads] is its "fine-grained" (batch dimensions included, except the axis of
    the individual examples).  None: every batch element has its own scales.  The returned
    array still has shape x.shape[:-1], with shared entries repeated.
    """
    x = _as_f32(x)
    if not np.all(np.isfinite(x)):
        raise ValueError("non-finite input")
    a = np.abs(x)
    if gran == "tensor":
        amax = np.array([a.max() if a.size else 0.0], dtype=np.float32)
    elif gran == "channel":
        amax = a.max(axis=-1).astype(np.float32) if a.shape[-1] else np.zeros(a.shape[:-1], np.float32)
        if batch_groups is not None:
            if x.ndim != 3 or batch_groups < 1 or x.shape[0] % batch_groups:
                raise ValueError("batch_groups must divide the batch of a [b, nc, c] operand")
            g = batch_groups
            shared = amax.reshape(x.shape[0] // g, g, x.shape[1]).max(axis=0)      # over the examples
            amax = np.broadcast_to(shared, (x.shape[0] // g, g, x.shape[1])).reshape(x.shape[:2]).copy()
    else:
        raise ValueError(gran)
    delta = amax / np.float32(qmax(fmt))          # one float32 division
    delta = np.where(amax == 0, np.float32(1.0), delta).astype(np.float32)
    return delta


def _expand(delta, x):
    """Broadcast delta ([1] or x.shape[:-1]) against x."""
    delta = np.asarray(delta, dtype=np.float32)
    if delta.shape == (1,):
        return delta.reshape((1,) * x.ndim)
    if delta.shape != x.shape[:-1]:
        raise ValueError("delta shape")
    return delta[..., None]


def quantize(x, fmt, delta, rounding="rtne", seed=0, stream=0):
    """Eq. 1, left half, with the saturation rule of the Methodology section.

    rounding == "stochastic" (second rounding mode of the Methodology section): see
    _quantize_stochastic.  What follows describes the default, round-to-nearest-even.

    t = x / delta in float32; the code is the grid value nearest to t, a tie
    going to the value whose code is even (round-to-nearest-even); |t| above the
    largest expressible value saturates to it.  Magnitudes below half the
    smallest positive grid value therefore become zero (FP8: a zero that keeps
    the sign bit of the input; INT8 has one zero).  Returns uint8 bytes
    (INT8: two's complement).
    The nearest value is found by comparing t with the midpoints of adjacent
    grid values, so no conversion instruction is involved.
    """
    x = _as_f32(x)
    if not (np.all(np.isfinite(x)) and np.all(np.isfinite(np.asarray(delta)))):
        raise ValueError("non-finite input")
    with np.errstate(over="ignore"):
        # IEEE float32 division.  With a scale that is not the tensor's own (a stale or shared one)
        # the quotient of finite numbers can exceed the float32 range; it is then a magnitude above
        # the largest expressible value and saturates like any other (the saturation rule).
        t = (x / _expand(delta, x)).astype(np.float32)
    if rounding == "stochastic":
        return _quantize_stochastic(t, fmt, seed, stream)
    if rounding != "rtne":
        raise ValueError(rounding)
    g = positive_grid(fmt)                               # g[c] = value of code c
    mid = (g[:-1] + g[1:]) / 2.0                         # exact in float64
    a = np.abs(t.astype(np.float64))
    idx = np.searchsorted(mid, a, side="left")           # number of midpoints < a
    below_top = idx < len(g) - 1
    tie = below_top & (a == mid[np.minimum(idx, len(mid) - 1)])
    idx = idx + (tie & (idx % 2 == 1))                   # tie: take the even code
    if fmt == "int8":
        code = np.where(np.signbit(t) & (idx > 0), 256 - idx, idx)
    else:
        # FP8 is sign-magnitude with IEEE conventions (the FP8 rules the paper cites): the sign
        # bit of the input survives rounding, so a negative value that rounds to zero is -0.
        code = np.where(np.signbit(t), idx + 128, idx)
    return code.astype(np.uint8)


def _quantize_stochastic(t, fmt, seed, stream):
    """Stochastic rounding of t = x / delta onto the format's grid.

    With lo <= |t| <= hi the two neighbouring expressible magnitudes (|t| first capped at the
    largest one: the saturation rule), the result is hi with probability
    p = (|t| - lo) / (hi - lo) and lo otherwise, so its expectation is t.  The draw of element
    number i (C order over the operand in its [.., nc, c] orientation) is the uniform number
    u_i of rng.element_uniforms(seed, stream): hi iff u_i < p.  A value on the grid has p = 0 and
    never moves; the sign is kept (FP8 keeps it on a zero result as RTNE does).
    All of it is exact in float64: |t| - lo and hi - lo are exact differences of float32 values.
    """
    g = positive_grid(fmt)
    a = np.minimum(np.abs(t.astype(np.float64)), g[-1])
    lo_i = np.searchsorted(g, a, side="right") - 1        # largest grid value <= a
    hi_i = np.minimum(lo_i + 1, len(g) - 1)
    lo, hi = g[lo_i], g[hi_i]
    with np.errstate(divide="ignore", invalid="ignore"):
        p = np.where(hi > lo, (a - lo) / (hi - lo), 0.0)
    u = element_uniforms(t.shape, seed, stream)
    idx = np.where(u < p, hi_i, lo_i)
    if fmt == "int8":
        code = np.where(np.signbit(t) & (idx > 0), 256 - idx, idx)
    else:
        code = np.where(np.signbit(t), idx + 128, idx)
    return code.astype(np.uint8)


def dequantize(codes, fmt, delta=None):
    """Code -> value (float64), times delta when given."""
    v = decode_table(fmt)[np.asarray(codes, dtype=np.uint8)]
    if delta is not None:
        v = v * _expand(delta, v).astype(np.float64)
    return v


def gemm_lp(codes_l, fmt_l, codes_r, fmt_r):
    """A = Lbar . Rbar on decoded code values, float64 accumulation (exact for
    INT8 and E4M3: every partial sum is a multiple of the smallest product
    below 2**53 of them).  codes_l [.., M, K], codes_r [.., N, K]."""
    a = dequantize(codes_l, fmt_l)
    b = dequantize(codes_r, fmt_r)
    return np.matmul(a, np.swapaxes(b, -1, -2))


def descale(acc, delta_l, delta_r):
    """Q_ij = A_ij * delta_L[i] * delta_R[j] (descaling after the matmul)."""
    dl = np.asarray(delta_l, dtype=np.float64)
    dr = np.asarray(delta_r, dtype=np.float64)
    dl = dl.reshape((1,) * acc.ndim) if dl.shape == (1,) else dl[..., :, None]
    dr = dr.reshape((1,) * acc.ndim) if dr.shape == (1,) else dr[..., None, :]
    return acc * dl * dr


def gemm_ref(l, rt):
    """C = L . R in float64 on the stored values (numerator of Eq. 3)."""
    return np.matmul(_as_f32(l).astype(np.float64),
                     np.swapaxes(_as_f32(rt).astype(np.float64), -1, -2))


def gemm_den(l, rt):
    """D = |L| . |R|: elementwise absolute values, then the matrix product
    (denominator of Eq. 3, inner-product-level backward error)."""
    return np.matmul(np.abs(_as_f32(l).astype(np.float64)),
                     np.swapaxes(np.abs(_as_f32(rt).astype(np.float64)), -1, -2))


def metric(c, q, d):
    """Eq. 3 per inner product: BE_ij = |C_ij - Q_ij| / D_ij (0 where D_ij is
    0), reduced to the statistics record."""
    c = np.asarray(c, np.float64); q = np.asarray(q, np.float64); d = np.asarray(d, np.float64)
    diff = c - q
    be = np.zeros_like(diff)
    nz = d != 0
    be[nz] = np.abs(diff[nz]) / d[nz]
    return {
        "sum_be": float(be.sum()),
        "max_be": float(be.max()) if be.size else 0.0,
        "sum_diff2": float((diff * diff).sum()),
        "sum_ref2": float((c * c).sum()),
        "sum_den2": float((d * d).sum()),
        "count": int(be.size),
    }


def derived(rec):
    """Scalars derived from the record: mean BE (primary), norm-wise BE,
    relative L2 error and SNR in dB."""
    n = max(rec["count"], 1)
    sd, sr, sden = rec["sum_diff2"], rec["sum_ref2"], rec["sum_den2"]
    return {
        "mean_be": rec["sum_be"] / n,
        "max_be": rec["max_be"],
        "normwise_be": (sd / sden) ** 0.5 if sden > 0 else 0.0,
        "rel_l2": (sd / sr) ** 0.5 if sr > 0 else 0.0,
        "snr_db": 10.0 * np.log10(sr / sd) if sd > 0 and sr > 0 else float("inf"),
    }


def probe(l, r, fmt_l, fmt_r, gran_l, gran_r, rows=None, full=False, round_l="rtne", round_r="rtne", seed=0,
          groups_l=None, groups_r=None):
    """The whole probe for L [.., M, K] and R [.., K, N].

    rows: optional index array of output rows to evaluate (row-sampled mode;
    scales are still computed over the whole operands).  With full=True the
    intermediate arrays are returned too.  round_l / round_r choose the rounding mode per
    operand (the paper rounds gradients stochastically); stochastic draws are numbered over
    the whole operand in its [.., nc, c] orientation, stream 0 for L and 1 for R.
    groups_l / groups_r: batch_groups of scale() for an operand with channel granularity.
    """
    l = l_full = _as_f32(l)
    rt = np.swapaxes(_as_f32(r), -1, -2)
    dl = scale(l, fmt_l, gran_l, groups_l if gran_l == "channel" else None)
    dr = scale(rt, fmt_r, gran_r, groups_r if gran_r == "channel" else None)
    if rows is not None:
        l = l[..., rows, :]
        dl_rows = dl if dl.shape == (1,) else dl[..., rows]
    else:
        dl_rows = dl
    if round_l == "stochastic" and rows is not None:
        cl = quantize(_as_f32(l_full), fmt_l, dl, "stochastic", seed, 0)[..., rows, :]
    else:
        cl = quantize(l, fmt_l, dl_rows, round_l, seed, 0)
    cr = quantize(rt, fmt_r, dr, round_r, seed, 1)
    acc = gemm_lp(cl, fmt_l, cr, fmt_r)
    q = descale(acc, dl_rows, dr)
    c = gemm_ref(l, rt)
    d = gemm_den(l, rt)
    rec = metric(c, q, d)
    if full:
        return rec, {"delta_l": dl, "delta_r": dr, "codes_l": cl, "codes_r": cr,
                     "acc": acc, "q": q, "c": c, "d": d}
    return rec


def relative_error(v, v_tilde):
    """Eq. 2 with the denominator read as |v|; entries with v == 0 are NaN."""
    v = np.asarray(v, np.float64); v_tilde = np.asarray(v_tilde, np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        return np.where(v != 0, np.abs(v - v_tilde) / np.abs(v), np.nan)
