"""GPU parity: scales and codes against the oracle, bit for bit (Eq. 1, saturation rule)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from helpers import oriented, as3

pytestmark = pytest.mark.gpu
FMTS = ["int8", "e4m3", "e5m2"]


def make(shape, dtype, seed, dist="t"):
    rng = np.random.default_rng(seed)
    x = (rng.standard_t(3, shape) if dist == "t" else rng.standard_normal(shape)).astype(np.float32)
    return torch.from_numpy(x).to(dtype)


def check(t, contract_dim, fmt, gran, fused):
    td = t.cuda()
    op = qm.operand_of(td, contract_dim)
    x = as3(oriented(t, contract_dim))                     # [b, nc, c]
    want_d = oracle.scale(x, fmt, gran)
    want_c = oracle.quantize(x, fmt, want_d)
    d = qm.qm_scale(op, fmt, gran)
    assert np.array_equal(d.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32))
    if fused:
        codes, d2, ab, km = qm.qm_quantize(op, fmt, gran, None, want_abs=True, want_kmaj=(contract_dim == -2))
        assert np.array_equal(d2.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32))
    else:
        codes, _, ab, km = qm.qm_quantize(op, fmt, gran, d, want_abs=True, want_kmaj=True)
    torch.cuda.synchronize()
    c = codes.cpu().numpy()
    K = x.shape[-1]
    assert c.shape[-1] == (K + 15) // 16 * 16
    assert np.array_equal(c[..., :K], want_c)
    assert not c[..., K:].any()                            # padding bytes are zero
    xb = torch.from_numpy(x).to(torch.bfloat16)
    assert torch.equal(ab.cpu(), xb.abs())
    if km is not None:
        assert torch.equal(km.cpu(), xb)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("layout", ["rows", "cols"])
def test_codes_bf16(fmt, gran, fused, layout):
    # several 64-wide tiles plus ragged tails in both directions
    t = make((333, 200), torch.bfloat16, 1)
    check(t, -1 if layout == "rows" else -2, fmt, gran, fused)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("layout", ["rows", "cols"])
def test_codes_fp32(fmt, gran, layout):
    t = make((130, 264), torch.float32, 2, "n")
    check(t, -1 if layout == "rows" else -2, fmt, gran, True)


@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("layout", ["rows", "cols"])
def test_codes_batched(gran, layout):
    t = make((5, 72, 64), torch.bfloat16, 3)
    check(t, -1 if layout == "rows" else -2, "e4m3", gran, True)
    check(t, -1 if layout == "rows" else -2, "int8", gran, False)


def test_strided_view_and_long_rows():
    big = make((64, 4104), torch.bfloat16, 4)
    v = big[:, :4100]                                      # row stride 4104, ragged length
    td = big.cuda()[:, :4100]
    for gran in ("tensor", "channel"):
        op = qm.operand_of(td, -1)
        x = as3(v.float().numpy())
        want_d = oracle.scale(x, "e5m2", gran)
        codes, d, _, _ = qm.qm_quantize(op, "e5m2", gran, None)
        assert np.array_equal(d.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32))
        assert np.array_equal(codes.cpu().numpy()[..., :4100], oracle.quantize(x, "e5m2", want_d))


@pytest.mark.parametrize("fmt", FMTS)
def test_exhaustive_bf16_inputs(fmt):
    # every finite bf16 value, under several scales, including awkward non-power-of-two ones
    bits = np.arange(65536, dtype=np.uint32)
    vals = (bits << 16).view(np.float32)
    vals = vals[np.isfinite(vals)]
    for delta in (1.0, 0.75, 3.0, 1.0 / 3.0, 1e-3, 2.0 ** -20, 1.7e5, 7.3e-12):
        lim = np.float32(delta) * np.float32(oracle.qmax(fmt)) * np.float32(4.0)
        x = vals[np.abs(vals) <= lim]                      # include clear saturation cases
        pad = (-len(x)) % 16
        x = np.concatenate([x, np.zeros(pad, np.float32)])[None, None, :]
        d = np.array([delta], np.float32)
        want = oracle.quantize(x, fmt, d)
        t = torch.from_numpy(x[0]).to(torch.bfloat16).cuda()
        assert np.array_equal(t.float().cpu().numpy(), x[0])
        codes, _, _, _ = qm.qm_quantize(qm.operand_of(t, -1), fmt, "tensor", torch.from_numpy(d).cuda())
        got = codes.cpu().numpy()
        bad = np.nonzero(got != want)
        assert bad[0].size == 0, (fmt, delta, x[bad][:5], got[bad][:5], want[bad][:5])


def test_zero_tensor_and_zero_rows():
    t = torch.zeros((40, 64), dtype=torch.bfloat16)
    t[3, 5] = -2.0
    td = t.cuda()
    op = qm.operand_of(td, -1)
    d = qm.qm_scale(op, "e4m3", "channel").cpu().numpy()
    want = oracle.scale(as3(t.float().numpy()), "e4m3", "channel").ravel()
    assert np.array_equal(d, want) and d[0] == 1.0
    codes, _, _, _ = qm.qm_quantize(op, "e4m3", "channel", None)
    c = codes.cpu().numpy()[0]
    assert c[3, 5] == 0xFE and c.sum() == 0xFE
    z = torch.zeros((16, 32), dtype=torch.bfloat16).cuda()
    assert qm.qm_scale(qm.operand_of(z, -1), "int8", "tensor").item() == 1.0


def test_nonfinite_input_is_flagged_in_delta():
    t = torch.ones((8, 64), dtype=torch.bfloat16)
    t[2, 3] = float("inf")
    d = qm.qm_scale(qm.operand_of(t.cuda(), -1), "int8", "channel").cpu().numpy()
    assert not np.isfinite(d[2]) and np.isfinite(np.delete(d, 2)).all()
    t[2, 3] = float("nan")
    d = qm.qm_scale(qm.operand_of(t.cuda(), -1), "int8", "tensor").cpu().numpy()
    assert not np.isfinite(d[0])


def test_large_tensor_sampled():
    # a size that spans every SM several times; scales exact, codes compared on sampled rows
    t = make((4096, 3072), torch.bfloat16, 5, "n")
    td = t.cuda()
    x = as3(t.float().numpy())
    for gran in ("tensor", "channel"):
        for cd in (-1, -2):
            op = qm.operand_of(td, cd)
            xo = as3(oriented(t, cd))
            want_d = oracle.scale(xo, "e4m3", gran)
            codes, d, _, _ = qm.qm_quantize(op, "e4m3", gran, None)
            assert np.array_equal(d.cpu().numpy(), want_d.ravel())
            rows = np.random.default_rng(6).choice(xo.shape[1], 64, replace=False)
            dsel = want_d if gran == "tensor" else want_d[:, rows]
            want_c = oracle.quantize(xo[:, rows, :], "e4m3", dsel)
            assert np.array_equal(codes.cpu().numpy()[:, rows, :xo.shape[2]], want_c)


def adversarial_deltas(rng, n_random):
    """Scales whose reciprocal or quotients are awkward: significands of all ones, one ulp above a
    power of two, thirds and sevenths, plus log-uniform random ones."""
    bits = []
    for e in (100, 117, 127, 130, 150):                     # biased exponents well inside the range
        for m in (0x7FFFFF, 0x7FFFFE, 0x000001, 0x000000, 0x2AAAAB, 0x555555, 0x124925, 0x400000, 0x7FF000):
            bits.append((e << 23) | m)
    d = np.array(bits, dtype=np.uint32).view(np.float32)
    r = np.exp(rng.uniform(np.log(1e-6), np.log(1e6), n_random)).astype(np.float32)
    return np.concatenate([d, r])


@pytest.mark.parametrize("fmt", FMTS)
def test_quotient_is_exact_for_many_scales_bf16(fmt):
    # all finite bf16 inputs against ~250 scales in one call (one scale per row)
    rng = np.random.default_rng(50)
    deltas = adversarial_deltas(rng, 203)          # 248 rows: a multiple of 8 for the transposed view
    bits = np.arange(65536, dtype=np.uint32)
    vals = (bits << 16).view(np.float32)
    vals = np.where(np.isfinite(vals), vals, 0.0).astype(np.float32)
    x = np.tile(vals, (len(deltas), 1))
    lim = (deltas * np.float32(oracle.qmax(fmt)) * np.float32(4.0))[:, None]
    x = np.where(np.abs(x) <= lim, x, 0.0).astype(np.float32)[None]       # [1, rows, 65536]
    want = oracle.quantize(x, fmt, deltas[None, :])
    t = torch.from_numpy(x[0]).to(torch.bfloat16).cuda()
    codes, _, _, _ = qm.qm_quantize(qm.operand_of(t, -1), fmt, "channel", torch.from_numpy(deltas).cuda())
    got = codes.cpu().numpy()
    bad = np.nonzero(got != want)
    assert bad[0].size == 0, (fmt, bad[0].size, deltas[bad[1][:5]], x[bad][:5], got[bad][:5], want[bad][:5])
    # the same scales through the transposing kernel (one scale per column)
    tt = t.t().contiguous()                                               # [65536, rows]
    codes_t, _, _, _ = qm.qm_quantize(qm.operand_of(tt, -2), fmt, "channel", torch.from_numpy(deltas).cuda())
    assert np.array_equal(codes_t.cpu().numpy(), want)


@pytest.mark.parametrize("fmt", FMTS)
def test_quotient_is_exact_for_fp32_inputs(fmt):
    # fp32 operands have full 24-bit significands: random values near the rounding boundaries
    rng = np.random.default_rng(51)
    deltas = adversarial_deltas(rng, 150)
    g = oracle.positive_grid(fmt)
    mid = ((g[:-1] + g[1:]) / 2).astype(np.float32)
    base = rng.choice(np.concatenate([mid, g[1:].astype(np.float32)]), (len(deltas), 2048)).astype(np.float32)
    x = base * deltas[:, None]                                            # lands near ties and grid points
    jitter = rng.integers(-3, 4, x.shape)
    x = (x.view(np.int32) + jitter).view(np.float32)                      # a few ulps either side
    x = (x * rng.choice([-1.0, 1.0], x.shape)).astype(np.float32)[None]
    want = oracle.quantize(x, fmt, deltas[None, :])
    t = torch.from_numpy(x[0]).cuda()
    codes, _, _, _ = qm.qm_quantize(qm.operand_of(t, -1), fmt, "channel", torch.from_numpy(deltas).cuda())
    got = codes.cpu().numpy()
    bad = np.nonzero(got != want)
    assert bad[0].size == 0, (fmt, bad[0].size, deltas[bad[1][:5]], x[bad][:5], got[bad][:5], want[bad][:5])


def test_extreme_scales_take_the_division_path():
    # deltas outside 2^-60 .. 2^60, including subnormal ones
    for d in (1e-30, 3e-39, 1e-44, 2.5e25, 1e32):
        d32 = np.float32(d)
        vals = (np.arange(1, 20000, dtype=np.float32) * d32 * np.float32(0.013)).astype(np.float32)
        vals = vals[np.isfinite(vals)]
        vals = np.concatenate([vals, -vals])
        pad = (-len(vals)) % 16
        x = np.concatenate([vals, np.zeros(pad, np.float32)])[None, None, :]
        dd = np.array([d32], np.float32)
        want = oracle.quantize(x, "e4m3", dd)
        t = torch.from_numpy(x[0]).cuda()
        codes, _, _, _ = qm.qm_quantize(qm.operand_of(t, -1), "e4m3", "tensor", torch.from_numpy(dd).cuda())
        assert np.array_equal(codes.cpu().numpy(), want), d


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_supplied_scale_that_overflows_the_quotient_saturates(fmt, dtype):
    """A scale handed in from elsewhere can make x / delta exceed the float32 range; such elements
    saturate at the largest expressible value (codes against the oracle, bit for bit)."""
    t = make((40, 64), dtype, 9)
    t[0, 0] = 3e38; t[1, 5] = -3e38; t[2, 7] = 1e30; t[3, 3] = -2.5e35
    for dv in (1e-12, 3e-9, 2.0 ** -70):          # the corrected-reciprocal path and the division path
        d = np.array([dv], dtype=np.float32)
        x = as3(oriented(t, -1))
        want = oracle.quantize(x, fmt, d)
        codes, _, _, _ = qm.qm_quantize(qm.operand_of(t.cuda(), -1), fmt, "tensor", torch.from_numpy(d).cuda())
        assert np.array_equal(codes.cpu().numpy()[..., :64], want)
        v = oracle.dequantize(want, fmt)
        assert v[0, 0, 0] == oracle.qmax(fmt) and v[0, 1, 5] == -oracle.qmax(fmt)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("fused", [False, True])
def test_codes_bf16_strided_in_whole_tiles(fmt, gran, fused):
    """Strided contraction in whole 128 x 64 tiles: the shared-memory transposing kernel (several
    tiles in both directions, batched, scales per tensor and per output row, finished or fused)."""
    t = make((3, 256, 192), torch.bfloat16, 5)             # [b][c = 256][nc = 192], contraction strided
    td = t.cuda()
    op = qm.operand_of(td, -2)
    x = as3(oriented(t, -2))
    want_d = oracle.scale(x, fmt, gran)
    want_c = oracle.quantize(x, fmt, want_d)
    if fused:
        codes, d, _, km = qm.qm_quantize(op, fmt, gran, None, want_kmaj=True)
    else:
        d = qm.qm_scale(op, fmt, gran)
        codes, _, _, km = qm.qm_quantize(op, fmt, gran, d, want_kmaj=True)
    torch.cuda.synchronize()
    assert np.array_equal(d.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32))
    assert np.array_equal(codes.cpu().numpy(), want_c)
    assert torch.equal(km.cpu(), torch.from_numpy(x).to(torch.bfloat16))


@pytest.mark.parametrize("fmt", FMTS)
def test_strided_tiles_with_a_scale_from_elsewhere_saturate(fmt):
    """A supplied scale far below the operand's own drives x / delta past the float range: the codes
    saturate at the format's largest magnitude (Methodology, saturation rule), as the oracle's do."""
    t = make((256, 128), torch.bfloat16, 6) * 1e30
    op = qm.operand_of(t.cuda(), -2)
    x = as3(oriented(t, -2))
    tiny = np.array([1e-12], dtype=np.float32)
    want = oracle.quantize(x, fmt, tiny)
    codes, _, _, _ = qm.qm_quantize(op, fmt, "tensor", torch.from_numpy(tiny).cuda())
    assert np.array_equal(codes.cpu().numpy(), want)
    dense, _, _, _ = qm.qm_quantize(qm.operand_of(t.cuda(), -1), fmt, "tensor", torch.from_numpy(tiny).cuda())
    assert np.array_equal(dense.cpu().numpy(), oracle.quantize(as3(oriented(t, -1)), fmt, tiny))


@pytest.mark.parametrize("fmt", ["e4m3", "int8"])
def test_dense_tensors_off_the_32_byte_grid(fmt):
    """The dense kernels use 256-bit loads on the 32-byte aligned middle of a tensor: a tensor that
    starts 16 bytes past such a boundary, and one whose size leaves a 16-byte tail, still give the
    oracle's scale and codes (the ends go through the general kernels or the 128-bit variant)."""
    base = make((1 << 20) + 64, torch.bfloat16, 7).reshape(-1)
    dev = base.cuda()
    for off, rows, cols in ((8, 512, 1024), (0, 33, 72), (8, 129, 4088), (24, 1024, 512)):
        t = base[off:off + rows * cols].reshape(rows, cols)
        td = dev[off:off + rows * cols].view(rows, cols)
        assert td.data_ptr() % 16 == 0
        op = qm.operand_of(td, -1)
        x = as3(oriented(t, -1))
        want_d = oracle.scale(x, fmt, "tensor")
        d = qm.qm_scale(op, fmt, "tensor")
        assert np.array_equal(d.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32)), (off, rows, cols)
        if cols % 16 == 0:
            codes, _, _, _ = qm.qm_quantize(op, fmt, "tensor", d)
            assert np.array_equal(codes.cpu().numpy()[..., :cols], oracle.quantize(x, fmt, want_d)), (off, rows, cols)
