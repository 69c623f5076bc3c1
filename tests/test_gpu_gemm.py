"""GPU parity: 8-bit products (exact for INT8), reference/denominator products and the
stand-alone Eq. 3 reduction."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm

pytestmark = pytest.mark.gpu


def rand_codes(rng, fmt, shape):
    t = oracle.decode_table(fmt)
    ok = np.array([c for c in range(256) if np.isfinite(t[c]) and not (fmt == "int8" and c == 128)], np.uint8)
    return rng.choice(ok, shape).astype(np.uint8)


def pad_codes(c):
    K = c.shape[-1]
    ld = (K + 15) // 16 * 16
    out = np.zeros(c.shape[:-1] + (ld,), np.uint8)
    out[..., :K] = c
    return out


def run_gemm(fl, fr, b, M, N, K, gl, gr, simt, seed, small=False):
    rng = np.random.default_rng(seed)
    if small:   # small-magnitude FP8 codes so that every fp32 sum is exact
        cl = rng.choice(np.array([0x30, 0x38, 0x3C, 0x40, 0xB8, 0xC0, 0x00], np.uint8), (b, M, K))
        cr = rng.choice(np.array([0x30, 0x38, 0x3C, 0x40, 0xB8, 0xC0, 0x00], np.uint8), (b, N, K))
    else:
        cl, cr = rand_codes(rng, fl, (b, M, K)), rand_codes(rng, fr, (b, N, K))
    dl = rng.uniform(0.5, 2.0, (1,) if gl == "tensor" else (b, M)).astype(np.float32)
    dr = rng.uniform(0.5, 2.0, (1,) if gr == "tensor" else (b, N)).astype(np.float32)
    acc = oracle.gemm_lp(cl, fl, cr, fr)
    from oracle.probe import descale
    want = descale(acc, dl, dr)
    out, raw = qm.qm_gemm(torch.from_numpy(pad_codes(cl)).cuda(), fl, torch.from_numpy(dl.ravel()).cuda(), gl,
                          torch.from_numpy(pad_codes(cr)).cuda(), fr, torch.from_numpy(dr.ravel()).cuda(), gr,
                          K, want_raw=True, use_simt=simt)
    torch.cuda.synchronize()
    return acc, want, out.cpu().numpy().astype(np.float64), raw.cpu().numpy(), (cl, cr, dl, dr)


@pytest.mark.parametrize("simt", [False, True])
@pytest.mark.parametrize("shape", [(1, 128, 128, 64), (1, 200, 136, 176), (3, 130, 72, 48), (1, 384, 256, 1024)])
@pytest.mark.parametrize("gran", [("tensor", "tensor"), ("channel", "channel")])
def test_int8_gemm_exact(simt, shape, gran):
    b, M, N, K = shape
    acc, want, out, raw, _ = run_gemm("int8", "int8", b, M, N, K, gran[0], gran[1], simt, 20)
    assert raw.dtype == np.int32
    assert np.array_equal(raw.astype(np.int64), acc.astype(np.int64))      # bit-exact accumulators
    assert np.allclose(out, want, rtol=3e-7, atol=0)


@pytest.mark.parametrize("simt", [False, True])
@pytest.mark.parametrize("fmts", [("e4m3", "e4m3"), ("e5m2", "e4m3"), ("e4m3", "e5m2"), ("e5m2", "e5m2")])
def test_fp8_gemm_exact_on_small_values(simt, fmts):
    # operands chosen so that all partial sums are exactly representable: equality required
    acc, want, out, raw, _ = run_gemm(fmts[0], fmts[1], 2, 136, 200, 192, "tensor", "tensor", simt, 21, small=True)
    assert np.array_equal(raw.astype(np.float64), acc)


@pytest.mark.parametrize("simt", [False, True])
@pytest.mark.parametrize("fmts", [("e4m3", "e4m3"), ("e5m2", "e4m3"), ("e4m3", "e5m2")])
@pytest.mark.parametrize("shape", [(1, 256, 384, 512), (2, 100, 260, 1040)])
def test_fp8_gemm_within_tolerance(simt, fmts, shape):
    b, M, N, K = shape
    acc, want, out, raw, (cl, cr, dl, dr) = run_gemm(fmts[0], fmts[1], b, M, N, K, "channel", "channel", simt, 22)
    # tolerance on outputs: 1e-3 of the backward-error scale |Lbar|.|Rbar| delta_l delta_r
    from oracle.probe import descale
    scale = descale(np.matmul(np.abs(oracle.dequantize(cl, fmts[0])),
                              np.swapaxes(np.abs(oracle.dequantize(cr, fmts[1])), -1, -2)), dl, dr)
    err = np.abs(out - want) / scale
    assert err.max() <= 1e-3, err.max()
    assert np.abs(out - want).max() / np.abs(want).max() <= 1e-3
    print("fp8 gemm", fmts, "simt" if simt else "tc", "max err / scale =", err.max())


@pytest.mark.parametrize("shape", [(1, 128, 128, 64), (1, 300, 200, 528), (4, 64, 136, 128), (1, 512, 512, 2048)])
def test_reference_and_denominator_products(shape):
    b, M, N, K = shape
    rng = np.random.default_rng(23)
    l = torch.from_numpy(rng.standard_normal((b, M, K)).astype(np.float32)).to(torch.bfloat16)
    r = torch.from_numpy(rng.standard_normal((b, N, K)).astype(np.float32)).to(torch.bfloat16)
    c = qm.qm_gemm_ref(l.cuda(), r.cuda()).cpu().numpy().astype(np.float64)
    d = qm.qm_gemm_ref(l.abs().cuda(), r.abs().cuda()).cpu().numpy().astype(np.float64)
    want_c = oracle.gemm_ref(l.float().numpy(), r.float().numpy())
    want_d = oracle.gemm_den(l.float().numpy(), r.float().numpy())
    assert (np.abs(c - want_c) / want_d).max() <= 1e-3
    assert (np.abs(d - want_d) / want_d).max() <= 1e-3
    print("ref gemm max err / D =", (np.abs(c - want_c) / want_d).max(), (np.abs(d - want_d) / want_d).max())


def test_reference_product_exact_on_small_integers():
    rng = np.random.default_rng(24)
    l = torch.from_numpy(rng.integers(-8, 9, (1, 200, 320)).astype(np.float32)).to(torch.bfloat16)
    r = torch.from_numpy(rng.integers(-8, 9, (1, 136, 320)).astype(np.float32)).to(torch.bfloat16)
    c = qm.qm_gemm_ref(l.cuda(), r.cuda()).cpu().numpy().astype(np.float64)
    assert np.array_equal(c, oracle.gemm_ref(l.float().numpy(), r.float().numpy()))


@pytest.mark.parametrize("n", [1, 1000, 128 * 128, 1234567])
def test_metric_reduction(n):
    rng = np.random.default_rng(25)
    c = rng.standard_normal(n).astype(np.float32)
    d = (np.abs(c) + rng.uniform(0, 2, n)).astype(np.float32)
    q = (c + rng.standard_normal(n) * 0.01 * d).astype(np.float32)
    d[:: 97] = 0.0
    res = qm.qm_metric(torch.from_numpy(c).cuda(), torch.from_numpy(q).cuda(), torch.from_numpy(d).cuda())
    want = oracle.metric(c, q, d)
    got = res.record()
    assert got["count"] == n and res.device_error == 0
    for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(got[k] - want[k]) <= 1e-5 * abs(want[k]) + 1e-30, (k, got[k], want[k])
    assert abs(got["max_be"] - want["max_be"]) <= 1e-6 * want["max_be"]


# ------------------------------------------------------------------ 256-column tiles (outputs at least 256 wide)
@pytest.mark.parametrize("shape", [(1, 300, 600, 144), (2, 130, 258, 272), (1, 4096, 3072, 256), (3, 256, 512, 1040)])
@pytest.mark.parametrize("gran", [("tensor", "tensor"), ("channel", "channel")])
def test_int8_gemm_exact_on_wide_outputs(shape, gran):
    # ragged last tile, a width that is not a multiple of 4 (scalar stores), a contraction that is
    # not a multiple of the 128-code k-block, several tiles per CTA pair (both accumulator buffers
    # reused), batches
    b, M, N, K = shape
    acc, want, out, raw, _ = run_gemm("int8", "int8", b, M, N, K, gran[0], gran[1], False, 27)
    assert np.array_equal(raw.astype(np.int64), acc.astype(np.int64))
    assert np.allclose(out, want, rtol=3e-7, atol=0)


@pytest.mark.parametrize("fmts", [("e4m3", "e4m3"), ("e5m2", "e4m3")])
def test_fp8_gemm_exact_on_wide_outputs(fmts):
    acc, want, out, raw, _ = run_gemm(fmts[0], fmts[1], 1, 2304, 2560, 400, "channel", "tensor", False, 28, small=True)
    assert np.array_equal(raw.view(np.float32).astype(np.float64), acc)


def test_reference_product_wide_many_tiles():
    rng = np.random.default_rng(29)
    l = torch.from_numpy(rng.integers(-4, 5, (1, 4096, 192)).astype(np.float32)).to(torch.bfloat16)
    r = torch.from_numpy(rng.integers(-4, 5, (1, 2816, 192)).astype(np.float32)).to(torch.bfloat16)
    out = qm.qm_gemm_ref(l.cuda(), r.cuda()).cpu().numpy()
    want = l.float().numpy().astype(np.float64) @ np.swapaxes(r.float().numpy().astype(np.float64), -1, -2)
    assert np.array_equal(out.astype(np.float64), want)          # small integers: every sum exact
