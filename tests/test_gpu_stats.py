"""GPU parity of the single-tensor passes against the oracle: the tensor statistics of the
Experiments section and the Eq. 2 clipping / rounding split of the Results section.

Tolerances (from the arithmetic: per-element values carry one or two fp32 roundings, 32 of
them are summed in fp32, everything above that in fp64): counts and max|x| exact; a sum of
positive terms within 2e-6 relative; a signed sum within 2e-6 of the sum of magnitudes; derived
statistics of well-conditioned tensors within 1e-4; RE sums within 1e-5."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from helpers import oriented, as3

pytestmark = pytest.mark.gpu
FMTS = ["int8", "e4m3", "e5m2"]


def tensor(shape, dtype, seed, scale=1.0, dist="t"):
    rng = np.random.default_rng(seed)
    x = (rng.standard_t(4, shape) if dist == "t" else rng.gamma(2.0, 1.0, shape)) * scale
    return torch.from_numpy(x.astype(np.float32)).to(dtype)


def to_dev(t):
    """The tensor on the GPU with the strides it has on the CPU (a view of its base tensor)."""
    if t.is_contiguous():
        return t.cuda()
    return torch.as_strided(t._base.cuda(), t.shape, t.stride(), t.storage_offset())


def check_stats(t, contract_dim=-1):
    got = qm.qm_tensor_stats(qm.operand_of(to_dev(t), contract_dim))
    x = t.float().numpy().astype(np.float64)
    want = oracle.tensor_stats(t.float().numpy())
    assert got.device_error == 0
    assert got.count == want["count"] and got.max_abs == want["max_abs"]
    a = np.abs(x)
    assert abs(got.sum1 - want["sum1"]) <= 2e-6 * a.sum() + 1e-300
    assert abs(got.sum2 - want["sum2"]) <= 2e-6 * want["sum2"] + 1e-300
    assert abs(got.sum3 - want["sum3"]) <= 2e-6 * (a ** 3).sum() + 1e-300
    assert abs(got.sum4 - want["sum4"]) <= 2e-6 * want["sum4"] + 1e-300
    return got, want


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(1, 8), (3, 40), (257, 1000), (2, 130, 72), (1, 1)])
def test_stats_small(dtype, shape):
    check_stats(tensor(shape, dtype, 11))


def test_stats_derived_on_a_skewed_law():
    got, want = check_stats(tensor((512, 2048), torch.bfloat16, 12, dist="gamma"))
    d = got.derived()
    assert d["mean"] == pytest.approx(want["mean"], rel=1e-6)
    assert d["variance"] == pytest.approx(want["variance"], rel=1e-4)
    assert d["skew"] == pytest.approx(want["skew"], abs=1e-4)          # gamma(2): skew sqrt(2), kurtosis 6
    assert d["kurtosis"] == pytest.approx(want["kurtosis"], rel=1e-4)
    assert d["skew"] == pytest.approx(2 ** 0.5, abs=0.05) and d["kurtosis"] == pytest.approx(6.0, rel=0.1)


def test_stats_views_and_ragged_rows():
    base = tensor((300, 256), torch.bfloat16, 13)
    check_stats(base[:, :70])                         # rows of 70 inside rows of 256: ragged tail
    check_stats(base, contract_dim=-2)                # contraction strided: same elements
    b3 = tensor((4, 64, 128), torch.float32, 14)
    check_stats(b3[:, :, :33])
    check_stats(b3, contract_dim=-2)


def test_stats_large_dense_many_blocks():
    got, want = check_stats(tensor((4096, 4096), torch.bfloat16, 15, scale=0.02))
    assert got.derived()["kurtosis"] == pytest.approx(want["kurtosis"], rel=1e-4)
    again = qm.qm_tensor_stats(qm.operand_of(tensor((4096, 4096), torch.bfloat16, 15, scale=0.02).cuda(), -1))
    assert (again.sum1, again.sum2, again.sum3, again.sum4) == (got.sum1, got.sum2, got.sum3, got.sum4)


def test_stats_zero_constant_and_nonfinite():
    z = qm.qm_tensor_stats(qm.operand_of(torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda"), -1))
    assert (z.sum1, z.sum2, z.max_abs, z.count, z.device_error) == (0.0, 0.0, 0.0, 1024, 0)
    c = qm.qm_tensor_stats(qm.operand_of(torch.full((16, 64), 2.5, device="cuda"), -1))
    assert c.sum1 == 2.5 * 1024 and c.derived()["variance"] == 0.0 and c.derived()["skew"] == 0.0
    bad = torch.ones((8, 64), device="cuda")
    bad[3, 5] = float("inf")
    assert qm.qm_tensor_stats(qm.operand_of(bad, -1)).device_error == 1


def check_error(t, contract_dim, fmt, gran, delta=None):
    td = to_dev(t)
    op = qm.operand_of(td, contract_dim)
    x = as3(oriented(t, contract_dim))
    if delta is None:
        want = oracle.quantize_error(x, fmt, gran)
        got = qm.qm_quantize_error(op, fmt, gran)
    else:
        want = oracle.quantize_error(x, fmt, gran, delta=delta)
        got = qm.qm_quantize_error(op, fmt, gran, delta=torch.from_numpy(delta.ravel()).cuda())
    assert got.device_error == 0
    for k in ("count", "n_nonzero", "n_overflow", "n_underflow"):
        assert getattr(got, k) == want[k], (k, getattr(got, k), want[k])
    # the kernel squares in float32: a square below the normal range (2^-126) is lost there, so a sum
    # of squares carries that much absolute slack per element
    tiny = want["count"] * 2.0 ** -126
    for k in ("sum_re", "sum_re_round", "err2_round", "err2_overflow", "err2_underflow", "sum_x2"):
        slack = tiny if k.startswith("err2") or k == "sum_x2" else 1e-300
        assert abs(getattr(got, k) - want[k]) <= 1e-5 * abs(want[k]) + slack, (k, getattr(got, k), want[k])
    assert abs(got.max_re_round - want["max_re_round"]) <= 1e-6 * want["max_re_round"] + 1e-300
    return got, want


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_error_contiguous(fmt, gran, dtype):
    rng = np.random.default_rng(21)
    t = tensor((96, 200), dtype, 21) * torch.from_numpy(10.0 ** rng.uniform(-3, 1, (96, 1)).astype(np.float32)).to(dtype)
    t[5] = 0
    got, want = check_error(t, -1, fmt, gran)
    if fmt == "int8" and gran == "tensor":
        assert want["n_underflow"] > 0              # the case does exercise the underflow class


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_error_strided_contraction_and_batches(fmt, gran):
    check_error(tensor((176, 136), torch.bfloat16, 22), -2, fmt, gran)      # deltas follow the contiguous index
    check_error(tensor((3, 40, 72), torch.bfloat16, 23)[:, :, :70], -1, fmt, gran)
    check_error(tensor((3, 72, 40), torch.float32, 24), -2, fmt, gran)


@pytest.mark.parametrize("fmt", FMTS)
def test_error_with_outside_scale_overflows(fmt):
    t = tensor((64, 128), torch.float32, 25, scale=3.0)
    small = np.array([np.abs(t.numpy()).max() / oracle.qmax(fmt) / 8], dtype=np.float32)   # an eighth of the Eq. 1 scale
    got, want = check_error(t, -1, fmt, "tensor", delta=small)
    assert want["n_overflow"] > 0 and want["err2_overflow"] > 0


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_error_with_subnormal_elements(fmt, dtype):
    """Non-zero elements below the normal range of float32 (bf16 subnormals are float32 subnormals):
    their code is zero, so each is an underflow with RE exactly 1 and the sums stay finite."""
    t = tensor((32, 64), dtype, 27)
    sub = torch.tensor([1e-39, -3e-40, 2.0 ** -133, -2.0 ** -130], dtype=torch.float32).to(dtype)
    assert (sub != 0).all()
    t[3, 10:14] = sub
    t[7, 0] = sub[0]
    got, want = check_error(t, -1, fmt, "tensor")
    assert want["n_underflow"] >= 5 and np.isfinite(got.sum_re)
    check_error(t, -1, fmt, "channel")
    got_s, _ = check_stats(t)
    assert got_s.device_error == 0


def test_error_large_dense_and_repeatable():
    t = tensor((2048, 4096), torch.bfloat16, 26, scale=0.02)
    got, _ = check_error(t, -1, "e4m3", "tensor")
    again = qm.qm_quantize_error(qm.operand_of(t.cuda(), -1), "e4m3", "tensor")
    assert again.record() == got.record()


def test_error_argument_checks():
    t = torch.ones((8, 64), device="cuda")
    op = qm.operand_of(t, -1)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(qm.QmError):
        qm.qm_tensor_stats(op, ws=ws)                 # workspace too small
    bad = torch.ones((8, 64), device="cuda")
    bad[0, 0] = float("nan")
    r = qm.qm_quantize_error(qm.operand_of(bad, -1), "int8", "tensor", delta=torch.ones(1, device="cuda"))
    assert r.device_error == 1


def test_stats_dense_kernel_and_its_fallbacks_agree_with_the_oracle():
    """Large dense tensors take the 256-bit kernel; the same data 16 bytes off the 32-byte grid takes
    the general one: both against the oracle."""
    big = tensor((2048, 1024), torch.bfloat16, 16, scale=0.5)
    check_stats(big)                                           # 4 MB, aligned: the 256-bit kernel
    flat = torch.cat([big.reshape(-1), big.reshape(-1)[:8]])
    dev = flat.cuda()
    shifted = dev[8:].view(2048, 1024)
    got = qm.qm_tensor_stats(qm.operand_of(shifted, -1))
    want = oracle.tensor_stats(flat[8:].float().numpy().reshape(2048, 1024))
    assert got.count == want["count"] and got.max_abs == want["max_abs"]
    assert abs(got.sum2 - want["sum2"]) <= 2e-6 * want["sum2"] and abs(got.sum4 - want["sum4"]) <= 2e-6 * want["sum4"]
    f32 = tensor((1024, 1024), torch.float32, 17)
    check_stats(f32)                                           # fp32 through the same kernel
