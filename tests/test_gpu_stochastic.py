"""GPU parity of stochastic rounding (second rounding mode of the Methodology section): codes
bit for bit against the oracle, which draws the same Philox4x32-10 numbers by element index, and
the probe with a stochastically rounded operand."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oriented, as3, assert_record_close

pytestmark = pytest.mark.gpu
FMTS = ["int8", "e4m3", "e5m2"]


def to_dev(t):
    if t.is_contiguous():
        return t.cuda()
    return torch.as_strided(t._base.cuda(), t.shape, t.stride(), t.storage_offset())


def check_codes(t, contract_dim, fmt, gran, seed, stream_id, fused=False):
    op = qm.operand_of(to_dev(t), contract_dim)
    x = as3(oriented(t, contract_dim))
    d = oracle.scale(x, fmt, gran)
    want = oracle.quantize(x, fmt, d, "stochastic", seed, stream_id)
    if fused:
        codes, dout, ab, km = qm.qm_quantize(op, fmt, gran, None, want_abs=True, stochastic=(seed, stream_id))
        assert np.array_equal(dout.cpu().numpy().view(np.uint32), d.ravel().view(np.uint32))
    else:
        codes, _, ab, km = qm.qm_quantize(op, fmt, gran, qm.qm_scale(op, fmt, gran), want_abs=True,
                                          want_kmaj=(contract_dim == -2), stochastic=(seed, stream_id))
    torch.cuda.synchronize()
    c = codes.cpu().numpy()
    K = x.shape[-1]
    assert np.array_equal(c[..., :K], want)
    assert not c[..., K:].any()
    assert torch.equal(ab.cpu(), torch.from_numpy(x).to(torch.bfloat16).abs())
    rt = oracle.quantize(x, fmt, d)
    assert (want != rt).mean() > 0.05                 # the case is not accidentally all on the grid
    return want


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_codes_contiguous(fmt, gran, dtype):
    rng = workloads._rng(41)
    t = workloads.student_t(rng, (200, 176), 4.0, dtype=dtype)
    check_codes(t, -1, fmt, gran, seed=(5 << 32) | 77, stream_id=0)
    check_codes(t, -1, fmt, gran, seed=3, stream_id=1, fused=True)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_codes_strided_ragged_and_batched(fmt, gran):
    rng = workloads._rng(42)
    check_codes(workloads.normal(rng, (176, 136), 1e-3), -2, fmt, gran, 9, 1)       # contraction strided
    base = workloads.normal(rng, (3, 40, 72))
    check_codes(base[:, :, :70], -1, fmt, gran, 10, 0)                               # odd row length: blocks of 4 straddle rows
    check_codes(workloads.normal(rng, (2, 72, 40)), -2, fmt, gran, 11, 0)


def test_same_draws_on_either_layout():
    rng = workloads._rng(43)
    t = workloads.normal(rng, (128, 96))
    a = check_codes(t, -1, "e4m3", "tensor", 21, 0)
    b = check_codes(t.t().contiguous().t(), -1, "e4m3", "tensor", 21, 0)             # same values, other strides
    assert np.array_equal(a, b)


def test_round_up_frequency_on_the_gpu():
    n = 1 << 20
    x = torch.full((1024, n // 1024), 0.3)
    x[0, 0] = 127.0
    codes, *_ = qm.qm_quantize(qm.operand_of(x.cuda(), -1), "int8", "tensor", None, stochastic=(1234, 0))
    c = codes.cpu().numpy().astype(np.int8).ravel()[1:]
    assert set(np.unique(c)) == {0, 1}
    assert abs(c.mean() - 0.3) < 4 * (0.21 / n) ** 0.5 + 1e-4     # fp32(0.3) is 0.3 to 1e-8


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("which", ["stochastic_l", "stochastic_r", "stochastic_both"])
def test_probe_with_stochastic_operands(fmt, which):
    rng = workloads._rng(44)
    M, N, K = 200, 136, 176
    L = workloads.normal(rng, (M, K))
    R = workloads.lognormal_signed(rng, (K, N), -8.0, 2.0)
    res = qm.qm_probe_layer(qm.operand_of(L.cuda(), -1), qm.operand_of(R.cuda(), -2), fmt, fmt, "tensor", "tensor",
                            rounding=which, seed=99)
    assert res.device_error == 0
    want = oracle.probe(L.float().numpy(), R.float().numpy(), fmt, fmt, "tensor", "tensor",
                        round_l="stochastic" if which in ("stochastic_l", "stochastic_both") else "rtne",
                        round_r="stochastic" if which in ("stochastic_r", "stochastic_both") else "rtne", seed=99)
    assert_record_close(res.record(), want, what=f"{fmt} {which}")
    rt = qm.qm_probe_layer(qm.operand_of(L.cuda(), -1), qm.operand_of(R.cuda(), -2), fmt, fmt, "tensor", "tensor")
    assert rt.sum_be != res.sum_be


def test_probe_channel_scales_and_wgrad_layout():
    rng = workloads._rng(45)
    X = workloads.normal(rng, (256, 96))                 # [tokens, features]
    dY = workloads.normal(rng, (256, 64), 1e-3)          # [tokens, out]; wgrad contracts over tokens: both strided
    res = qm.qm_probe_layer(qm.operand_of(X.cuda(), -2), qm.operand_of(dY.cuda(), -2), "e4m3", "e5m2", "channel",
                            "channel", rounding="stochastic_r", seed=7)
    want = oracle.probe(X.float().numpy().T.copy(), dY.float().numpy(), "e4m3", "e5m2", "channel", "channel",
                        round_r="stochastic", seed=7)
    assert_record_close(res.record(), want, what="wgrad")
