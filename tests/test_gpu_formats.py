"""qm_quantize_formats: the codes and scales of several formats from one pass over an operand are,
bit for bit, the oracle's codes and scales of each format alone (Eq. 1 per format)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from helpers import oriented, as3

pytestmark = pytest.mark.gpu
SETS = [("e4m3", "int8"), ("int8", "e5m2"), ("e5m2", "e4m3"), ("e4m3", "e5m2", "int8"), ("e5m2",)]


def tensor(shape, dtype, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return torch.from_numpy((rng.standard_t(3, shape) * scale).astype(np.float32)).to(dtype)


def check(t, contract_dim, fmts, gran, want_kmaj=False):
    td = t.cuda()
    op = qm.operand_of(td, contract_dim)
    x = as3(oriented(t, contract_dim))
    codes, deltas, km = qm.qm_quantize_formats(op, list(fmts), gran, want_kmaj=want_kmaj)
    torch.cuda.synchronize()
    K = x.shape[-1]
    for f, c, d in zip(fmts, codes, deltas):
        want_d = oracle.scale(x, f, gran)
        want_c = oracle.quantize(x, f, want_d)
        assert np.array_equal(d.cpu().numpy().view(np.uint32), want_d.ravel().view(np.uint32)), f
        got = c.cpu().numpy()
        assert np.array_equal(got[..., :K], want_c), f
        assert not got[..., K:].any(), f
    if km is not None:
        assert torch.equal(km.cpu(), torch.from_numpy(x).to(torch.bfloat16))


@pytest.mark.parametrize("fmts", SETS)
def test_dense_bf16_one_pass(fmts):
    check(tensor((520, 1024), torch.bfloat16, 41), -1, fmts, "tensor")            # small grid variant
    check(tensor((3, 136, 64), torch.bfloat16, 42, 1e-3), -1, fmts, "tensor")      # batched, dense


@pytest.mark.parametrize("fmts", SETS)
def test_transposing_bf16_one_pass(fmts):
    # strided contraction, enough tiles for the register-tiled kernel: [c = 4096][nc = 2048]
    check(tensor((4096, 2048), torch.bfloat16, 43), -2, fmts, "tensor", want_kmaj=True)


def test_large_dense_takes_the_four_chunk_variant():
    check(tensor((16384, 4096), torch.bfloat16, 44, 0.02), -1, ("e4m3", "e5m2", "int8"), "tensor")


@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_cases_served_format_by_format(gran):
    fm = ("e4m3", "int8", "e5m2")
    check(tensor((333, 200), torch.bfloat16, 45), -1, fm, gran)                    # ragged rows
    check(tensor((333, 200), torch.bfloat16, 46), -2, fm, gran, want_kmaj=True)    # small strided contraction
    check(tensor((130, 264), torch.float32, 47), -1, fm, gran)                     # fp32 input
    check(tensor((2, 72, 40), torch.float32, 48), -2, fm, gran)


def test_signed_zero_subnormals_and_extreme_scales():
    """Negative zeros keep their sign in the FP8 codes, subnormal inputs quantize to zero codes, and
    scales outside the fast range of the two-wide quotient fall back to the division."""
    t = tensor((64, 64), torch.bfloat16, 49)
    t[0, :8] = torch.tensor([-0.0, 0.0, -1e-39, 1e-39, -2.0 ** -130, 2.0 ** -133, -0.0, 3.0]).to(torch.bfloat16)
    check(t, -1, ("e4m3", "e5m2", "int8"), "tensor")
    check((t.float() * 2.0 ** 80).to(torch.bfloat16), -1, ("e4m3", "e5m2", "int8"), "tensor")    # delta above 2^60 for int8/e4m3
    check((t.float() * 2.0 ** -90).to(torch.bfloat16), -1, ("e4m3", "e5m2", "int8"), "tensor")   # delta below 2^-60
    z = torch.zeros((32, 64), dtype=torch.bfloat16)
    check(z, -1, ("e4m3", "int8"), "tensor")                                                     # all-zero group: delta = 1


def test_argument_checks():
    op = qm.operand_of(torch.ones((8, 64), dtype=torch.bfloat16, device="cuda"), -1)
    with pytest.raises(qm.QmError):
        qm.qm_quantize_formats(op, ["e4m3", "e4m3"], "tensor")          # formats must be distinct
    with pytest.raises(qm.QmError):
        qm.qm_quantize_formats(op, [], "tensor")
