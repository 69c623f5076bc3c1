"""Two formats in one pass (qm_probe_layer2): the reference and denominator products are
computed once, each format keeps its own 8-bit accumulator; every record must be the record the
one-format probe gives, and must match the oracle's probe of that format."""
import numpy as np
import pytest
import torch

import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oracle_probe, assert_record_close

pytestmark = pytest.mark.gpu


def both(o, fa, fb, **kw):
    Ld, Rd = o["L"].cuda(), o["R"].cuda()
    Lop, Rop = qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"])
    two = qm.qm_probe_layer2(Lop, Rop, fa, fb, o["gran_l"], o["gran_r"], **kw)
    one = [qm.qm_probe_layer(Lop, Rop, f[0], f[1], o["gran_l"], o["gran_r"], **kw) for f in (fa, fb)]
    return two, one


def agree(a, b):
    """The two-format kernel and the one-format kernel evaluate Eq. 3 in fp32 per row of a tile with
    the operations in a different order (the one-format kernel folds the two scales into one factor
    and splits narrow tiles 32 columns per warp), so their records agree to fp32 rounding of those
    row sums, not bit for bit: 1e-6 on the sums, 1e-5 on the maximum (one element's quotient)."""
    assert a["count"] == b["count"]
    for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(a[k] - b[k]) <= 1e-6 * abs(b[k]), (k, a[k], b[k])
    assert abs(a["max_be"] - b["max_be"]) <= 1e-5 * abs(b["max_be"]), (a["max_be"], b["max_be"])
    return True


PAIRS = [(("e4m3", "e4m3"), ("int8", "int8")), (("int8", "int8"), ("e5m2", "e5m2")),
         (("e4m3", "e4m3"), ("e5m2", "e5m2")), (("e5m2", "e4m3"), ("e4m3", "e5m2"))]


@pytest.mark.parametrize("fa,fb", PAIRS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("layout", [(-1, -2), (-1, -1), (-2, -2)])
def test_two_formats_small_ragged(fa, fb, gran, layout):
    rng = workloads._rng(60)
    M, N, K = 200, 136, 176
    L = workloads.student_t(rng, (M, K) if layout[0] == -1 else (K, M), 4.0)
    R = workloads.normal(rng, (K, N) if layout[1] == -2 else (N, K), 0.05)
    o = workloads.op("small", L, layout[0], R, layout[1], fa[0], fa[1], gran, gran)
    two, one = both(o, fa, fb)
    for got, single, f in zip(two, one, (fa, fb)):
        assert got.device_error == 0
        assert agree(got.record(), single.record()), f
        oo = dict(o, fmt_l=f[0], fmt_r=f[1])
        assert_record_close(got.record(), oracle_probe(oo), what=str((f, gran, layout)))


def test_two_formats_many_tiles_and_batches():
    rng = workloads._rng(61)
    # several tiles per CTA pair, ragged M and N, 40 k-blocks
    o = workloads.op("big", workloads.normal(rng, (2000, 2560)), -1, workloads.normal(rng, (2560, 1096), 0.02), -2,
                     "e4m3", "e4m3")
    two, one = both(o, ("e4m3", "e4m3"), ("int8", "int8"))
    assert agree(two[0].record(), one[0].record()) and agree(two[1].record(), one[1].record())
    # batched attention-like product, channel scales shared per head
    Q = workloads.normal(rng, (12, 136, 64))
    Kt = workloads.normal(rng, (12, 200, 64))
    o = workloads.op("attn", Q, -1, Kt, -1, "e5m2", "e5m2", "channel", "channel")
    two, one = both(o, ("e5m2", "e5m2"), ("int8", "int8"), groups=(4, 4))
    assert agree(two[0].record(), one[0].record()) and agree(two[1].record(), one[1].record())
    # a stochastically rounded gradient operand
    dY = workloads.lognormal_signed(rng, (256, 64), -8.0, 2.0)
    X = workloads.normal(rng, (256, 96))
    o = workloads.op("wgrad", X, -2, dY, -2, "e4m3", "e5m2")
    two, one = both(o, ("e4m3", "e5m2"), ("int8", "int8"), rounding="stochastic_r", seed=5)
    assert agree(two[0].record(), one[0].record()) and agree(two[1].record(), one[1].record())


def test_two_formats_k64_and_repeat():
    rng = workloads._rng(62)
    o = workloads.op("k64", workloads.normal(rng, (512, 64)), -1, workloads.normal(rng, (64, 384)), -2, "e4m3", "e4m3")
    Ld, Rd = o["L"].cuda(), o["R"].cuda()
    Lop, Rop = qm.operand_of(Ld, -1), qm.operand_of(Rd, -2)
    plan = qm.ProbePlan2(Lop, Rop, ("e4m3", "e4m3"), ("int8", "int8"), "tensor", "tensor")
    recs = []
    for _ in range(3):                       # the workspace is reused as it is
        plan.launch(Lop, Rop)
        torch.cuda.synchronize()
        recs.append([r.record() for r in plan.results()])
    assert recs[0] == recs[1] == recs[2]
    assert agree(recs[0][0], qm.qm_probe_layer(Lop, Rop, "e4m3", "e4m3", "tensor", "tensor").record())


def test_two_formats_refusals():
    rng = workloads._rng(63)
    Lop = qm.operand_of(workloads.normal(rng, (128, 64)).cuda(), -1)
    Rop = qm.operand_of(workloads.normal(rng, (64, 128)).cuda(), -2)
    with pytest.raises(qm.QmError):
        qm.qm_probe_layer2(Lop, Rop, ("int8", "int8"), ("int8", "int8"), "tensor", "tensor")
    with pytest.raises(qm.QmError):
        qm.qm_probe_layer2(Lop, Rop, ("e4m3", "int8"), ("e5m2", "e5m2"), "tensor", "tensor")
