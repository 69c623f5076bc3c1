"""Inside a batch, operands over the same memory are prepared once (max|x|, contraction-major copy,
codes); every probe's record must still be the one it gets when probed alone, and the oracle's."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import assert_record_close, oracle_probe

pytestmark = pytest.mark.gpu


def _same(a, b):
    ra, rb = a.record(), b.record()
    if a.device_error != b.device_error or ra["count"] != rb["count"] or ra["max_be"] != rb["max_be"]:
        return False
    return all(abs(ra[k] - rb[k]) <= 1e-12 * abs(rb[k]) for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"))


def layer_ops(M=512, H=256, F=384):
    """A small layer in the sweep's form: X feeds three products and appears transposed in their
    wgrads, every gradient appears as the left operand of a dgrad and the right one of a wgrad,
    every weight in forward (strided) and dgrad (contiguous), each in three formats."""
    t = workloads.config5_layer_tensors(3, M=M, H=H, F=F, heads=2, S=128)
    return [o for f in ("e4m3", "e5m2", "int8") for o in workloads.config5_layer(3, f, tensors=t, M=M, H=H, F=F, heads=2, S=128)]


def test_layer_batch_equals_single_probes_and_the_oracle():
    ops = layer_ops()
    on = {}

    def dev(t):
        return on.setdefault(id(t), t.cuda())
    probes = [(qm.operand_of(dev(o["L"]), o["cl"]), qm.operand_of(dev(o["R"]), o["cr"]), o["fmt_l"], o["fmt_r"],
               o["gran_l"], o["gran_r"]) for o in ops]
    batch = qm.ProbeBatch(probes)
    for _ in range(2):
        batch.launch()
        torch.cuda.synchronize()
    got = batch.results()
    for o, p, g in zip(ops, probes, got):
        assert _same(g, qm.qm_probe_layer(*p)), o["name"]
    for i in (0, 1, 2, 13, 15, 17, 20, 38, 53):               # a sample against the oracle, whole matrices
        assert_record_close(got[i].record(), oracle_probe(ops[i]), what=ops[i]["name"])


def test_same_request_twice_and_both_sides():
    """The same (tensor, format) as the left operand of one probe and the right operand of another,
    and a probe repeated verbatim: codes are made once, records are unchanged."""
    rng = workloads._rng(140)
    A = workloads.normal(rng, (256, 192)).cuda()
    B = workloads.normal(rng, (320, 192), 0.1).cuda()
    A2 = workloads.normal(rng, (256, 192), 0.1).cuda()       # same extents as A: the pair contracts over the rows
    a, b = qm.operand_of(A, -1), qm.operand_of(B, -1)
    probes = [(a, b, "e4m3", "e4m3", "tensor", "tensor"), (b, a, "e4m3", "e4m3", "tensor", "tensor"),
              (a, b, "e4m3", "e4m3", "tensor", "tensor"), (a, a, "int8", "int8", "channel", "channel"),
              (qm.operand_of(A, -2), qm.operand_of(A2, -2), "e4m3", "e4m3", "tensor", "tensor")]
    batch = qm.ProbeBatch(probes)
    batch.launch()
    torch.cuda.synchronize()
    for p, g in zip(probes, batch.results()):
        assert _same(g, qm.qm_probe_layer(*p))


def test_a_nonfinite_operand_is_reported_by_every_probe_that_uses_it():
    rng = workloads._rng(141)
    A = workloads.normal(rng, (256, 128))
    A[17, 5] = float("inf")
    A = A.cuda()
    B = workloads.normal(rng, (128, 128), 0.1).cuda()
    Cm = workloads.normal(rng, (256, 128)).cuda()
    a, b, c = qm.operand_of(A, -1), qm.operand_of(B, -1), qm.operand_of(Cm, -1)
    probes = [(a, b, "e4m3", "e4m3", "tensor", "tensor"), (a, b, "e4m3", "e4m3", "tensor", "tensor"),
              (a, b, "int8", "int8", "tensor", "tensor"), (c, b, "e4m3", "e4m3", "tensor", "tensor")]
    batch = qm.ProbeBatch(probes)
    batch.launch()
    torch.cuda.synchronize()
    flags = [r.device_error for r in batch.results()]
    assert flags[0] & 1 and flags[1] & 1 and flags[2] & 1 and flags[3] == 0


def test_host_batch_copies_every_distinct_operand_once():
    ops = layer_ops(M=256, H=128, F=256)
    pinned = {}

    def pin(t):
        return pinned.setdefault(id(t), t.pin_memory())
    hb = qm.HostProbeBatch([(pin(o["L"]), o["cl"], pin(o["R"]), o["cr"], o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
                            for o in ops])
    distinct = {}
    for o in ops:
        for t in (o["L"], o["R"]):
            distinct[id(t)] = t.numel() * t.element_size()
    assert hb.h2d_bytes == sum(distinct.values())
    got = hb.run()
    again = hb.run()
    for o, g, g2 in zip(ops, got, again):
        assert g.record() == g2.record()
    for i in (0, 7, 12, 16, 30, 50):
        assert_record_close(got[i].record(), oracle_probe(ops[i]), what=ops[i]["name"])
