"""GPU parity of per-channel scales shared along the matmul batch: the 'channel' and
'fine-grained' granularity levels of the Results section (batch laid out [examples][heads])."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oriented, assert_record_close

pytestmark = pytest.mark.gpu
E, H = 3, 4            # examples x heads


def batched(seed, shape, spread=True):
    rng = workloads._rng(seed)
    t = workloads.normal(rng, shape)
    if spread:         # a different magnitude per batch element, so that sharing changes the scales
        t = t * torch.from_numpy((10.0 ** rng.uniform(-2, 1, (shape[0], 1, 1))).astype(np.float32)).to(t.dtype)
    return t


@pytest.mark.parametrize("fmt", ["int8", "e4m3", "e5m2"])
@pytest.mark.parametrize("groups", [1, H, E * H])
@pytest.mark.parametrize("contract", [-1, -2])
def test_shared_scales_and_codes(fmt, groups, contract):
    t = batched(51, (E * H, 72, 40))
    op = qm.operand_of(t.cuda(), contract)
    x = oriented(t, contract)
    want = oracle.scale(x, fmt, "channel", batch_groups=groups)
    d = qm.qm_scale_shared(op, fmt, groups)
    assert np.array_equal(d.cpu().numpy().view(np.uint32), want.ravel().view(np.uint32))
    if groups == E * H:
        assert torch.equal(d, qm.qm_scale(op, fmt, "channel"))
    codes, *_ = qm.qm_quantize(op, fmt, "channel", d)
    K = x.shape[-1]
    assert np.array_equal(codes.cpu().numpy()[..., :K], oracle.quantize(x, fmt, want))


def test_shared_scale_argument_checks():
    op = qm.operand_of(batched(52, (6, 16, 32)).cuda(), -1)
    with pytest.raises(qm.QmError):
        qm.qm_scale_shared(op, "int8", 4)            # does not divide the batch
    with pytest.raises(qm.QmError):
        qm.qm_scale_shared(op, "int8", 0)
    with pytest.raises(qm.QmError):
        qm.qm_probe_layer(op, op, "int8", "int8", "channel", "channel", groups=(4, 0))


@pytest.mark.parametrize("fmt", ["int8", "e4m3"])
@pytest.mark.parametrize("groups", [(1, 1), (H, H), (H, 0), (0, 1)])
@pytest.mark.parametrize("ref", ["bf16", "fp32"])
def test_attention_probe_with_shared_scales(fmt, groups, ref):
    # scores = Q . K^T per (example, head): L = Q [b, S, D], R = K stored [b, S, D] (contract -1)
    Q = batched(53, (E * H, 136, 64))
    Kt = batched(54, (E * H, 200, 64))
    res = qm.qm_probe_layer(qm.operand_of(Q.cuda(), -1), qm.operand_of(Kt.cuda(), -1), fmt, fmt, "channel", "channel",
                            ref, groups=groups)
    assert res.device_error == 0
    want = oracle.probe(Q.float().numpy(), np.swapaxes(Kt.float().numpy(), -1, -2), fmt, fmt, "channel", "channel",
                        groups_l=groups[0] or None, groups_r=groups[1] or None)
    assert_record_close(res.record(), want, what=f"{fmt} {groups} {ref}")
    own = qm.qm_probe_layer(qm.operand_of(Q.cuda(), -1), qm.operand_of(Kt.cuda(), -1), fmt, fmt, "channel", "channel", ref)
    assert own.sum_be != res.sum_be                  # sharing really changed the scales


def test_int8_error_grows_as_scales_are_shared_more_widely():
    Q = batched(55, (E * H, 128, 64))
    Kt = batched(56, (E * H, 128, 64))
    be = []
    for g in (0, H, 1):                               # own scales, fine-grained, channel
        r = qm.qm_probe_layer(qm.operand_of(Q.cuda(), -1), qm.operand_of(Kt.cuda(), -1), "int8", "int8", "channel",
                              "channel", groups=(g, g))
        be.append(r.derived()["mean_be"])
    t = qm.qm_probe_layer(qm.operand_of(Q.cuda(), -1), qm.operand_of(Kt.cuda(), -1), "int8", "int8", "tensor", "tensor")
    assert be[0] < be[1] < be[2] < t.derived()["mean_be"]
