"""The give-up path of the fused probe kernel: a barrier wait that nothing will ever satisfy runs
into its time limit, the kernel reports QM_DEVERR_TIMEOUT and returns, and the next probe on
the same GPU is right.  The wait is starved on purpose and safely: the loading warp simply stops
issuing loads (a hook of the library), so nothing is in flight that is never awaited; no trap, no
bad address, no unbounded loop."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import binding, workloads

pytestmark = pytest.mark.gpu

QM_DEVERR_TIMEOUT = 2
QM_ERR_TIMEOUT = 7


@pytest.fixture
def starved_producer():
    L = qm.lib()
    L.qm_debug_set_wait_limit_ns(2_000_000)          # 2 ms instead of 1 s
    yield L
    L.qm_debug_stop_producer_after(0xffffffff)
    L.qm_debug_set_wait_limit_ns(0)


def small_op(seed=31, M=256, N=128, K=256):
    rng = workloads._rng(seed)
    return workloads.op("giveup", workloads.normal(rng, (M, K)), -1, workloads.normal(rng, (K, N), 0.02), -2,
                        "e4m3", "e4m3")


def probe(o):
    Ld, Rd = o["L"].cuda(), o["R"].cuda()
    return qm.qm_probe_layer(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                             o["gran_l"], o["gran_r"])


def check_against_oracle(o, res):
    L, R = workloads.orient(o)
    want = oracle.probe(L, R, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
    got = res.record()
    assert res.device_error == 0 and got["count"] == want["count"]
    for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(got[k] - want[k]) <= 1e-4 * abs(want[k]), (k, got[k], want[k])


@pytest.mark.parametrize("stop_after", [0, 2])
def test_wait_runs_out_and_the_kernel_returns(starved_producer, stop_after):
    o = small_op()                                    # one tile of four k-blocks
    starved_producer.qm_debug_stop_producer_after(stop_after)
    res = probe(o)
    torch.cuda.synchronize()                          # the context is alive: no sticky error
    assert res.device_error & QM_DEVERR_TIMEOUT
    # the hook off again: the same probe is right, on the same GPU, in the same process
    starved_producer.qm_debug_stop_producer_after(0xffffffff)
    check_against_oracle(o, probe(o))


def test_host_entry_point_maps_the_flag_to_its_status(starved_producer):
    o = small_op(seed=32)
    Lh, Rh = o["L"].pin_memory(), o["R"].pin_memory()
    starved_producer.qm_debug_stop_producer_after(1)
    with pytest.raises(qm.QmError) as e:
        qm.qm_probe_layer_host(Lh, Rh, o["cl"], o["cr"], o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
    assert e.value.status == QM_ERR_TIMEOUT
    starved_producer.qm_debug_stop_producer_after(0xffffffff)
    res, _ = qm.qm_probe_layer_host(Lh, Rh, o["cl"], o["cr"], o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
    check_against_oracle(o, res)


def test_a_batch_reports_the_timeout_in_every_record(starved_producer):
    ops = [small_op(seed=33), small_op(seed=34, M=512, N=256, K=128)]
    dev = [(o["L"].cuda(), o["R"].cuda()) for o in ops]
    batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                            o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev)])
    starved_producer.qm_debug_stop_producer_after(1)
    batch.launch()
    torch.cuda.synchronize()
    assert all(r.device_error & QM_DEVERR_TIMEOUT for r in batch.results())
    starved_producer.qm_debug_stop_producer_after(0xffffffff)
    batch.launch()
    torch.cuda.synchronize()
    for o, r in zip(ops, batch.results()):
        check_against_oracle(o, r)
