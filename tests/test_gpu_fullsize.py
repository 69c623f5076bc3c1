"""GPU parity at the full sizes of the BERT-large configurations, in the launch configuration
the benchmark uses.  The oracle cannot evaluate whole products of this size, so each case is
checked three ways:
  * scales exactly, codes bit for bit on sampled rows;
  * sampled output rows of the 8-bit, reference and denominator products, one by one, against
    the oracle (exact for INT8, the stated tolerance otherwise);
  * properties that hold at any size: the fused probe's record equals the stand-alone Eq. 3
    reduction over the materialised products, and the oracle's row-sampled record equals the
    same reduction restricted to those rows.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle.probe import descale
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oriented, as3, assert_record_close

pytestmark = pytest.mark.gpu


def check_full(o, n_rows=24, seed=60):
    Ld, Rd = o["L"].cuda(), o["R"].cuda()
    Lop, Rop = qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"])
    xl, xr = as3(oriented(o["L"], o["cl"])), as3(oriented(o["R"], o["cr"]))     # [b, M, K], [b, N, K]
    B, M, K = xl.shape
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(M, min(n_rows, M), replace=False))
    bsel = np.sort(rng.choice(B, min(B, 3), replace=False))

    # ---- scales (exact) and codes (sampled rows, bit-exact)
    dl = oracle.scale(xl, o["fmt_l"], o["gran_l"]); dr = oracle.scale(xr, o["fmt_r"], o["gran_r"])
    cl, dlg, al, kl = qm.qm_quantize(Lop, o["fmt_l"], o["gran_l"], None, want_abs=True, want_kmaj=True)
    cr, drg, ar, kr = qm.qm_quantize(Rop, o["fmt_r"], o["gran_r"], None, want_abs=True, want_kmaj=True)
    assert np.array_equal(dlg.cpu().numpy(), dl.ravel()) and np.array_equal(drg.cpu().numpy(), dr.ravel())
    dl_rows = dl if dl.shape == (1,) else dl[np.ix_(bsel, rows)]
    want_cl = oracle.quantize(xl[np.ix_(bsel, rows)], o["fmt_l"], dl_rows)
    sel = (torch.as_tensor(bsel)[:, None], torch.as_tensor(rows)[None, :])
    assert np.array_equal(cl[sel].cpu().numpy()[..., :K], want_cl)
    dr_b = dr if dr.shape == (1,) else dr[bsel]
    want_cr = oracle.quantize(xr[bsel], o["fmt_r"], dr_b)
    assert np.array_equal(cr[torch.as_tensor(bsel)].cpu().numpy()[..., :K], want_cr)

    # ---- the three products, full size on the GPU, sampled rows against the oracle
    q, raw = qm.qm_gemm(cl, o["fmt_l"], dlg, o["gran_l"], cr, o["fmt_r"], drg, o["gran_r"], K, want_raw=True)
    c = qm.qm_gemm_ref(kl, kr)
    d = qm.qm_gemm_ref(al, ar)
    acc = oracle.gemm_lp(want_cl, o["fmt_l"], want_cr, o["fmt_r"])
    want_q = descale(acc, dl_rows, dr_b)
    want_c = oracle.gemm_ref(xl[np.ix_(bsel, rows)], xr[bsel])
    want_d = oracle.gemm_den(xl[np.ix_(bsel, rows)], xr[bsel])
    got_q = q[sel].cpu().numpy().astype(np.float64)
    got_c = c[sel].cpu().numpy().astype(np.float64)
    got_d = d[sel].cpu().numpy().astype(np.float64)
    if o["fmt_l"] == "int8":
        assert np.array_equal(raw[sel].cpu().numpy().astype(np.int64), acc.astype(np.int64))
    scale_q = descale(np.matmul(np.abs(oracle.dequantize(want_cl, o["fmt_l"])),
                                np.swapaxes(np.abs(oracle.dequantize(want_cr, o["fmt_r"])), -1, -2)), dl_rows, dr_b)
    assert (np.abs(got_q - want_q) / scale_q).max() <= 1e-3
    assert (np.abs(got_c - want_c) / want_d).max() <= 1e-3
    assert (np.abs(got_d - want_d) / want_d).max() <= 1e-3

    # ---- the oracle's record of the sampled rows == Eq. 3 reduction of the same GPU rows
    want_rec = oracle.metric(want_c, want_q, want_d)
    got_rec = qm.qm_metric(c[sel].contiguous(), q[sel].contiguous(), d[sel].contiguous()).record()
    assert_record_close(got_rec, want_rec, what=o["name"] + " sampled rows", K=K)

    # ---- fused probe == stand-alone reduction over the materialised products (any size)
    full = qm.qm_metric(c, q, d).record()
    res = qm.qm_probe_layer(Lop, Rop, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"])
    assert res.device_error == 0
    assert_record_close(res.record(), full, what=o["name"] + " fused vs materialised")
    return res


def pick(ops, name):
    return next(o for o in ops if o["name"] == name)


@pytest.fixture(scope="module")
def cfg3():
    return workloads.config3()


@pytest.mark.parametrize("name", ["qkv-fwd", "ffn1-dgrad", "ffn2-wgrad", "attn_out-wgrad", "ffn2-fwd"])
def test_config3_bert_large_layer(cfg3, name):
    check_full(pick(cfg3, name))


def test_config4_outlier_stress():
    ops = workloads.config4()
    res = {}
    for name in ("ffn1-int8-tensor", "ffn1-int8-channel", "ffn1-e4m3-tensor", "ffn1-e5m2-channel"):
        res[name] = check_full(pick(ops, name)).derived()["mean_be"]
    # finer granularity helps INT8 on heavy-tailed activations (the paper's observation)
    assert res["ffn1-int8-channel"] < res["ffn1-int8-tensor"]


def test_config5_attention_batched():
    ops = workloads.attention_ops(workloads._rng(61), 512, 512, 64, "e4m3")
    for name in ("qk-fwd-e4m3", "pv-fwd-e4m3", "qk-dk-e4m3", "pv-dv-e4m3"):
        check_full(pick(ops, name), n_rows=16)
    ops = workloads.attention_ops(workloads._rng(62), 512, 512, 64, "int8")
    check_full(pick(ops, "qk-dq-int8"), n_rows=16)


def test_config2_whole_records_through_the_batch_entry_point():
    """The benchmark's workload in the benchmark's launch configuration (one qm_probe_batch call for
    the step's eight probes): every whole-matrix record against the oracle's full probe."""
    ops = workloads.config2()
    dev = [(o["L"].cuda(), o["R"].cuda()) for o in ops]
    batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                            o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev)])
    for _ in range(2):
        batch.launch()
    torch.cuda.synchronize()
    for o, got in zip(ops, batch.results()):
        assert got.device_error == 0
        L, R = workloads.orient(o)
        want = oracle.probe(L, R, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
        assert_record_close(got.record(), want, what=o["name"], K=L.shape[-1])
