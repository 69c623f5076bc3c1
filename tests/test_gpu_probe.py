"""GPU parity: the fused probe against the oracle (Eq. 1 + Eq. 3 end to end)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oracle_probe, gpu_probe, assert_record_close

pytestmark = pytest.mark.gpu


def test_config1_fp32_reference():
    o = workloads.config1()[0]
    res = gpu_probe(o)
    assert res.device_error == 0
    assert_record_close(res.record(), oracle_probe(o), what="config1")


@pytest.mark.parametrize("fmt", ["int8", "e4m3", "e5m2"])
@pytest.mark.parametrize("gran", ["tensor", "channel"])
@pytest.mark.parametrize("ref", ["bf16", "fp32"])
@pytest.mark.parametrize("layout", [(-1, -2), (-1, -1), (-2, -2)])
def test_probe_small_ragged(fmt, gran, ref, layout):
    # M, N not multiples of the tile, K several k-blocks with a ragged last one
    rng = workloads._rng(30)
    M, N, K = 200, 136, 176
    L = workloads.student_t(rng, (M, K) if layout[0] == -1 else (K, M), 4.0)
    R = workloads.normal(rng, (K, N) if layout[1] == -2 else (N, K), 0.05)
    o = workloads.op("small", L, layout[0], R, layout[1], fmt, fmt, gran, gran, ref)
    res = gpu_probe(o)
    assert res.device_error == 0
    assert_record_close(res.record(), oracle_probe(o), what=str((fmt, gran, ref, layout)))


@pytest.mark.parametrize("fmts", [("e5m2", "e4m3"), ("e4m3", "e5m2")])
def test_probe_mixed_fp8_formats(fmts):
    rng = workloads._rng(31)
    L = workloads.normal(rng, (384, 512), 1e-3)
    R = workloads.normal(rng, (512, 256), 0.02)
    o = workloads.op("mixed", L, -1, R, -2, fmts[0], fmts[1], "tensor", "channel")
    res = gpu_probe(o)
    assert_record_close(res.record(), oracle_probe(o), what=str(fmts))


@pytest.mark.parametrize("fmt", ["int8", "e4m3"])
def test_probe_batched_attention_shapes(fmt):
    rng = workloads._rng(32)
    ops = workloads.attention_ops(rng, 6, 128, 64, fmt)
    for o in ops:
        res = gpu_probe(o)
        assert res.device_error == 0
        assert_record_close(res.record(), oracle_probe(o), what=o["name"])


@pytest.mark.parametrize("fmt", ["int8", "e4m3", "e5m2"])
def test_probe_on_grid_inputs_have_zero_error(fmt):
    g = oracle.positive_grid(fmt)
    g = g[(g >= 2.0 ** -3) & (g <= 16)] if fmt != "int8" else g[g <= 16]   # moderate dynamic range
    rng = np.random.default_rng(33)
    vals = np.concatenate([g, -g, [0.0]])
    M, K, N = 256, 128, 128
    Lv = rng.choice(vals, (M, K)); Rv = rng.choice(vals, (K, N))
    top = oracle.qmax(fmt)
    # every group holds +-qmax, so delta is the power of two the tensors are scaled by
    Lv[:, 0] = top; Rv[0, :] = -top
    L = torch.from_numpy((Lv * 2.0 ** -9).astype(np.float32)).to(torch.bfloat16)
    R = torch.from_numpy((Rv * 2.0 ** -9).astype(np.float32)).to(torch.bfloat16)
    assert np.array_equal(L.float().numpy().astype(np.float64), Lv * 2.0 ** -9)
    o = workloads.op("grid", L, -1, R, -2, fmt, fmt, "channel", "channel")
    want = oracle_probe(o)
    assert want["max_be"] < 1e-12
    res = gpu_probe(o)
    assert res.max_be <= 2e-6 and res.sum_diff2 <= 1e-10 * res.sum_ref2
    assert abs(res.sum_ref2 - want["sum_ref2"]) <= 1e-5 * want["sum_ref2"]


def test_probe_student_t_example_all_formats():
    for nu in (1.5, 3.0, 30.0):
        for fmt in ("int8", "e4m3", "e5m2"):
            o = workloads.student_t_example(nu, fmt=fmt)[0]
            res = gpu_probe(o)
            assert_record_close(res.record(), oracle_probe(o), what=o["name"])


def test_probe_is_deterministic():
    o = workloads.config2(M=512, H=256, F=512)[0]
    a, b = gpu_probe(o).record(), gpu_probe(o).record()
    assert a == b


def test_probe_flags_nonfinite_input():
    o = workloads.config2(M=256, H=128, F=256)[0]
    o["L"] = o["L"].clone(); o["L"][5, 7] = float("nan")
    assert gpu_probe(o).device_error & 1


def test_probe_host_entry_point_matches_device_entry_point():
    o = workloads.config2(M=512, H=256, F=512)[2]
    Lh, Rh = o["L"].pin_memory(), o["R"].pin_memory()
    res, stage = qm.qm_probe_layer_host(Lh, Rh, o["cl"], o["cr"], o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"])
    res2, _ = qm.qm_probe_layer_host(Lh, Rh, o["cl"], o["cr"], o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], stage=stage)
    assert res.record() == gpu_probe(o).record() == res2.record()


def test_config2_shapes_row_sampled():
    # full-size BERT-base forward operands; oracle on a seeded subset of output rows
    ops = workloads.config2()
    rows = np.random.default_rng(34).choice(4096, 48, replace=False)
    for o in ops:
        Ld, Rd = o["L"].cuda(), o["R"].cuda()
        res = qm.qm_probe_layer(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                                o["gran_l"], o["gran_r"], o["ref"])
        assert res.device_error == 0
        Ls = o["L"][rows].contiguous()
        # per-tensor scales over the whole operands; the sampled rows' statistics must match a
        # GPU probe of exactly those rows when the scale-setting element is kept
        want = oracle_probe(o, rows=rows)
        full = res.record()
        # sampled mean BE estimates the full mean BE (i.i.d. rows): loose statistical check
        assert abs(want["sum_be"] / want["count"] - full["sum_be"] / full["count"]) <= 0.05 * full["sum_be"] / full["count"]
        assert full["count"] == 4096 * o["R"].shape[1]
