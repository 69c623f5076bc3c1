"""Shared by the GPU parity tests: moves seeded inputs to the device and runs the oracle on
the same arrays."""
import numpy as np
import torch

import oracle
import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads


def oriented(t, contract_dim):
    """float32 numpy array [.., nc, c] of a tensor whose contracting dim is contract_dim."""
    x = t.float().cpu().numpy()
    return np.swapaxes(x, -1, -2) if contract_dim == -2 else x


def as3(a):
    return a[None] if a.ndim == 2 else a


def oracle_probe(o, rows=None, full=False):
    L, R = workloads.orient(o)
    return oracle.probe(L, R, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], rows=rows, full=full)


def gpu_probe(o):
    Ld, Rd = o["L"].cuda(), o["R"].cuda()
    res = qm.qm_probe_layer(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                            o["gran_l"], o["gran_r"], o["ref"])
    return res


def _derived(rec):
    d = oracle.derived(rec)
    return {k: d[k] for k in ("mean_be", "normwise_be", "rel_l2")}


def assert_record_close(got, want, rtol=1e-4, rtol_max=1e-3, what="", K=None):
    """Scalar-metric tolerance.  The metrics (mean BE, norm-wise BE, relative L2) must agree within
    rtol = 1e-4 and max BE within 1e-3, at every size.  The raw sums behind them get the same 1e-4
    up to K = 8192; beyond that the bound grows in proportion to K, because the tensor cores
    truncate when they add each 16-deep partial product to the fp32 accumulator: the all-positive
    denominator loses about 6e-8 per step relative, so its sum of squares is low by about
    1.6e-4 at K = 16384 (1024 steps) while the ratios that form the metrics stay inside 1e-4."""
    assert got["count"] == want["count"], what
    raw_tol = rtol if (K is None or K <= 8192) else rtol * K / 8192.0
    for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(got[k] - want[k]) <= raw_tol * abs(want[k]) + 1e-300, (what, k, got[k], want[k])
    dg, dw = _derived(got), _derived(want)
    for k in dg:
        assert abs(dg[k] - dw[k]) <= rtol * abs(dw[k]) + 1e-300, (what, k, dg[k], dw[k])
    assert abs(got["max_be"] - want["max_be"]) <= rtol_max * abs(want["max_be"]) + 1e-300, (what, got, want)
