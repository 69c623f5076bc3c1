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


def assert_record_close(got, want, rtol=1e-4, rtol_max=1e-3, what=""):
    """Scalar-metric tolerance: sums within rtol relative, max BE within rtol_max."""
    assert got["count"] == want["count"], what
    for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(got[k] - want[k]) <= rtol * abs(want[k]) + 1e-300, (what, k, got[k], want[k])
    assert abs(got["max_be"] - want["max_be"]) <= rtol_max * abs(want["max_be"]) + 1e-300, (what, got, want)
