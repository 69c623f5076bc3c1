"""GPU parity of the fused kernel's tile walk and column split: output widths on both sides of
every boundary the epilogue distinguishes (a warp's share of a tile is 32 or 64 columns, read in
chunks of 16, ragged at the edge of the matrix), outputs wider than tall (tiles walked down the
rows first), several batch elements, scales per tensor and per channel.  Every probe is checked
twice: its record against the oracle's, and every output row's Eq. 3 sums (the kernel's check
output) against the oracle's sums of that row."""
import numpy as np
import pytest
import torch

import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads
from helpers import oracle_probe, oracle_row_stats, assert_record_close

pytestmark = pytest.mark.gpu


def run_with_rows(ops):
    dev = [(o["L"].cuda(), o["R"].cuda()) for o in ops]
    batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                            o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev)], row_stats=True)
    batch.launch()
    torch.cuda.synchronize()
    return batch


def check(o, res, rows_out):
    (M, N, K, B), _ = workloads.op_flops(o)
    assert res.device_error == 0, o["name"]
    rec = res.record()
    assert_record_close(rec, oracle_probe(o), what=o["name"])
    rs = rows_out.cpu().numpy().reshape(B, M, 5)
    # the record is the sum (max) of the per-row output, and no row was skipped or written twice
    for k, name in ((0, "sum_be"), (2, "sum_diff2"), (3, "sum_ref2"), (4, "sum_den2")):
        assert abs(rs[..., k].sum() - rec[name]) <= 1e-9 * abs(rec[name]) + 1e-300, (o["name"], name)
    assert rs[..., 1].max() == rec["max_be"], o["name"]
    want = oracle_row_stats(o, np.arange(M))                           # every row of every batch element
    got = rs.reshape(-1, 5); want = want.reshape(-1, 5)
    # sums of squares of one row carry no cancellation: 1e-3; a row's BE terms are each off by up to
    # a few 1e-3 relative (fp32 products against an error of 1e-3 D) and a short row averages little
    for k in (3, 4):
        assert (np.abs(got[:, k] - want[:, k]) <= 1e-3 * want[:, k] + 1e-300).all(), (o["name"], k)
    for k in (0, 2):
        assert (np.abs(got[:, k] - want[:, k]) <= 2e-2 * want[:, k] + 1e-300).all(), (o["name"], k)
    assert (np.abs(got[:, 1] - want[:, 1]) <= 2e-2 * want[:, 1] + 1e-300).all(), (o["name"], "max_be")


WIDTHS = [8, 16, 17, 32, 33, 48, 49, 64, 65, 80, 81, 96, 112, 113, 128, 129, 200]


@pytest.mark.parametrize("fmt,gran", [("e4m3", "tensor"), ("int8", "channel")])
def test_every_width_class(fmt, gran):
    """One batch of probes, one per width: the narrow path (N <= 64: MMAs of N = 64, 32 columns per
    epilogue warp) and the wide path, every count of live 16-column chunks, ragged and whole."""
    rng = workloads._rng(90)
    ops = []
    for N in WIDTHS:
        L = workloads.student_t(rng, (2, 300, 144), 5.0)               # two batch elements, two row tiles, ragged K
        R = workloads.normal(rng, (2, N, 144), 0.05)
        ops.append(workloads.op(f"w{N}", L, -1, R, -1, fmt, fmt, gran, gran))
    batch = run_with_rows(ops)
    for i, (o, res) in enumerate(zip(ops, batch.results())):
        check(o, res, batch.row_stats[i])


@pytest.mark.parametrize("fmt,gran", [("e5m2", "channel"), ("int8", "tensor")])
def test_outputs_wider_than_tall_walk_down_the_rows(fmt, gran):
    """M < N: the tiles of a batch element are dealt row tile fastest.  Three row tiles by five
    column tiles (both ragged), three batch elements, beside a tall probe and a square one in the
    same launch, so that the pairs change probe and walk order in mid-launch."""
    rng = workloads._rng(91)
    shapes = [(3, 600, 620, 208), (1, 1100, 300, 272), (2, 384, 384, 80), (1, 130, 1000, 512)]
    ops = []
    for b, M, N, K in shapes:
        L = workloads.normal(rng, (b, M, K))
        R = workloads.normal(rng, (b, N, K), 0.02)
        ops.append(workloads.op(f"s{M}x{N}x{K}", L, -1, R, -1, fmt, fmt, gran, gran))
    batch = run_with_rows(ops)
    for i, (o, res) in enumerate(zip(ops, batch.results())):
        check(o, res, batch.row_stats[i])
    # each probe alone gives the same record: the walk order is per probe, not per launch
    for o, res in zip(ops, batch.results()):
        alone = qm.qm_probe_layer(qm.operand_of(o["L"].cuda(), o["cl"]), qm.operand_of(o["R"].cuda(), o["cr"]),
                                  o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"]).record()
        got = res.record()
        assert got["count"] == alone["count"] and got["max_be"] == alone["max_be"]
        for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"):
            assert abs(got[k] - alone[k]) <= 1e-12 * abs(alone[k]), (o["name"], k)
