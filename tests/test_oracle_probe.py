"""Pins for the oracle's GEMMs and the backward-error metric (Eq. 3)."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import positive_grid, qmax

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FMTS = ["int8", "e4m3", "e5m2"]


def frac_table(fmt):
    t = oracle.decode_table(fmt)
    return [Fraction(float(v)) if np.isfinite(v) else None for v in t]


@pytest.mark.parametrize("fl,fr", [("int8", "int8"), ("e4m3", "e4m3"), ("e5m2", "e4m3"), ("e5m2", "e5m2")])
def test_gemm_lp_brute_force_exact(fl, fr):
    # triple loop in exact rational arithmetic on tiny shapes
    rng = np.random.default_rng(10)
    M, N, K = 3, 4, 7
    tl, tr = frac_table(fl), frac_table(fr)
    okl = [c for c in range(256) if tl[c] is not None and not (fl == "int8" and c == 128)]
    okr = [c for c in range(256) if tr[c] is not None and not (fr == "int8" and c == 128)]
    cl = rng.choice(okl, (M, K)).astype(np.uint8)
    cr = rng.choice(okr, (N, K)).astype(np.uint8)
    got = oracle.gemm_lp(cl, fl, cr, fr)
    for i in range(M):
        for j in range(N):
            s = Fraction(0)
            for k in range(K):
                s += tl[cl[i, k]] * tr[cr[j, k]]
            assert abs(Fraction(float(got[i, j])) - s) <= abs(s) * Fraction(1, 2 ** 50)
            if fl != "e5m2" and fr != "e5m2":
                assert Fraction(float(got[i, j])) == s


def test_ref_and_den_brute_force():
    rng = np.random.default_rng(11)
    B, M, N, K = 2, 3, 5, 6
    l = rng.integers(-9, 10, (B, M, K)).astype(np.float32)      # small integers: sums exact
    r = rng.integers(-9, 10, (B, K, N)).astype(np.float32)
    rt = np.swapaxes(r, -1, -2)
    c = oracle.gemm_ref(l, rt); d = oracle.gemm_den(l, rt)
    for b in range(B):
        for i in range(M):
            for j in range(N):
                sc = sd = 0
                for k in range(K):
                    sc += int(l[b, i, k]) * int(r[b, k, j])
                    sd += abs(int(l[b, i, k])) * abs(int(r[b, k, j]))
                assert c[b, i, j] == sc and d[b, i, j] == sd
    assert np.all(d >= np.abs(c))


def test_hand_computed_2x2x2():
    be = codes_l = codes_r = None
    lit = {}
    for line in open(os.path.join(GOLDEN, "hand_2x2x2.txt")):
        if line.startswith("be "):
            be = [Fraction(t) for t in line.split()[1:]]
        elif line.startswith("codes_l "):
            codes_l = [int(t) for t in line.split()[1:]]
        elif line.startswith("codes_r_kxn "):
            codes_r = [int(t) for t in line.split()[1:]]
        elif not line.startswith("#") and len(line.split()) == 2:
            lit[line.split()[0]] = float(line.split()[1])
    L = np.array([[127, -63.5], [0.5, 2.5]], np.float32)
    R = np.array([[1.5, 127], [-3.5, 10.25]], np.float32)
    rec, full = oracle.probe(L, R, "int8", "int8", "tensor", "tensor", full=True)
    assert full["delta_l"][0] == 1.0 and full["delta_r"][0] == 1.0
    assert oracle.dequantize(full["codes_l"], "int8").ravel().tolist() == codes_l
    assert oracle.dequantize(full["codes_r"], "int8").T.ravel().tolist() == codes_r
    assert full["c"].ravel().tolist() == [412.75, 15478.125, -8.0, 89.125]
    assert full["q"].ravel().tolist() == [510, 15489, -8, 20]
    assert full["d"].ravel().tolist() == [412.75, 16779.875, 9.5, 89.125]
    assert rec["count"] == 4
    assert abs(rec["sum_be"] - float(sum(be))) < 1e-15
    assert abs(rec["max_be"] - float(max(be))) < 1e-15
    assert abs(rec["sum_diff2"] - (97.25 ** 2 + 10.875 ** 2 + 69.125 ** 2)) < 1e-9
    assert rec["sum_ref2"] == 412.75 ** 2 + 15478.125 ** 2 + 64 + 89.125 ** 2
    assert rec["sum_den2"] == 412.75 ** 2 + 16779.875 ** 2 + 9.5 ** 2 + 89.125 ** 2
    # the record's sums and every derived scalar against the stored hand-worked literals
    for k in ("sum_diff2", "sum_ref2", "sum_den2"):
        assert abs(rec[k] - lit[k]) <= 1e-15 * lit[k], k
    dv = oracle.derived(rec)
    assert set(dv) == {"mean_be", "max_be", "normwise_be", "rel_l2", "snr_db"}
    for k in dv:
        assert abs(dv[k] - lit[k]) <= 1e-14 * abs(lit[k]), (k, dv[k], lit[k])
    # degenerate records: an exact product has infinite SNR and zero errors, an empty one is all zero
    exact = oracle.derived({"sum_be": 0.0, "max_be": 0.0, "sum_diff2": 0.0, "sum_ref2": 5.0, "sum_den2": 7.0, "count": 3})
    assert exact["snr_db"] == float("inf") and exact["rel_l2"] == 0 and exact["normwise_be"] == 0 and exact["mean_be"] == 0
    empty = oracle.derived({"sum_be": 0.0, "max_be": 0.0, "sum_diff2": 0.0, "sum_ref2": 0.0, "sum_den2": 0.0, "count": 0})
    assert empty["mean_be"] == 0 and empty["rel_l2"] == 0 and empty["normwise_be"] == 0


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("gran", ["tensor", "channel"])
def test_on_grid_inputs_have_zero_error(fmt, gran):
    # inputs exactly representable after scaling  =>  Q == C and BE == 0 everywhere
    rng = np.random.default_rng(12)
    g = positive_grid(fmt)
    vals = np.concatenate([g, -g])
    M, K, N = 8, 32, 6
    L = rng.choice(vals, (M, K)); R = rng.choice(vals, (K, N))
    L[:, 0] = qmax(fmt); R[0, :] = -qmax(fmt)            # every group has absmax = qmax
    L = (L * 2.0 ** -3).astype(np.float32); R = (R * 2.0 ** 2).astype(np.float32)
    rec, full = oracle.probe(L, R, fmt, fmt, gran, gran, full=True)
    assert np.all(full["delta_l"] == np.float32(2.0 ** -3)) and np.all(full["delta_r"] == np.float32(4.0))
    if fmt == "e5m2":      # products span more than 53 bits: the two fp64 sums may round differently
        assert rec["max_be"] < 2.0 ** -45
    else:
        assert rec["sum_be"] == 0 and rec["max_be"] == 0 and rec["sum_diff2"] == 0
    assert rec["sum_ref2"] > 0 and rec["count"] == M * N


def test_descale_uses_row_and_column_scales():
    # per-channel: row i of L scaled by 2^i and column j of R by 2^-j must leave BE unchanged
    rng = np.random.default_rng(13)
    L = rng.standard_normal((4, 64)).astype(np.float32); R = rng.standard_normal((64, 5)).astype(np.float32)
    rec0, f0 = oracle.probe(L, R, "e4m3", "int8", "channel", "channel", full=True)
    Ls = (L * (2.0 ** np.arange(4))[:, None]).astype(np.float32)
    Rs = (R * (2.0 ** -np.arange(5))[None, :]).astype(np.float32)
    rec1, f1 = oracle.probe(Ls, Rs, "e4m3", "int8", "channel", "channel", full=True)
    assert np.array_equal(f0["codes_l"], f1["codes_l"]) and np.array_equal(f0["codes_r"], f1["codes_r"])
    be0 = np.abs(f0["c"] - f0["q"]) / f0["d"]; be1 = np.abs(f1["c"] - f1["q"]) / f1["d"]
    assert np.allclose(be0, be1, rtol=1e-12, atol=0)
    assert abs(rec0["sum_be"] - rec1["sum_be"]) < 1e-12 * rec0["sum_be"]
    # q really is acc * dl_i * dr_j
    i, j = 2, 3
    assert f1["q"][i, j] == f1["acc"][i, j] * float(f1["delta_l"][i]) * float(f1["delta_r"][j])


def test_metric_invariants():
    rng = np.random.default_rng(14)
    c = rng.standard_normal((5, 7)); d = np.abs(c) + rng.uniform(0, 1, c.shape)
    rec = oracle.metric(c, c, d)
    assert rec["sum_be"] == 0 and rec["max_be"] == 0 and rec["sum_diff2"] == 0
    q = c + 0.5 * d                                  # BE = 0.5 everywhere
    rec = oracle.metric(c, q, d)
    assert abs(rec["sum_be"] - 0.5 * 35) < 1e-12 and abs(rec["max_be"] - 0.5) < 1e-15
    d0 = d.copy(); d0[0, 0] = 0                       # D == 0 contributes BE 0 but still counts
    rec0 = oracle.metric(c, q, d0)
    assert rec0["count"] == 35 and abs(rec0["sum_be"] - 0.5 * 34) < 1e-12
    assert oracle.derived(oracle.metric(c, c, d))["snr_db"] == float("inf")


def test_row_sampled_mode_matches_full():
    rng = np.random.default_rng(15)
    L = rng.standard_t(3, (40, 96)).astype(np.float32); R = rng.standard_normal((96, 24)).astype(np.float32)
    rows = np.array([0, 7, 39])
    for gran in ("tensor", "channel"):
        _, full = oracle.probe(L, R, "int8", "e5m2", gran, "channel", full=True)
        rec = oracle.probe(L, R, "int8", "e5m2", gran, "channel", rows=rows)
        want = oracle.metric(full["c"][rows], full["q"][rows], full["d"][rows])
        assert rec == want


def test_batched_probe_equals_per_batch():
    rng = np.random.default_rng(16)
    L = rng.standard_normal((3, 8, 32)).astype(np.float32); R = rng.standard_normal((3, 32, 8)).astype(np.float32)
    rec, full = oracle.probe(L, R, "e4m3", "e4m3", "channel", "channel", full=True)
    s = 0.0
    for b in range(3):
        s += oracle.probe(L[b], R[b], "e4m3", "e4m3", "channel", "channel")["sum_be"]
    assert abs(s - rec["sum_be"]) < 1e-12
    # per-tensor over a batched operand is ONE delta for the whole batched tensor
    assert oracle.scale(L, "e4m3", "tensor").shape == (1,)


def test_paper_qualitative_claims_on_student_t():
    # "Quantized matrix multiplication: an illustrative example": 512x512 Student-t, per-vector
    # scaling; INT8 error grows with heavy-tailedness, FP8 is much more constrained, E4M3 < E5M2.
    rng = np.random.default_rng(17)
    mean_be = {}
    for nu in (1.5, 3.0, 30.0):
        L = rng.standard_t(nu, (512, 512)).astype(np.float32)
        R = rng.standard_t(nu, (512, 512)).astype(np.float32)
        for fmt in FMTS:
            mean_be[(fmt, nu)] = oracle.derived(oracle.probe(L, R, fmt, fmt, "channel", "channel"))["mean_be"]
    for nu in (1.5, 3.0, 30.0):
        assert mean_be[("e4m3", nu)] < mean_be[("e5m2", nu)]
        assert 1.5 < mean_be[("e5m2", nu)] / mean_be[("e4m3", nu)] < 2.5
    int8_spread = mean_be[("int8", 1.5)] / mean_be[("int8", 30.0)]
    e4m3_spread = mean_be[("e4m3", 1.5)] / mean_be[("e4m3", 30.0)]
    assert int8_spread > 5 and e4m3_spread < 4 and int8_spread > 4 * e4m3_spread
    # light tails: INT8 is at least as precise as FP8
    assert mean_be[("int8", 30.0)] < mean_be[("e4m3", 30.0)]


def test_finer_granularity_helps_int8_on_heavy_tails_and_k_scaling():
    rng = np.random.default_rng(18)
    L = rng.standard_t(2.0, (256, 512)).astype(np.float32); R = (rng.standard_normal((512, 128)) * 0.02).astype(np.float32)
    t = oracle.derived(oracle.probe(L, R, "int8", "int8", "tensor", "tensor"))["mean_be"]
    c = oracle.derived(oracle.probe(L, R, "int8", "int8", "channel", "channel"))["mean_be"]
    assert c < t
    # i.i.d. inputs: mean BE falls roughly like 1/sqrt(K)
    be = []
    for K in (256, 1024):
        L = rng.standard_normal((128, K)).astype(np.float32); R = rng.standard_normal((K, 128)).astype(np.float32)
        be.append(oracle.derived(oracle.probe(L, R, "e4m3", "e4m3", "tensor", "tensor"))["mean_be"])
    assert 1.6 < be[0] / be[1] < 2.4
