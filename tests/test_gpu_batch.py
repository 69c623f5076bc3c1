"""qm_probe_batch / qm_probe_batch_host: the probes of a measurement pass issued together give
the records of the same probes issued one by one."""
import ctypes as C

import pytest
import torch

import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import workloads

pytestmark = pytest.mark.gpu


def _ops():
    shapes = [(300, 200, 128, "e4m3", "tensor", "tensor"), (256, 128, 64, "int8", "channel", "tensor"),
              (130, 264, 256, "e5m2", "tensor", "channel"), (512, 384, 192, "e4m3", "channel", "channel"),
              (64, 64, 1024, "int8", "tensor", "tensor")]
    out = []
    for i, (M, N, K, fmt, gl, gr) in enumerate(shapes):
        rng = workloads._rng(100 + i)
        out.append((workloads.normal(rng, (M, K)), workloads.normal(rng, (K, N), 0.05), fmt, gl, gr))
    return out


def _same(a, b):
    """Equal records.  A batch sums the same per-row statistics in fp64, but over the tiles of a
    different CTA-to-tile assignment, so the sums may differ in the last bits."""
    ra, rb = a.record(), b.record()
    if a.device_error != b.device_error or ra["count"] != rb["count"] or ra["max_be"] != rb["max_be"]:
        return False
    return all(abs(ra[k] - rb[k]) <= 1e-12 * abs(rb[k]) for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2"))


def test_batch_equals_single_probes():
    ops = _ops()
    dev = [(L.cuda(), R.cuda()) for L, R, *_ in ops]
    single = [qm.qm_probe_layer(qm.operand_of(Ld, -1), qm.operand_of(Rd, -2), f, f, gl, gr)
              for (Ld, Rd), (_, _, f, gl, gr) in zip(dev, ops)]
    batch = qm.ProbeBatch([(qm.operand_of(Ld, -1), qm.operand_of(Rd, -2), f, f, gl, gr)
                           for (Ld, Rd), (_, _, f, gl, gr) in zip(dev, ops)])
    for _ in range(3):                      # workspaces are reused without clearing by the caller
        batch.launch()
        torch.cuda.synchronize()
        assert all(_same(g, s) for g, s in zip(batch.results(), single))
    batch.launch_serial()
    torch.cuda.synchronize()
    assert all(_same(g, s) for g, s in zip(batch.results(), single))


def test_batch_orders_after_and_before_the_callers_stream():
    L0, R0, f, gl, gr = _ops()[0]
    Ld, Rd = torch.zeros_like(L0, device="cuda"), R0.cuda()
    want = qm.qm_probe_layer(qm.operand_of(L0.cuda(), -1), qm.operand_of(Rd, -2), f, f, gl, gr)
    batch = qm.ProbeBatch([(qm.operand_of(Ld, -1), qm.operand_of(Rd, -2), f, f, gl, gr)] * 4)
    s = torch.cuda.Stream()
    src = L0.cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        Ld.copy_(src)                       # the batch must see this write ...
        batch.launch(stream=s)
        snapshot = batch.out.clone()        # ... and this read must see the batch's records
    s.synchronize()
    sz = C.sizeof(qm.MetricResult)
    raw = snapshot.cpu().numpy().tobytes()
    for i in range(4):
        assert _same(qm.MetricResult.from_buffer_copy(raw[i * sz:(i + 1) * sz]), want)


def test_host_batch_equals_single_probes():
    ops = _ops()
    single = [qm.qm_probe_layer(qm.operand_of(L.cuda(), -1), qm.operand_of(R.cuda(), -2), f, f, gl, gr)
              for L, R, f, gl, gr in ops]
    hb = qm.HostProbeBatch([(L.pin_memory(), -1, R.pin_memory(), -2, f, f, gl, gr) for L, R, f, gl, gr in ops])
    for _ in range(2):
        assert all(_same(g, s) for g, s in zip(hb.run(), single))
    assert hb.h2d_bytes == sum(L.numel() * 2 + R.numel() * 2 for L, R, *_ in ops)


def test_empty_and_bad_batches():
    lib = qm.lib()
    assert lib.qm_probe_batch(0, None, None, None, None, None, None, None) == 0
    assert lib.qm_probe_batch(-1, None, None, None, None, None, None, None) != 0
    assert lib.qm_probe_batch(2, None, None, None, None, None, None, None) != 0
    # a refused probe in the middle: the ones before it still complete, the call reports the error
    L0, R0, f, gl, gr = _ops()[0]
    Ld, Rd = L0.cuda(), R0.cuda()
    want = qm.qm_probe_layer(qm.operand_of(Ld, -1), qm.operand_of(Rd, -2), f, f, gl, gr)
    batch = qm.ProbeBatch([(qm.operand_of(Ld, -1), qm.operand_of(Rd, -2), f, f, gl, gr)] * 3)
    batch.ws_bytes[1] = 16                  # too small
    with pytest.raises(qm.QmError):
        batch.launch()
    torch.cuda.synchronize()
    assert _same(batch.results()[0], want)


def test_format_sweep_over_the_same_tensors_borrows_prepared_operands():
    """Probes of one batch that quantize the very same tensors into different formats share the
    format-independent part of the preparation; every record must still be the single probe's."""
    rng = workloads._rng(120)
    X = workloads.normal(rng, (520, 256)).cuda()              # activations, contraction contiguous
    W = workloads.normal(rng, (256, 392), 0.05).cuda()        # weights stored [K, N]: contraction strided
    Q = workloads.normal(rng, (6, 136, 64)).cuda()            # batched, for shared channel scales
    Kt = workloads.normal(rng, (6, 200, 64)).cuda()
    cases = []
    for gl, gr in (("tensor", "tensor"), ("channel", "channel"), ("tensor", "channel")):
        for f in ("e4m3", "int8", "e5m2"):
            cases.append((qm.operand_of(X, -1), qm.operand_of(W, -2), f, f, gl, gr, {}))
    for f in ("e4m3", "int8"):
        cases.append((qm.operand_of(Q, -1), qm.operand_of(Kt, -1), f, f, "channel", "channel", {"groups": (2, 2)}))
        cases.append((qm.operand_of(X, -1), qm.operand_of(W, -2), f, f, "tensor", "tensor",
                      {"rounding": "stochastic_r", "seed": 3}))
    single = [qm.qm_probe_layer(Lo, Ro, fl, fr, gl, gr, **kw) for Lo, Ro, fl, fr, gl, gr, kw in cases]
    batch = qm.ProbeBatch([c[:6] for c in cases])
    for i, c in enumerate(cases):                             # per-probe extras of the configuration
        kw = c[6]
        batch.cfg[i].round = qm.binding.ROUND[kw.get("rounding", "rtne")]
        batch.cfg[i].seed = kw.get("seed", 0)
        batch.cfg[i].batch_groups_l, batch.cfg[i].batch_groups_r = kw.get("groups", (0, 0))
    for _ in range(2):
        batch.launch()
        torch.cuda.synchronize()
        got = batch.results()
        for i, (g, s) in enumerate(zip(got, single)):
            assert _same(g, s), (i, cases[i][2:], g.record(), s.record())


def test_large_mixed_batch_spans_several_grouped_launches():
    """More probes than one grouped launch takes (16), shapes from a single tile to many, one
    k-block to many, batched operands, both reference modes in one batch."""
    rng = workloads._rng(130)
    shapes = [(64, 64, 64), (256, 128, 64), (300, 200, 128), (1000, 520, 192), (128, 1024, 320), (520, 136, 1040)]
    cases = []
    for i in range(21):
        M, N, K = shapes[i % len(shapes)]
        fmt = ("e4m3", "int8", "e5m2")[i % 3]
        gran = ("tensor", "channel")[(i // 3) % 2]
        ref = "fp32" if i in (4, 11) else "bf16"
        if i % 7 == 6:
            L, R = workloads.normal(rng, (3, M, K)), workloads.normal(rng, (3, N, K), 0.1)
            cases.append((L.cuda(), -1, R.cuda(), -1, fmt, gran, ref))
        else:
            L, R = workloads.student_t(rng, (M, K), 4.0), workloads.normal(rng, (K, N), 0.05)
            cases.append((L.cuda(), -1, R.cuda(), -2, fmt, gran, ref))
    probes = [(qm.operand_of(L, cl), qm.operand_of(R, cr), f, f, g, g, ref) for L, cl, R, cr, f, g, ref in cases]
    single = [qm.qm_probe_layer(*p) for p in probes]
    batch = qm.ProbeBatch(probes)
    for _ in range(2):
        batch.launch()
        torch.cuda.synchronize()
        for i, (g, s) in enumerate(zip(batch.results(), single)):
            assert _same(g, s), (i, cases[i][4:], g.record(), s.record())
