"""CPU-only checks of the C-ABI boundary: the library loads, exports every declared symbol,
and rejects bad arguments on the host before anything is launched."""
import ctypes as C
import os
import re

import pytest

import paper_2408_02897_b200 as qm
from paper_2408_02897_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qm_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = qm.lib()
    names = declared_functions()
    assert {"qm_scale", "qm_quantize", "qm_gemm", "qm_metric", "qm_probe_layer", "qm_workspace_bytes",
            "qm_status_string", "qm_version"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_struct_layouts_match_header(tmp_path):
    """The ctypes mirrors have the sizes and field offsets a C compiler gives the header's structs."""
    import subprocess
    pairs = [("qm_metric_result", binding.MetricResult), ("qm_operand", binding.Operand),
             ("qm_probe_cfg", binding.ProbeCfg), ("qm_tensor_stats_result", binding.TensorStats),
             ("qm_quant_error_result", binding.QuantError), ("qm_metric_scalars_t", binding.MetricScalars),
             ("qm_tensor_moments_t", binding.TensorMoments)]
    lines = []
    for cname, cls in pairs:
        lines.append(f'printf("{cname} %zu", sizeof({cname}));')
        for fname, _ in cls._fields_:
            lines.append(f'printf(" %zu", offsetof({cname}, {fname}));')
        lines.append('printf("\\n");')
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "qm.h"\nint main(void) {\n' + "\n".join(lines) + "\nreturn 0; }\n")
    exe = tmp_path / "layout"
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    subprocess.check_call(["gcc", "-std=c99", "-I", inc, str(src), "-o", str(exe)])
    out = subprocess.check_output([str(exe)], text=True).strip().splitlines()
    for (cname, cls), line in zip(pairs, out):
        w = line.split()
        assert w[0] == cname and int(w[1]) == C.sizeof(cls), line
        assert [int(x) for x in w[2:]] == [getattr(cls, f).offset for f, _ in cls._fields_], line
    assert C.sizeof(binding.MetricResult) == 56 and C.sizeof(binding.ProbeCfg) == 48


def test_host_side_argument_checks():
    L = qm.lib()
    assert L.qm_code_ld(1) == 16 and L.qm_code_ld(16) == 16 and L.qm_code_ld(17) == 32
    assert L.qm_status_string(0) == b"ok"
    op = binding.Operand()
    assert L.qm_scale(C.byref(op), 1, 0, None, None) == 1           # null data
    op.data = 0x1000; op.dtype = 1; op.noncontract = 8; op.contract = 32
    op.stride_nc = 32; op.stride_c = 1; op.batch = 1
    assert L.qm_scale(C.byref(op), 7, 0, C.c_void_p(0x2000), None) == 1    # bad format
    assert L.qm_scale(C.byref(op), 1, 0, None, None) == 1                  # null output
    op.stride_nc = 33
    assert L.qm_scale(C.byref(op), 1, 0, C.c_void_p(0x2000), None) == 3    # stride alignment
    op.stride_nc = 32; op.data = 0x1004
    assert L.qm_scale(C.byref(op), 1, 0, C.c_void_p(0x2000), None) == 3    # pointer alignment
    op.data = 0x1000; op.stride_c = 2
    assert L.qm_scale(C.byref(op), 1, 0, C.c_void_p(0x2000), None) == 2    # no unit stride
    op.stride_c = 1; op.stride_nc = 16
    assert L.qm_scale(C.byref(op), 1, 0, C.c_void_p(0x2000), None) == 1    # overlapping rows
    # probe configuration checks
    a = binding.Operand(); b = binding.Operand()
    for o, nc in ((a, 64), (b, 48)):
        o.data = 0x1000; o.dtype = 1; o.noncontract = nc; o.contract = 32
        o.stride_nc = 32; o.stride_c = 1; o.batch = 1
    cfg = binding.ProbeCfg(1, 1, 0, 0, 0, 0)
    assert L.qm_workspace_bytes(C.byref(a), C.byref(b), C.byref(cfg)) > 0
    cfg.fmt_r = 0                                                          # INT8 mixed with FP8
    assert L.qm_workspace_bytes(C.byref(a), C.byref(b), C.byref(cfg)) == 0
    assert L.qm_probe_layer(C.byref(a), C.byref(b), C.byref(cfg), C.c_void_p(0x100), C.c_void_p(0x100), 1 << 30, None) == 2
    cfg.fmt_r = 1; b.contract = 64; b.stride_nc = 64                       # K mismatch
    assert L.qm_probe_layer(C.byref(a), C.byref(b), C.byref(cfg), C.c_void_p(0x100), C.c_void_p(0x100), 1 << 30, None) == 1
    b.contract = 32; b.stride_nc = 32
    assert L.qm_probe_layer(C.byref(a), C.byref(b), C.byref(cfg), C.c_void_p(0x100), C.c_void_p(0x100), 16, None) == 4
    assert L.qm_probe_layer(C.byref(a), C.byref(b), C.byref(cfg), C.c_void_p(0x100), C.c_void_p(0x104), 1 << 30, None) == 3
    a.dtype = 0                                                            # fp32 operand on the bf16 path
    assert L.qm_probe_layer(C.byref(a), C.byref(b), C.byref(cfg), C.c_void_p(0x100), C.c_void_p(0x100), 1 << 30, None) == 2
    assert L.qm_metric(None, None, None, 4, None, None, 0, None) == 1
    assert L.qm_gemm(None, 0, None, 0, None, 0, None, 0, 1, 1, 16, 1, None, None, 0, None) == 1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libqm.so")
    with pytest.raises(qm.QmError):
        binding.lib()


def test_batch_and_two_format_argument_checks_need_no_gpu():
    L = qm.lib()
    assert L.qm_probe_batch(0, None, None, None, None, None, None, None) == 0       # empty batch: nothing to do
    assert L.qm_probe_batch(-1, None, None, None, None, None, None, None) == 1
    assert L.qm_probe_batch(3, None, None, None, None, None, None, None) == 1
    assert L.qm_probe_batch_host(0, None, None, None, None, None, None, None, None, None, None) == 0
    assert L.qm_probe_layer2(None, None, None, None, None, None, 0, None) == 1
    assert L.qm_workspace_bytes2(None, None, None, None) == 0
    assert L.qm_stats_workspace_bytes() >= 4096
    op = binding.Operand()
    assert L.qm_tensor_stats(C.byref(op), None, None, 0, None) == 1                   # null data
    assert L.qm_scale_shared(C.byref(op), 1, 1, None, None) == 1


def test_derived_scalars_come_from_the_library():
    """qm_metric_scalars on the record of the hand-computed 2x2x2 case (tests/golden/hand_2x2x2.txt
    holds the record's sums and the scalars worked out by hand), and qm_tensor_moments on small
    arrays whose moments are known in closed form."""
    lit = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "hand_2x2x2.txt")):
        w = line.split()
        if len(w) == 2 and not line.startswith("#"):
            lit[w[0]] = float(w[1])
    rec = binding.MetricResult(4 * lit["mean_be"], lit["max_be"], lit["sum_diff2"], lit["sum_ref2"], lit["sum_den2"], 4, 0, 0)
    got = rec.derived()
    assert set(got) == {"mean_be", "max_be", "normwise_be", "rel_l2", "snr_db"}
    for k, v in got.items():
        assert abs(v - lit[k]) <= 1e-14 * abs(lit[k]), (k, v, lit[k])
    exact = binding.MetricResult(0.0, 0.0, 0.0, 5.0, 7.0, 3, 0, 0).derived()
    assert exact["snr_db"] == float("inf") and exact["rel_l2"] == 0 and exact["normwise_be"] == 0
    empty = binding.MetricResult(0.0, 0.0, 0.0, 0.0, 0.0, 0, 0, 0).derived()
    assert all(empty[k] == 0 for k in ("mean_be", "max_be", "normwise_be", "rel_l2"))
    L = qm.lib()
    assert L.qm_metric_scalars(None, None) == 1 and L.qm_tensor_moments(None, None) == 1

    def moments(xs):
        t = binding.TensorStats(sum(xs), sum(x ** 2 for x in xs), sum(x ** 3 for x in xs), sum(x ** 4 for x in xs),
                                max(abs(x) for x in xs), len(xs), 0, 0)
        return t.derived()
    m = moments([1, 2, 3, 4])                     # mean 5/2, variance 5/4, symmetric, m4 = 41/16
    assert m["mean"] == 2.5 and m["variance"] == 1.25 and m["skew"] == 0.0 and abs(m["kurtosis"] - 1.64) < 1e-15
    m = moments([0, 0, 0, 4])                     # mean 1, m2 = 3, m3 = 6, m4 = 21
    assert m["mean"] == 1 and m["variance"] == 3 and abs(m["skew"] - 6 / 3 ** 1.5) < 1e-15 and abs(m["kurtosis"] - 21 / 9) < 1e-15
    m = moments([7, 7, 7])                        # constant tensor: no spread, skew and kurtosis reported as 0
    assert m == {"mean": 7.0, "variance": 0.0, "skew": 0.0, "kurtosis": 0.0}
    # a badly centred tensor (mean / sigma = 1e4): the extended-precision evaluation keeps the variance
    xs = [10000 + d for d in (-1, 0, 1)] * 5
    m = moments(xs)
    assert abs(m["variance"] - 2 / 3) < 1e-6 and abs(m["skew"]) < 1e-3
