#!/usr/bin/env python
"""Benchmark of the quantized-matmul error probe on B200.

A step is one pass of the whole probe path (scale, quantize, 8-bit product, reference and
denominator products, Eq. 3 reduction) over every product of the workload, repeated `repeat`
times so that a step lasts tens of milliseconds.  The default workload is the unit of the
24-layer BERT-large sweep: one encoder layer (batch 32 x seq 512), its four projections forward,
dgrad and wgrad plus the six batched attention products, each in E4M3, E5M2 and INT8: 54 probes.

  python bench.py --gpus 1 --steps K --warmup W            -> one JSON line (this library)
  python bench.py --impl reference ...                     -> one JSON line (CPU oracle)
  python bench.py --case quantize|stats|gemm|probe|batch   -> a few launches of one small case
                                                              (the command profiler captures run)

With N > 1 ranks (torchrun) every rank probes its own copy of the workload: the probes of a
table are independent, there is no exchange step, so scaling is weak and no collective runs
in the data path.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2408_02897_b200 import workloads  # noqa: E402

# DRAM bytes (read + write) of the fused probe kernel per byte of distinct operand data it reads
# (bf16 L and R and both code tensors), from a profiler capture of one launch over the 12 probes of
# the BERT-large layer workload (2.56 GB moved for 1.485 GB of distinct operand bytes: activations
# larger than L2 are re-read for part of the column tiles; other captures of the same launch
# moved 2.38 and 3.00 GB, so the figure varies by a fifth; 1.07 on the BERT-base workload, which
# fits in L2).  A launch of the default workload has the same projection shapes and is scaled by its
# distinct operand bytes.  None: the kernel has changed since the counters were taken.
TC_DRAM_BYTES_PER_OPERAND_BYTE = 1.72


METRIC = "probe TFLOPS"
UNIT = "TFLOP/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "peak_run_sm_mhz": (d.get("clocks_under_load") or {}).get("sm_mhz_median"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "peak_run_sm_mhz": 1300.0,
            "source": "fallback"}


def build_workload(name):
    if name == "bert_large_sweep_layer":
        t = workloads.config5_layer_tensors(0)
        per_fmt = [workloads.config5_layer(0, fmt, tensors=t) for fmt in ("e4m3", "e5m2", "int8")]
        ops = [o for triple in zip(*per_fmt) for o in triple]        # the three formats of a product side by side
        return ops, ("one layer of the BERT-large 24-layer sweep (batch 32 x seq 512): projections fwd+dgrad+wgrad and "
                     "batched attention products fwd+bwd, each in E4M3, E5M2 and INT8, per-tensor scales")
    if name == "bert_base_fwd":
        return workloads.config2(), "BERT-base forward matmuls (batch 8 x seq 512), E4M3 + INT8, per-tensor scales"
    if name == "bert_large_layer":
        return workloads.config3(), "BERT-large layer fwd+dgrad+wgrad (batch 32 x seq 512), E4M3/E5M2, per-channel weights"
    if name == "outlier":
        return workloads.config4(), "FFN1 outlier stress [16384x1024]x[1024x4096], 3 formats x 2 granularities"
    if name == "single":
        return workloads.config1(), "single fp32 probe 128x256x256"
    raise SystemExit(f"unknown workload {name}")


def distinct_operand_bytes(ops):
    """Bytes the fused kernels of a step read when every distinct tensor is counted once: the bf16
    values of each distinct (tensor, orientation) and one code tensor per distinct (tensor,
    orientation, format)."""
    seen_x, seen_c, total = set(), set(), 0
    for o in ops:
        for t, cd, fmt in ((o["L"], o["cl"], o["fmt_l"]), (o["R"], o["cr"], o["fmt_r"])):
            if (id(t), cd) not in seen_x:
                seen_x.add((id(t), cd))
                total += 2 * t.numel()
            if (id(t), cd, fmt) not in seen_c:
                seen_c.add((id(t), cd, fmt))
                total += t.numel()
    return total


def probe_flops(ops):
    """Flops of one step: the three products of Eq. 3 (8-bit, reference, denominator)."""
    return sum(3.0 * workloads.op_flops(o)[1] for o in ops)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0=None, t1=None):
        """Median SM clock and throttle reasons of the samples that arrived between host times t0
        and t1 (the timed region); all samples when no window is given."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if len(r) < 7 or (t0 is not None and not (t0 <= ts <= t1)):
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "samples_total": len(self.rows), "window": "timed region only",
                "reasons": sorted(reasons)}


def oracle_sample_ops(ops, max_ops=4):
    """The bounded sample of a workload the CPU oracle is timed on: the first `max_ops` distinct
    products (one format each) among the probes whose operands are plain 2-D matrices (the
    projections), or among all probes if there are none."""
    flat = [o for o in ops if o["L"].dim() == 2] or ops
    seen, out = set(), []
    for o in flat:
        key = (id(o["L"]), o["cl"], id(o["R"]), o["cr"])
        if key not in seen:
            seen.add(key)
            out.append(o)
    return out[:max_ops]


def time_oracle_sample(ops, rows_per_op, seed=7):
    """The CPU oracle, as it stands, on a bounded sample: `rows_per_op` output rows (all
    columns) of every given probe; scales and codes are still computed over the whole operands."""
    import oracle
    t0 = time.perf_counter()
    flops = 0.0
    for i, o in enumerate(ops):
        (M, N, K, b), _ = workloads.op_flops(o)
        rows = np.random.default_rng(seed + i).choice(M, min(rows_per_op, M), replace=False)
        L, R = workloads.orient(o)
        oracle.probe(L, R, o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], rows=np.sort(rows))
        flops += 3.0 * 2.0 * len(rows) * N * K * b
    dt = time.perf_counter() - t0
    return flops, dt


def gemm_rates(qm, n=8192, iters=10):
    """T(FL)OP/s of the stand-alone products qm_gemm (E4M3, INT8) and qm_gemm_ref (bf16) at n^3, and,
    as the achievable reference of the same run, of the library GEMMs torch reaches (harness only)."""
    import ctypes as C

    def timed(fn):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e-3

    x = torch.randn(n, n, device="cuda").to(torch.bfloat16)
    w = (torch.randn(n, n, device="cuda") * 0.02).to(torch.bfloat16)
    opx, opw = qm.operand_of(x, -1), qm.operand_of(w, -1)
    F = 2.0 * n ** 3
    L = qm.lib()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    out = torch.empty((1, n, n), dtype=torch.float32, device="cuda")
    res = {"shape": f"{n}^3, fp32 output written"}
    for fmt in ("e4m3", "int8"):
        cx, dx, _, _ = qm.qm_quantize(opx, fmt, "tensor")
        cw, dw, _, _ = qm.qm_quantize(opw, fmt, "tensor")

        def run():
            rc = L.qm_gemm(C.c_void_p(cx.data_ptr()), qm.FMT[fmt], C.c_void_p(dx.data_ptr()), 0,
                           C.c_void_p(cw.data_ptr()), qm.FMT[fmt], C.c_void_p(dw.data_ptr()), 0, n, n, n, 1,
                           C.c_void_p(out.data_ptr()), None, 0, st)
            assert rc == 0, rc
        res[f"qm_gemm_{fmt}_tops"] = F / timed(run) / 1e12
    res["qm_gemm_ref_bf16_tflops"] = F / timed(lambda: qm.qm_gemm_ref(x[None], w[None])) / 1e12
    del out
    try:
        res["library_bf16_tflops"] = F / timed(lambda: torch.matmul(x, w.t())) / 1e12
        xf, wf = x.to(torch.float8_e4m3fn), w.to(torch.float8_e4m3fn)
        one = torch.ones((), device="cuda")
        res["library_e4m3_tflops"] = F / timed(lambda: torch._scaled_mm(xf, wf.t(), scale_a=one, scale_b=one,
                                                                        out_dtype=torch.bfloat16)) / 1e12
        xi = torch.randint(-127, 127, (n, n), device="cuda", dtype=torch.int8)
        res["library_int8_tops"] = F / timed(lambda: torch._int_mm(xi, xi.t())) / 1e12
    except Exception as e:      # the library reference is context only
        res["library_note"] = repr(e)[:120]
    return res


def scale_quantize_rates(qm, hbm_gbs, rows=16384, cols=4096, iters=10):
    """Algorithmic GB/s of the scale / quantize kernels on one FFN-activation-sized bf16 tensor
    (rows x cols, 134 MB: larger than L2), each timed with CUDA events after a warm-up."""
    x = torch.randn(rows, cols, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    n = x.numel()
    op_rows, op_cols = qm.operand_of(x, -1), qm.operand_of(x, -2)

    def timed(fn):
        for _ in range(2):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(iters):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters * 1e-3

    delta = qm.qm_scale(op_rows, "e4m3", "tensor")
    ldc = qm.qm_code_ld(cols)
    codes = torch.empty((1, rows, ldc), dtype=torch.uint8, device="cuda")
    codes_t = torch.empty((1, cols, qm.qm_code_ld(rows)), dtype=torch.uint8, device="cuda")
    dch = torch.empty(rows, dtype=torch.float32, device="cuda")
    d1 = torch.empty(1, dtype=torch.float32, device="cuda")
    import ctypes as C
    L = qm.lib()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def raw_quant(op, gran, dl, dout, cod):
        rc = L.qm_quantize(C.byref(op), 1, gran, 0, C.c_void_p(dl.data_ptr()) if dl is not None else None,
                           C.c_void_p(dout.data_ptr()) if dout is not None else None, C.c_void_p(cod.data_ptr()),
                           None, None, st)
        assert rc == 0, rc

    t_scale = timed(lambda: L.qm_scale(C.byref(op_rows), 1, 0, C.c_void_p(d1.data_ptr()), st))
    t_quant = timed(lambda: raw_quant(op_rows, 0, delta, None, codes))
    t_fused = timed(lambda: raw_quant(op_rows, 1, None, dch, codes))
    t_trans = timed(lambda: raw_quant(op_cols, 0, delta, None, codes_t))
    def raw_quant_sr(op, cod):
        rc = L.qm_quantize_stochastic(C.byref(op), 1, 0, 12345, 0, C.c_void_p(delta.data_ptr()), None,
                                      C.c_void_p(cod.data_ptr()), None, None, st)
        assert rc == 0, rc

    t_sr = timed(lambda: raw_quant_sr(op_rows, codes))
    ws_n = L.qm_stats_workspace_bytes()
    ws = torch.empty(ws_n, dtype=torch.uint8, device="cuda")
    rec = torch.empty(128, dtype=torch.uint8, device="cuda")

    def raw_stats():
        rc = L.qm_tensor_stats(C.byref(op_rows), C.c_void_p(rec.data_ptr()), C.c_void_p(ws.data_ptr()), ws_n, st)
        assert rc == 0, rc

    def raw_error(gran, dl):
        rc = L.qm_quantize_error(C.byref(op_rows), 1, gran, C.c_void_p(dl.data_ptr()), C.c_void_p(rec.data_ptr()),
                                 C.c_void_p(ws.data_ptr()), ws_n, st)
        assert rc == 0, rc

    t_stats = timed(raw_stats)
    t_err = timed(lambda: raw_error(0, delta))
    t_err_ch = timed(lambda: raw_error(1, dch))
    out = {"tensor": f"bf16 [{rows} x {cols}] ({n * 2 / 1e6:.0f} MB)", "hbm_peak_gbs": hbm_gbs,
           "scale_tensor_gbs": 2 * n / t_scale / 1e9,                 # 2 B/elem read
           "quantize_gbs": 3 * n / t_quant / 1e9,                     # 2 B read + 1 B code
           "scale_quantize_rows_gbs": 3 * n / t_fused / 1e9,          # fused per-row scale + codes, input read once
           "quantize_transpose_gbs": 3 * n / t_trans / 1e9,
           "quantize_stochastic_gbs": 3 * n / t_sr / 1e9,              # 2 B read + 1 B code, Philox draws
           "tensor_stats_gbs": 2 * n / t_stats / 1e9,                  # 2 B/elem read, power sums + max
           "quantize_error_gbs": 2 * n / t_err / 1e9,                  # 2 B/elem read, Eq. 2 split, one scale
           "quantize_error_rows_gbs": 2 * n / t_err_ch / 1e9}         # one scale per row
    for k in ("scale_tensor", "quantize", "scale_quantize_rows", "quantize_transpose", "quantize_stochastic", "tensor_stats",
              "quantize_error", "quantize_error_rows"):
        out[k + "_frac_of_hbm"] = out[k + "_gbs"] / hbm_gbs
    return out


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def config_of(args, desc):
    """The `config` object of the JSON line, identical for both arms."""
    return {"workload": args.workload, "description": desc,
            "flops_counted": "3 x 2MNK per probe (8-bit, reference and denominator products)",
            "l2": "256 MiB buffer written between timed steps; the inputs of the default workload are larger than L2 as well"}


def oracle_sample_text(sample, rows, n_all):
    return (f"{rows} of the output rows of each of {len(sample)} of the workload's {n_all} probes "
            f"({', '.join(o['name'] for o in sample)}); scales and codes over whole operands")


def run_reference(args, ops, desc):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = args.oracle_rows
    sample = oracle_sample_ops(ops)
    for _ in range(min(args.warmup, 1)):
        time_oracle_sample(sample, rows)
    flops = secs = 0.0
    for _ in range(args.steps):
        f, t = time_oracle_sample(sample, rows)
        flops += f; secs += t
    val = flops / secs / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(args, desc),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                             "sample": oracle_sample_text(sample, rows, len(ops)) + " per step"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_case(a):
    """--case: a few launches of one kernel family on a small synthetic case and nothing else; the
    command that profiler captures run."""
    import paper_2408_02897_b200 as qm
    torch.cuda.set_device(0)
    rng = workloads._rng(11)
    if a.case == "batch":
        ops, _ = build_workload(a.workload)
        on_dev = {}
        dev = [(on_dev.setdefault(id(o["L"]), o["L"].cuda()), on_dev.setdefault(id(o["R"]), o["R"].cuda())) for o in ops]
        batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                                o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev)])
        for _ in range(a.iters):
            batch.launch()
        torch.cuda.synchronize()
        print("mean_be", [round(r.derived()["mean_be"], 6) for r in batch.results()])
        return
    lead = (a.batch,) if a.batch > 1 else ()
    L = workloads.normal(rng, lead + (a.M, a.K)).cuda()
    R = workloads.normal(rng, lead + ((a.K, a.N) if a.r_layout == "kn" else (a.N, a.K)), 0.02).cuda()
    Lop = qm.operand_of(L, -1)
    Rop = qm.operand_of(R, -2 if a.r_layout == "kn" else -1)
    if a.case == "probe":
        plan = qm.ProbePlan(Lop, Rop, a.fmt, a.fmt, a.gran, a.gran)
        for _ in range(a.iters):
            plan.launch(Lop, Rop)
        torch.cuda.synchronize()
        r = plan.result()
        print("mean_be", r.derived()["mean_be"], "device_error", r.device_error)
    elif a.case == "gemm":
        Rk = R.transpose(-1, -2).contiguous() if a.r_layout == "kn" else R
        cl, dl, _, _ = qm.qm_quantize(Lop, a.fmt, a.gran)
        cr, dr, _, _ = qm.qm_quantize(qm.operand_of(Rk, -1), a.fmt, a.gran)
        L3 = L if L.dim() == 3 else L[None]
        R3 = Rk if Rk.dim() == 3 else Rk[None]
        for _ in range(a.iters):
            out, _ = qm.qm_gemm(cl, a.fmt, dl, a.gran, cr, a.fmt, dr, a.gran, a.K)
            ref = qm.qm_gemm_ref(L3, R3)
        torch.cuda.synchronize()
        print("rel diff of the two products", float((out - ref).norm() / ref.norm()))
    elif a.case == "stats":
        for _ in range(a.iters):
            st = qm.qm_tensor_stats(Lop)
            er = qm.qm_quantize_error(Lop, a.fmt, a.gran)
        print("kurtosis", st.derived()["kurtosis"], "mean RE", er.sum_re / max(er.n_nonzero, 1))
    elif a.case == "quantize":
        Lt = qm.operand_of(L, -2)
        for _ in range(a.iters):
            qm.qm_scale(Lop, a.fmt, "tensor")
            qm.qm_quantize(Lop, a.fmt, "tensor", None)
            qm.qm_quantize(Lop, a.fmt, "channel", None)
            qm.qm_quantize(Lt, a.fmt, "tensor", None)
            qm.qm_quantize_formats(Lop, ["e4m3", "e5m2", "int8"], "tensor")
            qm.qm_quantize_formats(Lt, ["e4m3", "e5m2", "int8"], "tensor", want_kmaj=True)
        torch.cuda.synchronize()
        print("done")
    else:
        raise SystemExit(f"unknown case {a.case}")


def time_workload(qm, ranks, world, name, steps, warmup, target_ms=50.0, clock_index=None):
    """Times `steps` steps of a workload resident in HBM.  A step is `repeat` passes over the
    workload's probes (one qm_probe_batch call per pass) between one CUDA-event pair, with the L2
    flushed before it.  Returns a dict of the measurements."""
    ops, desc = build_workload(name)
    on_dev = {}

    def resident(t):
        # a tensor that several probes share (a layer probed in several formats, an activation that
        # feeds several products) is resident once
        if id(t) not in on_dev:
            on_dev[id(t)] = t.cuda()
        return on_dev[id(t)]
    batch = qm.ProbeBatch([(qm.operand_of(resident(o["L"]), o["cl"]), qm.operand_of(resident(o["R"]), o["cr"]),
                            o["fmt_l"], o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"]) for o in ops])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB L2

    def barrier():
        torch.cuda.synchronize()
        ranks.barrier(world)
        torch.cuda.synchronize()

    # repeat count from one measured pass, so that a step lasts about target_ms
    batch.launch()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(); batch.launch(); b.record()
    barrier()
    pass_ms = ranks.max_over_ranks(a.elapsed_time(b), world, "cuda")
    repeat = max(1, int(np.ceil(target_ms / pass_ms)))

    def step():
        for _ in range(repeat):
            batch.launch()

    for _ in range(max(warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(clock_index) if clock_index is not None else None
    if sampler:
        sampler.start()
        time.sleep(0.5)               # nvidia-smi needs a moment to start; samples outside the window are dropped
    launches0 = qm.kernel_launches()
    qm.profile_enable(True)           # the library records an event pair around each fused launch
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    t0 = time.time()
    for a, b in evs:
        flush.zero_()
        a.record()
        step()
        b.record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    step_ms = [a.elapsed_time(b) for a, b in evs]
    tc_ms, tc_launches = qm.profile_read()
    qm.profile_enable(False)
    launches = qm.kernel_launches() - launches0
    total_ms = ranks.max_over_ranks(float(sum(step_ms)), world, "cuda")
    results = batch.results()
    if any(r.device_error for r in results):
        raise SystemExit("device error flagged in a probe result")
    flops_pass = probe_flops(ops)
    return {"ops": ops, "desc": desc, "results": results, "repeat": repeat, "total_ms": total_ms, "steps": steps,
            "flops_step": flops_pass * repeat, "flops_pass": flops_pass, "tc_ms": tc_ms, "tc_launches": tc_launches,
            "launches": int(launches), "clocks": clocks, "wall_s": t1 - t0,
            "value": ranks.whole_job_rate(flops_pass * repeat * steps, world, total_ms) / 1e12}


def roofline_of(m, peaks, bench_mhz):
    """The roofline block of the dominant kernel (the grouped fused probe kernel) of a measurement.

    Composite tensor bound: per 2MNK one product at the 8-bit rate (2 x bf16) and two at the bf16
    rate -> 3 / (1/(2P) + 2/P) = 1.2 P in summed flops.  P is the sustained bf16 figure when the
    timed region lasted seconds (the kernel then runs under the same power cap as that
    measurement), the burst figure otherwise."""
    long_region = m["wall_s"] >= 1.0 and peaks.get("bf16_tflops_sustained")
    p16 = peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"]
    peak = 1.2 * p16
    achieved = m["flops_step"] * m["steps"] / (m["tc_ms"] * 1e-3) / 1e12 if m["tc_ms"] > 0 else None
    traffic = None
    if TC_DRAM_BYTES_PER_OPERAND_BYTE is not None and m["tc_launches"]:
        traffic = TC_DRAM_BYTES_PER_OPERAND_BYTE * distinct_operand_bytes(m["ops"]) * m["repeat"] * m["steps"] / m["tc_launches"]
    r = {"bound": "tensor",
         "kernel": "tc_group_kernel (fused 8-bit + reference + denominator products and Eq. 3 epilogue of up to 16 "
                   "probes per persistent launch)",
         "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak if achieved else None,
         "traffic": traffic,
         "traffic_note": "DRAM bytes per launch, scaled from a profiler capture of a smaller workload by distinct operand bytes",
         "peak_source": f"1.2 x {'bf16_tflops_sustained' if long_region else 'bf16_tflops'} ({p16}) of {peaks['source']}",
         "launches": m["tc_launches"], "avg_launch_ms": m["tc_ms"] / max(m["tc_launches"], 1),
         "timing": "CUDA event pair around every launch, recorded by the library on the launching stream inside the timed steps",
         "frac_of_burst_peak": achieved / (1.2 * peaks["bf16_tflops"]) if achieved else None,
         "whole_step_frac": m["value"] / peak,
         "whole_step_note": "the step's rate (scale/quantize kernels included) against the same composite peak",
         "frac_of_nominal": achieved / (1.2 * 2250.0) if achieved else None,
         "nominal_note": "against 1.2 x 2250 TFLOP/s (nominal dense bf16; 8-bit = 2x), context only",
         "targets": {"fused_probe_ge_0.70_of_composite_peak": bool(achieved and achieved / peak >= 0.70)}}
    if bench_mhz and peaks.get("peak_run_sm_mhz"):
        scaled = peak * bench_mhz / peaks["peak_run_sm_mhz"]
        r["clock_normalised"] = {"frac": achieved / scaled if achieved else None, "bench_sm_mhz": bench_mhz,
                                 "peak_run_sm_mhz": peaks["peak_run_sm_mhz"],
                                 "note": "achieved / (peak x bench MHz / MHz of the run that measured the peak)"}
    return r


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="timed steps (each at least --step-ms long)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bert_large_sweep_layer")
    ap.add_argument("--step-ms", type=float, default=50.0,
                    help="the workload is repeated inside a step until the step lasts about this long")
    ap.add_argument("--oracle-rows", type=int, default=8192)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads, the scale/quantize and the stand-alone GEMM rate blocks")
    ap.add_argument("--case", default=None, help="run a few launches of one small case and exit (profiler runs)")
    ap.add_argument("--M", type=int, default=4096)
    ap.add_argument("--N", type=int, default=3072)
    ap.add_argument("--K", type=int, default=768)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--fmt", default="e4m3")
    ap.add_argument("--gran", default="tensor")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--r-layout", default="kn", choices=["kn", "nk"], help="--case: R stored [K,N] or [N,K]")
    args = ap.parse_args()

    if args.case:
        run_case(args)
        return
    if args.impl == "reference":
        ops, desc = build_workload(args.workload)
        if args.steps == 20 and args.warmup == 3:
            args.steps, args.warmup = 3, 1
        run_reference(args, ops, desc)
        return

    import paper_2408_02897_b200 as qm
    import torch.distributed as dist

    from paper_2408_02897_b200 import ranks
    rank, world, local = ranks.rank_info()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    qm.lib()   # fail now if the CUDA library is missing

    m = time_workload(qm, ranks, world, args.workload, args.steps, args.warmup, args.step_ms, clock_index=local)
    ops, desc, results = m["ops"], m["desc"], m["results"]

    # ---- end to end through the host-buffer entry point: H2D of every operand and D2H of the
    # records inside the timed region; the copies of one probe overlap the kernels of another
    pinned = {}

    def pin(t):
        if id(t) not in pinned:
            pinned[id(t)] = t.pin_memory()
        return pinned[id(t)]
    host_batch = qm.HostProbeBatch([(pin(o["L"]), o["cl"], pin(o["R"]), o["cr"], o["fmt_l"],
                                     o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"]) for o in ops])
    h2d, d2h = host_batch.h2d_bytes, host_batch.d2h_bytes

    def barrier():
        torch.cuda.synchronize()
        ranks.barrier(world)
        torch.cuda.synchronize()
    for _ in range(2):
        host_batch.run()
    barrier()
    e2e_steps = max(3, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_results = host_batch.run()   # waits for the records itself
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_value = ranks.whole_job_rate(m["flops_pass"] * e2e_steps, world, ranks.max_over_ranks(e2e_ms, world, "cuda")) / 1e12
    for o, a, b in zip(ops, e2e_results, results):
        ra, rb = a.record(), b.record()
        # the two paths sum the same tile values over different tile-to-CTA assignments
        if ra["count"] != rb["count"] or any(abs(ra[k] - rb[k]) > 1e-9 * abs(rb[k]) for k in ("sum_be", "sum_diff2", "sum_ref2", "sum_den2")):
            raise SystemExit(f"end-to-end record of {o['name']} differs from the device-resident one")
    del host_batch, pinned

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    clocks = m["clocks"]
    roofline = roofline_of(m, peaks, clocks["sm_mhz"] if clocks else None)
    line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": m["total_ms"] / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "fp8/int8 x bf16 (fp32/int32 accumulate)",
            "data": "synthetic", "config": config_of(args, desc),
            "run": {"probes_per_pass": len(ops), "passes_per_step": m["repeat"], "timed_region_s": m["wall_s"],
                    "issue": "qm_probe_batch: one call per pass; every distinct operand is scaled and quantized once "
                             "(all its formats in one pass over it) on the library's 8 streams, then fused launches of "
                             "up to 16 probes on the caller's stream"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "one pass per step through qm_probe_batch_host: every distinct pinned host operand copied in "
                            "once, records copied out, inside the timed region"},
            "gpu_launches": m["launches"], "roofline": roofline,
            "mean_be": {o["name"]: r.derived()["mean_be"] for o, r in zip(ops, results)}}
    if not args.no_extras:
        others = {}
        for name in ("bert_large_layer", "bert_base_fwd"):
            if name == args.workload:
                continue
            mo = time_workload(qm, ranks, world, name, 10, 3, args.step_ms)
            ro = roofline_of(mo, peaks, None)
            others[name] = {"value": mo["value"], "unit": UNIT, "ms_per_pass": mo["total_ms"] / mo["steps"] / mo["repeat"],
                            "passes_per_step": mo["repeat"], "fused_kernel_tflops": ro["achieved"],
                            "fused_kernel_frac": ro["frac"], "peak": ro["peak"], "peak_source": ro["peak_source"]}
        line["other_workloads"] = others
        sq = scale_quantize_rates(qm, peaks["hbm_gbs"])
        sq["targets"] = {"scale_quantize_ge_0.80_of_hbm": bool(min(sq["scale_tensor_frac_of_hbm"], sq["quantize_frac_of_hbm"]) >= 0.80)}
        line["scale_quantize"] = sq
        line["gemm"] = gemm_rates(qm)
    if not args.no_cpu_baseline and world == 1:
        sample = oracle_sample_ops(ops)
        f, sec = time_oracle_sample(sample, args.oracle_rows)
        line["cpu_baseline"] = {"value": f / sec / 1e12, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": oracle_sample_text(sample, args.oracle_rows, len(ops)) + f", {sec:.1f} s"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
