#!/usr/bin/env python
"""Benchmark of the quantized-matmul error probe on B200.

A step is one pass of the whole probe path (scale, quantize, 8-bit product, reference and
denominator products, Eq. 3 reduction) over every product of the workload.  The default
workload is the BERT-base forward set (batch 8 x seq 512: QKV, attention output, FFN1, FFN2;
E4M3 and INT8 with per-tensor scales): 8 probes per step.

  python bench.py --gpus 1 --steps K --warmup W            -> one JSON line (this library)
  python bench.py --impl reference ...                     -> one JSON line (CPU oracle)

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

# DRAM traffic of the fused probe kernel from one ncu capture (profiles/tc_kernel_probe_*.md):
# dram__bytes_read + dram__bytes_write for M=4096 N=2304 K=768 E4M3, and the library's kernel
# revision the counters were taken at.  Traffic grows with the operand bytes (every operand is
# read from DRAM once), so a launch of another shape is scaled by its operand bytes.
NCU_TC = {"revision": "tc-group-rot4-refahead-2", "workload": "bert_base_fwd", "dram_bytes": 200.0e6}


def tc_operand_bytes(M, N, K, b=1):
    """Bytes the fused kernel reads per launch: L, |L| (bf16), R, |R| (bf16) and both code tensors."""
    return b * ((M + N) * K * 2 * 2 + (M + N) * K)


METRIC = "probe TFLOPS"
UNIT = "TFLOP/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def build_workload(name):
    if name == "bert_base_fwd":
        return workloads.config2(), "BERT-base forward matmuls (batch 8 x seq 512), E4M3 + INT8, per-tensor scales"
    if name == "bert_large_layer":
        return workloads.config3(), "BERT-large layer fwd+dgrad+wgrad (batch 32 x seq 512), E4M3/E5M2, per-channel weights"
    if name == "outlier":
        return workloads.config4(), "FFN1 outlier stress [16384x1024]x[1024x4096], 3 formats x 2 granularities"
    if name == "single":
        return workloads.config1(), "single fp32 probe 128x256x256"
    raise SystemExit(f"unknown workload {name}")


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
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle_sample(ops, rows_per_op, seed=7):
    """The CPU oracle, as it stands, on a bounded sample: `rows_per_op` output rows (all
    columns) of every probe; scales and codes are still computed over the whole operands."""
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


def run_reference(args, ops, desc):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = args.oracle_rows
    for _ in range(min(args.warmup, 1)):
        time_oracle_sample(ops, rows)
    flops = secs = 0.0
    for _ in range(args.steps):
        f, t = time_oracle_sample(ops, rows)
        flops += f; secs += t
    val = flops / secs / 1e12
    sample = f"{rows} of the output rows of each of the {len(ops)} probes per step (scales and codes over whole operands)"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "description": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500,
                    help="timed steps (0.4 ms each: the default keeps the GPU under load long enough for the clock samples)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bert_base_fwd")
    ap.add_argument("--oracle-rows", type=int, default=4096)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the scale/quantize and stand-alone GEMM rate blocks (profiling runs)")
    args = ap.parse_args()

    ops, desc = build_workload(args.workload)
    if args.impl == "reference":
        if args.steps == 500 and args.warmup == 3:
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

    # ---- inputs resident in HBM; one workspace and one result record per probe
    # (a tensor that several probes of the step share, here the same layer probed in two formats,
    # is resident once)
    on_dev = {}

    def resident(t):
        if id(t) not in on_dev:
            on_dev[id(t)] = t.cuda()
        return on_dev[id(t)]
    dev_tensors = [(resident(o["L"]), resident(o["R"])) for o in ops]
    batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                            o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev_tensors)])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB L2

    def step():
        batch.launch()      # qm_probe_batch: the step's probes, spread over the library's streams

    def barrier():
        torch.cuda.synchronize()
        ranks.barrier(world)
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- timed region: K steps, each between its own event pair, L2 flushed in between
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = qm.kernel_launches()
    # the step's fused kernels are ONE grouped launch on this stream, issued after every scale /
    # quantize chain has been joined: the library's event pair around it times it alone
    qm.profile_enable(True)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in evs:
        flush.zero_()
        a.record()
        step()
        b.record()
    barrier()
    step_ms = [a.elapsed_time(b) for a, b in evs]
    tc_ms, tc_launches = qm.profile_read()
    qm.profile_enable(False)
    launches = qm.kernel_launches() - launches0
    total_ms = ranks.max_over_ranks(float(sum(step_ms)), world, "cuda")
    results = batch.results()
    if any(r.device_error for r in results):
        raise SystemExit("device error flagged in a probe result")

    clocks = sampler.stop()

    flops_step = probe_flops(ops)
    value = ranks.whole_job_rate(flops_step * args.steps, world, total_ms) / 1e12

    # ---- end to end through the host-buffer entry point: H2D of every operand and D2H of the
    # records inside the timed region; the copies of one probe overlap the kernels of another
    host_batch = qm.HostProbeBatch([(o["L"].pin_memory(), o["cl"], o["R"].pin_memory(), o["cr"], o["fmt_l"],
                                     o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"]) for o in ops])
    h2d, d2h = host_batch.h2d_bytes, host_batch.d2h_bytes

    for _ in range(3):
        host_batch.run()
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_results = host_batch.run()   # waits for the records itself
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_value = ranks.whole_job_rate(flops_step * e2e_steps, world, ranks.max_over_ranks(e2e_ms, world, "cuda")) / 1e12
    if any(a.record() != b.record() for a, b in zip(e2e_results, results)):
        raise SystemExit("end-to-end records differ from the device-resident ones")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    sq = None if args.no_extras else scale_quantize_rates(qm, peaks["hbm_gbs"])
    # composite tensor bound of the fused kernel: per 2MNK, one product at the 8-bit rate
    # (2 x bf16) and two at the bf16 rate  ->  3 / (1/(2P) + 2/P) = 1.2 P in summed flops
    peak_tflops = 1.2 * peaks["bf16_tflops"]
    achieved = flops_step * args.steps / (tc_ms * 1e-3) / 1e12 if tc_ms > 0 else None
    traffic = None
    if qm.lib().qm_kernel_revision().decode() == NCU_TC["revision"] and args.workload == NCU_TC["workload"]:
        traffic = NCU_TC["dram_bytes"]
    roofline = {"bound": "tensor",
                "kernel": "tc_group_kernel (fused 8-bit + reference + denominator products and Eq. 3 epilogue of the "
                          "step's probes, one persistent launch per step)",
                "achieved": achieved, "peak": peak_tflops, "unit": "TFLOP/s",
                "frac": achieved / peak_tflops if achieved else None, "traffic": traffic,
                "traffic_note": "DRAM bytes of one grouped launch of this workload, from the ncu capture in profiles/",
                "peak_source": f"1.2 x bf16_tflops ({peaks['bf16_tflops']}) of {peaks['source']}",
                "launches": tc_launches, "avg_launch_ms": tc_ms / max(tc_launches, 1),
                "timing": "CUDA event pair around every launch, recorded by the library on the launching stream "
                          "inside the timed steps"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8/int8 x bf16 (fp32/int32 accumulate)", "data": "synthetic",
            "config": {"workload": args.workload, "description": desc, "probes_per_step": len(ops),
                       "flops_counted": "3 x 2MNK per probe (8-bit, reference and denominator products)",
                       "issue": "qm_probe_batch: one call per step, probes spread over 3 library streams",
                       "l2": "256 MiB buffer written between timed steps"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches), "roofline": roofline,
            "pct_of_composite_tensor_peak": 100.0 * value / peak_tflops,
            "scale_quantize": sq, "gemm": None if args.no_extras else gemm_rates(qm),
            "mean_be": {o["name"]: r.derived()["mean_be"] for o, r in zip(ops, results)}}
    if not args.no_cpu_baseline and world == 1:
        f, s = time_oracle_sample(ops, args.oracle_rows)
        line["cpu_baseline"] = {"value": f / s / 1e12, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": f"{args.oracle_rows} of the output rows of each of the {len(ops)} probes "
                                          f"(scales and codes over whole operands), {s:.1f} s"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
