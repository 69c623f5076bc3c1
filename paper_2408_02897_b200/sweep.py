"""The per-operation metric table of a whole encoder stack: every compute-intensive matmul of
every layer (the four projections forward, dgrad and wgrad, and the batched attention score and
context products forward and backward) probed in each 8-bit format.

This is the measurement the method is built on ("per operation quantization error" of every
matmul, Results section; the table's layout follows Table 1: tensor category x format x
granularity).  One layer's probes of all formats go to the library as one qm_probe_batch call,
so tensors shared by several probes (the same activation under three formats, the same weight in
forward and dgrad) are scaled once.  One JSON line per op is appended to the output file as soon
as its layer is done; a rerun with the same file skips the layers it already holds.

  python -m paper_2408_02897_b200.sweep --layers 24 --formats e4m3,e5m2,int8 --out table.jsonl
"""
import argparse
import json
import os
import time

import torch

from . import binding as qm
from . import workloads


def finished_layers(path, formats):
    """Layers whose every (op, format) line is already in the file."""
    per_layer = {}
    if os.path.exists(path):
        for line in open(path):
            try:
                r = json.loads(line)
            except ValueError:
                continue                      # a line cut off by an interrupted run
            per_layer.setdefault(r.get("layer"), set()).add((r.get("op"), r.get("sweep_format")))
    done = set()
    for layer, have in per_layer.items():
        if len(have) >= 18 * len(formats) and {f for _, f in have} >= set(formats):
            done.add(layer)
    return done


def layer_records(layer, formats, shape, per_op_time=True):
    """Probes one layer in all formats; returns (list of per-op dicts, milliseconds of the batch)."""
    tensors = workloads.config5_layer_tensors(layer, **shape)
    ops = [o for fmt in formats for o in workloads.config5_layer(layer, fmt, tensors=tensors, **shape)]
    on_dev = {}

    def resident(t):
        if id(t) not in on_dev:
            on_dev[id(t)] = t.cuda()
        return on_dev[id(t)]
    probes = [(qm.operand_of(resident(o["L"]), o["cl"]), qm.operand_of(resident(o["R"]), o["cr"]), o["fmt_l"],
               o["fmt_r"], o["gran_l"], o["gran_r"], o["ref"]) for o in ops]
    batch = qm.ProbeBatch(probes)
    batch.launch()                                   # warm-up: first-use set-up of streams and kernels
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    batch.launch()
    e1.record()
    torch.cuda.synchronize()
    batch_ms = e0.elapsed_time(e1)
    results = batch.results()
    op_us = [None] * len(ops)
    if per_op_time:
        # each probe on its own (its scale / quantize kernels and its fused kernel), one after the other
        evs = []
        for i, p in enumerate(probes):
            plan = qm.ProbePlan(*p)
            plan.launch(p[0], p[1])
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            plan.launch(p[0], p[1])
            b.record()
            evs.append((a, b))
            del plan
        torch.cuda.synchronize()
        op_us = [a.elapsed_time(b) * 1e3 for a, b in evs]
    rows = []
    n_fmt = len(formats)
    for i, (o, r) in enumerate(zip(ops, results)):
        if r.device_error:
            raise RuntimeError(f"device error {r.device_error} in {o['name']}")
        (M, N, K, b), flops = workloads.op_flops(o)
        ps, role_l, role_r = workloads.op_roles(o["name"])
        fmt = formats[i // (len(ops) // n_fmt)]
        row = {"layer": layer, "op": o["name"].rsplit("-", 1)[0].split("-", 1)[1], "pass": ps, "sweep_format": fmt,
               "role_l": role_l, "role_r": role_r, "fmt_l": o["fmt_l"], "fmt_r": o["fmt_r"],
               "gran_l": o["gran_l"], "gran_r": o["gran_r"], "M": M, "N": N, "K": K, "batch": b,
               "weight_std": tensors["wstd"], "record": r.record(), **r.derived()}
        if op_us[i] is not None:
            row["us"] = op_us[i]
            row["tflops_3_products"] = 3.0 * flops / (op_us[i] * 1e-6) / 1e12
        rows.append(row)
    return rows, batch_ms


def markdown_table(path, out_path):
    """Mean backward error per (op, pass) and format, averaged over the layers, as a markdown table."""
    acc = {}
    fmts = []
    for line in open(path):
        try:
            r = json.loads(line)
        except ValueError:
            continue
        if r["sweep_format"] not in fmts:
            fmts.append(r["sweep_format"])
        acc.setdefault((r["op"], r["role_l"], r["role_r"]), {}).setdefault(r["sweep_format"], []).append(
            (r["mean_be"], r["snr_db"]))
    with open(out_path, "w") as f:
        f.write("| op | L | R | " + " | ".join(f"mean BE {x} | SNR dB {x}" for x in fmts) + " |\n")
        f.write("|---|---|---|" + "---|---|" * len(fmts) + "\n")
        for (op, rl, rr), per in acc.items():
            cells = []
            for x in fmts:
                v = per.get(x, [])
                cells.append(f"{sum(a for a, _ in v) / len(v):.3e} | {sum(b for _, b in v) / len(v):.2f}" if v else "- | -")
            f.write(f"| {op} | {rl} | {rr} | " + " | ".join(cells) + " |\n")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=24)
    ap.add_argument("--formats", default="e4m3,e5m2,int8")
    ap.add_argument("--out", default="sweep.jsonl")
    ap.add_argument("--table", default=None, help="also write a markdown summary to this path")
    ap.add_argument("--tokens", type=int, default=16384, help="batch x sequence length (M)")
    ap.add_argument("--hidden", type=int, default=1024)
    ap.add_argument("--ffn", type=int, default=4096)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--seq", type=int, default=512)
    ap.add_argument("--no-per-op-time", action="store_true")
    a = ap.parse_args()
    formats = a.formats.split(",")
    shape = dict(M=a.tokens, H=a.hidden, F=a.ffn, heads=a.heads, S=a.seq)
    qm.lib()
    done = finished_layers(a.out, formats)
    t_all = time.time()
    for layer in range(a.layers):
        if layer in done:
            continue
        rows, batch_ms = layer_records(layer, formats, shape, not a.no_per_op_time)
        with open(a.out, "a") as f:
            for r in rows:
                r["layer_batch_ms"] = batch_ms
                f.write(json.dumps(r) + "\n")
        print(f"layer {layer}: {len(rows)} ops, {batch_ms:.2f} ms as one batch, "
              f"mean BE {min(r['mean_be'] for r in rows):.2e}..{max(r['mean_be'] for r in rows):.2e}", flush=True)
        torch.cuda.empty_cache()
    if a.table:
        markdown_table(a.out, a.table)
    print(f"done in {time.time() - t_all:.0f} s")


if __name__ == "__main__":
    main()
