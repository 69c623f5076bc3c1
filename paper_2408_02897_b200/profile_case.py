"""Runs one probe (or only its scale/quantize stage) a few times on synthetic operands.

Meant to be the command profiled by ncu on a small case, e.g.
  python -m paper_2408_02897_b200.profile_case --M 4096 --N 3072 --K 768 --fmt e4m3 --iters 3
"""
import argparse

import torch

from . import binding as qm
from . import workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--M", type=int, default=4096)
    ap.add_argument("--N", type=int, default=3072)
    ap.add_argument("--K", type=int, default=768)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--fmt", default="e4m3")
    ap.add_argument("--gran", default="tensor")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--stage", default="probe", choices=["probe", "quantize", "stats", "gemm", "batch"])
    ap.add_argument("--r-layout", default="kn", choices=["kn", "nk"], help="R stored [K,N] or [N,K]")
    a = ap.parse_args()
    if a.stage == "batch":
        # the benchmark's step: the eight probes of the BERT-base forward workload as one batch
        ops = workloads.config2()
        on_dev = {}
        dev = [(on_dev.setdefault(id(o["L"]), o["L"].cuda()), on_dev.setdefault(id(o["R"]), o["R"].cuda())) for o in ops]
        batch = qm.ProbeBatch([(qm.operand_of(Ld, o["cl"]), qm.operand_of(Rd, o["cr"]), o["fmt_l"], o["fmt_r"],
                                o["gran_l"], o["gran_r"], o["ref"]) for o, (Ld, Rd) in zip(ops, dev)])
        for _ in range(a.iters):
            batch.launch()
        torch.cuda.synchronize()
        print("mean_be", [round(r.derived()["mean_be"], 6) for r in batch.results()])
        return
    rng = workloads._rng(11)
    lead = (a.batch,) if a.batch > 1 else ()
    L = workloads.normal(rng, lead + (a.M, a.K)).cuda()
    R = workloads.normal(rng, lead + ((a.K, a.N) if a.r_layout == "kn" else (a.N, a.K)), 0.02).cuda()
    Lop = qm.operand_of(L, -1)
    Rop = qm.operand_of(R, -2 if a.r_layout == "kn" else -1)
    if a.stage == "probe":
        plan = qm.ProbePlan(Lop, Rop, a.fmt, a.fmt, a.gran, a.gran)
        for _ in range(a.iters):
            plan.launch(Lop, Rop)
        torch.cuda.synchronize()
        r = plan.result()
        print("mean_be", r.derived()["mean_be"], "device_error", r.device_error)
    elif a.stage == "gemm":
        # the stand-alone products: 8-bit codes of both operands, then qm_gemm and qm_gemm_ref
        Rk = R.transpose(-1, -2).contiguous() if a.r_layout == "kn" else R
        Rk_op = qm.operand_of(Rk, -1)
        cl, dl, _, _ = qm.qm_quantize(Lop, a.fmt, a.gran)
        cr, dr, _, _ = qm.qm_quantize(Rk_op, a.fmt, a.gran)
        L3 = L if L.dim() == 3 else L[None]
        R3 = Rk if Rk.dim() == 3 else Rk[None]
        for _ in range(a.iters):
            out, _ = qm.qm_gemm(cl, a.fmt, dl, a.gran, cr, a.fmt, dr, a.gran, a.K)
            ref = qm.qm_gemm_ref(L3, R3)
        torch.cuda.synchronize()
        print("rel diff of the two products", float((out - ref).norm() / ref.norm()))
    elif a.stage == "stats":
        # the single-tensor passes on the left operand
        for _ in range(a.iters):
            st = qm.qm_tensor_stats(Lop)
            er = qm.qm_quantize_error(Lop, a.fmt, a.gran)
        print("kurtosis", st.derived()["kurtosis"], "mean RE", er.sum_re / max(er.n_nonzero, 1))
    else:
        for _ in range(a.iters):
            qm.qm_quantize(Lop, a.fmt, a.gran, None, want_abs=True)
            qm.qm_quantize(Rop, a.fmt, a.gran, None, want_abs=True, want_kmaj=(a.r_layout == "kn"))
        torch.cuda.synchronize()
        print("done")


if __name__ == "__main__":
    main()
