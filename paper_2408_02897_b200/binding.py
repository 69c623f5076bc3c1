"""ctypes binding of include/qm.h.  Argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams); an operand of a
product L.R is described by `operand_of(tensor, contract_dim)`.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libqm.so")

FMT = {"int8": 0, "e4m3": 1, "e5m2": 2}
GRAN = {"tensor": 0, "channel": 1}
REF = {"bf16": 0, "fp32": 1}
_DT = {torch.float32: 0, torch.bfloat16: 1}


class QmError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(what)


class Operand(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("noncontract", C.c_int64),
                ("contract", C.c_int64), ("stride_nc", C.c_int64), ("stride_c", C.c_int64),
                ("batch", C.c_int64), ("stride_batch", C.c_int64)]


class MetricResult(C.Structure):
    _fields_ = [("sum_be", C.c_double), ("max_be", C.c_double), ("sum_diff2", C.c_double),
                ("sum_ref2", C.c_double), ("sum_den2", C.c_double), ("count", C.c_uint64),
                ("device_error", C.c_uint32), ("reserved", C.c_uint32)]

    def record(self):
        return {k: getattr(self, k) for k in ("sum_be", "max_be", "sum_diff2", "sum_ref2", "sum_den2", "count")}

    def derived(self):
        """mean BE, max BE, norm-wise BE, relative L2, SNR [dB] of the record (qm_metric_scalars)."""
        out = MetricScalars()
        _check(lib().qm_metric_scalars(C.byref(self), C.byref(out)), "qm_metric_scalars")
        return {k: getattr(out, k) for k, _ in out._fields_}


class MetricScalars(C.Structure):
    _fields_ = [("mean_be", C.c_double), ("max_be", C.c_double), ("normwise_be", C.c_double),
                ("rel_l2", C.c_double), ("snr_db", C.c_double)]


class TensorMoments(C.Structure):
    _fields_ = [("mean", C.c_double), ("variance", C.c_double), ("skew", C.c_double), ("kurtosis", C.c_double)]


class TensorStats(C.Structure):
    _fields_ = [("sum1", C.c_double), ("sum2", C.c_double), ("sum3", C.c_double), ("sum4", C.c_double),
                ("max_abs", C.c_double), ("count", C.c_uint64), ("device_error", C.c_uint32),
                ("reserved", C.c_uint32)]

    def derived(self):
        """mean, variance, skew, kurtosis of the tensor (qm_tensor_moments)."""
        out = TensorMoments()
        _check(lib().qm_tensor_moments(C.byref(self), C.byref(out)), "qm_tensor_moments")
        return {k: getattr(out, k) for k, _ in out._fields_}


class QuantError(C.Structure):
    _fields_ = [("sum_re", C.c_double), ("sum_re_round", C.c_double), ("max_re_round", C.c_double),
                ("err2_round", C.c_double), ("err2_overflow", C.c_double), ("err2_underflow", C.c_double),
                ("sum_x2", C.c_double), ("count", C.c_uint64), ("n_nonzero", C.c_uint64),
                ("n_overflow", C.c_uint64), ("n_underflow", C.c_uint64), ("device_error", C.c_uint32),
                ("reserved", C.c_uint32)]

    def record(self):
        return {k: getattr(self, k) for k, _ in self._fields_ if k not in ("device_error", "reserved")}


class ProbeCfg(C.Structure):
    _fields_ = [("fmt_l", C.c_int32), ("fmt_r", C.c_int32), ("gran_l", C.c_int32), ("gran_r", C.c_int32),
                ("round", C.c_int32), ("ref", C.c_int32), ("seed", C.c_uint64),
                ("batch_groups_l", C.c_int32), ("batch_groups_r", C.c_int32), ("row_stats", C.c_void_p)]


_lib = None


def lib():
    """The loaded library.  Raises if it is missing: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise QmError(-1, f"{_LIB_PATH} not built; run: python -m paper_2408_02897_b200.build")
        L = C.CDLL(_LIB_PATH)
        P, I32, I64, SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        OP = C.POINTER(Operand)
        sig = {
            "qm_code_ld": (I64, [I64]),
            "qm_scale": (I32, [OP, I32, I32, P, P]),
            "qm_scale_shared": (I32, [OP, I32, I32, P, P]),
            "qm_quantize": (I32, [OP, I32, I32, I32, P, P, P, P, P, P]),
            "qm_quantize_stochastic": (I32, [OP, I32, I32, C.c_uint64, C.c_uint32, P, P, P, P, P, P]),
            "qm_quantize_formats": (I32, [OP, I32, C.POINTER(I32), I32, C.POINTER(P), C.POINTER(P), P, P, P]),
            "qm_gemm": (I32, [P, I32, P, I32, P, I32, P, I32, I64, I64, I64, I64, P, P, I32, P]),
            "qm_gemm_ref": (I32, [P, P, I64, I64, I64, I64, P, P]),
            "qm_metric_workspace_bytes": (SZ, [I64]),
            "qm_metric": (I32, [P, P, P, I64, P, P, SZ, P]),
            "qm_metric_scalars": (I32, [C.POINTER(MetricResult), C.POINTER(MetricScalars)]),
            "qm_tensor_moments": (I32, [C.POINTER(TensorStats), C.POINTER(TensorMoments)]),
            "qm_workspace_bytes": (SZ, [OP, OP, C.POINTER(ProbeCfg)]),
            "qm_probe_layer": (I32, [OP, OP, C.POINTER(ProbeCfg), P, P, SZ, P]),
            "qm_workspace_bytes2": (SZ, [OP, OP, C.POINTER(ProbeCfg), C.POINTER(ProbeCfg)]),
            "qm_probe_layer2": (I32, [OP, OP, C.POINTER(ProbeCfg), C.POINTER(ProbeCfg), P, P, SZ, P]),
            "qm_operand_span_bytes": (SZ, [OP]),
            "qm_probe_layer_host": (I32, [OP, OP, C.POINTER(ProbeCfg), P, P, C.POINTER(MetricResult), P, P, SZ, P]),
            "qm_stats_workspace_bytes": (SZ, []),
            "qm_tensor_stats": (I32, [OP, P, P, SZ, P]),
            "qm_quantize_error": (I32, [OP, I32, I32, P, P, P, SZ, P]),
            "qm_probe_batch": (I32, [I32, OP, OP, C.POINTER(ProbeCfg), P, C.POINTER(P), C.POINTER(SZ), P]),
            "qm_probe_batch_host": (I32, [I32, OP, OP, C.POINTER(ProbeCfg), C.POINTER(P), C.POINTER(P),
                                          C.POINTER(MetricResult), P, C.POINTER(P), C.POINTER(SZ), P]),
            "qm_probe_batch_host_bytes": (I32, [I32, OP, OP, C.POINTER(SZ), C.POINTER(SZ)]),
            "qm_status_string": (C.c_char_p, [I32]),
            "qm_version": (I32, []),
            "qm_last_cuda_error": (C.c_char_p, []),
            "qm_metric_noalloc": (I32, [P, P, P, I64, P, P]),
            "qm_metric_noalloc_max_count": (I64, []),
            "qm_kernel_launches": (I64, []),
            "qm_debug_read_pass": (I32, [P, SZ, I32, I32, P, P]),
            "qm_debug_set_wait_limit_ns": (None, [C.c_uint64]),
            "qm_debug_stop_producer_after": (None, [C.c_uint32]),
            "qm_profile_enable": (I32, [I32]),
            "qm_profile_read": (I32, [C.POINTER(C.c_double), C.POINTER(I32)]),
            "qm_profile_samples": (I32, [C.POINTER(C.c_double), C.POINTER(C.c_double), I32, C.POINTER(I32)]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(st, what):
    if st != 0:
        L = lib()
        msg = L.qm_status_string(st).decode()
        if st == 6:
            msg += " (" + L.qm_last_cuda_error().decode() + ")"
        raise QmError(st, f"{what}: {msg}")


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def qm_code_ld(contract):
    return (contract + 15) // 16 * 16


def operand_of(t, contract_dim):
    """Describes a 2-D [.., .] or batched 3-D [b, ., .] tensor as an operand whose contracting
    dimension is `contract_dim` (-1 or -2).  No data is touched."""
    if t.dim() not in (2, 3) or t.dtype not in _DT:
        raise QmError(1, "operand must be a 2-D or 3-D float32/bfloat16 tensor")
    cd = contract_dim % t.dim()
    nd = t.dim() - 1 if cd == t.dim() - 2 else t.dim() - 2
    if cd == nd or cd < t.dim() - 2:
        raise QmError(1, "contract_dim must be one of the last two dimensions")
    o = Operand()
    o.data = t.data_ptr(); o.dtype = _DT[t.dtype]
    o.noncontract = t.shape[nd]; o.contract = t.shape[cd]
    o.stride_nc = t.stride(nd); o.stride_c = t.stride(cd)
    o.batch = t.shape[0] if t.dim() == 3 else 1
    o.stride_batch = t.stride(0) if t.dim() == 3 else 0
    o._keep = t
    return o


def _n_delta(op, gran):
    return 1 if GRAN[gran] == 0 else op.batch * op.noncontract


def qm_scale(op, fmt, gran, stream=None):
    """Eq. 1 scales of an operand -> float32 CUDA tensor (1 or batch*noncontract values)."""
    delta = torch.empty(_n_delta(op, gran), dtype=torch.float32, device="cuda")
    _check(lib().qm_scale(C.byref(op), FMT[fmt], GRAN[gran], _ptr(delta), _stream(stream)), "qm_scale")
    return delta


def qm_scale_shared(op, fmt, batch_groups, stream=None):
    """Per-channel Eq. 1 scales shared along the matmul batch (batch element b in group b % batch_groups)
    -> float32 CUDA tensor of batch*noncontract values, usable wherever "channel" scales are."""
    delta = torch.empty(op.batch * op.noncontract, dtype=torch.float32, device="cuda")
    _check(lib().qm_scale_shared(C.byref(op), FMT[fmt], batch_groups, _ptr(delta), _stream(stream)), "qm_scale_shared")
    return delta


def qm_quantize(op, fmt, gran, delta=None, want_abs=False, want_kmaj=False, stream=None, stochastic=None):
    """Codes of an operand.  delta=None fuses the scale step.  Returns (codes, delta, abs, kmaj).
    stochastic=(seed, stream_id) rounds stochastically (qm_quantize_stochastic) instead of RTNE."""
    ldc = qm_code_ld(op.contract)
    codes = torch.empty((op.batch, op.noncontract, ldc), dtype=torch.uint8, device="cuda")
    shape = (op.batch, op.noncontract, op.contract)
    ab = torch.empty(shape, dtype=torch.bfloat16, device="cuda") if want_abs else None
    km = torch.empty(shape, dtype=torch.bfloat16, device="cuda") if want_kmaj else None
    dout = None
    if delta is None:
        dout = torch.empty(_n_delta(op, gran), dtype=torch.float32, device="cuda")
    if stochastic is not None:
        _check(lib().qm_quantize_stochastic(C.byref(op), FMT[fmt], GRAN[gran], stochastic[0], stochastic[1],
                                            _ptr(delta), _ptr(dout), _ptr(codes), _ptr(ab), _ptr(km),
                                            _stream(stream)), "qm_quantize_stochastic")
    else:
        _check(lib().qm_quantize(C.byref(op), FMT[fmt], GRAN[gran], 0, _ptr(delta), _ptr(dout), _ptr(codes),
                                 _ptr(ab), _ptr(km), _stream(stream)), "qm_quantize")
    return codes, (delta if delta is not None else dout), ab, km


def qm_quantize_formats(op, fmts, gran, want_kmaj=False, stream=None):
    """Codes of several formats of one operand from one pass (qm_quantize_formats).
    Returns ([codes per format], [delta per format], kmaj or None)."""
    n = len(fmts)
    ldc = qm_code_ld(op.contract)
    codes = [torch.empty((op.batch, op.noncontract, ldc), dtype=torch.uint8, device="cuda") for _ in fmts]
    deltas = [torch.empty(_n_delta(op, gran), dtype=torch.float32, device="cuda") for _ in fmts]
    km = torch.empty((op.batch, op.noncontract, op.contract), dtype=torch.bfloat16, device="cuda") if want_kmaj else None
    scratch = torch.empty(_n_delta(op, gran), dtype=torch.int32, device="cuda")
    _check(lib().qm_quantize_formats(C.byref(op), n, (C.c_int32 * n)(*[FMT[f] for f in fmts]), GRAN[gran],
                                     (C.c_void_p * n)(*[t.data_ptr() for t in deltas]),
                                     (C.c_void_p * n)(*[t.data_ptr() for t in codes]), _ptr(km), _ptr(scratch),
                                     _stream(stream)), "qm_quantize_formats")
    return codes, deltas, km


def qm_gemm(codes_l, fmt_l, delta_l, gran_l, codes_r, fmt_r, delta_r, gran_r, K, want_raw=False,
            use_simt=False, stream=None):
    """Descaled 8-bit product from codes [b, M, ldc] x [b, N, ldc] -> (fp32 [b, M, N], raw or None)."""
    b, M, _ = codes_l.shape
    N = codes_r.shape[1]
    out = torch.empty((b, M, N), dtype=torch.float32, device="cuda")
    raw = None
    if want_raw:
        raw = torch.empty((b, M, N), dtype=torch.int32 if fmt_l == "int8" else torch.float32, device="cuda")
    _check(lib().qm_gemm(_ptr(codes_l), FMT[fmt_l], _ptr(delta_l), GRAN[gran_l], _ptr(codes_r), FMT[fmt_r],
                         _ptr(delta_r), GRAN[gran_r], M, N, K, b, _ptr(out), _ptr(raw), int(use_simt),
                         _stream(stream)), "qm_gemm")
    return out, raw


def qm_gemm_ref(l, r, stream=None):
    """out = l . r^T for dense bf16 [b, M, K] and [b, N, K] -> fp32 [b, M, N]."""
    b, M, K = l.shape
    N = r.shape[1]
    assert l.is_contiguous() and r.is_contiguous() and l.dtype == torch.bfloat16 and r.dtype == torch.bfloat16
    out = torch.empty((b, M, N), dtype=torch.float32, device="cuda")
    _check(lib().qm_gemm_ref(_ptr(l), _ptr(r), M, N, K, b, _ptr(out), _stream(stream)), "qm_gemm_ref")
    return out


def _read_result(dev_buf):
    host = dev_buf.cpu().numpy().tobytes()
    return MetricResult.from_buffer_copy(host)


def qm_metric(ref, q, den, stream=None):
    """Eq. 3 record of three fp32 arrays of equal size."""
    n = ref.numel()
    L = lib()
    ws_bytes = L.qm_metric_workspace_bytes(n)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    out = torch.empty(C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")
    _check(L.qm_metric(_ptr(ref), _ptr(q), _ptr(den), n, _ptr(out), _ptr(ws), ws_bytes, _stream(stream)), "qm_metric")
    return _read_result(out)


def qm_metric_noalloc(ref, q, den, out=None, stream=None):
    """Eq. 3 record through the entry point that keeps its scratch inside the library, for
    callers that cannot allocate device memory.  `out` is a caller-owned CUDA byte tensor of
    sizeof(qm_metric_result) bytes; one is made here only when none is passed."""
    if out is None:
        out = torch.empty(C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")
    _check(lib().qm_metric_noalloc(_ptr(ref), _ptr(q), _ptr(den), ref.numel(), _ptr(out), _stream(stream)),
           "qm_metric_noalloc")
    return _read_result(out)


def _stats_ws():
    n = lib().qm_stats_workspace_bytes()
    return torch.empty(n, dtype=torch.uint8, device="cuda"), n


def qm_tensor_stats(op, ws=None, stream=None):
    """Power sums and max|x| of a tensor -> TensorStats (synchronises to read the record)."""
    ws, n = (ws, ws.numel()) if ws is not None else _stats_ws()
    out = torch.empty(C.sizeof(TensorStats), dtype=torch.uint8, device="cuda")
    _check(lib().qm_tensor_stats(C.byref(op), _ptr(out), _ptr(ws), n, _stream(stream)), "qm_tensor_stats")
    return TensorStats.from_buffer_copy(out.cpu().numpy().tobytes())


def qm_quantize_error(op, fmt, gran, delta=None, ws=None, stream=None):
    """Eq. 2 sums and the clipping / rounding split of an operand -> QuantError.  delta=None
    takes the Eq. 1 scales of the operand itself (qm_scale)."""
    if delta is None:
        delta = qm_scale(op, fmt, gran, stream)
    ws, n = (ws, ws.numel()) if ws is not None else _stats_ws()
    out = torch.empty(C.sizeof(QuantError), dtype=torch.uint8, device="cuda")
    _check(lib().qm_quantize_error(C.byref(op), FMT[fmt], GRAN[gran], _ptr(delta), _ptr(out), _ptr(ws), n,
                                   _stream(stream)), "qm_quantize_error")
    return QuantError.from_buffer_copy(out.cpu().numpy().tobytes())


ROUND = {"rtne": 0, "stochastic_l": 1, "stochastic_r": 2, "stochastic_both": 3}


def _cfg(fmt_l, fmt_r, gran_l, gran_r, ref, rounding="rtne", seed=0, groups=(0, 0), row_stats=None):
    c = ProbeCfg()
    c.row_stats = row_stats.data_ptr() if row_stats is not None else None
    c.batch_groups_l, c.batch_groups_r = groups
    c.fmt_l, c.fmt_r, c.gran_l, c.gran_r, c.ref = FMT[fmt_l], FMT[fmt_r], GRAN[gran_l], GRAN[gran_r], REF[ref]
    c.round, c.seed = ROUND[rounding], seed
    return c


def qm_workspace_bytes(L_op, R_op, fmt_l, fmt_r, gran_l, gran_r, ref="bf16"):
    c = _cfg(fmt_l, fmt_r, gran_l, gran_r, ref)
    n = lib().qm_workspace_bytes(C.byref(L_op), C.byref(R_op), C.byref(c))
    if n == 0:
        raise QmError(1, "qm_workspace_bytes: configuration rejected")
    return n


def _row_stats_buffer(L_op):
    return torch.empty((L_op.batch * L_op.noncontract, 5), dtype=torch.float64, device="cuda")


class ProbePlan:
    """Pre-allocated workspace and result buffer for repeated probes of one shape."""

    def __init__(self, L_op, R_op, fmt_l, fmt_r, gran_l, gran_r, ref="bf16", rounding="rtne", seed=0,
                 groups=(0, 0), row_stats=False):
        # row_stats: also collect the per-row Eq. 3 sums [batch * M, 5] (check output of the fused kernel)
        self.row_stats = _row_stats_buffer(L_op) if row_stats else None
        self.cfg = _cfg(fmt_l, fmt_r, gran_l, gran_r, ref, rounding, seed, groups, self.row_stats)
        self.ws_bytes = qm_workspace_bytes(L_op, R_op, fmt_l, fmt_r, gran_l, gran_r, ref)
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")
        self.out = torch.zeros(C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")

    def launch(self, L_op, R_op, stream=None):
        _check(lib().qm_probe_layer(C.byref(L_op), C.byref(R_op), C.byref(self.cfg), _ptr(self.out),
                                    _ptr(self.ws), self.ws_bytes, _stream(stream)), "qm_probe_layer")

    def result(self):
        return _read_result(self.out)


class ProbePlan2:
    """Workspace and the two result records of a two-format probe (qm_probe_layer2).
    fmts_a / fmts_b are (fmt_l, fmt_r) of the two configurations; everything else is shared."""

    def __init__(self, L_op, R_op, fmts_a, fmts_b, gran_l, gran_r, rounding="rtne", seed=0, groups=(0, 0)):
        self.cfg_a = _cfg(fmts_a[0], fmts_a[1], gran_l, gran_r, "bf16", rounding, seed, groups)
        self.cfg_b = _cfg(fmts_b[0], fmts_b[1], gran_l, gran_r, "bf16", rounding, seed, groups)
        self.ws_bytes = lib().qm_workspace_bytes2(C.byref(L_op), C.byref(R_op), C.byref(self.cfg_a), C.byref(self.cfg_b))
        if self.ws_bytes == 0:
            raise QmError(2, "qm_workspace_bytes2: the two configurations cannot share a pass")
        self.ws = torch.empty(self.ws_bytes, dtype=torch.uint8, device="cuda")
        self.out = torch.zeros(2 * C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")

    def launch(self, L_op, R_op, stream=None):
        _check(lib().qm_probe_layer2(C.byref(L_op), C.byref(R_op), C.byref(self.cfg_a), C.byref(self.cfg_b),
                                     _ptr(self.out), _ptr(self.ws), self.ws_bytes, _stream(stream)), "qm_probe_layer2")

    def results(self):
        return _records(self.out.cpu().numpy().tobytes(), 2)


def qm_probe_layer2(L_op, R_op, fmts_a, fmts_b, gran_l, gran_r, stream=None, rounding="rtne", seed=0, groups=(0, 0)):
    """Both formats' records of one product from a single pass; returns [MetricResult, MetricResult]."""
    plan = ProbePlan2(L_op, R_op, fmts_a, fmts_b, gran_l, gran_r, rounding, seed, groups)
    plan.launch(L_op, R_op, stream)
    return plan.results()


def qm_probe_layer(L_op, R_op, fmt_l, fmt_r, gran_l, gran_r, ref="bf16", stream=None, rounding="rtne", seed=0,
                   groups=(0, 0)):
    """The whole probe for one product; returns the MetricResult (synchronises to read it).
    rounding: "rtne", or "stochastic_l" / "stochastic_r" / "stochastic_both" with `seed`.
    groups: batch_groups of (L, R) for channel scales shared along the batch (0 = not shared)."""
    plan = ProbePlan(L_op, R_op, fmt_l, fmt_r, gran_l, gran_r, ref, rounding, seed, groups)
    plan.launch(L_op, R_op, stream)
    return plan.result()


def qm_probe_layer_host(L_host, R_host, contract_l, contract_r, fmt_l, fmt_r, gran_l, gran_r, ref="bf16",
                        stage=None, stream=None):
    """Probe of operands held in (pinned) host tensors; copies are part of the call.
    `stage` may carry (l_stage, r_stage, plan) from an earlier call to avoid re-allocation."""
    Lh, Rh = operand_of(L_host, contract_l), operand_of(R_host, contract_r)
    if stage is None:
        l_stage = torch.empty(L_host.numel() if L_host.is_contiguous() else lib().qm_operand_span_bytes(C.byref(Lh)),
                              dtype=L_host.dtype if L_host.is_contiguous() else torch.uint8, device="cuda")
        r_stage = torch.empty(R_host.numel() if R_host.is_contiguous() else lib().qm_operand_span_bytes(C.byref(Rh)),
                              dtype=R_host.dtype if R_host.is_contiguous() else torch.uint8, device="cuda")
        Ld, Rd = Operand(), Operand()
        C.memmove(C.byref(Ld), C.byref(Lh), C.sizeof(Operand)); C.memmove(C.byref(Rd), C.byref(Rh), C.sizeof(Operand))
        Ld.data, Rd.data = l_stage.data_ptr(), r_stage.data_ptr()
        plan = ProbePlan(Ld, Rd, fmt_l, fmt_r, gran_l, gran_r, ref)
        stage = (l_stage, r_stage, plan)
    l_stage, r_stage, plan = stage
    res = MetricResult()
    st = lib().qm_probe_layer_host(C.byref(Lh), C.byref(Rh), C.byref(plan.cfg), _ptr(l_stage), _ptr(r_stage),
                                   C.byref(res), _ptr(plan.out), _ptr(plan.ws), plan.ws_bytes, _stream(stream))
    _check(st, "qm_probe_layer_host")
    return res, stage


def _copy_operand(op, data_ptr=None):
    o = Operand()
    C.memmove(C.byref(o), C.byref(op), C.sizeof(Operand))
    if data_ptr is not None:
        o.data = data_ptr
    return o


def _records(raw, n):
    sz = C.sizeof(MetricResult)
    return [MetricResult.from_buffer_copy(raw[i * sz:(i + 1) * sz]) for i in range(n)]


class ProbeBatch:
    """Workspaces and result records of a fixed list of probes that are issued together
    (qm_probe_batch).  `probes` is a list of (L_op, R_op, fmt_l, fmt_r, gran_l, gran_r[, ref])."""

    def __init__(self, probes, row_stats=False):
        n = self.n = len(probes)
        self._keep = [(p[0], p[1]) for p in probes]
        self.L = (Operand * n)(*[_copy_operand(p[0]) for p in probes])
        self.R = (Operand * n)(*[_copy_operand(p[1]) for p in probes])
        refs = [p[6] if len(p) > 6 else "bf16" for p in probes]
        # row_stats: per probe, also collect the per-row Eq. 3 sums (check output of the fused kernel)
        self.row_stats = [_row_stats_buffer(p[0]) if row_stats and r == "bf16" else None for p, r in zip(probes, refs)]
        self.cfg = (ProbeCfg * n)(*[_cfg(p[2], p[3], p[4], p[5], r, row_stats=rs)
                                    for p, r, rs in zip(probes, refs, self.row_stats)])
        sizes = [qm_workspace_bytes(p[0], p[1], p[2], p[3], p[4], p[5], r) for p, r in zip(probes, refs)]
        self._ws = [torch.empty(b, dtype=torch.uint8, device="cuda") for b in sizes]
        self.ws = (C.c_void_p * n)(*[t.data_ptr() for t in self._ws])
        self.ws_bytes = (C.c_size_t * n)(*sizes)
        self.out = torch.zeros(n * C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")

    def launch(self, stream=None):
        _check(lib().qm_probe_batch(self.n, self.L, self.R, self.cfg, _ptr(self.out), self.ws, self.ws_bytes,
                                    _stream(stream)), "qm_probe_batch")

    def launch_serial(self, stream=None):
        """The same probes one after the other on one stream (qm_probe_layer per probe)."""
        sz = C.sizeof(MetricResult)
        for i in range(self.n):
            _check(lib().qm_probe_layer(C.byref(self.L[i]), C.byref(self.R[i]), C.byref(self.cfg[i]),
                                        C.c_void_p(self.out.data_ptr() + i * sz), self.ws[i], self.ws_bytes[i],
                                        _stream(stream)), "qm_probe_layer")

    def results(self):
        return _records(self.out.cpu().numpy().tobytes(), self.n)


class HostProbeBatch:
    """The same for operands in (pinned) host tensors (qm_probe_batch_host): device staging
    buffers, workspaces and records are made once; run() copies, probes and returns the records.
    `probes` is a list of (L_host, contract_l, R_host, contract_r, fmt_l, fmt_r, gran_l, gran_r[, ref])."""

    def __init__(self, probes):
        n = self.n = len(probes)
        Lh = [operand_of(p[0], p[1]) for p in probes]
        Rh = [operand_of(p[2], p[3]) for p in probes]
        self._keep = (Lh, Rh)
        span = lib().qm_operand_span_bytes
        self._ls = [torch.empty(span(C.byref(o)), dtype=torch.uint8, device="cuda") for o in Lh]
        self._rs = [torch.empty(span(C.byref(o)), dtype=torch.uint8, device="cuda") for o in Rh]
        self.L = (Operand * n)(*[_copy_operand(o) for o in Lh])
        self.R = (Operand * n)(*[_copy_operand(o) for o in Rh])
        self.l_stage = (C.c_void_p * n)(*[t.data_ptr() for t in self._ls])
        self.r_stage = (C.c_void_p * n)(*[t.data_ptr() for t in self._rs])
        refs = [p[8] if len(p) > 8 else "bf16" for p in probes]
        self.cfg = (ProbeCfg * n)(*[_cfg(p[4], p[5], p[6], p[7], r) for p, r in zip(probes, refs)])
        sizes = []
        for i, (p, r) in enumerate(zip(probes, refs)):
            Ld, Rd = _copy_operand(Lh[i], self._ls[i].data_ptr()), _copy_operand(Rh[i], self._rs[i].data_ptr())
            sizes.append(qm_workspace_bytes(Ld, Rd, p[4], p[5], p[6], p[7], r))
        self._ws = [torch.empty(b, dtype=torch.uint8, device="cuda") for b in sizes]
        self.ws = (C.c_void_p * n)(*[t.data_ptr() for t in self._ws])
        self.ws_bytes = (C.c_size_t * n)(*sizes)
        self.out_dev = torch.zeros(n * C.sizeof(MetricResult), dtype=torch.uint8, device="cuda")
        self._out_host = torch.zeros(n * C.sizeof(MetricResult), dtype=torch.uint8).pin_memory()
        h2d, d2h = C.c_size_t(0), C.c_size_t(0)
        _check(lib().qm_probe_batch_host_bytes(n, self.L, self.R, C.byref(h2d), C.byref(d2h)), "qm_probe_batch_host_bytes")
        self.h2d_bytes, self.d2h_bytes = h2d.value, d2h.value      # what one run() copies

    def run(self, stream=None):
        out = C.cast(C.c_void_p(self._out_host.data_ptr()), C.POINTER(MetricResult))
        _check(lib().qm_probe_batch_host(self.n, self.L, self.R, self.cfg, self.l_stage, self.r_stage, out,
                                         _ptr(self.out_dev), self.ws, self.ws_bytes, _stream(stream)),
               "qm_probe_batch_host")
        return _records(self._out_host.numpy().tobytes(), self.n)


def kernel_launches():
    """Kernels launched by the library in this process so far."""
    return lib().qm_kernel_launches()


def profile_enable(on=True):
    _check(lib().qm_profile_enable(1 if on else 0), "qm_profile_enable")


def profile_samples(cap=4096):
    """[(start_ms, duration_ms)] of the fused probe launches recorded since profiling was enabled or
    last read, starts relative to the first one; does not end the interval."""
    st, du, n = (C.c_double * cap)(), (C.c_double * cap)(), C.c_int32(0)
    _check(lib().qm_profile_samples(st, du, cap, C.byref(n)), "qm_profile_samples")
    return [(st[i], du[i]) for i in range(min(n.value, cap))]


def profile_read():
    """(summed milliseconds, launches) of the fused tensor-core probe kernel since the last read."""
    ms, n = C.c_double(0), C.c_int32(0)
    _check(lib().qm_profile_read(C.byref(ms), C.byref(n)), "qm_profile_read")
    return ms.value, n.value
