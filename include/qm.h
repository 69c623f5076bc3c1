/*
 * qm.h - C ABI of the quantized-matmul error probe for NVIDIA B200 (sm_100a).
 *
 * The probe measures, for one matrix product L.R of a network, how much error
 * an 8-bit format would introduce.  Following the paper's Methodology section
 * it (1) computes the dynamic symmetric absmax scale of each operand (Eq. 1),
 * (2) quantizes each operand to INT8, FP8 E4M3 or FP8 E5M2 with
 * round-to-nearest-even and saturation (Eq. 1 and the saturation rule),
 * (3) multiplies the 8-bit operands on the tensor cores with a wide
 * accumulator and descales the result, (4) multiplies the unquantized
 * operands in high precision, and (5) reduces the two results into the
 * inner-product-level backward error of Eq. 3,
 *        BE_ij = |(L.R)_ij - Q(L,R)_ij| / (|L|.|R|)_ij ,
 * together with the sums needed for relative L2 error and SNR.
 *
 * Conventions that hold for every entry point
 *  - All data pointers are DEVICE memory owned by the caller unless a
 *    parameter says "host".  The library allocates no device memory.
 *  - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it and
 *    the call returns without waiting; results are valid once the caller has
 *    synchronised the stream (the *_host entry point is the one exception).
 *  - Argument errors are found on the host before anything is launched and
 *    come back as a qm_status.  Nothing throws, prints, traps or exits.
 *  - Conditions only the device can see (a NaN/Inf operand, a bounded wait
 *    that ran out) set bits in qm_metric_result.device_error; the numbers in
 *    that record are then meaningless.
 *  - An operand is a (batched) 2-D view named by its NON-CONTRACTING and
 *    CONTRACTING extents.  For L [M x K] of L.R these are M and K; for R
 *    [K x N] they are N and K.  One of the two strides must be 1; the other
 *    and the batch stride must be multiples of 8 elements.
 *  - Codes are bytes: INT8 two's complement in -127..127, FP8 bit patterns.
 *    A code tensor is [batch][noncontract][ldc] with the contracting index
 *    contiguous and ldc = qm_code_ld(contract) (rows padded to 16 bytes,
 *    padding bytes are zero).
 */
#ifndef QM_H_
#define QM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  QM_OK = 0,
  QM_ERR_INVALID_ARG = 1,        /* null pointer, non-positive extent, bad enum           */
  QM_ERR_UNSUPPORTED = 2,        /* valid request this build has no kernel for            */
  QM_ERR_ALIGNMENT = 3,          /* pointer or stride breaks a stated alignment rule      */
  QM_ERR_WORKSPACE_TOO_SMALL = 4,
  QM_ERR_NONFINITE_INPUT = 5,    /* reported by the *_host entry point only               */
  QM_ERR_CUDA = 6,               /* a CUDA runtime/driver call failed                     */
  QM_ERR_TIMEOUT = 7             /* reported by the *_host entry point only               */
} qm_status;

typedef enum { QM_FMT_INT8 = 0, QM_FMT_E4M3 = 1, QM_FMT_E5M2 = 2 } qm_format;
typedef enum { QM_DT_F32 = 0, QM_DT_BF16 = 1 } qm_dtype;
/* Scale granularity (Methodology, 4th bullet): one number for the whole tensor,
 * or one per index of the non-contracting dimension (and per batch element). */
typedef enum { QM_GRAN_TENSOR = 0, QM_GRAN_CHANNEL = 1 } qm_gran;
/* Rounding function of Eq. 1 (Methodology, 2nd bullet: round-to-nearest-even and stochastic
 * rounding).  In qm_probe_cfg.round the two STOCHASTIC flags may be OR-ed: the paper rounds
 * only the gradient operand stochastically, and which side that is depends on the product. */
typedef enum { QM_ROUND_RTNE = 0, QM_ROUND_STOCHASTIC_L = 1, QM_ROUND_STOCHASTIC_R = 2 } qm_round;
/* How the high-precision side of Eq. 3 is evaluated:
 *  BF16_FP32ACC: bf16 operands on the tensor cores, fp32 accumulation (every
 *                bf16 x bf16 product is exact in fp32);
 *  FP32:         fp32 multiply-add on the CUDA cores (fp32 or bf16 operands). */
typedef enum { QM_REF_BF16_FP32ACC = 0, QM_REF_FP32 = 1 } qm_ref;

typedef struct {
  const void* data;        /* device; 16-byte aligned                                     */
  int32_t dtype;           /* qm_dtype                                                    */
  int64_t noncontract;     /* extent of the non-contracting dimension (M for L, N for R)  */
  int64_t contract;        /* extent of the contracting dimension (K)                     */
  int64_t stride_nc;       /* element stride between non-contracting indices              */
  int64_t stride_c;        /* element stride between contracting indices                  */
  int64_t batch;           /* matmul batch count, 1 for a plain product                   */
  int64_t stride_batch;    /* element stride between batch elements (ignored if batch==1) */
} qm_operand;

/* Bits of qm_metric_result.device_error */
#define QM_DEVERR_NONFINITE 1u   /* an operand held NaN or Inf                            */
#define QM_DEVERR_TIMEOUT   2u   /* a bounded device-side wait gave up                    */

/* The statistics record of Eq. 3 over all count = batch*M*N inner products.
 * mean BE = sum_be/count; norm-wise BE = sqrt(sum_diff2/sum_den2);
 * relative L2 = sqrt(sum_diff2/sum_ref2); SNR = 10 log10(sum_ref2/sum_diff2). */
typedef struct {
  double sum_be;           /* sum of BE_ij (BE_ij = 0 where the denominator is 0)         */
  double max_be;           /* max of BE_ij                                                */
  double sum_diff2;        /* sum (C_ij - Q_ij)^2                                         */
  double sum_ref2;         /* sum C_ij^2                                                  */
  double sum_den2;         /* sum D_ij^2, D = |L|.|R|                                     */
  uint64_t count;
  uint32_t device_error;   /* QM_DEVERR_* bits, 0 when the record is valid                */
  uint32_t reserved;
} qm_metric_result;

/* The scalars the probe reports, all from one statistics record (host arithmetic on a host
 * copy of the record): mean and max of the inner-product-level backward error of Eq. 3, its
 * norm-wise form sqrt(sum (C-Q)^2 / sum D^2), the relative L2 error sqrt(sum (C-Q)^2 / sum C^2)
 * and the signal-to-noise ratio 10 log10(sum C^2 / sum (C-Q)^2) in dB (+inf for an exact
 * product).  A ratio whose denominator sum is zero is reported as 0; count == 0 gives mean 0.
 * rec and out are HOST pointers. */
typedef struct { double mean_be, max_be, normwise_be, rel_l2, snr_db; } qm_metric_scalars_t;
qm_status qm_metric_scalars(const qm_metric_result* rec, qm_metric_scalars_t* out);

/* Power sums of all elements of one tensor (Experiments section: "mean, variance,
 * skew and Kurtosis" of the matmul inputs of the baseline).  With n = count,
 * mu = sum1/n and the raw moments r_k = sum_k/n:  variance m2 = r2 - mu^2,
 * m3 = r3 - 3 mu r2 + 2 mu^3,  m4 = r4 - 4 mu r3 + 6 mu^2 r2 - 3 mu^4,
 * skew = m3 / m2^1.5, kurtosis = m4 / m2^2 (3 for a normal law). */
typedef struct {
  double sum1, sum2, sum3, sum4;
  double max_abs;
  uint64_t count;
  uint32_t device_error;   /* QM_DEVERR_NONFINITE when a NaN or Inf was seen                */
  uint32_t reserved;
} qm_tensor_stats_result;

/* "mean, variance, skew and Kurtosis" (Experiments section) from the power sums of a record, by
 * the formulas above: population central moments, kurtosis as the plain fourth standardised
 * moment.  Evaluated in long double; an empty or constant tensor gives skew = kurtosis = 0.
 * rec and out are HOST pointers. */
typedef struct { double mean, variance, skew, kurtosis; } qm_tensor_moments_t;
qm_status qm_tensor_moments(const qm_tensor_stats_result* rec, qm_tensor_moments_t* out);

/* Eq. 2, RE = |v - v~| / |v|, over the non-zero elements of one tensor under Eq. 1,
 * split as in the Results section: an element is OVERFLOW when |v/delta| exceeds the
 * largest expressible magnitude (it is capped), UNDERFLOW when it is not zero but its
 * code is, ROUNDING otherwise.  err2_* are sums of (v - v~)^2 per class, each square formed
 * in fp32 (an error below about 1e-19 in magnitude contributes 0 to them). */
typedef struct {
  double sum_re;           /* over all non-zero elements (an underflow contributes 1)     */
  double sum_re_round;     /* over the rounding class                                     */
  double max_re_round;
  double err2_round, err2_overflow, err2_underflow;
  double sum_x2;
  uint64_t count, n_nonzero, n_overflow, n_underflow;
  uint32_t device_error;
  uint32_t reserved;
} qm_quant_error_result;

typedef struct {
  int32_t fmt_l, fmt_r;    /* qm_format per operand                                       */
  int32_t gran_l, gran_r;  /* qm_gran per operand                                         */
  int32_t round;           /* qm_round flags                                              */
  int32_t ref;             /* qm_ref                                                      */
  uint64_t seed;           /* of the stochastic draws; unused with QM_ROUND_RTNE          */
  int32_t batch_groups_l;  /* QM_GRAN_CHANNEL on a batched operand: see qm_scale_shared;  */
  int32_t batch_groups_r;  /* 0 = every batch element has its own scales                  */
  /* Optional (NULL = off) check output of the fused tensor-core probe: device fp64
   * [batch * M][QM_ROW_STATS] = for every output row the Eq. 3 sums over its N inner products,
   * {sum BE, max BE, sum (C-Q)^2, sum C^2, sum D^2}.  The call zeroes it and the kernel adds each
   * tile's share with atomics, so a CPU evaluation of a few sampled rows can be compared with
   * the fused kernel itself at sizes whose whole product the CPU cannot evaluate.  The record in
   * `out` is unchanged by it.  QM_REF_BF16_FP32ACC only; not with qm_probe_layer2. */
  double* row_stats;
} qm_probe_cfg;
#define QM_ROW_STATS 5

/* Row length in bytes of a code tensor whose contracting extent is `contract`. */
int64_t qm_code_ld(int64_t contract);

/*
 * Eq. 1 (right half) with the "align absmax to the largest expressible value"
 * rule: delta = max|X| / qmax, qmax = 127 / 448 / 57344, one IEEE fp32
 * division.  `delta` (device, fp32) receives 1 value for QM_GRAN_TENSOR (the
 * whole batched tensor shares it) or batch*noncontract values, batch-major,
 * for QM_GRAN_CHANNEL.  An all-zero group gets delta = 1.  A NaN/Inf input
 * makes the group's delta NaN/Inf.
 */
qm_status qm_scale(const qm_operand* x, int32_t fmt, int32_t gran, float* delta, void* stream);

/*
 * Per-channel scales shared along the matmul batch (the granularity levels of the
 * Results section).  Batch element b belongs to group b % batch_groups, and the
 * batch elements of a group share one scale per non-contracting index, taken
 * over all of them:  batch_groups = 1 is the paper's "channel" level (a scale
 * tensor over the non-batch, non-contracting dimension), batch_groups = number
 * of heads, for a batch laid out [examples][heads], is its "fine-grained" level
 * (batch dimensions included, except the axis of the individual examples), and
 * batch_groups = batch is QM_GRAN_CHANNEL of qm_scale.  batch_groups must divide
 * the batch.  `delta` receives batch * noncontract values, shared ones repeated,
 * so it can be handed to qm_quantize / qm_gemm with QM_GRAN_CHANNEL as it is.
 */
qm_status qm_scale_shared(const qm_operand* x, int32_t fmt, int32_t batch_groups, float* delta,
                          void* stream);

/*
 * Eq. 1 (left half) and the saturation rule: code = sat(RTNE(x / delta)), the
 * division in IEEE fp32, ties to the even code, magnitudes above qmax clamp to
 * +-qmax, magnitudes below half the smallest grid value become 0.
 *  delta      device fp32 scales as produced by qm_scale, or NULL: the call
 *             then computes them itself (scale and quantize fused) and stores
 *             them in delta_out, which is then REQUIRED (it is the scratch the
 *             scales live in).
 *  codes      device bytes, [batch][noncontract][qm_code_ld(contract)].
 *  abs_copy   optional (may be NULL) device bf16 [batch][noncontract][contract]:
 *             |x| rounded to bf16, contracting index contiguous (operand of the
 *             denominator product of Eq. 3).
 *  kmaj_copy  optional (may be NULL) device bf16, same shape: x itself with the
 *             contracting index contiguous (for operands stored the other way).
 */
qm_status qm_quantize(const qm_operand* x, int32_t fmt, int32_t gran, int32_t round,
                      const float* delta, float* delta_out, uint8_t* codes,
                      void* abs_copy, void* kmaj_copy, void* stream);

/*
 * Eq. 1 with stochastic rounding (Methodology, 2nd bullet).  t = x / delta as in
 * qm_quantize; with lo <= |t| <= hi the neighbouring expressible magnitudes (|t|
 * capped at the largest one first), the code is hi's with probability
 * (|t| - lo) / (hi - lo) and lo's otherwise, so the expectation is t; values on
 * the grid never move and the sign is kept.  The paper does not say where the
 * random numbers come from.  Here element number i of the operand (numbered
 * batch-major, then noncontract, then contract, whatever the strides) uses
 * u = (w >> 8) / 2^24 with w = word (i mod 4) of Philox4x32-10 (Salmon et al.,
 * SC'11) on counter (i div 4: low word, high word, stream_id, 0) and key
 * (seed: low word, high word); hi iff u (hi - lo) < |t| - lo.  The same
 * (seed, stream_id) therefore reproduces the same codes on any layout.
 * Other arguments as for qm_quantize (round is implied; qm_quantize itself
 * accepts QM_ROUND_RTNE only).
 */
qm_status qm_quantize_stochastic(const qm_operand* x, int32_t fmt, int32_t gran, uint64_t seed,
                                 uint32_t stream_id, const float* delta, float* delta_out,
                                 uint8_t* codes, void* abs_copy, void* kmaj_copy, void* stream);

/*
 * The codes of several formats of one operand (Eq. 1 once per format): the
 * measurement sweeps the 8-bit formats over the same tensors (Table 1), and
 * max|x| and the pass over the tensor do not depend on the format.  fmts holds
 * n_fmt (1..3) distinct formats; delta_out[k] (device, 1 value or one per batch
 * element and non-contracting index) and codes[k] (device, laid out as for
 * qm_quantize) receive format k's scales and codes, round-to-nearest-even;
 * kmaj_copy as for qm_quantize.  amax_scratch is device scratch of as many
 * 32-bit words as one delta_out array has values; the call clears it.  Every
 * result equals what qm_quantize gives for that format alone.  Per-tensor
 * scales of a bf16 operand are produced by one kernel that reads the operand
 * once; other cases by one quantize launch per format after a common max|x|.
 * A non-finite operand yields NaN scales, as in qm_scale.
 */
qm_status qm_quantize_formats(const qm_operand* x, int32_t n_fmt, const int32_t* fmts, int32_t gran,
                              float* const* delta_out, uint8_t* const* codes, void* kmaj_copy,
                              uint32_t* amax_scratch, void* stream);

/*
 * The 8-bit product and its descaling (Methodology, 3rd bullet):
 *   A = Lbar . Rbar^T accumulated in int32 (INT8, exact) or fp32 (FP8, any mix
 *   of E4M3 and E5M2), Q_ij = A_ij * delta_l[i] * delta_r[j].
 * codes_l [batch][M][qm_code_ld(K)], codes_r [batch][N][qm_code_ld(K)];
 * delta_l has 1 value (gran_l TENSOR) or batch*M, delta_r 1 or batch*N.
 * out_descaled (optional) fp32 [batch][M][N]; out_raw (optional) the raw
 * accumulator [batch][M][N]: int32 for INT8 x INT8, fp32 bit patterns for FP8.
 * Mixing INT8 with an FP8 format is QM_ERR_UNSUPPORTED.  use_simt != 0 selects
 * the CUDA-core kernel (any K; test cross-check); the tensor-core kernel needs
 * K to be a multiple of 16.
 */
qm_status qm_gemm(const uint8_t* codes_l, int32_t fmt_l, const float* delta_l, int32_t gran_l,
                  const uint8_t* codes_r, int32_t fmt_r, const float* delta_r, int32_t gran_r,
                  int64_t M, int64_t N, int64_t K, int64_t batch,
                  float* out_descaled, void* out_raw, int32_t use_simt, void* stream);

/*
 * The high-precision side of Eq. 3 on its own: out = l . r^T with bf16 operands
 * and fp32 accumulation on the tensor cores.  Passing L and R gives the
 * numerator product C = L.R; passing the |x| copies that qm_quantize writes
 * gives the denominator product D = |L|.|R|.  l [batch][M][K] and
 * r [batch][N][K], contracting index contiguous, dense.  out fp32
 * [batch][M][N].  K must be a multiple of 16.
 */
qm_status qm_gemm_ref(const void* l_bf16, const void* r_bf16, int64_t M, int64_t N, int64_t K,
                      int64_t batch, float* out, void* stream);

/*
 * Eq. 3 on materialised arrays: ref = C, q = Q, den = D, each `count` fp32
 * values.  `out` (device) receives the record.  `ws` is device scratch of at
 * least qm_metric_workspace_bytes(count) bytes, 8-byte aligned.
 */
size_t qm_metric_workspace_bytes(int64_t count);
qm_status qm_metric(const float* ref, const float* q, const float* den, int64_t count,
                    qm_metric_result* out, void* ws, size_t ws_bytes, void* stream);

/*
 * The whole probe for one product L.R: scale, quantize, the three products
 * (8-bit, reference, denominator) and the Eq. 3 reduction fused so that no
 * M x N matrix is written.  L: noncontract = M, contract = K.  R: noncontract
 * = N, contract = K, same batch.  `out` (device) receives the record; `ws` is
 * device scratch of at least qm_workspace_bytes(L, R, cfg) bytes, 256-byte
 * aligned; its contents on entry do not matter and concurrent calls must not
 * share it.
 * QM_REF_BF16_FP32ACC needs bf16 operands and K a multiple of 16;
 * QM_REF_FP32 takes fp32 or bf16 operands of any shape.
 * cfg->round: an operand flagged stochastic is quantized as by
 * qm_quantize_stochastic with cfg->seed and stream_id 0 (L) or 1 (R).
 */
size_t qm_workspace_bytes(const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg);
qm_status qm_probe_layer(const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg,
                         qm_metric_result* out, void* ws, size_t ws_bytes, void* stream);

/*
 * Two formats in one pass.  The paper sweeps the 8-bit formats over the same
 * tensors (Table 1): the reference product L.R and the denominator product
 * |L|.|R| do not depend on the format, so this call computes them once and keeps
 * one 8-bit accumulator per format beside them.  cfg_a and cfg_b must agree in
 * everything except fmt_l / fmt_r, use QM_REF_BF16_FP32ACC, and at most one of
 * them may be the INT8 format.  out[0] receives the record of cfg_a, out[1]
 * that of cfg_b; each equals what qm_probe_layer gives for that configuration.
 * `ws`: at least qm_workspace_bytes2(...) bytes, otherwise as for qm_probe_layer.
 */
size_t qm_workspace_bytes2(const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg_a,
                           const qm_probe_cfg* cfg_b);
qm_status qm_probe_layer2(const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg_a,
                          const qm_probe_cfg* cfg_b, qm_metric_result* out, void* ws, size_t ws_bytes,
                          void* stream);

/*
 * Same probe for operands that live in HOST memory (pinned memory makes the
 * copies asynchronous).  L->data and R->data are host pointers; l_stage and
 * r_stage are device buffers the caller owns, large enough for the operands'
 * storage span (qm_operand_span_bytes), 16-byte aligned.  The call copies the
 * operands to the device, runs the probe, copies the record back into
 * *out_host and WAITS for the stream.  Device-detected conditions are returned
 * as QM_ERR_NONFINITE_INPUT / QM_ERR_TIMEOUT.
 */
size_t qm_operand_span_bytes(const qm_operand* x);
qm_status qm_probe_layer_host(const qm_operand* L_host, const qm_operand* R_host,
                              const qm_probe_cfg* cfg, void* l_stage, void* r_stage,
                              qm_metric_result* out_host, qm_metric_result* out_dev,
                              void* ws, size_t ws_bytes, void* stream);

/*
 * Single-tensor passes beside the probe, one read of the tensor each.
 * qm_tensor_stats: the power sums from which mean, variance, skew and kurtosis of
 * the tensor follow (Experiments section), and max|x|.  Powers are formed in fp32
 * (|x| up to 2^31 keeps x^4 finite), summed in fp32 over 32 elements and in fp64
 * from there on.
 * qm_quantize_error: Eq. 2 and the clipping / rounding split of the Results
 * section for the codes qm_quantize would produce with these scales.  `delta`
 * (device) holds finished Eq. 1 scales as written by qm_scale or qm_quantize:
 * one value (QM_GRAN_TENSOR) or batch * noncontract values (QM_GRAN_CHANNEL).
 * `out` (device) receives the record.  `ws` is device scratch of at least
 * qm_stats_workspace_bytes() bytes, 256-byte aligned; its contents on entry do
 * not matter and concurrent calls must not share it.  The operand needs a unit
 * stride in one of its two dimensions and fewer than 2^32 groups of 8 elements.
 */
size_t qm_stats_workspace_bytes(void);
qm_status qm_tensor_stats(const qm_operand* x, qm_tensor_stats_result* out, void* ws, size_t ws_bytes,
                          void* stream);
qm_status qm_quantize_error(const qm_operand* x, int32_t fmt, int32_t gran, const float* delta,
                            qm_quant_error_result* out, void* ws, size_t ws_bytes, void* stream);

/*
 * The probes of one measurement pass (the per-layer loop of the Methodology
 * section: every matmul of a network is probed on its own), issued together.
 * Probe i computes what qm_probe_layer(&L[i], &R[i], &cfg[i], out + i, ws[i],
 * ws_bytes[i]) computes.  The probes are independent, so the library runs the
 * scale/quantize kernels of all operands beside one another on a few streams of
 * its own (created on the first call on each device, kept until the process
 * exits) and then the fused kernels of all tensor-core probes as one persistent
 * launches of up to 16 probes over the tiles of all of them (the sums of a
 * record are then taken over another tile-to-CTA assignment than in
 * qm_probe_layer and may differ in the last bits).  A measurement pass asks
 * for the same preparation many times over (a sweep of formats over one layer,
 * an activation that feeds several products, a gradient that appears in dgrad
 * and wgrad): inside a batch, operands that describe the same memory (same
 * address, extents and strides) under the same scale grouping are prepared
 * once.  Their max|x| is reduced once (for per-tensor scales also across the
 * two orientations of a tensor), the contraction-major copy is made once, the
 * codes of up to three formats come from one pass over the tensor, and equal
 * (format, rounding) requests share scales and codes outright; a probe then
 * reads those results from the workspace of the probe that made them, and a
 * non-finite operand is reported in the record of every probe that uses it.
 * All of it is ordered after the work already in `stream`, and work put into
 * `stream` after the call waits for every probe.  `out` is a device array of n
 * records; the n workspaces must be distinct and sized per probe.  With
 * qm_probe_batch_host the operands live in host memory as for
 * qm_probe_layer_host (l_stage[i], r_stage[i]: distinct device staging buffers,
 * each as large as its operand): every distinct host operand (same address and
 * extent) is copied to the device once, into the staging buffer of the first
 * probe that names it, on a stream of the library's own and in the order in
 * which the probes first name them; the probes run as device batches of 16
 * consecutive probes, each waiting only for the copies it needs, so that the
 * copies of later probes run under the kernels of earlier ones (keep the
 * probes of one product next to each other: operands are shared within such a
 * batch of 16); out_host receives the n records and the call waits for them;
 * the first device-detected condition is returned.  n == 0 is a no-op.  On an argument
 * error of probe i the probes before it are completed as described; the rest
 * are not issued.  Make the first call on a device outside any stream capture.
 */
qm_status qm_probe_batch(int32_t n, const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg,
                         qm_metric_result* out, void* const* ws, const size_t* ws_bytes, void* stream);
qm_status qm_probe_batch_host(int32_t n, const qm_operand* L_host, const qm_operand* R_host,
                              const qm_probe_cfg* cfg, void* const* l_stage, void* const* r_stage,
                              qm_metric_result* out_host, qm_metric_result* out_dev, void* const* ws,
                              const size_t* ws_bytes, void* stream);
/* The bytes one qm_probe_batch_host call copies to the device (every distinct host operand once:
 * operands with the same host address and extent share one copy) and back (n records). */
qm_status qm_probe_batch_host_bytes(int32_t n, const qm_operand* L_host, const qm_operand* R_host, size_t* h2d_bytes,
                                    size_t* d2h_bytes);

const char* qm_status_string(int32_t status);
int32_t qm_version(void);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* qm_last_cuda_error(void);


/*
 * qm_metric for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).  Some users of this library
 * run where cudaMalloc is unavailable to them: a plug-in that only receives
 * input and output pointers from its host application, code that must stay
 * inside a region managed by somebody else's memory pool, or a loop that may
 * not call the allocator for latency reasons.  Such a caller cannot produce
 * the `ws` scratch that qm_metric asks for, so this variant keeps its scratch
 * inside the library: a fixed 40 KiB array in the device image, held by every
 * GPU that loads the library until the process exits.  It computes exactly
 * what qm_metric computes: ref, q, den are `count` fp32 values each (device),
 * `out` (device) receives the record.
 *  - count may be at most qm_metric_noalloc_max_count() (2^30); larger inputs
 *    are refused with QM_ERR_WORKSPACE_TOO_SMALL and nothing is launched.
 *  - The call allocates nothing, on the host or on the device.
 *  - The first call on each device looks up the array's device address; make
 *    that first call outside any stream capture.
 *  - All calls on a device share the one array, which still holds the previous
 *    call's partial sums.  Each call overwrites every entry it later reads, so
 *    no clearing is needed, but two calls whose kernels overlap on the GPU
 *    (different streams, no ordering between them) race on it: serialise them.
 */
int64_t qm_metric_noalloc_max_count(void);
qm_status qm_metric_noalloc(const float* ref, const float* q, const float* den, int64_t count,
                            qm_metric_result* out, void* stream);

/*
 * Measurement aids (no counterpart in the paper).
 * qm_kernel_launches: how many kernels the library has launched in this
 * process so far.  qm_profile_enable(1) makes every later qm_probe_layer record
 * a CUDA event pair on the caller's stream around its fused tensor-core probe
 * kernel; qm_profile_read waits for those events, returns the summed kernel
 * time in milliseconds and the number of launches, and starts a new interval.
 * Events are host objects; no device memory is involved.
 */
int64_t qm_kernel_launches(void);
qm_status qm_profile_enable(int32_t on);
qm_status qm_profile_read(double* tc_probe_ms, int32_t* tc_probe_launches);
/* The same interval launch by launch, without ending it: for launch i (in issue order, up to
 * `cap`) its start relative to the first recorded launch's start and its duration, both in
 * milliseconds; *launches receives the number recorded so far. */
qm_status qm_profile_samples(double* start_ms, double* dur_ms, int32_t cap, int32_t* launches);

/*
 * Read-bandwidth calibration (measurement aid, no counterpart in the paper): one
 * read-only pass over `bytes` of device memory at `data` (16-byte aligned) and
 * nothing else, so that the library's read-mostly kernels (max|x|, tensor
 * statistics) can be compared with what a pure read stream reaches on the same
 * buffer.  variant: 0 = 8 plain 128-bit loads in flight per thread, 3 = 16 of
 * them; 1 and 2 = 4 and 8 256-bit loads in flight with streaming cache hints
 * (data 32-byte aligned); blocks_per_sm (1..32) blocks of 256 threads per SM.
 * sink may be NULL.  Time it with events.
 */
qm_status qm_debug_read_pass(const void* data, size_t bytes, int32_t variant, int32_t blocks_per_sm, uint32_t* sink,
                             void* stream);

/*
 * Testing aids for the bounded device waits (no counterpart in the paper).
 * Every barrier wait inside the fused probe kernel gives up after a time limit
 * (one second by default): the kernel then raises QM_DEVERR_TIMEOUT in the
 * record, lets its outstanding loads and tensor-core work finish, frees its
 * tensor memory and returns, and the context stays usable.
 * qm_debug_set_wait_limit_ns sets that limit for later launches (0 restores
 * the default).  qm_debug_stop_producer_after(k) makes the loading warp of
 * every CTA of later launches stop after its first k k-blocks (64-deep slices
 * of the contraction), so that the warps waiting for the next slice run into
 * the limit; 0xffffffff (the default) switches the hook off.  Both are
 * process-wide and meant for tests only.
 */
void qm_debug_set_wait_limit_ns(uint64_t ns);
void qm_debug_stop_producer_after(uint32_t k_blocks);

#ifdef __cplusplus
}
#endif
#endif /* QM_H_ */
