// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "qm.h"

namespace qm {

// A validated operand view, extents as 64-bit, element strides.
struct View {
  const void* data;
  int dtype;            // qm_dtype
  int64_t nc, c;        // non-contracting / contracting extents
  int64_t s_nc, s_c;    // element strides
  int64_t batch, s_b;   // batch count / element stride
  bool c_contig() const { return s_c == 1; }
};

// Largest expressible magnitude of a format (127, 448, 57344).
__host__ __device__ inline float fmt_qmax(int fmt) {
  return fmt == QM_FMT_INT8 ? 127.0f : (fmt == QM_FMT_E4M3 ? 448.0f : 57344.0f);
}

// Per-thread record of the last CUDA error text.
void note_cuda_error(cudaError_t e, const char* where);
#define QM_CUDA_OK(expr)                                   \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) {                              \
      ::qm::note_cuda_error(e__, #expr);                   \
      return QM_ERR_CUDA;                                  \
    }                                                      \
  } while (0)

// One-time host state (function attributes, occupancy, SM counts, stream pools, symbol addresses)
// is kept per device, indexed by the current device's ordinal.
constexpr int kMaxDevices = 64;
int current_device();   // the ordinal, or -1 when it cannot be read or is not below kMaxDevices
int sm_count();         // of the current device

// Programmatic dependent launch.  Every kernel of the probe's chain is launched with the
// attribute that lets its CTAs be scheduled while the kernel before it in the stream is still
// draining, and starts with pdl_prologue(): wait until that kernel's results are visible, then
// allow the next kernel in the stream to be scheduled early in the same way.  This removes the
// launch gap between the short dependent kernels of a probe.
bool pdl_enabled();   // on unless the environment has QM_PDL=0
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_prologue() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... P, typename... A>
inline cudaError_t launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}
#endif

// Cumulative count of kernels this library has launched (profiling aid).
void count_launch(int n = 1);
// When profiling is on, returns an event pair to record around the fused tensor-core probe
// kernel; nullptrs otherwise.
void profile_events(cudaEvent_t* start, cudaEvent_t* stop);

// ---- scale / quantize (scale_quantize.cu) ---------------------------------
// amax: uint32 buffer (1 or batch*nc entries) that must be zero on entry; on exit it holds
// the bit pattern of max|x| per group.
qm_status launch_absmax(const View& x, int gran, uint32_t* amax_bits, cudaStream_t s);
// In place on the per-(batch element, channel) maxima of launch_absmax: entries of batch elements
// b with equal b % groups are replaced by their common maximum (scales shared along the batch).
qm_status launch_share_amax(uint32_t* amax_bits, int64_t batch, int64_t groups, int64_t nc, cudaStream_t s);
// In place: bit pattern of max|x| -> delta = max|x| / qmax (1 where max|x| == 0).
// err_word (optional): gets QM_DEVERR_NONFINITE or-ed in when a group max is NaN/Inf.
qm_status launch_finalize_delta(float* delta, int64_t n, int fmt, uint32_t* err_word, cudaStream_t s);
// codes (+ optional |x| and x as bf16, contraction-major).  `delta` holds finished deltas, or,
// with from_amax, the max|x| bit patterns of launch_absmax: the kernel then does the division
// itself, writes the deltas to delta_out and raises QM_DEVERR_NONFINITE in err_word (optional).
// draw != nullptr: stochastic rounding with these draws instead of round-to-nearest-even.
struct StochasticDraw { uint64_t seed; uint32_t stream; };
qm_status launch_quantize(const View& x, int fmt, int gran, const float* delta, bool from_amax,
                          float* delta_out, uint32_t* err_word, uint8_t* codes, void* abs_copy,
                          void* kmaj_copy, cudaStream_t s, const StochasticDraw* draw = nullptr);
// The codes of nf (1..3) distinct formats of one operand from the max|x| bit patterns of
// launch_absmax, round-to-nearest-even; per format k its scales go to delta_out[k], its codes to
// codes[k] and a non-finite maximum is flagged in err_word[k] (optional).  Per-tensor scales of a
// bf16 operand are served by one kernel that reads the operand once; everything else by one
// launch per format.  kmaj_copy as in launch_quantize.
qm_status launch_quantize_multi(const View& x, int gran, const uint32_t* amax, int nf, const int* fmts,
                                float* const* delta_out, uint32_t* const* err_word, uint8_t* const* codes,
                                void* kmaj_copy, cudaStream_t s);
// Single pass per row: absmax, delta, codes (contiguous contraction, per-channel).
qm_status launch_scale_quantize_rows(const View& x, int fmt, float* delta_out, uint8_t* codes,
                                     void* abs_copy, uint32_t* err_word, cudaStream_t s);

// ---- single-tensor passes (tensor_stats.cu) --------------------------------
size_t stats_workspace_bytes();
qm_status launch_tensor_stats(const View& x, qm_tensor_stats_result* out, void* ws, cudaStream_t s);
// delta: finished Eq. 1 scales (1 value, or one per batch element and non-contracting index)
qm_status launch_quantize_error(const View& x, int fmt, int gran, const float* delta,
                                qm_quant_error_result* out, void* ws, cudaStream_t s);

// ---- metric (metric.cu) ----------------------------------------------------
// One partial record per CTA: {sum_be, max_be, sum_diff2, sum_ref2, sum_den2} as doubles.
constexpr int kPartialDoubles = 5;
int metric_blocks(int64_t count);
qm_status launch_metric_partials(const float* ref, const float* q, const float* den, int64_t count,
                                 double* partials, int nblocks, cudaStream_t s);
// Sums `n` partial records in a fixed order and writes the result record.
qm_status launch_metric_finalize(const double* partials, int n, uint64_t count,
                                 const uint32_t* err_word, qm_metric_result* out, cudaStream_t s);

// Zeroes up to kClearMax regions of 32-bit words (4-byte aligned) in one launch: the control words
// of the workspaces of a batch.
constexpr int kClearMax = 32;
struct ClearList { int n; void* ptr[kClearMax]; uint32_t words[kClearMax]; };
qm_status launch_clear_many(const ClearList& list, cudaStream_t s);

// ---- CUDA-core GEMMs (gemm_simt.cu) ---------------------------------------
struct GemmShape { int64_t M, N, K, batch; };
qm_status launch_simt_gemm_lp(const uint8_t* cl, int fmt_l, const float* dl, int gran_l,
                              const uint8_t* cr, int fmt_r, const float* dr, int gran_r,
                              GemmShape g, float* out_descaled, void* out_raw, cudaStream_t s);
int simt_probe_blocks(GemmShape g);
// Fused CUDA-core probe: three accumulators per output, Eq. 3 partials per CTA.
qm_status launch_simt_probe(const View& L, const View& R, const uint8_t* cl, int fmt_l,
                            const float* dl, int gran_l, const uint8_t* cr, int fmt_r,
                            const float* dr, int gran_r, double* partials, cudaStream_t s);

// ---- tensor-core GEMMs (gemm_tc.cu) ---------------------------------------
struct TcProbeArgs {
  // bf16, contraction contiguous; element strides between rows / batches
  const void* l; int64_t l_ld, l_sb;
  const void* r; int64_t r_ld, r_sb;
  const void* l_abs; const void* r_abs;     // dense [batch][rows][K]
  const uint8_t* cl; const uint8_t* cr;     // codes, rows of qm_code_ld(K) bytes
  int fmt_l, fmt_r;
  const float* dl; int gran_l;
  const float* dr; int gran_r;
  GemmShape g;
  double* partials;                         // tc_probe_records(g) records
  uint32_t* done_counter;                   // zero on entry; counts finished CTAs
  qm_metric_result* result;                 // written by the last CTA to finish
  uint32_t* err_word;
  const uint32_t* err_also[2] = {nullptr, nullptr};   // error words of other probes whose kernels made this probe's codes
  double* row_stats = nullptr;              // optional per-row Eq. 3 sums (zeroed by the caller), one-format probes only
  // Two formats in one pass (cl2 != nullptr): codes and scales of the second format, same
  // granularities; `result` then points at two records and `partials` holds 2 x tc_probe_records.
  // The first format must be an FP8 one.
  const uint8_t* cl2 = nullptr; const uint8_t* cr2 = nullptr;
  int fmt_l2 = 0, fmt_r2 = 0;
  const float* dl2 = nullptr; const float* dr2 = nullptr;
};
int tc_probe_records(GemmShape g);
qm_status launch_tc_probe(const TcProbeArgs& a, cudaStream_t s);
// Up to tc_group_max() one-format probes as one persistent launch (every probe's operands must be
// prepared already; each writes its own record; the first probe's done_counter counts the CTAs).
int tc_group_max();
qm_status launch_tc_probe_group(const TcProbeArgs* ps, int n, cudaStream_t s);
// Bound of every barrier wait of the fused probe kernel (0 restores the default of one second), and
// a hook for testing the give-up path: the producer issues no more than this many k-blocks
// per CTA (0xffffffff: off), so that the consumers' waits run out.
void set_wait_limit_ns(uint64_t ns);
void set_stop_after_kb(uint32_t kb);
qm_status launch_tc_gemm_lp(const uint8_t* cl, int fmt_l, const float* dl, int gran_l,
                            const uint8_t* cr, int fmt_r, const float* dr, int gran_r,
                            GemmShape g, float* out_descaled, void* out_raw, uint32_t* err_word,
                            cudaStream_t s);
qm_status launch_tc_gemm_ref(const void* l, const void* r, GemmShape g, float* out,
                             uint32_t* err_word, cudaStream_t s);

}  // namespace qm
