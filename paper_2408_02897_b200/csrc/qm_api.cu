// The C ABI: argument checks, workspace layout and launch sequencing.  All arithmetic of the
// probe runs in the kernels of the other translation units.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "qm_internal.h"

namespace qm {

static thread_local char g_last_error[256] = "";

void note_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
  (void)cudaGetLastError();   // do not let a non-sticky error be blamed on a later call
}

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int sm_count() {
  static std::atomic<int> n[kMaxDevices];
  const int dev = current_device();
  if (dev < 0) return 148;
  int v = n[dev].load(std::memory_order_relaxed);
  if (v == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n[dev].store(v, std::memory_order_relaxed);
  }
  return v;
}

bool pdl_enabled() {
  static const bool on = [] {
    const char* e = getenv("QM_PDL");
    return !(e && e[0] == '0');
  }();
  return on;
}

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// profiling: a pool of event pairs recorded around the fused tensor-core probe kernel
static std::mutex g_prof_mutex;
static bool g_prof_on = false;
static std::vector<cudaEvent_t> g_prof_events;   // start0, stop0, start1, stop1, ...
static size_t g_prof_used = 0;

void profile_events(cudaEvent_t* start, cudaEvent_t* stop) {
  *start = *stop = nullptr;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (!g_prof_on) return;
  if (g_prof_used + 2 > g_prof_events.size()) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess) return;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return; }
    g_prof_events.push_back(a); g_prof_events.push_back(b);
  }
  *start = g_prof_events[g_prof_used]; *stop = g_prof_events[g_prof_used + 1];
  g_prof_used += 2;
}

namespace {

bool valid_fmt(int f) { return f == QM_FMT_INT8 || f == QM_FMT_E4M3 || f == QM_FMT_E5M2; }
bool valid_gran(int g) { return g == QM_GRAN_TENSOR || g == QM_GRAN_CHANNEL; }

qm_status to_view(const qm_operand* x, View* v) {
  if (!x || !x->data) return QM_ERR_INVALID_ARG;
  if (x->dtype != QM_DT_F32 && x->dtype != QM_DT_BF16) return QM_ERR_INVALID_ARG;
  if (x->noncontract <= 0 || x->contract <= 0 || x->batch <= 0) return QM_ERR_INVALID_ARG;
  // the stride of an extent-1 dimension carries no information: give it the dense value
  int64_t s_nc = x->stride_nc, s_c = x->stride_c;
  if (x->noncontract == 1 && x->contract == 1) { s_nc = 8; s_c = 1; }
  else if (x->noncontract == 1) s_nc = s_c == 1 ? ((x->contract + 7) & ~(int64_t)7) : 1;
  else if (x->contract == 1) s_c = s_nc == 1 ? ((x->noncontract + 7) & ~(int64_t)7) : 1;
  if (s_nc <= 0 || s_c <= 0) return QM_ERR_INVALID_ARG;
  if (s_nc != 1 && s_c != 1) return QM_ERR_UNSUPPORTED;
  if (x->batch > 1 && x->stride_batch <= 0) return QM_ERR_INVALID_ARG;
  v->data = x->data; v->dtype = x->dtype;
  v->nc = x->noncontract; v->c = x->contract;
  v->s_nc = s_nc; v->s_c = s_c;
  v->batch = x->batch;
  // rows must not overlap
  if (v->s_c == 1 && v->nc > 1 && v->s_nc < v->c) return QM_ERR_INVALID_ARG;
  if (v->s_c != 1 && v->c > 1 && v->s_c < v->nc) return QM_ERR_INVALID_ARG;
  const int64_t span = (v->nc - 1) * v->s_nc + (v->c - 1) * v->s_c + 1;
  v->s_b = x->batch > 1 ? x->stride_batch : ((span + 7) & ~(int64_t)7);
  if (v->batch > 1 && v->s_b < span) return QM_ERR_INVALID_ARG;
  // 128-bit loads: base, the non-unit stride and the batch stride must keep 16-byte alignment
  if (reinterpret_cast<uintptr_t>(x->data) & 15) return QM_ERR_ALIGNMENT;
  const int64_t big = v->s_c == 1 ? v->s_nc : v->s_c;
  if ((big & 7) || (v->batch > 1 && (v->s_b & 7))) return QM_ERR_ALIGNMENT;
  return QM_OK;
}

int64_t delta_count(const View& v, int gran) { return gran == QM_GRAN_TENSOR ? 1 : v.nc * v.batch; }

size_t align256(size_t n) { return (n + 255) & ~(size_t)255; }

struct Workspace {
  size_t off_err, off_ml, off_mr, off_dl, off_dr, off_cl, off_cr, off_al, off_ar, off_kl, off_kr, off_part, total;
  int n_part;
  bool tc;
};

Workspace plan(const View& L, const View& R, const qm_probe_cfg& cfg) {
  Workspace w{};
  w.tc = cfg.ref == QM_REF_BF16_FP32ACC;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += align256(bytes); return at; };
  w.off_err = take(256);
  w.off_ml = take(sizeof(float) * delta_count(L, cfg.gran_l));      // max|x| bit patterns (cleared)
  w.off_mr = take(sizeof(float) * delta_count(R, cfg.gran_r));
  w.off_dl = take(sizeof(float) * delta_count(L, cfg.gran_l));
  w.off_dr = take(sizeof(float) * delta_count(R, cfg.gran_r));
  const int64_t ldc = qm_code_ld(L.c);
  w.off_cl = take((size_t)(L.batch * L.nc * ldc));
  w.off_cr = take((size_t)(R.batch * R.nc * ldc));
  if (w.tc) {
    w.off_al = take((size_t)(L.batch * L.nc * L.c) * 2);
    w.off_ar = take((size_t)(R.batch * R.nc * R.c) * 2);
    w.off_kl = L.c_contig() ? 0 : take((size_t)(L.batch * L.nc * L.c) * 2);
    w.off_kr = R.c_contig() ? 0 : take((size_t)(R.batch * R.nc * R.c) * 2);
  }
  GemmShape g{L.nc, R.nc, L.c, L.batch};
  w.n_part = w.tc ? tc_probe_records(g) : simt_probe_blocks(g);
  w.off_part = take(sizeof(double) * kPartialDoubles * (size_t)w.n_part);
  w.total = o;
  return w;
}

qm_status check_probe(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg, View* L, View* R) {
  if (!cfg) return QM_ERR_INVALID_ARG;
  qm_status st = to_view(Lo, L);
  if (st != QM_OK) return st;
  st = to_view(Ro, R);
  if (st != QM_OK) return st;
  if (!valid_fmt(cfg->fmt_l) || !valid_fmt(cfg->fmt_r) || !valid_gran(cfg->gran_l) || !valid_gran(cfg->gran_r))
    return QM_ERR_INVALID_ARG;
  if (cfg->round & ~(QM_ROUND_STOCHASTIC_L | QM_ROUND_STOCHASTIC_R)) return QM_ERR_INVALID_ARG;
  if (cfg->batch_groups_l < 0 || cfg->batch_groups_r < 0) return QM_ERR_INVALID_ARG;
  if ((cfg->batch_groups_l && L->batch % cfg->batch_groups_l) || (cfg->batch_groups_r && R->batch % cfg->batch_groups_r))
    return QM_ERR_INVALID_ARG;
  if (cfg->ref != QM_REF_BF16_FP32ACC && cfg->ref != QM_REF_FP32) return QM_ERR_INVALID_ARG;
  if (L->c != R->c || L->batch != R->batch) return QM_ERR_INVALID_ARG;
  if ((cfg->fmt_l == QM_FMT_INT8) != (cfg->fmt_r == QM_FMT_INT8)) return QM_ERR_UNSUPPORTED;
  if (cfg->ref == QM_REF_BF16_FP32ACC) {
    if (L->dtype != QM_DT_BF16 || R->dtype != QM_DT_BF16) return QM_ERR_UNSUPPORTED;
    if (L->c % 16) return QM_ERR_UNSUPPORTED;
  } else if (cfg->row_stats) {
    return QM_ERR_UNSUPPORTED;
  }
  if (reinterpret_cast<uintptr_t>(cfg->row_stats) & 7) return QM_ERR_ALIGNMENT;
  return QM_OK;
}

// scale + quantize of one operand inside the probe
qm_status prepare_operand(const View& x, int fmt, int gran, uint32_t* amax, float* delta, uint8_t* codes,
                          void* abs_copy, void* kmaj_copy, uint32_t* err_word, const StochasticDraw* draw,
                          int batch_groups, cudaStream_t s) {
  const bool shared = gran == QM_GRAN_CHANNEL && batch_groups > 0 && batch_groups < x.batch;
  if (!draw && !shared && gran == QM_GRAN_CHANNEL && x.c_contig())
    return launch_scale_quantize_rows(x, fmt, delta, codes, abs_copy, err_word, s);
  qm_status st = launch_absmax(x, gran, amax, s);
  if (st != QM_OK) return st;
  if (shared) {
    st = launch_share_amax(amax, x.batch, batch_groups, x.nc, s);
    if (st != QM_OK) return st;
  }
  // the quantize kernel turns max|x| into delta itself
  return launch_quantize(x, fmt, gran, reinterpret_cast<const float*>(amax), true, delta, err_word, codes,
                         abs_copy, kmaj_copy, s, draw);
}

}  // namespace
}  // namespace qm

using namespace qm;

extern "C" {

int64_t qm_code_ld(int64_t contract) { return (contract + 15) & ~(int64_t)15; }

qm_status qm_scale(const qm_operand* x, int32_t fmt, int32_t gran, float* delta, void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (!valid_fmt(fmt) || !valid_gran(gran) || !delta) return QM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t n = delta_count(v, gran);
  QM_CUDA_OK(cudaMemsetAsync(delta, 0, sizeof(float) * n, s));
  st = launch_absmax(v, gran, reinterpret_cast<uint32_t*>(delta), s);
  if (st != QM_OK) return st;
  return launch_finalize_delta(delta, n, fmt, nullptr, s);
}

qm_status qm_scale_shared(const qm_operand* x, int32_t fmt, int32_t batch_groups, float* delta, void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (!valid_fmt(fmt) || !delta) return QM_ERR_INVALID_ARG;
  if (batch_groups < 1 || v.batch % batch_groups) return QM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t n = v.nc * v.batch;
  QM_CUDA_OK(cudaMemsetAsync(delta, 0, sizeof(float) * n, s));
  st = launch_absmax(v, QM_GRAN_CHANNEL, reinterpret_cast<uint32_t*>(delta), s);
  if (st != QM_OK) return st;
  if (batch_groups < v.batch) {
    st = launch_share_amax(reinterpret_cast<uint32_t*>(delta), v.batch, batch_groups, v.nc, s);
    if (st != QM_OK) return st;
  }
  return launch_finalize_delta(delta, n, fmt, nullptr, s);
}

static qm_status quantize_entry(const qm_operand* x, int32_t fmt, int32_t gran, const StochasticDraw* draw,
                                const float* delta, float* delta_out, uint8_t* codes, void* abs_copy,
                                void* kmaj_copy, void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (!valid_fmt(fmt) || !valid_gran(gran) || !codes) return QM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(codes) & 15) || (reinterpret_cast<uintptr_t>(abs_copy) & 15) ||
      (reinterpret_cast<uintptr_t>(kmaj_copy) & 15))
    return QM_ERR_ALIGNMENT;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (delta)
    return launch_quantize(v, fmt, gran, delta, false, nullptr, nullptr, codes, abs_copy, kmaj_copy, s, draw);
  if (!delta_out) return QM_ERR_INVALID_ARG;
  const int64_t n = delta_count(v, gran);
  if (!draw && gran == QM_GRAN_CHANNEL && v.c_contig() && !kmaj_copy)
    return launch_scale_quantize_rows(v, fmt, delta_out, codes, abs_copy, nullptr, s);
  QM_CUDA_OK(cudaMemsetAsync(delta_out, 0, sizeof(float) * n, s));
  st = launch_absmax(v, gran, reinterpret_cast<uint32_t*>(delta_out), s);
  if (st != QM_OK) return st;
  st = launch_finalize_delta(delta_out, n, fmt, nullptr, s);
  if (st != QM_OK) return st;
  return launch_quantize(v, fmt, gran, delta_out, false, nullptr, nullptr, codes, abs_copy, kmaj_copy, s, draw);
}

qm_status qm_quantize(const qm_operand* x, int32_t fmt, int32_t gran, int32_t round, const float* delta,
                      float* delta_out, uint8_t* codes, void* abs_copy, void* kmaj_copy, void* stream) {
  if (round != QM_ROUND_RTNE) return QM_ERR_UNSUPPORTED;   // stochastic rounding: qm_quantize_stochastic
  return quantize_entry(x, fmt, gran, nullptr, delta, delta_out, codes, abs_copy, kmaj_copy, stream);
}

qm_status qm_quantize_stochastic(const qm_operand* x, int32_t fmt, int32_t gran, uint64_t seed, uint32_t stream_id,
                                 const float* delta, float* delta_out, uint8_t* codes, void* abs_copy,
                                 void* kmaj_copy, void* stream) {
  const StochasticDraw draw{seed, stream_id};
  return quantize_entry(x, fmt, gran, &draw, delta, delta_out, codes, abs_copy, kmaj_copy, stream);
}

qm_status qm_gemm(const uint8_t* codes_l, int32_t fmt_l, const float* delta_l, int32_t gran_l,
                  const uint8_t* codes_r, int32_t fmt_r, const float* delta_r, int32_t gran_r, int64_t M,
                  int64_t N, int64_t K, int64_t batch, float* out_descaled, void* out_raw, int32_t use_simt,
                  void* stream) {
  if (!codes_l || !codes_r || !delta_l || !delta_r || (!out_descaled && !out_raw)) return QM_ERR_INVALID_ARG;
  if (!valid_fmt(fmt_l) || !valid_fmt(fmt_r) || !valid_gran(gran_l) || !valid_gran(gran_r)) return QM_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || batch <= 0) return QM_ERR_INVALID_ARG;
  if ((fmt_l == QM_FMT_INT8) != (fmt_r == QM_FMT_INT8)) return QM_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(codes_l) & 15) || (reinterpret_cast<uintptr_t>(codes_r) & 15)) return QM_ERR_ALIGNMENT;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  GemmShape g{M, N, K, batch};
  if (use_simt)
    return launch_simt_gemm_lp(codes_l, fmt_l, delta_l, gran_l, codes_r, fmt_r, delta_r, gran_r, g,
                               out_descaled, out_raw, s);
  if (K % 16) return QM_ERR_UNSUPPORTED;
  return launch_tc_gemm_lp(codes_l, fmt_l, delta_l, gran_l, codes_r, fmt_r, delta_r, gran_r, g, out_descaled,
                           out_raw, nullptr, s);
}

qm_status qm_gemm_ref(const void* l_bf16, const void* r_bf16, int64_t M, int64_t N, int64_t K, int64_t batch,
                      float* out, void* stream) {
  if (!l_bf16 || !r_bf16 || !out) return QM_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K <= 0 || batch <= 0) return QM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(l_bf16) & 15) || (reinterpret_cast<uintptr_t>(r_bf16) & 15)) return QM_ERR_ALIGNMENT;
  if (K % 16) return QM_ERR_UNSUPPORTED;
  GemmShape g{M, N, K, batch};
  return launch_tc_gemm_ref(l_bf16, r_bf16, g, out, nullptr, static_cast<cudaStream_t>(stream));
}

size_t qm_metric_workspace_bytes(int64_t count) {
  if (count <= 0) return 0;
  return align256(sizeof(double) * kPartialDoubles * (size_t)metric_blocks(count));
}

qm_status qm_metric(const float* ref, const float* q, const float* den, int64_t count, qm_metric_result* out,
                    void* ws, size_t ws_bytes, void* stream) {
  if (!ref || !q || !den || !out || !ws || count <= 0) return QM_ERR_INVALID_ARG;
  if (ws_bytes < qm_metric_workspace_bytes(count)) return QM_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(ws) & 7) return QM_ERR_ALIGNMENT;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int nb = metric_blocks(count);
  qm_status st = launch_metric_partials(ref, q, den, count, static_cast<double*>(ws), nb, s);
  if (st != QM_OK) return st;
  return launch_metric_finalize(static_cast<double*>(ws), nb, (uint64_t)count, nullptr, out, s);
}

size_t qm_workspace_bytes(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg) {
  View L, R;
  if (check_probe(Lo, Ro, cfg, &L, &R) != QM_OK) return 0;
  return plan(L, R, *cfg).total;
}

// The probe in phases that may be issued apart, on different streams (same arguments every time):
// kClear clears the workspace words, kPrepareL / kPrepareR run scale + quantize of one operand
// (after kClear), kProducts the products and the Eq. 3 reduction (after both).  With `defer` set and a tensor-core configuration, kProducts only describes the
// fused kernel's work in *defer (for a grouped launch) instead of launching it.
// What one prepared operand leaves behind that does not depend on the 8-bit format: the max|x|
// bit patterns, the |x| copy and (for a strided contraction) the contraction-major copy.  Inside
// a batch a later probe whose operand is the same tensor under the same scale grouping borrows
// them and runs only its own quantize kernel.
struct OperandShare {
  const uint32_t* amax = nullptr;
  void* abs_copy = nullptr;
  void* kmaj_copy = nullptr;
};
struct ProbeShare {
  const OperandShare* from_l = nullptr;   // borrow (inputs)
  const OperandShare* from_r = nullptr;
  OperandShare* own_l = nullptr;          // what this probe's own chains produce (outputs)
  OperandShare* own_r = nullptr;
};

enum { kClear = 1, kPrepareL = 2, kPrepareR = 4, kPrepare = kClear | kPrepareL | kPrepareR, kProducts = 8 };
static qm_status probe_phases(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg,
                              qm_metric_result* out, void* ws, size_t ws_bytes, void* stream, int phases,
                              TcProbeArgs* defer, bool* deferred, const ProbeShare* share = nullptr,
                              ClearList* clear_later = nullptr) {
  if (deferred) *deferred = false;
  View L, R;
  qm_status st = check_probe(Lo, Ro, cfg, &L, &R);
  if (st != QM_OK) return st;
  if (!out || !ws) return QM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return QM_ERR_ALIGNMENT;
  const Workspace w = plan(L, R, *cfg);
  if (ws_bytes < w.total) return QM_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  uint32_t* err = reinterpret_cast<uint32_t*>(base + w.off_err);
  float* dl = reinterpret_cast<float*>(base + w.off_dl);
  float* dr = reinterpret_cast<float*>(base + w.off_dr);
  uint8_t* cl = base + w.off_cl;
  uint8_t* cr = base + w.off_cr;
  double* part = reinterpret_cast<double*>(base + w.off_part);
  // the error word, the finished-CTA counter and both max|x| buffers are adjacent: one clear
  if ((phases & kClear) && clear_later && clear_later->n < kClearMax) {
    clear_later->ptr[clear_later->n] = base;                 // cleared with others by one kernel
    clear_later->words[clear_later->n++] = (uint32_t)(w.off_dl / 4);
  } else if (phases & kClear) {
    QM_CUDA_OK(cudaMemsetAsync(base, 0, w.off_dl, s));
  }
  if ((phases & kClear) && cfg->row_stats)
    QM_CUDA_OK(cudaMemsetAsync(cfg->row_stats, 0, sizeof(double) * QM_ROW_STATS * (size_t)(L.batch * L.nc), s));
  uint32_t* ml = reinterpret_cast<uint32_t*>(base + w.off_ml);
  uint32_t* mr = reinterpret_cast<uint32_t*>(base + w.off_mr);
  void* al = w.tc ? base + w.off_al : nullptr;
  void* ar = w.tc ? base + w.off_ar : nullptr;
  void* kl = (w.tc && !L.c_contig()) ? base + w.off_kl : nullptr;
  void* kr = (w.tc && !R.c_contig()) ? base + w.off_kr : nullptr;
  const StochasticDraw draw_l{cfg->seed, 0u}, draw_r{cfg->seed, 1u};
  const StochasticDraw* dl_draw = (cfg->round & QM_ROUND_STOCHASTIC_L) ? &draw_l : nullptr;
  const StochasticDraw* dr_draw = (cfg->round & QM_ROUND_STOCHASTIC_R) ? &draw_r : nullptr;
  const OperandShare* from_l = share ? share->from_l : nullptr;
  const OperandShare* from_r = share ? share->from_r : nullptr;
  if (share && share->own_l) *share->own_l = OperandShare{ml, al, kl};
  if (share && share->own_r) *share->own_r = OperandShare{mr, ar, kr};
  if (phases & kPrepareL) {
    st = from_l ? launch_quantize(L, cfg->fmt_l, cfg->gran_l, reinterpret_cast<const float*>(from_l->amax), true, dl,
                                  err, cl, nullptr, nullptr, s, dl_draw)
                : prepare_operand(L, cfg->fmt_l, cfg->gran_l, ml, dl, cl, al, kl, err, dl_draw, cfg->batch_groups_l, s);
    if (st != QM_OK) return st;
  }
  if (phases & kPrepareR) {
    st = from_r ? launch_quantize(R, cfg->fmt_r, cfg->gran_r, reinterpret_cast<const float*>(from_r->amax), true, dr,
                                  err, cr, nullptr, nullptr, s, dr_draw)
                : prepare_operand(R, cfg->fmt_r, cfg->gran_r, mr, dr, cr, ar, kr, err, dr_draw, cfg->batch_groups_r, s);
    if (st != QM_OK) return st;
  }
  if (from_l) { al = from_l->abs_copy; kl = from_l->kmaj_copy; }
  if (from_r) { ar = from_r->abs_copy; kr = from_r->kmaj_copy; }
  if (!(phases & kProducts)) return QM_OK;
  GemmShape g{L.nc, R.nc, L.c, L.batch};
  if (w.tc) {
    TcProbeArgs p{};
    p.l = kl ? kl : L.data; p.l_ld = kl ? L.c : L.s_nc; p.l_sb = kl ? L.nc * L.c : L.s_b;
    p.r = kr ? kr : R.data; p.r_ld = kr ? R.c : R.s_nc; p.r_sb = kr ? R.nc * R.c : R.s_b;
    p.l_abs = al; p.r_abs = ar; p.cl = cl; p.cr = cr;
    p.fmt_l = cfg->fmt_l; p.fmt_r = cfg->fmt_r;
    p.dl = dl; p.gran_l = cfg->gran_l; p.dr = dr; p.gran_r = cfg->gran_r;
    p.g = g; p.partials = part; p.err_word = err;
    p.done_counter = err + 1;               // second word of the cleared error slot
    p.result = out;
    p.row_stats = cfg->row_stats;
    if (defer) {
      *defer = p;
      *deferred = true;
      return QM_OK;
    }
    return launch_tc_probe(p, s);           // the last CTA writes the record
  }
  st = launch_simt_probe(L, R, cl, cfg->fmt_l, dl, cfg->gran_l, cr, cfg->fmt_r, dr, cfg->gran_r, part, s);
  if (st != QM_OK) return st;
  return launch_metric_finalize(part, w.n_part, (uint64_t)(g.M * g.N * g.batch), err, out, s);
}

qm_status qm_probe_layer(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg,
                         qm_metric_result* out, void* ws, size_t ws_bytes, void* stream) {
  return probe_phases(Lo, Ro, cfg, out, ws, ws_bytes, stream, kPrepare | kProducts, nullptr, nullptr);
}

// ---- two formats in one pass -------------------------------------------------------------------
}  // extern "C"
namespace {
struct Workspace2 {
  Workspace a;                 // everything of the first format's probe
  size_t off_dl2, off_dr2, off_cl2, off_cr2, off_part2, total;
};
// Orders the two configurations so that an FP8 one comes first; returns false when they cannot
// share a pass.
bool order2(const qm_probe_cfg* ca, const qm_probe_cfg* cb, const qm_probe_cfg** first, const qm_probe_cfg** second,
            bool* swapped) {
  if (!ca || !cb) return false;
  if (ca->gran_l != cb->gran_l || ca->gran_r != cb->gran_r || ca->round != cb->round || ca->seed != cb->seed ||
      ca->batch_groups_l != cb->batch_groups_l || ca->batch_groups_r != cb->batch_groups_r)
    return false;
  if (ca->ref != QM_REF_BF16_FP32ACC || cb->ref != QM_REF_BF16_FP32ACC) return false;
  if (ca->row_stats || cb->row_stats) return false;
  const bool a_int = ca->fmt_l == QM_FMT_INT8, b_int = cb->fmt_l == QM_FMT_INT8;
  if (a_int && b_int) return false;
  *swapped = a_int;
  *first = a_int ? cb : ca;
  *second = a_int ? ca : cb;
  return true;
}
Workspace2 plan2(const View& L, const View& R, const qm_probe_cfg& first) {
  Workspace2 w{};
  w.a = plan(L, R, first);
  size_t o = w.a.total;
  auto take = [&](size_t bytes) { size_t at = o; o += align256(bytes); return at; };
  w.off_dl2 = take(sizeof(float) * delta_count(L, first.gran_l));
  w.off_dr2 = take(sizeof(float) * delta_count(R, first.gran_r));
  const int64_t ldc = qm_code_ld(L.c);
  w.off_cl2 = take((size_t)(L.batch * L.nc * ldc));
  w.off_cr2 = take((size_t)(R.batch * R.nc * ldc));
  w.off_part2 = take(sizeof(double) * kPartialDoubles * 2 * (size_t)w.a.n_part);
  w.total = o;
  return w;
}
// absmax once, then the codes of both formats from the same maxima
qm_status prepare_operand2(const View& x, int fmt_a, int fmt_b, int gran, uint32_t* amax, float* delta_a,
                           float* delta_b, uint8_t* codes_a, uint8_t* codes_b, void* abs_copy, void* kmaj_copy,
                           uint32_t* err_word, const StochasticDraw* draw, int batch_groups, cudaStream_t s) {
  qm_status st = launch_absmax(x, gran, amax, s);
  if (st != QM_OK) return st;
  if (gran == QM_GRAN_CHANNEL && batch_groups > 0 && batch_groups < x.batch) {
    st = launch_share_amax(amax, x.batch, batch_groups, x.nc, s);
    if (st != QM_OK) return st;
  }
  st = launch_quantize(x, fmt_a, gran, reinterpret_cast<const float*>(amax), true, delta_a, err_word, codes_a,
                       abs_copy, kmaj_copy, s, draw);
  if (st != QM_OK) return st;
  return launch_quantize(x, fmt_b, gran, reinterpret_cast<const float*>(amax), true, delta_b, err_word, codes_b,
                         nullptr, nullptr, s, draw);
}
}  // namespace
extern "C" {

size_t qm_workspace_bytes2(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg_a,
                           const qm_probe_cfg* cfg_b) {
  const qm_probe_cfg *c1, *c2;
  bool swapped;
  View L, R;
  if (!order2(cfg_a, cfg_b, &c1, &c2, &swapped)) return 0;
  if (check_probe(Lo, Ro, c1, &L, &R) != QM_OK || check_probe(Lo, Ro, c2, &L, &R) != QM_OK) return 0;
  return plan2(L, R, *c1).total;
}

qm_status qm_probe_layer2(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg_a,
                          const qm_probe_cfg* cfg_b, qm_metric_result* out, void* ws, size_t ws_bytes,
                          void* stream) {
  const qm_probe_cfg *c1, *c2;
  bool swapped;
  if (!cfg_a || !cfg_b) return QM_ERR_INVALID_ARG;
  if (!order2(cfg_a, cfg_b, &c1, &c2, &swapped)) return QM_ERR_UNSUPPORTED;
  View L, R;
  qm_status st = check_probe(Lo, Ro, c1, &L, &R);
  if (st == QM_OK) st = check_probe(Lo, Ro, c2, &L, &R);
  if (st != QM_OK) return st;
  if (!out || !ws) return QM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return QM_ERR_ALIGNMENT;
  const Workspace2 w = plan2(L, R, *c1);
  if (ws_bytes < w.total) return QM_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* base = static_cast<uint8_t*>(ws);
  uint32_t* err = reinterpret_cast<uint32_t*>(base + w.a.off_err);
  QM_CUDA_OK(cudaMemsetAsync(base, 0, w.a.off_dl, s));      // error word, CTA counter, both max|x| buffers
  uint32_t* ml = reinterpret_cast<uint32_t*>(base + w.a.off_ml);
  uint32_t* mr = reinterpret_cast<uint32_t*>(base + w.a.off_mr);
  float* dl = reinterpret_cast<float*>(base + w.a.off_dl);
  float* dr = reinterpret_cast<float*>(base + w.a.off_dr);
  float* dl2 = reinterpret_cast<float*>(base + w.off_dl2);
  float* dr2 = reinterpret_cast<float*>(base + w.off_dr2);
  void* kl = L.c_contig() ? nullptr : base + w.a.off_kl;
  void* kr = R.c_contig() ? nullptr : base + w.a.off_kr;
  const StochasticDraw draw_l{c1->seed, 0u}, draw_r{c1->seed, 1u};
  st = prepare_operand2(L, c1->fmt_l, c2->fmt_l, c1->gran_l, ml, dl, dl2, base + w.a.off_cl, base + w.off_cl2,
                        base + w.a.off_al, kl, err, (c1->round & QM_ROUND_STOCHASTIC_L) ? &draw_l : nullptr,
                        c1->batch_groups_l, s);
  if (st != QM_OK) return st;
  st = prepare_operand2(R, c1->fmt_r, c2->fmt_r, c1->gran_r, mr, dr, dr2, base + w.a.off_cr, base + w.off_cr2,
                        base + w.a.off_ar, kr, err, (c1->round & QM_ROUND_STOCHASTIC_R) ? &draw_r : nullptr,
                        c1->batch_groups_r, s);
  if (st != QM_OK) return st;
  TcProbeArgs p{};
  p.l = kl ? kl : L.data; p.l_ld = kl ? L.c : L.s_nc; p.l_sb = kl ? L.nc * L.c : L.s_b;
  p.r = kr ? kr : R.data; p.r_ld = kr ? R.c : R.s_nc; p.r_sb = kr ? R.nc * R.c : R.s_b;
  p.l_abs = base + w.a.off_al; p.r_abs = base + w.a.off_ar;
  p.cl = base + w.a.off_cl; p.cr = base + w.a.off_cr; p.cl2 = base + w.off_cl2; p.cr2 = base + w.off_cr2;
  p.fmt_l = c1->fmt_l; p.fmt_r = c1->fmt_r; p.fmt_l2 = c2->fmt_l; p.fmt_r2 = c2->fmt_r;
  p.dl = dl; p.dr = dr; p.dl2 = dl2; p.dr2 = dr2; p.gran_l = c1->gran_l; p.gran_r = c1->gran_r;
  p.g = GemmShape{L.nc, R.nc, L.c, L.batch};
  p.partials = reinterpret_cast<double*>(base + w.off_part2);
  p.err_word = err; p.done_counter = err + 1;
  // the kernel writes record 0 for its first format: give it scratch records when the caller's
  // order is the other way round, and copy them across
  if (!swapped) {
    p.result = out;
    return launch_tc_probe(p, s);
  }
  qm_metric_result* tmp = reinterpret_cast<qm_metric_result*>(base + w.a.off_part);   // unused by this path
  p.result = tmp;
  st = launch_tc_probe(p, s);
  if (st != QM_OK) return st;
  QM_CUDA_OK(cudaMemcpyAsync(out, tmp + 1, sizeof(qm_metric_result), cudaMemcpyDeviceToDevice, s));
  QM_CUDA_OK(cudaMemcpyAsync(out + 1, tmp, sizeof(qm_metric_result), cudaMemcpyDeviceToDevice, s));
  return QM_OK;
}

size_t qm_operand_span_bytes(const qm_operand* x) {
  View v;
  if (to_view(x, &v) != QM_OK) return 0;
  const int64_t last = (v.batch - 1) * v.s_b + (v.nc - 1) * v.s_nc + (v.c - 1) * v.s_c;
  return (size_t)(last + 1) * (v.dtype == QM_DT_BF16 ? 2 : 4);
}

size_t qm_stats_workspace_bytes(void) { return stats_workspace_bytes(); }

qm_status qm_tensor_stats(const qm_operand* x, qm_tensor_stats_result* out, void* ws, size_t ws_bytes,
                          void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (!out || !ws) return QM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return QM_ERR_ALIGNMENT;
  if (ws_bytes < stats_workspace_bytes()) return QM_ERR_WORKSPACE_TOO_SMALL;
  return launch_tensor_stats(v, out, ws, static_cast<cudaStream_t>(stream));
}

qm_status qm_quantize_error(const qm_operand* x, int32_t fmt, int32_t gran, const float* delta,
                            qm_quant_error_result* out, void* ws, size_t ws_bytes, void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (!valid_fmt(fmt) || !valid_gran(gran) || !delta || !out || !ws) return QM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) & 255) return QM_ERR_ALIGNMENT;
  if (ws_bytes < stats_workspace_bytes()) return QM_ERR_WORKSPACE_TOO_SMALL;
  return launch_quantize_error(v, fmt, gran, delta, out, ws, static_cast<cudaStream_t>(stream));
}

// copies in, probe, record out: everything qm_probe_layer_host puts into the stream
static qm_status enqueue_host_probe(const qm_operand* L_host, const qm_operand* R_host, const qm_probe_cfg* cfg,
                                    void* l_stage, void* r_stage, qm_metric_result* out_host,
                                    qm_metric_result* out_dev, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!L_host || !R_host || !l_stage || !r_stage || !out_host || !out_dev) return QM_ERR_INVALID_ARG;
  const size_t lb = qm_operand_span_bytes(L_host), rb = qm_operand_span_bytes(R_host);
  if (lb == 0 || rb == 0) return QM_ERR_INVALID_ARG;
  QM_CUDA_OK(cudaMemcpyAsync(l_stage, L_host->data, lb, cudaMemcpyHostToDevice, s));
  QM_CUDA_OK(cudaMemcpyAsync(r_stage, R_host->data, rb, cudaMemcpyHostToDevice, s));
  qm_operand L = *L_host, R = *R_host;
  L.data = l_stage; R.data = r_stage;
  qm_status st = qm_probe_layer(&L, &R, cfg, out_dev, ws, ws_bytes, s);
  if (st != QM_OK) return st;
  QM_CUDA_OK(cudaMemcpyAsync(out_host, out_dev, sizeof(qm_metric_result), cudaMemcpyDeviceToHost, s));
  return QM_OK;
}

static qm_status host_record_status(const qm_metric_result* r) {
  if (r->device_error & QM_DEVERR_TIMEOUT) return QM_ERR_TIMEOUT;
  if (r->device_error & QM_DEVERR_NONFINITE) return QM_ERR_NONFINITE_INPUT;
  return QM_OK;
}

qm_status qm_probe_layer_host(const qm_operand* L_host, const qm_operand* R_host, const qm_probe_cfg* cfg,
                              void* l_stage, void* r_stage, qm_metric_result* out_host,
                              qm_metric_result* out_dev, void* ws, size_t ws_bytes, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  qm_status st = enqueue_host_probe(L_host, R_host, cfg, l_stage, r_stage, out_host, out_dev, ws, ws_bytes, s);
  if (st != QM_OK) return st;
  QM_CUDA_OK(cudaStreamSynchronize(s));
  return host_record_status(out_host);
}

}  // extern "C"

// ---- batches of probes over the library's own streams ------------------------------------------
namespace {
constexpr int kBatchStreams = 8;      // streams of the pool
constexpr int kHostBatchStreams = 3;  // of which the host-operand batches use this many
struct BatchStreams {
  std::mutex issue;            // one batch at a time is put into the streams (host side only)
  bool ready = false;
  cudaStream_t s[kBatchStreams];
  cudaEvent_t fork, join[kBatchStreams];
};
// One set per device, created on first use (never inside a stream capture) and kept.
qm_status batch_streams(BatchStreams** out) {
  static BatchStreams pool[kMaxDevices];
  static std::mutex mu;
  const int dev = current_device();
  if (dev < 0) return QM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  BatchStreams& b = pool[dev];
  if (!b.ready) {
    for (int i = 0; i < kBatchStreams; ++i) {
      QM_CUDA_OK(cudaStreamCreateWithFlags(&b.s[i], cudaStreamNonBlocking));
      QM_CUDA_OK(cudaEventCreateWithFlags(&b.join[i], cudaEventDisableTiming));
    }
    QM_CUDA_OK(cudaEventCreateWithFlags(&b.fork, cudaEventDisableTiming));
    b.ready = true;
  }
  *out = &b;
  return QM_OK;
}

// The earlier probe (j < i) of a batch whose operand on side `side` (0 = L, 1 = R) is the very
// tensor of probe i's, scaled in the same groups, and that has prepared it itself through the
// absmax -> quantize route (so that its max|x| array exists); -1 if there is none.
int find_lender(const qm_operand* ops, const qm_probe_cfg* cfg, int i, int side, const std::vector<int>& lender) {
  const qm_operand& x = ops[i];
  const int gran = side ? cfg[i].gran_r : cfg[i].gran_l;
  const int groups = side ? cfg[i].batch_groups_r : cfg[i].batch_groups_l;
  const bool grouped = gran == QM_GRAN_CHANNEL && groups > 0 && groups < x.batch;
  // per-channel scales of a contiguous contraction take the single-pass kernel, which keeps no maxima
  if (gran == QM_GRAN_CHANNEL && !grouped && (x.stride_c == 1 || x.contract == 1)) return -1;
  for (int j = 0; j < i; ++j) {
    if (cfg[j].ref != QM_REF_BF16_FP32ACC || lender[2 * j + side] >= 0) continue;
    const qm_operand& y = ops[j];
    const int gj = side ? cfg[j].gran_r : cfg[j].gran_l, pj = side ? cfg[j].batch_groups_r : cfg[j].batch_groups_l;
    if (y.data == x.data && y.dtype == x.dtype && y.noncontract == x.noncontract && y.contract == x.contract &&
        y.stride_nc == x.stride_nc && y.stride_c == x.stride_c && y.batch == x.batch &&
        y.stride_batch == x.stride_batch && gj == gran && pj == groups)
      return j;
  }
  return -1;
}

// Runs issue(i, stream_i) for i < n round-robin over the library's streams, between a fork from
// and a join back into the caller's stream.  The join happens even when a probe was refused.
template <typename F>
qm_status run_batch(int32_t n, cudaStream_t user, F issue) {
  if (n < 0) return QM_ERR_INVALID_ARG;
  if (n == 0) return QM_OK;
  BatchStreams* b = nullptr;
  qm_status st = batch_streams(&b);
  if (st != QM_OK) return st;
  const int used = n < kHostBatchStreams ? n : kHostBatchStreams;
  // the fork and join events are reused by every call: calls from several host threads take turns
  std::lock_guard<std::mutex> lock(b->issue);
  QM_CUDA_OK(cudaEventRecord(b->fork, user));
  for (int j = 0; j < used; ++j) QM_CUDA_OK(cudaStreamWaitEvent(b->s[j], b->fork, 0));
  for (int32_t i = 0; i < n && st == QM_OK; ++i) st = issue(i, b->s[i % kHostBatchStreams]);
  for (int j = 0; j < used; ++j) {
    QM_CUDA_OK(cudaEventRecord(b->join[j], b->s[j]));
    QM_CUDA_OK(cudaStreamWaitEvent(user, b->join[j], 0));
  }
  return st;
}
}  // namespace

extern "C" {

qm_status qm_probe_batch(int32_t n, const qm_operand* L, const qm_operand* R, const qm_probe_cfg* cfg,
                         qm_metric_result* out, void* const* ws, const size_t* ws_bytes, void* stream) {
  if (n > 0 && (!L || !R || !cfg || !out || !ws || !ws_bytes)) return QM_ERR_INVALID_ARG;
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  if (n < 0) return QM_ERR_INVALID_ARG;
  if (n == 0) return QM_OK;
  BatchStreams* b = nullptr;
  qm_status st = batch_streams(&b);
  if (st != QM_OK) return st;
  std::lock_guard<std::mutex> lock(b->issue);
  // Scale + quantize of every OPERAND is a chain of two or three short, latency-bound kernels, and
  // all 2n chains are independent: the workspace words of every probe are cleared on the caller's
  // stream, then the chains are spread over the library's streams so that they run beside one
  // another.  Probes that do not take the fused tensor-core kernel (fp32 reference) run whole on
  // one of those streams.  A refused probe ends the issue there; the ones before it complete.
  std::vector<int32_t> fused;
  int32_t good = 0;
  ClearList clears{};
  for (; good < n && st == QM_OK; ++good)
    if (cfg[good].ref == QM_REF_BF16_FP32ACC)
      st = probe_phases(&L[good], &R[good], &cfg[good], out + good, ws[good], ws_bytes[good], user, kClear, nullptr,
                        nullptr, nullptr, &clears);
  if (st != QM_OK) --good;
  if (clears.n > 0) {
    const qm_status e = launch_clear_many(clears, user);
    if (e != QM_OK) return e;
  }
  QM_CUDA_OK(cudaEventRecord(b->fork, user));
  const int used = 2 * good < kBatchStreams ? 2 * good : kBatchStreams;
  for (int j = 0; j < used; ++j) QM_CUDA_OK(cudaStreamWaitEvent(b->s[j], b->fork, 0));
  // One chunk: all chains, then the caller's stream waits for the library's streams and takes the
  // fused kernels as one persistent launch.  (Two chunks, the second one's chains running under
  // the first one's launch, measured slower: the chains wait for the SMs the launch holds.)
  const int32_t chunk = good;
  std::vector<OperandShare> own(2 * (size_t)n);
  std::vector<int> lender(2 * (size_t)n, -1);     // per operand: the probe it borrows from, or -1
  std::vector<ProbeShare> shares((size_t)n);
  std::vector<TcProbeArgs> args;
  for (int32_t c0 = 0; c0 < good; c0 += chunk) {
    const int32_t c1 = c0 + chunk < good ? c0 + chunk : good;
    fused.clear();
    for (int32_t i = c0; i < c1; ++i) {
      cudaStream_t sl = b->s[(2 * i) % kBatchStreams], sr = b->s[(2 * i + 1) % kBatchStreams];
      qm_status e;
      if (cfg[i].ref == QM_REF_BF16_FP32ACC) {
        // An operand that an earlier probe of the batch has already prepared (the same tensor under
        // the same scale grouping: a sweep of formats over one layer) borrows that probe's max|x|,
        // |x| copy and contraction-major copy and only quantizes, on the lender's stream.
        ProbeShare sh;
        sh.own_l = &own[2 * i]; sh.own_r = &own[2 * i + 1];
        const int dl_i = find_lender(L, cfg, i, 0, lender), dr_i = find_lender(R, cfg, i, 1, lender);
        lender[2 * i] = dl_i; lender[2 * i + 1] = dr_i;
        if (dl_i >= 0) { sh.from_l = &own[2 * dl_i]; sl = b->s[(2 * dl_i) % kBatchStreams]; }
        if (dr_i >= 0) { sh.from_r = &own[2 * dr_i + 1]; sr = b->s[(2 * dr_i + 1) % kBatchStreams]; }
        shares[i] = sh;
        e = probe_phases(&L[i], &R[i], &cfg[i], out + i, ws[i], ws_bytes[i], sl, kPrepareL, nullptr, nullptr, &sh);
        if (e == QM_OK)
          e = probe_phases(&L[i], &R[i], &cfg[i], out + i, ws[i], ws_bytes[i], sr, kPrepareR, nullptr, nullptr, &sh);
        if (e == QM_OK) fused.push_back(i);
      } else {
        e = probe_phases(&L[i], &R[i], &cfg[i], out + i, ws[i], ws_bytes[i], sl, kPrepare | kProducts, nullptr, nullptr);
      }
      if (e != QM_OK && st == QM_OK) st = e;
    }
    for (int j = 0; j < used; ++j) {
      QM_CUDA_OK(cudaEventRecord(b->join[j], b->s[j]));
      QM_CUDA_OK(cudaStreamWaitEvent(user, b->join[j], 0));
    }
    // up to tc_group_max() probes per persistent launch
    auto flush_group = [&]() -> qm_status {
      if (args.empty()) return QM_OK;
      const qm_status e = args.size() == 1 ? launch_tc_probe(args[0], user)
                                           : launch_tc_probe_group(args.data(), (int)args.size(), user);
      args.clear();
      return e;
    };
    for (int32_t i : fused) {
      TcProbeArgs p{};
      bool deferred = false;
      const qm_status e = probe_phases(&L[i], &R[i], &cfg[i], out + i, ws[i], ws_bytes[i], user, kProducts, &p, &deferred,
                                       &shares[i]);
      if (e != QM_OK) { if (st == QM_OK) st = e; continue; }
      if (deferred) args.push_back(p);
      if ((int)args.size() == tc_group_max()) {
        const qm_status g = flush_group();
        if (g != QM_OK && st == QM_OK) st = g;
      }
    }
    const qm_status g = flush_group();
    if (g != QM_OK && st == QM_OK) st = g;
  }
  return st;
}

qm_status qm_probe_batch_host(int32_t n, const qm_operand* L_host, const qm_operand* R_host,
                              const qm_probe_cfg* cfg, void* const* l_stage, void* const* r_stage,
                              qm_metric_result* out_host, qm_metric_result* out_dev, void* const* ws,
                              const size_t* ws_bytes, void* stream) {
  if (n > 0 && (!L_host || !R_host || !cfg || !l_stage || !r_stage || !out_host || !out_dev || !ws || !ws_bytes))
    return QM_ERR_INVALID_ARG;
  if (n == 0) return QM_OK;
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  int32_t issued = 0;
  qm_status st = run_batch(n, user, [&](int32_t i, cudaStream_t s) {
    qm_status e = enqueue_host_probe(&L_host[i], &R_host[i], &cfg[i], l_stage[i], r_stage[i], out_host + i,
                                     out_dev + i, ws[i], ws_bytes[i], s);
    if (e == QM_OK) ++issued;
    return e;
  });
  QM_CUDA_OK(cudaStreamSynchronize(user));
  if (st != QM_OK) return st;
  for (int32_t i = 0; i < issued; ++i) {
    st = host_record_status(out_host + i);
    if (st != QM_OK) return st;
  }
  return QM_OK;
}

const char* qm_status_string(int32_t st) {
  switch (st) {
    case QM_OK: return "ok";
    case QM_ERR_INVALID_ARG: return "invalid argument";
    case QM_ERR_UNSUPPORTED: return "unsupported configuration";
    case QM_ERR_ALIGNMENT: return "alignment";
    case QM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case QM_ERR_NONFINITE_INPUT: return "non-finite input";
    case QM_ERR_CUDA: return "CUDA error";
    case QM_ERR_TIMEOUT: return "device wait timed out";
    default: return "unknown status";
  }
}

int32_t qm_version(void) { return 100; }

const char* qm_last_cuda_error(void) { return qm::g_last_error; }

int64_t qm_kernel_launches(void) { return (int64_t)qm::g_launches.load(); }

qm_status qm_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> lock(qm::g_prof_mutex);
  qm::g_prof_on = on != 0;
  qm::g_prof_used = 0;
  return QM_OK;
}

qm_status qm_profile_samples(double* start_ms, double* dur_ms, int32_t cap, int32_t* launches) {
  if (!start_ms || !dur_ms || !launches || cap < 0) return QM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(qm::g_prof_mutex);
  const int32_t n = (int32_t)(qm::g_prof_used / 2);
  for (int32_t i = 0; i < n && i < cap; ++i) {
    QM_CUDA_OK(cudaEventSynchronize(qm::g_prof_events[2 * i + 1]));
    float t0 = 0, t1 = 0;
    QM_CUDA_OK(cudaEventElapsedTime(&t0, qm::g_prof_events[0], qm::g_prof_events[2 * i]));
    QM_CUDA_OK(cudaEventElapsedTime(&t1, qm::g_prof_events[2 * i], qm::g_prof_events[2 * i + 1]));
    start_ms[i] = t0; dur_ms[i] = t1;
  }
  *launches = n;
  return QM_OK;
}

qm_status qm_profile_read(double* ms, int32_t* launches) {
  if (!ms || !launches) return QM_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(qm::g_prof_mutex);
  double total = 0;
  for (size_t i = 0; i + 1 < qm::g_prof_used; i += 2) {
    QM_CUDA_OK(cudaEventSynchronize(qm::g_prof_events[i + 1]));
    float t = 0;
    QM_CUDA_OK(cudaEventElapsedTime(&t, qm::g_prof_events[i], qm::g_prof_events[i + 1]));
    total += t;
  }
  *ms = total;
  *launches = (int32_t)(qm::g_prof_used / 2);
  qm::g_prof_used = 0;
  return QM_OK;
}

}  // extern "C"
