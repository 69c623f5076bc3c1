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

// with_abs: room for the bf16 |x| copies (only the two-format kernel still loads them)
Workspace plan(const View& L, const View& R, const qm_probe_cfg& cfg, bool with_abs = false) {
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
    if (with_abs) {
      w.off_al = take((size_t)(L.batch * L.nc * L.c) * 2);
      w.off_ar = take((size_t)(R.batch * R.nc * R.c) * 2);
    }
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

qm_status qm_quantize_formats(const qm_operand* x, int32_t n_fmt, const int32_t* fmts, int32_t gran,
                              float* const* delta_out, uint8_t* const* codes, void* kmaj_copy,
                              uint32_t* amax_scratch, void* stream) {
  View v;
  qm_status st = to_view(x, &v);
  if (st != QM_OK) return st;
  if (n_fmt < 1 || n_fmt > 3 || !fmts || !valid_gran(gran) || !delta_out || !codes || !amax_scratch) return QM_ERR_INVALID_ARG;
  int f[3]; float* d[3]; uint8_t* c[3]; uint32_t* e[3] = {nullptr, nullptr, nullptr};
  for (int k = 0; k < n_fmt; ++k) {
    if (!valid_fmt(fmts[k]) || !delta_out[k] || !codes[k]) return QM_ERR_INVALID_ARG;
    for (int j = 0; j < k; ++j)
      if (fmts[j] == fmts[k]) return QM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(codes[k]) & 15) return QM_ERR_ALIGNMENT;
    f[k] = fmts[k]; d[k] = delta_out[k]; c[k] = codes[k];
  }
  if (reinterpret_cast<uintptr_t>(kmaj_copy) & 15) return QM_ERR_ALIGNMENT;
  if (kmaj_copy && v.dtype != QM_DT_BF16) return QM_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  QM_CUDA_OK(cudaMemsetAsync(amax_scratch, 0, sizeof(uint32_t) * delta_count(v, gran), s));
  st = launch_absmax(v, gran, amax_scratch, s);
  if (st != QM_OK) return st;
  return launch_quantize_multi(v, gran, amax_scratch, n_fmt, f, d, e, c, kmaj_copy, s);
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

// The probe in phases that may be issued apart (same arguments every time): kClear clears the
// workspace words (or only lists them in *clear_later, for one clearing kernel over a batch),
// kPrepareL / kPrepareR run scale + quantize of one operand (after kClear), kProducts the
// products and the Eq. 3 reduction (after both).
enum { kClear = 1, kPrepareL = 2, kPrepareR = 4, kPrepare = kClear | kPrepareL | kPrepareR, kProducts = 8 };
static qm_status probe_phases(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg,
                              qm_metric_result* out, void* ws, size_t ws_bytes, void* stream, int phases,
                              ClearList* clear_later = nullptr) {
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
  // the fused kernel forms |L| and |R| tiles in shared memory: no |x| copy is written
  void* al = nullptr;
  void* ar = nullptr;
  void* kl = (w.tc && !L.c_contig()) ? base + w.off_kl : nullptr;
  void* kr = (w.tc && !R.c_contig()) ? base + w.off_kr : nullptr;
  const StochasticDraw draw_l{cfg->seed, 0u}, draw_r{cfg->seed, 1u};
  const StochasticDraw* dl_draw = (cfg->round & QM_ROUND_STOCHASTIC_L) ? &draw_l : nullptr;
  const StochasticDraw* dr_draw = (cfg->round & QM_ROUND_STOCHASTIC_R) ? &draw_r : nullptr;
  if (phases & kPrepareL) {
    st = prepare_operand(L, cfg->fmt_l, cfg->gran_l, ml, dl, cl, al, kl, err, dl_draw, cfg->batch_groups_l, s);
    if (st != QM_OK) return st;
  }
  if (phases & kPrepareR) {
    st = prepare_operand(R, cfg->fmt_r, cfg->gran_r, mr, dr, cr, ar, kr, err, dr_draw, cfg->batch_groups_r, s);
    if (st != QM_OK) return st;
  }
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
    return launch_tc_probe(p, s);           // the last CTA writes the record
  }
  st = launch_simt_probe(L, R, cl, cfg->fmt_l, dl, cfg->gran_l, cr, cfg->fmt_r, dr, cfg->gran_r, part, s);
  if (st != QM_OK) return st;
  return launch_metric_finalize(part, w.n_part, (uint64_t)(g.M * g.N * g.batch), err, out, s);
}

qm_status qm_probe_layer(const qm_operand* Lo, const qm_operand* Ro, const qm_probe_cfg* cfg,
                         qm_metric_result* out, void* ws, size_t ws_bytes, void* stream) {
  return probe_phases(Lo, Ro, cfg, out, ws, ws_bytes, stream, kPrepare | kProducts);
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
  w.a = plan(L, R, first, true);
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
constexpr int kCopyEvents = 64;       // chunks of a host batch that can wait for their own copies
struct BatchStreams {
  std::mutex issue;            // one batch at a time is put into the streams (host side only)
  bool ready = false;
  cudaStream_t s[kBatchStreams];
  cudaEvent_t fork, join[kBatchStreams];
  std::mutex host_issue;       // one host batch at a time uses the copy stream and its events
  cudaStream_t copy;           // host batches: the host-to-device copies, beside the probes of earlier chunks
  cudaEvent_t copy_fork, copied[kCopyEvents];
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
    QM_CUDA_OK(cudaStreamCreateWithFlags(&b.copy, cudaStreamNonBlocking));
    QM_CUDA_OK(cudaEventCreateWithFlags(&b.copy_fork, cudaEventDisableTiming));
    for (int i = 0; i < kCopyEvents; ++i) QM_CUDA_OK(cudaEventCreateWithFlags(&b.copied[i], cudaEventDisableTiming));
    b.ready = true;
  }
  *out = &b;
  return QM_OK;
}

// One operand of one tensor-core probe of a batch: what has to be prepared, where this probe's own
// buffers for it are, and whose results it uses.  Preparing an operand leaves four things behind:
// the max|x| bit patterns, the contraction-major bf16 copy (strided contraction only), the
// scales and the codes.  A sweep of formats over a layer, and a layer whose activations feed
// several products, ask for the same things many times over; inside a batch each is made once:
//   code_root: the earlier operand with the same view, scale grouping, format and rounding: its
//              scales, codes and copy are used as they are and nothing is launched;
//   copy_root: the earlier operand with the same view and scale grouping under another format:
//              its max|x| and contraction-major copy are borrowed, only the codes are made;
//   amax_root: per-tensor scales only: the earlier operand over the same elements in either
//              orientation (max|x| does not depend on which dimension contracts).
// A root index equal to the slot's own index means "makes it itself".
struct Slot {
  View v;
  int fmt, gran, groups;
  bool stochastic;
  StochasticDraw draw;
  uint32_t* amax; float* delta; uint8_t* codes; void* kmaj; uint32_t* err;
  bool keeps_amax;                 // false when the single-pass per-row kernel prepares it (no maxima are stored)
  int code_root, copy_root, amax_root;
  int stream;                      // index of the library stream its kernels go to
};

bool same_view(const View& a, const View& b) {
  return a.data == b.data && a.dtype == b.dtype && a.nc == b.nc && a.c == b.c && a.s_nc == b.s_nc && a.s_c == b.s_c &&
         a.batch == b.batch && a.s_b == b.s_b;
}
// the same elements with the two matrix dimensions exchanged
bool transposed_view(const View& a, const View& b) {
  return a.data == b.data && a.dtype == b.dtype && a.nc == b.c && a.c == b.nc && a.s_nc == b.s_c && a.s_c == b.s_nc &&
         a.batch == b.batch && a.s_b == b.s_b;
}
bool grouped_scales(const Slot& x) { return x.gran == QM_GRAN_CHANNEL && x.groups > 0 && x.groups < x.v.batch; }

void find_roots(std::vector<Slot>& slots, int t) {
  Slot& x = slots[t];
  x.code_root = x.copy_root = x.amax_root = t;
  const int gx = grouped_scales(x) ? x.groups : 0;
  for (int u = 0; u < t; ++u) {
    const Slot& y = slots[u];
    if (y.code_root != u || !same_view(x.v, y.v) || y.gran != x.gran || (grouped_scales(y) ? y.groups : 0) != gx) continue;
    const bool same_round = x.stochastic == y.stochastic &&
                            (!x.stochastic || (x.draw.seed == y.draw.seed && x.draw.stream == y.draw.stream));
    if (y.fmt == x.fmt && same_round) { x.code_root = u; x.copy_root = y.copy_root; x.amax_root = y.amax_root; return; }
  }
  for (int u = 0; u < t; ++u) {
    const Slot& y = slots[u];
    if (y.code_root != u || y.copy_root != u || !y.keeps_amax) continue;
    if (same_view(x.v, y.v) && y.gran == x.gran && (grouped_scales(y) ? y.groups : 0) == gx) {
      x.copy_root = u; x.amax_root = y.amax_root;
      return;
    }
  }
  if (x.gran != QM_GRAN_TENSOR) return;
  for (int u = 0; u < t; ++u) {
    const Slot& y = slots[u];
    if (y.code_root != u || y.copy_root != u || y.amax_root != u || y.gran != QM_GRAN_TENSOR) continue;
    if (same_view(x.v, y.v) || transposed_view(x.v, y.v)) { x.amax_root = u; return; }
  }
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
  // Pass 1 (host only): check every probe, lay out its workspace, list the control words to clear
  // and describe the two operands of every tensor-core probe.  A refused probe ends the batch
  // there; the ones before it complete.
  struct Planned { View Lv, Rv; Workspace w; bool tc; };
  std::vector<Planned> plans;
  std::vector<Slot> slots;
  std::vector<int> slot_of((size_t)n, -1);            // probe -> index of its left operand's slot
  ClearList clears{};
  int32_t good = 0;
  qm_status refused = QM_OK;                          // why probe `good` was not taken, if one was not
  for (; good < n; ++good) {
    const int32_t i = good;
    Planned pl{};
    refused = check_probe(&L[i], &R[i], &cfg[i], &pl.Lv, &pl.Rv);
    if (refused == QM_OK && (!ws[i] || (reinterpret_cast<uintptr_t>(ws[i]) & 255)))
      refused = ws[i] ? QM_ERR_ALIGNMENT : QM_ERR_INVALID_ARG;
    if (refused != QM_OK) break;
    pl.w = plan(pl.Lv, pl.Rv, cfg[i]);
    pl.tc = pl.w.tc;
    if (ws_bytes[i] < pl.w.total) { refused = QM_ERR_WORKSPACE_TOO_SMALL; break; }
    plans.push_back(pl);
    if (!pl.tc) continue;
    uint8_t* base = static_cast<uint8_t*>(ws[i]);
    if (clears.n == kClearMax) {
      const qm_status e = launch_clear_many(clears, user);
      if (e != QM_OK) return e;
      clears.n = 0;
    }
    clears.ptr[clears.n] = base;                       // error word, CTA counter and both max|x| buffers are adjacent
    clears.words[clears.n++] = (uint32_t)(pl.w.off_dl / 4);
    if (cfg[i].row_stats)
      QM_CUDA_OK(cudaMemsetAsync(cfg[i].row_stats, 0, sizeof(double) * QM_ROW_STATS * (size_t)(pl.Lv.batch * pl.Lv.nc), user));
    slot_of[i] = (int)slots.size();
    for (int side = 0; side < 2; ++side) {
      const View& v = side ? pl.Rv : pl.Lv;
      Slot x{};
      x.v = v;
      x.fmt = side ? cfg[i].fmt_r : cfg[i].fmt_l;
      x.gran = side ? cfg[i].gran_r : cfg[i].gran_l;
      x.groups = side ? cfg[i].batch_groups_r : cfg[i].batch_groups_l;
      x.stochastic = (cfg[i].round & (side ? QM_ROUND_STOCHASTIC_R : QM_ROUND_STOCHASTIC_L)) != 0;
      x.draw = StochasticDraw{cfg[i].seed, (uint32_t)side};
      x.amax = reinterpret_cast<uint32_t*>(base + (side ? pl.w.off_mr : pl.w.off_ml));
      x.delta = reinterpret_cast<float*>(base + (side ? pl.w.off_dr : pl.w.off_dl));
      x.codes = base + (side ? pl.w.off_cr : pl.w.off_cl);
      x.kmaj = v.c_contig() ? nullptr : base + (side ? pl.w.off_kr : pl.w.off_kl);
      // words 2 and 3 of the control block: "this operand is not finite", raised by the kernel that scales it
      x.err = reinterpret_cast<uint32_t*>(base + pl.w.off_err) + 2 + side;
      x.keeps_amax = !(!x.stochastic && !grouped_scales(x) && x.gran == QM_GRAN_CHANNEL && v.c_contig());
      slots.push_back(x);
      find_roots(slots, (int)slots.size() - 1);
    }
  }
  if (clears.n > 0) {
    const qm_status e = launch_clear_many(clears, user);
    if (e != QM_OK) return e;
  }
  // Pass 2: the scale / quantize chains.  Each chain is two or three short kernels and the chains
  // of different tensors are independent, so they are spread over the library's streams and run
  // beside one another; whatever borrows from an earlier operand goes to that operand's stream,
  // behind the kernels that make what it borrows.  Probes that do not take the fused tensor-core
  // kernel (fp32 reference) run whole on one of those streams.
  QM_CUDA_OK(cudaEventRecord(b->fork, user));
  for (int j = 0; j < kBatchStreams; ++j) QM_CUDA_OK(cudaStreamWaitEvent(b->s[j], b->fork, 0));
  int next_stream = 0;
  std::vector<char> done(slots.size(), 0);
  for (size_t t = 0; t < slots.size(); ++t) {
    Slot& x = slots[t];
    if (x.code_root != (int)t) { x.stream = slots[x.code_root].stream; continue; }     // nothing to launch
    if (done[t]) continue;
    qm_status e = QM_OK;
    const StochasticDraw* draw = x.stochastic ? &x.draw : nullptr;
    if (x.copy_root != (int)t) {
      // borrows max|x| and the contraction-major copy, and was not served with its lender's formats
      x.stream = slots[x.copy_root].stream;
      e = launch_quantize(x.v, x.fmt, x.gran, reinterpret_cast<const float*>(slots[x.amax_root].amax), true, x.delta, x.err,
                          x.codes, nullptr, nullptr, b->s[x.stream], draw);
    } else if (!x.keeps_amax) {
      x.stream = next_stream; next_stream = (next_stream + 1) % kBatchStreams;
      e = prepare_operand(x.v, x.fmt, x.gran, x.amax, x.delta, x.codes, nullptr, x.kmaj, x.err, draw, x.groups, b->s[x.stream]);
    } else {
      if (x.amax_root == (int)t) {
        x.stream = next_stream; next_stream = (next_stream + 1) % kBatchStreams;
        e = launch_absmax(x.v, x.gran, x.amax, b->s[x.stream]);
        if (e == QM_OK && grouped_scales(x)) e = launch_share_amax(x.amax, x.v.batch, x.groups, x.v.nc, b->s[x.stream]);
      } else {
        x.stream = slots[x.amax_root].stream;
      }
      cudaStream_t s = b->s[x.stream];
      const uint32_t* amax = slots[x.amax_root].amax;
      // this operand's format and those of the later operands that borrow its copy: one pass over
      // the tensor writes all their codes (round-to-nearest-even ones; stochastic ones go singly)
      int fmts[3]; float* deltas[3]; uint32_t* errs[3]; uint8_t* codes[3];
      int nf = 0;
      bool kmaj_written = false;
      if (!x.stochastic) { fmts[nf] = x.fmt; deltas[nf] = x.delta; errs[nf] = x.err; codes[nf] = x.codes; ++nf; }
      for (size_t u = t + 1; u < slots.size() && nf < 3; ++u) {
        Slot& y = slots[u];
        if (y.code_root != (int)u || y.copy_root != (int)t || y.stochastic || done[u]) continue;
        bool dup = false;
        for (int k = 0; k < nf; ++k) dup |= fmts[k] == y.fmt;
        if (dup) continue;
        fmts[nf] = y.fmt; deltas[nf] = y.delta; errs[nf] = y.err; codes[nf] = y.codes; ++nf;
        y.stream = x.stream; done[u] = 1;
      }
      if (e == QM_OK && x.stochastic) {
        e = launch_quantize(x.v, x.fmt, x.gran, reinterpret_cast<const float*>(amax), true, x.delta, x.err, x.codes, nullptr,
                            x.kmaj, s, draw);
        kmaj_written = true;
      }
      if (e == QM_OK && nf > 0)
        e = launch_quantize_multi(x.v, x.gran, amax, nf, fmts, deltas, errs, codes, kmaj_written ? nullptr : x.kmaj, s);
    }
    done[t] = 1;
    if (e != QM_OK && st == QM_OK) st = e;
  }
  for (int32_t i = 0; i < good; ++i) {
    if (plans[i].tc) continue;
    cudaStream_t s = b->s[next_stream]; next_stream = (next_stream + 1) % kBatchStreams;
    const qm_status e = probe_phases(&L[i], &R[i], &cfg[i], out + i, ws[i], ws_bytes[i], s, kPrepare | kProducts);
    if (e != QM_OK && st == QM_OK) st = e;
  }
  for (int j = 0; j < kBatchStreams; ++j) {
    QM_CUDA_OK(cudaEventRecord(b->join[j], b->s[j]));
    QM_CUDA_OK(cudaStreamWaitEvent(user, b->join[j], 0));
  }
  // Pass 3: the caller's stream has waited for every chain; the fused kernels go to it as
  // persistent launches of up to tc_group_max() probes.  (Running a second chunk's chains under
  // the first chunk's launch measured slower: the chains wait for the SMs the launch holds.)
  std::vector<TcProbeArgs> args;
  auto flush_group = [&]() -> qm_status {
    if (args.empty()) return QM_OK;
    const qm_status e = launch_tc_probe_group(args.data(), (int)args.size(), user);
    args.clear();
    return e;
  };
  for (int32_t i = 0; i < good && st == QM_OK; ++i) {
    if (!plans[i].tc) continue;
    const Planned& pl = plans[i];
    uint8_t* base = static_cast<uint8_t*>(ws[i]);
    const Slot& xl = slots[slot_of[i]];
    const Slot& xr = slots[slot_of[i] + 1];
    const Slot& cl = slots[xl.code_root];
    const Slot& cr = slots[xr.code_root];
    void* kl = slots[cl.copy_root].kmaj;
    void* kr = slots[cr.copy_root].kmaj;
    TcProbeArgs p{};
    p.l = kl ? kl : pl.Lv.data; p.l_ld = kl ? pl.Lv.c : pl.Lv.s_nc; p.l_sb = kl ? pl.Lv.nc * pl.Lv.c : pl.Lv.s_b;
    p.r = kr ? kr : pl.Rv.data; p.r_ld = kr ? pl.Rv.c : pl.Rv.s_nc; p.r_sb = kr ? pl.Rv.nc * pl.Rv.c : pl.Rv.s_b;
    p.cl = cl.codes; p.cr = cr.codes;
    p.fmt_l = cfg[i].fmt_l; p.fmt_r = cfg[i].fmt_r;
    p.dl = cl.delta; p.gran_l = cfg[i].gran_l; p.dr = cr.delta; p.gran_r = cfg[i].gran_r;
    p.g = GemmShape{pl.Lv.nc, pl.Rv.nc, pl.Lv.c, pl.Lv.batch};
    p.partials = reinterpret_cast<double*>(base + pl.w.off_part);
    p.err_word = reinterpret_cast<uint32_t*>(base + pl.w.off_err);
    p.done_counter = p.err_word + 1;        // second word of the cleared control block
    // a non-finite operand is flagged in the control block of the probe whose kernel scaled it
    p.err_also[0] = cl.err;
    p.err_also[1] = cr.err;
    p.result = out + i;
    p.row_stats = cfg[i].row_stats;
    args.push_back(p);
    if ((int)args.size() == tc_group_max()) {
      const qm_status g = flush_group();
      if (g != QM_OK && st == QM_OK) st = g;
    }
  }
  const qm_status g = flush_group();
  if (g != QM_OK && st == QM_OK) st = g;
  return st != QM_OK ? st : refused;
}

// Which host operands of a host batch are copied: an operand whose host bytes an earlier operand of
// the batch has already brought to the device (same address, same extent) uses that copy.
namespace {
struct HostCopy { const void* host; size_t bytes; void* dev; };
void* find_copy(const std::vector<HostCopy>& seen, const void* host, size_t bytes) {
  for (const HostCopy& c : seen)
    if (c.host == host && c.bytes == bytes) return c.dev;
  return nullptr;
}
}  // namespace

qm_status qm_probe_batch_host_bytes(int32_t n, const qm_operand* L_host, const qm_operand* R_host, size_t* h2d_bytes,
                                    size_t* d2h_bytes) {
  if (n < 0 || (n > 0 && (!L_host || !R_host)) || !h2d_bytes || !d2h_bytes) return QM_ERR_INVALID_ARG;
  std::vector<HostCopy> seen;
  size_t total = 0;
  for (int32_t i = 0; i < n; ++i)
    for (int side = 0; side < 2; ++side) {
      const qm_operand& x = side ? R_host[i] : L_host[i];
      const size_t bytes = qm_operand_span_bytes(&x);
      if (bytes == 0) return QM_ERR_INVALID_ARG;
      if (find_copy(seen, x.data, bytes)) continue;
      seen.push_back(HostCopy{x.data, bytes, const_cast<void*>(x.data)});
      total += bytes;
    }
  *h2d_bytes = total;
  *d2h_bytes = sizeof(qm_metric_result) * (size_t)n;
  return QM_OK;
}

qm_status qm_probe_batch_host(int32_t n, const qm_operand* L_host, const qm_operand* R_host,
                              const qm_probe_cfg* cfg, void* const* l_stage, void* const* r_stage,
                              qm_metric_result* out_host, qm_metric_result* out_dev, void* const* ws,
                              const size_t* ws_bytes, void* stream) {
  if (n > 0 && (!L_host || !R_host || !cfg || !l_stage || !r_stage || !out_host || !out_dev || !ws || !ws_bytes))
    return QM_ERR_INVALID_ARG;
  if (n < 0) return QM_ERR_INVALID_ARG;
  if (n == 0) return QM_OK;
  cudaStream_t user = static_cast<cudaStream_t>(stream);
  BatchStreams* bs = nullptr;
  qm_status st = batch_streams(&bs);
  if (st != QM_OK) return st;
  // Every distinct host operand is copied once, on a stream of the library's own and in the order
  // in which the probes first name them.  The probes go to the device in chunks of one fused
  // launch's worth, each chunk as a device batch (which prepares every distinct operand of the
  // chunk once) that waits only for the copies it needs: the copies of later chunks run under the
  // kernels of earlier ones.  Order the probes so that those of one product are neighbours and the
  // first chunks need only the first tensors.
  std::vector<qm_operand> Ld((size_t)n), Rd((size_t)n);
  std::vector<HostCopy> seen;
  const int32_t chunk = tc_group_max();
  const bool pipelined = (n + chunk - 1) / chunk <= kCopyEvents;
  std::lock_guard<std::mutex> lock(bs->host_issue);
  QM_CUDA_OK(cudaEventRecord(bs->copy_fork, user));               // the copies follow the work already in the stream
  QM_CUDA_OK(cudaStreamWaitEvent(bs->copy, bs->copy_fork, 0));
  qm_status refused = QM_OK;
  int32_t good = 0, issued = 0;
  for (int32_t c0 = 0; c0 < n && st == QM_OK && refused == QM_OK; c0 += chunk) {
    const int32_t c1 = c0 + chunk < n ? c0 + chunk : n;
    for (good = c0; good < c1; ++good) {
      for (int side = 0; side < 2 && refused == QM_OK; ++side) {
        const qm_operand& x = side ? R_host[good] : L_host[good];
        void* stage = side ? r_stage[good] : l_stage[good];
        const size_t bytes = qm_operand_span_bytes(&x);
        if (bytes == 0 || !stage) { refused = QM_ERR_INVALID_ARG; break; }
        void* dev = find_copy(seen, x.data, bytes);
        if (!dev) {
          QM_CUDA_OK(cudaMemcpyAsync(stage, x.data, bytes, cudaMemcpyHostToDevice, bs->copy));
          seen.push_back(HostCopy{x.data, bytes, stage});
          dev = stage;
        }
        qm_operand& d = side ? Rd[good] : Ld[good];
        d = x;
        d.data = dev;
      }
      if (refused != QM_OK) break;
    }
    // this chunk's copies (and all earlier ones) are in the copy stream: the caller's stream waits for them
    cudaEvent_t ev = bs->copied[pipelined ? c0 / chunk : 0];
    QM_CUDA_OK(cudaEventRecord(ev, bs->copy));
    QM_CUDA_OK(cudaStreamWaitEvent(user, ev, 0));
    if (good > c0) {
      st = qm_probe_batch(good - c0, Ld.data() + c0, Rd.data() + c0, cfg + c0, out_dev + c0, ws + c0, ws_bytes + c0, user);
      if (st == QM_OK) issued = good;
    }
    if (!pipelined) QM_CUDA_OK(cudaStreamSynchronize(user));       // the one event is about to be recorded again
  }
  if (issued > 0)
    QM_CUDA_OK(cudaMemcpyAsync(out_host, out_dev, sizeof(qm_metric_result) * (size_t)issued, cudaMemcpyDeviceToHost, user));
  QM_CUDA_OK(cudaStreamSynchronize(user));
  if (st != QM_OK) return st;
  if (refused != QM_OK) return refused;
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

void qm_debug_set_wait_limit_ns(uint64_t ns) { qm::set_wait_limit_ns(ns); }
void qm_debug_stop_producer_after(uint32_t k_blocks) { qm::set_stop_after_kb(k_blocks); }

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
