// Single-tensor passes beside the probe: the baseline tensor statistics of the Experiments
// section (power sums for mean, variance, skew, kurtosis, and max|x|) and the per-element
// quantization error of Eq. 2 split into clipping (overflow, underflow) and rounding error as in
// the Results section.  Both are one HBM pass over the tensor: 128-bit loads, four loads in
// flight per thread, fp32 arithmetic per element, fp32 sums over the 32 elements of a batch of
// loads, fp64 from there on, one record per block and a fixed-order sum by the last block.
#include "quant_device.cuh"

namespace qm {
namespace {

constexpr int kRec = 10;                 // doubles per partial record
constexpr int kMaxBlocks = 2048;
constexpr size_t kCounterBytes = 256;

// A tensor as `lines` contiguous runs of `inner` elements.
struct Lines {
  const void* x;
  int64_t inner, line_stride, batch_stride;   // elements
  uint32_t groups_per_line;                   // ceil(inner / 8)
  uint32_t total_groups;
  FastDiv by_gpl, by_outer;
  uint32_t outer;                             // lines per batch element
  const float* delta;                         // Eq. 2 pass only
  int delta_mode;                             // 0: one delta; 1: one per line; 2: one per position in the line
  int64_t delta_batch;                        // deltas per batch element (modes 1, 2)
};

enum { kStats = 0, kError = 1 };

// value of one code byte
template <int FMT>
__device__ __forceinline__ void decode2(uint32_t two_codes, float& a, float& b) {
  if (FMT == QM_FMT_INT8) {
    a = (float)(int)(signed char)(two_codes & 0xff);
    b = (float)(int)(signed char)((two_codes >> 8) & 0xff);
  } else {
    uint32_t h2;
    const uint16_t c = (uint16_t)two_codes;
    if (FMT == QM_FMT_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(c));
    else asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(c));
    const __half2 h = *reinterpret_cast<__half2*>(&h2);
    a = __low2float(h);
    b = __high2float(h);
  }
}

struct Acc {
  double d[kRec];
};

// which entries of a record combine by max instead of sum
template <int KIND> __device__ __forceinline__ bool is_max(int i) { return KIND == kStats ? i == 4 : i == 9; }

template <typename T, int KIND, int FMT>
__global__ void __launch_bounds__(kThreads)
tensor_pass_kernel(const Lines p, double* __restrict__ partials, uint32_t* __restrict__ counter,
                   void* __restrict__ result, uint64_t count) {
  pdl_prologue();
  Acc acc;
#pragma unroll
  for (int i = 0; i < kRec; ++i) acc.d[i] = 0.0;
  const float qmaxv = fmt_qmax(FMT);
  const uint32_t stride = gridDim.x * kThreads;
  for (uint32_t g0 = blockIdx.x * kThreads + threadIdx.x; g0 < p.total_groups; g0 += 4 * stride) {
    Vec8 v[4];
    float dl[4][8];
    int live[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t g = g0 + u * stride;
      live[u] = 0;
      if (g < p.total_groups) {
        const uint32_t line = p.by_gpl.div(g), j = g - line * p.groups_per_line;
        const uint32_t b = p.by_outer.div(line), o = line - b * p.outer;
        const int64_t off = (int64_t)b * p.batch_stride + (int64_t)o * p.line_stride + (int64_t)j * 8;
        const int64_t left = p.inner - (int64_t)j * 8;
        live[u] = left < 8 ? (int)left : 8;
        const char* base = reinterpret_cast<const char*>(p.x) + off * (int64_t)sizeof(T);
        if (live[u] == 8) {
          v[u] = Loader<T>::load8(base);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) v[u].v[e] = e < live[u] ? Loader<T>::load1(base, e) : 0.f;
        }
        if (KIND == kError) {
          if (p.delta_mode == 2) {
            const float* d = p.delta + (int64_t)b * p.delta_batch + (int64_t)j * 8;
#pragma unroll
            for (int e = 0; e < 8; ++e) dl[u][e] = e < live[u] ? __ldg(d + e) : 1.f;
          } else {
            const float d = p.delta_mode == 0 ? __ldg(p.delta) : __ldg(p.delta + (int64_t)b * p.delta_batch + o);
#pragma unroll
            for (int e = 0; e < 8; ++e) dl[u][e] = d;
          }
        }
      }
    }
    if (KIND == kStats) {
      float s1 = 0.f, s2 = 0.f, s3 = 0.f, s4 = 0.f;
      uint32_t mx = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (live[u] == 0) continue;
        mx = absmax8(v[u], mx);          // padded entries are zero and change nothing
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x = v[u].v[e], x2 = x * x;
          s1 += x; s2 += x2; s3 = fmaf(x2, x, s3); s4 = fmaf(x2, x2, s4);
        }
      }
      acc.d[0] += (double)s1; acc.d[1] += (double)s2; acc.d[2] += (double)s3; acc.d[3] += (double)s4;
      acc.d[4] = fmax(acc.d[4], (double)mx);
    } else {
      float sre = 0.f, srr = 0.f, e2r = 0.f, e2o = 0.f, e2u = 0.f, sx2 = 0.f, mrr = 0.f;
      uint32_t nnz = 0, nov = 0, nun = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (live[u] == 0) continue;
        const bool one_delta = p.delta_mode != 2;
        const Quotient q0(dl[u][0]);
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          const float xa = v[u].v[e], xb = v[u].v[e + 1];
          const float da = dl[u][e], db = dl[u][e + 1];
          float ta, tb;
          if (one_delta) { ta = q0(xa); tb = q0(xb); }
          else { ta = Quotient(da)(xa); tb = Quotient(db)(xb); }
          float ga, gb;
          decode2<FMT>(quant2<FMT>(ta, tb), ga, gb);
          const float xs[2] = {xa, xb}, ts[2] = {ta, tb}, gs[2] = {ga, gb}, ds[2] = {da, db};
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float x = xs[h];
            if (x != 0.f) {                                   // padded entries are zero
              const float err = fabsf(fmaf(-gs[h], ds[h], x));  // |x - value(code) delta|, one rounding
              const float re = __fdividef(err, fabsf(x));
              const bool over = fabsf(ts[h]) > qmaxv;
              const bool under = !over && gs[h] == 0.f;
              ++nnz;
              sre += re;
              sx2 = fmaf(x, x, sx2);
              if (over) { ++nov; e2o = fmaf(err, err, e2o); }
              else if (under) { ++nun; e2u = fmaf(err, err, e2u); }
              else { srr += re; e2r = fmaf(err, err, e2r); mrr = fmaxf(mrr, re); }
            }
          }
        }
      }
      acc.d[0] += (double)sre; acc.d[1] += (double)srr; acc.d[2] += (double)e2r; acc.d[3] += (double)e2o;
      acc.d[4] += (double)e2u; acc.d[5] += (double)sx2; acc.d[6] += (double)nnz; acc.d[7] += (double)nov;
      acc.d[8] += (double)nun; acc.d[9] = fmax(acc.d[9], (double)mrr);
    }
  }

  // block record
  __shared__ double red[kRec][kThreads / 32];
  __shared__ uint32_t is_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < kRec; ++i) {
    double x = acc.d[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double y = __shfl_xor_sync(0xffffffffu, x, o);
      x = is_max<KIND>(i) ? fmax(x, y) : x + y;
    }
    if (lane == 0) red[i][warp] = x;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double* rec = partials + (int64_t)blockIdx.x * kRec;
    for (int i = 0; i < kRec; ++i) {
      double x = red[i][0];
      for (int w = 1; w < kThreads / 32; ++w) x = is_max<KIND>(i) ? fmax(x, red[i][w]) : x + red[i][w];
      __stcg(rec + i, x);
    }
    __threadfence();
    is_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1u : 0u;
  }
  __syncthreads();
  if (!is_last || warp != 0) return;
  __threadfence();
  double tot[kRec];
#pragma unroll
  for (int i = 0; i < kRec; ++i) tot[i] = 0.0;
  for (int b = lane; b < (int)gridDim.x; b += 32) {            // fixed order: deterministic
    const double* rec = partials + (int64_t)b * kRec;
#pragma unroll
    for (int i = 0; i < kRec; ++i) {
      const double y = __ldcg(rec + i);
      tot[i] = is_max<KIND>(i) ? fmax(tot[i], y) : tot[i] + y;
    }
  }
#pragma unroll
  for (int i = 0; i < kRec; ++i) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double y = __shfl_xor_sync(0xffffffffu, tot[i], o);
      tot[i] = is_max<KIND>(i) ? fmax(tot[i], y) : tot[i] + y;
    }
  }
  if (lane != 0) return;
  if (KIND == kStats) {
    qm_tensor_stats_result* r = static_cast<qm_tensor_stats_result*>(result);
    const uint32_t mx = (uint32_t)tot[4];
    r->sum1 = tot[0]; r->sum2 = tot[1]; r->sum3 = tot[2]; r->sum4 = tot[3];
    r->max_abs = (double)__uint_as_float(mx);
    r->count = count;
    r->device_error = mx >= 0x7f800000u ? QM_DEVERR_NONFINITE : 0u;
    r->reserved = 0;
  } else {
    qm_quant_error_result* r = static_cast<qm_quant_error_result*>(result);
    r->sum_re = tot[0]; r->sum_re_round = tot[1]; r->max_re_round = tot[9];
    r->err2_round = tot[2]; r->err2_overflow = tot[3]; r->err2_underflow = tot[4]; r->sum_x2 = tot[5];
    r->count = count;
    r->n_nonzero = (uint64_t)tot[6]; r->n_overflow = (uint64_t)tot[7]; r->n_underflow = (uint64_t)tot[8];
    r->device_error = (tot[5] != tot[5] || tot[5] > 1.7e308) ? QM_DEVERR_NONFINITE : 0u;   // NaN / Inf seen
    r->reserved = 0;
  }
}

// Describes the view as contiguous lines.  channel_delta: deltas follow the non-contracting index.
qm_status make_lines(const View& x, bool channel_delta, const float* delta, Lines* out) {
  Lines p{};
  p.x = x.data;
  p.delta = delta;
  const bool c_inner = x.s_c == 1;
  if (!c_inner && x.s_nc != 1) return QM_ERR_UNSUPPORTED;
  int64_t inner = c_inner ? x.c : x.nc, outer = c_inner ? x.nc : x.c, batch = x.batch;
  int64_t line_stride = c_inner ? x.s_nc : x.s_c, batch_stride = x.s_b;
  p.delta_mode = !channel_delta ? 0 : (c_inner ? 1 : 2);
  p.delta_batch = x.nc;
  // dense tensors whose deltas do not depend on the position are one long line per tensor
  const bool dense = line_stride == inner && (batch == 1 || batch_stride == inner * outer);
  if (dense && p.delta_mode == 0) {
    inner = inner * outer * batch; outer = 1; batch = 1; line_stride = inner; batch_stride = inner;
  }
  const int64_t gpl = (inner + 7) / 8, total = gpl * outer * batch;
  if (gpl >= (1ll << 32) || total >= (1ll << 32) || outer >= (1ll << 32)) return QM_ERR_UNSUPPORTED;
  p.inner = inner; p.line_stride = line_stride; p.batch_stride = batch_stride;
  p.groups_per_line = (uint32_t)gpl; p.total_groups = (uint32_t)total; p.outer = (uint32_t)outer;
  p.by_gpl = FastDiv((uint32_t)gpl); p.by_outer = FastDiv((uint32_t)outer);
  *out = p;
  return QM_OK;
}

int pass_blocks(const Lines& p) {
  const int64_t want = ((int64_t)p.total_groups + 4 * kThreads - 1) / (4 * kThreads);
  const int64_t cap = (int64_t)sm_count() * 8 < kMaxBlocks ? (int64_t)sm_count() * 8 : kMaxBlocks;
  return (int)(want < 1 ? 1 : (want > cap ? cap : want));
}

template <typename T, int KIND, int FMT>
qm_status launch_pass(const Lines& p, void* result, uint64_t count, void* ws, cudaStream_t s) {
  uint32_t* counter = static_cast<uint32_t*>(ws);
  double* partials = reinterpret_cast<double*>(static_cast<char*>(ws) + kCounterBytes);
  QM_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(uint32_t), s));
  QM_CUDA_OK(launch_pdl(tensor_pass_kernel<T, KIND, FMT>, dim3(pass_blocks(p)), dim3(kThreads), 0, s, p, partials,
                        counter, result, count));
  count_launch();
  return QM_OK;
}

}  // namespace

size_t stats_workspace_bytes() { return kCounterBytes + (size_t)kMaxBlocks * kRec * sizeof(double); }

qm_status launch_tensor_stats(const View& x, qm_tensor_stats_result* out, void* ws, cudaStream_t s) {
  Lines p;
  qm_status st = make_lines(x, false, nullptr, &p);
  if (st != QM_OK) return st;
  const uint64_t n = (uint64_t)(x.nc * x.c * x.batch);
  return x.dtype == QM_DT_BF16 ? launch_pass<__nv_bfloat16, kStats, 0>(p, out, n, ws, s)
                               : launch_pass<float, kStats, 0>(p, out, n, ws, s);
}

qm_status launch_quantize_error(const View& x, int fmt, int gran, const float* delta, qm_quant_error_result* out,
                                void* ws, cudaStream_t s) {
  Lines p;
  qm_status st = make_lines(x, gran == QM_GRAN_CHANNEL, delta, &p);
  if (st != QM_OK) return st;
  const uint64_t n = (uint64_t)(x.nc * x.c * x.batch);
#define QM_PASS(T)                                                                           \
  (fmt == QM_FMT_INT8 ? launch_pass<T, kError, QM_FMT_INT8>(p, out, n, ws, s)                 \
   : fmt == QM_FMT_E4M3 ? launch_pass<T, kError, QM_FMT_E4M3>(p, out, n, ws, s)               \
                        : launch_pass<T, kError, QM_FMT_E5M2>(p, out, n, ws, s))
  return x.dtype == QM_DT_BF16 ? QM_PASS(__nv_bfloat16) : QM_PASS(float);
#undef QM_PASS
}

}  // namespace qm
