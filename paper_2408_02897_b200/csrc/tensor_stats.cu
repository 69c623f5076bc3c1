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

// Per-thread sums of one batch of up to four groups of 8 elements: fp32 inside the batch.
template <int KIND, int FMT>
struct Batch {
  float f[7];
  uint32_t n[3];
  uint32_t mx;
  __device__ __forceinline__ Batch() : mx(0) {
#pragma unroll
    for (int i = 0; i < 7; ++i) f[i] = 0.f;
    n[0] = n[1] = n[2] = 0;
  }
  // statistics: f = {sum x, sum x^2, sum x^3, sum x^4}; padded entries are zero and add nothing.
  // Two elements per instruction (packed fp32 pairs): p[k] holds the even-lane and odd-lane halves
  // of the k-th power sum, folded into f by fold_stats().
  uint64_t p2[4] = {0ull, 0ull, 0ull, 0ull};
  __device__ __forceinline__ void stats(const Vec8& v) {
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      // max |x| as a three-input fp32 max (a NaN input shows up in the sums instead)
      asm("max.f32 %0, %0, %1, %2;" : "+f"(f[4]) : "f"(fabsf(v.v[e])), "f"(fabsf(v.v[e + 1])));
      uint64_t x, x2;
      asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "f"(v.v[e]), "f"(v.v[e + 1]));
      asm("mul.rn.f32x2 %0, %1, %1;" : "=l"(x2) : "l"(x));
      asm("add.rn.f32x2 %0, %0, %1;" : "+l"(p2[0]) : "l"(x));
      asm("add.rn.f32x2 %0, %0, %1;" : "+l"(p2[1]) : "l"(x2));
      asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(p2[2]) : "l"(x2), "l"(x));
      asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(p2[3]) : "l"(x2));
    }
  }
  __device__ __forceinline__ void fold_stats() {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float a, b;
      asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(p2[k]));
      f[k] = a + b;
    }
  }
  // Eq. 2 split: f = {sum RE, sum RE rounding, err2 rounding, err2 overflow, err2 underflow,
  // sum x^2, max RE rounding}; n = {non-zero, overflow, underflow}.  Branch-free per element.
  __device__ __forceinline__ void error2(float xa, float xb, float ta, float tb, float da, float db) {
    float ga, gb;
    decode2<FMT>(quant2<FMT>(ta, tb), ga, gb);
    const float qmaxv = fmt_qmax(FMT);
    const float xs[2] = {xa, xb}, ts[2] = {ta, tb}, gs[2] = {ga, gb}, ds[2] = {da, db};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float x = xs[h];
      const bool nz = x != 0.f;
      const float err = fabsf(fmaf(-gs[h], ds[h], x));        // |x - value(code) delta|, one rounding
      // |x| below the normal range (a subnormal bf16 or fp32 element) would be flushed by the
      // approximate reciprocal: those rare elements take the division, which also makes the RE
      // of an underflowed one (err == |x|) exactly 1
      const float ax = fabsf(x);
      float re;
      if (ax >= 1e-36f) {
        float rcp;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rcp) : "f"(ax));
        re = err * rcp;
      } else {
        re = nz ? __fdiv_rn(err, ax) : 0.f;
      }
      const float e2 = err * err;
      const bool over = fabsf(ts[h]) > qmaxv;
      const bool under = nz && !over && gs[h] == 0.f;
      const bool rnd = nz && !over && !under;
      n[0] += nz; n[1] += over; n[2] += under;
      f[0] += re;
      f[5] = fmaf(x, x, f[5]);
      f[3] += over ? e2 : 0.f;
      f[4] += under ? e2 : 0.f;
      f[2] += rnd ? e2 : 0.f;
      const float rr = rnd ? re : 0.f;
      f[1] += rr;
      f[6] = fmaxf(f[6], rr);
    }
  }
  __device__ __forceinline__ void flush(Acc& acc) {
    if (KIND == kStats) {
      fold_stats();
      acc.d[0] += (double)f[0]; acc.d[1] += (double)f[1]; acc.d[2] += (double)f[2]; acc.d[3] += (double)f[3];
      acc.d[4] = fmax(acc.d[4], (double)f[4]);
    } else {
#pragma unroll
      for (int i = 0; i < 6; ++i) acc.d[i] += (double)f[i];
      acc.d[6] += (double)n[0]; acc.d[7] += (double)n[1]; acc.d[8] += (double)n[2];
      acc.d[9] = fmax(acc.d[9], (double)f[6]);
    }
  }
};

// The block's record from its threads' sums, and, in the last block to finish, the fixed-order
// sum of all records into the result.
template <int KIND>
__device__ __forceinline__ void finish_pass(Acc& acc, double* __restrict__ partials, uint32_t* __restrict__ counter,
                                            void* __restrict__ result, uint64_t count) {
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
  if (!is_last) return;
  // last block: every record is visible.  Thread t adds records t, t + 256, ... (all 256 threads, so
  // that the loads of this last step run side by side), then warps and block combine in a fixed order.
  __threadfence();
  double tot[kRec];
#pragma unroll
  for (int i = 0; i < kRec; ++i) tot[i] = 0.0;
  for (int b = threadIdx.x; b < (int)gridDim.x; b += kThreads) {
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
    if (lane == 0) red[i][warp] = tot[i];
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
#pragma unroll
  for (int i = 0; i < kRec; ++i) {
    double x = red[i][0];
    for (int w = 1; w < kThreads / 32; ++w) x = is_max<KIND>(i) ? fmax(x, red[i][w]) : x + red[i][w];
    tot[i] = x;
  }
  if (KIND == kStats) {
    qm_tensor_stats_result* r = static_cast<qm_tensor_stats_result*>(result);
    r->sum1 = tot[0]; r->sum2 = tot[1]; r->sum3 = tot[2]; r->sum4 = tot[3];
    r->max_abs = tot[4];
    r->count = count;
    // a NaN or Inf element (or a power that left the fp32 range) makes sum x^4 NaN or Inf
    r->device_error = (tot[3] != tot[3] || tot[3] > 1.7e308 || tot[4] > 3.5e38) ? QM_DEVERR_NONFINITE : 0u;
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

// Statistics of a dense tensor that starts on a 32-byte boundary and is a whole number of 32-byte
// vectors long: 256-bit loads, four in flight per thread, the same arithmetic (fp32 inside the 64
// or 32 elements of a batch of loads, fp64 above).
template <typename T, bool STREAM>
__global__ void __launch_bounds__(kThreads)
tensor_stats_dense_kernel(const uint8_t* __restrict__ x, uint64_t n_vec, double* __restrict__ partials,
                          uint32_t* __restrict__ counter, void* __restrict__ result, uint64_t count) {
  pdl_prologue();
  Acc acc;
#pragma unroll
  for (int i = 0; i < kRec; ++i) acc.d[i] = 0.0;
  constexpr int U = 4;
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  auto eat = [&](Batch<kStats, 0>& bt, const Vec256& v) {
    Vec8 a, b;
    if (sizeof(T) == 2) {
      a.v[0] = bf16_lo(v.lo.x); a.v[1] = bf16_hi(v.lo.x); a.v[2] = bf16_lo(v.lo.y); a.v[3] = bf16_hi(v.lo.y);
      a.v[4] = bf16_lo(v.lo.z); a.v[5] = bf16_hi(v.lo.z); a.v[6] = bf16_lo(v.lo.w); a.v[7] = bf16_hi(v.lo.w);
      b.v[0] = bf16_lo(v.hi.x); b.v[1] = bf16_hi(v.hi.x); b.v[2] = bf16_lo(v.hi.y); b.v[3] = bf16_hi(v.hi.y);
      b.v[4] = bf16_lo(v.hi.z); b.v[5] = bf16_hi(v.hi.z); b.v[6] = bf16_lo(v.hi.w); b.v[7] = bf16_hi(v.hi.w);
      bt.stats(a); bt.stats(b);
    } else {
      a.v[0] = __uint_as_float(v.lo.x); a.v[1] = __uint_as_float(v.lo.y); a.v[2] = __uint_as_float(v.lo.z); a.v[3] = __uint_as_float(v.lo.w);
      a.v[4] = __uint_as_float(v.hi.x); a.v[5] = __uint_as_float(v.hi.y); a.v[6] = __uint_as_float(v.hi.z); a.v[7] = __uint_as_float(v.hi.w);
      bt.stats(a);
    }
  };
  uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  for (; i + (U - 1) * stride < n_vec; i += U * stride) {
    Vec256 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = ld256<STREAM>(x + (i + u * stride) * 32);
    Batch<kStats, 0> bt;
#pragma unroll
    for (int u = 0; u < U; ++u) eat(bt, v[u]);
    bt.flush(acc);
  }
  for (; i < n_vec; i += stride) {
    Batch<kStats, 0> bt;
    eat(bt, ld256<STREAM>(x + i * 32));
    bt.flush(acc);
  }
  finish_pass<kStats>(acc, partials, counter, result, count);
}

template <typename T, int KIND, int FMT>
__global__ void __launch_bounds__(kThreads, KIND == kError ? 3 : 1)
tensor_pass_kernel(const Lines p, double* __restrict__ partials, uint32_t* __restrict__ counter,
                   void* __restrict__ result, uint64_t count) {
  pdl_prologue();
  Acc acc;
#pragma unroll
  for (int i = 0; i < kRec; ++i) acc.d[i] = 0.0;
  const uint32_t stride = gridDim.x * kThreads;
  const bool whole_groups = (p.inner & 7) == 0;               // no ragged tail anywhere
  const bool flat = p.outer == 1 && p.groups_per_line == p.total_groups;

  // where group g starts, and which deltas it takes
  auto locate = [&](uint32_t g, uint32_t& b, uint32_t& o, uint32_t& j) -> int64_t {
    if (flat) { b = 0; o = 0; j = g; return (int64_t)g * 8; }
    const uint32_t line = p.by_gpl.div(g);
    j = g - line * p.groups_per_line;
    b = p.by_outer.div(line);
    o = line - b * p.outer;
    return (int64_t)b * p.batch_stride + (int64_t)o * p.line_stride + (int64_t)j * 8;
  };
  auto process = [&](Batch<KIND, FMT>& bt, const Vec8& v, uint32_t b, uint32_t o, uint32_t j, int live) {
    if (KIND == kStats) { bt.stats(v); return; }
    if (p.delta_mode != 2) {
      const float d = p.delta_mode == 0 ? __ldg(p.delta) : __ldg(p.delta + (int64_t)b * p.delta_batch + o);
      const Quotient q(d);
#pragma unroll
      for (int e = 0; e < 8; e += 2) bt.error2(v.v[e], v.v[e + 1], q(v.v[e]), q(v.v[e + 1]), d, d);
    } else {
      const float* dp = p.delta + (int64_t)b * p.delta_batch + (int64_t)j * 8;
      float d[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) d[e] = e < live ? __ldg(dp + e) : 1.f;
#pragma unroll
      for (int e = 0; e < 8; e += 2)
        bt.error2(v.v[e], v.v[e + 1], Quotient(d[e])(v.v[e]), Quotient(d[e + 1])(v.v[e + 1]), d[e], d[e + 1]);
    }
  };

  // loads in flight per thread: four for the bandwidth-bound statistics, two for the
  // arithmetic-bound error split (fewer registers, more resident warps)
  constexpr int U = KIND == kError ? 2 : 4;
  for (uint32_t g0 = blockIdx.x * kThreads + threadIdx.x; g0 < p.total_groups; g0 += U * stride) {
    Batch<KIND, FMT> bt;
    const bool full = whole_groups && (uint64_t)g0 + (uint64_t)(U - 1) * stride < p.total_groups;
    if (full) {
      // all loads of the batch are issued before any arithmetic
      Vec8 v[U];
      uint32_t b[U], o[U], j[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int64_t off = locate(g0 + u * stride, b[u], o[u], j[u]);
        v[u] = Loader<T>::load8(reinterpret_cast<const char*>(p.x) + off * (int64_t)sizeof(T));
      }
#pragma unroll
      for (int u = 0; u < U; ++u) process(bt, v[u], b[u], o[u], j[u], 8);
    } else {
      for (int u = 0; u < U; ++u) {
        const uint64_t g = (uint64_t)g0 + (uint64_t)u * stride;
        if (g >= p.total_groups) break;
        uint32_t b, o, j;
        const int64_t off = locate((uint32_t)g, b, o, j);
        const int64_t left = p.inner - (int64_t)j * 8;
        const int live = left < 8 ? (int)left : 8;
        const char* base = reinterpret_cast<const char*>(p.x) + off * (int64_t)sizeof(T);
        Vec8 v;
        if (live == 8) {
          v = Loader<T>::load8(base);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) v.v[e] = e < live ? Loader<T>::load1(base, e) : 0.f;
        }
        process(bt, v, b, o, j, live);
      }
    }
    bt.flush(acc);
  }

  finish_pass<KIND>(acc, partials, counter, result, count);
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

// One wave of resident blocks (or fewer when the tensor is small).
int pass_blocks(const Lines& p, int resident_per_sm) {
  const int64_t want = ((int64_t)p.total_groups + 2 * kThreads - 1) / (2 * kThreads);
  int64_t cap = (int64_t)sm_count() * resident_per_sm;
  if (cap > kMaxBlocks) cap = kMaxBlocks;
  return (int)(want < 1 ? 1 : (want > cap ? cap : want));
}

template <typename T, int KIND, int FMT>
qm_status launch_pass(const Lines& p, void* result, uint64_t count, void* ws, cudaStream_t s) {
  static int resident_of[kMaxDevices] = {};      // per instantiation and device
  const int dev = current_device();
  if (dev < 0) return QM_ERR_UNSUPPORTED;
  if (resident_of[dev] == 0) {
    int nb = 0;
    QM_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, tensor_pass_kernel<T, KIND, FMT>, kThreads, 0));
    resident_of[dev] = nb > 0 ? nb : 1;
  }
  const int resident = resident_of[dev];
  uint32_t* counter = static_cast<uint32_t*>(ws);
  double* partials = reinterpret_cast<double*>(static_cast<char*>(ws) + kCounterBytes);
  QM_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(uint32_t), s));
  QM_CUDA_OK(launch_pdl(tensor_pass_kernel<T, KIND, FMT>, dim3(pass_blocks(p, resident)), dim3(kThreads), 0, s, p,
                        partials, counter, result, count));
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
  const uint64_t bytes = n * (x.dtype == QM_DT_BF16 ? 2 : 4);
  if (p.outer == 1 && p.groups_per_line == p.total_groups && (reinterpret_cast<uintptr_t>(x.data) & 31) == 0 &&
      (bytes & 31) == 0 && bytes >= (1u << 20)) {
    // dense, aligned and large enough to be worth it: the 256-bit kernel
    uint32_t* counter = static_cast<uint32_t*>(ws);
    double* partials = reinterpret_cast<double*>(static_cast<char*>(ws) + kCounterBytes);
    QM_CUDA_OK(cudaMemsetAsync(counter, 0, sizeof(uint32_t), s));
    const uint64_t n_vec = bytes / 32;
    int64_t blocks = (int64_t)((n_vec + kThreads - 1) / kThreads);
    const int64_t cap = (int64_t)sm_count() * 8 < kMaxBlocks ? (int64_t)sm_count() * 8 : kMaxBlocks;
    if (blocks > cap) blocks = cap;
    const uint8_t* src = static_cast<const uint8_t*>(x.data);
    const bool stream = bytes > (64u << 20);
#define QM_TS(T, S) launch_pdl(tensor_stats_dense_kernel<T, S>, dim3((unsigned)blocks), dim3(kThreads), 0, s, src, n_vec, partials, counter, static_cast<void*>(out), n)
    if (x.dtype == QM_DT_BF16) { if (stream) QM_CUDA_OK(QM_TS(__nv_bfloat16, true)); else QM_CUDA_OK(QM_TS(__nv_bfloat16, false)); }
    else { if (stream) QM_CUDA_OK(QM_TS(float, true)); else QM_CUDA_OK(QM_TS(float, false)); }
#undef QM_TS
    count_launch();
    return QM_OK;
  }
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
