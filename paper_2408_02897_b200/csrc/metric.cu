// Eq. 3 on materialised arrays, and the deterministic final reduction shared with the fused
// probe kernels.
#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_maxd(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Each block owns a contiguous slice; the order of additions is fixed by the launch shape.
__global__ void __launch_bounds__(kThreads)
metric_partials_kernel(const float* __restrict__ ref, const float* __restrict__ q,
                       const float* __restrict__ den, int64_t count, double* __restrict__ partials) {
  __shared__ double s[5][kThreads / 32];
  const int64_t per_block = (count + gridDim.x - 1) / gridDim.x;
  const int64_t i0 = (int64_t)blockIdx.x * per_block;
  const int64_t i1 = min(count, i0 + per_block);
  double sbe = 0, mbe = 0, sd2 = 0, sr2 = 0, sn2 = 0;
  for (int64_t base = i0; base < i1; base += kThreads * 8) {
    // fp32 inside a short run, fp64 across runs
    float fbe = 0, fmx = 0, fd2 = 0, fr2 = 0, fn2 = 0;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int64_t i = base + u * kThreads + threadIdx.x;
      if (i < i1) {
        const float c = __ldg(ref + i), qq = __ldg(q + i), d = __ldg(den + i);
        const float diff = c - qq;
        const float be = d != 0.f ? __fdiv_rn(fabsf(diff), d) : 0.f;
        fbe += be; fmx = fmaxf(fmx, be);
        fd2 = fmaf(diff, diff, fd2); fr2 = fmaf(c, c, fr2); fn2 = fmaf(d, d, fn2);
      }
    }
    sbe += fbe; mbe = fmax(mbe, (double)fmx); sd2 += fd2; sr2 += fr2; sn2 += fn2;
  }
  sbe = warp_sum(sbe); sd2 = warp_sum(sd2); sr2 = warp_sum(sr2); sn2 = warp_sum(sn2);
  mbe = warp_maxd(mbe);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { s[0][w] = sbe; s[1][w] = mbe; s[2][w] = sd2; s[3][w] = sr2; s[4][w] = sn2; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0, m = 0, b = 0, c = 0, d = 0;
    for (int i = 0; i < kThreads / 32; ++i) {
      a += s[0][i]; m = fmax(m, s[1][i]); b += s[2][i]; c += s[3][i]; d += s[4][i];
    }
    double* o = partials + (int64_t)blockIdx.x * kPartialDoubles;
    o[0] = a; o[1] = m; o[2] = b; o[3] = c; o[4] = d;
  }
}

// One block; thread t sums records t, t+256, ... in order, then a fixed tree.
__global__ void __launch_bounds__(kThreads)
metric_finalize_kernel(const double* __restrict__ partials, int n, uint64_t count,
                       const uint32_t* __restrict__ err_word, qm_metric_result* __restrict__ out) {
  __shared__ double s[5][kThreads];
  double a = 0, m = 0, b = 0, c = 0, d = 0;
  for (int i = threadIdx.x; i < n; i += kThreads) {
    const double* p = partials + (int64_t)i * kPartialDoubles;
    a += p[0]; m = fmax(m, p[1]); b += p[2]; c += p[3]; d += p[4];
  }
  s[0][threadIdx.x] = a; s[1][threadIdx.x] = m; s[2][threadIdx.x] = b;
  s[3][threadIdx.x] = c; s[4][threadIdx.x] = d;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      s[0][threadIdx.x] += s[0][threadIdx.x + o];
      s[1][threadIdx.x] = fmax(s[1][threadIdx.x], s[1][threadIdx.x + o]);
      s[2][threadIdx.x] += s[2][threadIdx.x + o];
      s[3][threadIdx.x] += s[3][threadIdx.x + o];
      s[4][threadIdx.x] += s[4][threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    out->sum_be = s[0][0]; out->max_be = s[1][0]; out->sum_diff2 = s[2][0];
    out->sum_ref2 = s[3][0]; out->sum_den2 = s[4][0];
    out->count = count;
    out->device_error = err_word ? *err_word : 0u;
    out->reserved = 0;
  }
}

}  // namespace

int metric_blocks(int64_t count) {
  int64_t want = (count + kThreads * 8 - 1) / (kThreads * 8);
  int64_t cap = (int64_t)sm_count() * 8;
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

qm_status launch_metric_partials(const float* ref, const float* q, const float* den, int64_t count,
                                 double* partials, int nblocks, cudaStream_t s) {
  metric_partials_kernel<<<nblocks, kThreads, 0, s>>>(ref, q, den, count, partials);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

qm_status launch_metric_finalize(const double* partials, int n, uint64_t count,
                                 const uint32_t* err_word, qm_metric_result* out, cudaStream_t s) {
  metric_finalize_kernel<<<1, kThreads, 0, s>>>(partials, n, count, err_word, out);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

}  // namespace qm

// ---------------------------------------------------------------------------------------------
// qm_metric_noalloc: Eq. 3 reduction for callers that cannot allocate device memory.
//
// The per-block partial records of qm_metric normally live in a caller-provided workspace.  A
// caller that runs where cudaMalloc is off limits (a plug-in that is handed raw input/output
// pointers by its host application, code running inside a memory-pool-managed region, a
// latency-critical loop that must not touch the allocator) has nowhere to get that workspace
// from.  For them the library carries the scratch itself, as a fixed array in the module's
// device image: kNoAllocRecords partial records (40 KiB), present on every GPU that loads the
// library until the process ends.
namespace qm {
namespace {

constexpr int kNoAllocRecords = 1024;                         // 1024 x 5 doubles = 40 KiB
constexpr int64_t kNoAllocMaxCount = (int64_t)1 << 30;        // elements per input array

static __device__ __align__(256) double g_noalloc_partials[kNoAllocRecords * kPartialDoubles];

// In host code the array's name is only a handle for the runtime, not a device address: the
// address the kernels need is looked up once per device (with that device current) and cached.
double* g_noalloc_ptr[kMaxDevices] = {};

qm_status noalloc_scratch(double** out) {
  int dev = -1;
  QM_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return QM_ERR_UNSUPPORTED;
  if (!g_noalloc_ptr[dev]) {
    double* p = nullptr;
    QM_CUDA_OK(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_partials));
    if (!p) return QM_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return QM_OK;
}

}  // namespace
// ---- clearing the control words of several workspaces in one launch --------------------------
namespace {
__global__ void clear_many_kernel(const ClearList list) {
  pdl_prologue();
  const int w = blockIdx.x;                      // gridDim.y blocks per region
  uint32_t* p = static_cast<uint32_t*>(list.ptr[w]);
  for (uint32_t i = blockIdx.y * blockDim.x + threadIdx.x; i < list.words[w]; i += gridDim.y * blockDim.x) p[i] = 0u;
}
}  // namespace

qm_status launch_clear_many(const ClearList& list, cudaStream_t s) {
  if (list.n < 1 || list.n > kClearMax) return QM_ERR_INVALID_ARG;
  QM_CUDA_OK(launch_pdl(clear_many_kernel, dim3((unsigned)list.n, 8), dim3(256), 0, s, list));
  count_launch();
  return QM_OK;
}

}  // namespace qm

extern "C" qm_status qm_metric_noalloc(const float* ref, const float* q, const float* den, int64_t count,
                                       qm_metric_result* out, void* stream) {
  using namespace qm;
  if (!ref || !q || !den || !out || count <= 0) return QM_ERR_INVALID_ARG;
  if (count > kNoAllocMaxCount) return QM_ERR_WORKSPACE_TOO_SMALL;   // beyond the built-in scratch's stated limit
  double* scratch = nullptr;
  qm_status st = noalloc_scratch(&scratch);
  if (st != QM_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int nb = metric_blocks(count);
  if (nb > kNoAllocRecords) nb = kNoAllocRecords;
  // Every record that the final reduction reads is overwritten by its block first, so nothing
  // in the shared array has to be cleared between calls.
  st = launch_metric_partials(ref, q, den, count, scratch, nb, s);
  if (st != QM_OK) return st;
  return launch_metric_finalize(scratch, nb, (uint64_t)count, nullptr, out, s);
}

extern "C" int64_t qm_metric_noalloc_max_count(void) { return qm::kNoAllocMaxCount; }
