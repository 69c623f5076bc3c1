// Measurement aid: a read-only pass over a device buffer, the ceiling that the read-mostly
// kernels of this library (max|x|, tensor statistics) are compared with.  It does nothing but
// load: every thread keeps kInFlight independent 128-bit loads outstanding, folds what arrives
// into one word and the block writes that word only if it is an impossible value, so the
// compiler keeps the loads and the memory system sees no stores.
#include "qm_internal.h"

namespace qm {
namespace {

// WIDE: 256-bit loads with streaming hints (no L1 allocation, evict-first in L2: a stream that is
// read once); otherwise plain 128-bit read-only loads.
template <int IN_FLIGHT, bool WIDE>
__global__ void __launch_bounds__(256)
read_pass_kernel(const uint8_t* __restrict__ p, uint64_t n_vec, uint32_t* __restrict__ sink) {
  constexpr int kVecBytes = WIDE ? 32 : 16;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  auto load = [&](uint64_t j) -> uint32_t {
    const uint8_t* q = p + j * kVecBytes;
    if (WIDE) {
      uint32_t a, b, c, d, e, f, g, h;
      asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(a), "=r"(b), "=r"(c), "=r"(d), "=r"(e), "=r"(f), "=r"(g), "=r"(h) : "l"(q));
      return ((a ^ b) & (c ^ d)) | ((e ^ f) & (g ^ h));
    } else {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(q));
      return (v.x ^ v.y) & (v.z ^ v.w);
    }
  };
  for (; i + (IN_FLIGHT - 1) * stride < n_vec; i += IN_FLIGHT * stride) {
    uint32_t v[IN_FLIGHT];
#pragma unroll
    for (int u = 0; u < IN_FLIGHT; ++u) v[u] = load(i + u * stride);
#pragma unroll
    for (int u = 0; u < IN_FLIGHT; ++u) acc |= v[u];
  }
  for (; i < n_vec; i += stride) acc |= load(i);
  acc = __reduce_or_sync(0xffffffffu, acc);
  if ((threadIdx.x & 31) == 0 && acc == 0x5a5a5a5bu && sink) atomicOr(sink, acc);
}

}  // namespace
}  // namespace qm

extern "C" qm_status qm_debug_read_pass(const void* data, size_t bytes, int32_t variant, int32_t blocks_per_sm,
                                        uint32_t* sink, void* stream) {
  using namespace qm;
  if (!data || bytes < 16 || (reinterpret_cast<uintptr_t>(data) & 15) || blocks_per_sm < 1 || blocks_per_sm > 32)
    return QM_ERR_INVALID_ARG;
  const dim3 grid((unsigned)(sm_count() * blocks_per_sm)), block(256);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint8_t* p = static_cast<const uint8_t*>(data);
  if (variant >= 1 && (reinterpret_cast<uintptr_t>(data) & 31)) return QM_ERR_ALIGNMENT;
  switch (variant) {
    case 0: read_pass_kernel<8, false><<<grid, block, 0, s>>>(p, bytes / 16, sink); break;
    case 1: read_pass_kernel<4, true><<<grid, block, 0, s>>>(p, bytes / 32, sink); break;
    case 2: read_pass_kernel<8, true><<<grid, block, 0, s>>>(p, bytes / 32, sink); break;
    case 3: read_pass_kernel<16, false><<<grid, block, 0, s>>>(p, bytes / 16, sink); break;
    default: return QM_ERR_INVALID_ARG;
  }
  QM_CUDA_OK(cudaGetLastError());
  count_launch();
  return QM_OK;
}
