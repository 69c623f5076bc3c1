// Scale (Eq. 1, right half) and quantize (Eq. 1, left half + saturation rule) kernels.
// All of them are HBM-bound streaming kernels: 128-bit coalesced loads, warp-shuffle and
// shared-memory reductions, one atomicMax per block and group.
#include "quant_device.cuh"

namespace qm {
namespace {

// ---------------------------------------------------------------- absmax, whole tensor
// Rows of `c` contiguous elements (vector loads for the multiple-of-8 part, scalar loads for
// the tail).  When the rows are dense the host flattens the tensor into a single row so that
// every block gets an equal share.
template <typename T>
__global__ void __launch_bounds__(kThreads)
absmax_tensor_kernel(const T* __restrict__ x, int64_t rows, int64_t c, int64_t row_stride,
                     uint32_t* __restrict__ amax) {
  pdl_prologue();
  const int64_t vec_per_row = c >> 3;
  const int64_t total_vec = rows * vec_per_row;
  uint32_t acc = 0;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (rows == 1) {
    // dense tensor walked as one row: no index arithmetic beyond the stride;
    // eight independent 128-bit loads in flight per thread
    for (; i + 7 * stride < total_vec; i += 8 * stride) {
      Vec8 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = Loader<T>::load8(x + (i + u * stride) * 8);
#pragma unroll
      for (int u = 0; u < 8; ++u) acc = absmax8(v[u], acc);
    }
    if (i < total_vec) {
      // remainder (fewer than eight per thread): still issued together, not one after another;
      // lanes past the end re-read the last vector, which cannot change a maximum
      Vec8 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int64_t j = i + u * stride;
        v[u] = Loader<T>::load8(x + (j < total_vec ? j : total_vec - 1) * 8);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) acc = absmax8(v[u], acc);
    }
  } else {
    // four independent 128-bit loads in flight per thread
    for (; i + 3 * stride < total_vec; i += 4 * stride) {
      Vec8 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        int64_t j = i + u * stride;
        int64_t r = j / vec_per_row, k = j - r * vec_per_row;
        v[u] = Loader<T>::load8(x + r * row_stride + k * 8);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) acc = absmax8(v[u], acc);
    }
    for (; i < total_vec; i += stride) {
      int64_t r = i / vec_per_row, k = i - r * vec_per_row;
      acc = absmax8(Loader<T>::load8(x + r * row_stride + k * 8), acc);
    }
  }
  const int64_t tail = c & 7;
  if (tail) {
    const int64_t total_tail = rows * tail;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < total_tail; j += stride) {
      int64_t r = j / tail, k = j - r * tail;
      acc = max(acc, absbits_f32(__float_as_uint(Loader<T>::load1(x, r * row_stride + (c - tail) + k))));
    }
  }
  acc = block_max(acc);
  if (threadIdx.x == 0 && acc) atomicMax(amax, acc);
}

// ---------------------------------------------------------------- absmax, dense tensor
// One flat run of 32-byte vectors (base 32-byte aligned): 256-bit loads, IN_FLIGHT of them
// outstanding per thread, and the maximum taken on packed words: for bf16 two sign-cleared 16-bit
// patterns per word (unsigned 16-bit maxima order like the magnitudes), for fp32 one 31-bit pattern.
template <typename T, int IN_FLIGHT, bool STREAM>
__global__ void __launch_bounds__(kThreads)
absmax_dense_kernel(const uint8_t* __restrict__ x, uint64_t n_vec, uint32_t* __restrict__ amax) {
  pdl_prologue();
  constexpr bool kBf16 = sizeof(T) == 2;
  const uint32_t mask = kBf16 ? 0x7fff7fffu : 0x7fffffffu;
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t m = 0;
  auto fold = [&](const Vec256& v) {
    if (kBf16) {
      const uint32_t a = __vmaxu2(__vmaxu2(v.lo.x & mask, v.lo.y & mask), __vmaxu2(v.lo.z & mask, v.lo.w & mask));
      const uint32_t b = __vmaxu2(__vmaxu2(v.hi.x & mask, v.hi.y & mask), __vmaxu2(v.hi.z & mask, v.hi.w & mask));
      m = __vmaxu2(m, __vmaxu2(a, b));
    } else {
      const uint32_t a = max(max(v.lo.x & mask, v.lo.y & mask), max(v.lo.z & mask, v.lo.w & mask));
      const uint32_t b = max(max(v.hi.x & mask, v.hi.y & mask), max(v.hi.z & mask, v.hi.w & mask));
      m = max(m, max(a, b));
    }
  };
  for (; i + (IN_FLIGHT - 1) * stride < n_vec; i += IN_FLIGHT * stride) {
    Vec256 v[IN_FLIGHT];
#pragma unroll
    for (int u = 0; u < IN_FLIGHT; ++u) v[u] = ld256<STREAM>(x + (i + u * stride) * 32);
#pragma unroll
    for (int u = 0; u < IN_FLIGHT; ++u) fold(v[u]);
  }
  for (; i < n_vec; i += stride) fold(ld256<STREAM>(x + i * 32));
  uint32_t acc = kBf16 ? (max(m & 0xffffu, m >> 16) << 16) : m;      // as an fp32 bit pattern
  acc = block_max(acc);
  if (threadIdx.x == 0 && acc) atomicMax(amax, acc);
}

// ---------------------------------------------------------------- absmax per row (contiguous rows)
// G lanes share a row; rows are (batch, nc) pairs.
template <typename T, int G>
__global__ void __launch_bounds__(kThreads)
absmax_rows_kernel(const T* __restrict__ x, int64_t nc, int64_t c, int64_t s_nc, int64_t batch,
                   int64_t s_b, uint32_t* __restrict__ amax) {
  pdl_prologue();
  const int64_t rows = nc * batch;
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int sub = threadIdx.x % G;
  uint32_t acc = 0;
  if (row < rows) {
    const int64_t b = row / nc, r = row - b * nc;
    const T* p = x + b * s_b + r * s_nc;
    const int64_t nvec = c >> 3;
    for (int64_t k = sub; k < nvec; k += G) acc = absmax8(Loader<T>::load8(p + k * 8), acc);
    for (int64_t k = (nvec << 3) + sub; k < c; k += G)
      acc = max(acc, absbits_f32(__float_as_uint(Loader<T>::load1(p, k))));
  }
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) acc = max(acc, __shfl_xor_sync(0xffffffffu, acc, o, G));
  if (row < rows && sub == 0) amax[row] = acc;
}

// ---------------------------------------------------------------- absmax per column (strided contraction)
// Storage is [c][nc] with nc contiguous; one value per column.  Each thread owns 8 adjacent
// columns; blockDim = (32, 8): 256 columns wide, 8 row slices; grid.y splits the rows.
template <typename T>
__global__ void __launch_bounds__(kThreads)
absmax_cols_kernel(const T* __restrict__ x, int64_t nc, int64_t c, int64_t s_c, int64_t s_b,
                   int64_t rows_per_block, uint32_t* __restrict__ amax) {
  pdl_prologue();
  __shared__ uint32_t s[8][256];
  const int64_t b = blockIdx.z;
  const int64_t col0 = ((int64_t)blockIdx.x * 32 + threadIdx.x) * 8;
  const int64_t r0 = (int64_t)blockIdx.y * rows_per_block;
  const int64_t r1 = min(c, r0 + rows_per_block);
  uint32_t acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0;
  const T* base = x + b * s_b;
  if (col0 + 8 <= nc) {
    for (int64_t r = r0 + threadIdx.y; r < r1; r += 8) {
      Vec8 v = Loader<T>::load8(base + r * s_c + col0);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = max(acc[i], absbits_f32(__float_as_uint(v.v[i])));
    }
  } else if (col0 < nc) {
    for (int64_t r = r0 + threadIdx.y; r < r1; r += 8)
      for (int i = 0; i < 8 && col0 + i < nc; ++i)
        acc[i] = max(acc[i], absbits_f32(__float_as_uint(Loader<T>::load1(base, r * s_c + col0 + i))));
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) s[threadIdx.y][threadIdx.x * 8 + i] = acc[i];
  __syncthreads();
  const int t = threadIdx.y * 32 + threadIdx.x;      // 0..255: one column each
  uint32_t m = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) m = max(m, s[j][t]);
  const int64_t col = (int64_t)blockIdx.x * 256 + t;
  if (col < nc && m) atomicMax(amax + b * nc + col, m);
}

// Per-channel maxima shared along the batch: batch element b belongs to group b % groups, and
// every (group, channel) entry becomes the maximum over the group's batch elements (integer max
// of the order-preserving bit patterns), written back to each of them.  One thread per entry.
__global__ void share_amax_kernel(uint32_t* __restrict__ amax, int64_t batch, int64_t groups, int64_t nc) {
  pdl_prologue();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= groups * nc) return;
  const int64_t g = i / nc, ch = i - g * nc;
  uint32_t m = 0;
  for (int64_t b = g; b < batch; b += groups) m = max(m, amax[b * nc + ch]);
  for (int64_t b = g; b < batch; b += groups) amax[b * nc + ch] = m;
}

__global__ void finalize_delta_kernel(float* __restrict__ delta, int64_t n, float qmax,
                                      uint32_t* __restrict__ err_word) {
  pdl_prologue();
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t bits = __float_as_uint(delta[i]);
  float amax = __uint_as_float(bits);
  if (bits >= 0x7f800000u && err_word) atomicOr(err_word, QM_DEVERR_NONFINITE);
  delta[i] = bits == 0 ? 1.0f : __fdiv_rn(amax, qmax);
}

// Where a quantize kernel gets its scales from.  Either finished deltas, or (from_amax) the bit
// patterns of max|x| left by an absmax kernel: the division of Eq. 1 is then done here, which
// saves a launch; the thread named `writer` stores the delta for later consumers and raises
// the non-finite flag.
struct DeltaSrc {
  const float* p;
  int per_channel;
  int from_amax;
  float qmax;
  float* out;           // from_amax only: where the finished deltas go
  uint32_t* err_word;   // from_amax only, optional
  __device__ __forceinline__ float get(int64_t i, bool writer) const {
    if (!from_amax) return __ldg(p + i);
    const uint32_t bits = __ldg(reinterpret_cast<const uint32_t*>(p) + i);
    const float d = bits == 0 ? 1.0f : __fdiv_rn(__uint_as_float(bits), qmax);
    if (writer) {
      out[i] = d;
      if (bits >= 0x7f800000u && err_word) atomicOr(err_word, QM_DEVERR_NONFINITE);
    }
    return d;
  }
};

// ---------------------------------------------------------------- quantize, contiguous contraction
// One thread handles 16 consecutive elements of a row: two 128-bit loads (bf16), one 128-bit
// code store, optionally two 128-bit stores of |x| as bf16.
template <typename T, int FMT>
__global__ void __launch_bounds__(kThreads)
quantize_rows_kernel(const T* __restrict__ x, int64_t nc, int64_t c, int64_t s_nc, int64_t batch,
                     int64_t s_b, const DeltaSrc ds, const FastDiv by_chunks, const FastDiv by_nc,
                     uint8_t* __restrict__ codes, int64_t ldc, __nv_bfloat16* __restrict__ abs_copy,
                     const Rounding rnd) {
  pdl_prologue();
  const uint32_t chunks_per_row = (uint32_t)(ldc >> 4);     // 16 codes per chunk, padding included
  const uint32_t total = (uint32_t)(nc * batch) * chunks_per_row;   // < 2^32, checked by the host
  const uint32_t stride = gridDim.x * blockDim.x;
  const float d_tensor = ds.per_channel ? 0.f : ds.get(0, blockIdx.x == 0 && threadIdx.x == 0);
  const Quotient quot_tensor(d_tensor);
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const uint32_t row = by_chunks.div(i), ch = i - row * chunks_per_row;
    const uint32_t b = by_nc.div(row), r = row - b * (uint32_t)nc;
    const T* p = x + (int64_t)b * s_b + (int64_t)r * s_nc + ch * 16;
    const Quotient quot = ds.per_channel ? Quotient(ds.get(row, ch == 0)) : quot_tensor;
    const int64_t k0 = ch * 16;
    Vec8 v0, v1;
    if (k0 + 16 <= c) {
      v0 = Loader<T>::load8(p);
      v1 = Loader<T>::load8(p + 8);
    } else {                                                // ragged end of the row: zero fill
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        v0.v[j] = k0 + j < c ? Loader<T>::load1(p, j) : 0.f;
        v1.v[j] = k0 + 8 + j < c ? Loader<T>::load1(p, 8 + j) : 0.f;
      }
    }
    uint2 q0, q1;
    if (rnd.stochastic) {
      const uint64_t e0 = (uint64_t)row * (uint64_t)c + (uint64_t)k0;   // number of the chunk's first element
      q0 = quant8_sr<FMT>(v0, quot, rnd, e0);
      q1 = quant8_sr<FMT>(v1, quot, rnd, e0 + 8);
    } else {
      q0 = quant8<FMT>(v0, quot);
      q1 = quant8<FMT>(v1, quot);
    }
    *reinterpret_cast<uint4*>(codes + row * ldc + k0) = make_uint4(q0.x, q0.y, q1.x, q1.y);
    if (abs_copy) {
      __nv_bfloat16* a = abs_copy + row * c + k0;
      if (k0 + 16 <= c && (c & 7) == 0) {
        *reinterpret_cast<uint4*>(a) = abs_bf16x8(v0);
        *reinterpret_cast<uint4*>(a + 8) = abs_bf16x8(v1);
      } else {
        for (int j = 0; j < 8; ++j) {
          if (k0 + j < c) a[j] = __float2bfloat16_rn(fabsf(v0.v[j]));
          if (k0 + 8 + j < c) a[8 + j] = __float2bfloat16_rn(fabsf(v1.v[j]));
        }
      }
    }
  }
}

// ---------------------------------------------------------------- quantize, dense bf16 fast path
// The common case of the probe: a dense bf16 tensor whose rows are a multiple of 16 long, so the
// whole tensor is one flat run of 16-element chunks and codes have no padding.  Each thread
// takes CHUNKS chunks a block-width apart and issues all of their 128-bit loads before touching
// any of them (2 x CHUNKS loads in flight per thread; 4 for tensors that fill the GPU several
// times over, 1 for small ones, which need the parallelism more); |x| copies are the raw
// bit patterns with the sign bits cleared.
// WIDE: the tensor starts on a 32-byte boundary and a chunk is fetched with one 256-bit load (the
// four-chunk variant, used for tensors far larger than L2, also asks for evict-first).
template <int FMT, int CHUNKS, bool WIDE>
__global__ void __launch_bounds__(kThreads)
quantize_dense_kernel(const uint4* __restrict__ x, uint32_t total_chunks, const DeltaSrc ds,
                      const FastDiv by_chunks, uint32_t chunks_per_row, uint4* __restrict__ codes,
                      uint4* __restrict__ abs_copy) {
  pdl_prologue();
  const uint32_t base = blockIdx.x * (kThreads * CHUNKS) + threadIdx.x;
  uint4 w[CHUNKS][2];
#pragma unroll
  for (int u = 0; u < CHUNKS; ++u) {
    const uint32_t i = base + u * kThreads;
    const uint32_t j = i < total_chunks ? i : total_chunks - 1;     // clamp: results of dead lanes are dropped
    if (WIDE) {
      const Vec256 v = ld256<CHUNKS == 4>(x + 2 * (size_t)j);
      w[u][0] = v.lo; w[u][1] = v.hi;
    } else {
      w[u][0] = __ldg(x + 2 * (size_t)j);
      w[u][1] = __ldg(x + 2 * (size_t)j + 1);
    }
  }
  const float d_tensor = ds.per_channel ? 0.f : ds.get(0, blockIdx.x == 0 && threadIdx.x == 0);
  if (!ds.per_channel && !abs_copy && QuotientPair::serves(d_tensor)) {
    // one scale for the whole tensor: the two-wide exact quotient (guarded against overflow
    // when the scale was handed in rather than taken from the tensor's own max|x|)
    const QuotientPair qp(d_tensor);
#pragma unroll
    for (int u = 0; u < CHUNKS; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < total_chunks)
        codes[i] = ds.from_amax ? quant_bf16x16<FMT, false>(w[u][0], w[u][1], qp) : quant_bf16x16<FMT, true>(w[u][0], w[u][1], qp);
    }
    return;
  }
  const Quotient quot_tensor(d_tensor);
#pragma unroll
  for (int u = 0; u < CHUNKS; ++u) {
    const uint32_t i = base + u * kThreads;
    if (i >= total_chunks) break;
    Quotient quot = quot_tensor;
    if (ds.per_channel) {
      const uint32_t row = by_chunks.div(i);
      quot = Quotient(ds.get(row, i == row * chunks_per_row));
    }
    uint4 out;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint4 v = w[u][h];
      Vec8 f;
      f.v[0] = bf16_lo(v.x); f.v[1] = bf16_hi(v.x); f.v[2] = bf16_lo(v.y); f.v[3] = bf16_hi(v.y);
      f.v[4] = bf16_lo(v.z); f.v[5] = bf16_hi(v.z); f.v[6] = bf16_lo(v.w); f.v[7] = bf16_hi(v.w);
      const uint2 q = quant8<FMT>(f, quot);
      if (h == 0) { out.x = q.x; out.y = q.y; } else { out.z = q.x; out.w = q.y; }
      if (abs_copy) {
        const uint32_t m = 0x7fff7fffu;
        abs_copy[2 * (size_t)i + h] = make_uint4(v.x & m, v.y & m, v.z & m, v.w & m);
      }
    }
    codes[i] = out;
  }
}

// ---------------------------------------------------------------- several formats in one pass
// A sweep of formats quantizes the same tensor two or three times (Table 1).  These kernels read
// it once and write the codes of every format in MASK (bit f = qm_format f), with per-tensor
// scales taken from the tensor's max|x| bit pattern: delta_f = max|x| / qmax_f.  Thread 0 of
// block 0 stores the scales and raises the non-finite flag for each format's probe.
struct MultiOut {
  uint8_t* codes[3];      // indexed by qm_format; null where MASK has no bit
  float* delta_out[3];
  uint32_t* err_word[3];
};

template <int MASK>
__device__ __forceinline__ void multi_scales(const uint32_t* amax, const MultiOut& o, bool writer, float (&d)[3]) {
  const uint32_t bits = __ldg(amax);
#pragma unroll
  for (int f = 0; f < 3; ++f) {
    if (!(MASK & (1 << f))) { d[f] = 1.f; continue; }
    d[f] = bits == 0 ? 1.0f : __fdiv_rn(__uint_as_float(bits), fmt_qmax(f));
    if (writer) {
      o.delta_out[f][0] = d[f];
      if (bits >= 0x7f800000u && o.err_word[f]) atomicOr(o.err_word[f], QM_DEVERR_NONFINITE);
    }
  }
}

// Dense bf16 tensor, rows a multiple of 16 long: one flat run of 16-element chunks.
template <int MASK, int CHUNKS, bool WIDE>
__global__ void __launch_bounds__(kThreads)
quantize_dense_multi_kernel(const uint4* __restrict__ x, uint32_t total_chunks, const uint32_t* __restrict__ amax,
                            const MultiOut o) {
  pdl_prologue();
  const uint32_t base = blockIdx.x * (kThreads * CHUNKS) + threadIdx.x;
  uint4 w[CHUNKS][2];
#pragma unroll
  for (int u = 0; u < CHUNKS; ++u) {
    const uint32_t i = base + u * kThreads;
    const uint32_t j = i < total_chunks ? i : total_chunks - 1;     // clamp: results of dead lanes are dropped
    if (WIDE) {
      const Vec256 v = ld256<CHUNKS == 4>(x + 2 * (size_t)j);
      w[u][0] = v.lo; w[u][1] = v.hi;
    } else {
      w[u][0] = __ldg(x + 2 * (size_t)j);
      w[u][1] = __ldg(x + 2 * (size_t)j + 1);
    }
  }
  float d[3];
  multi_scales<MASK>(amax, o, blockIdx.x == 0 && threadIdx.x == 0, d);
  const bool pair_ok = QuotientPair::serves(d[0]) && QuotientPair::serves(d[1]) && QuotientPair::serves(d[2]);
#pragma unroll
  for (int f = 0; f < 3; ++f) {
    if (!(MASK & (1 << f))) continue;
    uint4* codes = reinterpret_cast<uint4*>(o.codes[f]);
    if (pair_ok) {
      const QuotientPair quot(d[f]);
#pragma unroll
      for (int u = 0; u < CHUNKS; ++u) {
        const uint32_t i = base + u * kThreads;
        if (i < total_chunks) {
          codes[i] = f == 0   ? quant_bf16x16<0>(w[u][0], w[u][1], quot)
                     : f == 1 ? quant_bf16x16<1>(w[u][0], w[u][1], quot)
                              : quant_bf16x16<2>(w[u][0], w[u][1], quot);
        }
      }
    } else {
      const Quotient quot(d[f]);
#pragma unroll 1
      for (int u = 0; u < CHUNKS; ++u) {
        const uint32_t i = base + u * kThreads;
        if (i >= total_chunks) break;
        uint4 out;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint4 v = w[u][h];
          Vec8 t;
          t.v[0] = bf16_lo(v.x); t.v[1] = bf16_hi(v.x); t.v[2] = bf16_lo(v.y); t.v[3] = bf16_hi(v.y);
          t.v[4] = bf16_lo(v.z); t.v[5] = bf16_hi(v.z); t.v[6] = bf16_lo(v.w); t.v[7] = bf16_hi(v.w);
          const uint2 q = f == 0 ? quant8<0>(t, quot) : f == 1 ? quant8<1>(t, quot) : quant8<2>(t, quot);
          if (h == 0) { out.x = q.x; out.y = q.y; } else { out.z = q.x; out.w = q.y; }
        }
        codes[i] = out;
      }
    }
  }
}

// ---------------------------------------------------------------- quantize + transpose through shared memory
// Storage [c][nc] (nc contiguous, bf16), c a multiple of 128 and nc a multiple of 64.  A block
// takes a tile of 128 contraction rows x 64 columns: it loads the tile with whole-line reads (8
// threads per 128-byte row), reads it back column-wise (a thread takes 16 contraction entries of two
// adjacent columns; consecutive lanes read consecutive words: conflict-free), quantizes, and hands
// the codes (128 bytes per output row and format) and the contraction-major copy (256 bytes per
// output row) to global memory through a second shared-memory tile so that every store instruction
// writes whole lines: 16-byte chunk ch of output row n sits at ch ^ ((n >> 1) & 7), which keeps
// both the column-wise writes and the row-wise reads of that tile conflict-free.
// d_lo / d_hi: the scales of the thread's two columns, per format in MASK (bit f = qm_format f).
template <int MASK, bool GUARD>
__device__ __forceinline__ void transpose_tile(const __nv_bfloat16* __restrict__ x, int64_t nc, int64_t c, int64_t s_c,
                                               int64_t s_b, const float (&d_lo)[3], const float (&d_hi)[3],
                                               uint8_t* const (&codes)[3], int64_t ldc,
                                               __nv_bfloat16* __restrict__ kmaj_copy, uint4* smem) {
  const int t = threadIdx.x;
  const int64_t b = blockIdx.z, n0 = (int64_t)blockIdx.x * 64, k0 = (int64_t)blockIdx.y * 128;
  // phase 1: 128 rows x 128 bytes, four 16-byte loads per thread in flight
  {
    const uint4* src = reinterpret_cast<const uint4*>(x + b * s_b + k0 * s_c + n0);
    const int64_t pitch = s_c >> 3;                                   // row stride in 16-byte units
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = __ldg(src + (int64_t)((t >> 3) + 32 * i) * pitch + (t & 7));
#pragma unroll
    for (int i = 0; i < 4; ++i) smem[((t >> 3) + 32 * i) * 8 + (t & 7)] = v[i];
  }
  __syncthreads();
  // phase 2: columns 2p, 2p + 1, contraction entries 16g .. 16g + 15
  const int pcol = t & 31, g = t >> 5;
  uint32_t w[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) w[j] = reinterpret_cast<const uint32_t*>(smem)[(16 * g + j) * 32 + pcol];
  __syncthreads();                                                     // the output tiles reuse the input tile's memory
  uint4* const s_codes = smem;                                         // [3][64 rows][8 chunks]
  uint4* const s_kmaj = smem + 3 * 64 * 8;                             // [64 rows][16 chunks]
  const uint32_t sw = (uint32_t)pcol & 7u;
#pragma unroll
  for (int col = 0; col < 2; ++col) {
    const int n = 2 * pcol + col;
    uint32_t pw[8];                                                    // this column's 16 values, two bf16 per word
#pragma unroll
    for (int j = 0; j < 8; ++j)
      pw[j] = col == 0 ? __byte_perm(w[2 * j], w[2 * j + 1], 0x5410) : __byte_perm(w[2 * j], w[2 * j + 1], 0x7632);
    const uint4 a = make_uint4(pw[0], pw[1], pw[2], pw[3]), bb = make_uint4(pw[4], pw[5], pw[6], pw[7]);
    if (kmaj_copy) {
      s_kmaj[n * 16 + ((2 * g) ^ sw)] = a;
      s_kmaj[n * 16 + ((2 * g + 1) ^ sw)] = bb;
    }
#pragma unroll
    for (int f = 0; f < 3; ++f) {
      if (!(MASK & (1 << f))) continue;
      const float d = col == 0 ? d_lo[f] : d_hi[f];
      uint4 cw;
      if (QuotientPair::serves(d)) {
        const QuotientPair qp(d);
        cw = f == 0 ? quant_bf16x16<0, GUARD>(a, bb, qp) : f == 1 ? quant_bf16x16<1, GUARD>(a, bb, qp) : quant_bf16x16<2, GUARD>(a, bb, qp);
      } else {
        const Quotient quot(d);
        Vec8 lo, hi;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          lo.v[2 * j] = bf16_lo(pw[j]); lo.v[2 * j + 1] = bf16_hi(pw[j]);
          hi.v[2 * j] = bf16_lo(pw[4 + j]); hi.v[2 * j + 1] = bf16_hi(pw[4 + j]);
        }
        const uint2 q0 = f == 0 ? quant8<0>(lo, quot) : f == 1 ? quant8<1>(lo, quot) : quant8<2>(lo, quot);
        const uint2 q1 = f == 0 ? quant8<0>(hi, quot) : f == 1 ? quant8<1>(hi, quot) : quant8<2>(hi, quot);
        cw = make_uint4(q0.x, q0.y, q1.x, q1.y);
      }
      s_codes[(f * 64 + n) * 8 + ((uint32_t)g ^ sw)] = cw;
    }
  }
  __syncthreads();
  // phase 3: whole output rows
#pragma unroll
  for (int f = 0; f < 3; ++f) {
    if (!(MASK & (1 << f))) continue;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = (t >> 3) + 32 * i, ch = t & 7;
      const uint4 v = s_codes[(f * 64 + row) * 8 + (ch ^ ((row >> 1) & 7))];
      *reinterpret_cast<uint4*>(codes[f] + (b * nc + n0 + row) * ldc + k0 + ch * 16) = v;
    }
  }
  if (kmaj_copy) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = (t >> 4) + 16 * i, ch = t & 15;
      const uint4 v = s_kmaj[row * 16 + (ch ^ ((row >> 1) & 7))];
      *reinterpret_cast<uint4*>(kmaj_copy + (b * nc + n0 + row) * c + k0 + ch * 8) = v;
    }
  }
}

constexpr int kTileSmemVec = 3 * 64 * 8 + 64 * 16;                    // 40 KB in 16-byte units

// One format, scales from a DeltaSrc (per tensor or per output row, finished or from max|x|).
template <int FMT>
__global__ void __launch_bounds__(kThreads)
quantize_transpose_tile_kernel(const __nv_bfloat16* __restrict__ x, int64_t nc, int64_t c, int64_t s_c, int64_t s_b,
                               const DeltaSrc ds, uint8_t* __restrict__ codes, int64_t ldc,
                               __nv_bfloat16* __restrict__ kmaj_copy) {
  pdl_prologue();
  __shared__ uint4 smem[kTileSmemVec];
  const int pcol = threadIdx.x & 31, g = threadIdx.x >> 5;
  const int64_t orow = (int64_t)blockIdx.z * nc + (int64_t)blockIdx.x * 64 + 2 * pcol;
  float d_lo[3] = {1.f, 1.f, 1.f}, d_hi[3] = {1.f, 1.f, 1.f};
  if (ds.per_channel) {
    d_lo[FMT] = ds.get(orow, blockIdx.y == 0 && g == 0);
    d_hi[FMT] = ds.get(orow + 1, blockIdx.y == 0 && g == 0);
  } else {
    d_lo[FMT] = d_hi[FMT] = ds.get(0, blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0);
  }
  uint8_t* const cd[3] = {codes, codes, codes};
  if (ds.from_amax) transpose_tile<1 << FMT, false>(x, nc, c, s_c, s_b, d_lo, d_hi, cd, ldc, kmaj_copy, smem);
  else transpose_tile<1 << FMT, true>(x, nc, c, s_c, s_b, d_lo, d_hi, cd, ldc, kmaj_copy, smem);
}

// Every format in MASK from one read, per-tensor scales from the tensor's max|x|.
template <int MASK>
__global__ void __launch_bounds__(kThreads)
quantize_transpose_tile_multi_kernel(const __nv_bfloat16* __restrict__ x, int64_t nc, int64_t c, int64_t s_c,
                                     int64_t s_b, const uint32_t* __restrict__ amax, const MultiOut o, int64_t ldc,
                                     __nv_bfloat16* __restrict__ kmaj_copy) {
  pdl_prologue();
  __shared__ uint4 smem[kTileSmemVec];
  float d[3];
  multi_scales<MASK>(amax, o, blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0, d);
  uint8_t* const cd[3] = {o.codes[0], o.codes[1], o.codes[2]};
  transpose_tile<MASK, false>(x, nc, c, s_c, s_b, d, d, cd, ldc, kmaj_copy, smem);
}

// ---------------------------------------------------------------- fused per-row scale + quantize
// G lanes own one row: pass 1 reduces max|x| over the row, pass 2 re-reads it (from L1/L2: the
// same lanes touched it a moment ago) and writes codes.  HBM sees each element once.
template <typename T, int FMT, int G>
__global__ void __launch_bounds__(kThreads)
scale_quantize_rows_kernel(const T* __restrict__ x, int64_t nc, int64_t c, int64_t s_nc,
                           int64_t batch, int64_t s_b, float qmax, float* __restrict__ delta_out,
                           uint8_t* __restrict__ codes, int64_t ldc,
                           __nv_bfloat16* __restrict__ abs_copy, uint32_t* __restrict__ err_word) {
  pdl_prologue();
  const int64_t rows = nc * batch;
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int sub = threadIdx.x % G;
  const bool live = row < rows;
  const int64_t b = live ? row / nc : 0, r = live ? row - b * nc : 0;
  const T* p = x + b * s_b + r * s_nc;
  const int64_t nvec = c >> 3;
  uint32_t acc = 0;
  if (live) {
    for (int64_t k = sub; k < nvec; k += G) acc = absmax8(Loader<T>::load8(p + k * 8), acc);
    for (int64_t k = (nvec << 3) + sub; k < c; k += G)
      acc = max(acc, absbits_f32(__float_as_uint(Loader<T>::load1(p, k))));
  }
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) acc = max(acc, __shfl_xor_sync(0xffffffffu, acc, o, G));
  if (!live) return;
  const float d = acc == 0 ? 1.0f : __fdiv_rn(__uint_as_float(acc), qmax);
  if (sub == 0) {
    delta_out[row] = d;
    if (acc >= 0x7f800000u && err_word) atomicOr(err_word, QM_DEVERR_NONFINITE);
  }
  const Quotient quot(d);
  const bool pair_ok = sizeof(T) == 2 && !abs_copy && QuotientPair::serves(d);
  const QuotientPair qp(pair_ok ? d : 1.f);                 // the row's own scale: nothing can overflow
  const int64_t nchunk = ldc >> 3;                          // 8 codes per step, padding included
  for (int64_t k = sub; k < nchunk; k += G) {
    const int64_t k0 = k * 8;
    if (pair_ok && k0 + 8 <= c) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p + k0));
      *reinterpret_cast<uint2*>(codes + row * ldc + k0) = quant_bf16x8<FMT>(raw, qp);
      continue;
    }
    Vec8 v;
    if (k0 + 8 <= c) v = Loader<T>::load8(p + k0);
    else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v.v[j] = k0 + j < c ? Loader<T>::load1(p, k0 + j) : 0.f;
    }
    *reinterpret_cast<uint2*>(codes + row * ldc + k0) = quant8<FMT>(v, quot);
    if (abs_copy) {
      __nv_bfloat16* a = abs_copy + row * c + k0;
      if (k0 + 8 <= c && (c & 7) == 0) *reinterpret_cast<uint4*>(a) = abs_bf16x8(v);
      else
        for (int j = 0; j < 8 && k0 + j < c; ++j) a[j] = __float2bfloat16_rn(fabsf(v.v[j]));
    }
  }
}

// ---------------------------------------------------------------- fused per-row, row held in registers
// bf16 rows of at most VPL * 256 elements (a multiple of 16): one warp per row loads the whole row
// with VPL independent 128-bit loads per lane, reduces max|x| with shuffles, and quantizes from
// the registers.  Every element crosses the memory system once.
template <int FMT, int VPL>
__global__ void __launch_bounds__(kThreads)
scale_quantize_rows_reg_kernel(const __nv_bfloat16* __restrict__ x, int64_t nc, int nvec, int64_t s_nc,
                               int64_t batch, int64_t s_b, float qmax, float* __restrict__ delta_out,
                               uint2* __restrict__ codes, uint4* __restrict__ abs_copy,
                               uint32_t* __restrict__ err_word) {
  pdl_prologue();
  const int64_t rows = nc * batch;
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;                                  // whole warps leave together
  const int64_t b = row / nc, r = row - b * nc;
  const uint4* p = reinterpret_cast<const uint4*>(x + b * s_b + r * s_nc);
  uint4 w[VPL];
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    const int k = lane + 32 * u;
    w[u] = k < nvec ? __ldg(p + k) : make_uint4(0u, 0u, 0u, 0u);
  }
  // max over sign-cleared 16-bit patterns, two per word
  uint32_t m2 = 0;
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    const uint32_t k = 0x7fff7fffu;
    m2 = __vmaxu2(m2, __vmaxu2(__vmaxu2(w[u].x & k, w[u].y & k), __vmaxu2(w[u].z & k, w[u].w & k)));
  }
  uint32_t acc = max(m2 & 0xffffu, m2 >> 16) << 16;         // as an fp32 bit pattern
  acc = warp_max(acc);
  const float d = acc == 0 ? 1.0f : __fdiv_rn(__uint_as_float(acc), qmax);
  if (lane == 0) {
    delta_out[row] = d;
    if (acc >= 0x7f800000u && err_word) atomicOr(err_word, QM_DEVERR_NONFINITE);
  }
  if (!abs_copy && QuotientPair::serves(d)) {
    const QuotientPair qp(d);                                // the row's own scale: nothing can overflow
#pragma unroll
    for (int u = 0; u < VPL; ++u) {
      const int k = lane + 32 * u;
      if (k < nvec) codes[row * nvec + k] = quant_bf16x8<FMT>(w[u], qp);
    }
    return;
  }
  const Quotient quot(d);
#pragma unroll
  for (int u = 0; u < VPL; ++u) {
    const int k = lane + 32 * u;
    if (k >= nvec) break;
    const uint4 v = w[u];
    Vec8 f;
    f.v[0] = bf16_lo(v.x); f.v[1] = bf16_hi(v.x); f.v[2] = bf16_lo(v.y); f.v[3] = bf16_hi(v.y);
    f.v[4] = bf16_lo(v.z); f.v[5] = bf16_hi(v.z); f.v[6] = bf16_lo(v.w); f.v[7] = bf16_hi(v.w);
    codes[row * nvec + k] = quant8<FMT>(f, quot);
    if (abs_copy) {
      const uint32_t m = 0x7fff7fffu;
      abs_copy[row * nvec + k] = make_uint4(v.x & m, v.y & m, v.z & m, v.w & m);
    }
  }
}

// ---------------------------------------------------------------- quantize + transpose
// Storage [c][nc] (nc contiguous) -> codes [nc][ldc] and optional bf16 copies [nc][c].
// A 64(c) x 64(nc) tile goes through shared memory.
template <typename T, int FMT>
__global__ void __launch_bounds__(kThreads)
quantize_transpose_kernel(const T* __restrict__ x, int64_t nc, int64_t c, int64_t s_c, int64_t s_b,
                          const DeltaSrc ds,
                          uint8_t* __restrict__ codes, int64_t ldc,
                          __nv_bfloat16* __restrict__ abs_copy, __nv_bfloat16* __restrict__ kmaj_copy,
                          const Rounding rnd) {
  pdl_prologue();
  __shared__ float tile[64][65];     // +1 column spreads the transposed accesses over the banks
  const int64_t b = blockIdx.z;
  const int64_t c0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
  const T* base = x + b * s_b;
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;    // 8 column-chunks x 32 rows
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int rr = ty + it * 32;
    const int64_t cc = c0 + rr, nn = n0 + tx * 8;
    Vec8 v;
    if (cc < c && nn + 8 <= nc) v = Loader<T>::load8(base + cc * s_c + nn);
    else {
#pragma unroll
      for (int j = 0; j < 8; ++j)
        v.v[j] = (cc < c && nn + j < nc) ? Loader<T>::load1(base, cc * s_c + nn + j) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) tile[rr][tx * 8 + j] = v.v[j];
  }
  __syncthreads();
  // output: row n (64 of them), 64 contraction entries = 8 chunks of 8
  const float d_tensor = ds.per_channel
                             ? 0.f
                             : ds.get(0, blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0);
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int nrow = ty + it * 32;
    const int64_t nn = n0 + nrow;
    if (nn >= nc) continue;
    const int64_t k0 = c0 + tx * 8;
    if (k0 >= ldc) continue;
    Vec8 v;
#pragma unroll
    for (int j = 0; j < 8; ++j) v.v[j] = tile[tx * 8 + j][nrow];
    const Quotient quot(ds.per_channel ? ds.get(b * nc + nn, blockIdx.y == 0 && tx == 0) : d_tensor);
    const int64_t orow = b * nc + nn;
    *reinterpret_cast<uint2*>(codes + orow * ldc + k0) =
        rnd.stochastic ? quant8_sr<FMT>(v, quot, rnd, (uint64_t)orow * (uint64_t)c + (uint64_t)k0)
                       : quant8<FMT>(v, quot);
    if (abs_copy || kmaj_copy) {
      if (k0 + 8 <= c && (c & 7) == 0) {
        if (abs_copy) *reinterpret_cast<uint4*>(abs_copy + orow * c + k0) = abs_bf16x8(v);
        if (kmaj_copy) *reinterpret_cast<uint4*>(kmaj_copy + orow * c + k0) = to_bf16x8(v);
      } else {
        for (int j = 0; j < 8 && k0 + j < c; ++j) {
          if (abs_copy) abs_copy[orow * c + k0 + j] = __float2bfloat16_rn(fabsf(v.v[j]));
          if (kmaj_copy) kmaj_copy[orow * c + k0 + j] = __float2bfloat16_rn(v.v[j]);
        }
      }
    }
  }
}

// ---------------------------------------------------------------- quantize + transpose, bf16 fast path
// Storage [c][nc] (nc contiguous, bf16) with c a multiple of 32 and nc even.  A thread owns two
// adjacent columns and 32 consecutive contraction rows: it issues its 32 four-byte loads (each
// warp-wide load is one 128-byte row segment) before using any, then writes 32 bytes of codes
// and 64 bytes of each bf16 copy per column - whole sectors, no shared memory, no barrier.
// Block = 8 warps = 64 columns x 256 rows.
template <int FMT>
__global__ void __launch_bounds__(kThreads)
quantize_transpose_bf16_kernel(const __nv_bfloat16* __restrict__ x, int64_t nc, int64_t c, int64_t s_c,
                               int64_t s_b, const DeltaSrc ds, uint8_t* __restrict__ codes, int64_t ldc,
                               __nv_bfloat16* __restrict__ abs_copy, __nv_bfloat16* __restrict__ kmaj_copy) {
  pdl_prologue();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t b = blockIdx.z;
  const int64_t n = ((int64_t)blockIdx.x * 32 + lane) * 2;                 // first of this thread's two columns
  const int64_t k0 = ((int64_t)blockIdx.y * 8 + warp) * 32;                // first contraction row
  const float d_tensor =
      ds.per_channel ? 0.f : ds.get(0, blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0);
  if (n >= nc || k0 >= c) return;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(x + b * s_b + k0 * s_c + n);
  const int64_t step = s_c >> 1;                                           // row stride in 32-bit words
  uint32_t w[32];
#pragma unroll
  for (int r = 0; r < 32; ++r) w[r] = __ldg(src + r * step);
#pragma unroll
  for (int col = 0; col < 2; ++col) {
    const int64_t orow = b * nc + n + col;
    const float dv = ds.per_channel ? ds.get(orow, k0 == 0) : d_tensor;
    // this column's 32 values as 16 words of two bf16 each
    uint32_t pw[16];
#pragma unroll
    for (int j = 0; j < 16; ++j)
      pw[j] = col == 0 ? __byte_perm(w[2 * j], w[2 * j + 1], 0x5410) : __byte_perm(w[2 * j], w[2 * j + 1], 0x7632);
    uint4* cdst = reinterpret_cast<uint4*>(codes + orow * ldc + k0);
    if (QuotientPair::serves(dv)) {
      const QuotientPair qp(dv);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint4 a = make_uint4(pw[8 * h], pw[8 * h + 1], pw[8 * h + 2], pw[8 * h + 3]);
        const uint4 bb = make_uint4(pw[8 * h + 4], pw[8 * h + 5], pw[8 * h + 6], pw[8 * h + 7]);
        cdst[h] = ds.from_amax ? quant_bf16x16<FMT, false>(a, bb, qp) : quant_bf16x16<FMT, true>(a, bb, qp);
      }
    } else {
      const Quotient quot(dv);
      uint32_t cw[8];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        Vec8 f;
#pragma unroll
        for (int j = 0; j < 4; ++j) { f.v[2 * j] = bf16_lo(pw[4 * g + j]); f.v[2 * j + 1] = bf16_hi(pw[4 * g + j]); }
        const uint2 q = quant8<FMT>(f, quot);
        cw[2 * g] = q.x; cw[2 * g + 1] = q.y;
      }
      cdst[0] = make_uint4(cw[0], cw[1], cw[2], cw[3]);
      cdst[1] = make_uint4(cw[4], cw[5], cw[6], cw[7]);
    }
    if (abs_copy || kmaj_copy) {
      if (kmaj_copy) {
        uint4* d = reinterpret_cast<uint4*>(kmaj_copy + orow * c + k0);
#pragma unroll
        for (int j = 0; j < 4; ++j) d[j] = make_uint4(pw[4 * j], pw[4 * j + 1], pw[4 * j + 2], pw[4 * j + 3]);
      }
      if (abs_copy) {
        const uint32_t m = 0x7fff7fffu;
        uint4* d = reinterpret_cast<uint4*>(abs_copy + orow * c + k0);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          d[j] = make_uint4(pw[4 * j] & m, pw[4 * j + 1] & m, pw[4 * j + 2] & m, pw[4 * j + 3] & m);
      }
    }
  }
}

int grid_for(int64_t work_items, int per_sm) {
  int64_t want = (work_items + kThreads - 1) / kThreads;
  int64_t cap = (int64_t)sm_count() * per_sm;
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

// max|x| over n dense elements: the 32-byte aligned middle by the 256-bit kernel, what is left at
// either end (less than 32 bytes each) by the general one.
template <typename T>
void absmax_dense(const T* p, int64_t n, uint32_t* amax, cudaStream_t s) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(p), a1 = a0 + (uintptr_t)n * sizeof(T);
  const uintptr_t m0 = (a0 + 31) & ~(uintptr_t)31, m1 = a1 & ~(uintptr_t)31;
  if (m1 <= m0) {
    launch_pdl(absmax_tensor_kernel<T>, dim3(1), dim3(kThreads), 0, s, p, 1, n, n, amax);
    return;
  }
  const uint64_t n_vec = (m1 - m0) / 32;
  const dim3 grid((unsigned)grid_for((int64_t)n_vec, 8));
  const uint8_t* mid = reinterpret_cast<const uint8_t*>(m0);
  if (m1 - m0 > (64u << 20))        // read once and far larger than what stays in L2: evict first
    launch_pdl(absmax_dense_kernel<T, 4, true>, grid, dim3(kThreads), 0, s, mid, n_vec, amax);
  else
    launch_pdl(absmax_dense_kernel<T, 4, false>, grid, dim3(kThreads), 0, s, mid, n_vec, amax);
  const int64_t head = (int64_t)((m0 - a0) / sizeof(T)), tail = (int64_t)((a1 - m1) / sizeof(T));
  if (head > 0) launch_pdl(absmax_tensor_kernel<T>, dim3(1), dim3(32), 0, s, p, 1, head, head, amax);
  if (tail > 0) launch_pdl(absmax_tensor_kernel<T>, dim3(1), dim3(32), 0, s, p + (n - tail), 1, tail, tail, amax);
}

template <typename T>
qm_status absmax_t(const View& x, int gran, uint32_t* amax, cudaStream_t s) {
  const T* p = static_cast<const T*>(x.data);
  if (x.c_contig()) {
    if (gran == QM_GRAN_TENSOR) {
      const bool dense = x.s_nc == x.c && (x.batch == 1 || x.s_b == x.nc * x.c);
      const bool even = x.batch == 1 || x.s_b == x.nc * x.s_nc;
      if (dense) {
        const int64_t n = x.nc * x.batch * x.c;
        absmax_dense<T>(p, n, amax, s);
      } else if (even) {
        launch_pdl(absmax_tensor_kernel<T>, dim3(grid_for(x.nc * x.batch * x.c / 8 + 1, 8)), dim3(kThreads), 0, s, 
            p, x.nc * x.batch, x.c, x.s_nc, amax);
      } else {
        for (int64_t b = 0; b < x.batch; ++b)
          launch_pdl(absmax_tensor_kernel<T>, dim3(grid_for(x.nc * x.c / 8 + 1, 8)), dim3(kThreads), 0, s, 
              p + b * x.s_b, x.nc, x.c, x.s_nc, amax);
      }
    } else {
      const int64_t rows = x.nc * x.batch;
      const int64_t nvec = x.c / 8;
#define QM_ROWS(G)                                                                              \
  launch_pdl(absmax_rows_kernel<T, G>, dim3((unsigned)((rows * G + kThreads - 1) / kThreads)), dim3(kThreads), 0, s,  \
      p, x.nc, x.c, x.s_nc, x.batch, x.s_b, amax)
      if (nvec <= 4) QM_ROWS(4);
      else if (nvec <= 8) QM_ROWS(8);
      else if (nvec <= 16) QM_ROWS(16);
      else QM_ROWS(32);
#undef QM_ROWS
    }
  } else {
    if (gran == QM_GRAN_TENSOR) {
      // storage rows are the contracting index: walk them as rows of nc contiguous elements; the
      // rows of all batch elements form one run when the batch stride continues the row stride
      if (x.batch == 1 || x.s_b == x.c * x.s_c) {
        const bool dense = x.s_c == x.nc;
        const int64_t n = x.nc * x.c * x.batch;
        if (dense)
          absmax_dense<T>(p, n, amax, s);
        else
          launch_pdl(absmax_tensor_kernel<T>, dim3(grid_for(n / 8 + 1, 8)), dim3(kThreads), 0, s,
              p, x.c * x.batch, x.nc, x.s_c, amax);
      } else {
        for (int64_t b = 0; b < x.batch; ++b)
          launch_pdl(absmax_tensor_kernel<T>, dim3(grid_for(x.nc * x.c / 8 + 1, 8)), dim3(kThreads), 0, s,
              p + b * x.s_b, x.c, x.nc, x.s_c, amax);
      }
    } else {
      const int64_t col_blocks = (x.nc + 255) / 256;
      int64_t want_y = ((int64_t)sm_count() * 8 + col_blocks * x.batch - 1) / (col_blocks * x.batch);
      int64_t rows_per_block = (x.c + want_y - 1) / want_y;
      rows_per_block = (rows_per_block + 7) / 8 * 8;
      if (rows_per_block < 64) rows_per_block = 64;
      const int64_t gy = (x.c + rows_per_block - 1) / rows_per_block;
      dim3 grid((unsigned)col_blocks, (unsigned)gy, (unsigned)x.batch), block(32, 8);
      launch_pdl(absmax_cols_kernel<T>, dim3(grid), dim3(block), 0, s, p, x.nc, x.c, x.s_c, x.s_b, rows_per_block, amax);
    }
  }
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

// The shared-memory transposing kernels serve bf16 views whose contraction is strided, in whole
// tiles of 128 contraction entries x 64 columns.
bool tile_transposable(const View& x) {
  return x.dtype == QM_DT_BF16 && !x.c_contig() && (x.c & 127) == 0 && (x.nc & 63) == 0 && x.c / 128 <= 65535 &&
         x.batch <= 65535;
}

template <typename T, int FMT>
qm_status quantize_t(const View& x, int gran, const float* delta, bool from_amax, float* delta_out,
                     uint32_t* err_word, uint8_t* codes, void* abs_copy, void* kmaj_copy, const Rounding& rnd,
                     cudaStream_t s) {
  const T* p = static_cast<const T*>(x.data);
  const int64_t ldc = qm_code_ld(x.c);
  DeltaSrc ds;
  ds.p = delta; ds.per_channel = gran == QM_GRAN_CHANNEL; ds.from_amax = from_amax ? 1 : 0;
  ds.qmax = fmt_qmax(FMT); ds.out = delta_out; ds.err_word = err_word;
  if (x.c_contig()) {
    const int64_t total = x.nc * x.batch * (ldc >> 4);
    if (total >= (1ll << 32) || x.nc >= (1ll << 32)) return QM_ERR_UNSUPPORTED;   // 32-bit chunk index
    // (stochastic rounding takes the general kernels: the draws cost more than the fast paths save)
    const bool dense = !rnd.stochastic && x.dtype == QM_DT_BF16 && x.s_nc == x.c && (x.c & 15) == 0 &&
                       (x.batch == 1 || x.s_b == x.nc * x.c);
    if (dense) {
      const uint4* src = reinterpret_cast<const uint4*>(x.data);
      const FastDiv by_chunks((uint32_t)(ldc >> 4));
      const bool big = total >= (int64_t)sm_count() * 8 * kThreads * 4;
      const bool wide = (reinterpret_cast<uintptr_t>(x.data) & 31) == 0;
      const int64_t per_block = (int64_t)kThreads * (big ? 4 : 1);
      const dim3 grid((unsigned)((total + per_block - 1) / per_block));
#define QM_QD(C, W)                                                                                                 \
  launch_pdl(quantize_dense_kernel<FMT, C, W>, grid, dim3(kThreads), 0, s, src, (uint32_t)total, ds, by_chunks, \
             (uint32_t)(ldc >> 4), reinterpret_cast<uint4*>(codes), reinterpret_cast<uint4*>(abs_copy))
      if (big) { if (wide) QM_QD(4, true); else QM_QD(4, false); }
      else { if (wide) QM_QD(1, true); else QM_QD(1, false); }
#undef QM_QD
    } else
    launch_pdl(quantize_rows_kernel<T, FMT>, dim3(grid_for(total, 16)), dim3(kThreads), 0, s, 
        p, x.nc, x.c, x.s_nc, x.batch, x.s_b, ds, FastDiv((uint32_t)(ldc >> 4)), FastDiv((uint32_t)x.nc),
        codes, ldc, static_cast<__nv_bfloat16*>(abs_copy), rnd);
    if (kmaj_copy) {
      // already contraction-major: a strided copy honours the parameter
      if (x.dtype != QM_DT_BF16) return QM_ERR_UNSUPPORTED;
      for (int64_t b = 0; b < x.batch; ++b)
        QM_CUDA_OK(cudaMemcpy2DAsync(static_cast<uint8_t*>(kmaj_copy) + b * x.nc * x.c * 2, x.c * 2,
                                     static_cast<const uint8_t*>(x.data) + b * x.s_b * 2, x.s_nc * 2,
                                     x.c * 2, x.nc, cudaMemcpyDeviceToDevice, s));
    }
  } else {
    if (!rnd.stochastic && !abs_copy && tile_transposable(x)) {
      dim3 grid((unsigned)(x.nc / 64), (unsigned)(x.c / 128), (unsigned)x.batch);
      launch_pdl(quantize_transpose_tile_kernel<FMT>, dim3(grid), dim3(kThreads), 0, s,
                 static_cast<const __nv_bfloat16*>(x.data), x.nc, x.c, x.s_c, x.s_b, ds, codes, ldc,
                 static_cast<__nv_bfloat16*>(kmaj_copy));
      count_launch();
      QM_CUDA_OK(cudaGetLastError());
      return QM_OK;
    }
    if (!rnd.stochastic && x.dtype == QM_DT_BF16 && (x.c & 31) == 0 && (x.nc & 1) == 0 && (x.c + 255) / 256 <= 65535 &&
        ((x.nc + 63) / 64) * ((x.c + 255) / 256) * x.batch >= 4 * (int64_t)sm_count()) {
      dim3 grid((unsigned)((x.nc + 63) / 64), (unsigned)((x.c + 255) / 256), (unsigned)x.batch);
      launch_pdl(quantize_transpose_bf16_kernel<FMT>, dim3(grid), dim3(kThreads), 0, s, 
          static_cast<const __nv_bfloat16*>(x.data), x.nc, x.c, x.s_c, x.s_b, ds, codes, ldc,
          static_cast<__nv_bfloat16*>(abs_copy), static_cast<__nv_bfloat16*>(kmaj_copy));
      count_launch();
      QM_CUDA_OK(cudaGetLastError());
      return QM_OK;
    }
    dim3 grid((unsigned)((x.nc + 63) / 64), (unsigned)((ldc + 63) / 64), (unsigned)x.batch);
    launch_pdl(quantize_transpose_kernel<T, FMT>, dim3(grid), dim3(kThreads), 0, s, 
        p, x.nc, x.c, x.s_c, x.s_b, ds, codes, ldc, static_cast<__nv_bfloat16*>(abs_copy),
        static_cast<__nv_bfloat16*>(kmaj_copy), rnd);
  }
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

template <typename T, int FMT>
qm_status scale_quantize_rows_t(const View& x, float* delta_out, uint8_t* codes, void* abs_copy,
                                uint32_t* err_word, cudaStream_t s) {
  const T* p = static_cast<const T*>(x.data);
  const int64_t rows = x.nc * x.batch, ldc = qm_code_ld(x.c), nvec = x.c / 8;
  const float qmax = fmt_qmax(FMT);
  if (x.dtype == QM_DT_BF16 && (x.c & 15) == 0 && x.c <= 4 * 256) {
    // the row fits in one warp's registers
    const unsigned blocks = (unsigned)((rows * 32 + kThreads - 1) / kThreads);
    const __nv_bfloat16* pb = static_cast<const __nv_bfloat16*>(x.data);
#define QM_SQR(V)                                                                                 \
  launch_pdl(scale_quantize_rows_reg_kernel<FMT, V>, dim3(blocks), dim3(kThreads), 0, s,                              \
      pb, x.nc, (int)nvec, x.s_nc, x.batch, x.s_b, qmax, delta_out, reinterpret_cast<uint2*>(codes), \
      reinterpret_cast<uint4*>(abs_copy), err_word)
    if (nvec <= 32) QM_SQR(1);
    else if (nvec <= 64) QM_SQR(2);
    else if (nvec <= 128) QM_SQR(4);
    else if (nvec <= 256) QM_SQR(8);
    else QM_SQR(16);
#undef QM_SQR
    count_launch();
    QM_CUDA_OK(cudaGetLastError());
    return QM_OK;
  }
#define QM_SQ(G)                                                                                   \
  launch_pdl(scale_quantize_rows_kernel<T, FMT, G>,                                                \
             dim3((unsigned)((rows * G + kThreads - 1) / kThreads)), dim3(kThreads), 0, s,         \
             p, x.nc, x.c, x.s_nc, x.batch, x.s_b, qmax, delta_out, codes, ldc,                    \
             static_cast<__nv_bfloat16*>(abs_copy), err_word)
  if (nvec <= 4) QM_SQ(4);
  else if (nvec <= 8) QM_SQ(8);
  else if (nvec <= 16) QM_SQ(16);
  else QM_SQ(32);
#undef QM_SQ
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

}  // namespace

qm_status launch_absmax(const View& x, int gran, uint32_t* amax_bits, cudaStream_t s) {
  return x.dtype == QM_DT_BF16 ? absmax_t<__nv_bfloat16>(x, gran, amax_bits, s)
                               : absmax_t<float>(x, gran, amax_bits, s);
}

qm_status launch_share_amax(uint32_t* amax_bits, int64_t batch, int64_t groups, int64_t nc, cudaStream_t s) {
  const int64_t n = groups * nc;
  launch_pdl(share_amax_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, s, amax_bits, batch, groups, nc);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

qm_status launch_finalize_delta(float* delta, int64_t n, int fmt, uint32_t* err_word, cudaStream_t s) {
  launch_pdl(finalize_delta_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, s, delta, n, fmt_qmax(fmt), err_word);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

qm_status launch_quantize(const View& x, int fmt, int gran, const float* delta, bool from_amax,
                          float* delta_out, uint32_t* err_word, uint8_t* codes, void* abs_copy,
                          void* kmaj_copy, cudaStream_t s, const StochasticDraw* draw) {
  Rounding rnd{};
  if (draw) {
    rnd.stochastic = 1;
    rnd.k0 = (uint32_t)draw->seed; rnd.k1 = (uint32_t)(draw->seed >> 32); rnd.stream = draw->stream;
  }
#define QM_ARGS x, gran, delta, from_amax, delta_out, err_word, codes, abs_copy, kmaj_copy, rnd, s
#define QM_Q(T)                                                    \
  (fmt == QM_FMT_INT8   ? quantize_t<T, QM_FMT_INT8>(QM_ARGS)      \
   : fmt == QM_FMT_E4M3 ? quantize_t<T, QM_FMT_E4M3>(QM_ARGS)      \
                        : quantize_t<T, QM_FMT_E5M2>(QM_ARGS))
  return x.dtype == QM_DT_BF16 ? QM_Q(__nv_bfloat16) : QM_Q(float);
#undef QM_Q
#undef QM_ARGS
}

qm_status launch_quantize_multi(const View& x, int gran, const uint32_t* amax, int nf, const int* fmts,
                                float* const* delta_out, uint32_t* const* err_word, uint8_t* const* codes,
                                void* kmaj_copy, cudaStream_t s) {
  if (nf < 1 || nf > 3) return QM_ERR_INVALID_ARG;
  const int64_t ldc = qm_code_ld(x.c);
  int mask = 0;
  MultiOut o{};
  for (int k = 0; k < nf; ++k) {
    const int f = fmts[k];
    if (f < 0 || f > 2 || (mask & (1 << f))) return QM_ERR_INVALID_ARG;
    mask |= 1 << f;
    o.codes[f] = codes[k]; o.delta_out[f] = delta_out[k]; o.err_word[f] = err_word[k];
  }
  bool one_pass = nf > 1 && gran == QM_GRAN_TENSOR && x.dtype == QM_DT_BF16;
  const int64_t total = x.nc * x.batch * (ldc >> 4);
  bool dense = false, transposing = false;
  if (one_pass && x.c_contig()) {
    dense = x.s_nc == x.c && (x.c & 15) == 0 && (x.batch == 1 || x.s_b == x.nc * x.c) && total < (1ll << 32);
    one_pass = dense && !kmaj_copy;
  } else if (one_pass) {
    transposing = tile_transposable(x);
    one_pass = transposing;
  }
  if (!one_pass) {
    // one launch per format; the first one also writes the contraction-major copy
    for (int k = 0; k < nf; ++k) {
      const qm_status st = launch_quantize(x, fmts[k], gran, reinterpret_cast<const float*>(amax), true, delta_out[k],
                                           err_word[k], codes[k], nullptr, k == 0 ? kmaj_copy : nullptr, s);
      if (st != QM_OK) return st;
    }
    return QM_OK;
  }
  if (dense) {
    const uint4* src = reinterpret_cast<const uint4*>(x.data);
    const bool big = total >= (int64_t)sm_count() * 8 * kThreads * 4;
    const int64_t per_block = (int64_t)kThreads * (big ? 4 : 1);
    const dim3 grid((unsigned)((total + per_block - 1) / per_block));
    const bool wide = (reinterpret_cast<uintptr_t>(x.data) & 31) == 0;
#define QM_DM(M)                                                                                                           \
  (big ? (wide ? launch_pdl(quantize_dense_multi_kernel<M, 4, true>, grid, dim3(kThreads), 0, s, src, (uint32_t)total, amax, o)    \
               : launch_pdl(quantize_dense_multi_kernel<M, 4, false>, grid, dim3(kThreads), 0, s, src, (uint32_t)total, amax, o))  \
       : (wide ? launch_pdl(quantize_dense_multi_kernel<M, 1, true>, grid, dim3(kThreads), 0, s, src, (uint32_t)total, amax, o)    \
               : launch_pdl(quantize_dense_multi_kernel<M, 1, false>, grid, dim3(kThreads), 0, s, src, (uint32_t)total, amax, o)))
    switch (mask) {
      case 3: QM_DM(3); break;
      case 5: QM_DM(5); break;
      case 6: QM_DM(6); break;
      default: QM_DM(7); break;
    }
#undef QM_DM
  } else {
    dim3 grid((unsigned)(x.nc / 64), (unsigned)(x.c / 128), (unsigned)x.batch);
    const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(x.data);
    __nv_bfloat16* km = static_cast<__nv_bfloat16*>(kmaj_copy);
#define QM_TM(M) launch_pdl(quantize_transpose_tile_multi_kernel<M>, grid, dim3(kThreads), 0, s, src, x.nc, x.c, x.s_c, x.s_b, amax, o, ldc, km)
    switch (mask) {
      case 3: QM_TM(3); break;
      case 5: QM_TM(5); break;
      case 6: QM_TM(6); break;
      default: QM_TM(7); break;
    }
#undef QM_TM
  }
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

qm_status launch_scale_quantize_rows(const View& x, int fmt, float* delta_out, uint8_t* codes,
                                     void* abs_copy, uint32_t* err_word, cudaStream_t s) {
#define QM_Q(T)                                                                                       \
  (fmt == QM_FMT_INT8   ? scale_quantize_rows_t<T, QM_FMT_INT8>(x, delta_out, codes, abs_copy, err_word, s) \
   : fmt == QM_FMT_E4M3 ? scale_quantize_rows_t<T, QM_FMT_E4M3>(x, delta_out, codes, abs_copy, err_word, s) \
                        : scale_quantize_rows_t<T, QM_FMT_E5M2>(x, delta_out, codes, abs_copy, err_word, s))
  return x.dtype == QM_DT_BF16 ? QM_Q(__nv_bfloat16) : QM_Q(float);
#undef QM_Q
}

}  // namespace qm
