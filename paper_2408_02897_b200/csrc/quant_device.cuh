// Device helpers shared by the streaming kernels (scale, quantize, tensor statistics, Eq. 2
// error split): element loads, the exact quotient of Eq. 1, the 8-bit conversions, small
// reductions.  Included by .cu files only; everything sits in the including file's anonymous
// namespace.
#pragma once
#include <cuda_bf16.h>

#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kThreads = 256;

// ---------------------------------------------------------------- element helpers
// |x| as an order-preserving unsigned integer: for IEEE formats the bit pattern with the sign
// cleared orders like the magnitude, and Inf / NaN patterns sort above every finite value, so
// an integer max also carries "non-finite seen" to the end.  bf16 patterns are widened to the
// fp32 pattern (shift by 16) so one code path serves both input types.
__device__ __forceinline__ uint32_t absbits_f32(uint32_t w) { return w & 0x7fffffffu; }

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// 32 bytes in one load (sm_100 has 256-bit global loads), read-only path, no L1 allocation.
// STREAM adds evict-first in L2: for tensors much larger than L2 that are read once per pass.
struct Vec256 { uint4 lo, hi; };
template <bool STREAM>
__device__ __forceinline__ Vec256 ld256(const void* p) {
  Vec256 v;
  if (STREAM)
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.lo.x), "=r"(v.lo.y), "=r"(v.lo.z), "=r"(v.lo.w), "=r"(v.hi.x), "=r"(v.hi.y), "=r"(v.hi.z), "=r"(v.hi.w)
                 : "l"(p));
  else
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v.lo.x), "=r"(v.lo.y), "=r"(v.lo.z), "=r"(v.lo.w), "=r"(v.hi.x), "=r"(v.hi.y), "=r"(v.hi.z), "=r"(v.hi.w)
                 : "l"(p));
  return v;
}

// Two quantized bytes from t = x / delta: t0 in bits 0..7, t1 in bits 8..15.
// RTNE, saturating at the largest finite magnitude.
template <int FMT>
__device__ __forceinline__ uint32_t quant2(float t0, float t1) {
  if (FMT == QM_FMT_INT8) {
    int a = __float2int_rn(t0), b = __float2int_rn(t1);      // round to nearest even
    a = max(-127, min(127, a));
    b = max(-127, min(127, b));
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8);
  } else {
    uint16_t r;
    if (FMT == QM_FMT_E4M3)
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(t1), "f"(t0));
    else
      asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(t1), "f"(t0));
    return r;
  }
}

// 8 consecutive elements held as fp32.
struct Vec8 { float v[8]; };

template <typename T> struct Loader;
template <> struct Loader<__nv_bfloat16> {
  static __device__ __forceinline__ Vec8 load8(const void* p) {
    uint4 w = __ldg(reinterpret_cast<const uint4*>(p));
    Vec8 r;
    r.v[0] = bf16_lo(w.x); r.v[1] = bf16_hi(w.x); r.v[2] = bf16_lo(w.y); r.v[3] = bf16_hi(w.y);
    r.v[4] = bf16_lo(w.z); r.v[5] = bf16_hi(w.z); r.v[6] = bf16_lo(w.w); r.v[7] = bf16_hi(w.w);
    return r;
  }
  static __device__ __forceinline__ float load1(const void* p, int64_t i) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p) + i) << 16);
  }
};
template <> struct Loader<float> {
  static __device__ __forceinline__ Vec8 load8(const void* p) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    Vec8 r;
    r.v[0] = a.x; r.v[1] = a.y; r.v[2] = a.z; r.v[3] = a.w;
    r.v[4] = b.x; r.v[5] = b.y; r.v[6] = b.z; r.v[7] = b.w;
    return r;
  }
  static __device__ __forceinline__ float load1(const void* p, int64_t i) {
    return __ldg(reinterpret_cast<const float*>(p) + i);
  }
};

__device__ __forceinline__ uint32_t absmax8(const Vec8& x, uint32_t acc) {
#pragma unroll
  for (int i = 0; i < 8; ++i) acc = max(acc, absbits_f32(__float_as_uint(x.v[i])));
  return acc;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // round to nearest even
  return *reinterpret_cast<uint32_t*>(&h);
}

// x / delta, correctly rounded (the IEEE quotient Eq. 1 asks for), for many x under one delta.
// With r = RN(1/delta) computed once per scaling group, a product and two residual corrections
//   q0 = x r;  q1 = q0 + (x - q0 delta) r;  q = q1 + (x - q1 delta) r      (residuals exact by FMA)
// give RN(x / delta): q1 is within one ulp of the quotient, and one more correction of a
// faithful quotient with the correctly rounded reciprocal rounds correctly (Markstein's
// theorem).  This needs the intermediate values inside the normal range, so it is used only for
// 2^-60 <= delta <= 2^60, where any |x| small enough to leave that range quantizes to zero in
// every format; other deltas take the division instruction sequence.
struct Quotient {
  float delta, recip;
  bool fast;
  __device__ __forceinline__ explicit Quotient(float d) : delta(d) {
    fast = d >= 8.6736174e-19f && d <= 1.1529215e18f;        // 2^-60 .. 2^60
    recip = fast ? __frcp_rn(d) : 0.f;
  }
  __device__ __forceinline__ float operator()(float x) const {
    if (!fast) return __fdiv_rn(x, delta);
    const float q0 = x * recip;
    const float q1 = fmaf(fmaf(-q0, delta, x), recip, q0);
    const float q = fmaf(fmaf(-q1, delta, x), recip, q1);
    // A delta handed in from elsewhere (stale, shared) can make x * recip overflow; the corrections
    // then evaluate inf - inf.  fminf returns its non-NaN operand, so that case comes out as the
    // largest float and saturates in the conversion, as the division would.
    return copysignf(fminf(fabsf(q), 3.402823466e38f), x);    // keeps the sign of a zero input
  }
};

// The same correctly rounded quotient for two elements at once with the two-wide fp32
// instructions (one mul and four fma for a pair), for scales taken from the operand's own max|x|:
// |x / delta| then never exceeds the format's largest value by more than a rounding, so nothing
// overflows and the guard of Quotient is not needed.  Only the fast range of delta is served;
// callers fall back to Quotient otherwise.
struct QuotientPair {
  uint64_t recip2, ndelta2;
  __device__ __forceinline__ explicit QuotientPair(float d) {
    const float r = __frcp_rn(d), nd = -d;
    asm("mov.b64 %0, {%1, %1};" : "=l"(recip2) : "f"(r));
    asm("mov.b64 %0, {%1, %1};" : "=l"(ndelta2) : "f"(nd));
  }
  static __device__ __forceinline__ bool serves(float d) { return d >= 8.6736174e-19f && d <= 1.1529215e18f; }
  // x2 = {x0, x1} packed; returns {RN(x0 / delta), RN(x1 / delta)} packed (a zero comes out as +0)
  __device__ __forceinline__ uint64_t operator()(uint64_t x2) const {
    uint64_t q0, t, q1, q;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(q0) : "l"(x2), "l"(recip2));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t) : "l"(q0), "l"(ndelta2), "l"(x2));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q1) : "l"(t), "l"(recip2), "l"(q0));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(t) : "l"(q1), "l"(ndelta2), "l"(x2));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(q) : "l"(t), "l"(recip2), "l"(q1));
    return q;
  }
};

// Two codes (bits 0..7 and 8..15) of the bf16 pair held in word w (low half = first element).
// GUARD: the scale may come from elsewhere, so x r can overflow and the corrections then evaluate
// inf - inf; fminf returns its non-NaN operand, which turns that case into the largest float and
// lets the conversion saturate, as the division would.
template <int FMT, bool GUARD = false>
__device__ __forceinline__ uint32_t quant_bf16_pair(uint32_t w, const QuotientPair& quot) {
  uint64_t x2;
  asm("mov.b64 %0, {%1, %2};" : "=l"(x2) : "r"(w << 16), "r"(w & 0xffff0000u));
  const uint64_t q2 = quot(x2);
  uint32_t q0, q1;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(q0), "=r"(q1) : "l"(q2));
  if (GUARD) {
    q0 = __float_as_uint(fminf(fabsf(__uint_as_float(q0)), 3.402823466e38f)) | ((w << 16) & 0x80000000u);
    q1 = __float_as_uint(fminf(fabsf(__uint_as_float(q1)), 3.402823466e38f)) | (w & 0x80000000u);
    return quant2<FMT>(__uint_as_float(q0), __uint_as_float(q1));
  }
  if (FMT == QM_FMT_INT8) {
    return quant2<FMT>(__uint_as_float(q0), __uint_as_float(q1));
  } else {
    // a negative input that rounds to zero is -0 in the FP8 formats: give the quotient its sign back
    q0 |= (w << 16) & 0x80000000u;
    q1 |= w & 0x80000000u;
    return quant2<FMT>(__uint_as_float(q0), __uint_as_float(q1));
  }
}

// Sixteen codes of sixteen consecutive bf16 values (two 128-bit words).
template <int FMT, bool GUARD = false>
__device__ __forceinline__ uint4 quant_bf16x16(const uint4& a, const uint4& b, const QuotientPair& quot) {
  uint4 r;
  r.x = quant_bf16_pair<FMT, GUARD>(a.x, quot) | (quant_bf16_pair<FMT, GUARD>(a.y, quot) << 16);
  r.y = quant_bf16_pair<FMT, GUARD>(a.z, quot) | (quant_bf16_pair<FMT, GUARD>(a.w, quot) << 16);
  r.z = quant_bf16_pair<FMT, GUARD>(b.x, quot) | (quant_bf16_pair<FMT, GUARD>(b.y, quot) << 16);
  r.w = quant_bf16_pair<FMT, GUARD>(b.z, quot) | (quant_bf16_pair<FMT, GUARD>(b.w, quot) << 16);
  return r;
}

// Eight codes of eight consecutive bf16 values (one 128-bit word).
template <int FMT, bool GUARD = false>
__device__ __forceinline__ uint2 quant_bf16x8(const uint4& a, const QuotientPair& quot) {
  uint2 r;
  r.x = quant_bf16_pair<FMT, GUARD>(a.x, quot) | (quant_bf16_pair<FMT, GUARD>(a.y, quot) << 16);
  r.y = quant_bf16_pair<FMT, GUARD>(a.z, quot) | (quant_bf16_pair<FMT, GUARD>(a.w, quot) << 16);
  return r;
}

template <int FMT>
__device__ __forceinline__ uint2 quant8(const Vec8& x, const Quotient& quot) {
  float t[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) t[i] = quot(x.v[i]);
  uint2 r;
  r.x = quant2<FMT>(t[0], t[1]) | (quant2<FMT>(t[2], t[3]) << 16);
  r.y = quant2<FMT>(t[4], t[5]) | (quant2<FMT>(t[6], t[7]) << 16);
  return r;
}

// ---------------------------------------------------------------- stochastic rounding
// Second rounding mode of the Methodology section.  The uniform number of element i of an operand
// is word (i mod 4) of Philox4x32-10 (Salmon et al., SC'11) with counter (i div 4 as two words,
// stream, 0) and the seed's two words as key; u = (word >> 8) / 2^24.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Rounding mode of one quantize launch, passed by value.
struct Rounding {
  int stochastic;
  uint32_t k0, k1;      // seed, low and high word
  uint32_t stream;      // which operand of the probe draws (0 = left, 1 = right)
};

// t = x / delta moved onto the format's grid: with lo <= |t| <= hi the neighbouring expressible
// magnitudes (|t| capped at the largest one first), hi when u (hi - lo) < |t| - lo and lo
// otherwise.  Both sides of the comparison are exact in fp32 (hi - lo is a power of two and
// |t| - lo a difference inside one binade), so the decision equals the one taken in exact
// arithmetic.  The sign of t is kept.
template <int FMT>
__device__ __forceinline__ float sr_value(float t, uint32_t word) {
  const float a = fminf(fabsf(t), fmt_qmax(FMT));
  const float u = (float)(word >> 8) * 5.9604644775390625e-8f;          // 2^-24, exact
  float lo, spacing;
  if (FMT == QM_FMT_INT8) {
    lo = floorf(a);
    spacing = 1.f;
  } else {
    constexpr int m = FMT == QM_FMT_E4M3 ? 3 : 2;                        // mantissa bits
    constexpr int emin = FMT == QM_FMT_E4M3 ? -6 : -14;                  // smallest normal exponent
    const float min_normal = __uint_as_float((uint32_t)(127 + emin) << 23);
    if (a >= min_normal) {
      const uint32_t bits = __float_as_uint(a) & ~((1u << (23 - m)) - 1u);   // mantissa cut to m bits
      lo = __uint_as_float(bits);
      spacing = __uint_as_float(((bits >> 23) - m) << 23);
    } else {
      spacing = __uint_as_float((uint32_t)(127 + emin - m) << 23);       // the subnormal step
      lo = floorf(a * __uint_as_float((uint32_t)(127 - emin + m) << 23)) * spacing;
    }
  }
  const float r = (u * spacing < a - lo) ? lo + spacing : lo;
  return copysignf(r, t);
}

// Eight consecutive elements whose first has number idx0 in the operand.  ALIGNED: idx0 is a
// multiple of 4 (rows whose length is one, the common case), so the eight draws are exactly the
// words of two counter blocks; otherwise they straddle three.
template <int FMT, bool ALIGNED>
__device__ __forceinline__ uint2 quant8_sr(const Vec8& x, const Quotient& quot, const Rounding& rnd,
                                           uint64_t idx0) {
  uint32_t w[12];
  const uint64_t blk = idx0 >> 2;
  const int first = ALIGNED ? 0 : (int)(idx0 & 3);
#pragma unroll
  for (int b = 0; b < (ALIGNED ? 2 : 3); ++b) {
    const uint64_t c = blk + b;
    philox4x32_10((uint32_t)c, (uint32_t)(c >> 32), rnd.stream, 0u, rnd.k0, rnd.k1,
                  *reinterpret_cast<uint32_t(*)[4]>(&w[4 * b]));
  }
  float t[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t word = w[i];
    if (!ALIGNED) {
      // word first + i without dynamic indexing of the register array
#pragma unroll
      for (int f = 1; f < 4; ++f)
        if (first == f) word = w[f + i];
    }
    t[i] = sr_value<FMT>(quot(x.v[i]), word);
  }
  uint2 r;
  r.x = quant2<FMT>(t[0], t[1]) | (quant2<FMT>(t[2], t[3]) << 16);
  r.y = quant2<FMT>(t[4], t[5]) | (quant2<FMT>(t[6], t[7]) << 16);
  return r;
}
// The same, choosing the variant from idx0 (uniform over a launch whenever rows are a multiple of 4 long).
template <int FMT>
__device__ __forceinline__ uint2 quant8_sr(const Vec8& x, const Quotient& quot, const Rounding& rnd,
                                           uint64_t idx0) {
  return (idx0 & 3) == 0 ? quant8_sr<FMT, true>(x, quot, rnd, idx0) : quant8_sr<FMT, false>(x, quot, rnd, idx0);
}

__device__ __forceinline__ uint4 abs_bf16x8(const Vec8& x) {
  uint4 r;
  r.x = pack_bf16x2(fabsf(x.v[0]), fabsf(x.v[1]));
  r.y = pack_bf16x2(fabsf(x.v[2]), fabsf(x.v[3]));
  r.z = pack_bf16x2(fabsf(x.v[4]), fabsf(x.v[5]));
  r.w = pack_bf16x2(fabsf(x.v[6]), fabsf(x.v[7]));
  return r;
}
__device__ __forceinline__ uint4 to_bf16x8(const Vec8& x) {
  uint4 r;
  r.x = pack_bf16x2(x.v[0], x.v[1]); r.y = pack_bf16x2(x.v[2], x.v[3]);
  r.z = pack_bf16x2(x.v[4], x.v[5]); r.w = pack_bf16x2(x.v[6], x.v[7]);
  return r;
}

__device__ __forceinline__ uint32_t warp_max(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ uint32_t block_max(uint32_t v) {
  __shared__ uint32_t s[32];
  v = warp_max(v);
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) s[w] = v;
  __syncthreads();
  if (w == 0) {
    v = lane < (int)(blockDim.x >> 5) ? s[lane] : 0u;
    v = warp_max(v);
  }
  return v;   // valid in warp 0
}

// Division of a 32-bit index by a launch-time constant without a divide instruction
// (multiply-high and shift; the magic numbers come from the host).
struct FastDiv {
  uint32_t d, m, s;
  __host__ FastDiv(uint32_t div = 1) : d(div), m(0), s(0) {
    if (d > 1) {
      while ((1ull << s) < d) ++s;                          // s = ceil(log2 d)
      m = (uint32_t)((((1ull << s) - d) << 32) / d + 1);
    }
  }
  __device__ __forceinline__ uint32_t div(uint32_t n) const {
    if (d == 1) return n;
    const uint32_t t = __umulhi(m, n);
    return (t + ((n - t) >> 1)) >> (s - 1);
  }
};

}  // namespace
}  // namespace qm
