// CUDA-core versions of the probe's products.  They serve the fp32-reference configuration
// (fp32 operands have no tensor-core path with an fp32 multiply) and act as a second opinion
// for the tensor-core kernels in the tests.  Not tuned.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kTile = 64;     // output tile edge
constexpr int kStep = 16;     // contraction step
constexpr int kThreads = 256; // 16 x 16 threads, 4 x 4 outputs each

__device__ __forceinline__ float decode_code(uint8_t c, int fmt) {
  if (fmt == QM_FMT_INT8) return (float)(int8_t)c;
  uint32_t h2;
  uint16_t in = c;
  if (fmt == QM_FMT_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
  else asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(in));
  __half lo = __ushort_as_half((unsigned short)(h2 & 0xffffu));
  return __half2float(lo);
}

__device__ __forceinline__ float load_elem(const void* p, int dtype, int64_t off) {
  if (dtype == QM_DT_BF16)
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p) + off) << 16);
  return __ldg(reinterpret_cast<const float*>(p) + off);
}

struct SimtArgs {
  const void* l; int l_dt; int64_t l_snc, l_sc, l_sb;
  const void* r; int r_dt; int64_t r_snc, r_sc, r_sb;
  const uint8_t* cl; const uint8_t* cr; int64_t ldc;
  int fmt_l, fmt_r;
  const float* dl; int pc_l;
  const float* dr; int pc_r;
  int64_t M, N, K;
  float* out_descaled; void* out_raw;
  double* partials;
};

// PROBE: three accumulators (reference, denominator, 8-bit) and the Eq. 3 partial sums.
// otherwise: the 8-bit product only, written out.
template <bool IS_INT, bool PROBE>
__global__ void __launch_bounds__(kThreads) simt_kernel(SimtArgs a) {
  __shared__ float sL[kStep][kTile + 1], sR[kStep][kTile + 1];
  __shared__ float sLq[kStep][kTile + 1], sRq[kStep][kTile + 1];
  __shared__ double sred[5][kThreads / 32];
  const int64_t b = blockIdx.z;
  const int64_t m0 = (int64_t)blockIdx.y * kTile, n0 = (int64_t)blockIdx.x * kTile;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

  float accC[4][4], accD[4][4], accF[4][4];
  int accI[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { accC[i][j] = 0.f; accD[i][j] = 0.f; accF[i][j] = 0.f; accI[i][j] = 0; }

  for (int64_t k0 = 0; k0 < a.K; k0 += kStep) {
    // fill: 64 rows x 16 k per operand, 4 elements per thread
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = threadIdx.x + e * kThreads;   // 0..1023
      const int row = idx >> 4, kk = idx & 15;
      const int64_t k = k0 + kk;
      const int64_t mi = m0 + row, ni = n0 + row;
      const bool okl = mi < a.M && k < a.K, okr = ni < a.N && k < a.K;
      if (PROBE) {
        sL[kk][row] = okl ? load_elem(a.l, a.l_dt, b * a.l_sb + mi * a.l_snc + k * a.l_sc) : 0.f;
        sR[kk][row] = okr ? load_elem(a.r, a.r_dt, b * a.r_sb + ni * a.r_snc + k * a.r_sc) : 0.f;
      }
      sLq[kk][row] = okl ? decode_code(__ldg(a.cl + (b * a.M + mi) * a.ldc + k), a.fmt_l) : 0.f;
      sRq[kk][row] = okr ? decode_code(__ldg(a.cr + (b * a.N + ni) * a.ldc + k), a.fmt_r) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kStep; ++kk) {
      float lv[4], rv[4], lq[4], rq[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        lq[i] = sLq[kk][ty * 4 + i]; rq[i] = sRq[kk][tx * 4 + i];
        if (PROBE) { lv[i] = sL[kk][ty * 4 + i]; rv[i] = sR[kk][tx * 4 + i]; }
        else { lv[i] = 0.f; rv[i] = 0.f; }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (PROBE) {
            accC[i][j] = fmaf(lv[i], rv[j], accC[i][j]);
            accD[i][j] = fmaf(fabsf(lv[i]), fabsf(rv[j]), accD[i][j]);
          }
          if (IS_INT) accI[i][j] += (int)lq[i] * (int)rq[j];
          else accF[i][j] = fmaf(lq[i], rq[j], accF[i][j]);
        }
    }
    __syncthreads();
  }

  const float dl_t = a.pc_l ? 0.f : __ldg(a.dl), dr_t = a.pc_r ? 0.f : __ldg(a.dr);
  float fbe = 0, fmx = 0, fd2 = 0, fr2 = 0, fn2 = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t mi = m0 + ty * 4 + i;
    if (mi >= a.M) continue;
    const float dl = a.pc_l ? __ldg(a.dl + b * a.M + mi) : dl_t;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t ni = n0 + tx * 4 + j;
      if (ni >= a.N) continue;
      const float dr = a.pc_r ? __ldg(a.dr + b * a.N + ni) : dr_t;
      const float acc = IS_INT ? (float)accI[i][j] : accF[i][j];
      const float q = acc * (dl * dr);
      if (PROBE) {
        const float c = accC[i][j], d = accD[i][j];
        const float diff = c - q;
        const float be = d != 0.f ? __fdiv_rn(fabsf(diff), d) : 0.f;
        fbe += be; fmx = fmaxf(fmx, be);
        fd2 = fmaf(diff, diff, fd2); fr2 = fmaf(c, c, fr2); fn2 = fmaf(d, d, fn2);
      } else {
        const int64_t o = (b * a.M + mi) * a.N + ni;
        if (a.out_descaled) a.out_descaled[o] = q;
        if (a.out_raw) {
          if (IS_INT) reinterpret_cast<int*>(a.out_raw)[o] = accI[i][j];
          else reinterpret_cast<float*>(a.out_raw)[o] = accF[i][j];
        }
      }
    }
  }
  if (PROBE) {
    double v[5] = {fbe, fmx, fd2, fr2, fn2};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
      v[1] = fmax(v[1], __shfl_xor_sync(0xffffffffu, v[1], o));
      v[2] += __shfl_xor_sync(0xffffffffu, v[2], o);
      v[3] += __shfl_xor_sync(0xffffffffu, v[3], o);
      v[4] += __shfl_xor_sync(0xffffffffu, v[4], o);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0)
      for (int i = 0; i < 5; ++i) sred[i][w] = v[i];
    __syncthreads();
    if (threadIdx.x == 0) {
      double r[5] = {0, 0, 0, 0, 0};
      for (int i = 0; i < kThreads / 32; ++i) {
        r[0] += sred[0][i]; r[1] = fmax(r[1], sred[1][i]); r[2] += sred[2][i];
        r[3] += sred[3][i]; r[4] += sred[4][i];
      }
      const int64_t blk = ((int64_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
      for (int i = 0; i < 5; ++i) a.partials[blk * kPartialDoubles + i] = r[i];
    }
  }
}

dim3 grid_of(GemmShape g) {
  return dim3((unsigned)((g.N + kTile - 1) / kTile), (unsigned)((g.M + kTile - 1) / kTile),
              (unsigned)g.batch);
}

}  // namespace

int simt_probe_blocks(GemmShape g) {
  dim3 d = grid_of(g);
  return (int)(d.x * d.y * d.z);
}

qm_status launch_simt_gemm_lp(const uint8_t* cl, int fmt_l, const float* dl, int gran_l,
                              const uint8_t* cr, int fmt_r, const float* dr, int gran_r,
                              GemmShape g, float* out_descaled, void* out_raw, cudaStream_t s) {
  if (g.batch > 65535 || (g.M + kTile - 1) / kTile > 65535) return QM_ERR_UNSUPPORTED;
  SimtArgs a{};
  a.cl = cl; a.cr = cr; a.ldc = qm_code_ld(g.K); a.fmt_l = fmt_l; a.fmt_r = fmt_r;
  a.dl = dl; a.pc_l = gran_l == QM_GRAN_CHANNEL; a.dr = dr; a.pc_r = gran_r == QM_GRAN_CHANNEL;
  a.M = g.M; a.N = g.N; a.K = g.K; a.out_descaled = out_descaled; a.out_raw = out_raw;
  if (fmt_l == QM_FMT_INT8) simt_kernel<true, false><<<grid_of(g), kThreads, 0, s>>>(a);
  else simt_kernel<false, false><<<grid_of(g), kThreads, 0, s>>>(a);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

qm_status launch_simt_probe(const View& L, const View& R, const uint8_t* cl, int fmt_l,
                            const float* dl, int gran_l, const uint8_t* cr, int fmt_r,
                            const float* dr, int gran_r, double* partials, cudaStream_t s) {
  GemmShape g{L.nc, R.nc, L.c, L.batch};
  if (g.batch > 65535 || (g.M + kTile - 1) / kTile > 65535) return QM_ERR_UNSUPPORTED;
  SimtArgs a{};
  a.l = L.data; a.l_dt = L.dtype; a.l_snc = L.s_nc; a.l_sc = L.s_c; a.l_sb = L.s_b;
  a.r = R.data; a.r_dt = R.dtype; a.r_snc = R.s_nc; a.r_sc = R.s_c; a.r_sb = R.s_b;
  a.cl = cl; a.cr = cr; a.ldc = qm_code_ld(L.c); a.fmt_l = fmt_l; a.fmt_r = fmt_r;
  a.dl = dl; a.pc_l = gran_l == QM_GRAN_CHANNEL; a.dr = dr; a.pc_r = gran_r == QM_GRAN_CHANNEL;
  a.M = L.nc; a.N = R.nc; a.K = L.c; a.partials = partials;
  if (fmt_l == QM_FMT_INT8) simt_kernel<true, true><<<grid_of(g), kThreads, 0, s>>>(a);
  else simt_kernel<false, true><<<grid_of(g), kThreads, 0, s>>>(a);
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

}  // namespace qm
