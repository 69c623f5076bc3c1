// Tensor-core products of the probe for sm_100a: tcgen05.mma with accumulators in tensor
// memory, operands staged in shared memory by TMA, warp-specialised roles.
//
// One CTA owns one 128 x 128 output tile.  Roles:
//   warp 0      TMA producer: per k-block, bulk-tensor loads of every operand tile into a ring
//   warp 1      allocates tensor memory; one lane issues the MMAs of each k-block
//   warps 2..5  epilogue: read the accumulators with tcgen05.ld and either reduce the Eq. 3
//               statistics (probe) or store the product.
// In probe mode three accumulators live side by side in tensor memory: the reference L.R
// (bf16 operands, kind::f16), the denominator |L|.|R| (bf16, kind::f16) and the 8-bit product
// (kind::f8f6f4 or kind::i8), so no M x N matrix ever goes to HBM.
//
// Every wait is bounded: when one gives up it raises QM_DEVERR_TIMEOUT in the caller's error
// word and flags the CTA, after which every role falls through to the common exit, tensor
// memory is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kBlockM = 128, kBlockN = 128, kBlockK = 64;
constexpr int kThreads = 192;
constexpr uint32_t kBf16TileBytes = kBlockM * kBlockK * 2;   // 16 KB, 128-byte rows
constexpr uint32_t kLpTileBytes = kBlockM * kBlockK;         //  8 KB,  64-byte rows

enum Mode { kProbe = 0, kLpOnly = 1, kRefOnly = 2 };

template <int MODE> struct Cfg;
template <> struct Cfg<kProbe> {
  static constexpr int kStages = 2;
  static constexpr uint32_t kStageBytes = 4 * kBf16TileBytes + 2 * kLpTileBytes;
  static constexpr uint32_t kTmemCols = 512;
};
template <> struct Cfg<kLpOnly> {
  static constexpr int kStages = 8;
  static constexpr uint32_t kStageBytes = 2 * kLpTileBytes;
  static constexpr uint32_t kTmemCols = 128;
};
template <> struct Cfg<kRefOnly> {
  static constexpr int kStages = 6;
  static constexpr uint32_t kStageBytes = 2 * kBf16TileBytes;
  static constexpr uint32_t kTmemCols = 128;
};

struct KernelArgs {
  int64_t M, N, K;
  const float* dl; int pc_l;      // per-channel flags: delta indexed by batch*M + row
  const float* dr; int pc_r;
  float* out_descaled;            // LpOnly / RefOnly
  void* out_raw;                  // LpOnly
  double* partials;               // Probe
  uint32_t* err_word;
  uint32_t idesc_lp;              // instruction descriptor of the 8-bit MMA
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when the CTA has been flagged or the time limit (1 s) ran out;
// in the second case it flags the CTA and the caller's error word.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* err_word) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  uint32_t polls = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++polls & 0xffu) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > 1000000000ull) {
        *abort_flag = 1u;
        if (err_word) atomicOr(err_word, QM_DEVERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

// Shared-memory matrix descriptor, contraction-major tile with a 128- or 64-byte swizzle:
// rows are one swizzle span wide, eight consecutive rows form one swizzle atom, atoms follow
// each other every 8 * span bytes (the "stride byte offset").
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t span_bytes) {
  const uint64_t layout = span_bytes == 128 ? 2ull : 4ull;      // SWIZZLE_128B : SWIZZLE_64B
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);                      // start address / 16
  d |= (uint64_t)1 << 16;                                       // leading byte offset (unused here)
  d |= (uint64_t)((8u * span_bytes) >> 4) << 32;                // stride byte offset / 16
  d |= (uint64_t)1 << 46;                                       // descriptor version of sm_100
  d |= layout << 61;
  return d;
}

enum MmaKind { kKindF16 = 0, kKindF8 = 1, kKindI8 = 2 };

template <int KIND>
__device__ __forceinline__ void mma_ss(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc,
                                       uint32_t accumulate) {
  if (KIND == kKindF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  } else if (KIND == kKindF8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  }
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (base lane + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Instruction descriptor: D format [4,6), A format [7,10), B format [10,13), majors [15],[16]
// (0 = contraction-major), N/8 at [17,23), M/16 at [24,29).
__host__ __device__ constexpr uint32_t make_idesc(uint32_t c_fmt, uint32_t a_fmt, uint32_t b_fmt,
                                                  uint32_t m, uint32_t n) {
  return (c_fmt << 4) | (a_fmt << 7) | (b_fmt << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

struct Shared {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t tmem_full;
  uint32_t tmem_base;
  uint32_t abort_flag;
  float delta_r[kBlockN];
  double red[5][4];
};

template <int MODE, int LPKIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_kernel(const __grid_constant__ CUtensorMap map_l, const __grid_constant__ CUtensorMap map_r,
          const __grid_constant__ CUtensorMap map_la, const __grid_constant__ CUtensorMap map_ra,
          const __grid_constant__ CUtensorMap map_cl, const __grid_constant__ CUtensorMap map_cr,
          const KernelArgs a) {
  using C = Cfg<MODE>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + (size_t)kStages * C::kStageBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tile = blockIdx.x, m_tile = blockIdx.y, b = blockIdx.z;
  const int num_kb = (int)((a.K + kBlockK - 1) / kBlockK);
  volatile uint32_t* abort_flag = &sh->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kStages;
        const uint32_t use = kb / kStages;
        if (use > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (use - 1) & 1, abort_flag, a.err_word)) break;
        const uint32_t bar = smem_u32(&sh->full[s]);
        mbar_expect_tx(bar, C::kStageBytes);
        uint32_t dst = smem_u32(tiles + (size_t)s * C::kStageBytes);
        const int k0 = kb * kBlockK, r0 = m_tile * kBlockM, c0 = n_tile * kBlockN;
        if (MODE == kProbe || MODE == kRefOnly) {
          tma_load_3d(dst, &map_l, bar, k0, r0, b); dst += kBf16TileBytes;
          tma_load_3d(dst, &map_r, bar, k0, c0, b); dst += kBf16TileBytes;
        }
        if (MODE == kProbe) {
          tma_load_3d(dst, &map_la, bar, k0, r0, b); dst += kBf16TileBytes;
          tma_load_3d(dst, &map_ra, bar, k0, c0, b); dst += kBf16TileBytes;
        }
        if (MODE == kProbe || MODE == kLpOnly) {
          tma_load_3d(dst, &map_cl, bar, k0, r0, b); dst += kLpTileBytes;
          tma_load_3d(dst, &map_cr, bar, k0, c0, b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_bf16 = make_idesc(1, 1, 1, kBlockM, kBlockN);
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kStages;
        const uint32_t use = kb / kStages;
        if (!mbar_wait(smem_u32(&sh->full[s]), use & 1, abort_flag, a.err_word)) break;
        tc_fence_after();
        uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
        if (MODE == kProbe || MODE == kRefOnly) {
          const uint64_t dl = smem_desc(base, 128), dr = smem_desc(base + kBf16TileBytes, 128);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
            mma_ss<kKindF16>(tmem_base, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0);
          base += 2 * kBf16TileBytes;
        }
        if (MODE == kProbe) {
          const uint64_t dl = smem_desc(base, 128), dr = smem_desc(base + kBf16TileBytes, 128);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)
            mma_ss<kKindF16>(tmem_base + 128, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0);
          base += 2 * kBf16TileBytes;
        }
        if (MODE == kProbe || MODE == kLpOnly) {
          const uint32_t col = MODE == kProbe ? 256u : 0u;
          const uint64_t dl = smem_desc(base, 64), dr = smem_desc(base + kLpTileBytes, 64);
#pragma unroll
          for (int k = 0; k < kBlockK / 32; ++k)   // 32 bytes per step
            mma_ss<LPKIND>(tmem_base + col, dl + 2 * k, dr + 2 * k, a.idesc_lp, (kb | k) != 0);
        }
        tc_commit(smem_u32(&sh->empty[s]));       // frees the stage once these MMAs have read it
      }
      tc_commit(smem_u32(&sh->tmem_full));        // accumulators complete
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const int et = (warp - 2) * 32 + lane;        // 0..127
    {
      const int64_t col = (int64_t)n_tile * kBlockN + et;
      float d = 1.f;
      if (MODE != kRefOnly) d = a.pc_r ? (col < a.N ? __ldg(a.dr + (int64_t)b * a.N + col) : 0.f) : __ldg(a.dr);
      sh->delta_r[et] = d;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    const int64_t row = (int64_t)m_tile * kBlockM + q * 32 + lane;
    const bool row_ok = row < a.M;
    float dlv = 1.f;
    if (MODE != kRefOnly) dlv = a.pc_l ? (row_ok ? __ldg(a.dl + (int64_t)b * a.M + row) : 0.f) : __ldg(a.dl);

    const bool ok = mbar_wait(smem_u32(&sh->tmem_full), 0, abort_flag, a.err_word);
    tc_fence_after();
    double sbe = 0, mbe = 0, sd2 = 0, sr2 = 0, sn2 = 0;
    if (ok) {
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < kBlockN / 32; ++c) {
        const int64_t col0 = (int64_t)n_tile * kBlockN + c * 32;
        if (col0 >= a.N) break;                   // uniform across the warp
        if (MODE == kProbe) {
          uint32_t rc[32], rd[32], rq[32];
          tmem_ld32(lane_addr + c * 32, rc);
          tmem_ld32(lane_addr + 128 + c * 32, rd);
          tmem_ld32(lane_addr + 256 + c * 32, rq);
          tmem_ld_wait();
          float fbe = 0, fmx = 0, fd2 = 0, fr2 = 0, fn2 = 0;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float cc = __uint_as_float(rc[j]), dd = __uint_as_float(rd[j]);
            const float acc = LPKIND == kKindI8 ? (float)(int)rq[j] : __uint_as_float(rq[j]);
            const float qq = acc * (dlv * sh->delta_r[c * 32 + j]);
            const float diff = cc - qq;
            const bool live = col0 + j < a.N;
            float be = dd != 0.f ? __fdividef(fabsf(diff), dd) : 0.f;
            if (!live) be = 0.f;
            fbe += be; fmx = fmaxf(fmx, be);
            if (live) { fd2 = fmaf(diff, diff, fd2); fr2 = fmaf(cc, cc, fr2); fn2 = fmaf(dd, dd, fn2); }
          }
          if (row_ok) { sbe += fbe; mbe = fmax(mbe, (double)fmx); sd2 += fd2; sr2 += fr2; sn2 += fn2; }
        } else {
          uint32_t r[32];
          tmem_ld32(lane_addr + c * 32, r);
          tmem_ld_wait();
          if (row_ok) {
            const int64_t o = ((int64_t)b * a.M + row) * a.N + col0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (col0 + j < a.N) {
                if (MODE == kRefOnly) {
                  a.out_descaled[o + j] = __uint_as_float(r[j]);
                } else {
                  const float acc = LPKIND == kKindI8 ? (float)(int)r[j] : __uint_as_float(r[j]);
                  if (a.out_descaled) a.out_descaled[o + j] = acc * (dlv * sh->delta_r[c * 32 + j]);
                  if (a.out_raw) reinterpret_cast<uint32_t*>(a.out_raw)[o + j] = r[j];
                }
              }
            }
          }
        }
      }
    }
    if (MODE == kProbe) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sbe += __shfl_xor_sync(0xffffffffu, sbe, o);
        mbe = fmax(mbe, __shfl_xor_sync(0xffffffffu, mbe, o));
        sd2 += __shfl_xor_sync(0xffffffffu, sd2, o);
        sr2 += __shfl_xor_sync(0xffffffffu, sr2, o);
        sn2 += __shfl_xor_sync(0xffffffffu, sn2, o);
      }
      if (lane == 0) {
        sh->red[0][warp - 2] = sbe; sh->red[1][warp - 2] = mbe; sh->red[2][warp - 2] = sd2;
        sh->red[3][warp - 2] = sr2; sh->red[4][warp - 2] = sn2;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0) {
        double r[5] = {0, 0, 0, 0, 0};
        for (int i = 0; i < 4; ++i) {
          r[0] += sh->red[0][i]; r[1] = fmax(r[1], sh->red[1][i]); r[2] += sh->red[2][i];
          r[3] += sh->red[3][i]; r[4] += sh->red[4][i];
        }
        const int64_t blk = ((int64_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
        for (int i = 0; i < 5; ++i) a.partials[blk * kPartialDoubles + i] = r[i];
      }
    }
  }

  // ---------------------------------------------------------------- common exit
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols)
                 : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Tensor map over [batch][rows][K] with the contracting index contiguous; box = 64 x 128 x 1.
bool make_map(CUtensorMap* m, const void* base, bool bf16, int64_t K, int64_t rows, int64_t batch,
              int64_t ld_elems, int64_t sb_elems) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const uint64_t es = bf16 ? 2 : 1;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t sb = batch > 1 ? (cuuint64_t)sb_elems * es : (cuuint64_t)rows * ld_elems * es;
  cuuint64_t strides[2] = {(cuuint64_t)ld_elems * es, sb};
  cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)kBlockM, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  bf16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

uint32_t lp_idesc(int fmt_l, int fmt_r) {
  if (fmt_l == QM_FMT_INT8) return make_idesc(2, 1, 1, kBlockM, kBlockN);          // s8 x s8 -> s32
  const uint32_t fa = fmt_l == QM_FMT_E4M3 ? 0u : 1u, fb = fmt_r == QM_FMT_E4M3 ? 0u : 1u;
  return make_idesc(1, fa, fb, kBlockM, kBlockN);                                  // fp8 x fp8 -> f32
}

template <int MODE>
size_t smem_bytes() {
  return (size_t)Cfg<MODE>::kStages * Cfg<MODE>::kStageBytes + sizeof(Shared) + 1024;
}

template <int MODE, int LPKIND>
qm_status launch(const CUtensorMap* maps, const KernelArgs& ka, GemmShape g, cudaStream_t s) {
  auto kern = tc_kernel<MODE, LPKIND>;
  static bool attr_done = false;     // per instantiation
  if (!attr_done) {
    QM_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<MODE>()));
    attr_done = true;
  }
  dim3 grid((unsigned)((g.N + kBlockN - 1) / kBlockN), (unsigned)((g.M + kBlockM - 1) / kBlockM),
            (unsigned)g.batch);
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (MODE == kProbe) profile_events(&ev0, &ev1);
  if (ev0) QM_CUDA_OK(cudaEventRecord(ev0, s));
  kern<<<grid, kThreads, smem_bytes<MODE>(), s>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], ka);
  if (ev1) QM_CUDA_OK(cudaEventRecord(ev1, s));
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

bool shape_ok(GemmShape g) {
  return g.M > 0 && g.N > 0 && g.K > 0 && g.batch > 0 && (g.K % 16) == 0 && g.batch <= 65535 &&
         (g.M + kBlockM - 1) / kBlockM <= 65535 && g.M < (1ll << 31) && g.N < (1ll << 31) && g.K < (1ll << 31);
}

}  // namespace

int tc_probe_tiles(GemmShape g) {
  return (int)(((g.N + kBlockN - 1) / kBlockN) * ((g.M + kBlockM - 1) / kBlockM) * g.batch);
}

qm_status launch_tc_probe(const TcProbeArgs& p, cudaStream_t s) {
  if (!shape_ok(p.g)) return QM_ERR_UNSUPPORTED;
  const GemmShape g = p.g;
  const int64_t ldc = qm_code_ld(g.K);
  CUtensorMap maps[6];
  bool ok = make_map(&maps[0], p.l, true, g.K, g.M, g.batch, p.l_ld, p.l_sb) &&
            make_map(&maps[1], p.r, true, g.K, g.N, g.batch, p.r_ld, p.r_sb) &&
            make_map(&maps[2], p.l_abs, true, g.K, g.M, g.batch, g.K, g.M * g.K) &&
            make_map(&maps[3], p.r_abs, true, g.K, g.N, g.batch, g.K, g.N * g.K) &&
            make_map(&maps[4], p.cl, false, g.K, g.M, g.batch, ldc, g.M * ldc) &&
            make_map(&maps[5], p.cr, false, g.K, g.N, g.batch, ldc, g.N * ldc);
  if (!ok) return QM_ERR_CUDA;
  KernelArgs ka{};
  ka.M = g.M; ka.N = g.N; ka.K = g.K;
  ka.dl = p.dl; ka.pc_l = p.gran_l == QM_GRAN_CHANNEL; ka.dr = p.dr; ka.pc_r = p.gran_r == QM_GRAN_CHANNEL;
  ka.partials = p.partials; ka.err_word = p.err_word; ka.idesc_lp = lp_idesc(p.fmt_l, p.fmt_r);
  return p.fmt_l == QM_FMT_INT8 ? launch<kProbe, kKindI8>(maps, ka, g, s)
                                : launch<kProbe, kKindF8>(maps, ka, g, s);
}

qm_status launch_tc_gemm_lp(const uint8_t* cl, int fmt_l, const float* dl, int gran_l,
                            const uint8_t* cr, int fmt_r, const float* dr, int gran_r, GemmShape g,
                            float* out_descaled, void* out_raw, uint32_t* err_word, cudaStream_t s) {
  if (!shape_ok(g)) return QM_ERR_UNSUPPORTED;
  const int64_t ldc = qm_code_ld(g.K);
  CUtensorMap maps[6];
  bool ok = make_map(&maps[4], cl, false, g.K, g.M, g.batch, ldc, g.M * ldc) &&
            make_map(&maps[5], cr, false, g.K, g.N, g.batch, ldc, g.N * ldc);
  if (!ok) return QM_ERR_CUDA;
  maps[0] = maps[1] = maps[2] = maps[3] = maps[4];
  KernelArgs ka{};
  ka.M = g.M; ka.N = g.N; ka.K = g.K;
  ka.dl = dl; ka.pc_l = gran_l == QM_GRAN_CHANNEL; ka.dr = dr; ka.pc_r = gran_r == QM_GRAN_CHANNEL;
  ka.out_descaled = out_descaled; ka.out_raw = out_raw; ka.err_word = err_word;
  ka.idesc_lp = lp_idesc(fmt_l, fmt_r);
  return fmt_l == QM_FMT_INT8 ? launch<kLpOnly, kKindI8>(maps, ka, g, s)
                              : launch<kLpOnly, kKindF8>(maps, ka, g, s);
}

qm_status launch_tc_gemm_ref(const void* l, const void* r, GemmShape g, float* out, uint32_t* err_word,
                             cudaStream_t s) {
  if (!shape_ok(g)) return QM_ERR_UNSUPPORTED;
  CUtensorMap maps[6];
  bool ok = make_map(&maps[0], l, true, g.K, g.M, g.batch, g.K, g.M * g.K) &&
            make_map(&maps[1], r, true, g.K, g.N, g.batch, g.K, g.N * g.K);
  if (!ok) return QM_ERR_CUDA;
  maps[2] = maps[3] = maps[4] = maps[5] = maps[0];
  KernelArgs ka{};
  ka.M = g.M; ka.N = g.N; ka.K = g.K; ka.out_descaled = out; ka.err_word = err_word;
  return launch<kRefOnly, kKindF8>(maps, ka, g, s);
}

}  // namespace qm
