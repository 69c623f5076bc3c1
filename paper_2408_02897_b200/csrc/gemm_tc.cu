// Tensor-core products of the probe for sm_100a: tcgen05.mma with accumulators in tensor
// memory, operands staged in shared memory by TMA, warp-specialised persistent CTAs.
//
// Each CTA walks a static list of 128 x 128 output tiles (tile = blockIdx.x + i * gridDim.x).
//   warp 0      TMA producer: per 32-wide k-block, bulk-tensor loads of every operand tile into
//               a ring of stages; it runs ahead across tile boundaries, so the next tile's first
//               stages arrive while the current tile is still in its epilogue
//   warp 1      allocates tensor memory once; one lane issues the MMAs of each k-block
//   warps 2..9  epilogue: read the accumulators with tcgen05.ld (a warp may touch the lane
//               quarter warp_id % 4; the two warps of a quarter split the columns) and either
//               reduce the Eq. 3 statistics (probe) or store the product.
// In probe mode three accumulators live side by side in tensor memory: the reference L.R
// (bf16 operands, kind::f16, columns 0..127), the denominator |L|.|R| (bf16, kind::f16, columns
// 128..255) and the 8-bit product (kind::f8f6f4 or kind::i8, columns 256..383), so no M x N
// matrix ever goes to HBM.  The CTA keeps its Eq. 3 statistics in registers across tiles and
// writes one record; the last CTA to finish adds the records up in a fixed order.
//
// Every wait is bounded: when one gives up it raises QM_DEVERR_TIMEOUT in the caller's error
// word and flags the CTA, after which every role falls through to the common exit, tensor
// memory is freed and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kBlockM = 128, kBlockN = 128, kBlockK = 32;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;                // 320
constexpr uint32_t kBf16TileBytes = kBlockM * kBlockK * 2;   // 8 KB, 64-byte rows
constexpr uint32_t kLpTileBytes = kBlockM * kBlockK;         // 4 KB, 32-byte rows
constexpr int kMaxStages = 10;

enum Mode { kProbe = 0, kLpOnly = 1, kRefOnly = 2 };

template <int MODE> struct Cfg;
template <> struct Cfg<kProbe> {
  static constexpr int kStages = 5;
  static constexpr uint32_t kStageBytes = 4 * kBf16TileBytes + 2 * kLpTileBytes;   // 40 KB
  static constexpr uint32_t kTmemCols = 512;
};
template <> struct Cfg<kLpOnly> {
  static constexpr int kStages = 10;
  static constexpr uint32_t kStageBytes = 2 * kLpTileBytes;                        // 8 KB
  static constexpr uint32_t kTmemCols = 128;
};
template <> struct Cfg<kRefOnly> {
  static constexpr int kStages = 10;
  static constexpr uint32_t kStageBytes = 2 * kBf16TileBytes;                      // 16 KB
  static constexpr uint32_t kTmemCols = 128;
};

struct KernelArgs {
  int64_t M, N, K;
  int32_t tiles_m, tiles_n, num_tiles;
  const float* dl; int pc_l;      // per-channel flags: delta indexed by batch*M + row
  const float* dr; int pc_r;
  float* out_descaled;            // LpOnly / RefOnly
  void* out_raw;                  // LpOnly
  double* partials;               // Probe: gridDim.x records
  uint32_t* done_counter;         // Probe: zero on entry
  qm_metric_result* result;       // Probe
  uint64_t count;                 // Probe: batch * M * N
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

// Shared-memory matrix descriptor, contraction-major tile whose rows are exactly one swizzle
// span wide (64 bytes for the bf16 tiles, 32 bytes for the code tiles): eight consecutive rows
// form one swizzle atom, atoms follow each other every 8 * span bytes ("stride byte offset").
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t span_bytes) {
  const uint64_t layout = span_bytes == 128 ? 2ull : (span_bytes == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);                      // start address / 16
  d |= (uint64_t)1 << 16;                                       // leading byte offset (unused here)
  d |= (uint64_t)((8u * span_bytes) >> 4) << 32;                // stride byte offset / 16
  d |= (uint64_t)1 << 46;                                       // descriptor version of sm_100
  d |= layout << 61;                                            // swizzle mode
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
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full;
  uint64_t tmem_empty;
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t is_last;
  uint32_t pad;
  float delta_r[2][kBlockN];
  double red[5][kEpiWarps];
};

// Named barrier 1 over the 256 epilogue threads, returning the OR of `flag` over all of them.
__device__ __forceinline__ bool epi_barrier_any(bool flag) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"((uint32_t)flag)
      : "memory");
  return out != 0;
}

struct TileCoord { int m_tile, n_tile, b; };
__device__ __forceinline__ TileCoord tile_coord(int t, const KernelArgs& a) {
  TileCoord c;
  const int per_b = a.tiles_m * a.tiles_n;
  c.b = t / per_b;
  const int r = t - c.b * per_b;
  c.m_tile = r / a.tiles_n;
  c.n_tile = r - c.m_tile * a.tiles_n;
  return c;
}

template <int MODE, int LPKIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_kernel(const __grid_constant__ CUtensorMap map_l, const __grid_constant__ CUtensorMap map_r,
          const __grid_constant__ CUtensorMap map_la, const __grid_constant__ CUtensorMap map_ra,
          const __grid_constant__ CUtensorMap map_cl, const __grid_constant__ CUtensorMap map_cr,
          const KernelArgs a) {
  using C = Cfg<MODE>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  // tiles start on a 1024-byte boundary (a multiple of every swizzle atom size)
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + (size_t)kStages * C::kStageBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (int)((a.K + kBlockK - 1) / kBlockK);
  volatile uint32_t* abort_flag = &sh->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), kEpiWarps);
    sh->abort_flag = 0;
    sh->is_last = 0;
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
      uint32_t g = 0;                                           // running k-block count
      bool ok = true;
      for (int t = blockIdx.x; t < a.num_tiles && ok; t += gridDim.x) {
        const TileCoord tc = tile_coord(t, a);
        const int r0 = tc.m_tile * kBlockM, c0 = tc.n_tile * kBlockN;
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t use = g / kStages;
          if (use > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (use - 1) & 1, abort_flag, a.err_word)) {
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&sh->full[s]);
          mbar_expect_tx(bar, C::kStageBytes);
          uint32_t dst = smem_u32(tiles + (size_t)s * C::kStageBytes);
          const int k0 = kb * kBlockK;
          if (MODE == kProbe || MODE == kRefOnly) {
            tma_load_3d(dst, &map_l, bar, k0, r0, tc.b); dst += kBf16TileBytes;
            tma_load_3d(dst, &map_r, bar, k0, c0, tc.b); dst += kBf16TileBytes;
          }
          if (MODE == kProbe) {
            tma_load_3d(dst, &map_la, bar, k0, r0, tc.b); dst += kBf16TileBytes;
            tma_load_3d(dst, &map_ra, bar, k0, c0, tc.b); dst += kBf16TileBytes;
          }
          if (MODE == kProbe || MODE == kLpOnly) {
            tma_load_3d(dst, &map_cl, bar, k0, r0, tc.b); dst += kLpTileBytes;
            tma_load_3d(dst, &map_cr, bar, k0, c0, tc.b);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_bf16 = make_idesc(1, 1, 1, kBlockM, kBlockN);
      uint32_t g = 0, it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < a.num_tiles && ok; t += gridDim.x, ++it) {
        // the epilogue must have drained the previous tile's accumulators
        if (it > 0 && !mbar_wait(smem_u32(&sh->tmem_empty), (it - 1) & 1, abort_flag, a.err_word)) break;
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t use = g / kStages;
          if (!mbar_wait(smem_u32(&sh->full[s]), use & 1, abort_flag, a.err_word)) { ok = false; break; }
          tc_fence_after();
          uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
          if (MODE == kProbe || MODE == kRefOnly) {
            const uint64_t dl = smem_desc(base, 64), dr = smem_desc(base + kBf16TileBytes, 64);
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
              mma_ss<kKindF16>(tmem_base, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0);
            base += 2 * kBf16TileBytes;
          }
          if (MODE == kProbe) {
            const uint64_t dl = smem_desc(base, 64), dr = smem_desc(base + kBf16TileBytes, 64);
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
              mma_ss<kKindF16>(tmem_base + 128, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0);
            base += 2 * kBf16TileBytes;
          }
          if (MODE == kProbe || MODE == kLpOnly) {
            const uint32_t col = MODE == kProbe ? 256u : 0u;
            // one 32-byte step covers the whole k-block
            mma_ss<LPKIND>(tmem_base + col, smem_desc(base, 32), smem_desc(base + kLpTileBytes, 32),
                           a.idesc_lp, kb != 0);
          }
          tc_commit(smem_u32(&sh->empty[s]));       // frees the stage once these MMAs have read it
        }
        if (ok) tc_commit(smem_u32(&sh->tmem_full));  // accumulators of this tile complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const int h = (warp - 2) >> 2;                // which 64-column half of the tile
    const int et = (warp - 2) * 32 + lane;        // 0..255
    const float dl_tensor = (MODE != kRefOnly && !a.pc_l) ? __ldg(a.dl) : 1.f;
    const float dr_tensor = (MODE != kRefOnly && !a.pc_r) ? __ldg(a.dr) : 1.f;
    double sbe = 0, mbe = 0, sd2 = 0, sr2 = 0, sn2 = 0;
    uint32_t it = 0;
    for (int t = blockIdx.x; t < a.num_tiles; t += gridDim.x, ++it) {
      const TileCoord tc = tile_coord(t, a);
      float* dr_s = sh->delta_r[it & 1];
      if (et < kBlockN) {
        const int64_t col = (int64_t)tc.n_tile * kBlockN + et;
        float d = dr_tensor;
        if (MODE != kRefOnly && a.pc_r) d = col < a.N ? __ldg(a.dr + (int64_t)tc.b * a.N + col) : 0.f;
        dr_s[et] = d;
      }
      const int64_t row = (int64_t)tc.m_tile * kBlockM + q * 32 + lane;
      const bool row_ok = row < a.M;
      float dlv = dl_tensor;
      if (MODE != kRefOnly && a.pc_l) dlv = row_ok ? __ldg(a.dl + (int64_t)tc.b * a.M + row) : 0.f;

      const bool ok = mbar_wait(smem_u32(&sh->tmem_full), it & 1, abort_flag, a.err_word);
      // one barrier publishes delta_r and makes the give-up decision uniform over the epilogue
      if (epi_barrier_any(!ok)) break;
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        const int cc0 = h * 64 + c * 32;          // first column of this chunk inside the tile
        const int64_t col0 = (int64_t)tc.n_tile * kBlockN + cc0;
        if (col0 >= a.N) break;                   // uniform across the warp
        if (MODE == kProbe) {
          uint32_t rc[32], rd[32], rq[32];
          tmem_ld32(lane_addr + cc0, rc);
          tmem_ld32(lane_addr + 128 + cc0, rd);
          tmem_ld32(lane_addr + 256 + cc0, rq);
          tmem_ld_wait();
          float fbe = 0, fmx = 0, fd2 = 0, fr2 = 0, fn2 = 0;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float cv = __uint_as_float(rc[j]), dd = __uint_as_float(rd[j]);
            const float acc = LPKIND == kKindI8 ? (float)(int)rq[j] : __uint_as_float(rq[j]);
            const float diff = fmaf(-(acc * dlv), dr_s[cc0 + j], cv);      // C - A * dl * dr
            const bool live = col0 + j < a.N;
            float be = dd != 0.f ? __fdividef(fabsf(diff), dd) : 0.f;
            if (!live) be = 0.f;
            fbe += be; fmx = fmaxf(fmx, be);
            if (live) { fd2 = fmaf(diff, diff, fd2); fr2 = fmaf(cv, cv, fr2); fn2 = fmaf(dd, dd, fn2); }
          }
          if (row_ok) { sbe += fbe; mbe = fmax(mbe, (double)fmx); sd2 += fd2; sr2 += fr2; sn2 += fn2; }
        } else {
          uint32_t r[32];
          tmem_ld32(lane_addr + cc0, r);
          tmem_ld_wait();
          if (row_ok) {
            const int64_t o = ((int64_t)tc.b * a.M + row) * a.N + col0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (col0 + j < a.N) {
                if (MODE == kRefOnly) {
                  a.out_descaled[o + j] = __uint_as_float(r[j]);
                } else {
                  const float acc = LPKIND == kKindI8 ? (float)(int)r[j] : __uint_as_float(r[j]);
                  if (a.out_descaled) a.out_descaled[o + j] = acc * (dlv * dr_s[cc0 + j]);
                  if (a.out_raw) reinterpret_cast<uint32_t*>(a.out_raw)[o + j] = r[j];
                }
              }
            }
          }
        }
      }
      // this warp has finished reading the accumulators of the tile
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty));
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
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (et == 0) {
        double r[5] = {0, 0, 0, 0, 0};
        for (int i = 0; i < kEpiWarps; ++i) {
          r[0] += sh->red[0][i]; r[1] = fmax(r[1], sh->red[1][i]); r[2] += sh->red[2][i];
          r[3] += sh->red[3][i]; r[4] += sh->red[4][i];
        }
        double* rec = a.partials + (int64_t)blockIdx.x * kPartialDoubles;
        for (int i = 0; i < 5; ++i) __stcg(rec + i, r[i]);
        __threadfence();
        const uint32_t prev = atomicAdd(a.done_counter, 1u);
        sh->is_last = prev == gridDim.x - 1 ? 1u : 0u;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (sh->is_last && warp == 2) {
        // last CTA: every record is visible; fixed-order sum (lane l takes records l, l+32, ...)
        __threadfence();
        double r[5] = {0, 0, 0, 0, 0};
        for (int i = lane; i < (int)gridDim.x; i += 32) {
          const double* rec = a.partials + (int64_t)i * kPartialDoubles;
          r[0] += __ldcg(rec); r[1] = fmax(r[1], __ldcg(rec + 1)); r[2] += __ldcg(rec + 2);
          r[3] += __ldcg(rec + 3); r[4] += __ldcg(rec + 4);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          r[0] += __shfl_xor_sync(0xffffffffu, r[0], o);
          r[1] = fmax(r[1], __shfl_xor_sync(0xffffffffu, r[1], o));
          r[2] += __shfl_xor_sync(0xffffffffu, r[2], o);
          r[3] += __shfl_xor_sync(0xffffffffu, r[3], o);
          r[4] += __shfl_xor_sync(0xffffffffu, r[4], o);
        }
        if (lane == 0) {
          a.result->sum_be = r[0]; a.result->max_be = r[1]; a.result->sum_diff2 = r[2];
          a.result->sum_ref2 = r[3]; a.result->sum_den2 = r[4];
          a.result->count = a.count;
          a.result->device_error = a.err_word ? *reinterpret_cast<volatile uint32_t*>(a.err_word) : 0u;
          a.result->reserved = 0;
        }
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

// Tensor map over [batch][rows][K] with the contracting index contiguous; box = 32 x 128 x 1,
// swizzle span = row width of the box (64 bytes for bf16, 32 bytes for codes).
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
                  bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B,
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

bool shape_ok(GemmShape g) {
  if (!(g.M > 0 && g.N > 0 && g.K > 0 && g.batch > 0 && (g.K % 16) == 0)) return false;
  if (g.M >= (1ll << 31) || g.N >= (1ll << 31) || g.K >= (1ll << 31) || g.batch >= (1ll << 31)) return false;
  const int64_t tiles = ((g.M + kBlockM - 1) / kBlockM) * ((g.N + kBlockN - 1) / kBlockN) * g.batch;
  return tiles < (1ll << 31);
}

void fill_tiles(KernelArgs* ka, GemmShape g) {
  ka->M = g.M; ka->N = g.N; ka->K = g.K;
  ka->tiles_m = (int32_t)((g.M + kBlockM - 1) / kBlockM);
  ka->tiles_n = (int32_t)((g.N + kBlockN - 1) / kBlockN);
  ka->num_tiles = (int32_t)((int64_t)ka->tiles_m * ka->tiles_n * g.batch);
}

int grid_size(GemmShape g) {
  const int64_t tiles = ((g.M + kBlockM - 1) / kBlockM) * ((g.N + kBlockN - 1) / kBlockN) * g.batch;
  const int sms = sm_count();
  return (int)(tiles < sms ? tiles : sms);
}

template <int MODE, int LPKIND>
qm_status launch(const CUtensorMap* maps, const KernelArgs& ka, GemmShape g, cudaStream_t s) {
  auto kern = tc_kernel<MODE, LPKIND>;
  static bool attr_done = false;     // per instantiation
  if (!attr_done) {
    QM_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<MODE>()));
    attr_done = true;
  }
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (MODE == kProbe) profile_events(&ev0, &ev1);
  if (ev0) QM_CUDA_OK(cudaEventRecord(ev0, s));
  kern<<<grid_size(g), kThreads, smem_bytes<MODE>(), s>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], ka);
  if (ev1) QM_CUDA_OK(cudaEventRecord(ev1, s));
  count_launch();
  QM_CUDA_OK(cudaGetLastError());
  return QM_OK;
}

}  // namespace

int tc_probe_records(GemmShape g) { return grid_size(g); }

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
  fill_tiles(&ka, g);
  ka.dl = p.dl; ka.pc_l = p.gran_l == QM_GRAN_CHANNEL; ka.dr = p.dr; ka.pc_r = p.gran_r == QM_GRAN_CHANNEL;
  ka.partials = p.partials; ka.done_counter = p.done_counter; ka.result = p.result;
  ka.count = (uint64_t)(g.M * g.N * g.batch);
  ka.err_word = p.err_word; ka.idesc_lp = lp_idesc(p.fmt_l, p.fmt_r);
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
  fill_tiles(&ka, g);
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
  fill_tiles(&ka, g);
  ka.out_descaled = out; ka.err_word = err_word;
  return launch<kRefOnly, kKindF8>(maps, ka, g, s);
}

}  // namespace qm
