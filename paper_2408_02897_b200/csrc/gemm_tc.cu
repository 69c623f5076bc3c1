// Tensor-core products of the probe for sm_100a: tcgen05.mma with accumulators in tensor
// memory, operands staged in shared memory by TMA, warp-specialised persistent CTA pairs.
//
// Two CTAs on the two SMs of a TPC form a cluster and work on one output tile with cta_group::2
// MMAs: each CTA stages its own 128 rows of the left operand and HALF of the right operand's
// tile, so every byte of the right operand enters and leaves shared memory once per pair instead
// of once per SM.  Three kernels, in this order in the file:
//   tc_kernel            256 x 128 tiles, 320 threads (TMA warp, MMA warp, 8 epilogue warps): the
//                        stand-alone 8-bit and reference products on narrow outputs, and the
//                        two-formats-in-one-pass probe (four accumulators fill tensor memory);
//   tc_gemm_wide_kernel  256 x 256 tiles, two accumulator buffers: stand-alone products on outputs at
//                        least 256 wide;
//   tc_group_kernel      the fused probe (Eq. 3 record of one probe, or of up to 16 probes, per
//                        persistent launch): reference L.R, denominator |L|.|R| and 8-bit product side
//                        by side in tensor memory, |L| fed to the MMAs from tensor memory by converter
//                        warps, the Eq. 3 statistics reduced in the epilogue; no M x N matrix ever
//                        goes to HBM.  Its own comment describes roles and barriers.
// Common to all: the MMA warp runs its loop converged and one elected lane issues; the epilogue
// warps read the accumulators with tcgen05.ld (a warp may touch the lane quarter warp_id % 4; the
// two warps of a quarter split the columns); a CTA keeps Eq. 3 statistics in registers across tiles
// and writes one record, and the last CTA to finish adds the records up in a fixed order.
//
// Every mbarrier wait is bounded: when one gives up it raises QM_DEVERR_TIMEOUT in the caller's
// error word and flags the CTA, after which every role falls through to the common exit, tensor
// memory is freed and the kernel returns.  No load uses cluster multicast.
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>
#include <cstdlib>
#include <mutex>

#include "qm_internal.h"

namespace qm {
namespace {

constexpr int kBlockM = 128;             // rows per CTA
constexpr int kPairM = 256;              // rows per CTA pair
constexpr int kBlockN = 128;             // columns per tile
constexpr int kHalfN = 64;               // right-operand rows staged by each CTA
constexpr int kBlockK = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;                     // 320
constexpr uint32_t kABf16 = kBlockM * kBlockK * 2;                // 16 KB, 128-byte rows
constexpr uint32_t kALp = kBlockM * kBlockK;                      //  8 KB,  64-byte rows
constexpr uint32_t kBBf16 = kHalfN * kBlockK * 2;                 //  8 KB
constexpr uint32_t kBLp = kHalfN * kBlockK;                       //  4 KB
constexpr int kMaxStages = 8;

enum Mode { kLpOnly = 1, kRefOnly = 2, kProbe2 = 3 };

// Stage layout: left-operand tiles first (L, |L|, codes), then the right-operand halves.
template <int MODE> struct Cfg;
// Two 8-bit formats in one pass: the reference and denominator products are shared, each format
// has its own code tiles and its own accumulator.
template <> struct Cfg<kProbe2> {
  static constexpr int kStages = 3;
  static constexpr uint32_t kOffL = 0, kOffLa = kABf16, kOffCl = 2 * kABf16, kOffCl2 = kOffCl + kALp;
  static constexpr uint32_t kOffR = kOffCl2 + kALp, kOffRa = kOffR + kBBf16, kOffCr = kOffRa + kBBf16;
  static constexpr uint32_t kOffCr2 = kOffCr + kBLp;
  static constexpr uint32_t kStageBytes = kOffCr2 + kBLp;         // 72 KB
  static constexpr uint32_t kTmemCols = 512;
};
template <> struct Cfg<kLpOnly> {
  static constexpr int kStages = 8;
  static constexpr uint32_t kOffL = 0, kOffLa = 0, kOffCl = 0, kOffR = 0, kOffRa = 0, kOffCr = kALp;
  static constexpr uint32_t kStageBytes = kALp + kBLp;            // 12 KB
  static constexpr uint32_t kTmemCols = 128;
};
template <> struct Cfg<kRefOnly> {
  static constexpr int kStages = 6;
  static constexpr uint32_t kOffL = 0, kOffLa = 0, kOffCl = 0, kOffR = kABf16, kOffRa = 0, kOffCr = 0;
  static constexpr uint32_t kStageBytes = kABf16 + kBBf16;        // 24 KB
  static constexpr uint32_t kTmemCols = 128;
};

struct KernelArgs {
  int64_t M, N, K;
  int32_t tiles_m, tiles_n, num_tiles;   // tiles of 256 x 128
  const float* dl; int pc_l;             // per-channel flags: delta indexed by batch*M + row
  const float* dr; int pc_r;
  float* out_descaled;                   // LpOnly / RefOnly
  void* out_raw;                         // LpOnly
  double* partials;                      // Probe: gridDim.x records
  uint32_t* done_counter;                // Probe: zero on entry
  qm_metric_result* result;              // Probe
  uint64_t count;                        // Probe: batch * M * N
  uint32_t* err_word;
  uint32_t idesc_lp;                     // instruction descriptor of the 8-bit MMA
  // Probe2: scales and descriptor of the second format (granularities are shared); its record
  // is result[1] and its per-CTA records follow the first format's gridDim.x records
  const float* dl2; const float* dr2;
  uint32_t idesc_lp2;
  double* row_stats;                     // Probe (one format): optional [batch * M][5] per-row sums
  const uint32_t* err_also[2];           // Probe (one format): further error words to report in the record, or null
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank`
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
// arrive on a barrier given by its shared::cluster address (own CTA or the peer)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  // default semantics (release at CTA scope): the data this barrier orders lives in tensor
  // memory and is fenced by tcgen05.fence; a cluster-scope release costs a long memory fence
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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

// The same for a converged warp: every lane waits, and all lanes take the same decision.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                               uint32_t* err_word) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, err_word));
}

// Tile load into this CTA's shared memory; the byte count is credited to the barrier at
// `bar_cluster_addr`, which may live in the peer CTA (cta_group::2 form).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One lane of a fully converged warp.  The MMA warp runs its whole loop (waits, descriptor
// arithmetic, loop control) convergently and narrows to one lane only around each tcgen05
// instruction: issued from a loop that a single lane runs alone, every MMA cost about 100 cycles
// of issue time, which was the limit of the main loop; issued this way it costs about 60.
__device__ __forceinline__ bool elect_one() {
  uint32_t p;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(p));
  return p != 0;
}

// Arrive on the barrier at this shared-memory offset in BOTH CTAs of the pair once all MMAs
// issued so far have completed.  Called by a converged warp; one lane issues.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, bool lead) {
  if (!lead) return;
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"(mask) : "memory");
}

// Shared-memory matrix descriptor, contraction-major tile whose rows are exactly one swizzle
// span wide (128 bytes for the bf16 tiles, 64 bytes for the code tiles): eight consecutive rows
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

// D[256 x N] (+)= A[256 x k] . B[N x k]^T across the CTA pair; called by a converged warp of the
// leader, one lane issues.
template <int KIND>
__device__ __forceinline__ void mma_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc,
                                         uint32_t accumulate, bool lead) {
  if (!lead) return;
  if (KIND == kKindF16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  } else if (KIND == kKindF8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
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
  uint64_t full[kMaxStages];     // used in the leader CTA: both CTAs' loads of a stage have landed
  uint64_t empty[kMaxStages];    // per CTA: the pair's MMAs have finished reading the stage
  uint64_t tmem_full;            // per CTA: the tile's accumulators are complete
  uint64_t tmem_empty;           // leader: both CTAs' epilogues have drained the accumulators
  uint64_t lp_done;              // leader (probe): both CTAs' epilogues have finished a tile
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t is_last;
  uint32_t pad;
  float delta_r[2][kBlockN];
  float delta_r2[2][kBlockN];    // Probe2: column scales of the second format
  double red[10][kEpiWarps];
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

// 32 lanes x 16 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// Two-wide fp32 arithmetic (one instruction for a pair of values).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t x, uint64_t y, uint64_t z) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(x), "l"(y), "l"(z));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t x, uint64_t y) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(x), "l"(y));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t x, uint64_t y) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(x), "l"(y));
  return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float max3(float x, float y, float z) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(x), "f"(y), "f"(z));
  return r;
}

// Eq. 3 statistics of one row, kept two-wide across the columns of a tile.
struct Stats2 {
  uint64_t be, d2, r2, n2;
  float mx;
};

// 16 consecutive columns of one row: reference rc, denominator rd, raw 8-bit accumulator rq.
// ndl2 holds (-delta_l, -delta_l); dr_s points at the 16 column scales (per_col) or is unused.
// n_live < 16 only in the last, ragged column chunk of a matrix.
template <int LPKIND, bool RAGGED>
__device__ __forceinline__ void stats16(const uint32_t* rc, const uint32_t* rd, const uint32_t* rq,
                                        uint64_t ndl2, const float* dr_s, bool per_col, uint64_t dr_tensor2,
                                        int n_live, Stats2& s) {
#pragma unroll
  for (int j = 0; j < 16; j += 2) {
    const bool live0 = !RAGGED || j < n_live, live1 = !RAGGED || j + 1 < n_live;
    const float a0 = LPKIND == kKindI8 ? (float)(int)rq[j] : __uint_as_float(rq[j]);
    const float a1 = LPKIND == kKindI8 ? (float)(int)rq[j + 1] : __uint_as_float(rq[j + 1]);
    const uint64_t dr2 = per_col ? *reinterpret_cast<const uint64_t*>(dr_s + j) : dr_tensor2;
    float c0 = __uint_as_float(rc[j]), c1 = __uint_as_float(rc[j + 1]);
    float d0 = __uint_as_float(rd[j]), d1 = __uint_as_float(rd[j + 1]);
    if (!live0) { c0 = 0.f; d0 = 0.f; }
    if (!live1) { c1 = 0.f; d1 = 0.f; }
    const uint64_t cv2 = pack2(c0, c1), dd2 = pack2(d0, d1);
    uint64_t diff2 = fma2(mul2(pack2(live0 ? a0 : 0.f, live1 ? a1 : 0.f), ndl2), dr2, cv2);   // C - A dl dr
    float e0, e1;
    unpack2(diff2, e0, e1);
    // D == 0 implies C == Q == 0, so clamping the divisor keeps BE = 0 there without a branch
    const float r0 = rcp_approx(fmaxf(d0, 1e-37f)), r1 = rcp_approx(fmaxf(d1, 1e-37f));
    const uint64_t be2 = mul2(pack2(fabsf(e0), fabsf(e1)), pack2(r0, r1));
    float b0, b1;
    unpack2(be2, b0, b1);
    s.be = add2(s.be, be2);
    s.mx = max3(s.mx, b0, b1);
    s.d2 = fma2(diff2, diff2, s.d2);
    s.r2 = fma2(cv2, cv2, s.r2);
    s.n2 = fma2(dd2, dd2, s.n2);
  }
}

// The same statistics for the grouped kernel, which first brings a chunk into one form (the
// 8-bit accumulator as fp32, dead columns zeroed) so that one instantiation per scale layout
// serves every format and the ragged edge.  PER_COL: the right operand has a scale per column
// (dr_s), otherwise kd2 holds (-delta_l delta_r) twice.
struct StatsG {
  float be0, be1;
  uint64_t d2, r2, n2;
  float mx;
};
template <bool PER_COL>
__device__ __forceinline__ void stats16g(const uint32_t* rc, const uint32_t* rd, const uint32_t* rq, uint64_t kd2,
                                         const float* dr_s, StatsG& s) {
#pragma unroll
  for (int j = 0; j < 16; j += 2) {
    const uint64_t a2 = pack2(__uint_as_float(rq[j]), __uint_as_float(rq[j + 1]));
    const uint64_t cv2 = pack2(__uint_as_float(rc[j]), __uint_as_float(rc[j + 1]));
    const float d0 = __uint_as_float(rd[j]), d1 = __uint_as_float(rd[j + 1]);
    const uint64_t dd2 = pack2(d0, d1);
    uint64_t diff2;                                              // C - A dl dr
    if (PER_COL) diff2 = fma2(mul2(a2, kd2), *reinterpret_cast<const uint64_t*>(dr_s + j), cv2);
    else diff2 = fma2(a2, kd2, cv2);
    // D == 0 implies C == Q == 0, so clamping the divisor keeps BE = 0 there without a branch
    const uint64_t be2 = mul2(diff2, pack2(rcp_approx(fmaxf(d0, 1e-37f)), rcp_approx(fmaxf(d1, 1e-37f))));
    float b0, b1;
    unpack2(be2, b0, b1);
    s.be0 += fabsf(b0);
    s.be1 += fabsf(b1);
    s.mx = fmaxf(s.mx, fmaxf(fabsf(b0), fabsf(b1)));
    s.d2 = fma2(diff2, diff2, s.d2);
    s.r2 = fma2(cv2, cv2, s.r2);
    s.n2 = fma2(dd2, dd2, s.n2);
  }
}
// Chunk CH (16 columns) of a warp's share of a tile: rq holds its 8-bit accumulators as read from
// tensor memory; n_live < 16 only at the ragged edge of the matrix, whose dead columns count as zeros.
template <int CH>
__device__ __forceinline__ void stats_chunk(uint32_t (&rc)[64], uint32_t (&rd)[64], uint32_t (&rq)[16], int n_live,
                                            bool is_i8, bool per_col, uint64_t kd2, const float* dr_s, StatsG& st) {
  if (is_i8) {
#pragma unroll
    for (int k = 0; k < 16; ++k) rq[k] = __float_as_uint((float)(int)rq[k]);
  }
  if (n_live < 16) {
#pragma unroll
    for (int k = 0; k < 16; ++k)
      if (k >= n_live) { rc[CH * 16 + k] = 0u; rd[CH * 16 + k] = 0u; rq[k] = 0u; }
  }
  if (per_col) stats16g<true>(&rc[CH * 16], &rd[CH * 16], rq, kd2, dr_s + CH * 16, st);
  else stats16g<false>(&rc[CH * 16], &rd[CH * 16], rq, kd2, nullptr, st);
}
// Adds one tile's share of a row's Eq. 3 sums to the optional per-row check output.
__device__ __forceinline__ void row_stats_add(double* rs, const StatsG& st) {
  float x0, x1;
  atomicAdd(rs + 0, (double)st.be0 + (double)st.be1);
  atomicMax(reinterpret_cast<unsigned long long*>(rs + 1), (unsigned long long)__double_as_longlong((double)st.mx));
  unpack2(st.d2, x0, x1); atomicAdd(rs + 2, (double)x0 + (double)x1);
  unpack2(st.r2, x0, x1); atomicAdd(rs + 3, (double)x0 + (double)x1);
  unpack2(st.n2, x0, x1); atomicAdd(rs + 4, (double)x0 + (double)x1);
}

template <int MODE, int LPKIND, int LPKIND2>
__global__ void __launch_bounds__(kThreads, 1)
tc_kernel(const __grid_constant__ CUtensorMap map_l, const __grid_constant__ CUtensorMap map_r,
          const __grid_constant__ CUtensorMap map_la, const __grid_constant__ CUtensorMap map_ra,
          const __grid_constant__ CUtensorMap map_cl, const __grid_constant__ CUtensorMap map_cr,
          const __grid_constant__ CUtensorMap map_cl2, const __grid_constant__ CUtensorMap map_cr2,
          const KernelArgs a) {
  constexpr bool kAnyProbe = MODE == kProbe2;
  constexpr int kFormats = MODE == kProbe2 ? 2 : 1;
  using C = Cfg<MODE>;
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  // tiles start on a 1024-byte boundary (the 128-byte swizzle atom); the offset is the same in
  // both CTAs of the pair because their dynamic shared memory starts at the same address
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + (size_t)kStages * C::kStageBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();                   // 0 = leader
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_kb = (int)((a.K + kBlockK - 1) / kBlockK);
  volatile uint32_t* abort_flag = &sh->abort_flag;

  if (warp == 0 && lane < 8) {
    // fetch the tensor maps into the descriptor cache while the CTA sets itself up
    const CUtensorMap* maps[8] = {&map_l, &map_r, &map_la, &map_ra, &map_cl, &map_cr, &map_cl2, &map_cr2};
    asm volatile("prefetch.tensormap [%0];" ::"l"(maps[lane]) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), 2 * kEpiWarps);
    mbar_init(smem_u32(&sh->lp_done), 2 * kEpiWarps);
    sh->abort_flag = 0;
    sh->is_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)), "r"(C::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync();          // the peer's barriers and tensor memory exist before anyone uses them
  pdl_prologue();          // everything above overlapped the tail of the previous kernel
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t g = 0;                                           // running k-block count
      bool ok = true;
      for (int t = pair; t < a.num_tiles && ok; t += num_pairs) {
        const TileCoord tc = tile_coord(t, a);
        const int r0 = tc.m_tile * kPairM + (int)rank * kBlockM;     // this CTA's left-operand rows
        const int c0 = tc.n_tile * kBlockN + (int)rank * kHalfN;     // this CTA's half of the right operand
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t use = g / kStages;
          if (use > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (use - 1) & 1, abort_flag, a.err_word)) {
            ok = false;
            break;
          }
          // one barrier (the leader's) collects the bytes of both CTAs
          if (rank == 0) mbar_expect_tx(smem_u32(&sh->full[s]), 2 * C::kStageBytes);
          const uint32_t bar = map_to_cta(smem_u32(&sh->full[s]), 0);
          const uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
          const int k0 = kb * kBlockK;
          if (kAnyProbe || MODE == kRefOnly) {
            tma_load_3d(base + C::kOffL, &map_l, bar, k0, r0, tc.b);
            tma_load_3d(base + C::kOffR, &map_r, bar, k0, c0, tc.b);
          }
          if (kAnyProbe) {
            tma_load_3d(base + C::kOffLa, &map_la, bar, k0, r0, tc.b);
            tma_load_3d(base + C::kOffRa, &map_ra, bar, k0, c0, tc.b);
          }
          if (kAnyProbe || MODE == kLpOnly) {
            tma_load_3d(base + C::kOffCl, &map_cl, bar, k0, r0, tc.b);
            tma_load_3d(base + C::kOffCr, &map_cr, bar, k0, c0, tc.b);
          }
          if constexpr (MODE == kProbe2) {
            tma_load_3d(base + C::kOffCl2, &map_cl2, bar, k0, r0, tc.b);
            tma_load_3d(base + C::kOffCr2, &map_cr2, bar, k0, c0, tc.b);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (rank == 0) {   // the whole warp, converged: see elect_one()
      const bool lead = elect_one();
      constexpr uint32_t idesc_bf16 = make_idesc(1, 1, 1, kPairM, kBlockN);
      uint32_t g = 0, it = 0;
      bool ok = true;
      for (int t = pair; t < a.num_tiles && ok; t += num_pairs, ++it) {
        const uint32_t col_ref = 0u, col_den = 128u;
        const uint32_t col_lp = MODE == kProbe2 ? 256u : 0u;
        auto issue_ref = [&](uint32_t base, int kb) {
          const uint64_t dl = smem_desc(base + C::kOffL, 128), dr = smem_desc(base + C::kOffR, 128);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
            mma_pair<kKindF16>(tmem_base + col_ref, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0, lead);
        };
        auto issue_den = [&](uint32_t base, int kb) {
          const uint64_t dl = smem_desc(base + C::kOffLa, 128), dr = smem_desc(base + C::kOffRa, 128);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k)
            mma_pair<kKindF16>(tmem_base + col_den, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0, lead);
        };
        auto issue_lp = [&](uint32_t base, int kb) {
          const uint64_t dl = smem_desc(base + C::kOffCl, 64), dr = smem_desc(base + C::kOffCr, 64);
#pragma unroll
          for (int k = 0; k < kBlockK / 32; ++k)   // 32 codes = 32 bytes per step
            mma_pair<LPKIND>(tmem_base + col_lp, dl + 2 * k, dr + 2 * k, a.idesc_lp, (kb | k) != 0, lead);
        };
        // Probe2: the second format's accumulator takes the fourth block (columns 384..511), so
        // nothing rotates.  The reference and denominator blocks come back when both epilogues
        // have copied them out (tmem_empty), the two 8-bit blocks when they have finished the tile
        // (lp_done); the reference and denominator MMAs of as many k-blocks as there are stages
        // are therefore issued between the two signals.
        auto issue_lp2 = [&](uint32_t base, int kb) {
          if constexpr (MODE == kProbe2) {
            const uint64_t dl = smem_desc(base + C::kOffCl2, 64), dr = smem_desc(base + C::kOffCr2, 64);
#pragma unroll
            for (int k = 0; k < kBlockK / 32; ++k)
              mma_pair<LPKIND2>(tmem_base + 384u, dl + 2 * k, dr + 2 * k, a.idesc_lp2, (kb | k) != 0, lead);
          }
        };
        int kb = 0;
        if (MODE == kProbe2) {
          if (it > 0 && !mbar_wait_warp(smem_u32(&sh->tmem_empty), (it - 1) & 1, abort_flag, a.err_word)) break;
          tc_fence_after();
          const int n_ahead = num_kb < kStages ? num_kb : kStages;
          for (int j = 0; j < n_ahead && ok; ++j) {
            const int s = (g + j) % kStages;
            if (!mbar_wait_warp(smem_u32(&sh->full[s]), ((g + j) / kStages) & 1, abort_flag, a.err_word)) ok = false;
            tc_fence_after();
            if (ok) {
              const uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
              issue_ref(base, j);
              issue_den(base, j);
            }
          }
          if (!ok) break;
          if (it > 0 && !mbar_wait_warp(smem_u32(&sh->lp_done), (it - 1) & 1, abort_flag, a.err_word)) break;
          tc_fence_after();
          for (; kb < n_ahead; ++kb, ++g) {
            const int s = g % kStages;
            const uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
            issue_lp(base, kb);
            issue_lp2(base, kb);
            tc_commit_pair(smem_u32(&sh->empty[s]), lead);
          }
        }
        if (MODE != kProbe2 && it > 0 &&
            !mbar_wait_warp(smem_u32(&sh->tmem_empty), (it - 1) & 1, abort_flag, a.err_word))
          break;
        tc_fence_after();
        for (; kb < num_kb; ++kb, ++g) {
          const int s = g % kStages;
          const uint32_t use = g / kStages;
          if (!mbar_wait_warp(smem_u32(&sh->full[s]), use & 1, abort_flag, a.err_word)) { ok = false; break; }
          tc_fence_after();
          const uint32_t base = smem_u32(tiles + (size_t)s * C::kStageBytes);
          if (kAnyProbe || MODE == kRefOnly) issue_ref(base, kb);
          if (kAnyProbe) issue_den(base, kb);
          if (kAnyProbe || MODE == kLpOnly) issue_lp(base, kb);
          issue_lp2(base, kb);
          tc_commit_pair(smem_u32(&sh->empty[s]), lead);        // frees the stage in both CTAs
        }
        if (ok) tc_commit_pair(smem_u32(&sh->tmem_full), lead); // this tile's accumulators are complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const int h = (warp - 2) >> 2;                // which 64-column half of the tile
    const int et = (warp - 2) * 32 + lane;        // 0..255
    const float dl_tensor = (MODE != kRefOnly && !a.pc_l) ? __ldg(a.dl) : 1.f;
    const float dr_tensor = (MODE != kRefOnly && !a.pc_r) ? __ldg(a.dr) : 1.f;
    const bool per_col = MODE != kRefOnly && a.pc_r;
    const uint32_t tmem_empty_leader = map_to_cta(smem_u32(&sh->tmem_empty), 0);
    double acc[kFormats][5];                       // per format: sum BE, max BE, sum diff^2, sum C^2, sum D^2
#pragma unroll
    for (int f = 0; f < kFormats; ++f)
#pragma unroll
      for (int i = 0; i < 5; ++i) acc[f][i] = 0.0;
    [[maybe_unused]] const float dl_tensor2 = (MODE == kProbe2 && !a.pc_l) ? __ldg(a.dl2) : 1.f;
    [[maybe_unused]] const float dr_tensor2 = (MODE == kProbe2 && !a.pc_r) ? __ldg(a.dr2) : 1.f;
    auto add_stats = [&](int f, const Stats2& st) {
      float x0, x1;
      unpack2(st.be, x0, x1); acc[f][0] += (double)x0 + (double)x1;
      unpack2(st.d2, x0, x1); acc[f][2] += (double)x0 + (double)x1;
      unpack2(st.r2, x0, x1); acc[f][3] += (double)x0 + (double)x1;
      unpack2(st.n2, x0, x1); acc[f][4] += (double)x0 + (double)x1;
      acc[f][1] = fmax(acc[f][1], (double)st.mx);
    };
    uint32_t it = 0;
    for (int t = pair; t < a.num_tiles; t += num_pairs, ++it) {
      const TileCoord tc = tile_coord(t, a);
      float* dr_s = sh->delta_r[it & 1];
      [[maybe_unused]] float* dr_s2 = sh->delta_r2[it & 1];
      if (per_col && et < kBlockN) {
        const int64_t col = (int64_t)tc.n_tile * kBlockN + et;
        dr_s[et] = col < a.N ? __ldg(a.dr + (int64_t)tc.b * a.N + col) : 0.f;
        if (MODE == kProbe2) dr_s2[et] = col < a.N ? __ldg(a.dr2 + (int64_t)tc.b * a.N + col) : 0.f;
      }
      const int64_t row = (int64_t)tc.m_tile * kPairM + rank * kBlockM + q * 32 + lane;
      const bool row_ok = row < a.M;
      float dlv = dl_tensor;
      if (MODE != kRefOnly && a.pc_l) dlv = row_ok ? __ldg(a.dl + (int64_t)tc.b * a.M + row) : 0.f;
      [[maybe_unused]] float dlv2 = dl_tensor2;
      if (MODE == kProbe2 && a.pc_l) dlv2 = row_ok ? __ldg(a.dl2 + (int64_t)tc.b * a.M + row) : 0.f;

      const bool ok = mbar_wait(smem_u32(&sh->tmem_full), it & 1, abort_flag, a.err_word);
      // one barrier publishes delta_r and makes the give-up decision uniform over the epilogue
      if (epi_barrier_any(!ok)) break;
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
      if (MODE == kProbe2) {
        // Fixed blocks: reference 0, denominator 128, first format 256, second format 384.  Copy
        // this warp's 64 reference and denominator columns into registers and hand those two
        // blocks back (the next tile's reference and denominator MMAs start), walk both 8-bit
        // blocks in chunks of 16 columns, then report the tile finished (lp_done).
        const int64_t colw = (int64_t)tc.n_tile * kBlockN + h * 64;
        uint32_t rc[64], rd[64], rq[16];
        tmem_ld32(lane_addr + 0u + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&rc[0]));
        tmem_ld32(lane_addr + 0u + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&rc[32]));
        tmem_ld32(lane_addr + 128u + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&rd[0]));
        tmem_ld32(lane_addr + 128u + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&rd[32]));
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
        Stats2 st{0ull, 0ull, 0ull, 0ull, 0.f}, st2{0ull, 0ull, 0ull, 0ull, 0.f};
        const uint64_t ndl2 = pack2(-dlv, -dlv), drt2 = pack2(dr_tensor, dr_tensor);
        const uint64_t ndl2b = pack2(-dlv2, -dlv2), drt2b = pack2(dr_tensor2, dr_tensor2);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int cc0 = h * 64 + c * 16;
          const int64_t col0 = colw + c * 16;
          if (col0 < a.N) {                       // uniform across the warp
            const int n_live = (int)(a.N - col0 < 16 ? a.N - col0 : 16);
            tmem_ld16(lane_addr + 256u + cc0, rq);
            tmem_ld_wait();
            if (n_live == 16) stats16<LPKIND, false>(&rc[c * 16], &rd[c * 16], rq, ndl2, dr_s + cc0, per_col, drt2, 16, st);
            else stats16<LPKIND, true>(&rc[c * 16], &rd[c * 16], rq, ndl2, dr_s + cc0, per_col, drt2, n_live, st);
            tmem_ld16(lane_addr + 384u + cc0, rq);
            tmem_ld_wait();
            if (n_live == 16) stats16<LPKIND2, false>(&rc[c * 16], &rd[c * 16], rq, ndl2b, dr_s2 + cc0, per_col, drt2b, 16, st2);
            else stats16<LPKIND2, true>(&rc[c * 16], &rd[c * 16], rq, ndl2b, dr_s2 + cc0, per_col, drt2b, n_live, st2);
          }
        }
        if (row_ok) {
          add_stats(0, st);
          if constexpr (kFormats == 2) add_stats(1, st2);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&sh->lp_done), 0));
      } else {
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          const int cc0 = h * 64 + c * 32;          // first column of this chunk inside the tile
          const int64_t col0 = (int64_t)tc.n_tile * kBlockN + cc0;
          if (col0 >= a.N) break;                   // uniform across the warp
          const int n_live = (int)(a.N - col0 < 32 ? a.N - col0 : 32);
          uint32_t r[32];
          tmem_ld32(lane_addr + cc0, r);
          tmem_ld_wait();
          if (row_ok) {
            const int64_t o = ((int64_t)tc.b * a.M + row) * a.N + col0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < n_live) {
                if (MODE == kRefOnly) {
                  a.out_descaled[o + j] = __uint_as_float(r[j]);
                } else {
                  const float acc = LPKIND == kKindI8 ? (float)(int)r[j] : __uint_as_float(r[j]);
                  const float drj = per_col ? dr_s[cc0 + j] : dr_tensor;
                  if (a.out_descaled) a.out_descaled[o + j] = acc * (dlv * drj);
                  if (a.out_raw) reinterpret_cast<uint32_t*>(a.out_raw)[o + j] = r[j];
                }
              }
            }
          }
        }
      }
      if (!kAnyProbe) {
        // this warp has finished reading the accumulator of the tile: tell the leader's MMA lane
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
      }
    }
    if (kAnyProbe) {
      // per format: warp sums -> CTA record -> (last CTA) fixed-order sum of all records
#pragma unroll
      for (int f = 0; f < kFormats; ++f) {
#pragma unroll
        for (int i = 0; i < 5; ++i) {
          double x = acc[f][i];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const double y = __shfl_xor_sync(0xffffffffu, x, o);
            x = i == 1 ? fmax(x, y) : x + y;
          }
          if (lane == 0) sh->red[f * 5 + i][warp - 2] = x;
        }
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (et == 0) {
        for (int f = 0; f < kFormats; ++f) {
          double* rec = a.partials + ((int64_t)f * gridDim.x + blockIdx.x) * kPartialDoubles;
          for (int i = 0; i < 5; ++i) {
            double x = 0.0;
            for (int w = 0; w < kEpiWarps; ++w) x = i == 1 ? fmax(x, sh->red[f * 5 + i][w]) : x + sh->red[f * 5 + i][w];
            __stcg(rec + i, x);
          }
        }
        __threadfence();
        const uint32_t prev = atomicAdd(a.done_counter, 1u);
        sh->is_last = prev == gridDim.x - 1 ? 1u : 0u;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (sh->is_last && warp == 2) {
        // last CTA: every record is visible; fixed-order sum (lane l takes records l, l+32, ...)
        __threadfence();
        for (int f = 0; f < kFormats; ++f) {
          double r[5] = {0, 0, 0, 0, 0};
          for (int i = lane; i < (int)gridDim.x; i += 32) {
            const double* rec = a.partials + ((int64_t)f * gridDim.x + i) * kPartialDoubles;
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
            qm_metric_result* out = a.result + f;
            out->sum_be = r[0]; out->max_be = r[1]; out->sum_diff2 = r[2];
            out->sum_ref2 = r[3]; out->sum_den2 = r[4];
            out->count = a.count;
            out->device_error = a.err_word ? *reinterpret_cast<volatile uint32_t*>(a.err_word) : 0u;
            out->reserved = 0;
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- common exit
  // Neither CTA may leave while the other can still read its shared memory, signal its
  // barriers or write its tensor memory.
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols)
                 : "memory");
  }
}

// ------------------------------------------------------------------ plain products on 256 x 256 tiles
// qm_gemm and qm_gemm_ref on wide outputs.  One accumulator per tile leaves room for 256-column
// tiles, which halves the MMA instructions and the left-operand traffic per flop, and for two
// accumulator buffers (2 x 256 tensor-memory columns), so the epilogue of one tile runs under the
// main loop of the next.  A k-block is 128 BYTES of contraction per row for every operand type
// (64 bf16 or 128 codes), so all tiles are 128-byte-swizzled 16 KB blocks: a stage is this CTA's
// 128 left rows and its 128-row half of the right tile, 32 KB, six stages.  Roles, barriers,
// bounded waits and the exit protocol are those of tc_kernel.
constexpr int kWideN = 256;
constexpr int kWideHalfN = 128;
constexpr int kWideStages = 6;
constexpr uint32_t kWideTile = 128 * 128;                 // 16 KB
constexpr uint32_t kWideStageBytes = 2 * kWideTile;

struct SharedWide {
  uint64_t full[kWideStages];
  uint64_t empty[kWideStages];
  uint64_t tmem_full[2];         // per CTA, per accumulator buffer
  uint64_t tmem_empty[2];        // leader, per accumulator buffer
  uint32_t tmem_base;
  uint32_t abort_flag;
  float delta_r[2][kWideN];
};

// KIND: kKindF16 (bf16 x bf16 -> fp32 output), kKindF8 / kKindI8 (descaled and/or raw output)
template <int KIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_wide_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const KernelArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedWide* sh = reinterpret_cast<SharedWide*>(tiles + (size_t)kWideStages * kWideStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  constexpr int kElemsPerBlock = KIND == kKindF16 ? 64 : 128;          // contraction elements per k-block
  const int num_kb = (int)((a.K + kElemsPerBlock - 1) / kElemsPerBlock);
  volatile uint32_t* abort_flag = &sh->abort_flag;

  if (warp == 0 && lane < 2) {
    const CUtensorMap* maps[2] = {&map_a, &map_b};
    asm volatile("prefetch.tensormap [%0];" ::"l"(maps[lane]) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kWideStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->tmem_full[b]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[b]), 2 * kEpiWarps);
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync();
  pdl_prologue();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t g = 0;
      bool ok = true;
      for (int t = pair; t < a.num_tiles && ok; t += num_pairs) {
        const TileCoord tc = tile_coord(t, a);
        const int r0 = tc.m_tile * kPairM + (int)rank * kBlockM;
        const int c0 = tc.n_tile * kWideN + (int)rank * kWideHalfN;
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kWideStages;
          const uint32_t use = g / kWideStages;
          if (use > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (use - 1) & 1, abort_flag, a.err_word)) {
            ok = false;
            break;
          }
          if (rank == 0) mbar_expect_tx(smem_u32(&sh->full[s]), 2 * kWideStageBytes);
          const uint32_t bar = map_to_cta(smem_u32(&sh->full[s]), 0);
          const uint32_t base = smem_u32(tiles + (size_t)s * kWideStageBytes);
          tma_load_3d(base, &map_a, bar, kb * kElemsPerBlock, r0, tc.b);
          tma_load_3d(base + kWideTile, &map_b, bar, kb * kElemsPerBlock, c0, tc.b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA, converged warp)
    if (rank == 0) {
      const bool lead = elect_one();
      const uint32_t idesc = KIND == kKindF16 ? make_idesc(1, 1, 1, kPairM, kWideN) : a.idesc_lp;
      uint32_t g = 0, it = 0;
      bool ok = true;
      for (int t = pair; t < a.num_tiles && ok; t += num_pairs, ++it) {
        const uint32_t buf = it & 1;
        // the buffer was last used by tile it-2: wait until both epilogues have drained it
        if (it >= 2 && !mbar_wait_warp(smem_u32(&sh->tmem_empty[buf]), ((it >> 1) - 1) & 1, abort_flag, a.err_word))
          break;
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb, ++g) {
          const int s = g % kWideStages;
          if (!mbar_wait_warp(smem_u32(&sh->full[s]), (g / kWideStages) & 1, abort_flag, a.err_word)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t base = smem_u32(tiles + (size_t)s * kWideStageBytes);
          const uint64_t da = smem_desc(base, 128), db = smem_desc(base + kWideTile, 128);
#pragma unroll
          for (int k = 0; k < 4; ++k)             // 32 bytes of contraction per instruction
            mma_pair<KIND>(tmem_base + buf * kWideN, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0, lead);
          tc_commit_pair(smem_u32(&sh->empty[s]), lead);
        }
        if (ok) tc_commit_pair(smem_u32(&sh->tmem_full[buf]), lead);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;                // which 128-column half of the tile
    const int et = (warp - 2) * 32 + lane;        // 0..255
    const float dl_tensor = (KIND != kKindF16 && !a.pc_l) ? __ldg(a.dl) : 1.f;
    const float dr_tensor = (KIND != kKindF16 && !a.pc_r) ? __ldg(a.dr) : 1.f;
    const bool per_col = KIND != kKindF16 && a.pc_r;
    // 16-byte stores need 16-byte aligned rows: output bases aligned and N a multiple of 4
    const bool vec_ok = (a.N & 3) == 0 && (reinterpret_cast<uintptr_t>(a.out_descaled) & 15) == 0 &&
                        (reinterpret_cast<uintptr_t>(a.out_raw) & 15) == 0;
    uint32_t it = 0;
    for (int t = pair; t < a.num_tiles; t += num_pairs, ++it) {
      const TileCoord tc = tile_coord(t, a);
      const uint32_t buf = it & 1;
      float* dr_s = sh->delta_r[buf];
      if (per_col) {
        const int64_t col = (int64_t)tc.n_tile * kWideN + et;
        dr_s[et] = col < a.N ? __ldg(a.dr + (int64_t)tc.b * a.N + col) : 0.f;
      }
      const int64_t row = (int64_t)tc.m_tile * kPairM + rank * kBlockM + q * 32 + lane;
      const bool row_ok = row < a.M;
      float dlv = dl_tensor;
      if (KIND != kKindF16 && a.pc_l) dlv = row_ok ? __ldg(a.dl + (int64_t)tc.b * a.M + row) : 0.f;
      const bool ok = mbar_wait(smem_u32(&sh->tmem_full[buf]), (it >> 1) & 1, abort_flag, a.err_word);
      if (epi_barrier_any(!ok)) break;            // also publishes delta_r
      tc_fence_after();
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kWideN;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        const int cc0 = h * 128 + c * 32;
        const int64_t col0 = (int64_t)tc.n_tile * kWideN + cc0;
        if (col0 >= a.N) break;                   // uniform across the warp
        const int n_live = (int)(a.N - col0 < 32 ? a.N - col0 : 32);
        uint32_t r[32];
        tmem_ld32(lane_addr + cc0, r);
        tmem_ld_wait();
        if (row_ok) {
          const int64_t o = ((int64_t)tc.b * a.M + row) * a.N + col0;
          if (n_live == 32 && vec_ok) {
            // 128 bytes per thread and chunk: whole lines
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              if (KIND == kKindF16) {
                *reinterpret_cast<uint4*>(a.out_descaled + o + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
              } else {
                if (a.out_raw)
                  *reinterpret_cast<uint4*>(reinterpret_cast<uint32_t*>(a.out_raw) + o + j) =
                      make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                if (a.out_descaled) {
                  float4 v;
                  float* pv = &v.x;
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    const float acc = KIND == kKindI8 ? (float)(int)r[j + e] : __uint_as_float(r[j + e]);
                    pv[e] = acc * (dlv * (per_col ? dr_s[cc0 + j + e] : dr_tensor));
                  }
                  *reinterpret_cast<float4*>(a.out_descaled + o + j) = v;
                }
              }
            }
          } else {
            for (int j = 0; j < n_live; ++j) {
              if (KIND == kKindF16) {
                a.out_descaled[o + j] = __uint_as_float(r[j]);
              } else {
                const float acc = KIND == kKindI8 ? (float)(int)r[j] : __uint_as_float(r[j]);
                if (a.out_descaled) a.out_descaled[o + j] = acc * (dlv * (per_col ? dr_s[cc0 + j] : dr_tensor));
                if (a.out_raw) reinterpret_cast<uint32_t*>(a.out_raw)[o + j] = r[j];
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&sh->tmem_empty[buf]), 0));
    }
  }

  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------ the fused probe kernel
// One persistent launch computes the Eq. 3 records of up to kMaxGroup probes (one probe is a
// group of one).  A launch per probe pays, each time, the kernel's set-up and drain, the launch
// gap, and the last wave of a tile count that is not a multiple of the 74 CTA pairs; here the
// tiles of all probes form one sequence.  The host orders the probes by descending contraction
// length (tile cost) and the sequence is dealt to the pairs back and forth (round r gives pair p
// position r P + p when r is even and r P + P-1-p when it is odd), which for descending costs
// balances the pairs to within one tile of the cheapest kind.  The operand maps, scales, shapes
// and the 8-bit MMA kind are read per tile from a table in the kernel's parameter space.  A
// pair's positions increase, so it meets each probe in one run: when the probe changes, the
// epilogue warps reduce their statistics and write the CTA's record of the probe they leave.
//
// What bounds this kernel is shared-memory bandwidth: per 64-deep k-block the tensor cores need
// 640 cycles, and with all six operand tiles (L, |L|, codes, R, |R|, codes) staged in shared
// memory an SM writes 60 KB and reads 60 KB per k-block, which takes it 940.  So the left operand
// of the denominator product |L|.|R| is not staged in shared memory: converter warps read this
// CTA's 128 rows of the L tile, clear the sign bits and store the result into TENSOR memory, from
// where the denominator MMAs take their A operand; the same warps write the |R| half-tile into
// the stage.  No |x| copy exists in HBM, TMA brings 36 KB per k-block, the MMAs read 44 KB and the
// converters move 32 KB.
//
// Roles in each CTA (512 threads = 4 warpgroups; registers are re-divided with setmaxnreg):
//   warp 0        TMA producer: per k-block the bf16 tiles of L and R and both code tiles into a
//                 ring of kStages stages; a CTA's loads complete on its own `full` barrier.
//   warp 1        allocates tensor memory; in the leader CTA it runs the MMA loop converged and
//                 one elected lane issues the pair's MMAs; tcgen05.commit frees a stage (shared
//                 and tensor memory) in both CTAs (`empty`).
//   warps 2, 3    idle (they fill the first warpgroup).
//   warps 4..7    converters, one per tensor-memory lane quarter: thread = one of the CTA's 128
//                 left-operand rows.
//   warps 8..15   epilogue.
// Tensor memory: columns 0..127 reference L.R, 128..255 denominator |L|.|R|, 256..383 the 8-bit
// product, 384..511 four stages of |L| (32 columns of two bf16 each per stage; the shared-memory
// ring has five stages, so TMA runs a k-block further ahead than the converters can).  The epilogue
// copies its reference and denominator columns into registers and hands those two blocks back
// at once (`tmem_empty`), after which the MMA warp issues the next tile's reference and
// denominator MMAs for as many k-blocks as there are stages; the 8-bit MMAs of those k-blocks
// follow when the epilogue has finished the 8-bit block (`lp_done`).  No M x N matrix ever goes
// to HBM.
constexpr int kMaxGroup = 16;
constexpr int kProbeThreads = 512;
constexpr int kFirstEpiWarp = 8;               // warps 8..15: lane quarter = warp % 4 holds for both groups
// registers per thread after the split (launch: 128 each): 56 + 104 + 176 + 176 = 4 x 128
constexpr int kRegsCtl = 56, kRegsConv = 104, kRegsEpi = 176;
static_assert(kRegsCtl + kRegsConv + 2 * kRegsEpi <= 4 * 128, "the split must fit what the block was launched with");

struct CfgP {
  static constexpr int kStages = 5;          // stages of shared memory (TMA ring)
  static constexpr int kAbsStages = 4;       // stages of |L| in tensor memory (128 columns / 32)
  // stage: L, R, |R| (written by the converters), codes of L, codes of R
  static constexpr uint32_t kOffL = 0, kOffR = kABf16, kOffRa = kOffR + kBBf16, kOffCl = kOffRa + kBBf16;
  static constexpr uint32_t kOffCr = kOffCl + kALp;
  static constexpr uint32_t kStageBytes = kOffCr + kBLp;             // 44 KB
  static constexpr uint32_t kTileBytes = kStages * kStageBytes;      // 220 KB
  static constexpr uint32_t kColRef = 0, kColDen = 128, kColLp = 256, kColAbsL = 384;   // tensor-memory columns
};

// What the roles need of a probe for every tile, copied to shared memory once per CTA: the
// launch's table sits in the kernel's parameter space, and reads of it with an index known only
// at run time go through the small constant cache, which eleven kilobytes of table thrash.
struct WalkInfo {
  int32_t tile_begin, per_b, inner, num_kb;         // per_b = tiles_m * tiles_n (tiles per batch element);
                                                    // inner = tiles_n: column tiles run fastest, -tiles_m: row tiles do
  int32_t half_n, kind;
  uint32_t idesc_ref, idesc_lp;
};

struct SharedP {
  uint64_t full[CfgP::kStages];     // per CTA: this CTA's loads of a stage have landed
  uint64_t ready[CfgP::kAbsStages]; // leader: both CTAs' converters have seen their loads land and have written
                                    //         |L| (tensor memory) and |R| (stage)
  uint64_t empty[CfgP::kStages];    // per CTA: the pair's MMAs have finished with the k-block of the stage
  uint64_t tmem_full;               // per CTA: the tile's accumulators are complete
  uint64_t tmem_empty;              // leader: both CTAs' epilogues have copied out reference and denominator
  uint64_t lp_done;                 // leader: both CTAs' epilogues have finished a tile
  uint64_t drain;                   // leader, give-up path only: every MMA issued so far has completed
  uint32_t tmem_base;
  uint32_t abort_flag;
  uint32_t is_last;
  uint32_t issued;                  // k-blocks whose loads the producer has issued (read on the give-up path)
  float delta_r[2][kBlockN];
  double red[5][kEpiWarps];
  WalkInfo walk[kMaxGroup];
};

struct GroupProblem {
  CUtensorMap maps[4];        // L, R, codes L, codes R
  KernelArgs a;               // num_tiles, tiles_m, tiles_n: of this probe
  int32_t tile_begin;         // position of its first tile in the sequence
  int32_t kind;               // kKindF8 or kKindI8
  int32_t half_n;             // right-operand rows each CTA stages: 64, or 32 for outputs at most 64 wide
  int32_t m_fastest;          // the tiles of a batch element are walked down the rows first (below)
  uint32_t idesc_ref;         // instruction descriptor of the bf16 MMAs (N = 2 * half_n)
};
struct GroupTable {
  int32_t n, total_tiles;
  uint32_t stop_after_kb;     // test hook: the producer issues no k-block beyond this many (0xffffffff: off)
  uint32_t pad0;
  uint64_t wait_limit_ns;     // bound of every barrier wait
  int32_t pad[10];
  GroupProblem p[kMaxGroup];
};

// position of pair `pair` in round r of the back-and-forth deal
__device__ __forceinline__ int group_position(int r, int pair, int num_pairs) {
  return r * num_pairs + ((r & 1) ? num_pairs - 1 - pair : pair);
}

// The tiles of one CTA pair in order, k-block by k-block: every role walks the same sequence.
// A pair's positions ascend, so the search for a position's probe continues from the probe in hand.
struct TileWalk {
  const WalkInfo* wk;
  int n, total_tiles;
  int r, pair, num_pairs;
  int pi, num_kb, kb, half_n;
  TileCoord tc;
  bool valid;
  __device__ __forceinline__ void start(const WalkInfo* wk_, int n_, int total_tiles_, int pair_, int num_pairs_) {
    wk = wk_; n = n_; total_tiles = total_tiles_;
    r = -1; pair = pair_; num_pairs = num_pairs_; kb = 0; num_kb = 0; pi = 0; half_n = 0; valid = true;
    next_tile();
  }
  // moves to the pair's next tile; valid = false when there is none
  __device__ __forceinline__ void next_tile() {
    while (true) {
      ++r;
      const int pos = group_position(r, pair, num_pairs);
      if (pos >= total_tiles) {
        if (r * num_pairs >= total_tiles) { valid = false; return; }   // no round reaches further
        continue;
      }
      while (pi + 1 < n && pos >= wk[pi + 1].tile_begin) ++pi;
      const int4 w4 = *reinterpret_cast<const int4*>(&wk[pi]);          // tile_begin, per_b, inner, num_kb
      const int t = pos - w4.x;
      tc.b = t / w4.y;
      const int rem = t - tc.b * w4.y;
      const int inner = w4.z < 0 ? -w4.z : w4.z;
      const int outer_i = rem / inner, inner_i = rem - outer_i * inner;
      tc.m_tile = w4.z < 0 ? inner_i : outer_i;
      tc.n_tile = w4.z < 0 ? outer_i : inner_i;
      num_kb = w4.w;
      half_n = wk[pi].half_n;
      kb = 0;
      return;
    }
  }
  // moves to the next k-block of the sequence
  __device__ __forceinline__ void next_kb() {
    if (++kb >= num_kb) next_tile();
  }
};

// Bounded wait with the launch's limit; see mbar_wait.
struct Waiter {
  volatile uint32_t* abort_flag;
  uint32_t* err_word;
  uint64_t limit_ns;
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t polls = 0;
    while (true) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((++polls & 0x3fu) == 0) {
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
          *abort_flag = 1u;
          if (err_word) atomicOr(err_word, QM_DEVERR_TIMEOUT);
          return false;
        }
      }
    }
  }
  __device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity) const {
    return __all_sync(0xffffffffu, wait(bar, parity));
  }
};

// Tile load into this CTA's shared memory, completing on this CTA's barrier.
__device__ __forceinline__ void tma_load_3d_local(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                  int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns of tensor memory from registers: lane (base + t) <- thread t.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// D[256 x N] (+)= A[256 x 16] . B[N x 16]^T across the CTA pair, A (bf16) taken from tensor memory:
// each CTA's 128 rows at the same column address, two values per 32-bit column.
__device__ __forceinline__ void mma_pair_a_tmem(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc,
                                                uint32_t accumulate, bool lead) {
  if (!lead) return;
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

__global__ void __launch_bounds__(kProbeThreads, 1)
tc_group_kernel(const __grid_constant__ GroupTable tab) {
  using C = CfgP;
  constexpr int kStages = C::kStages, kAbs = C::kAbsStages;
  extern __shared__ uint8_t smem_raw[];
  // tiles start on a 1024-byte boundary (the 128-byte swizzle atom); the offset is the same in
  // both CTAs of the pair because their dynamic shared memory starts at the same address
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedP* sh = reinterpret_cast<SharedP*>(tiles + C::kTileBytes);
  const uint32_t tile_base = smem_u32(tiles);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const Waiter w{&sh->abort_flag, tab.p[0].a.err_word, tab.wait_limit_ns};   // a timed-out wait is reported in probe 0's word

  if (warp == 0) {
    // fetch the tensor maps of this pair's first tile into the descriptor cache
    const int pos = group_position(0, pair, num_pairs);
    if (pos < tab.total_tiles && lane < 4) {
      int pi = 0;
      while (pi + 1 < tab.n && pos >= tab.p[pi + 1].tile_begin) ++pi;
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tab.p[pi].maps[lane]) : "memory");
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int s = 0; s < kAbs; ++s) mbar_init(smem_u32(&sh->ready[s]), 2 * 4);   // four converter warps in each CTA
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), 2 * kEpiWarps);
    mbar_init(smem_u32(&sh->lp_done), 2 * kEpiWarps);
    mbar_init(smem_u32(&sh->drain), 1);
    sh->abort_flag = 0;
    sh->is_last = 0;
    sh->issued = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&sh->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  if (warp == 2 && lane < tab.n) {
    const GroupProblem& pr = tab.p[lane];
    WalkInfo wi;
    wi.tile_begin = pr.tile_begin; wi.per_b = pr.a.tiles_m * pr.a.tiles_n;
    wi.inner = pr.m_fastest ? -pr.a.tiles_m : pr.a.tiles_n;
    wi.num_kb = (int)((pr.a.K + kBlockK - 1) / kBlockK);
    wi.half_n = pr.half_n; wi.kind = pr.kind; wi.idesc_ref = pr.idesc_ref; wi.idesc_lp = pr.a.idesc_lp;
    sh->walk[lane] = wi;
  }
  tc_fence_before();
  __syncthreads();
  __syncwarp();
  cluster_sync();          // the peer's barriers and tensor memory exist before anyone uses them
  pdl_prologue();          // everything above overlapped the tail of the previous kernel
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsCtl));
    if (warp == 0) {
      // ---------------------------------------------------------- TMA producer (both CTAs)
      if (lane == 0) {
        TileWalk tw;
        tw.start(sh->walk, tab.n, tab.total_tiles, pair, num_pairs);
        for (uint32_t g = 0; tw.valid; ++g, tw.next_kb()) {
          const int s = g % kStages;
          const uint32_t use = g / kStages;
          if (g >= tab.stop_after_kb) break;                  // test hook: the consumers' waits run out
          if (use > 0 && !w.wait(smem_u32(&sh->empty[s]), (use - 1) & 1)) break;
          const GroupProblem& pr = tab.p[tw.pi];
          const int r0 = tw.tc.m_tile * kPairM + (int)rank * kBlockM;     // this CTA's left-operand rows
          const int c0 = tw.tc.n_tile * kBlockN + (int)rank * tw.half_n;  // this CTA's half of the right operand
          const uint32_t bar = smem_u32(&sh->full[s]);
          mbar_expect_tx(bar, kABf16 + kALp + (uint32_t)tw.half_n * (kBlockK * 2 + kBlockK));
          const uint32_t base = tile_base + s * C::kStageBytes;
          const int k0 = tw.kb * kBlockK;
          tma_load_3d_local(base + C::kOffR, &pr.maps[1], bar, k0, c0, tw.tc.b);     // the converters read this one
          tma_load_3d_local(base + C::kOffL, &pr.maps[0], bar, k0, r0, tw.tc.b);
          tma_load_3d_local(base + C::kOffCl, &pr.maps[2], bar, k0, r0, tw.tc.b);
          tma_load_3d_local(base + C::kOffCr, &pr.maps[3], bar, k0, c0, tw.tc.b);
          sh->issued = g + 1;
        }
      }
    } else if (warp == 1 && rank == 0) {
      // ---------------------------------------------------------- MMA issuer (leader CTA, converged warp)
      const bool lead = elect_one();
      uint32_t idesc_bf16 = 0;                 // of the tile in hand
      auto issue_ref_den = [&](uint32_t gg, int kb) {
        const uint32_t s = gg % kStages, base = tile_base + s * C::kStageBytes;
        const uint64_t dl = smem_desc(base + C::kOffL, 128), dr = smem_desc(base + C::kOffR, 128);
#pragma unroll
        for (int k = 0; k < kBlockK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
          mma_pair<kKindF16>(tmem_base + C::kColRef, dl + 2 * k, dr + 2 * k, idesc_bf16, (kb | k) != 0, lead);
        const uint64_t da = smem_desc(base + C::kOffRa, 128);
        const uint32_t ta = tmem_base + C::kColAbsL + 32u * (gg % kAbs);
#pragma unroll
        for (int k = 0; k < kBlockK / 16; ++k)   // 16 bf16 = 8 columns of tensor memory per step
          mma_pair_a_tmem(tmem_base + C::kColDen, ta + 8u * k, da + 2 * k, idesc_bf16, (kb | k) != 0, lead);
      };
      auto issue_lp = [&](uint32_t gg, int kb, int kind, uint32_t idesc_lp) {
        const uint32_t base = tile_base + (gg % kStages) * C::kStageBytes;
        const uint64_t cl = smem_desc(base + C::kOffCl, 64), cr = smem_desc(base + C::kOffCr, 64);
#pragma unroll
        for (int k = 0; k < kBlockK / 32; ++k) {  // 32 codes = 32 bytes per step
          if (kind == kKindI8) mma_pair<kKindI8>(tmem_base + C::kColLp, cl + 2 * k, cr + 2 * k, idesc_lp, (kb | k) != 0, lead);
          else mma_pair<kKindF8>(tmem_base + C::kColLp, cl + 2 * k, cr + 2 * k, idesc_lp, (kb | k) != 0, lead);
        }
      };
      auto wait_stage = [&](uint32_t gg) {
        if (!w.wait_warp(smem_u32(&sh->ready[gg % kAbs]), (gg / kAbs) & 1)) return false;
        tc_fence_after();
        return true;
      };
      TileWalk tw;
      tw.start(sh->walk, tab.n, tab.total_tiles, pair, num_pairs);
      uint32_t g = 0;
      bool ok = true;
      for (uint32_t it = 0; tw.valid && ok; ++it, tw.next_tile()) {
        const WalkInfo& wi = sh->walk[tw.pi];
        const int num_kb = tw.num_kb, kind = wi.kind;
        const uint32_t idesc_lp = wi.idesc_lp;
        idesc_bf16 = wi.idesc_ref;
        // the reference and denominator blocks come back when both epilogues have copied the
        // previous tile's values out; the 8-bit block when they have finished that tile
        if (it > 0 && !w.wait_warp(smem_u32(&sh->tmem_empty), (it - 1) & 1)) break;
        tc_fence_after();
        const int n_ahead = num_kb < kAbs ? num_kb : kAbs;
        for (int j = 0; j < n_ahead && ok; ++j) {
          ok = wait_stage(g + j);
          if (ok) issue_ref_den(g + j, j);
        }
        if (!ok) break;
        if (it > 0 && !w.wait_warp(smem_u32(&sh->lp_done), (it - 1) & 1)) break;
        tc_fence_after();
        int kb = 0;
        for (; kb < n_ahead; ++kb, ++g) {
          issue_lp(g, kb, kind, idesc_lp);
          tc_commit_pair(smem_u32(&sh->empty[g % kStages]), lead);
        }
        for (; kb < num_kb && ok; ++kb, ++g) {
          ok = wait_stage(g);
          if (!ok) break;
          issue_ref_den(g, kb);
          issue_lp(g, kb, kind, idesc_lp);
          tc_commit_pair(smem_u32(&sh->empty[g % kStages]), lead);        // frees the k-block in both CTAs
        }
        if (ok) tc_commit_pair(smem_u32(&sh->tmem_full), lead);           // this tile's accumulators are complete
      }
    }
  } else if (warp < kFirstEpiWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsConv));
    // ------------------------------------------------------------ converters (both CTAs)
    // Thread t of the four warps owns row t of this CTA's 128 left-operand rows (its warp's
    // tensor-memory lane quarter holds that row): once the stage has landed it reads its row of the
    // L tile from shared memory (128-byte swizzle: 16-byte chunk c of row r sits at c ^ (r & 7),
    // which makes these row-per-thread reads conflict-free), clears the sign bits and stores the
    // 32 words into the stage's tensor-memory columns.  (Loading the rows with plain global loads
    // instead, to spare shared memory the 16 KB, was tried: a warp then touches 32 lines per
    // instruction and the converters became the bottleneck, 1.6 x slower overall.)  The |R|
    // half-tile is a flat sign-cleared copy of the R half-tile (8 KB: four vectors per thread).
    const int q = warp & 3;
    const int t = q * 32 + lane;                   // 0..127
    const uint32_t ready_leader = map_to_cta(smem_u32(&sh->ready[0]), 0);
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + C::kColAbsL;
    const uint32_t row_off = (uint32_t)t * 128u, sw = (uint32_t)t & 7u;
    TileWalk tw;
    tw.start(sh->walk, tab.n, tab.total_tiles, pair, num_pairs);
    bool ok = true;
    for (uint32_t g = 0; ok && tw.valid; ++g, tw.next_kb()) {
      const uint32_t s = g % kStages, sa = g % kAbs, m = 0x7fff7fffu;
      // the tensor-memory columns were last read by the MMAs of k-block g - kAbs (its commit also
      // covers every earlier k-block, so the |R| slot of the stage is free as well)
      if (g >= (uint32_t)kAbs) {
        const uint32_t gp = g - kAbs;
        if (!w.wait_warp(smem_u32(&sh->empty[gp % kStages]), (gp / kStages) & 1)) { ok = false; break; }
      }
      if (!w.wait_warp(smem_u32(&sh->full[s]), (g / kStages) & 1)) { ok = false; break; }
      tc_fence_after();
      const uint32_t base = tile_base + s * C::kStageBytes;
      uint4 v[8], u[4];
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = lds128(base + C::kOffL + row_off + (((uint32_t)j ^ sw) << 4));
      const uint32_t rsrc = base + C::kOffR + (uint32_t)t * 16u;
      const int r_vec = tw.half_n * 8;                           // 16-byte vectors of the R half-tile that are in use
#pragma unroll
      for (int j = 0; j < 4; ++j) u[j] = t + 128 * j < r_vec ? lds128(rsrc + (uint32_t)j * 2048u) : make_uint4(0u, 0u, 0u, 0u);
      uint32_t a[32];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        a[4 * j] = v[j].x & m; a[4 * j + 1] = v[j].y & m; a[4 * j + 2] = v[j].z & m; a[4 * j + 3] = v[j].w & m;
      }
      tmem_st32(taddr + 32u * sa, a);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (t + 128 * j < r_vec)
          sts128(rsrc + (C::kOffRa - C::kOffR) + (uint32_t)j * 2048u, make_uint4(u[j].x & m, u[j].y & m, u[j].z & m, u[j].w & m));
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> the tensor core's reads
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(ready_leader + sa * 8u);
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsEpi));
    // ------------------------------------------------------------ epilogue (warps 8..15, both CTAs)
    // A warp may touch the tensor-memory lane quarter warp % 4; the two warps of a quarter split
    // the columns.  Copy this warp's 64 columns of the reference and denominator blocks into
    // registers, hand those two blocks back to the MMA lane, then walk the 8-bit block in chunks
    // of 16 columns; the statistics arithmetic runs under the next tile's main loop.
    const int q = warp & 3;
    const int ew = warp - kFirstEpiWarp;           // 0..7
    const int h = ew >> 2;                         // which half of the tile's columns
    const int et = ew * 32 + lane;                 // 0..255
    const uint32_t tmem_empty_leader = map_to_cta(smem_u32(&sh->tmem_empty), 0);
    double acc[5] = {0, 0, 0, 0, 0};               // of the probe in hand: sum BE, max BE, sum diff^2, C^2, D^2
    int cur = -1;                                  // the probe in hand
    // reduce the statistics of probe `pi` over the CTA and write its record (all 256 threads call)
    auto flush = [&](int pi) {
#pragma unroll
      for (int i = 0; i < 5; ++i) {
        double x = acc[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const double y = __shfl_xor_sync(0xffffffffu, x, o);
          x = i == 1 ? fmax(x, y) : x + y;
        }
        if (lane == 0) sh->red[i][ew] = x;
        acc[i] = 0.0;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (et < 5) {
        double x = 0.0;
        for (int k = 0; k < kEpiWarps; ++k) x = et == 1 ? fmax(x, sh->red[et][k]) : x + sh->red[et][k];
        __stcg(tab.p[pi].a.partials + (int64_t)blockIdx.x * kPartialDoubles + et, x);
        __threadfence();
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");       // red[] may be reused
    };
    uint32_t met = 0;                              // bit pi: this CTA has had tiles of probe pi
    // of the probe in hand (reloaded when the probe changes, not per tile)
    bool per_col = false, pc_l = false, is_i8 = false, narrow = false;
    float dr_tensor = 1.f, dl_tensor = 0.f;
    int pM = 0, pN = 0;                            // a probe's M and N are below 2^31 (its tensor maps require it)
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    TileWalk tw;
    tw.start(sh->walk, tab.n, tab.total_tiles, pair, num_pairs);
    for (uint32_t it = 0; tw.valid; ++it) {
      const int pi = tw.pi;
      if (pi != cur) {
        if (cur >= 0) flush(cur);
        cur = pi;
        met |= 1u << pi;
        const GroupProblem& pr = tab.p[pi];
        per_col = pr.a.pc_r != 0; pc_l = pr.a.pc_l != 0; is_i8 = pr.kind == kKindI8; narrow = pr.half_n < 64;
        pM = (int)pr.a.M; pN = (int)pr.a.N;
        dr_tensor = per_col ? 1.f : __ldg(pr.a.dr);
        dl_tensor = pc_l ? 0.f : __ldg(pr.a.dl);
      }
      const TileCoord tc = tw.tc;
      float* dr_s = sh->delta_r[it & 1];
      if (per_col && et < kBlockN) {
        const int col = tc.n_tile * kBlockN + et;
        dr_s[et] = col < pN ? __ldg(tab.p[pi].a.dr + (int64_t)tc.b * pN + col) : 0.f;
      }
      const int row = tc.m_tile * kPairM + (int)rank * kBlockM + q * 32 + lane;
      const bool row_ok = row < pM;
      float dlv = dl_tensor;
      if (pc_l) dlv = row_ok ? __ldg(tab.p[pi].a.dl + (int64_t)tc.b * pM + row) : 0.f;
      // the two warps of a lane quarter split the tile's columns: 64 each, or 32 each where the
      // tile is 64 wide (outputs at most 64 wide)
      const int cw = narrow ? 32 : 64, cbase = h * cw;
      const int colw = tc.n_tile * kBlockN + cbase;                  // first column of this warp

      const bool ok = w.wait(smem_u32(&sh->tmem_full), it & 1);
      // one barrier publishes delta_r and makes the give-up decision uniform over the epilogue
      if (epi_barrier_any(!ok)) break;
      tc_fence_after();
      // live = columns of this warp that exist in the matrix
      const int live = pN - colw < cw ? pN - colw : cw;          // <= 0: none
      const uint32_t lp_addr = lane_addr + C::kColLp + cbase;
      const uint32_t lp_done_leader = map_to_cta(smem_u32(&sh->lp_done), 0);
      const float* const drc = dr_s + cbase;
      uint32_t rc[64], rd[64], rq0[16];
      tmem_ld32(lane_addr + C::kColRef + cbase, *reinterpret_cast<uint32_t(*)[32]>(&rc[0]));
      tmem_ld32(lane_addr + C::kColDen + cbase, *reinterpret_cast<uint32_t(*)[32]>(&rd[0]));
      if (!narrow) {
        tmem_ld32(lane_addr + C::kColRef + cbase + 32, *reinterpret_cast<uint32_t(*)[32]>(&rc[32]));
        tmem_ld32(lane_addr + C::kColDen + cbase + 32, *reinterpret_cast<uint32_t(*)[32]>(&rd[32]));
      }
      if (live > 0) tmem_ld16(lp_addr, rq0);
      tmem_ld_wait();
      // The reference and denominator blocks are in registers: the MMA lane may start the next
      // tile's bf16 MMAs.  The 8-bit block follows in two steps, its first 16 columns with the
      // loads above and the rest once the first chunk has been evaluated (which frees the
      // registers the rest is read into); then the MMA lane may start the next tile's 8-bit MMAs as well, while the
      // remaining chunks are still being evaluated.  Every warp arrives on each barrier exactly
      // once per tile.
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_cluster(tmem_empty_leader);
        if (live <= 16) mbar_arrive_cluster(lp_done_leader);      // nothing further to read
      }
      StatsG st{0.f, 0.f, 0ull, 0ull, 0ull, 0.f};
      const float kd = -dlv * dr_tensor;
      const uint64_t kd2 = per_col ? pack2(-dlv, -dlv) : pack2(kd, kd);
      if (live > 0) stats_chunk<0>(rc, rd, rq0, live, is_i8, per_col, kd2, drc, st);
      if (live > 16) {
        // chunk 1 into the first chunk's registers, chunks 2 and 3 into those of the first
        // chunk's reference and denominator values
        uint32_t(&rq2)[16] = *reinterpret_cast<uint32_t(*)[16]>(&rc[0]);
        uint32_t(&rq3)[16] = *reinterpret_cast<uint32_t(*)[16]>(&rd[0]);
        tmem_ld16(lp_addr + 16, rq0);
        if (live > 32) tmem_ld16(lp_addr + 32, rq2);
        if (live > 48) tmem_ld16(lp_addr + 48, rq3);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lp_done_leader);
        stats_chunk<1>(rc, rd, rq0, live - 16, is_i8, per_col, kd2, drc, st);
        if (live > 32) stats_chunk<2>(rc, rd, rq2, live - 32, is_i8, per_col, kd2, drc, st);
        if (live > 48) stats_chunk<3>(rc, rd, rq3, live - 48, is_i8, per_col, kd2, drc, st);
      }
      if (row_ok) {
        float x0, x1;
        acc[0] += (double)st.be0 + (double)st.be1;
        unpack2(st.d2, x0, x1); acc[2] += (double)x0 + (double)x1;
        unpack2(st.r2, x0, x1); acc[3] += (double)x0 + (double)x1;
        unpack2(st.n2, x0, x1); acc[4] += (double)x0 + (double)x1;
        acc[1] = fmax(acc[1], (double)st.mx);
        double* const rows = tab.p[pi].a.row_stats;
        if (rows) row_stats_add(rows + ((int64_t)tc.b * pM + row) * 5, st);
      }
      tw.next_tile();
    }
    if (cur >= 0) flush(cur);
    // the records of the probes this CTA never met are zero
    if (et == 0) {
      for (int pi = 0; pi < tab.n; ++pi) {
        if (met & (1u << pi)) continue;
        double* rec = tab.p[pi].a.partials + (int64_t)blockIdx.x * kPartialDoubles;
        for (int i = 0; i < 5; ++i) __stcg(rec + i, 0.0);
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (et == 0) {
      __threadfence();
      const uint32_t prev = atomicAdd(tab.p[0].a.done_counter, 1u);
      sh->is_last = prev == gridDim.x - 1 ? 1u : 0u;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (sh->is_last) {
      // last CTA: every record of every probe is visible; each epilogue warp takes probes
      // ew, ew + 8, ...; fixed-order sum (lane l takes records l, l+32, ...)
      __threadfence();
      uint32_t* const err0 = tab.p[0].a.err_word;
      const uint32_t timed_out = err0 ? (*reinterpret_cast<volatile uint32_t*>(err0) & QM_DEVERR_TIMEOUT) : 0u;
      for (int pi = ew; pi < tab.n; pi += kEpiWarps) {
        const KernelArgs& a = tab.p[pi].a;
        double s5[5] = {0, 0, 0, 0, 0};
        for (int i = lane; i < (int)gridDim.x; i += 32) {
          const double* rec = a.partials + (int64_t)i * kPartialDoubles;
          s5[0] += __ldcg(rec); s5[1] = fmax(s5[1], __ldcg(rec + 1)); s5[2] += __ldcg(rec + 2);
          s5[3] += __ldcg(rec + 3); s5[4] += __ldcg(rec + 4);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          s5[0] += __shfl_xor_sync(0xffffffffu, s5[0], o);
          s5[1] = fmax(s5[1], __shfl_xor_sync(0xffffffffu, s5[1], o));
          s5[2] += __shfl_xor_sync(0xffffffffu, s5[2], o);
          s5[3] += __shfl_xor_sync(0xffffffffu, s5[3], o);
          s5[4] += __shfl_xor_sync(0xffffffffu, s5[4], o);
        }
        if (lane == 0) {
          a.result->sum_be = s5[0]; a.result->max_be = s5[1]; a.result->sum_diff2 = s5[2];
          a.result->sum_ref2 = s5[3]; a.result->sum_den2 = s5[4];
          a.result->count = a.count;
          uint32_t flags = (a.err_word ? *reinterpret_cast<volatile uint32_t*>(a.err_word) : 0u) | timed_out;
          for (int k = 0; k < 2; ++k)
            if (a.err_also[k]) flags |= *reinterpret_cast<const volatile uint32_t*>(a.err_also[k]);
          a.result->device_error = flags;
          a.result->reserved = 0;
        }
      }
    }
  }

  // ---------------------------------------------------------------- common exit
  // Neither CTA may leave while the other can still read its shared memory, signal its barriers
  // or write its tensor memory, and no bulk load may still be writing into a CTA that retires.
  tc_fence_before();
  __syncthreads();
  if (sh->abort_flag && threadIdx.x == 0) {
    // give-up path: the loads of the last kStages k-blocks this producer issued may not have been
    // awaited by anyone; wait (bounded) until each has landed
    const uint32_t n = sh->issued;
    for (uint32_t j = n > (uint32_t)kStages ? n - kStages : 0u; j < n; ++j) {
      const uint32_t bar = smem_u32(&sh->full[j % kStages]), parity = (j / kStages) & 1;
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(bar, parity) && global_timer_ns() - t0 < tab.wait_limit_ns) {}
    }
  }
  if (sh->abort_flag && warp == 1 && rank == 0) {
    // ... and the MMAs issued so far may still be running: one more commit, awaited (bounded) here
    __syncwarp();
    if (elect_one())
      asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                       smem_u32(&sh->drain)) : "memory");
    __syncwarp();
    const uint64_t t0 = global_timer_ns();
    while (!mbar_try_wait(smem_u32(&sh->drain), 0) && global_timer_ns() - t0 < tab.wait_limit_ns) {}
    __syncwarp();
  }
  __syncthreads();
  __syncwarp();
  cluster_sync();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
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

// Tensor map over [batch][rows][K] with the contracting index contiguous; box = 64 x box_rows x 1,
// swizzle span = row width of the box (128 bytes for bf16, 64 bytes for codes).
// wide: 128-byte boxes and swizzle for the codes as well (the 256 x 256 tile kernel).
bool make_map(CUtensorMap* m, const void* base, bool bf16, int box_rows, int64_t K, int64_t rows, int64_t batch,
              int64_t ld_elems, int64_t sb_elems, bool wide = false) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const uint64_t es = bf16 ? 2 : 1;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t sb = batch > 1 ? (cuuint64_t)sb_elems * es : (cuuint64_t)rows * ld_elems * es;
  cuuint64_t strides[2] = {(cuuint64_t)ld_elems * es, sb};
  cuuint32_t box[3] = {(cuuint32_t)((wide && !bf16) ? 2 * kBlockK : kBlockK), (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  (bf16 || wide) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

uint32_t lp_idesc(int fmt_l, int fmt_r, int n = kBlockN) {
  if (fmt_l == QM_FMT_INT8) return make_idesc(2, 1, 1, kPairM, n);                 // s8 x s8 -> s32
  const uint32_t fa = fmt_l == QM_FMT_E4M3 ? 0u : 1u, fb = fmt_r == QM_FMT_E4M3 ? 0u : 1u;
  return make_idesc(1, fa, fb, kPairM, n);                                         // fp8 x fp8 -> f32
}

template <int MODE>
size_t smem_bytes() {
  return (size_t)Cfg<MODE>::kStages * Cfg<MODE>::kStageBytes + sizeof(Shared) + 1024;
}

int64_t tile_count(GemmShape g) {
  return ((g.M + kPairM - 1) / kPairM) * ((g.N + kBlockN - 1) / kBlockN) * g.batch;
}

bool shape_ok(GemmShape g) {
  if (!(g.M > 0 && g.N > 0 && g.K > 0 && g.batch > 0 && (g.K % 16) == 0)) return false;
  // row, column and contraction indices of a tile's far edge are formed in 32-bit integers
  constexpr int64_t kLimit = (1ll << 31) - 1024;
  if (g.M >= kLimit || g.N >= kLimit || g.K >= kLimit || g.batch >= (1ll << 31)) return false;
  return tile_count(g) < (1ll << 31);
}

void fill_tiles(KernelArgs* ka, GemmShape g) {
  ka->M = g.M; ka->N = g.N; ka->K = g.K;
  ka->tiles_m = (int32_t)((g.M + kPairM - 1) / kPairM);
  ka->tiles_n = (int32_t)((g.N + kBlockN - 1) / kBlockN);
  ka->num_tiles = (int32_t)tile_count(g);
}

// CTA pairs that can be resident at once (one per TPC unless the device says fewer).
int g_max_pairs[kMaxDevices] = {};     // per device; 0 = not yet queried
int max_pairs() {
  const int dev = current_device();
  return dev >= 0 && g_max_pairs[dev] > 0 ? g_max_pairs[dev] : sm_count() / 2;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device.
template <typename K>
qm_status allow_smem(K kern, size_t bytes, bool (&done)[kMaxDevices]) {
  const int dev = current_device();
  if (dev < 0) return QM_ERR_UNSUPPORTED;
  if (!done[dev]) {
    QM_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    done[dev] = true;
  }
  return QM_OK;
}

// CTAs to launch: two per tile, at most the resident number of pairs.
int grid_size(GemmShape g) {
  const int64_t tiles = tile_count(g);
  const int pairs = max_pairs();
  return 2 * (int)(tiles < pairs ? tiles : pairs);
}

// maps: eight tensor maps (L, R, |L|, |R|, codes L, codes R, second-format codes L, R).
template <int MODE, int LPKIND, int LPKIND2 = LPKIND>
qm_status launch(const CUtensorMap* maps, const KernelArgs& ka, GemmShape g, cudaStream_t s) {
  auto kern = tc_kernel<MODE, LPKIND, LPKIND2>;
  static bool attr_done[kMaxDevices] = {};     // per instantiation
  const qm_status as = allow_smem(kern, smem_bytes<MODE>(), attr_done);
  if (as != QM_OK) return as;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid_size(g));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem_bytes<MODE>();
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see pdl_prologue()
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (MODE == kProbe2) profile_events(&ev0, &ev1);
  if (ev0) QM_CUDA_OK(cudaEventRecord(ev0, s));
  QM_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], maps[6], maps[7],
                                ka));
  if (ev1) QM_CUDA_OK(cudaEventRecord(ev1, s));
  count_launch();
  return QM_OK;
}

// The 256 x 256 tile kernel: worth it once the output is at least one such tile wide.
bool use_wide(GemmShape g) { return g.N >= kWideN; }

template <int KIND>
qm_status launch_wide(const CUtensorMap& ma, const CUtensorMap& mb, KernelArgs ka, GemmShape g, cudaStream_t s) {
  auto kern = tc_gemm_wide_kernel<KIND>;
  constexpr size_t smem = (size_t)kWideStages * kWideStageBytes + sizeof(SharedWide) + 1024;
  static bool attr_done[kMaxDevices] = {};
  const qm_status as = allow_smem(kern, smem, attr_done);
  if (as != QM_OK) return as;
  ka.tiles_m = (int32_t)((g.M + kPairM - 1) / kPairM);
  ka.tiles_n = (int32_t)((g.N + kWideN - 1) / kWideN);
  const int64_t tiles = (int64_t)ka.tiles_m * ka.tiles_n * g.batch;
  if (tiles >= (1ll << 31)) return QM_ERR_UNSUPPORTED;
  ka.num_tiles = (int32_t)tiles;
  const int pairs = max_pairs();
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * (tiles < pairs ? tiles : pairs)));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  QM_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, ma, mb, ka));
  count_launch();
  return QM_OK;
}

}  // namespace

int tc_group_max() { return kMaxGroup; }

namespace {
constexpr size_t kProbeSmem = (size_t)CfgP::kTileBytes + sizeof(SharedP) + 1024;

// Bound of the fused kernels' barrier waits and the producer's test hook (see qm_debug_* in qm.h).
std::atomic<uint64_t> g_wait_limit_ns{1000000000ull};
std::atomic<uint32_t> g_stop_after_kb{0xffffffffu};

// CTA pairs of the fused probe kernel that can be resident at once (its footprint is the largest
// of all modes, so its residency bounds every grid); queried once per device.
qm_status probe_residency() {
  const int dev = current_device();
  if (dev < 0) return QM_ERR_UNSUPPORTED;
  static bool attr_done[kMaxDevices] = {};
  const qm_status as = allow_smem(tc_group_kernel, kProbeSmem, attr_done);
  if (as != QM_OK) return as;
  if (g_max_pairs[dev] == 0) {
    // the kernel re-divides the registers its block was launched with (setmaxnreg): refuse to
    // launch if the compiler gave it fewer than the split adds up to, because an increase that
    // cannot be served waits forever
    cudaFuncAttributes fa{};
    QM_CUDA_OK(cudaFuncGetAttributes(&fa, tc_group_kernel));
    if (fa.numRegs * 4 < kRegsCtl + kRegsConv + 2 * kRegsEpi) return QM_ERR_UNSUPPORTED;
    cudaLaunchConfig_t q{};
    q.gridDim = dim3((unsigned)(2 * (sm_count() / 2))); q.blockDim = dim3(kProbeThreads);
    q.dynamicSmemBytes = kProbeSmem;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
    q.attrs = qa; q.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_group_kernel, &q) == cudaSuccess && n > 0)
      g_max_pairs[dev] = n < sm_count() / 2 ? n : sm_count() / 2;
    else
      g_max_pairs[dev] = sm_count() / 2;
    (void)cudaGetLastError();
  }
  return QM_OK;
}
}  // namespace

void set_wait_limit_ns(uint64_t ns) { g_wait_limit_ns.store(ns ? ns : 1000000000ull); }
void set_stop_after_kb(uint32_t kb) { g_stop_after_kb.store(kb); }

qm_status launch_tc_probe_group(const TcProbeArgs* ps, int n, cudaStream_t s) {
  if (n < 1 || n > kMaxGroup) return QM_ERR_INVALID_ARG;
  // descending contraction length = descending tile cost
  int order[kMaxGroup];
  for (int i = 0; i < n; ++i) order[i] = i;
  for (int i = 1; i < n; ++i)
    for (int j = i; j > 0 && ps[order[j]].g.K > ps[order[j - 1]].g.K; --j) {
      const int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t;
    }
  static GroupTable tab;               // 11 KB: kept off the stack; guarded by the mutex below
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  tab.n = n;
  tab.wait_limit_ns = g_wait_limit_ns.load();
  tab.stop_after_kb = g_stop_after_kb.load();
  int64_t total = 0;
  for (int k = 0; k < n; ++k) {
    const TcProbeArgs& p = ps[order[k]];
    if (!shape_ok(p.g) || p.cl2) return QM_ERR_UNSUPPORTED;
    const GemmShape g = p.g;
    const int64_t ldc = qm_code_ld(g.K);
    GroupProblem& gp = tab.p[k];
    // outputs at most 64 wide (the context and score-gradient products of attention): MMAs of N = 64,
    // half as many right-operand rows staged
    const int half_n = g.N <= 64 ? 32 : kHalfN;
    const bool ok = make_map(&gp.maps[0], p.l, true, kBlockM, g.K, g.M, g.batch, p.l_ld, p.l_sb) &&
                    make_map(&gp.maps[1], p.r, true, half_n, g.K, g.N, g.batch, p.r_ld, p.r_sb) &&
                    make_map(&gp.maps[2], p.cl, false, kBlockM, g.K, g.M, g.batch, ldc, g.M * ldc) &&
                    make_map(&gp.maps[3], p.cr, false, half_n, g.K, g.N, g.batch, ldc, g.N * ldc);
    if (!ok) return QM_ERR_CUDA;
    KernelArgs ka{};
    fill_tiles(&ka, g);
    ka.dl = p.dl; ka.pc_l = p.gran_l == QM_GRAN_CHANNEL; ka.dr = p.dr; ka.pc_r = p.gran_r == QM_GRAN_CHANNEL;
    ka.partials = p.partials; ka.done_counter = p.done_counter; ka.result = p.result;
    ka.count = (uint64_t)(g.M * g.N * g.batch);
    ka.err_word = p.err_word; ka.idesc_lp = lp_idesc(p.fmt_l, p.fmt_r, 2 * half_n);
    ka.row_stats = p.row_stats;
    ka.err_also[0] = p.err_also[0]; ka.err_also[1] = p.err_also[1];
    gp.a = ka;
    gp.half_n = half_n;
    // Tiles that run at the same time should share the LARGER operand's blocks, so that it is
    // streamed from HBM once and the smaller one is what gets fetched again (from L2, if it fits):
    // the tiles of a batch element are walked along the shorter side first.
    gp.m_fastest = g.M < g.N ? 1 : 0;
    gp.idesc_ref = make_idesc(1, 1, 1, kPairM, 2 * half_n);
    gp.kind = p.fmt_l == QM_FMT_INT8 ? kKindI8 : kKindF8;
    gp.tile_begin = (int32_t)total;
    total += ka.num_tiles;
    if (total >= (1ll << 31)) return QM_ERR_UNSUPPORTED;
  }
  tab.total_tiles = (int32_t)total;
  const qm_status rs = probe_residency();
  if (rs != QM_OK) return rs;
  const int pairs = max_pairs();
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * (total < pairs ? total : pairs)));
  cfg.blockDim = dim3(kProbeThreads);
  cfg.dynamicSmemBytes = kProbeSmem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  profile_events(&ev0, &ev1);
  if (ev0) QM_CUDA_OK(cudaEventRecord(ev0, s));
  QM_CUDA_OK(cudaLaunchKernelEx(&cfg, tc_group_kernel, tab));
  if (ev1) QM_CUDA_OK(cudaEventRecord(ev1, s));
  count_launch();
  return QM_OK;
}

// per format; a launch writes one record per CTA of its grid
int tc_probe_records(GemmShape) {
  (void)probe_residency();
  return 2 * max_pairs();
}

qm_status launch_tc_probe(const TcProbeArgs& p, cudaStream_t s) {
  if (!p.cl2) return launch_tc_probe_group(&p, 1, s);       // one format: a group of one
  if (!shape_ok(p.g)) return QM_ERR_UNSUPPORTED;
  const qm_status rs = probe_residency();
  if (rs != QM_OK) return rs;
  const GemmShape g = p.g;
  const int64_t ldc = qm_code_ld(g.K);
  CUtensorMap maps[8];
  bool ok = make_map(&maps[0], p.l, true, kBlockM, g.K, g.M, g.batch, p.l_ld, p.l_sb) &&
            make_map(&maps[1], p.r, true, kHalfN, g.K, g.N, g.batch, p.r_ld, p.r_sb) &&
            make_map(&maps[2], p.l_abs, true, kBlockM, g.K, g.M, g.batch, g.K, g.M * g.K) &&
            make_map(&maps[3], p.r_abs, true, kHalfN, g.K, g.N, g.batch, g.K, g.N * g.K) &&
            make_map(&maps[4], p.cl, false, kBlockM, g.K, g.M, g.batch, ldc, g.M * ldc) &&
            make_map(&maps[5], p.cr, false, kHalfN, g.K, g.N, g.batch, ldc, g.N * ldc) &&
            make_map(&maps[6], p.cl2, false, kBlockM, g.K, g.M, g.batch, ldc, g.M * ldc) &&
            make_map(&maps[7], p.cr2, false, kHalfN, g.K, g.N, g.batch, ldc, g.N * ldc);
  if (!ok) return QM_ERR_CUDA;
  KernelArgs ka{};
  fill_tiles(&ka, g);
  ka.dl = p.dl; ka.pc_l = p.gran_l == QM_GRAN_CHANNEL; ka.dr = p.dr; ka.pc_r = p.gran_r == QM_GRAN_CHANNEL;
  ka.partials = p.partials; ka.done_counter = p.done_counter; ka.result = p.result;
  ka.count = (uint64_t)(g.M * g.N * g.batch);
  ka.err_word = p.err_word; ka.idesc_lp = lp_idesc(p.fmt_l, p.fmt_r);
  // the first format is an FP8 one (the caller orders them), the second FP8 or INT8
  if (p.fmt_l == QM_FMT_INT8) return QM_ERR_UNSUPPORTED;
  ka.dl2 = p.dl2; ka.dr2 = p.dr2; ka.idesc_lp2 = lp_idesc(p.fmt_l2, p.fmt_r2);
  return p.fmt_l2 == QM_FMT_INT8 ? launch<kProbe2, kKindF8, kKindI8>(maps, ka, g, s)
                                 : launch<kProbe2, kKindF8, kKindF8>(maps, ka, g, s);
}

qm_status launch_tc_gemm_lp(const uint8_t* cl, int fmt_l, const float* dl, int gran_l,
                            const uint8_t* cr, int fmt_r, const float* dr, int gran_r, GemmShape g,
                            float* out_descaled, void* out_raw, uint32_t* err_word, cudaStream_t s) {
  if (!shape_ok(g)) return QM_ERR_UNSUPPORTED;
  const int64_t ldc = qm_code_ld(g.K);
  CUtensorMap maps[8];
  if (use_wide(g)) {
    if (!make_map(&maps[0], cl, false, kBlockM, g.K, g.M, g.batch, ldc, g.M * ldc, true) ||
        !make_map(&maps[1], cr, false, kWideHalfN, g.K, g.N, g.batch, ldc, g.N * ldc, true))
      return QM_ERR_CUDA;
    KernelArgs kw{};
    kw.M = g.M; kw.N = g.N; kw.K = g.K;
    kw.dl = dl; kw.pc_l = gran_l == QM_GRAN_CHANNEL; kw.dr = dr; kw.pc_r = gran_r == QM_GRAN_CHANNEL;
    kw.out_descaled = out_descaled; kw.out_raw = out_raw; kw.err_word = err_word;
    const uint32_t fa = fmt_l == QM_FMT_E4M3 ? 0u : 1u, fb = fmt_r == QM_FMT_E4M3 ? 0u : 1u;
    kw.idesc_lp = fmt_l == QM_FMT_INT8 ? make_idesc(2, 1, 1, kPairM, kWideN) : make_idesc(1, fa, fb, kPairM, kWideN);
    return fmt_l == QM_FMT_INT8 ? launch_wide<kKindI8>(maps[0], maps[1], kw, g, s)
                                : launch_wide<kKindF8>(maps[0], maps[1], kw, g, s);
  }
  bool ok = make_map(&maps[4], cl, false, kBlockM, g.K, g.M, g.batch, ldc, g.M * ldc) &&
            make_map(&maps[5], cr, false, kHalfN, g.K, g.N, g.batch, ldc, g.N * ldc);
  if (!ok) return QM_ERR_CUDA;
  maps[0] = maps[1] = maps[2] = maps[3] = maps[6] = maps[7] = maps[4];
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
  CUtensorMap maps[8];
  if (use_wide(g)) {
    if (!make_map(&maps[0], l, true, kBlockM, g.K, g.M, g.batch, g.K, g.M * g.K, true) ||
        !make_map(&maps[1], r, true, kWideHalfN, g.K, g.N, g.batch, g.K, g.N * g.K, true))
      return QM_ERR_CUDA;
    KernelArgs kw{};
    kw.M = g.M; kw.N = g.N; kw.K = g.K;
    kw.out_descaled = out; kw.err_word = err_word;
    return launch_wide<kKindF16>(maps[0], maps[1], kw, g, s);
  }
  bool ok = make_map(&maps[0], l, true, kBlockM, g.K, g.M, g.batch, g.K, g.M * g.K) &&
            make_map(&maps[1], r, true, kHalfN, g.K, g.N, g.batch, g.K, g.N * g.K);
  if (!ok) return QM_ERR_CUDA;
  maps[2] = maps[3] = maps[4] = maps[5] = maps[6] = maps[7] = maps[0];
  KernelArgs ka{};
  fill_tiles(&ka, g);
  ka.out_descaled = out; ka.err_word = err_word;
  return launch<kRefOnly, kKindF8>(maps, ka, g, s);
}

}  // namespace qm
