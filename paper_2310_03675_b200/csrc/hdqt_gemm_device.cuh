// Device-side building blocks of the tiled integer GEMM kernels: tile constants, kernel parameters, PTX
// wrappers (mbarrier, TMA, tcgen05), and the epilogue of one output block (accumulator quantisation, packed
// 16-bit-lane sums, staged stores).  Included by hdqt_gemm.cu only (one translation unit).
#pragma once

#include <cuda.h>

#include "hdqt_common.cuh"

namespace hdqt {

namespace {


constexpr int BM = 128;          // output rows per CTA (= TMEM lanes)
constexpr int BN = 256;          // output columns per CTA (= one MMA's N)
constexpr int BKB = 128;         // bytes of K per stage row (one 128B swizzle atom = 4 tiles of 32)
constexpr int STAGES = 4;
constexpr int A_STAGE = BM * BKB;              // 16 KB
constexpr int B_STAGE = BN * BKB;              // 32 KB
constexpr int STAGE_BYTES = A_STAGE + B_STAGE; // 48 KB
constexpr int NUM_EPI_WARPS = 8;               // 2 per TMEM lane quarter, 128 accumulator columns each
constexpr int EPI_COLS = BN / (NUM_EPI_WARPS / 4);
constexpr int NUM_CTRL_WARPS = 4;   // warp group 0: TMA producer, MMA issuer, certificate builder, one spare
constexpr int GEMM_THREADS = 32 * (NUM_CTRL_WARPS + NUM_EPI_WARPS);
// Register split between the warp groups (setmaxnreg): the kernel is compiled for 168 registers per thread
// (384 threads), the control warps give most of theirs back and the epilogue warps take them:
// 128 * 72 + 256 * 216 = 384 * 168.
constexpr int CTRL_REGS = 72;
constexpr int EPI_REGS = 216;
constexpr int TMEM_COLS = 512;
constexpr int MAX_CERT_WORDS = 256;            // certificate bitmask: up to 8192 accumulator tiles
constexpr int OUT_STAGE_WARP = 32 * 16 * 4;    // per epilogue warp: a 32-row x 16-column fp32 box for the store transpose
constexpr int TILE_INFO_BYTES = 4 * MAX_CERT_WORDS + 16;
// the dynamic shared-memory window is declared 1024-byte aligned (checked in the kernel), so no slack is kept
// offset of the store boxes (128-byte aligned)
constexpr int OUT_STAGE_OFF = (STAGES * STAGE_BYTES + 256 /*barriers*/ + 2 * TILE_INFO_BYTES + 127) / 128 * 128;
// constant operand tiles of the offset MMA (see epilogue_packed): no swizzle, 8-row groups 256 bytes apart,
// the two 16-byte K chunks of a row group 128 bytes apart
constexpr int OFFS_A_OFF = OUT_STAGE_OFF + NUM_EPI_WARPS * OUT_STAGE_WARP;
constexpr int OFFS_A_BYTES = (BM / 8) * 256;   // 4 KB
constexpr int OFFS_B_OFF = OFFS_A_OFF + OFFS_A_BYTES;
constexpr int OFFS_B_BYTES = (BN / 8) * 256;   // 8 KB
constexpr int SMEM_BYTES = OFFS_B_OFF + OFFS_B_BYTES;
static_assert(OUT_STAGE_WARP % 128 == 0, "store boxes must stay 128-byte aligned");
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");

// instruction descriptor: D = s32, A = B = signed 8-bit, both K-major, N = 256, M = 128
constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                           ((uint32_t)(BM >> 4) << 24);

// Optional event timeline for kernel tuning (compiled in only with -DHDQT_TIMELINE): block 0 records the
// SM clock at a few points of its first 64 accumulator tiles into a device array that
// hdqt_debug_timeline copies out.  Slots: 0 MMA issuer got the accumulator, 1 MMA issuer committed the tile,
// 2 epilogue saw the tile, 4 accumulator released, 5 tile added up (first epilogue warp); 8..15 release time
// of each epilogue warp.
#ifndef HDQT_TL_Q
#define HDQT_TL_Q 0   // lane quarter of the epilogue warp whose events are recorded
#endif
#ifdef HDQT_TIMELINE
__device__ long long g_timeline[64 * 16];
#define HDQT_TL(slot, idx)                                                                            \
  do {                                                                                                \
    if (blockIdx.x == 0 && (idx) < 64) g_timeline[(idx) * 16 + (slot)] = clock64();                   \
  } while (0)
#else
#define HDQT_TL(slot, idx) do { } while (0)
#endif

struct GemmParams {
  int64_t M, N, K_pad;
  int32_t tiles32;        // K_pad / 32
  int32_t tiles_per_acc;  // acc_tile / 32 (tiles32 if acc_tile == 0)
  int32_t num_acc;        // accumulator tiles along K
  int32_t acc_shift;
  int32_t lo, hi;         // accumulator range
  int32_t had_block;
  int32_t flush_every;    // packed mode: accumulator tiles summed in 16-bit lanes before widening
  int32_t offset_mma;     // packed mode: every clamp-path accumulator tile starts from the constant 2^(b_a-1)
  const float* bias;      // optional fp32 [N]: added to the dequantised output (one fp32 add per element)
  int32_t relu;           // != 0: max(., 0) after the bias
  int32_t split_k;        // > 1: the contraction of every output block is cut into this many work items
  int32_t split_kblocks;  // shared-memory stages (4 tiles of 32) per work item
  // merging of provably clamp-free accumulator tiles
  int32_t merge;          // 0 = off, 1 = certificates from the tile norms, 2 = every tile is clamp-free
  int32_t merge_max_uncert_256;  // a CTA merges only if uncertified tiles <= this/256 of all tiles
  int64_t cert_thr_sq;    // a 32-wide sub-tile is certified iff norm_a*norm_b <= this
  const int32_t* norms_a; // [ceil(M/128), tiles32]
  const int32_t* norms_b; // [ceil(N/128), tiles32]
  const float* step_a;
  const float* step_b;
  float* out;
  int64_t ld_out;
  int32_t* S_out;
  void* tiles_out;
  int32_t tiles_elem_bytes;
  int32_t* dev_status;
  // optional work list (device): when set, the kernel processes block_count[0] output blocks whose ids
  // (row block * column blocks + column block) are in block_list, instead of all blocks
  const int32_t* block_list;
  const int32_t* block_count;
};

// ---- PTX wrappers ---------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded waits: each gives up after ~1 s, or as soon as another role has given up.
//
// mbar_wait: for the two single-thread roles (TMA producer, MMA issuer), whose waits are on the
// critical path of every K tile: polls without suspending first, then backs off.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int slow_polls = 1 << 20) {
  for (int i = 0; i < (1 << 12); ++i) {
    if (mbar_test_wait(bar, parity)) return true;
  }
  for (int i = 0; i < slow_polls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    __nanosleep(512);
  }
  *abort_flag = 1;
  return false;
}

// mbar_wait_suspend: for waits that are usually long (the TMA producer far ahead of the MMAs, the MMA issuer
// behind a slower epilogue): try_wait parks the thread in hardware until the phase completes or a short time
// limit passes, so the waiting warp takes no issue slots from the warps of its scheduler that have work.
__device__ __forceinline__ bool mbar_wait_suspend(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  long long limit_clk = 2000000000ll) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - start > limit_clk) break;
  }
  *abort_flag = 1;
  return false;
}
// mbar_wait_yield: for the epilogue warps. A warp that spins steals issue slots from the MMA issuer
// and from the warps that have work, so these waits suspend in hardware (try_wait) and sleep between
// polls; kSleepNs is the poll period (short for the per-tile handshake, long for the one wait on the
// merged accumulator that spans the whole main loop).
template <int kSleepNs>
__device__ __forceinline__ bool mbar_wait_yield(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                int polls = (kSleepNs >= 512) ? (1 << 21) : (1 << 24)) {
  if (mbar_try_wait(bar, parity)) return true;
  for (int i = 0; i < polls; ++i) {
    __nanosleep(kSleepNs);
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63) == 63 && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

template <int kRegs>
__device__ __forceinline__ void warpgroup_reg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegs));
}
template <int kRegs>
__device__ __forceinline__ void warpgroup_reg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegs));
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC), "r"(accumulate)
      : "memory");
}

// the two forms an issue loop needs, with the accumulate flag fixed at compile time (no predicate set-up)
__device__ __forceinline__ void tc_mma_i8_new(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC)
      : "memory");
}
__device__ __forceinline__ void tc_mma_i8_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.eq.b32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(IDESC)
      : "memory");
}

// K-major operand tile with 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                         // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // SWIZZLE_128B
  return d;
}

// K-major operand tile without swizzle: 8 rows x 16 bytes are contiguous (128 bytes); `lbo` = distance between
// the two 16-byte K chunks of a 32-byte K slice, `sbo` = distance between 8-row groups.
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}

#define HDQT_TMEM_LD32(taddr, v)                                                                        \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                         \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                         \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"         \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),      \
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),      \
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                           \
      : "r"(taddr)                                                                                      \
      : "memory")

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

#define HDQT_TMEM_LD32_PACK16(taddr, v)                                                                 \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x32.pack::16b.b32 "                                               \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                         \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"         \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),      \
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),      \
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                           \
      : "r"(taddr)                                                                                      \
      : "memory")

#define HDQT_TMEM_LD64_PACK16(taddr, v)                                                                 \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x64.pack::16b.b32 "                                               \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "                         \
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "                \
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "                \
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"         \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),      \
        "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),      \
        "=r"(v[29]), "=r"(v[30]), "=r"(v[31]), "=r"(v[32]), "=r"(v[33]), "=r"(v[34]), "=r"(v[35]),      \
        "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]), "=r"(v[40]), "=r"(v[41]), "=r"(v[42]),      \
        "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]), "=r"(v[48]), "=r"(v[49]),      \
        "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]), "=r"(v[56]),      \
        "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63])       \
      : "r"(taddr)                                                                                      \
      : "memory")

#define HDQT_TMEM_LD16_PACK16(taddr, v)                                                                 \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x16.pack::16b.b32 "                                               \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"                  \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15])                                                                                     \
      : "r"(taddr)                                                                                      \
      : "memory")

// tcgen05.wait::ld tied to the registers of the load it completes, so that the compiler cannot move
// their first use above the wait
#define HDQT_TMEM_WAIT16(v)                                                                             \
  asm volatile("tcgen05.wait::ld.sync.aligned;"                                                         \
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]),    \
                 "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), \
                 "+r"(v[14]), "+r"(v[15])                                                               \
               :                                                                                        \
               : "memory")

#define HDQT_TMEM_WAIT32(v)                                                                             \
  asm volatile("tcgen05.wait::ld.sync.aligned;"                                                         \
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]),    \
                 "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), \
                 "+r"(v[14]), "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]),          \
                 "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]),          \
                 "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])           \
               :                                                                                        \
               : "memory")

#define HDQT_TMEM_LD16(taddr, v)                                                                        \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                         \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"                  \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15])                                                                                     \
      : "r"(taddr)                                                                                      \
      : "memory")

// packed (two columns per register) load of half of a warp's columns, and the matching wait
#define HDQT_LD_HALF_PACK(taddr, v)                                    \
  do {                                                                 \
    if constexpr (EPI_COLS / 4 == 32) { HDQT_TMEM_LD32_PACK16(taddr, v); } \
    else { HDQT_TMEM_LD16_PACK16(taddr, v); }                          \
  } while (0)
#define HDQT_WAIT_HALF(v)                                              \
  do {                                                                 \
    if constexpr (EPI_COLS / 4 == 32) { HDQT_TMEM_WAIT32(v); }         \
    else { HDQT_TMEM_WAIT16(v); }                                      \
  } while (0)

// accumulator quantisation of one exact tile sum
template <bool kShift>
__device__ __forceinline__ int acc_quant(int P, int r, int lo, int hi) {
  if (kShift) {
    // round-half-even of P / 2^r:  (P + (2^(r-1) - 1) + ((P >> r) & 1)) >> r
    P = (P + ((1 << (r - 1)) - 1) + ((P >> r) & 1)) >> r;
  }
  return min(max(P, lo), hi);
}

// The fp32 tail of the dequantising epilogue (outside the quantized path: Section 3 quantizes the matmul's inputs
// and accumulators only): optional bias of the output column, optional ReLU.
__device__ __forceinline__ float finish1(const GemmParams& p, float x, int64_t n) {
  if (p.bias != nullptr) x = __fadd_rn(x, __ldg(p.bias + n));
  if (p.relu) x = fmaxf(x, 0.0f);
  return x;
}

// Writes 4 consecutive output columns of one row: the final fp32 values (and optionally the integer
// sums), or - for an intermediate widening of the packed sums - the int32 partial sums, which are
// parked in the output buffer itself until the final pass reads them back.
template <bool kFinal>
__device__ __forceinline__ void emit4(const GemmParams& p, int64_t gm, int64_t gn, int (&s)[4], bool have_prev,
                                      bool vec, float scale) {
  float* orow = p.out + gm * p.ld_out + gn;
  if (vec) {
    if (have_prev) {
      const int4 prev = *reinterpret_cast<const int4*>(orow);
      s[0] += prev.x; s[1] += prev.y; s[2] += prev.z; s[3] += prev.w;
    }
    if (kFinal) {
      float4 o;
      o.x = finish1(p, __fmul_rn((float)s[0], scale), gn);
      o.y = finish1(p, __fmul_rn((float)s[1], scale), gn + 1);
      o.z = finish1(p, __fmul_rn((float)s[2], scale), gn + 2);
      o.w = finish1(p, __fmul_rn((float)s[3], scale), gn + 3);
      *reinterpret_cast<float4*>(orow) = o;
    } else {
      *reinterpret_cast<int4*>(orow) = make_int4(s[0], s[1], s[2], s[3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (gn + i < p.N) {
        if (have_prev) s[i] += __float_as_int(orow[i]);
        orow[i] = kFinal ? finish1(p, __fmul_rn((float)s[i], scale), gn + i) : __int_as_float(s[i]);
      }
    }
  }
  if (kFinal && p.S_out != nullptr) {
    int32_t* srow = p.S_out + gm * p.N + gn;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (gn + i < p.N) srow[i] = s[i];
    }
  }
}

// ---- epilogue of one output block, as separate functions ---------------------------------------
// Each variant keeps its own register-resident state (sums, load buffers); keeping them out of the
// kernel body lets the compiler allocate registers per variant instead of for their union.

struct EpiCtx {               // constants of one epilogue warp
  uint32_t lane_addr;         // TMEM address of this warp's lane quarter and column group in accumulator 0
  uint32_t bar_tfull;         // [2] accumulator ready
  uint32_t bar_tempty;        // [2] accumulator drained
  volatile int* abort_flag;
  float* box;                 // this warp's 32 x 16 fp32 staging box in shared memory
  int q, grp, lane;
  float scale;                // dequantisation scale of the launch (formed once per warp, not per output block)
};

struct BlockJob {             // one output block as seen by the epilogue
  int m0 = 0, n0 = 0;
  int n_clamp_tiles = 0;      // accumulator tiles that arrive one by one for the clamp path
  int n_merged = 0;           // accumulator tiles merged in accumulator 0
  int merging = 0;            // clamp tiles use accumulator 1 only (else they alternate 0 / 1)
  int atomic = 0;             // split-K: add the integer sums into the output buffer instead of storing the result
};

__device__ __forceinline__ float dequant_scale(const GemmParams& p) {
  return (float)((double)__ldg(p.step_a) * (double)__ldg(p.step_b) * (double)(1u << p.acc_shift) /
                 (double)p.had_block);
}

// Final integer sums of columns [16c, 16c+16) of this thread's row -> fp32 output.
// Staged path: the warp's 32 x 16 block is transposed through a 2 KB shared-memory box so that every
// store instruction writes 8 rows x 64 contiguous bytes (whole sectors) instead of 32 rows x 16 bytes;
// stores are fire-and-forget, so the box can be reused as soon as the warp has read it back.
// raw = true parks the integer sums themselves (as bit patterns) for a later fix-up pass instead.
// kDirect: every thread stores its own row with 16-byte vector stores instead (no staging box, no warp syncs:
// less code and fewer registers around a long main loop; less efficient stores, so only where the final pass is
// rare: the long-contraction variant).
// kAtomic = false: the launch has no split-K work items; the atomic path is compiled out (the per-tile loops of the
// clamp path lost 12 % to its mere presence in the kernel's code).
template <bool kDirect = false, bool kAtomic = true>
__device__ __forceinline__ void store_chunk(const GemmParams& p, const EpiCtx& e, const BlockJob& job, int c,
                                            int (&val)[16], bool parked, float scale, bool raw = false) {
  const int64_t gm = (int64_t)job.m0 + e.q * 32 + e.lane;
  const int64_t gn = (int64_t)job.n0 + e.grp * EPI_COLS + c * 16;
  if (gn >= p.N) return;      // (warp-uniform) columns beyond the matrix: nothing to write
  if (kAtomic && job.atomic) {
    // split-K: integer partial sums of this K range (the buffer was cleared before the launch).  Through the box,
    // like the stores: a warp-wide atomic then covers 8 rows x 16 consecutive words (8 memory transactions)
    // instead of one word in each of 32 rows.
    if (gn + 16 <= p.N) {
      int4* dst = reinterpret_cast<int4*>(e.box + e.lane * 16);
      const int rot = (e.lane >> 1) & 3;
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[(i + rot) & 3] = make_int4(val[4 * i], val[4 * i + 1], val[4 * i + 2], val[4 * i + 3]);
      __syncwarp();
      const int sub = e.lane >> 2, quad = e.lane & 3;
#pragma unroll
      for (int rr = 0; rr < 32; rr += 8) {
        const int rloc = rr + sub;
        const int4 v = *reinterpret_cast<const int4*>(e.box + rloc * 16 + ((quad + ((rloc >> 1) & 3)) & 3) * 4);
        const int64_t grow = (int64_t)job.m0 + e.q * 32 + rloc;
        if (grow < p.M) {
          int* o = reinterpret_cast<int*>(p.out + grow * p.ld_out + gn + quad * 4);
          if (v.x != 0) atomicAdd(o, v.x);
          if (v.y != 0) atomicAdd(o + 1, v.y);
          if (v.z != 0) atomicAdd(o + 2, v.z);
          if (v.w != 0) atomicAdd(o + 3, v.w);
        }
      }
      __syncwarp();
    } else if (gm < p.M) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (gn + i < p.N && val[i] != 0) atomicAdd(reinterpret_cast<int*>(p.out + gm * p.ld_out + gn + i), val[i]);
      }
    }
    return;
  }
  const bool staged = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                      (gn + 16 <= p.N);    // warp-uniform
  if (kDirect && staged) {
    if (gm < p.M) {
#pragma unroll
      for (int i = 0; i < 16; i += 4) {
        int s4[4] = {val[i], val[i + 1], val[i + 2], val[i + 3]};
        if (raw) emit4<false>(p, gm, gn + i, s4, parked, true, scale);
        else emit4<true>(p, gm, gn + i, s4, parked, true, scale);
      }
    }
    return;
  }
  if (staged) {
    if (gm < p.M && (parked || (p.S_out != nullptr && !raw))) {
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (parked) val[i] += __float_as_int(p.out[gm * p.ld_out + gn + i]);
        if (p.S_out != nullptr && !raw) p.S_out[gm * p.N + gn + i] = val[i];
      }
    }
    // row r of the box starts at r*16 floats; the four float4 of a row are rotated by (r >> 1) & 3 so
    // that neither the row-wise writes nor the read-back hit a shared-memory bank twice
    float4* dst = reinterpret_cast<float4*>(e.box + e.lane * 16);
    const int rot = (e.lane >> 1) & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      dst[(i + rot) & 3] =
          raw ? make_float4(__int_as_float(val[4 * i]), __int_as_float(val[4 * i + 1]), __int_as_float(val[4 * i + 2]),
                            __int_as_float(val[4 * i + 3]))
              : make_float4(__fmul_rn((float)val[4 * i], scale), __fmul_rn((float)val[4 * i + 1], scale),
                            __fmul_rn((float)val[4 * i + 2], scale), __fmul_rn((float)val[4 * i + 3], scale));
    }
    __syncwarp();
    const int sub = e.lane >> 2, quad = e.lane & 3;       // 8 rows per instruction, 4 lanes per row
#pragma unroll
    for (int rr = 0; rr < 32; rr += 8) {
      const int rloc = rr + sub;
      float4 v = *reinterpret_cast<const float4*>(e.box + rloc * 16 + ((quad + ((rloc >> 1) & 3)) & 3) * 4);
      if (!raw && (p.bias != nullptr || p.relu)) {
        const int64_t n = gn + quad * 4;
        v.x = finish1(p, v.x, n); v.y = finish1(p, v.y, n + 1); v.z = finish1(p, v.z, n + 2); v.w = finish1(p, v.w, n + 3);
      }
      const int64_t grow = (int64_t)job.m0 + e.q * 32 + rloc;
      if (grow < p.M) *reinterpret_cast<float4*>(p.out + grow * p.ld_out + gn + quad * 4) = v;
    }
    __syncwarp();
  } else if (gm < p.M) {
#pragma unroll
    for (int i = 0; i < 16; i += 4) {
      int s4[4] = {val[i], val[i + 1], val[i + 2], val[i + 3]};
      if (raw) emit4<false>(p, gm, gn + i, s4, parked, false, scale);
      else emit4<true>(p, gm, gn + i, s4, parked, false, scale);
    }
  }
}

// The common case of the staged store with everything that does not depend on the column chunk formed once per
// output block: addresses of this lane's box slots and output rows, row predicates, the fp32 tail's flags.  A
// chunk is then ~70 instructions without a branch (the general store_chunk: ~200 with 27 branches, and the final
// pass of a block was bound by instruction fetch).  Usable for chunks that lie inside the matrix when the output
// is 16-byte aligned and nothing is parked, raw, atomic or wanted as integers.
struct FastStore {
  float* out0;                 // output address of this lane's first row group, first chunk
  int64_t row_step;            // 8 rows further
  uint32_t sts[4];             // shared-memory addresses of the four 16-byte slots this lane writes
  uint32_t lds[4];             // ... and of the four it reads back (one per row group)
  const float* bias0;          // bias of this lane's four columns in chunk 0, or null
  bool row_ok[4];
  bool relu;
  bool usable;
  int chunks_inside;           // chunks [0, chunks_inside) lie wholly inside the matrix
  bool ragged;                 // ... and one more lies partly inside
};

__device__ __forceinline__ FastStore make_fast_store(const GemmParams& p, const EpiCtx& e, const BlockJob& job,
                                                     bool parked) {
  FastStore f;
  const int64_t gn0 = (int64_t)job.n0 + e.grp * EPI_COLS;
  f.usable = !parked && !job.atomic && p.S_out == nullptr && ((p.ld_out & 3) == 0) &&
             ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && ((reinterpret_cast<uintptr_t>(p.bias) & 15) == 0);
  const int64_t left = p.N - gn0;
  f.chunks_inside = left <= 0 ? 0 : (left >= EPI_COLS ? EPI_COLS / 16 : (int)(left >> 4));
  f.ragged = left > 0 && left < EPI_COLS && (left & 15) != 0;
  const int sub = e.lane >> 2, quad = e.lane & 3;
  const int64_t row0 = (int64_t)job.m0 + e.q * 32 + sub;
  f.out0 = p.out + row0 * p.ld_out + gn0 + quad * 4;
  f.row_step = 8 * p.ld_out;
  const uint32_t box = smem_u32(e.box);
  const int rot = (e.lane >> 1) & 3;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f.sts[i] = box + (uint32_t)(e.lane * 64 + (((i + rot) & 3) << 4));
    const int rloc = 8 * i + sub;
    f.lds[i] = box + (uint32_t)(rloc * 64 + (((quad + ((rloc >> 1) & 3)) & 3) << 4));
    f.row_ok[i] = row0 + 8 * i < p.M;
  }
  f.bias0 = p.bias != nullptr ? p.bias + gn0 + quad * 4 : nullptr;
  f.relu = p.relu != 0;
  return f;
}

__device__ __forceinline__ void sts128(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}

// integer sums of columns [16c, 16c+16) of this thread's row -> fp32 output, chunk c inside the matrix
__device__ __forceinline__ void store_chunk_fast(const FastStore& f, int c, const int (&val)[16], float scale) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    sts128(f.sts[i], __fmul_rn((float)val[4 * i], scale), __fmul_rn((float)val[4 * i + 1], scale),
           __fmul_rn((float)val[4 * i + 2], scale), __fmul_rn((float)val[4 * i + 3], scale));
  }
  __syncwarp();
  float4 b4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  if (f.bias0 != nullptr) b4 = __ldg(reinterpret_cast<const float4*>(f.bias0 + c * 16));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float4 v = lds128(f.lds[i]);
    if (f.bias0 != nullptr) {
      v.x = __fadd_rn(v.x, b4.x); v.y = __fadd_rn(v.y, b4.y); v.z = __fadd_rn(v.z, b4.z); v.w = __fadd_rn(v.w, b4.w);
    }
    if (f.relu) { v.x = fmaxf(v.x, 0.0f); v.y = fmaxf(v.y, 0.0f); v.z = fmaxf(v.z, 0.0f); v.w = fmaxf(v.w, 0.0f); }
    if (f.row_ok[i]) *reinterpret_cast<float4*>(f.out0 + i * f.row_step + c * 16) = v;
  }
  __syncwarp();
}

// one elected lane arrives once the whole warp is here (elect.sync converges the warp; no divergent branch)
__device__ __forceinline__ void warp_arrive_one(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
      ::"r"(bar)
      : "memory");
}

__device__ __forceinline__ void release_accumulator(const EpiCtx& e, int buf, uint32_t& drain_par) {
  tc_fence_before();
  warp_arrive_one(e.bar_tempty + 8 * buf);
  drain_par ^= 1u << buf;
}

// Whole block merged (the common case on heavy-tailed operands): no per-tile sums exist, so the registers
// take the complete accumulator row at once and the accumulator goes back to the MMA issuer before any
// conversion or store work.
template <bool kDirect = false>
__device__ __forceinline__ bool epilogue_merged_only(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t& drain_par) {
  if (!mbar_wait_yield<64>(e.bar_tfull + 0, drain_par & 1u, e.abort_flag)) return false;
  tc_fence_after();
  const float scale = e.scale;
  uint32_t mv[EPI_COLS];
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_LD16(e.lane_addr + c * 16, (mv + c * 16));
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_WAIT16((mv + c * 16));
  release_accumulator(e, 0, drain_par);
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) {
    int val[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) val[i] = (int)mv[c * 16 + i];
    store_chunk<kDirect>(p, e, job, c, val, false, scale);
  }
  return true;
}

// 16-bit-lane path: tile sums fit int16, b_a <= 8, r = 0.
//
// Every clamp-path accumulator tile starts from the constant o = 2^(b_a-1) (the MMA issuer writes it with one
// MMA of constant operand tiles before the tile's data MMAs), so TMEM holds y = P + o, and the accumulator
// quantisation c = clamp(P, -o, o-1) becomes c + o = clamp(y, 0, 2^b_a - 1).  TMEM is read with two columns
// packed per register (low half = even column).  In range, y has no bit outside 2^b_a - 1, in either half:
// one OR-reduction over the warp's registers proves that no element of the tile clamps, and the registers are
// then added to the 16-bit lane sums as they are (one three-input logic operation per two registers and one
// add per register, instead of a clamp per register).  A tile with an element out of range takes the clamp
// instruction instead.  The sums stay unsigned 16-bit lanes (no carry can cross) and are widened through the
// output buffer every flush_every tiles; o times the tile count is subtracted when they are unpacked.
//
// The logic operations and adds are inline PTX on purpose: written in C++, the compiler pairs the 32-bit adds
// into two-element vector operations that cost two instructions each (measured: 3x the time).  Being volatile,
// they also stay behind the tcgen05.wait::ld that makes the registers valid.
__device__ __forceinline__ void packed_accumulate(uint32_t (&S)[EPI_COLS / 2], uint32_t (&v)[EPI_COLS / 2],
                                                  uint32_t rng2) {
  uint32_t any0 = 0u, any1 = 0u, any2 = 0u, any3 = 0u;    // four independent chains
#pragma unroll
  for (int i = 0; i < EPI_COLS / 2; i += 8) {
    asm volatile("lop3.b32 %0, %0, %1, %2, 0xFE;" : "+r"(any0) : "r"(v[i]), "r"(v[i + 1]));
    asm volatile("lop3.b32 %0, %0, %1, %2, 0xFE;" : "+r"(any1) : "r"(v[i + 2]), "r"(v[i + 3]));
    asm volatile("lop3.b32 %0, %0, %1, %2, 0xFE;" : "+r"(any2) : "r"(v[i + 4]), "r"(v[i + 5]));
    asm volatile("lop3.b32 %0, %0, %1, %2, 0xFE;" : "+r"(any3) : "r"(v[i + 6]), "r"(v[i + 7]));
  }
#pragma unroll
  for (int i = 0; i < EPI_COLS / 2; ++i) asm volatile("add.u32 %0, %0, %1;" : "+r"(S[i]) : "r"(v[i]));
  // Rare: some element of the warp's tile is out of range.  The plain add above may then have carried
  // between the two lanes of a register; taking the added value out again and putting the clamped one in is
  // exact all the same (32-bit wrap-around arithmetic).  Written as a loop over an opaque count (0 or 1) so
  // that the compiler emits a real, warp-uniform branch instead of predicating the clamps into the common path.
  int redo = __any_sync(0xFFFFFFFFu, (((any0 | any1) | (any2 | any3)) & ~rng2) != 0u) ? 1 : 0;
  asm volatile("" : "+r"(redo));
#pragma unroll 1
  for (int rep = 0; rep < redo; ++rep) {
#pragma unroll
    for (int i = 0; i < EPI_COLS / 2; ++i) S[i] += __viaddmin_s16x2_relu(v[i], 0u, rng2) - v[i];
  }
}

// kDeep (contractions of more than flush_every tiles, chosen by the host): a second set of 16-bit lanes takes the
// high bytes of the lane sums every flush_every tiles (sum = low + 256 * high), so that nothing is parked in memory
// for up to 256 * flush_every tiles; it costs 64 more registers, which is why it is a variant of its own.
template <bool kDeep, bool kMerge = true, bool kAtomic = true>
__device__ __forceinline__ bool epilogue_packed(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t& drain_par) {
  uint32_t S[EPI_COLS / 2];
  uint32_t Shi[kDeep ? EPI_COLS / 2 : 1];
#pragma unroll
  for (int i = 0; i < EPI_COLS / 2; ++i) S[i] = 0u;
#pragma unroll
  for (int i = 0; i < (kDeep ? EPI_COLS / 2 : 1); ++i) Shi[i] = 0u;
  int n_deep = 0;        // tiles whose high bytes have moved to Shi
  const uint32_t off = (uint32_t)(-p.lo);                    // c + off lies in [0, hi - lo]
  const uint32_t rng2 = (uint32_t)(p.hi - p.lo) | ((uint32_t)(p.hi - p.lo) << 16);
  int n_in_S = 0;
  bool parked = false;   // int32 partial sums are parked in the output buffer
  // One load of the warp's whole row segment (128 columns in 64 registers) per tile; the accumulator goes
  // back to the MMA issuer as soon as the load has landed, before any arithmetic.  (Arithmetic of a warp does
  // not overlap its own TMEM load in flight - measured: it gets slower -, so the load is not split or
  // prefetched; the other epilogue warp of the scheduler fills the load's latency.)
  // widen: park the int32 partial sums in the output buffer (added to what is parked there already)
  auto park_sums = [&]() {
    const int64_t gm = (int64_t)job.m0 + e.q * 32 + e.lane;
    const int64_t gn0 = (int64_t)job.n0 + e.grp * EPI_COLS;
    const bool vec = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                     (gn0 + EPI_COLS <= p.N);
    if (gm < p.M) {
#pragma unroll
      for (int i = 0; i < EPI_COLS / 2; i += 2) {
        int s4[4];
        s4[0] = (int)(S[i] & 0xFFFFu) - (int)off * n_in_S;
        s4[1] = (int)(S[i] >> 16) - (int)off * n_in_S;
        s4[2] = (int)(S[i + 1] & 0xFFFFu) - (int)off * n_in_S;
        s4[3] = (int)(S[i + 1] >> 16) - (int)off * n_in_S;
        emit4<false>(p, gm, gn0 + 2 * i, s4, parked, vec, 0.0f);
      }
    }
#pragma unroll
    for (int i = 0; i < EPI_COLS / 2; ++i) S[i] = 0u;
  };
  // Two nested loops: the widening step (rare, a lot of code) sits between runs of at most flush_every tiles,
  // outside the per-tile loop, so that the per-tile loop is one short stretch of code.
  for (int base = 0; base < job.n_clamp_tiles; base += p.flush_every) {
    const int run_end = min(job.n_clamp_tiles, base + p.flush_every);
    auto one_tile = [&](int ci, int buf) -> bool {
      const uint32_t par = buf ? (drain_par >> 1) : (drain_par & 1u);
      if (!mbar_wait_suspend(e.bar_tfull + 8 * buf, par & 1u, e.abort_flag)) return false;
      tc_fence_after();
      if (e.q == HDQT_TL_Q && e.grp == 0 && e.lane == 0) HDQT_TL(2, ci);
      uint32_t v[EPI_COLS / 2];
      HDQT_TMEM_LD64_PACK16(e.lane_addr + buf * BN, v);
      tmem_ld_wait();
      release_accumulator(e, buf, drain_par);
      if (e.q == HDQT_TL_Q && e.grp == 0 && e.lane == 0) HDQT_TL(4, ci);
      if (e.lane == 0) HDQT_TL(8 + e.grp * 4 + e.q, ci);      // release time of every epilogue warp
      packed_accumulate(S, v, rng2);
      if (e.q == HDQT_TL_Q && e.grp == 0 && e.lane == 0) HDQT_TL(5, ci);
      return true;
    };
    int ci = base;
    if (!(kMerge && job.merging) && (base & 1) == 0) {
      // tiles alternate between the two accumulators: pairs with the accumulator index fixed at compile time
      // (barrier and TMEM addresses then stay in uniform registers: 740 -> 876 TOPS at 8192^3; four per
      // iteration gave nothing more)
#pragma unroll 1
      for (; ci + 1 < run_end; ci += 2) {
        if (!one_tile(ci, 0)) return false;
        if (!one_tile(ci + 1, 1)) return false;
      }
    }
#pragma unroll 1
    for (; ci < run_end; ++ci) {
      if (!one_tile(ci, (kMerge && job.merging) ? 1 : (ci & 1))) return false;
    }
    n_in_S = run_end - base;
    if (run_end < job.n_clamp_tiles) {
      if constexpr (kDeep) {
#pragma unroll
        for (int i = 0; i < EPI_COLS / 2; ++i) {
          Shi[i] += (S[i] >> 8) & 0x00FF00FFu;
          S[i] &= 0x00FF00FFu;
        }
        n_deep += n_in_S;
      } else if constexpr (kMerge) {     // (the merge-free instantiations never get work items that long)
        park_sums();
        n_in_S = 0;
        parked = true;
      }
    }
  }
  if constexpr (kDeep) n_in_S += n_deep;     // every tile's offset is still in the two lane sets
  if (kMerge && job.n_merged > 0) {
    if (!mbar_wait_yield<64>(e.bar_tfull + 0, drain_par & 1u, e.abort_flag)) return false;
    tc_fence_after();
  }
  const FastStore fast = make_fast_store(p, e, job, parked);
  const float scale = e.scale;
  // the chunks of one output block, with the store routine chosen once for all of them (two separate stretches
  // of code: the common one stays compact)
  auto final_pass = [&]<bool kFast>() {
#pragma unroll
    for (int c = 0; c < EPI_COLS / 16; ++c) {
      uint32_t mv[16];
      if (kMerge && job.n_merged > 0) {   // uniform
        HDQT_TMEM_LD16(e.lane_addr + c * 16, mv);
        HDQT_TMEM_WAIT16(mv);
        // the last of the merged accumulator is in registers: hand it back to the MMA issuer
        if (c == EPI_COLS / 16 - 1) release_accumulator(e, 0, drain_par);
      }
      int val[16];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t sp = S[c * 8 + i];
        val[2 * i] = (int)(sp & 0xFFFFu) - (int)off * n_in_S;
        val[2 * i + 1] = (int)(sp >> 16) - (int)off * n_in_S;
        if constexpr (kDeep) {
          const uint32_t hp = Shi[c * 8 + i];
          val[2 * i] += (int)((hp & 0xFFFFu) << 8);
          val[2 * i + 1] += (int)((hp >> 16) << 8);
        }
        if (kMerge && job.n_merged > 0) {
          val[2 * i] += (int)mv[2 * i];
          val[2 * i + 1] += (int)mv[2 * i + 1];
        }
      }
      if constexpr (kFast) {
        if (c < fast.chunks_inside) store_chunk_fast(fast, c, val, scale);   // (the rest lies beyond the matrix)
      } else {
        store_chunk<kDeep, kAtomic>(p, e, job, c, val, parked, scale);
      }
    }
  };
  if (!kDeep && fast.usable && !fast.ragged) final_pass.template operator()<true>();
  else final_pass.template operator()<false>();
  return true;
}

// 32-bit path: one register per accumulator element, any b_a and shift r, optional per-tile debug output.
template <bool kShift, bool kTilesOut>
__device__ __forceinline__ bool epilogue_wide(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t& drain_par) {
  int S[EPI_COLS];
#pragma unroll
  for (int i = 0; i < EPI_COLS; ++i) S[i] = 0;
  const int r = p.acc_shift, lo = p.lo, hi = p.hi;
  for (int ci = 0; ci < job.n_clamp_tiles; ++ci) {
    const int buf = job.merging ? 1 : (ci & 1);
    if (!mbar_wait(e.bar_tfull + 8 * buf, (drain_par >> buf) & 1u, e.abort_flag)) return false;
    tc_fence_after();
#pragma unroll
    for (int c = 0; c < EPI_COLS / 16; ++c) {
      uint32_t v[16];
      HDQT_TMEM_LD16(e.lane_addr + buf * BN + c * 16, v);
      HDQT_TMEM_WAIT16(v);
      if (c == EPI_COLS / 16 - 1) release_accumulator(e, buf, drain_par);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int ct = acc_quant<kShift>((int)v[i], r, lo, hi);
        S[c * 16 + i] += ct;
        if (kTilesOut) {
          const int64_t gm = (int64_t)job.m0 + e.q * 32 + e.lane;
          const int64_t n = (int64_t)job.n0 + e.grp * EPI_COLS + c * 16 + i;
          if (gm < p.M && n < p.N) {
            const int64_t o = ((int64_t)ci * p.M + gm) * p.N + n;
            if (p.tiles_elem_bytes == 1) reinterpret_cast<int8_t*>(p.tiles_out)[o] = (int8_t)ct;
            else reinterpret_cast<int16_t*>(p.tiles_out)[o] = (int16_t)ct;
          }
        }
      }
    }
  }
  if (job.n_merged > 0) {
    if (!mbar_wait_yield<64>(e.bar_tfull + 0, drain_par & 1u, e.abort_flag)) return false;
    tc_fence_after();
  }
  const float scale = e.scale;
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) {
    int val[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) val[i] = S[c * 16 + i];
    if (job.n_merged > 0) {   // uniform
      uint32_t mv[16];
      HDQT_TMEM_LD16(e.lane_addr + c * 16, mv);
      HDQT_TMEM_WAIT16(mv);
      if (c == EPI_COLS / 16 - 1) release_accumulator(e, 0, drain_par);
#pragma unroll
      for (int i = 0; i < 16; ++i) val[i] += (int)mv[i];
    }
    store_chunk(p, e, job, c, val, false, scale);
  }
  return true;
}

}  // namespace

}  // namespace hdqt
