// Tiled integer GEMM with low-bit per-tile accumulators on the sm_100a tensor cores
// (paper Section 3, last paragraph: "tiled quantization ... tiles of size s"; Section 4:
// accumulator block size 32; Section 4.2: 8-bit accumulators in forward and backward pass).
//
//   P_t[m,n] = sum_{k in tile t} Aq[m,k]*Bq[n,k]   one tcgen05.mma.kind::i8 per 32 k (exact, s32 in TMEM)
//   c_t      = clamp(rne(P_t / 2^r), -2^(b_a-1), 2^(b_a-1)-1)            epilogue warps, registers
//   S        = sum_t c_t                                                   int32 registers
//   out      = fp32(S) * fp32(step_a*step_b*2^r / n_h)
//
// Output blocks are 128 x 256; persistent CTAs (one per SM) walk over them.  Warp 0 feeds a 4-stage
// shared-memory ring with TMA (128-byte swizzled rows = 4 tiles of 32 k per stage), warp 1 issues the
// MMAs into two TMEM accumulators of 256 columns, 8 epilogue warps drain the accumulators (tcgen05.ld),
// apply the accumulator quantisation per tile and keep the wide sums in registers.
// Tiles that provably cannot clamp (Cauchy-Schwarz bound from per-tile code norms) may be
// accumulated together in TMEM: the clamp is the identity there, so the integers are unchanged.
// Every wait is bounded; when one runs out the CTA records HDQT_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <string.h>

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
constexpr int GEMM_THREADS = 32 * (3 + NUM_EPI_WARPS);   // + TMA producer, MMA issuer, certificate builder
constexpr int TMEM_COLS = 512;
constexpr int MAX_CERT_WORDS = 256;            // certificate bitmask: up to 8192 accumulator tiles
constexpr int OUT_STAGE_WARP = 32 * 16 * 4;    // per epilogue warp: a 32-row x 16-column fp32 box for the store transpose
constexpr int TILE_INFO_BYTES = 4 * MAX_CERT_WORDS + 16;
// the dynamic shared-memory window is declared 1024-byte aligned (checked in the kernel), so no slack is kept
// offset of the store boxes (128-byte aligned)
constexpr int OUT_STAGE_OFF = (STAGES * STAGE_BYTES + 256 /*barriers*/ + 2 * TILE_INFO_BYTES + 127) / 128 * 128;
constexpr int SMEM_BYTES = OUT_STAGE_OFF + NUM_EPI_WARPS * OUT_STAGE_WARP;
static_assert(OUT_STAGE_WARP % 128 == 0, "store boxes must stay 128-byte aligned");
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");

// instruction descriptor: D = s32, A = B = signed 8-bit, both K-major, N = 256, M = 128
constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                           ((uint32_t)(BM >> 4) << 24);

struct GemmParams {
  int64_t M, N, K_pad;
  int32_t tiles32;        // K_pad / 32
  int32_t tiles_per_acc;  // acc_tile / 32 (tiles32 if acc_tile == 0)
  int32_t num_acc;        // accumulator tiles along K
  int32_t acc_shift;
  int32_t lo, hi;         // accumulator range
  int32_t had_block;
  int32_t flush_every;    // packed mode: accumulator tiles summed in 16-bit lanes before widening
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < (1 << 12); ++i) {
    if (mbar_test_wait(bar, parity)) return true;
  }
  for (int i = 0; i < (1 << 20); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    __nanosleep(512);
  }
  *abort_flag = 1;
  return false;
}

// mbar_wait_yield: for the epilogue warps. A warp that spins steals issue slots from the MMA issuer
// and from the warps that have work, so these waits suspend in hardware (try_wait) and sleep between
// polls; kSleepNs is the poll period (short for the per-tile handshake, long for the one wait on the
// merged accumulator that spans the whole main loop).
template <int kSleepNs>
__device__ __forceinline__ bool mbar_wait_yield(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  constexpr int kLimit = (kSleepNs >= 512) ? (1 << 21) : (1 << 24);
  for (int i = 0; i < kLimit; ++i) {
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
      o.x = __fmul_rn((float)s[0], scale);
      o.y = __fmul_rn((float)s[1], scale);
      o.z = __fmul_rn((float)s[2], scale);
      o.w = __fmul_rn((float)s[3], scale);
      *reinterpret_cast<float4*>(orow) = o;
    } else {
      *reinterpret_cast<int4*>(orow) = make_int4(s[0], s[1], s[2], s[3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (gn + i < p.N) {
        if (have_prev) s[i] += __float_as_int(orow[i]);
        orow[i] = kFinal ? __fmul_rn((float)s[i], scale) : __int_as_float(s[i]);
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
};

struct BlockJob {             // one output block as seen by the epilogue
  int m0, n0;
  int n_clamp_tiles;          // accumulator tiles that arrive one by one for the clamp path
  int n_merged;               // accumulator tiles merged in accumulator 0
  int merging;                // clamp tiles use accumulator 1 only (else they alternate 0 / 1)
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
__device__ __forceinline__ void store_chunk(const GemmParams& p, const EpiCtx& e, const BlockJob& job, int c,
                                            int (&val)[16], bool parked, float scale, bool raw = false) {
  const int64_t gm = (int64_t)job.m0 + e.q * 32 + e.lane;
  const int64_t gn = (int64_t)job.n0 + e.grp * EPI_COLS + c * 16;
  const bool staged = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                      (gn + 16 <= p.N);    // warp-uniform
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
      const float4 v = *reinterpret_cast<const float4*>(e.box + rloc * 16 + ((quad + ((rloc >> 1) & 3)) & 3) * 4);
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

__device__ __forceinline__ void release_accumulator(const EpiCtx& e, int buf, uint32_t* drains) {
  tc_fence_before();
  __syncwarp();
  if (e.lane == 0) mbar_arrive(e.bar_tempty + 8 * buf);
  ++drains[buf];
}

// Whole block merged (the common case on heavy-tailed operands): no per-tile sums exist, so the registers
// take the complete accumulator row at once and the accumulator goes back to the MMA issuer before any
// conversion or store work.
__device__ __forceinline__ bool epilogue_merged_only(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t* drains) {
  if (!mbar_wait_yield<64>(e.bar_tfull + 0, drains[0] & 1u, e.abort_flag)) return false;
  tc_fence_after();
  const float scale = dequant_scale(p);
  uint32_t mv[EPI_COLS];
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_LD16(e.lane_addr + c * 16, (mv + c * 16));
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_WAIT16((mv + c * 16));
  release_accumulator(e, 0, drains);
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) {
    int val[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) val[i] = (int)mv[c * 16 + i];
    store_chunk(p, e, job, c, val, false, scale);
  }
  return true;
}

// 16-bit-lane path: tile sums fit int16, b_a <= 8, r = 0.  TMEM is read with two columns packed per
// register (low half = even column); c - lo = relu(min(P - lo, hi - lo)) per lane in one instruction;
// sums stay unsigned 16-bit lanes and are widened through the output buffer every flush_every tiles.
__device__ __forceinline__ bool epilogue_packed(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t* drains) {
  uint32_t S[EPI_COLS / 2];
#pragma unroll
  for (int i = 0; i < EPI_COLS / 2; ++i) S[i] = 0u;
  const uint32_t off = (uint32_t)(-p.lo);                    // c - lo lies in [0, hi - lo]
  const uint32_t off2 = off | (off << 16);
  const uint32_t rng2 = (uint32_t)(p.hi - p.lo) | ((uint32_t)(p.hi - p.lo) << 16);
  int n_in_S = 0;
  bool parked = false;   // int32 partial sums are parked in the output buffer
  // Half of the warp's columns at a time through one load buffer; the other epilogue warp of the
  // scheduler covers the load latency.
  for (int ci = 0; ci < job.n_clamp_tiles; ++ci) {
    const int buf = job.merging ? 1 : (ci & 1);
    if (!mbar_wait(e.bar_tfull + 8 * buf, drains[buf] & 1u, e.abort_flag)) return false;
    tc_fence_after();
    uint32_t v[EPI_COLS / 4];
    HDQT_LD_HALF_PACK(e.lane_addr + buf * BN, v);
    HDQT_WAIT_HALF(v);
#pragma unroll
    for (int i = 0; i < EPI_COLS / 4; ++i) S[i] += __viaddmin_s16x2_relu(v[i], off2, rng2);
    HDQT_LD_HALF_PACK(e.lane_addr + buf * BN + EPI_COLS / 2, v);
    HDQT_WAIT_HALF(v);                                                 // the buffer is free
    release_accumulator(e, buf, drains);
#pragma unroll
    for (int i = 0; i < EPI_COLS / 4; ++i) S[EPI_COLS / 4 + i] += __viaddmin_s16x2_relu(v[i], off2, rng2);
    if (++n_in_S == p.flush_every && ci + 1 < job.n_clamp_tiles) {
      // widen: park int32 partial sums in the output buffer
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
      n_in_S = 0;
      parked = true;
    }
  }
  if (job.n_merged > 0) {
    if (!mbar_wait_yield<64>(e.bar_tfull + 0, drains[0] & 1u, e.abort_flag)) return false;
    tc_fence_after();
  }
  const float scale = dequant_scale(p);
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) {
    uint32_t mv[16];
    if (job.n_merged > 0) {   // uniform
      HDQT_TMEM_LD16(e.lane_addr + c * 16, mv);
      HDQT_TMEM_WAIT16(mv);
      // the last of the merged accumulator is in registers: hand it back to the MMA issuer
      if (c == EPI_COLS / 16 - 1) release_accumulator(e, 0, drains);
    }
    int val[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t sp = S[c * 8 + i];
      val[2 * i] = (int)(sp & 0xFFFFu) - (int)off * n_in_S;
      val[2 * i + 1] = (int)(sp >> 16) - (int)off * n_in_S;
      if (job.n_merged > 0) {
        val[2 * i] += (int)mv[2 * i];
        val[2 * i + 1] += (int)mv[2 * i + 1];
      }
    }
    store_chunk(p, e, job, c, val, parked, scale);
  }
  return true;
}

// 32-bit path: one register per accumulator element, any b_a and shift r, optional per-tile debug output.
template <bool kShift, bool kTilesOut>
__device__ __forceinline__ bool epilogue_wide(const GemmParams& p, EpiCtx e, BlockJob job, uint32_t* drains) {
  int S[EPI_COLS];
#pragma unroll
  for (int i = 0; i < EPI_COLS; ++i) S[i] = 0;
  const int r = p.acc_shift, lo = p.lo, hi = p.hi;
  for (int ci = 0; ci < job.n_clamp_tiles; ++ci) {
    const int buf = job.merging ? 1 : (ci & 1);
    if (!mbar_wait(e.bar_tfull + 8 * buf, drains[buf] & 1u, e.abort_flag)) return false;
    tc_fence_after();
#pragma unroll
    for (int c = 0; c < EPI_COLS / 16; ++c) {
      uint32_t v[16];
      HDQT_TMEM_LD16(e.lane_addr + buf * BN + c * 16, v);
      HDQT_TMEM_WAIT16(v);
      if (c == EPI_COLS / 16 - 1) release_accumulator(e, buf, drains);
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
    if (!mbar_wait_yield<64>(e.bar_tfull + 0, drains[0] & 1u, e.abort_flag)) return false;
    tc_fence_after();
  }
  const float scale = dequant_scale(p);
#pragma unroll
  for (int c = 0; c < EPI_COLS / 16; ++c) {
    int val[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) val[i] = S[c * 16 + i];
    if (job.n_merged > 0) {   // uniform
      uint32_t mv[16];
      HDQT_TMEM_LD16(e.lane_addr + c * 16, mv);
      HDQT_TMEM_WAIT16(mv);
      if (c == EPI_COLS / 16 - 1) release_accumulator(e, 0, drains);
#pragma unroll
      for (int i = 0; i < 16; ++i) val[i] += (int)mv[i];
    }
    store_chunk(p, e, job, c, val, false, scale);
  }
  return true;
}

// ---- the kernel -----------------------------------------------------------------------------
// Persistent: one CTA per SM walks over output blocks (block index = blockIdx.x + i*gridDim.x), so that the
// TMA producer runs ahead into the next block while the epilogue warps drain the previous one, and the
// per-block fixed costs (TMEM allocation, barrier set-up, pipeline fill) are paid once.
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer, 2 = certificate builder (clamp-free tile bitmask of the
// next block, from the tile norms), 3..10 = epilogue (TMEM lane quarter = warp % 4, 128 columns each;
// 11 warps leave each thread 168 registers: the sums of 128 columns plus a load buffer fit without spills).
//
// kPacked: the per-tile sums fit 16 bits and b_a <= 8, r = 0: TMEM is read with two columns packed
//          per register, clamp and add work on 16-bit lane pairs (half the ALU work per element).
// otherwise: one 32-bit register per accumulator element, any b_a and r.

struct TileInfo {                       // what the certificate warp publishes per output block
  uint32_t mask[MAX_CERT_WORDS];        // bit a: accumulator tile a provably cannot clamp
  int32_t n_uncert;                     // accumulator tiles without a certificate
  int32_t pad[3];
};
static_assert(sizeof(TileInfo) == TILE_INFO_BYTES, "TileInfo layout");

__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tile_m, int& tile_n) {
  // grouped order: co-resident CTAs form a roughly square patch (16 row blocks x ~9 column blocks on
  // 148 SMs), so both operands' panels are shared through L2
  constexpr int GROUP_M = 16;
  const int per_group = GROUP_M * tiles_n;
  const int group = t / per_group;
  const int first_m = group * GROUP_M;
  const int group_rows = min(tiles_m - first_m, GROUP_M);
  const int in_group = t - group * per_group;
  tile_m = first_m + in_group % group_rows;
  tile_n = in_group / group_rows;
}

// i-th output block of this launch: from the work list if there is one, else in grouped order
__device__ __forceinline__ void block_coords(const GemmParams& p, int i, int tiles_m, int tiles_n, int& tile_m,
                                             int& tile_n) {
  if (p.block_list != nullptr) {
    const int id = __ldg(p.block_list + i);
    tile_m = id / tiles_n;
    tile_n = id - tile_m * tiles_n;
  } else {
    tile_coords(i, tiles_m, tiles_n, tile_m, tile_n);
  }
}

template <bool kPacked, bool kShift, bool kTilesOut>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_i8_tiled_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ GemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  uint8_t* smem_al = smem_raw;
  if (smem_base & 1023u) {   // the 128-byte swizzle needs 1024-byte aligned stages: refuse rather than corrupt
    if (threadIdx.x == 0) report_status(p.dev_status, HDQT_ERR_CUDA);
    return;
  }
  // barrier block behind the stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * STAGE_BYTES);
  const uint32_t bar_full = smem_u32(bars);             // [STAGES]  TMA -> MMA
  const uint32_t bar_empty = bar_full + 8 * STAGES;     // [STAGES]  MMA -> TMA
  const uint32_t bar_tfull = bar_empty + 8 * STAGES;    // [2]       MMA -> epilogue (accumulator ready)
  const uint32_t bar_tempty = bar_tfull + 16;           // [2]       epilogue -> MMA (accumulator drained)
  const uint32_t bar_ifull = bar_tempty + 16;           // [2]       certificate warp -> MMA, epilogue
  const uint32_t bar_iempty = bar_ifull + 16;           // [2]       MMA, epilogue -> certificate warp
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  TileInfo* tile_info = reinterpret_cast<TileInfo*>(smem_al + STAGES * STAGE_BYTES + 256);   // [2]

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int tiles_m = (int)((p.M + BM - 1) / BM), tiles_n = (int)((p.N + BN - 1) / BN);
  const int num_tiles = (p.block_list != nullptr) ? __ldg(p.block_count) : tiles_m * tiles_n;
  const int num_kblocks = (p.tiles32 + 3) >> 2;
  const int num_acc = p.num_acc;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, NUM_EPI_WARPS);
      mbar_init(bar_ifull + 8 * b, 1);
      mbar_init(bar_iempty + 8 * b, NUM_EPI_WARPS + 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // A block merges its certified tiles only when few tiles need the clamp path (that path is
  // single-buffered while merging).
  auto block_merges = [&](int n_uncert) {
    return (p.merge == 2) ||
           (p.merge == 1 && (int64_t)n_uncert * 256 <= (int64_t)p.merge_max_uncert_256 * num_acc);
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;   // k-blocks issued so far, over all output blocks
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int tile_m, tile_n;
        block_coords(p, tile, tiles_m, tiles_n, tile_m, tile_n);
        for (int kb = 0; kb < num_kblocks; ++kb, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t par = ((it / STAGES) & 1u) ^ 1u;
          if (!mbar_wait(bar_empty + 8 * s, par, abort_flag)) { ok = false; break; }
          mbar_expect_tx(bar_full + 8 * s, STAGE_BYTES);
          const uint32_t a_dst = smem_base + s * STAGE_BYTES;
          tma_load_2d(a_dst, &map_a, kb * BKB, tile_m * BM, bar_full + 8 * s);
          tma_load_2d(a_dst + A_STAGE, &map_b, kb * BKB, tile_n * BN, bar_full + 8 * s);
        }
      }
      if (*abort_flag) {
        // let the copies that are still in flight land before the CTA gives its memory back
        for (uint32_t k = (it > STAGES ? it - STAGES : 0u); k < it; ++k) {
          const uint32_t bar = bar_full + 8 * (k % STAGES);
          const uint32_t par = (k / STAGES) & 1u;
          for (int i = 0; i < (1 << 16) && !mbar_try_wait(bar, par); ++i) __nanosleep(256);
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------ certificate builder ------------------------
    // bit a is set iff every 32-wide sub-tile of accumulator tile a satisfies
    // max_row ||a||^2 * max_col ||b||^2 <= (hi / tiles_per_acc)^2, so |P| <= hi for the whole block
    // (Cauchy-Schwarz) and the clamp is the identity there.
    if (p.merge == 1) {
      int ti = 0;
      for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++ti) {
        const int slot = ti & 1;
        if (!mbar_wait_yield<128>(bar_iempty + 8 * slot, (((uint32_t)ti >> 1) & 1u) ^ 1u, abort_flag)) break;
        int tile_m, tile_n;
        block_coords(p, tile, tiles_m, tiles_n, tile_m, tile_n);
        const int64_t T = p.tiles32;
        const int32_t* na = p.norms_a + (int64_t)tile_m * T;
        const int64_t nb_blk = (int64_t)tile_n * 2;
        const int32_t* nb0 = p.norms_b + nb_blk * T;
        const bool has1 = (nb_blk + 1) * 128 < p.N;
        const int32_t* nb1 = nb0 + T;
        TileInfo& info = tile_info[slot];
        int uncert = 0;
        const int acc_round = (num_acc + 31) & ~31;
        for (int a = lane; a < acc_round; a += 32) {
          bool cert = false;
          if (a < num_acc) {
            cert = true;
            const int t0 = a * p.tiles_per_acc;
            const int t1 = min(p.tiles32, t0 + p.tiles_per_acc);
            for (int t = t0; t < t1; ++t) {
              const int64_t a2 = __ldg(na + t);
              int64_t b2 = __ldg(nb0 + t);
              if (has1) b2 = max(b2, (int64_t)__ldg(nb1 + t));
              cert = cert && (a2 * b2 <= p.cert_thr_sq);
            }
          }
          const uint32_t bits = __ballot_sync(0xFFFFFFFFu, cert);
          if (lane == 0) {
            info.mask[a >> 5] = bits;
            const int valid = min(32, num_acc - a);
            uncert += valid - __popc(valid == 32 ? bits : (bits & ((1u << valid) - 1u)));
          }
        }
        if (lane == 0) {
          info.n_uncert = uncert;
          __threadfence_block();
          mbar_arrive(bar_ifull + 8 * slot);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (lane == 0) {
      // tcgen05.mma holds the issuing thread until the tensor pipe takes the operation, and the pipe
      // idles while this thread does anything else: bookkeeping between two MMAs is dead tensor time.
      // Stages whose four tiles are all merged are therefore issued as four back-to-back MMAs, with
      // the next stage's barrier polled ahead; only stages with clamp tiles take the per-tile code.
      const uint64_t desc_a0 = make_smem_desc(smem_base);
      const uint64_t desc_b0 = make_smem_desc(smem_base + A_STAGE);
      uint32_t s = 0;            // smem stage
      uint32_t full_par = 0;     // parity of the stage's next "full" phase
      uint32_t fills[2] = {0u, 0u};   // how many times each TMEM accumulator has been handed to the epilogue
      uint64_t desc_a = desc_a0, desc_b = desc_b0;
      bool ok = true;
      const int tiles32 = p.tiles32, tpa = p.tiles_per_acc;
      bool ready = false;
      int ti = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++ti) {
        const int slot = ti & 1;
        int n_uncert = (p.merge == 2) ? 0 : num_acc;
        if (p.merge == 1) {
          if (!mbar_wait(bar_ifull + 8 * slot, ((uint32_t)ti >> 1) & 1u, abort_flag)) { ok = false; break; }
          n_uncert = *reinterpret_cast<volatile int32_t*>(&tile_info[slot].n_uncert);
        }
        const bool merging = block_merges(n_uncert);
        const int n_merged = merging ? num_acc - n_uncert : 0;
        const uint32_t* cert_mask = tile_info[slot].mask;
        const bool nibble_ok = (p.merge == 2) || (merging && p.merge == 1 && tpa == 1);
        int j = 0;                 // position inside the current accumulator tile
        int acc = 0;               // accumulator tile index
        int clamp_idx = 0;         // index among this block's tiles that take the clamp path
        bool cert = (p.merge == 2);
        uint32_t merged_started = 0;
        uint32_t d_tmem = tmem_base;
        int cur_buf = 0;
        for (int kb = 0; kb < num_kblocks; ++kb) {
          if (!ready && !mbar_wait(bar_full + 8 * s, full_par, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t s_next = (s + 1 == STAGES) ? 0u : s + 1;
          const uint32_t par_next = (s + 1 == STAGES) ? (full_par ^ 1u) : full_par;
          const int kt0 = kb * 4;
          uint32_t nib = 0;
          if (p.merge == 2) nib = 0xFu;
          else if (nibble_ok) nib = (cert_mask[kb >> 3] >> ((kb & 7) * 4)) & 0xFu;
          if (nib == 0xFu && kt0 + 4 <= tiles32) {
            if (!merged_started) {
              // the merged accumulator (buffer 0) must have been drained by the previous user
              if (!mbar_wait(bar_tempty, (fills[0] & 1u) ^ 1u, abort_flag)) { ok = false; break; }
              tc_fence_after();
            }
            tc_mma_i8(tmem_base, desc_a, desc_b, merged_started);
            tc_mma_i8(tmem_base, desc_a + 2, desc_b + 2, 1u);
            tc_mma_i8(tmem_base, desc_a + 4, desc_b + 4, 1u);
            tc_mma_i8(tmem_base, desc_a + 6, desc_b + 6, 1u);
            merged_started = 1u;
            acc += 4;    // only meaningful (and only used) when tiles_per_acc == 1
          } else {
            const int kt1 = min(tiles32, kt0 + 4);
            for (int kt = kt0; kt < kt1; ++kt) {
              if (j == 0) {
                if (p.merge == 2) {
                  cert = true;
                } else if (merging) {
                  cert = (cert_mask[acc >> 5] >> (acc & 31)) & 1u;
                }
                // merged tiles accumulate in buffer 0; clamp tiles use buffer 1 when merging, else 0 / 1
                cur_buf = cert ? 0 : (merging ? 1 : (clamp_idx & 1));
                if (!cert || !merged_started) {
                  if (!mbar_wait(bar_tempty + 8 * cur_buf, (fills[cur_buf] & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                  tc_fence_after();
                }
                d_tmem = tmem_base + cur_buf * BN;
              }
              uint32_t sub2 = (uint32_t)(2 * (kt - kt0));
              uint32_t accumulate = cert ? merged_started : (uint32_t)(j != 0);
              tc_mma_i8(d_tmem, desc_a + sub2, desc_b + sub2, accumulate);
              if (tpa >= 4) {
                // long accumulator tiles: the rest of this stage's K tiles that belong to the same
                // accumulator tile go out back to back (bookkeeping between MMAs is dead tensor time)
                const int extra = min(kt1 - kt, tpa - j) - 1;
                for (int i = 0; i < extra; ++i) {
                  sub2 += 2;
                  tc_mma_i8(d_tmem, desc_a + sub2, desc_b + sub2, 1u);
                }
                kt += extra;
                j += extra;
              }
              if (cert) merged_started = 1u;
              if (++j == tpa || kt == tiles32 - 1) {
                if (!cert) {
                  tc_commit(bar_tfull + 8 * cur_buf);
                  ++fills[cur_buf];
                  ++clamp_idx;
                }
                j = 0;
                ++acc;
              }
            }
            if (!ok) break;
          }
          tc_commit(bar_empty + 8 * s);
          ready = mbar_test_wait(bar_full + 8 * s_next, par_next);
          s = s_next;
          full_par = par_next;
          if (s == 0) {
            desc_a = desc_a0;
            desc_b = desc_b0;
          } else {
            desc_a += (uint64_t)(STAGE_BYTES >> 4);
            desc_b += (uint64_t)(STAGE_BYTES >> 4);
          }
        }
        if (!ok) break;
        if (n_merged > 0) {
          tc_commit(bar_tfull + 0);
          ++fills[0];
        }
        if (p.merge == 1) mbar_arrive(bar_iempty + 8 * slot);
      }
    }
  } else {
    // ------------------------------ epilogue warps ----------------------------
    EpiCtx e;
    e.q = warp & 3;                     // TMEM lane quarter this warp may read
    e.grp = (warp - 3) >> 2;            // which EPI_COLS columns of the accumulator
    e.lane = lane;
    e.lane_addr = tmem_base + ((uint32_t)(e.q * 32) << 16) + (uint32_t)(e.grp * EPI_COLS);
    e.bar_tfull = bar_tfull;
    e.bar_tempty = bar_tempty;
    e.abort_flag = abort_flag;
    e.box = reinterpret_cast<float*>(smem_al + OUT_STAGE_OFF + (warp - 3) * OUT_STAGE_WARP);
    uint32_t drains[2] = {0u, 0u};      // how many times this warp has drained each accumulator
    int ti = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++ti) {
      const int slot = ti & 1;
      int n_uncert = (p.merge == 2) ? 0 : num_acc;
      if (p.merge == 1) {
        if (!mbar_wait_yield<128>(bar_ifull + 8 * slot, ((uint32_t)ti >> 1) & 1u, abort_flag)) break;
        n_uncert = *reinterpret_cast<volatile int32_t*>(&tile_info[slot].n_uncert);
      }
      BlockJob job;
      job.merging = block_merges(n_uncert) ? 1 : 0;
      job.n_clamp_tiles = job.merging ? n_uncert : num_acc;
      job.n_merged = job.merging ? num_acc - n_uncert : 0;
      int tile_m, tile_n;
      block_coords(p, tile, tiles_m, tiles_n, tile_m, tile_n);
      job.m0 = tile_m * BM;
      job.n0 = tile_n * BN;
      bool ok;
      if (job.n_clamp_tiles == 0 && job.n_merged > 0) ok = epilogue_merged_only(p, e, job, drains);
      else if (kPacked) ok = epilogue_packed(p, e, job, drains);
      else ok = epilogue_wide<kShift, kTilesOut>(p, e, job, drains);
      if (!ok) break;
      if (p.merge == 1) {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_iempty + 8 * slot);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) report_status(p.dev_status, HDQT_ERR_TIMEOUT);
}

// ---- work split for large problems ---------------------------------------------------------------
// A 256 x 256 "pair block" whose every K tile carries a clamp-free certificate needs no clamp path at all:
// such blocks go to the cta_group::2 kernel below (two accumulators of 256 columns, used alternately, so a
// block's drain overlaps the next block's main loop); all other blocks go to the general kernel above as two
// 128 x 256 blocks.  Two small kernels build the two work lists.

constexpr int PAIR_M = 2 * BM;

// Class of pair block t (grouped order over [tiles_m2, tiles_n]) from the number u of its accumulator tiles
// without a clamp-free certificate:  1 = none (pure),  2 = a few (u <= max_fix: the pair kernel accumulates them
// unclamped and a fix-up pass repairs the sums),  0 = many (general kernel).
constexpr int kFixFlag = 0x40000000;   // marks class-2 blocks in the pair kernel's work list

__device__ __forceinline__ bool pair_tile_certified(const int32_t* a0, const int32_t* b0, int64_t T, bool has_a1,
                                                    bool has_b1, int t0, int t1, int64_t thr_sq) {
  bool ok = true;
  for (int k = t0; k < t1; ++k) {
    int64_t a2 = __ldg(a0 + k), b2 = __ldg(b0 + k);
    if (has_a1) a2 = max(a2, (int64_t)__ldg(a0 + T + k));
    if (has_b1) b2 = max(b2, (int64_t)__ldg(b0 + T + k));
    ok = ok && (a2 * b2 <= thr_sq);
  }
  return ok;
}

__global__ void classify_pair_blocks_kernel(const int32_t* __restrict__ norms_a, const int32_t* __restrict__ norms_b,
                                            int64_t M, int64_t N, int tiles32, int tiles_per_acc, int num_acc,
                                            int64_t thr_sq, int max_fix, int tiles_m2, int tiles_n,
                                            uint8_t* __restrict__ flag) {
  const int warps_per_block = blockDim.x >> 5;
  const int t = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (t >= tiles_m2 * tiles_n) return;
  int tm, tn;
  tile_coords(t, tiles_m2, tiles_n, tm, tn);
  const int64_t T = tiles32;
  const int32_t* a0 = norms_a + (int64_t)(2 * tm) * T;
  const int32_t* b0 = norms_b + (int64_t)(2 * tn) * T;
  const bool has_a1 = (int64_t)(2 * tm + 1) * 128 < M;
  const bool has_b1 = (int64_t)(2 * tn + 1) * 128 < N;
  int u = 0;
  for (int a = lane; a < num_acc; a += 32) {
    const int t0 = a * tiles_per_acc, t1 = min(tiles32, t0 + tiles_per_acc);
    u += pair_tile_certified(a0, b0, T, has_a1, has_b1, t0, t1, thr_sq) ? 0 : 1;
  }
  u = __reduce_add_sync(0xFFFFFFFFu, u);
  if (lane == 0) flag[t] = (u == 0) ? 1 : (u <= max_fix ? 2 : 0);
}

// One thread block: ordered compaction of the flags into the list of clamp-free pair blocks and the list of
// 128 x 256 blocks (ids = row block * tiles_n + column block) that the general kernel has to do.
__global__ void __launch_bounds__(1024)
compact_blocks_kernel(const uint8_t* __restrict__ flag, int tiles_m2, int tiles_n, int64_t M,
                      int32_t* __restrict__ list_pair, int32_t* __restrict__ list_single,
                      int32_t* __restrict__ list_fix, int32_t* __restrict__ counts) {
  __shared__ int s_warp_pair[32], s_warp_single[32];
  __shared__ int s_base_pair, s_base_single, s_fix;
  const int n = tiles_m2 * tiles_n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { s_base_pair = 0; s_base_single = 0; s_fix = 0; }
  __syncthreads();
  for (int base = 0; base < n; base += 1024) {
    const int t = base + threadIdx.x;
    int tm = 0, tn = 0, is_pair = 0, singles = 0, cls = 0;
    if (t < n) {
      tile_coords(t, tiles_m2, tiles_n, tm, tn);
      cls = flag[t];
      is_pair = (cls != 0);
      if (!is_pair) singles = ((int64_t)(2 * tm + 1) * 128 < M) ? 2 : 1;
    }
    // exclusive scans inside the warp
    int sp = is_pair, ss = singles;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, sp, d), us = __shfl_up_sync(0xFFFFFFFFu, ss, d);
      if (lane >= d) { sp += up; ss += us; }
    }
    if (lane == 31) { s_warp_pair[warp] = sp; s_warp_single[warp] = ss; }
    __syncthreads();
    if (warp == 0) {
      int wp = s_warp_pair[lane], wsn = s_warp_single[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, wp, d), us = __shfl_up_sync(0xFFFFFFFFu, wsn, d);
        if (lane >= d) { wp += up; wsn += us; }
      }
      s_warp_pair[lane] = wp;       // inclusive over warps
      s_warp_single[lane] = wsn;
    }
    __syncthreads();
    const int off_pair = s_base_pair + (warp ? s_warp_pair[warp - 1] : 0) + sp - is_pair;
    const int off_single = s_base_single + (warp ? s_warp_single[warp - 1] : 0) + ss - singles;
    if (is_pair) list_pair[off_pair] = t | (cls == 2 ? kFixFlag : 0);
    if (cls == 2) list_fix[atomicAdd(&s_fix, 1)] = t;      // order is irrelevant for the fix-up pass
    if (singles >= 1) list_single[off_single] = (2 * tm) * tiles_n + tn;
    if (singles == 2) list_single[off_single + 1] = (2 * tm + 1) * tiles_n + tn;
    __syncthreads();
    if (threadIdx.x == 0) { s_base_pair += s_warp_pair[31]; s_base_single += s_warp_single[31]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { counts[0] = s_base_pair; counts[1] = s_base_single; counts[2] = s_fix; }
}

// ---- cta_group::2 kernel for clamp-free pair blocks ---------------------------------------------------
// Cluster of two CTAs = one 256 x 256 output block per step: CTA rank r loads rows [128r, 128r+128) of the
// A block and of the B block (32 KB per stage instead of 48: 6 stages, 2/3 of the L2->SM traffic), the
// leader (rank 0) issues M = 256 MMAs that read both CTAs' tiles, and each CTA's TMEM receives its 128 rows.
// Every K tile of such a block is clamp-free, so a block is ONE accumulation; the two 256-column
// accumulators alternate between blocks and the epilogue of a block overlaps the main loop of the next.
// Warps: 0 = TMA producer, 1 = MMA issuer (leader only), 2..9 = epilogue (lane quarter x 128 columns).

constexpr int P_STAGES = 6;
constexpr int P_B_STAGE = (BN / 2) * BKB;                 // this CTA's half of the B rows
constexpr int P_STAGE_BYTES = A_STAGE + P_B_STAGE;        // 32 KB
constexpr int P_EPI_WARPS = 8;
constexpr int P_THREADS = 32 * (2 + P_EPI_WARPS);
constexpr int P_OUT_OFF = P_STAGES * P_STAGE_BYTES + 256;
constexpr int P_SMEM_BYTES = P_OUT_OFF + P_EPI_WARPS * OUT_STAGE_WARP;
static_assert(P_OUT_OFF % 128 == 0 && P_SMEM_BYTES <= 232448, "pair kernel shared memory layout");
static_assert(EPI_COLS == 128, "the pair kernel's epilogue warps own 128 columns like the general kernel's");
constexpr uint32_t P_IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                             ((uint32_t)(PAIR_M >> 4) << 24);
// clearing the rank bit of a shared-window address gives the same offset in the pair leader's window
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y,
                                                 uint32_t bar_local) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_local & kPeerBitMask)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// arrives on the barrier at this offset in BOTH CTAs of the pair once the MMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(P_IDESC), "r"(accumulate)
      : "memory");
}

__global__ void __launch_bounds__(P_THREADS, 1) __cluster_dims__(2, 1, 1)
gemm_i8_merged_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                           const __grid_constant__ GemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  if (smem_base & 1023u) {   // (same outcome in both CTAs of a pair)
    if (threadIdx.x == 0) report_status(p.dev_status, HDQT_ERR_CUDA);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + P_STAGES * P_STAGE_BYTES);
  const uint32_t bar_full = smem_u32(bars);              // [P_STAGES] both CTAs' TMA -> leader's MMA issuer
  const uint32_t bar_empty = bar_full + 8 * P_STAGES;    // [P_STAGES] leader's MMA -> both producers
  const uint32_t bar_tfull = bar_empty + 8 * P_STAGES;   // [2] leader's MMA -> both CTAs' epilogue
  const uint32_t bar_tempty = bar_tfull + 16;            // [2] both CTAs' epilogue -> leader's MMA issuer
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * P_STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t cta_rank = cluster_ctarank();
  const bool leader = (cta_rank == 0);
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int tiles_m2 = (int)((p.M + PAIR_M - 1) / PAIR_M), tiles_n = (int)((p.N + BN - 1) / BN);
  const int num_blocks = (p.block_list != nullptr) ? __ldg(p.block_count) : tiles_m2 * tiles_n;
  const int num_kblocks = (p.tiles32 + 3) >> 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < P_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_tfull + 8 * b, 1);
      mbar_init(bar_tempty + 8 * b, 2 * P_EPI_WARPS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();     // the peer's barriers are initialised before anything is signalled across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // i-th block of this launch; returns true if its sums are to be parked as integers for the fix-up pass
  auto block_at = [&](int i, int& tm, int& tn) {
    const int t = (p.block_list != nullptr) ? __ldg(p.block_list + i) : i;
    tile_coords(t & ~kFixFlag, tiles_m2, tiles_n, tm, tn);
    return (t & kFixFlag) != 0;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int i = pair_id; i < num_blocks && ok; i += num_pairs) {
        int tm, tn;
        block_at(i, tm, tn);
        const int a_row0 = tm * PAIR_M + (int)cta_rank * BM;
        const int b_row0 = tn * BN + (int)cta_rank * (BN / 2);
        for (int kb = 0; kb < num_kblocks; ++kb, ++it) {
          const uint32_t s = it % P_STAGES;
          if (!mbar_wait(bar_empty + 8 * s, ((it / P_STAGES) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(bar_full + 8 * s, 2 * P_STAGE_BYTES);   // collects both CTAs' bytes
          const uint32_t dst = smem_base + s * P_STAGE_BYTES;
          tma_load_2d_pair(dst, &map_a, kb * BKB, a_row0, bar_full + 8 * s);
          tma_load_2d_pair(dst + A_STAGE, &map_b, kb * BKB, b_row0, bar_full + 8 * s);
        }
      }
      if (*abort_flag && leader) {
        for (uint32_t k = (it > P_STAGES ? it - P_STAGES : 0u); k < it; ++k) {
          const uint32_t bar = bar_full + 8 * (k % P_STAGES);
          for (int j = 0; j < (1 << 16) && !mbar_try_wait(bar, (k / P_STAGES) & 1u); ++j) __nanosleep(256);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) ------------------
    if (lane == 0 && leader) {
      uint32_t it = 0;
      int bi = 0;
      bool ok = true;
      for (int i = pair_id; i < num_blocks && ok; i += num_pairs, ++bi) {
        const int buf = bi & 1;
        if (!mbar_wait(bar_tempty + 8 * buf, (((uint32_t)bi >> 1) & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < num_kblocks; ++kb, ++it) {
          const uint32_t s = it % P_STAGES;
          if (!mbar_wait(bar_full + 8 * s, (it / P_STAGES) & 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = make_smem_desc(smem_base + s * P_STAGE_BYTES);
          const uint64_t db = make_smem_desc(smem_base + s * P_STAGE_BYTES + A_STAGE);
          if (kb * 4 + 4 <= p.tiles32) {
            tc_mma_i8_pair(d_tmem, da, db, kb > 0 ? 1u : 0u);
            tc_mma_i8_pair(d_tmem, da + 2, db + 2, 1u);
            tc_mma_i8_pair(d_tmem, da + 4, db + 4, 1u);
            tc_mma_i8_pair(d_tmem, da + 6, db + 6, 1u);
          } else {
            for (int sub = 0; kb * 4 + sub < p.tiles32; ++sub)
              tc_mma_i8_pair(d_tmem, da + 2 * sub, db + 2 * sub, (kb > 0 || sub > 0) ? 1u : 0u);
          }
          tc_commit_pair(bar_empty + 8 * s);
        }
        if (ok) tc_commit_pair(bar_tfull + 8 * buf);
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs) ----------------------
    EpiCtx e;
    e.q = warp & 3;
    e.grp = (warp - 2) >> 2;
    e.lane = lane;
    e.lane_addr = tmem_base + ((uint32_t)(e.q * 32) << 16) + (uint32_t)(e.grp * EPI_COLS);
    e.bar_tfull = bar_tfull;
    e.bar_tempty = map_to_cta(bar_tempty, 0);      // the leader's barriers, as cluster addresses
    e.abort_flag = abort_flag;
    e.box = reinterpret_cast<float*>(smem_raw + P_OUT_OFF + (warp - 2) * OUT_STAGE_WARP);
    const float scale = dequant_scale(p);
    int bi = 0;
    for (int i = pair_id; i < num_blocks; i += num_pairs, ++bi) {
      const int buf = bi & 1;
      int tm, tn;
      const bool raw = block_at(i, tm, tn);
      BlockJob job;
      job.m0 = tm * PAIR_M + (int)cta_rank * BM;
      job.n0 = tn * BN;
      job.n_clamp_tiles = 0;
      job.n_merged = p.num_acc;
      job.merging = 1;
      if (!mbar_wait_yield<64>(bar_tfull + 8 * buf, ((uint32_t)bi >> 1) & 1u, abort_flag)) break;
      tc_fence_after();
      uint32_t mv[EPI_COLS];
#pragma unroll
      for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_LD16(e.lane_addr + buf * BN + c * 16, (mv + c * 16));
#pragma unroll
      for (int c = 0; c < EPI_COLS / 16; ++c) HDQT_TMEM_WAIT16((mv + c * 16));
      // the accumulator is in registers: hand it back before converting and storing
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(e.bar_tempty + 8 * buf);
#pragma unroll
      for (int c = 0; c < EPI_COLS / 16; ++c) {
        int val[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) val[k] = (int)mv[c * 16 + k];
        store_chunk(p, e, job, c, val, false, scale, raw);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();     // neither CTA leaves while the other may still read its operands or signal its barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                 : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) report_status(p.dev_status, HDQT_ERR_TIMEOUT);
}

// ---- fix-up pass for pair blocks with a few uncertified accumulator tiles -----------------------------
// The pair kernel accumulated ALL their tiles unclamped and parked the integer sums in the output buffer.
// For an uncertified tile the accumulator quantisation may change the tile sum, so this pass recomputes
// exactly those tile sums P on the CUDA cores and adds clamp(P) - P; the result is sum_t clamp(P_t) bit for bit
// (on certified tiles the clamp is the identity).  Then it applies the dequantising scale.
// Work item = 64 rows of a 256 x 256 block (4 items per block, so that the few blocks spread over all SMs),
// 256 threads: warp w owns rows 8w..8w+7, lane l owns the columns l + 32 j.  Corrections are rare, so they are
// added to the parked sums in place as they are found.
constexpr int FIX_ROWS = 64;
constexpr int kMaxFixTiles = 256;   // the classification sends blocks with more uncertified tiles to the general kernel
constexpr int FIX_B_STRIDE = 36;    // bytes per staged B row (32 + 4: consecutive rows fall into different banks)

__global__ void __launch_bounds__(256, 2)
fixup_pair_blocks_kernel(const int8_t* __restrict__ Aq, const int8_t* __restrict__ Bq, const GemmParams p,
                         const int32_t* __restrict__ list_fix, const int32_t* __restrict__ counts) {
  __shared__ __align__(16) uint8_t sA[FIX_ROWS * 32];
  __shared__ __align__(16) uint8_t sB[256 * FIX_B_STRIDE];
  __shared__ int s_list[kMaxFixTiles];
  __shared__ int s_count;
  const int tiles_m2 = (int)((p.M + PAIR_M - 1) / PAIR_M), tiles_n = (int)((p.N + BN - 1) / BN);
  const int n_items = (PAIR_M / FIX_ROWS) * __ldg(counts + 2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t T = p.tiles32;
  const float scale = dequant_scale(p);
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    int tm, tn;
    tile_coords(__ldg(list_fix + item / (PAIR_M / FIX_ROWS)), tiles_m2, tiles_n, tm, tn);
    const int64_t m0 = (int64_t)tm * PAIR_M + (item % (PAIR_M / FIX_ROWS)) * FIX_ROWS, n0 = (int64_t)tn * BN;
    if (m0 >= p.M) continue;     // block-uniform: these rows of a ragged last block do not exist
    // certificates are those of the whole pair block (what the pair kernel relied on)
    const int32_t* a0 = p.norms_a + (int64_t)(2 * tm) * T;
    const int32_t* b0 = p.norms_b + (int64_t)(2 * tn) * T;
    const bool has_a1 = (int64_t)(2 * tm + 1) * 128 < p.M;
    const bool has_b1 = (int64_t)(2 * tn + 1) * 128 < p.N;
    // all threads look for the (few) uncertified accumulator tiles in parallel, then walk that short list
    __syncthreads();
    if (threadIdx.x == 0) s_count = 0;
    __syncthreads();
    for (int a = threadIdx.x; a < p.num_acc; a += blockDim.x) {
      const int t0 = a * p.tiles_per_acc, t1 = min(p.tiles32, t0 + p.tiles_per_acc);
      if (!pair_tile_certified(a0, b0, T, has_a1, has_b1, t0, t1, p.cert_thr_sq)) {
        const int slot = atomicAdd(&s_count, 1);
        if (slot < kMaxFixTiles) s_list[slot] = a;
      }
    }
    __syncthreads();
    const int n_uncert = min(s_count, kMaxFixTiles);
    for (int u = 0; u < n_uncert; ++u) {
      const int a = s_list[u];
      const int t0 = a * p.tiles_per_acc, t1 = min(p.tiles32, t0 + p.tiles_per_acc);
      int P[8][8];
#pragma unroll
      for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int j = 0; j < 8; ++j) P[r][j] = 0;
      for (int t = t0; t < t1; ++t) {
        __syncthreads();
        {   // stage the 32-byte K slice of 64 rows of A and 256 rows of B (rows beyond the matrices read as zero)
          const int row = threadIdx.x >> 2, part = threadIdx.x & 3;     // 4 threads x 8 bytes per row
          uint2 va = make_uint2(0u, 0u);
          if (m0 + row < p.M) va = __ldg(reinterpret_cast<const uint2*>(Aq + (m0 + row) * p.K_pad + (int64_t)t * 32 + part * 8));
          *reinterpret_cast<uint2*>(sA + row * 32 + part * 8) = va;
#pragma unroll
          for (int h = 0; h < 256 / FIX_ROWS; ++h) {
            const int brow = row + FIX_ROWS * h;
            uint2 vb = make_uint2(0u, 0u);
            if (n0 + brow < p.N) vb = __ldg(reinterpret_cast<const uint2*>(Bq + (n0 + brow) * p.K_pad + (int64_t)t * 32 + part * 8));
            uint32_t* db = reinterpret_cast<uint32_t*>(sB + brow * FIX_B_STRIDE + part * 8);
            db[0] = vb.x;
            db[1] = vb.y;
          }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          int av[8], bv[8];
#pragma unroll
          for (int r = 0; r < 8; ++r) av[r] = *reinterpret_cast<const int*>(sA + (warp * 8 + r) * 32 + k * 4);
#pragma unroll
          for (int j = 0; j < 8; ++j) bv[j] = *reinterpret_cast<const int*>(sB + (lane + 32 * j) * FIX_B_STRIDE + k * 4);
#pragma unroll
          for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int j = 0; j < 8; ++j) P[r][j] = __dp4a(av[r], bv[j], P[r][j]);
        }
      }
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const int64_t gm = m0 + warp * 8 + r;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int64_t gn = n0 + lane + 32 * j;
          const int d = min(max(P[r][j], p.lo), p.hi) - P[r][j];
          if (d != 0 && gm < p.M && gn < p.N) {
            int* o = reinterpret_cast<int*>(p.out + gm * p.ld_out + gn);   // only this thread touches this element
            *o += d;
          }
        }
      }
    }
    // parked (now exact) integer sums -> fp32, lanes on consecutive columns; all loads first, so that
    // they are in flight together (each element is touched by this thread only)
    int Sv[8][8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int64_t gm = m0 + warp * 8 + r;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int64_t gn = n0 + lane + 32 * j;
        Sv[r][j] = (gm < p.M && gn < p.N) ? __float_as_int(__ldcg(p.out + gm * p.ld_out + gn)) : 0;
      }
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const int64_t gm = m0 + warp * 8 + r;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int64_t gn = n0 + lane + 32 * j;
        if (gm < p.M && gn < p.N) {
          p.out[gm * p.ld_out + gn] = __fmul_rn((float)Sv[r][j], scale);
          if (p.S_out != nullptr) p.S_out[gm * p.N + gn] = Sv[r][j];
        }
      }
    }
    __syncthreads();
  }
}

// ---- smallest clamp-free accumulator shift (CUDA cores; a calibration utility, not the hot path)

__global__ void calibrate_shift_kernel(const int8_t* __restrict__ Aq, const int8_t* __restrict__ Bq, int64_t M,
                                       int64_t N, int64_t K_pad, int tile_k, int lo, int hi,
                                       int32_t* shift_out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int need = 0;
  if (idx < M * N) {
    const int64_t m = idx / N, n = idx - m * N;
    const int* a = reinterpret_cast<const int*>(Aq + m * K_pad);
    const int* b = reinterpret_cast<const int*>(Bq + n * K_pad);
    for (int64_t k0 = 0; k0 < K_pad; k0 += tile_k) {
      int P = 0;
      const int64_t k1 = min(K_pad, k0 + tile_k);
      for (int64_t k = k0; k < k1; k += 4) P = __dp4a(__ldg(a + (k >> 2)), __ldg(b + (k >> 2)), P);
      while (need < 31) {
        int c = P;
        if (need > 0) c = (P + ((1 << (need - 1)) - 1) + ((P >> need) & 1)) >> need;
        if (c >= lo && c <= hi) break;
        ++need;
      }
    }
  }
  need = __reduce_max_sync(0xFFFFFFFFu, need);
  if ((threadIdx.x & 31) == 0 && need > 0) atomicMax(shift_out, need);
}

// ---- host side --------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess) {
      return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// int8 matrix [rows, K_pad] (K contiguous) viewed as a 2-D tensor {K_pad, rows}; box {128 bytes, box_rows}
bool make_operand_map(CUtensorMap* map, const int8_t* base, int64_t rows, int64_t K_pad, int box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K_pad, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)K_pad};
  const cuuint32_t box[2] = {(cuuint32_t)BKB, (cuuint32_t)box_rows};
  const cuuint32_t elem_strides[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(base), dims, strides, box,
                         elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <bool kPacked, bool kShift, bool kTilesOut>
hdqt_status_t launch_variant(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& p, dim3 grid,
                             cudaStream_t s) {
  auto kern = gemm_i8_tiled_kernel<kPacked, kShift, kTilesOut>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return cuda_failure(e, "cudaFuncSetAttribute(gemm)");
  kern<<<grid, GEMM_THREADS, SMEM_BYTES, s>>>(ma, mb, p);
  e = cudaGetLastError();
  return e == cudaSuccess ? HDQT_OK : cuda_failure(e, "launch(gemm)");
}

}  // namespace

}  // namespace hdqt

using namespace hdqt;

namespace {
inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
// scratch of the work split: [counts 256 B | classes u8[npb] | pair list i32[npb] | single list i32[2 npb] | fix list i32[npb]]
struct SplitLayout {
  size_t flags, list_pair, list_single, list_fix, total;
  int64_t npb;
};
inline SplitLayout split_layout(int64_t M, int64_t N) {
  SplitLayout L;
  L.npb = ((M + PAIR_M - 1) / PAIR_M) * ((N + BN - 1) / BN);
  L.flags = 256;
  L.list_pair = L.flags + up256((size_t)L.npb);
  L.list_single = L.list_pair + up256((size_t)L.npb * 4);
  L.list_fix = L.list_single + up256((size_t)L.npb * 8);
  L.total = L.list_fix + up256((size_t)L.npb * 4);
  return L;
}
}  // namespace

extern "C" size_t hdqt_gemm_i8_workspace_bytes(int64_t M, int64_t N, int64_t) {
  if (M <= 0 || N <= 0) return 256;
  return split_layout(M, N).total;
}

extern "C" hdqt_status_t hdqt_gemm_i8_tiled(const int8_t* Aq, const int8_t* Bq, const float* step_a,
                                            const float* step_b, int64_t M, int64_t N, int64_t K_pad,
                                            int32_t code_bits, int32_t acc_bits, int32_t acc_tile,
                                            int32_t acc_shift, int32_t had_block, float* out, int64_t ld_out,
                                            int32_t* S_out, void* tiles_out, int32_t tiles_elem_bytes,
                                            const int32_t* norms_a, const int32_t* norms_b, uint32_t flags,
                                            void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                            void* stream) {
  if (!Aq || !Bq || !step_a || !step_b || !out) return HDQT_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K_pad <= 0 || ld_out < N) return HDQT_ERR_INVALID_ARG;
  if (K_pad % 32 != 0) return HDQT_ERR_INVALID_ARG;
  if (code_bits < 2 || code_bits > 8) return HDQT_ERR_INVALID_ARG;
  if (acc_bits < 2 || acc_bits > 32 || acc_shift < 0 || acc_shift > 24) return HDQT_ERR_INVALID_ARG;
  if (acc_tile < 0 || acc_tile % 32 != 0) return HDQT_ERR_INVALID_ARG;
  if (had_block < 1 || (had_block & (had_block - 1)) != 0) return HDQT_ERR_INVALID_ARG;
  if (M > INT32_MAX - BM || N > INT32_MAX - BN || K_pad > INT32_MAX - BKB) return HDQT_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(Aq) & 127) || (reinterpret_cast<uintptr_t>(Bq) & 127)) return HDQT_ERR_ALIGNMENT;
  if (reinterpret_cast<uintptr_t>(out) & 3) return HDQT_ERR_ALIGNMENT;
  if (workspace_bytes < hdqt_gemm_i8_workspace_bytes(M, N, K_pad)) return HDQT_ERR_WORKSPACE;
  if (tiles_out) {
    if (tiles_elem_bytes == 1) { if (acc_bits > 8) return HDQT_ERR_INVALID_ARG; }
    else if (tiles_elem_bytes == 2) { if (acc_bits > 16) return HDQT_ERR_INVALID_ARG; }
    else return HDQT_ERR_INVALID_ARG;
  }
  const int64_t tiles32 = K_pad / 32;
  const int64_t tpa = acc_tile == 0 ? tiles32 : acc_tile / 32;
  const int64_t num_acc = (tiles32 + tpa - 1) / tpa;
  // largest magnitude of one exact tile sum, given |code| <= 2^(code_bits-1)
  const int64_t code_max = int64_t(1) << (code_bits - 1);
  const int64_t p_max = tpa * 32 * code_max * code_max;
  if (p_max > INT32_MAX) return HDQT_ERR_UNSUPPORTED;
  // the wide sum must fit int32: |c_t| <= min(2^(b_a-1), p_max) per tile
  const int64_t acc_max = acc_bits >= 32 ? p_max : (int64_t(1) << (acc_bits - 1));
  const int64_t per_tile_max = acc_max < p_max ? acc_max : p_max;
  if (per_tile_max * num_acc > INT32_MAX) return HDQT_ERR_UNSUPPORTED;

  CUtensorMap ma, mb;
  if (!make_operand_map(&ma, Aq, M, K_pad, BM) || !make_operand_map(&mb, Bq, N, K_pad, BN)) return HDQT_ERR_CUDA;

  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = M; p.N = N; p.K_pad = K_pad;
  p.tiles32 = (int32_t)tiles32;
  p.tiles_per_acc = (int32_t)tpa;
  p.num_acc = (int32_t)num_acc;
  p.acc_shift = acc_shift;
  p.lo = acc_bits >= 32 ? INT32_MIN : -(1 << (acc_bits - 1));
  p.hi = acc_bits >= 32 ? INT32_MAX : (1 << (acc_bits - 1)) - 1;
  p.had_block = had_block;
  p.step_a = step_a; p.step_b = step_b;
  p.out = out; p.ld_out = ld_out; p.S_out = S_out;
  p.tiles_out = tiles_out; p.tiles_elem_bytes = tiles_elem_bytes;
  p.dev_status = dev_status;

  // 16-bit-lane epilogue: tile sums fit int16, the offset sums fit uint16 for flush_every tiles
  const bool packed = !tiles_out && acc_shift == 0 && acc_bits <= 8 && p_max <= 32767;
  p.flush_every = packed ? (int32_t)(65535 / ((int64_t)p.hi - p.lo)) : 0;
  if (p.flush_every > 256) p.flush_every = 256;

  // merging of clamp-free tiles: only without rounding shift (the shift is not the identity)
  p.merge = 0;
  if (!tiles_out && acc_shift == 0 && !(flags & HDQT_FLAG_NO_MERGE)) {
    if (p_max <= (int64_t)p.hi) {
      p.merge = 2;  // no tile can clamp whatever the data
    } else if (norms_a && norms_b && num_acc <= 32 * MAX_CERT_WORDS) {
      p.merge = 1;
      const int64_t thr = (int64_t)p.hi / tpa;
      p.cert_thr_sq = thr * thr;
      p.norms_a = norms_a;
      p.norms_b = norms_b;
      p.merge_max_uncert_256 = 32;  // merge in a CTA when at most 1/8 of its tiles need the clamp path
    }
  }

  const int64_t num_blocks = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  if (num_blocks > INT32_MAX) return HDQT_ERR_UNSUPPORTED;
  const int sms = sm_count();
  dim3 grid((unsigned)(num_blocks < sms ? num_blocks : sms));   // persistent: one CTA per SM
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

  // Large problems (at least 8 output blocks per SM; below that the extra launches cost more than they gain)
  // with clamp-free tiles: the cta_group::2 kernel takes the blocks whose K tiles are all, or all but a few,
  // certified (a fix-up pass repairs the few), the general kernel takes the rest.
  const bool split = (p.merge != 0) && !tiles_out && num_blocks >= 8 * (int64_t)sms && sms >= 2 && workspace != nullptr;
  if (split) {
    const SplitLayout L = split_layout(M, N);
    if (L.npb > INT32_MAX / 4) return HDQT_ERR_UNSUPPORTED;
    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
    int32_t* counts = reinterpret_cast<int32_t*>(ws);
    uint8_t* flags = ws + L.flags;
    int32_t* list_pair = reinterpret_cast<int32_t*>(ws + L.list_pair);
    int32_t* list_single = reinterpret_cast<int32_t*>(ws + L.list_single);
    const int tiles_m2 = (int)((M + PAIR_M - 1) / PAIR_M), tiles_n = (int)((N + BN - 1) / BN);
    CUtensorMap mb_half;
    if (!make_operand_map(&mb_half, Bq, N, K_pad, BN / 2)) return HDQT_ERR_CUDA;
    GemmParams pp = p;
    int32_t* list_fix = reinterpret_cast<int32_t*>(ws + L.list_fix);
    if (p.merge == 1) {
      // blocks with at most 1/32 of their accumulator tiles uncertified are repaired by the fix-up pass
      int max_fix = p.num_acc / 32 > 0 ? p.num_acc / 32 : 1;
      if (max_fix > kMaxFixTiles) max_fix = kMaxFixTiles;
      classify_pair_blocks_kernel<<<(unsigned)((L.npb + 7) / 8), 256, 0, s>>>(
          norms_a, norms_b, M, N, p.tiles32, p.tiles_per_acc, p.num_acc, p.cert_thr_sq, max_fix, tiles_m2, tiles_n, flags);
      compact_blocks_kernel<<<1, 1024, 0, s>>>(flags, tiles_m2, tiles_n, M, list_pair, list_single, list_fix, counts);
      pp.block_list = list_pair;
      pp.block_count = counts;
    }   // merge == 2: every block is clamp-free whatever the data, no lists needed
    cudaError_t e = cudaFuncSetAttribute(gemm_i8_merged_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         P_SMEM_BYTES);
    if (e != cudaSuccess) return cuda_failure(e, "cudaFuncSetAttribute(pair gemm)");
    const int64_t pairs = L.npb < sms / 2 ? L.npb : sms / 2;
    gemm_i8_merged_pair_kernel<<<(unsigned)(2 * pairs), P_THREADS, P_SMEM_BYTES, s>>>(ma, mb_half, pp);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_failure(e, "launch(pair gemm)");
    if (p.merge == 2) return HDQT_OK;
    fixup_pair_blocks_kernel<<<(unsigned)(2 * sms), 256, 0, s>>>(Aq, Bq, p, list_fix, counts);
    if (cudaGetLastError() != cudaSuccess) return HDQT_ERR_CUDA;
    p.block_list = list_single;     // the general kernel does what is left
    p.block_count = counts + 1;
  }
  if (tiles_out) {
    return acc_shift ? launch_variant<false, true, true>(ma, mb, p, grid, s)
                     : launch_variant<false, false, true>(ma, mb, p, grid, s);
  }
  if (packed) return launch_variant<true, false, false>(ma, mb, p, grid, s);
  return acc_shift ? launch_variant<false, true, false>(ma, mb, p, grid, s)
                   : launch_variant<false, false, false>(ma, mb, p, grid, s);
}

extern "C" hdqt_status_t hdqt_calibrate_acc_shift(const int8_t* Aq, const int8_t* Bq, int64_t M, int64_t N,
                                                  int64_t K_pad, int32_t acc_bits, int32_t acc_tile,
                                                  int32_t* shift_out, void* workspace, size_t workspace_bytes,
                                                  int32_t* dev_status, void* stream) {
  (void)workspace; (void)workspace_bytes; (void)dev_status;
  if (!Aq || !Bq || !shift_out) return HDQT_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K_pad <= 0 || K_pad % 32 != 0) return HDQT_ERR_INVALID_ARG;
  if (acc_bits < 2 || acc_bits > 32 || acc_tile < 0 || acc_tile % 32 != 0) return HDQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(Aq) & 3) || (reinterpret_cast<uintptr_t>(Bq) & 3)) return HDQT_ERR_ALIGNMENT;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(shift_out, 0, sizeof(int32_t), s) != cudaSuccess) return HDQT_ERR_CUDA;
  const int lo = acc_bits >= 32 ? INT32_MIN : -(1 << (acc_bits - 1));
  const int hi = acc_bits >= 32 ? INT32_MAX : (1 << (acc_bits - 1)) - 1;
  const int tile_k = acc_tile == 0 ? (int)K_pad : acc_tile;
  const int64_t total = M * N;
  calibrate_shift_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(Aq, Bq, M, N, K_pad, tile_k, lo, hi,
                                                                       shift_out);
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}
