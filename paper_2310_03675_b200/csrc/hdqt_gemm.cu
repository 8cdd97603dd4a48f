// Tiled integer GEMM with low-bit per-tile accumulators on the sm_100a tensor cores
// (paper Section 3, last paragraph: "tiled quantization ... tiles of size s"; Section 4:
// accumulator block size 32; Section 4.2: 8-bit accumulators in forward and backward pass).
//
//   P_t[m,n] = sum_{k in tile t} Aq[m,k]*Bq[n,k]   one tcgen05.mma.kind::i8 per 32 k (exact, s32 in TMEM)
//   c_t      = clamp(rne(P_t / 2^r), -2^(b_a-1), 2^(b_a-1)-1)            epilogue warps, registers
//   S        = sum_t c_t                                                   int32 registers
//   out      = fp32(S) * fp32(step_a*step_b*2^r / n_h)
//
// One CTA owns a 128 x 256 output block.  Warp 0 feeds a 4-stage shared-memory ring with TMA
// (128-byte swizzled rows = 4 tiles of 32 k per stage), warp 1 issues the MMAs into two TMEM
// accumulators of 256 columns, warps 2..17 drain the accumulators (tcgen05.ld), apply the
// accumulator quantisation per tile and keep the wide sums in registers.
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
constexpr int NUM_EPI_WARPS = 16;              // 4 per TMEM lane quarter, 64 accumulator columns each
constexpr int EPI_COLS = BN / (NUM_EPI_WARPS / 4);
constexpr int GEMM_THREADS = 32 * (2 + NUM_EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr int MAX_CERT_WORDS = 512;            // certificate bitmask: up to 16384 accumulator tiles
constexpr int STAGE_OUT_ROW = EPI_COLS + 4;     // floats per staged output row (+4: conflict-free float4 rows)
constexpr int STAGE_OUT_WARP = 32 * STAGE_OUT_ROW;   // floats per epilogue warp (32 rows x 64 columns)
static_assert(NUM_EPI_WARPS * STAGE_OUT_WARP * 4 <= STAGES * STAGE_BYTES, "output staging must fit the operand ring");
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/ + 4 * MAX_CERT_WORDS;

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

#define HDQT_TMEM_LD16(taddr, v)                                                                        \
  asm volatile(                                                                                         \
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                         \
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"                  \
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), \
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),        \
        "=r"(v[15])                                                                                     \
      : "r"(taddr)                                                                                      \
      : "memory")

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
// In the final pass of the vector path the fp32 values go to `stage` (this thread's row of the warp's
// shared-memory staging block) instead, and the warp copies the block out row by row afterwards, so
// that global stores are 256 contiguous bytes per half-warp rather than 16 bytes per row.
template <bool kFinal>
__device__ __forceinline__ void emit4(const GemmParams& p, int64_t gm, int64_t gn, int (&s)[4], bool have_prev,
                                      bool vec, float scale, float* stage = nullptr) {
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
      *reinterpret_cast<float4*>(stage != nullptr ? stage : orow) = o;
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

// ---- the kernel -----------------------------------------------------------------------------
// kPacked: the per-tile sums fit 16 bits and b_a <= 8, r = 0: TMEM is read with two columns packed
//          per register, clamp and add work on 16-bit lane pairs (half the ALU work per element).
// otherwise: one 32-bit register per accumulator element, any b_a and r.

template <bool kPacked, bool kShift, bool kTilesOut>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_i8_tiled_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  // barrier block behind the stages
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * STAGE_BYTES);
  const uint32_t bar_full = smem_u32(bars);             // [STAGES]
  const uint32_t bar_empty = bar_full + 8 * STAGES;     // [STAGES]
  const uint32_t bar_tfull = bar_empty + 8 * STAGES;    // [2]
  const uint32_t bar_tempty = bar_tfull + 16;           // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* s_uncert = reinterpret_cast<int*>(tmem_slot + 2);
  uint32_t* cert_mask = reinterpret_cast<uint32_t*>(smem_al + STAGES * STAGE_BYTES + 256);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // 1-D grid over output blocks, ordered so that co-resident CTAs form a roughly square patch
  // (16 row blocks x ~9 column blocks on 148 SMs): both operands' panels are then shared through L2
  const int tiles_m = (int)((p.M + BM - 1) / BM), tiles_n = (int)((p.N + BN - 1) / BN);
  int tile_m, tile_n;
  {
    constexpr int GROUP_M = 16;
    const int t = blockIdx.x;
    const int per_group = GROUP_M * tiles_n;
    const int group = t / per_group;
    const int first_m = group * GROUP_M;
    const int group_rows = min(tiles_m - first_m, GROUP_M);
    const int in_group = t - group * per_group;
    tile_m = first_m + in_group % group_rows;
    tile_n = in_group / group_rows;
  }
  const int m0 = tile_m * BM;
  const int n0 = tile_n * BN;
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
    }
    *abort_flag = 0;
    *s_uncert = 0;
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

  // ---- which accumulator tiles provably cannot clamp (Cauchy-Schwarz on the tile norms) ----
  // bit a of cert_mask is set iff every 32-wide sub-tile of accumulator tile a satisfies
  // max_row ||a||^2 * max_col ||b||^2 <= (hi / tiles_per_acc)^2, so |P| <= hi for the whole block.
  if (p.merge == 1) {
    if (warp >= 2) {
      const int et = threadIdx.x - 64;
      const int64_t T = p.tiles32;
      const int32_t* na = p.norms_a + (int64_t)tile_m * T;
      const int64_t nb_blk = (int64_t)tile_n * 2;
      const int32_t* nb0 = p.norms_b + nb_blk * T;
      const bool has1 = (nb_blk + 1) * 128 < p.N;
      const int32_t* nb1 = nb0 + T;
      int my_uncert = 0;
      const int acc_round = (num_acc + 31) & ~31;
      for (int a = et; a < acc_round; a += 32 * NUM_EPI_WARPS) {
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
          my_uncert += cert ? 0 : 1;
        }
        const uint32_t bits = __ballot_sync(0xFFFFFFFFu, cert);
        if (lane == 0) cert_mask[a >> 5] = bits;
      }
      my_uncert = __reduce_add_sync(0xFFFFFFFFu, my_uncert);
      if (lane == 0 && my_uncert) atomicAdd(s_uncert, my_uncert);
    }
    __syncthreads();
  }
  const int n_uncert = (p.merge == 2) ? 0 : *s_uncert;
  // merge in this CTA only when few tiles need the clamp path (it is single-buffered when merging)
  const bool merging = (p.merge == 2) ||
                       (p.merge == 1 && (int64_t)n_uncert * 256 <= (int64_t)p.merge_max_uncert_256 * num_acc);
  const int n_clamp_tiles = merging ? n_uncert : num_acc;
  const int n_merged = merging ? num_acc - n_uncert : 0;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < num_kblocks; ++kb) {
        const int s = kb % STAGES;
        const uint32_t par = ((kb / STAGES) & 1) ^ 1;
        if (!mbar_wait(bar_empty + 8 * s, par, abort_flag)) break;
        mbar_expect_tx(bar_full + 8 * s, STAGE_BYTES);
        const uint32_t a_dst = smem_base + s * STAGE_BYTES;
        tma_load_2d(a_dst, &map_a, kb * BKB, m0, bar_full + 8 * s);
        tma_load_2d(a_dst + A_STAGE, &map_b, kb * BKB, n0, bar_full + 8 * s);
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let the copies that are still in flight land before the CTA gives its memory back
        for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
          const uint32_t bar = bar_full + 8 * (kb % STAGES);
          const uint32_t par = (kb / STAGES) & 1;
          for (int i = 0; i < (1 << 16) && !mbar_try_wait(bar, par); ++i) __nanosleep(256);
        }
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
      int s = 0;                 // smem stage
      uint32_t full_par = 0;     // parity of the stage's next "full" phase
      int j = 0;                 // position inside the current accumulator tile
      int acc = 0;               // accumulator tile index
      int clamp_idx = 0;         // index among the tiles that take the clamp path
      bool cert = (p.merge == 2);
      uint32_t merged_started = 0;
      uint32_t d_tmem = tmem_base;
      uint32_t tfull_bar = bar_tfull;
      uint64_t desc_a = desc_a0, desc_b = desc_b0;
      bool ok = true;
      const int tiles32 = p.tiles32, tpa = p.tiles_per_acc;
      const bool nibble_ok = (p.merge == 2) || (merging && tpa == 1);
      bool ready = mbar_test_wait(bar_full, 0u);
      for (int kb = 0; kb < num_kblocks; ++kb) {
        if (!ready && !mbar_wait(bar_full + 8 * s, full_par, abort_flag)) { ok = false; break; }
        tc_fence_after();
        // poll the next stage now; the answer is needed only after this stage's MMAs
        const int s_next = (s + 1 == STAGES) ? 0 : s + 1;
        const uint32_t par_next = (s + 1 == STAGES) ? (full_par ^ 1u) : full_par;
        const int kt0 = kb * 4;
        uint32_t nib = 0;
        if (p.merge == 2) nib = 0xFu;
        else if (nibble_ok) nib = (cert_mask[kb >> 3] >> ((kb & 7) * 4)) & 0xFu;
        if (nib == 0xFu && kt0 + 4 <= tiles32) {
          tc_mma_i8(tmem_base, desc_a, desc_b, merged_started);
          tc_mma_i8(tmem_base, desc_a + 2, desc_b + 2, 1u);
          tc_mma_i8(tmem_base, desc_a + 4, desc_b + 4, 1u);
          tc_mma_i8(tmem_base, desc_a + 6, desc_b + 6, 1u);
          merged_started = 1u;
          acc += 4;    // only meaningful (and only used) when tiles_per_acc == 1
        } else {
          if (tpa < 4) {
            // short accumulator tiles: one MMA per pass keeps this thread's path between a released
            // accumulator and the next MMA as short as possible (it is on the critical chain of every tile)
            const int kt1 = min(tiles32, kt0 + 4);
            for (int kt = kt0; kt < kt1; ++kt) {
              if (j == 0) {
                if (p.merge == 2) {
                  cert = true;
                } else if (merging) {
                  cert = (cert_mask[acc >> 5] >> (acc & 31)) & 1u;
                }
                if (cert) {
                  d_tmem = tmem_base;                      // merged tiles accumulate in buffer 0
                } else {
                  // clamp tiles: buffer 1 when merging, else alternate 0 / 1
                  const int buf = merging ? 1 : (clamp_idx & 1);
                  const uint32_t use = merging ? (uint32_t)clamp_idx : (uint32_t)(clamp_idx >> 1);
                  if (!mbar_wait(bar_tempty + 8 * buf, (use & 1) ^ 1, abort_flag)) { ok = false; break; }
                  tc_fence_after();
                  d_tmem = tmem_base + buf * BN;
                  tfull_bar = bar_tfull + 8 * buf;
                }
              }
              const uint32_t sub2 = (uint32_t)(2 * (kt - kt0));
              tc_mma_i8(d_tmem, desc_a + sub2, desc_b + sub2, cert ? merged_started : (uint32_t)(j != 0));
              if (cert) merged_started = 1u;
              if (++j == tpa || kt == tiles32 - 1) {
                if (!cert) {
                  tc_commit(tfull_bar);
                  ++clamp_idx;
                }
                j = 0;
                ++acc;
              }
            }
          } else {
            // long accumulator tiles: the K tiles of this stage that belong to the current accumulator
            // tile go out back to back
            const int kt1 = min(tiles32, kt0 + 4);
            int kt = kt0;
            while (kt < kt1) {
              if (j == 0) {
                if (p.merge == 2) {
                  cert = true;
                } else if (merging) {
                  cert = (cert_mask[acc >> 5] >> (acc & 31)) & 1u;
                }
                if (cert) {
                  d_tmem = tmem_base;                      // merged tiles accumulate in buffer 0
                } else {
                  // clamp tiles: buffer 1 when merging, else alternate 0 / 1
                  const int buf = merging ? 1 : (clamp_idx & 1);
                  const uint32_t use = merging ? (uint32_t)clamp_idx : (uint32_t)(clamp_idx >> 1);
                  if (!mbar_wait(bar_tempty + 8 * buf, (use & 1) ^ 1, abort_flag)) { ok = false; break; }
                  tc_fence_after();
                  d_tmem = tmem_base + buf * BN;
                  tfull_bar = bar_tfull + 8 * buf;
                }
              }
              // the K tiles of this stage that belong to the current accumulator tile go out back to back
              uint32_t sub2 = (uint32_t)(2 * (kt - kt0));
              uint32_t accumulate = cert ? merged_started : (uint32_t)(j != 0);
              const int run = min(kt1 - kt, tpa - j);
              for (int i = 0; i < run; ++i) {
                tc_mma_i8(d_tmem, desc_a + sub2, desc_b + sub2, accumulate);
                sub2 += 2;
                accumulate = 1u;
              }
              if (cert) merged_started = 1u;
              j += run;
              kt += run;
              if (j == tpa || kt == tiles32) {
                if (!cert) {
                  tc_commit(tfull_bar);
                  ++clamp_idx;
                }
                j = 0;
                ++acc;
              }
            }
          }
          if (!ok) break;
        }
        tc_commit(bar_empty + 8 * s);
        ready = (kb + 1 < num_kblocks) && mbar_test_wait(bar_full + 8 * s_next, par_next);
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
      if (ok && n_merged > 0) tc_commit(bar_tfull + 0);
    }
  } else {
    // ------------------------------ epilogue warps ----------------------------
    const int q = warp & 3;                   // TMEM lane quarter this warp may read
    const int grp = (warp - 2) >> 2;          // which EPI_COLS columns of the accumulator
    const int row = q * 32 + lane;
    const int64_t gm = (int64_t)m0 + row;
    const int64_t gn0 = (int64_t)n0 + grp * EPI_COLS;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(grp * EPI_COLS);
    const int r = p.acc_shift, lo = p.lo, hi = p.hi;
    const bool vec = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                     (gn0 + EPI_COLS <= p.N);
    bool ok = true;
    // output staging reuses the operand ring: it is touched only after the last MMA has completed
    float* stage_warp = reinterpret_cast<float*>(smem_al) + (warp - 2) * STAGE_OUT_WARP;
    float* stage_row = stage_warp + lane * STAGE_OUT_ROW;
    // copies the warp's staged 32 x 64 block to global memory, two rows (2 x 256 bytes) per instruction
    auto copy_out = [&]() {
      __syncwarp();
      const int sub_row = lane >> 4, c4 = (lane & 15) * 4;
#pragma unroll 4
      for (int rr = 0; rr < 32; rr += 2) {
        const int rloc = rr + sub_row;
        const int64_t grow = (int64_t)m0 + q * 32 + rloc;
        if (grow < p.M) {
          const float4 v = *reinterpret_cast<const float4*>(stage_warp + rloc * STAGE_OUT_ROW + c4);
          *reinterpret_cast<float4*>(p.out + grow * p.ld_out + gn0 + c4) = v;
        }
      }
    };

    if (kPacked) {
      // two columns per register: low half = even column, high half = odd column
      uint32_t S[EPI_COLS / 2];
#pragma unroll
      for (int i = 0; i < EPI_COLS / 2; ++i) S[i] = 0u;
      const uint32_t off = (uint32_t)(-lo);                    // c - lo lies in [0, hi - lo]
      const uint32_t off2 = off | (off << 16);
      const uint32_t rng2 = (uint32_t)(hi - lo) | ((uint32_t)(hi - lo) << 16);
      int n_in_S = 0;
      bool parked = false;   // int32 partial sums are parked in the output buffer
      // Rolling pipeline over half-tiles (32 columns = 16 packed registers): while one half is clamped
      // and added, the load of the next half (possibly of the next tile) is in flight.
      uint32_t v0[EPI_COLS / 4], v1[EPI_COLS / 4];
      if (n_clamp_tiles > 0) {
        const int buf = merging ? 1 : 0;
        if (!mbar_wait(bar_tfull + 8 * buf, 0u, abort_flag)) ok = false;
        tc_fence_after();
        if (ok) HDQT_TMEM_LD16_PACK16(lane_addr + buf * BN, v0);
      }
      for (int ci = 0; ci < n_clamp_tiles && ok; ++ci) {
        const int buf = merging ? 1 : (ci & 1);
        HDQT_TMEM_WAIT16(v0);                                            // first half of tile ci has landed
        HDQT_TMEM_LD16_PACK16(lane_addr + buf * BN + EPI_COLS / 2, v1);  // second half in flight ...
#pragma unroll
        for (int i = 0; i < EPI_COLS / 4; ++i) S[i] += __viaddmin_s16x2_relu(v0[i], off2, rng2);
        HDQT_TMEM_WAIT16(v1);                                            // ... landed: the buffer is free
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
        if (ci + 1 < n_clamp_tiles) {
          const int nbuf = merging ? 1 : ((ci + 1) & 1);
          const uint32_t use = merging ? (uint32_t)(ci + 1) : (uint32_t)((ci + 1) >> 1);
          if (!mbar_wait(bar_tfull + 8 * nbuf, use & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          HDQT_TMEM_LD16_PACK16(lane_addr + nbuf * BN, v0);              // first half of the next tile in flight
        }
#pragma unroll
        for (int i = 0; i < EPI_COLS / 4; ++i) S[EPI_COLS / 4 + i] += __viaddmin_s16x2_relu(v1[i], off2, rng2);
        if (++n_in_S == p.flush_every && ci + 1 < n_clamp_tiles) {
          // widen: park int32 partial sums in the output buffer
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
      if (ok && n_merged > 0) {
        ok = mbar_wait_yield<256>(bar_tfull + 0, 0u, abort_flag);
        tc_fence_after();
      }
      if (ok) {
        const float scale = (float)((double)__ldg(p.step_a) * (double)__ldg(p.step_b) *
                                    (double)(1u << p.acc_shift) / (double)p.had_block);
#pragma unroll
        for (int c = 0; c < EPI_COLS / 16; ++c) {
          uint32_t mv[16];
          if (n_merged > 0) {   // uniform
            HDQT_TMEM_LD16(lane_addr + c * 16, mv);
            HDQT_TMEM_WAIT16(mv);
          }
          if (gm < p.M) {
#pragma unroll
            for (int i = 0; i < 8; i += 2) {
              const uint32_t s0 = S[c * 8 + i], s1 = S[c * 8 + i + 1];
              int s4[4];
              s4[0] = (int)(s0 & 0xFFFFu) - (int)off * n_in_S;
              s4[1] = (int)(s0 >> 16) - (int)off * n_in_S;
              s4[2] = (int)(s1 & 0xFFFFu) - (int)off * n_in_S;
              s4[3] = (int)(s1 >> 16) - (int)off * n_in_S;
              if (n_merged > 0) {
                s4[0] += (int)mv[2 * i]; s4[1] += (int)mv[2 * i + 1];
                s4[2] += (int)mv[2 * i + 2]; s4[3] += (int)mv[2 * i + 3];
              }
              emit4<true>(p, gm, gn0 + c * 16 + 2 * i, s4, parked, vec, scale,
                          vec ? stage_row + c * 16 + 2 * i : nullptr);
            }
          }
        }
        if (vec) copy_out();
      }
    } else {
      int S[EPI_COLS];
#pragma unroll
      for (int i = 0; i < EPI_COLS; ++i) S[i] = 0;
      for (int ci = 0; ci < n_clamp_tiles; ++ci) {
        const int buf = merging ? 1 : (ci & 1);
        const uint32_t use = merging ? (uint32_t)ci : (uint32_t)(ci >> 1);
        if (!mbar_wait(bar_tfull + 8 * buf, use & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < EPI_COLS / 16; ++c) {
          uint32_t v[16];
          HDQT_TMEM_LD16(lane_addr + buf * BN + c * 16, v);
          HDQT_TMEM_WAIT16(v);
          if (c == EPI_COLS / 16 - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int ct = acc_quant<kShift>((int)v[i], r, lo, hi);
            S[c * 16 + i] += ct;
            if (kTilesOut) {
              const int64_t n = gn0 + c * 16 + i;
              if (gm < p.M && n < p.N) {
                const int64_t o = ((int64_t)ci * p.M + gm) * p.N + n;
                if (p.tiles_elem_bytes == 1) reinterpret_cast<int8_t*>(p.tiles_out)[o] = (int8_t)ct;
                else reinterpret_cast<int16_t*>(p.tiles_out)[o] = (int16_t)ct;
              }
            }
          }
        }
      }
      if (ok && n_merged > 0) {
        ok = mbar_wait_yield<256>(bar_tfull + 0, 0u, abort_flag);
        tc_fence_after();
      }
      if (ok) {
        const float scale = (float)((double)__ldg(p.step_a) * (double)__ldg(p.step_b) *
                                    (double)(1u << p.acc_shift) / (double)p.had_block);
#pragma unroll
        for (int c = 0; c < EPI_COLS / 16; ++c) {
          uint32_t mv[16];
          if (n_merged > 0) {   // uniform
            HDQT_TMEM_LD16(lane_addr + c * 16, mv);
            HDQT_TMEM_WAIT16(mv);
          }
          if (gm < p.M) {
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
              int s4[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                s4[j] = S[c * 16 + i + j];
                if (n_merged > 0) s4[j] += (int)mv[i + j];
              }
              emit4<true>(p, gm, gn0 + c * 16 + i, s4, false, vec, scale, vec ? stage_row + c * 16 + i : nullptr);
            }
          }
        }
        if (vec) copy_out();
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

extern "C" size_t hdqt_gemm_i8_workspace_bytes(int64_t, int64_t, int64_t) { return 256; }

extern "C" hdqt_status_t hdqt_gemm_i8_tiled(const int8_t* Aq, const int8_t* Bq, const float* step_a,
                                            const float* step_b, int64_t M, int64_t N, int64_t K_pad,
                                            int32_t code_bits, int32_t acc_bits, int32_t acc_tile,
                                            int32_t acc_shift, int32_t had_block, float* out, int64_t ld_out,
                                            int32_t* S_out, void* tiles_out, int32_t tiles_elem_bytes,
                                            const int32_t* norms_a, const int32_t* norms_b, uint32_t flags,
                                            void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                            void* stream) {
  (void)workspace;
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
  const dim3 grid((unsigned)num_blocks);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
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
