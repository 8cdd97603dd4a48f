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
// (128-byte swizzled rows = 4 tiles of 32 k per stage), warp 1 issues the MMAs into a TMEM
// accumulator ring of 2 x 256 columns, warps 2..9 drain the accumulators (tcgen05.ld), apply
// the accumulator quantisation per tile and keep the wide sums in registers.
// Every wait is bounded; when one runs out the CTA records HDQT_ERR_TIMEOUT and leaves.
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
constexpr int NUM_EPI_WARPS = 8;
constexpr int GEMM_THREADS = 32 * (2 + NUM_EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;

// instruction descriptor: D = s32, A = B = signed 8-bit, both K-major, N = 256, M = 128
constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                           ((uint32_t)(BM >> 4) << 24);

struct GemmParams {
  int64_t M, N, K_pad;
  int32_t tiles32;        // K_pad / 32
  int32_t tiles_per_acc;  // acc_tile / 32 (tiles32 if acc_tile == 0)
  int32_t acc_shift;
  int32_t lo, hi;         // accumulator range
  int32_t had_block;
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

// Bounded wait: gives up after ~1 s, or as soon as another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < (1 << 14); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  for (int i = 0; i < (1 << 20); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    __nanosleep(512);
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

// accumulator quantisation of one exact tile sum
template <bool kShift>
__device__ __forceinline__ int acc_quant(int P, int r, int lo, int hi) {
  if (kShift) {
    // round-half-even of P / 2^r:  (P + (2^(r-1) - 1) + ((P >> r) & 1)) >> r
    P = (P + ((1 << (r - 1)) - 1) + ((P >> r) & 1)) >> r;
  }
  return min(max(P, lo), hi);
}

// ---- the kernel -----------------------------------------------------------------------------

template <bool kShift, bool kTilesOut>
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

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * BM;
  const int n0 = blockIdx.y * BN;
  const int num_kblocks = (p.tiles32 + 3) >> 2;
  const int num_acc = (p.tiles32 + p.tiles_per_acc - 1) / p.tiles_per_acc;

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
      for (int kt = 0; kt < p.tiles32; ++kt) {
        const int kb = kt >> 2, sub = kt & 3;
        const int s = kb % STAGES;
        if (sub == 0) {
          if (!mbar_wait(bar_full + 8 * s, (kb / STAGES) & 1, abort_flag)) break;
        }
        const int acc = kt / p.tiles_per_acc;
        const int j = kt - acc * p.tiles_per_acc;
        const int buf = acc & 1;
        if (j == 0) {
          if (!mbar_wait(bar_tempty + 8 * buf, ((acc >> 1) & 1) ^ 1, abort_flag)) break;
        }
        tc_fence_after();
        const uint32_t a_addr = smem_base + s * STAGE_BYTES + sub * 32;
        const uint64_t a_desc = make_smem_desc(a_addr);
        const uint64_t b_desc = make_smem_desc(a_addr + A_STAGE);
        tc_mma_i8(tmem_base + buf * BN, a_desc, b_desc, j != 0);
        const bool last = (kt == p.tiles32 - 1);
        if (j == p.tiles_per_acc - 1 || last) tc_commit(bar_tfull + 8 * buf);
        if (sub == 3 || last) tc_commit(bar_empty + 8 * s);
      }
    }
  } else {
    // ------------------------------ epilogue warps ----------------------------
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;       // which 128 columns of the accumulator
    const int row = q * 32 + lane;
    const int64_t gm = (int64_t)m0 + row;
    const int64_t gn0 = (int64_t)n0 + half * 128;
    int S[128];
#pragma unroll
    for (int i = 0; i < 128; ++i) S[i] = 0;
    const int r = p.acc_shift, lo = p.lo, hi = p.hi;
    bool ok = true;
    for (int acc = 0; acc < num_acc; ++acc) {
      const int buf = acc & 1;
      if (!mbar_wait(bar_tfull + 8 * buf, (acc >> 1) & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * 128);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t v[32];
        HDQT_TMEM_LD32(taddr + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int ct = acc_quant<kShift>((int)v[i], r, lo, hi);
          S[c * 32 + i] += ct;
          if (kTilesOut) {
            const int64_t n = gn0 + c * 32 + i;
            if (gm < p.M && n < p.N) {
              const int64_t off = ((int64_t)acc * p.M + gm) * p.N + n;
              if (p.tiles_elem_bytes == 1) reinterpret_cast<int8_t*>(p.tiles_out)[off] = (int8_t)ct;
              else reinterpret_cast<int16_t*>(p.tiles_out)[off] = (int16_t)ct;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
    }
    if (ok && gm < p.M) {
      const float scale = (float)((double)__ldg(p.step_a) * (double)__ldg(p.step_b) *
                                  (double)(1u << p.acc_shift) / (double)p.had_block);
      float* orow = p.out + gm * p.ld_out;
      const bool vec = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) &&
                       (gn0 + 128 <= p.N);
      if (vec) {
#pragma unroll
        for (int i = 0; i < 128; i += 4) {
          float4 o;
          o.x = __fmul_rn((float)S[i], scale);
          o.y = __fmul_rn((float)S[i + 1], scale);
          o.z = __fmul_rn((float)S[i + 2], scale);
          o.w = __fmul_rn((float)S[i + 3], scale);
          *reinterpret_cast<float4*>(orow + gn0 + i) = o;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          if (gn0 + i < p.N) orow[gn0 + i] = __fmul_rn((float)S[i], scale);
        }
      }
      if (p.S_out != nullptr) {
        int32_t* srow = p.S_out + gm * p.N;
#pragma unroll
        for (int i = 0; i < 128; ++i) {
          if (gn0 + i < p.N) srow[gn0 + i] = S[i];
        }
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

template <bool kShift, bool kTilesOut>
hdqt_status_t launch_variant(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& p, dim3 grid,
                             cudaStream_t s) {
  auto kern = gemm_i8_tiled_kernel<kShift, kTilesOut>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return HDQT_ERR_CUDA;
  kern<<<grid, GEMM_THREADS, SMEM_BYTES, s>>>(ma, mb, p);
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}

}  // namespace

}  // namespace hdqt

using namespace hdqt;

extern "C" size_t hdqt_gemm_i8_workspace_bytes(int64_t, int64_t, int64_t) { return 256; }

extern "C" hdqt_status_t hdqt_gemm_i8_tiled(const int8_t* Aq, const int8_t* Bq, const float* step_a,
                                            const float* step_b, int64_t M, int64_t N, int64_t K_pad,
                                            int32_t acc_bits, int32_t acc_tile, int32_t acc_shift,
                                            int32_t had_block, float* out, int64_t ld_out, int32_t* S_out,
                                            void* tiles_out, int32_t tiles_elem_bytes, const int32_t* norms_a,
                                            const int32_t* norms_b, uint32_t flags, void* workspace,
                                            size_t workspace_bytes, int32_t* dev_status, void* stream) {
  (void)norms_a; (void)norms_b; (void)flags; (void)workspace;
  if (!Aq || !Bq || !step_a || !step_b || !out) return HDQT_ERR_INVALID_ARG;
  if (M <= 0 || N <= 0 || K_pad <= 0 || ld_out < N) return HDQT_ERR_INVALID_ARG;
  if (K_pad % 32 != 0) return HDQT_ERR_INVALID_ARG;
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
  // the wide sum must fit int32: |c_t| <= 2^(b_a-1), T tiles
  const int64_t tiles32 = K_pad / 32;
  const int64_t tpa = acc_tile == 0 ? tiles32 : acc_tile / 32;
  const int64_t num_acc = (tiles32 + tpa - 1) / tpa;
  const int64_t per_tile_max = acc_bits >= 32 ? (tpa * 32 * 128 * 128) : (int64_t(1) << (acc_bits - 1));
  if (per_tile_max * num_acc > INT32_MAX || tpa * 32 * 128 * 128 > INT32_MAX) return HDQT_ERR_UNSUPPORTED;

  CUtensorMap ma, mb;
  if (!make_operand_map(&ma, Aq, M, K_pad, BM) || !make_operand_map(&mb, Bq, N, K_pad, BN)) return HDQT_ERR_CUDA;

  GemmParams p;
  p.M = M; p.N = N; p.K_pad = K_pad;
  p.tiles32 = (int32_t)tiles32;
  p.tiles_per_acc = (int32_t)tpa;
  p.acc_shift = acc_shift;
  p.lo = acc_bits >= 32 ? INT32_MIN : -(1 << (acc_bits - 1));
  p.hi = acc_bits >= 32 ? INT32_MAX : (1 << (acc_bits - 1)) - 1;
  p.had_block = had_block;
  p.step_a = step_a; p.step_b = step_b;
  p.out = out; p.ld_out = ld_out; p.S_out = S_out;
  p.tiles_out = tiles_out; p.tiles_elem_bytes = tiles_elem_bytes;
  p.dev_status = dev_status;

  const dim3 grid((unsigned)((M + BM - 1) / BM), (unsigned)((N + BN - 1) / BN));
  if (grid.y > 65535) return HDQT_ERR_UNSUPPORTED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (tiles_out) {
    return acc_shift ? launch_variant<true, true>(ma, mb, p, grid, s) : launch_variant<false, true>(ma, mb, p, grid, s);
  }
  return acc_shift ? launch_variant<true, false>(ma, mb, p, grid, s) : launch_variant<false, false>(ma, mb, p, grid, s);
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
