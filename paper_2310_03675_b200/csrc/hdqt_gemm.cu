// Tiled integer GEMM with low-bit per-tile accumulators on the sm_100a tensor cores
// (paper Section 3, last paragraph: "tiled quantization ... tiles of size s"; Section 4:
// accumulator block size 32; Section 4.2: 8-bit accumulators in forward and backward pass).
//
//   P_t[m,n] = sum_{k in tile t} Aq[m,k]*Bq[n,k]   one tcgen05.mma.kind::i8 per 32 k (exact, s32 in TMEM)
//   c_t      = clamp(rne(P_t / 2^r), -2^(b_a-1), 2^(b_a-1)-1)            epilogue warps, registers
//   S        = sum_t c_t                                                   int32 registers
//   out      = fp32(S) * fp32(step_a*step_b*2^r / n_h)
//
// This translation unit holds the host side (argument checks, tensor maps, kernel selection) and the
// calibration utility; the kernels live in the headers it includes:
//   hdqt_gemm_device.cuh   tile constants, parameters, PTX wrappers, per-block epilogues
//   hdqt_gemm_general.cuh  general kernel: persistent CTAs over 128 x 256 blocks; warp 0 feeds a shared-memory
//                          ring with TMA, warp 1 issues the MMAs into two TMEM accumulators, warp 2 builds the
//                          clamp-free certificates of the next block, 8 epilogue warps drain the accumulators,
//                          apply the accumulator quantisation per tile and keep the wide sums in registers
//   hdqt_gemm_pair.cuh     large problems: block classification, cta_group::2 kernel for certified 256 x 256
//                          blocks, fix-up pass for blocks with a few uncertified tiles
// Tiles that provably cannot clamp (Cauchy-Schwarz bound from per-tile code norms) may be
// accumulated together in TMEM: the clamp is the identity there, so the integers are unchanged.
// Every wait is bounded; when one runs out the CTA records HDQT_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include <string.h>

#include "hdqt_common.cuh"
#include "hdqt_gemm_device.cuh"
#include "hdqt_gemm_general.cuh"
#include "hdqt_gemm_pair.cuh"

namespace hdqt {

namespace {

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

// ---- self-test of the bounded waits ------------------------------------------------------------
// Both wait forms of the GEMM kernels, on a barrier that nothing ever arrives at, with a poll budget of about a
// millisecond instead of the kernels' second: each must give up, raise the block's abort flag and let the
// block end normally with HDQT_ERR_TIMEOUT in the status word.  No TMA copy or tensor-core operation is in
// flight, so there is nothing to drain.
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(int32_t* dev_status, int32_t* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, 1 << 10);          // spin, then back off
  if (threadIdx.x >= 32) ok = mbar_wait_yield<64>(smem_u32(&bar), 0u, &abort_flag, 1 << 12);   // suspend and sleep
  if (!ok && gave_up != nullptr) atomicAdd(gave_up, 1);
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) report_status(dev_status, HDQT_ERR_TIMEOUT);
}

// ---- tensor-pipe yardstick: back-to-back MMAs of the shape the GEMM kernels use, operands resident ----
// One CTA per SM, one thread issues `iters` tcgen05.mma.kind::i8 M128 N256 K32 into one accumulator from four
// K slices of a zero-filled shared-memory stage; no loads, no epilogue.  Timed by the caller, it gives the
// integer tensor rate this chip reaches at its current clocks: the ceiling the GEMM kernels are compared with.
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int iters, int32_t* dev_status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const uint32_t base = smem_u32(smem_raw);
  if (base & 1023u) {
    if (threadIdx.x == 0) report_status(dev_status, HDQT_ERR_CUDA);
    return;
  }
  for (int i = threadIdx.x; i < STAGE_BYTES / 16; i += blockDim.x) reinterpret_cast<uint4*>(smem_raw)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(BN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  if (threadIdx.x == 32) {
    const uint64_t da = make_smem_desc(base), db = make_smem_desc(base + A_STAGE);
    for (int it = 0; it < iters; ++it) {
      const uint64_t k = (uint64_t)(2 * (it & 3));
      tc_mma_i8(tmem, da + k, db + k, it > 0 ? 1u : 0u);
    }
    tc_commit(smem_u32(&bar));
    if (!mbar_wait(smem_u32(&bar), 0u, &abort_flag)) report_status(dev_status, HDQT_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(BN) : "memory");
  }
}

// ---- split-K: integer sums parked in the output buffer -> fp32 result (and optional integer output) ----
__global__ void split_k_finalize_kernel(const GemmParams p) {
  const float scale = dequant_scale(p);
  const int64_t total = p.M * p.N;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t m = i / p.N, n = i - m * p.N;
    float* o = p.out + m * p.ld_out + n;
    const int S = __float_as_int(*o);
    *o = finish1(p, __fmul_rn((float)S, scale), n);
    if (p.S_out != nullptr) p.S_out[i] = S;
  }
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

template <bool kPacked, bool kShift, bool kTilesOut, bool kDeep = false, bool kMerge = true, bool kAtomic = true>
hdqt_status_t launch_variant(const CUtensorMap& ma, const CUtensorMap& mb, const GemmParams& p, dim3 grid,
                             cudaStream_t s) {
  auto kern = gemm_i8_tiled_kernel<kPacked, kShift, kTilesOut, kDeep, kMerge, kAtomic>;
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
  return hdqt::gemm_i8_tiled_impl(Aq, Bq, step_a, step_b, M, N, K_pad, code_bits, acc_bits, acc_tile, acc_shift,
                                  had_block, out, ld_out, S_out, tiles_out, tiles_elem_bytes, norms_a, norms_b, flags,
                                  nullptr, workspace, workspace_bytes, dev_status, stream);
}

hdqt_status_t hdqt::gemm_i8_tiled_impl(const int8_t* Aq, const int8_t* Bq, const float* step_a,
                                       const float* step_b, int64_t M, int64_t N, int64_t K_pad,
                                       int32_t code_bits, int32_t acc_bits, int32_t acc_tile,
                                       int32_t acc_shift, int32_t had_block, float* out, int64_t ld_out,
                                       int32_t* S_out, void* tiles_out, int32_t tiles_elem_bytes,
                                       const int32_t* norms_a, const int32_t* norms_b, uint32_t flags,
                                       const float* bias, void* workspace, size_t workspace_bytes,
                                       int32_t* dev_status, void* stream) {
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
  p.bias = bias;
  p.relu = (flags & HDQT_FLAG_RELU) ? 1 : 0;

  // 16-bit-lane epilogue: tile sums fit int16, the offset sums fit uint16 for flush_every tiles
  // (the epilogue forms P + 2^(b_a-1) in signed 16-bit lanes before it takes the minimum)
  const bool packed = !tiles_out && acc_shift == 0 && acc_bits <= 8 && p_max + ((int64_t)p.hi + 1) <= 32767;
  p.offset_mma = packed ? 1 : 0;
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
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

  // Split-K: a long contraction with few output blocks (the weight gradient of a convolution: K = batch x
  // positions) would leave most SMs idle.  Only where every tile takes the clamp path anyway (no merging), in
  // whole shared-memory stages and whole accumulator tiles; with the 16-bit-lane epilogue a work item stays
  // within one widening period.  Integer addition is exact and order-free, so the result is unchanged.
  p.split_k = 1;
  p.split_kblocks = 0;
  if (p.merge == 0 && !tiles_out && num_blocks * 2 <= sms && (flags & HDQT_FLAG_NO_SPLIT_K) == 0) {
    const int64_t unit = (tpa % 4 == 0) ? tpa : ((tpa % 2 == 0) ? 2 * tpa : 4 * tpa);   // lcm(4, tpa) tiles
    const int64_t units = tiles32 / unit;                                              // whole units in K
    int64_t want = sms / num_blocks;
    // at least 8 stages per item (the fixed cost of an item is a few tiles' worth, and its sums are added with one
    // atomic per element), at most `want` items, and items of equal length (32 + 4 tiles is worse than 36 in one)
    const int64_t min_units = (32 + unit - 1) / unit;
    if (want > units / min_units) want = units / min_units;
    if (want < 1) want = 1;
    int64_t per_item = (units + want - 1) / want;
    if (per_item < min_units) per_item = min_units;
    if (packed && per_item * unit > (int64_t)p.flush_every * tpa) per_item = (int64_t)p.flush_every * tpa / unit;
    const int64_t items = per_item > 0 ? (tiles32 + per_item * unit - 1) / (per_item * unit) : 1;
    if (per_item > 0 && items > 1 && items <= 65535) {
      p.split_k = (int32_t)items;
      p.split_kblocks = (int32_t)(per_item * unit / 4);
    }
  }
  const int64_t num_items = num_blocks * p.split_k;
  dim3 grid((unsigned)(num_items < sms ? num_items : sms));   // persistent: one CTA per SM
  if (p.split_k > 1) {
    if (cudaMemset2DAsync(out, (size_t)ld_out * sizeof(float), 0, (size_t)N * sizeof(float), (size_t)M, s) != cudaSuccess)
      return HDQT_ERR_CUDA;
  }

  // Large problems (at least 2 output blocks per SM; below that the extra launches cost more than they gain)
  // with clamp-free tiles: the cta_group::2 kernel takes the blocks whose K tiles are all, or all but a few,
  // certified (a fix-up pass repairs the few), the general kernel takes the rest.
  const bool split = (p.merge != 0) && !tiles_out && num_blocks >= 2 * (int64_t)sms && sms >= 2 && workspace != nullptr;
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
  hdqt_status_t st;
  // The variant with a second set of lanes is needed when a work item has more clamp-path tiles than the 16-bit
  // lanes hold (up to 256 x flush_every tiles; beyond that the plain variant parks partial sums in the output
  // buffer).  It also stores the result straight from the registers, which costs a few thousand clocks more per
  // output block than the staged store but leaves a kernel with less code around the per-tile loops, and those
  // run ~4 % faster for it (measured: 893 -> 931 TOPS at 8192^3, break-even near 128 tiles): used from 128 tiles.
  const int64_t tiles_per_item = p.split_k > 1 ? (int64_t)p.split_kblocks * 4 / tpa : num_acc;
  const bool deep = packed && tiles_per_item >= 128 && tiles_per_item <= 256 * (int64_t)p.flush_every;
  if (packed && p.merge == 0 && (deep || tiles_per_item <= p.flush_every)) {
    // no merged tiles in this launch, no work item that would have to park partial sums: the lean kernels
    if (p.split_k > 1) {
      st = deep ? launch_variant<true, false, false, true, false, true>(ma, mb, p, grid, s)
                : launch_variant<true, false, false, false, false, true>(ma, mb, p, grid, s);
    } else {
      st = deep ? launch_variant<true, false, false, true, false, false>(ma, mb, p, grid, s)
                : launch_variant<true, false, false, false, false, false>(ma, mb, p, grid, s);
    }
  } else if (packed) {       // (split-K work items only exist in launches that merge nothing)
    st = deep ? launch_variant<true, false, false, true, true, false>(ma, mb, p, grid, s)
              : launch_variant<true, false, false, false, true, false>(ma, mb, p, grid, s);
  }
  else st = acc_shift ? launch_variant<false, true, false>(ma, mb, p, grid, s)
                      : launch_variant<false, false, false>(ma, mb, p, grid, s);
  if (st == HDQT_OK && p.split_k > 1) {
    const int64_t total = M * N;
    const int64_t blocks = (total + 255) / 256;
    split_k_finalize_kernel<<<(unsigned)(blocks < 4 * sms ? blocks : 4 * sms), 256, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return HDQT_ERR_CUDA;
  }
  return st;
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

extern "C" hdqt_status_t hdqt_selftest_bounded_wait(int32_t* dev_status, int32_t* gave_up, void* stream) {
  if (!dev_status) return HDQT_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 64, 0, reinterpret_cast<cudaStream_t>(stream)>>>(dev_status, gave_up);
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}

#ifdef HDQT_TIMELINE
// tuning builds only: copies the recorded event timeline (64 tiles x 16 slots of SM clock values) to the host
extern "C" int hdqt_debug_timeline(long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, g_timeline, sizeof(long long) * 64 * 16);
}
#endif

extern "C" hdqt_status_t hdqt_selftest_mma_rate(int32_t iters, int64_t* ops_out, int32_t* dev_status, void* stream) {
  if (iters <= 0 || iters > (1 << 22)) return HDQT_ERR_INVALID_ARG;
  cudaError_t e = cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, STAGE_BYTES);
  if (e != cudaSuccess) return cuda_failure(e, "cudaFuncSetAttribute(mma rate)");
  const int sms = sm_count();
  mma_rate_kernel<<<sms, 128, STAGE_BYTES, reinterpret_cast<cudaStream_t>(stream)>>>(iters, dev_status);
  if (cudaGetLastError() != cudaSuccess) return HDQT_ERR_CUDA;
  if (ops_out) *ops_out = 2ll * BM * BN * 32 * (int64_t)iters * sms;
  return HDQT_OK;
}
