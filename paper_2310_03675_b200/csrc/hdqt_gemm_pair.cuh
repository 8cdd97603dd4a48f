// Work split for large problems: classification of 256 x 256 pair blocks, the cta_group::2 kernel for blocks
// whose tiles are (nearly) all certified clamp-free, and the fix-up pass for their few uncertified tiles.  Included by hdqt_gemm.cu.
#pragma once

#include "hdqt_gemm_device.cuh"
#include "hdqt_gemm_general.cuh"

namespace hdqt {

namespace {

// ---- work split for large problems ---------------------------------------------------------------
// A 256 x 256 "pair block" whose every K tile carries a clamp-free certificate needs no clamp path at all:
// such blocks go to the cta_group::2 kernel below (two accumulators of 256 columns, used alternately, so a
// block's drain overlaps the next block's main loop); all other blocks go to the general kernel above as two
// 128 x 256 blocks.  Two small kernels build the two work lists.

constexpr int PAIR_M = 2 * BM;
// Pair blocks are walked in groups of PAIR_GROUP_M block rows: the CTA pairs that run together then share few
// enough operand panels (all of K) for the L2 to keep them between one wave of blocks and the next.
#ifndef HDQT_PAIR_GROUP_M
#define HDQT_PAIR_GROUP_M 16
#endif
constexpr int PAIR_GROUP_M = HDQT_PAIR_GROUP_M;

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
  tile_coords<PAIR_GROUP_M>(t, tiles_m2, tiles_n, tm, tn);
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
      tile_coords<PAIR_GROUP_M>(t, tiles_m2, tiles_n, tm, tn);
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
    tile_coords<PAIR_GROUP_M>(t & ~kFixFlag, tiles_m2, tiles_n, tm, tn);
    return (t & kFixFlag) != 0;
  };

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------
    if (lane == 0) {
      uint32_t it = 0;           // stages issued so far (for the drain after a timeout)
      uint32_t ps = 0, pe_par = 1u;   // stage slot and the parity its "empty" barrier is waited on with
      bool ok = true;
      for (int i = pair_id; i < num_blocks && ok; i += num_pairs) {
        int tm, tn;
        block_at(i, tm, tn);
        const int a_row0 = tm * PAIR_M + (int)cta_rank * BM;
        const int b_row0 = tn * BN + (int)cta_rank * (BN / 2);
        for (int kb = 0; kb < num_kblocks; ++kb, ++it) {
          if (!mbar_try_wait(bar_empty + 8 * ps, pe_par) && !mbar_wait(bar_empty + 8 * ps, pe_par, abort_flag)) { ok = false; break; }
          if (leader) mbar_expect_tx(bar_full + 8 * ps, 2 * P_STAGE_BYTES);   // collects both CTAs' bytes
          const uint32_t dst = smem_base + ps * P_STAGE_BYTES;
          tma_load_2d_pair(dst, &map_a, kb * BKB, a_row0, bar_full + 8 * ps);
          tma_load_2d_pair(dst + A_STAGE, &map_b, kb * BKB, b_row0, bar_full + 8 * ps);
          if (++ps == P_STAGES) { ps = 0; pe_par ^= 1u; }
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
      // The tensor pipe takes one MMA while it works on another, so whatever this thread does between the last MMA
      // of a stage and the first of the next must fit into one MMA's time: stage index, barrier addresses, parity and
      // descriptors advance incrementally (no division by the stage count, no descriptor rebuilt), and whole stages
      // take no test on the tile count.
      const uint64_t da0 = make_smem_desc(smem_base), db0 = make_smem_desc(smem_base + A_STAGE);
      uint64_t da = da0, db = db0;
      uint32_t s = 0, full_par = 0u;
      uint32_t fb = bar_full, eb = bar_empty;
      const int full_stages = p.tiles32 >> 2;
      int bi = 0;
      bool ok = true;
      auto next_stage = [&]() {
        if (++s == P_STAGES) {
          s = 0; full_par ^= 1u; da = da0; db = db0; fb = bar_full; eb = bar_empty;
        } else {
          da += (uint64_t)(P_STAGE_BYTES >> 4); db += (uint64_t)(P_STAGE_BYTES >> 4); fb += 8; eb += 8;
        }
      };
      for (int i = pair_id; i < num_blocks && ok; i += num_pairs, ++bi) {
        const int buf = bi & 1;
        if (!mbar_wait(bar_tempty + 8 * buf, (((uint32_t)bi >> 1) & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        uint32_t acc = 0u;
        for (int kb = 0; kb < full_stages; ++kb) {
          if (s == 0 && kb + P_STAGES <= full_stages) {
            // one turn of the stage ring with every address a compile-time offset
#pragma unroll
            for (int j = 0; j < P_STAGES; ++j) {
              if (!mbar_try_wait(bar_full + 8 * j, full_par) && !mbar_wait(bar_full + 8 * j, full_par, abort_flag)) { ok = false; break; }
              tc_fence_after();
              const uint64_t o = (uint64_t)(j * (P_STAGE_BYTES >> 4));
              tc_mma_i8_pair(d_tmem, da0 + o, db0 + o, acc);
              tc_mma_i8_pair(d_tmem, da0 + o + 2, db0 + o + 2, 1u);
              tc_mma_i8_pair(d_tmem, da0 + o + 4, db0 + o + 4, 1u);
              tc_mma_i8_pair(d_tmem, da0 + o + 6, db0 + o + 6, 1u);
              acc = 1u;
              tc_commit_pair(bar_empty + 8 * j);
            }
            if (!ok) break;
            full_par ^= 1u;
            kb += P_STAGES - 1;
            continue;
          }
          if (!mbar_try_wait(fb, full_par) && !mbar_wait(fb, full_par, abort_flag)) { ok = false; break; }
          tc_fence_after();
          tc_mma_i8_pair(d_tmem, da, db, acc);
          tc_mma_i8_pair(d_tmem, da + 2, db + 2, 1u);
          tc_mma_i8_pair(d_tmem, da + 4, db + 4, 1u);
          tc_mma_i8_pair(d_tmem, da + 6, db + 6, 1u);
          acc = 1u;
          tc_commit_pair(eb);
          next_stage();
        }
        if (ok && full_stages < num_kblocks) {       // ragged last stage
          if (!mbar_wait(fb, full_par, abort_flag)) { ok = false; break; }
          tc_fence_after();
          for (int sub = 0; full_stages * 4 + sub < p.tiles32; ++sub)
            tc_mma_i8_pair(d_tmem, da + 2 * sub, db + 2 * sub, (acc != 0u || sub > 0) ? 1u : 0u);
          tc_commit_pair(eb);
          next_stage();
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
    e.scale = scale;
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
// exactly those tile sums P (warp-level mma.sync m16n8k32 on staged 32-byte K slices) and adds clamp(P) - P;
// the result is sum_t clamp(P_t) bit for bit (on certified tiles the clamp is the identity).  Then it applies
// the dequantising scale.
// Work item = 64 rows of a 256 x 256 block (4 items per block, so that the few blocks spread over all SMs),
// 256 threads.  Corrections are rare, so they are added to the parked sums in place as they are found; the
// final conversion walks the item with warp w on rows 8w..8w+7 and lane l on the columns l + 32 j.
constexpr int FIX_ROWS = 64;
constexpr int kMaxFixTiles = 256;   // the classification sends blocks with more uncertified tiles to the general kernel
constexpr int FIX_B_STRIDE = 48;    // bytes per staged B row (32 + 16: the fragment loads of 8 rows x 4 lanes hit 32 banks)

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
    tile_coords<PAIR_GROUP_M>(__ldg(list_fix + item / (PAIR_M / FIX_ROWS)), tiles_m2, tiles_n, tm, tn);
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
      // exact tile sums on the (legacy) int8 tensor path: warp w owns rows 16 (w & 3) .. +15 and the 128
      // columns of half (w >> 2), as 16 m16n8k32 tiles; C[nt] = rows (g, g + 8) x columns 8 nt + 2 tig, + 1
      int Cf[16][4];
#pragma unroll
      for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) Cf[nt][i] = 0;
      const int g = lane >> 2, tig = lane & 3;
      const int arow = (warp & 3) * 16 + g, col_half = (warp >> 2) * 128;
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
            *reinterpret_cast<uint2*>(sB + brow * FIX_B_STRIDE + part * 8) = vb;
          }
        }
        __syncthreads();
        // A fragment: (row g, k 4 tig..), (row g + 8, same k), then the same rows at k + 16
        const int a0 = *reinterpret_cast<const int*>(sA + arow * 32 + tig * 4);
        const int a1 = *reinterpret_cast<const int*>(sA + (arow + 8) * 32 + tig * 4);
        const int a2 = *reinterpret_cast<const int*>(sA + arow * 32 + 16 + tig * 4);
        const int a3 = *reinterpret_cast<const int*>(sA + (arow + 8) * 32 + 16 + tig * 4);
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
          // B fragment: column n = 8 nt + g of the tile (= row n of the code matrix), k 4 tig.. and k + 16
          const uint8_t* brow = sB + (col_half + nt * 8 + g) * FIX_B_STRIDE;
          const int b0 = *reinterpret_cast<const int*>(brow + tig * 4);
          const int b1 = *reinterpret_cast<const int*>(brow + 16 + tig * 4);
          asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                       : "+r"(Cf[nt][0]), "+r"(Cf[nt][1]), "+r"(Cf[nt][2]), "+r"(Cf[nt][3])
                       : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
      }
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int64_t gm = m0 + arow + (i >> 1) * 8;
          const int64_t gn = n0 + col_half + nt * 8 + tig * 2 + (i & 1);
          const int P = Cf[nt][i];
          const int d = min(max(P, p.lo), p.hi) - P;
          if (d != 0 && gm < p.M && gn < p.N) {
            int* o = reinterpret_cast<int*>(p.out + gm * p.ld_out + gn);   // only this thread touches this element
            *o += d;
          }
        }
      }
    }
    __syncthreads();   // the corrections above and the conversion below use different thread-to-element maps
    // parked (now exact) integer sums -> fp32, lanes on consecutive columns; all loads first, so that
    // they are in flight together (each element is touched by this thread only)
    const bool vec4 = ((p.ld_out & 3) == 0) && ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (n0 + BN <= p.N) &&
                      (m0 + FIX_ROWS <= p.M) && p.S_out == nullptr;      // block-uniform
    if (vec4) {
      // whole 64 x 256 item inside the matrix: 16-byte accesses, lane l on columns 4 l .. 4 l + 3 (+ 128)
      int4 Sq[8][2];
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const float* row = p.out + (m0 + warp * 8 + r) * p.ld_out + n0 + 4 * lane;
        Sq[r][0] = __ldcg(reinterpret_cast<const int4*>(row));
        Sq[r][1] = __ldcg(reinterpret_cast<const int4*>(row + 128));
      }
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        float* row = p.out + (m0 + warp * 8 + r) * p.ld_out + n0 + 4 * lane;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int64_t gn = n0 + 4 * lane + 128 * h;
          float4 o;
          o.x = finish1(p, __fmul_rn((float)Sq[r][h].x, scale), gn);
          o.y = finish1(p, __fmul_rn((float)Sq[r][h].y, scale), gn + 1);
          o.z = finish1(p, __fmul_rn((float)Sq[r][h].z, scale), gn + 2);
          o.w = finish1(p, __fmul_rn((float)Sq[r][h].w, scale), gn + 3);
          *reinterpret_cast<float4*>(row + 128 * h) = o;
        }
      }
      __syncthreads();
      continue;
    }
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
          p.out[gm * p.ld_out + gn] = finish1(p, __fmul_rn((float)Sv[r][j], scale), gn);
          if (p.S_out != nullptr) p.S_out[gm * p.N + gn] = Sv[r][j];
        }
      }
    }
    __syncthreads();
  }
}

}  // namespace

}  // namespace hdqt
