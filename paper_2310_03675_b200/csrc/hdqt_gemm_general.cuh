// General tiled integer GEMM kernel: persistent single-CTA blocks of 128 x 256 with a clamp path (every tile
// through the low-bit accumulator epilogue) and per-block merging of certified tiles.  Included by hdqt_gemm.cu.
#pragma once

#include "hdqt_gemm_device.cuh"

namespace hdqt {

namespace {


// ---- the kernel -----------------------------------------------------------------------------
// Persistent: one CTA per SM walks over output blocks (block index = blockIdx.x + i*gridDim.x), so that the
// TMA producer runs ahead into the next block while the epilogue warps drain the previous one, and the
// per-block fixed costs (TMEM allocation, barrier set-up, pipeline fill) are paid once.
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer, 2 = certificate builder (clamp-free tile bitmask of the
// next block, from the tile norms), 3 = spare (completes the control warp group), 4..11 = epilogue (TMEM lane
// quarter = warp % 4, 128 columns each).  The control warp group hands most of its registers to the two
// epilogue warp groups (setmaxnreg), which hold the sums of 128 columns plus two TMEM load buffers.
//
// kPacked: the per-tile sums fit 16 bits and b_a <= 8, r = 0: TMEM is read with two columns packed
//          per register, clamp and add work on 16-bit lane pairs (half the ALU work per element).
// kDeep:   with kPacked, for contractions longer than flush_every tiles: two-level lane sums (see epilogue_packed).
// kMerge:  false = the launch merges no tiles; the merged paths are compiled out.
// kAtomic: false = no split-K work items in the launch; the atomic store path is compiled out (packed variants).
// otherwise: one 32-bit register per accumulator element, any b_a and r.

struct TileInfo {                       // what the certificate warp publishes per output block
  uint32_t mask[MAX_CERT_WORDS];        // bit a: accumulator tile a provably cannot clamp
  int32_t n_uncert;                     // accumulator tiles without a certificate
  int32_t pad[3];
};
static_assert(sizeof(TileInfo) == TILE_INFO_BYTES, "TileInfo layout");

template <int GROUP_M = 16>
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tile_m, int& tile_n) {
  // grouped order: co-resident CTAs form a roughly square patch (16 row blocks x ~9 column blocks on
  // 148 SMs), so both operands' panels are shared through L2
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

template <bool kPacked, bool kShift, bool kTilesOut, bool kDeep = false, bool kMerge = true, bool kAtomic = true>
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

  // kMerge = false (launches in which no tile is merged): all code of the merged paths drops out.  The per-tile
  // loops of the clamp path are sensitive to the size of the code around them (removing the unused staging-box
  // store of the merged-only epilogue from the long-contraction variant alone was worth 13 %).
  const int merge_mode = kMerge ? p.merge : 0;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int tiles_m = (int)((p.M + BM - 1) / BM), tiles_n = (int)((p.N + BN - 1) / BN);
  const int num_tiles = (p.block_list != nullptr) ? __ldg(p.block_count) : tiles_m * tiles_n;
  const int num_kblocks = (p.tiles32 + 3) >> 2;
  const int num_acc = p.num_acc;
  if (num_tiles == 0) return;   // an empty work list (uniform over the grid): nothing to set up or tear down
  // Split-K (host-selected for long contractions with few output blocks, clamp path only): a work item is then
  // (output block, K range of split_kblocks stages); the integer sums of the ranges are added up in the output
  // buffer with atomics (exact and order-free) and a small kernel applies the scale afterwards.
  const int split_k = p.split_k > 1 ? p.split_k : 1;
  const int num_items = num_tiles * split_k;
  struct ItemRange { int blk, kb_lo, kb_hi, t_end, n_acc; };
  auto item_range = [&](int item) {
    ItemRange r{item, 0, num_kblocks, p.tiles32, num_acc};
    if (split_k > 1) {
      r.blk = item / split_k;
      r.kb_lo = (item - r.blk * split_k) * p.split_kblocks;
      r.kb_hi = min(num_kblocks, r.kb_lo + p.split_kblocks);
      r.t_end = min(p.tiles32, r.kb_hi * 4);
      r.n_acc = (r.t_end - r.kb_lo * 4 + p.tiles_per_acc - 1) / p.tiles_per_acc;
    }
    return r;
  };

  if (threadIdx.x == 0) {
    // the first TMA load would otherwise wait for its descriptor: fetch both while the CTA sets itself up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
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
  if (p.offset_mma) {
    // Constant operand tiles of the offset MMA: every 16-byte K chunk of the A tile holds o/2 in its first
    // byte and zeros, every byte of the B tile is 1, so that a 32-byte K slice of any row pair multiplies to
    // o = 2^(b_a-1), wherever the 8-row groups and K chunks of the descriptor fall inside the tiles.
    const uint32_t half_off = (uint32_t)(-(p.lo / 2));
    uint4* ca = reinterpret_cast<uint4*>(smem_al + OFFS_A_OFF);
    uint4* cb = reinterpret_cast<uint4*>(smem_al + OFFS_B_OFF);
    for (int i = threadIdx.x; i < OFFS_A_BYTES / 16; i += GEMM_THREADS) ca[i] = make_uint4(half_off, 0u, 0u, 0u);
    for (int i = threadIdx.x; i < OFFS_B_BYTES / 16; i += GEMM_THREADS)
      cb[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads them through the async proxy
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // A block merges its certified tiles only when few tiles need the clamp path (that path is
  // single-buffered while merging).
  auto block_merges = [&](int n_uncert) {
    return (merge_mode == 2) ||
           (merge_mode == 1 && (int64_t)n_uncert * 256 <= (int64_t)p.merge_max_uncert_256 * num_acc);
  };

  if (warp < NUM_CTRL_WARPS) {
  warpgroup_reg_dec<CTRL_REGS>();
  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;   // k-blocks issued so far, over all output blocks
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_items && ok; tile += gridDim.x) {
        const ItemRange ir = item_range(tile);
        int tile_m, tile_n;
        block_coords(p, ir.blk, tiles_m, tiles_n, tile_m, tile_n);
        for (int kb = ir.kb_lo; kb < ir.kb_hi; ++kb, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t par = ((it / STAGES) & 1u) ^ 1u;
          if (!mbar_wait_suspend(bar_empty + 8 * s, par, abort_flag)) { ok = false; break; }
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
    if (merge_mode == 1) {
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
      const uint64_t desc_offs_a = make_smem_desc_plain(smem_base + OFFS_A_OFF, 128u, 256u);
      const uint64_t desc_offs_b = make_smem_desc_plain(smem_base + OFFS_B_OFF, 128u, 256u);
      const uint32_t offset_mma = (uint32_t)p.offset_mma;
      uint32_t s = 0;            // smem stage
      uint32_t full_par = 0;     // parity of the stage's next "full" phase
      uint32_t fill_par = 0u;   // bit b: parity of the times TMEM accumulator b has been handed to the epilogue
      uint64_t desc_a = desc_a0, desc_b = desc_b0;
      bool ok = true;
      const int tpa = p.tiles_per_acc;
      bool ready = false;
      int ti = 0;
      for (int tile = blockIdx.x; tile < num_items && ok; tile += gridDim.x, ++ti) {
        const ItemRange ir = item_range(tile);
        const int tiles32 = ir.t_end;      // end of this item's K range, in 32-wide tiles
        const int num_acc = ir.n_acc;      // (shadows the block-wide count: accumulator tiles of this item)
        const int slot = ti & 1;
        int n_uncert = (merge_mode == 2) ? 0 : num_acc;
        if (merge_mode == 1) {
          if (!mbar_wait(bar_ifull + 8 * slot, ((uint32_t)ti >> 1) & 1u, abort_flag)) { ok = false; break; }
          n_uncert = *reinterpret_cast<volatile int32_t*>(&tile_info[slot].n_uncert);
        }
        const bool merging = block_merges(n_uncert);
        const int n_merged = merging ? num_acc - n_uncert : 0;
        const uint32_t* cert_mask = tile_info[slot].mask;
        const bool nibble_ok = (merge_mode == 2) || (merging && merge_mode == 1 && tpa == 1);
        int j = 0;                 // position inside the current accumulator tile
        int acc = 0;               // accumulator tile index
        int clamp_idx = 0;         // index among this block's tiles that take the clamp path
        bool cert = (merge_mode == 2);
        uint32_t merged_started = 0;
        uint32_t d_tmem = tmem_base;
        int cur_buf = 0;
        for (int kb = ir.kb_lo; kb < ir.kb_hi; ++kb) {
          if (!ready && !mbar_wait(bar_full + 8 * s, full_par, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t s_next = (s + 1 == STAGES) ? 0u : s + 1;
          const uint32_t par_next = (s + 1 == STAGES) ? (full_par ^ 1u) : full_par;
          const int kt0 = kb * 4;
          uint32_t nib = 0;
          if (merge_mode == 2) nib = 0xFu;
          else if (nibble_ok) nib = (cert_mask[kb >> 3] >> ((kb & 7) * 4)) & 0xFu;
          if (!merging && tpa == 1 && offset_mma && kt0 + 4 <= tiles32 && (clamp_idx & 1) == 0) {
            // A whole stage of clamp-path tiles, straight-line: this thread's instructions are the pace of the
            // ring (each costs it tens of clocks beside the epilogue warps of its scheduler), so accumulator,
            // K slice and barrier parity of the four tiles are compile-time constants.  Each accumulator is
            // handed over twice per stage, which leaves the hand-over parities as they were.
            const uint32_t p0 = (fill_par & 1u) ^ 1u, p1 = ((fill_par >> 1) & 1u) ^ 1u;
#pragma unroll
            for (int sub = 0; sub < 4; ++sub) {
              const uint32_t b = (uint32_t)sub & 1u;
              const uint32_t par = (b ? p1 : p0) ^ (uint32_t)(sub >> 1);
              if (!mbar_wait_suspend(bar_tempty + 8 * b, par, abort_flag)) { ok = false; break; }
              tc_fence_after();
              HDQT_TL(0, clamp_idx + sub);
              tc_mma_i8_new(tmem_base + b * BN, desc_offs_a, desc_offs_b);
              tc_mma_i8_acc(tmem_base + b * BN, desc_a + (uint64_t)(2 * sub), desc_b + (uint64_t)(2 * sub));
              HDQT_TL(1, clamp_idx + sub);
              tc_commit(bar_tfull + 8 * b);
            }
            if (!ok) break;
            clamp_idx += 4;
          } else if (!merging && tpa == 1 && offset_mma) {
            // Every tile of this block takes the clamp path of the 16-bit-lane epilogue: a short, branch-free
            // sequence per tile.  (This thread shares its scheduler with two epilogue warps; every instruction
            // it spends between two tiles is taken from them, and they are the slowest of the eight.  Issuing
            // the odd tiles from a second thread on another scheduler was tried: the lag moved to that
            // scheduler's warps and the tile rate stayed the same.)
            const int nsub = min(tiles32 - kt0, 4);
            for (int sub = 0; sub < nsub; ++sub) {
              const uint32_t b = (uint32_t)clamp_idx & 1u;
              if (!mbar_wait_suspend(bar_tempty + 8 * b, ((fill_par >> b) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
              tc_fence_after();
              HDQT_TL(0, clamp_idx);
              const uint32_t d = tmem_base + b * BN;
              tc_mma_i8(d, desc_offs_a, desc_offs_b, 0u);
              tc_mma_i8(d, desc_a + (uint64_t)(2 * sub), desc_b + (uint64_t)(2 * sub), 1u);
              HDQT_TL(1, clamp_idx);
              tc_commit(bar_tfull + 8 * b);
              fill_par ^= 1u << b;
              ++clamp_idx;
            }
            if (!ok) break;
          } else if (nib == 0xFu && kt0 + 4 <= tiles32) {
            if (!merged_started) {
              // the merged accumulator (buffer 0) must have been drained by the previous user
              if (!mbar_wait(bar_tempty, (fill_par & 1u) ^ 1u, abort_flag)) { ok = false; break; }
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
                if (merge_mode == 2) {
                  cert = true;
                } else if (merging) {
                  cert = (cert_mask[acc >> 5] >> (acc & 31)) & 1u;
                }
                // merged tiles accumulate in buffer 0; clamp tiles use buffer 1 when merging, else 0 / 1
                cur_buf = cert ? 0 : (merging ? 1 : (clamp_idx & 1));
                if (!cert || !merged_started) {
                  if (!mbar_wait_suspend(bar_tempty + 8 * cur_buf, ((fill_par >> cur_buf) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                  tc_fence_after();
                }
                d_tmem = tmem_base + cur_buf * BN;
                if (!cert) HDQT_TL(0, clamp_idx);
                // a clamp-path tile of the 16-bit-lane epilogue starts from the constant 2^(b_a-1)
                if (!cert && offset_mma) tc_mma_i8(d_tmem, desc_offs_a, desc_offs_b, 0u);
              }
              uint32_t sub2 = (uint32_t)(2 * (kt - kt0));
              uint32_t accumulate = cert ? merged_started : ((uint32_t)(j != 0) | offset_mma);
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
                  HDQT_TL(1, clamp_idx);
                  tc_commit(bar_tfull + 8 * cur_buf);
                  fill_par ^= 1u << cur_buf;
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
          fill_par ^= 1u;
        }
        if (merge_mode == 1) mbar_arrive(bar_iempty + 8 * slot);
      }
    }
  }
  } else {
    // ------------------------------ epilogue warps ----------------------------
    warpgroup_reg_inc<EPI_REGS>();
    EpiCtx e;
    e.q = warp & 3;                     // TMEM lane quarter this warp may read
    e.grp = (warp - NUM_CTRL_WARPS) >> 2;   // which EPI_COLS columns of the accumulator
    e.lane = lane;
    e.lane_addr = tmem_base + ((uint32_t)(e.q * 32) << 16) + (uint32_t)(e.grp * EPI_COLS);
    e.bar_tfull = bar_tfull;
    e.bar_tempty = bar_tempty;
    e.abort_flag = abort_flag;
    e.box = reinterpret_cast<float*>(smem_al + OUT_STAGE_OFF + (warp - NUM_CTRL_WARPS) * OUT_STAGE_WARP);
    e.scale = dequant_scale(p);
    uint32_t drain_par = 0u;            // bit b: parity of the times this warp has drained accumulator b
    int ti = 0;
    for (int tile = blockIdx.x; tile < num_items; tile += gridDim.x, ++ti) {
      const ItemRange ir = item_range(tile);
      const int slot = ti & 1;
      int n_uncert = (merge_mode == 2) ? 0 : ir.n_acc;
      if (merge_mode == 1) {
        if (!mbar_wait_yield<128>(bar_ifull + 8 * slot, ((uint32_t)ti >> 1) & 1u, abort_flag)) break;
        n_uncert = *reinterpret_cast<volatile int32_t*>(&tile_info[slot].n_uncert);
      }
      BlockJob job;
      job.merging = block_merges(n_uncert) ? 1 : 0;
      job.n_clamp_tiles = job.merging ? n_uncert : ir.n_acc;
      job.n_merged = job.merging ? ir.n_acc - n_uncert : 0;
      job.atomic = split_k > 1 ? 1 : 0;
      int tile_m, tile_n;
      block_coords(p, ir.blk, tiles_m, tiles_n, tile_m, tile_n);
      job.m0 = tile_m * BM;
      job.n0 = tile_n * BN;
      bool ok;
      if (kMerge && job.n_clamp_tiles == 0 && job.n_merged > 0) ok = epilogue_merged_only<kDeep>(p, e, job, drain_par);
      else if (kPacked) ok = epilogue_packed<kDeep, kMerge, kAtomic>(p, e, job, drain_par);
      else ok = epilogue_wide<kShift, kTilesOut>(p, e, job, drain_par);
      if (!ok) break;
      if (merge_mode == 1) {
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

}  // namespace

}  // namespace hdqt
