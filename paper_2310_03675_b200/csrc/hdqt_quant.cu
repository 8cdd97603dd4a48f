// FWHT + calibration maximum + quantizer kernels (paper Section 3: Hadamard paragraph,
// definition of Q, stochastic rounding; Section 4: clip factor).
//
// Two memory layouts of the source operand are served:
//   * K contiguous ("kc"): a thread owns 8 consecutive k of one row; a 32-wide Hadamard
//     block is spread over 4 neighbouring lanes: strides 1,2,4 run in registers, strides 8,16
//     through warp shuffles.  Loads are 2 x 128-bit per thread, stores 64-bit per thread.
//   * K strided ("ks", the row index is contiguous): a thread owns one whole 32-wide block of
//     one row; a warp reads 32 consecutive rows per load instruction (128 bytes, coalesced),
//     all five butterfly stages run in registers, and the thread writes its 32 codes as one
//     32-byte segment of the K-contiguous code row (a fused transpose).
//
// Both are HBM-bound streaming kernels: 4 B/element read (+1 B/element written when
// quantizing).  Butterfly order is ascending stride, every add/sub is a single fp32 rounding,
// so the transformed values - and hence the codes - are bit-identical for both layouts.
#include <mutex>

#include "hdqt_common.cuh"

namespace hdqt {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// ---- butterflies ------------------------------------------------------------------------

// strides 1, 2, 4 on 8 register values (only those below had_block)
__device__ __forceinline__ void fwht8_regs(float (&x)[8], int had_block) {
  if (had_block > 1) {
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      const float a = x[i], b = x[i + 1];
      x[i] = __fadd_rn(a, b);
      x[i + 1] = __fsub_rn(a, b);
    }
  }
  if (had_block > 2) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if ((i & 2) == 0) {
        const float a = x[i], b = x[i + 2];
        x[i] = __fadd_rn(a, b);
        x[i + 2] = __fsub_rn(a, b);
      }
    }
  }
  if (had_block > 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float a = x[i], b = x[i + 4];
      x[i] = __fadd_rn(a, b);
      x[i + 4] = __fsub_rn(a, b);
    }
  }
}

// strides 8 and 16 across lanes (lane^1, lane^2); the whole warp must call this.
// The lower lane of a pair needs x + y, the upper one y - x: both are fma(sign, x, y) with sign = +-1
// (sign*x is exact, so the fused form rounds once, exactly like the add / subtract).
__device__ __forceinline__ void fwht8_lanes(float (&x)[8], int had_block, int lane) {
  if (had_block > 8) {
    const float sign = (lane & 1) ? -1.0f : 1.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float y = __shfl_xor_sync(0xFFFFFFFFu, x[i], 1);
      x[i] = __fmaf_rn(sign, x[i], y);
    }
  }
  if (had_block > 16) {
    const float sign = (lane & 2) ? -1.0f : 1.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float y = __shfl_xor_sync(0xFFFFFFFFu, x[i], 2);
      x[i] = __fmaf_rn(sign, x[i], y);
    }
  }
}

// all stages on 32 register values
__device__ __forceinline__ void fwht32_regs(float (&x)[32], int had_block) {
#pragma unroll
  for (int h = 1; h < 32; h <<= 1) {
    if (h < had_block) {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        if ((i & h) == 0) {
          const float a = x[i], b = x[i + h];
          x[i] = __fadd_rn(a, b);
          x[i + h] = __fsub_rn(a, b);
        }
      }
    }
  }
}

// ---- loads ------------------------------------------------------------------------------

// 8 consecutive k of one row, zero beyond K. `vec` = row base and stride are 16-byte aligned.
__device__ __forceinline__ void load8_kc(const float* __restrict__ row, int64_t k0, int64_t K, bool vec,
                                         float (&x)[8]) {
  if (vec && k0 + 8 <= K) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(row + k0));
    const float4 b = __ldg(reinterpret_cast<const float4*>(row + k0 + 4));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = (k0 + i < K) ? __ldg(row + k0 + i) : 0.0f;
  }
}

// ---- quantizer --------------------------------------------------------------------------

struct QuantParams {
  float m;
  int lo, hi;
  int mode;          // hdqt_round_t
  bool sr_magic;     // |v| < 64 guaranteed: fixed-point conversion through the fp32 adder
  uint32_t tag;
  const PhiloxKeys* keys;   // the launch's round keys (a kernel parameter)
};

// codes of 8 consecutive elements; `g` = (linear index of the first element) / 8
__device__ __forceinline__ void quantize8(const float (&x)[8], const QuantParams& p, uint64_t g,
                                          int (&c)[8]) {
  if (p.mode == HDQT_ROUND_NEAREST) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float v = __fmul_rn(x[i], p.m);
      // rint through the fp32 adder: exact for |v| < 2^22
      const int q = __float_as_int(__fadd_rn(v, 12582912.0f)) - 0x4B400000;
      c[i] = min(max(q, p.lo), p.hi);
    }
  } else {
    const Philox4 rnd = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), p.tag, 0u, *p.keys);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float v = __fmul_rn(x[i], p.m);
      const uint32_t word = rnd.w[i >> 1];
      const int u16 = (i & 1) ? (int)(word >> 16) : (int)(word & 0xFFFFu);
      int v_fx;  // rint(v * 2^16), a Q.16 fixed-point integer
      if (p.sr_magic) {
        // for v in [-64, 64): v + 192 lies in [128, 256) where one ulp is 2^-16
        v_fx = __float_as_int(__fadd_rn(v, 192.0f)) - 0x43400000;
      } else {
        v_fx = __float2int_rn(__fmul_rn(v, 65536.0f));
      }
      const int q = (v_fx + u16) >> 16;  // floor((v_fx + u16) / 2^16)
      c[i] = min(max(q, p.lo), p.hi);
    }
  }
}

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d) {
  return (uint32_t)(a & 0xFF) | ((uint32_t)(b & 0xFF) << 8) | ((uint32_t)(c & 0xFF) << 16) |
         ((uint32_t)(d & 0xFF) << 24);
}

__device__ __forceinline__ QuantParams make_params(const QuantScale& qs, int bits, float clip, int mode,
                                                   const PhiloxKeys* keys, uint32_t tag) {
  QuantParams p;
  p.m = qs.m;
  p.lo = -(1 << (bits - 1));
  p.hi = (1 << (bits - 1)) - 1;
  p.mode = mode;
  p.sr_magic = ((float)(1 << (bits - 1)) <= 32.0f * clip);  // |v| <= 32 (1 + eps)
  p.keys = keys;
  p.tag = tag;
  return p;
}

// ---- block-wide max -----------------------------------------------------------------------

__device__ __forceinline__ void block_absmax_commit(uint32_t mx, float* amax_out, int32_t* dev_status) {
  __shared__ uint32_t smax[kThreads / 32];
  mx = __reduce_max_sync(0xFFFFFFFFu, mx);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) smax[warp] = mx;
  __syncthreads();
  if (warp == 0) {
    uint32_t v = (lane < kThreads / 32) ? smax[lane] : 0u;
    v = __reduce_max_sync(0xFFFFFFFFu, v);
    if (lane == 0) {
      // non-negative floats order like their bit patterns
      atomicMax(reinterpret_cast<uint32_t*>(amax_out), v);
      if (v >= 0x7F800000u) report_status(dev_status, HDQT_ERR_NONFINITE);
    }
  }
}

// ---- K-contiguous kernels -------------------------------------------------------------------
// A thread block walks the tensor in slabs of kUnroll*kThreads chunks (a chunk = 8 consecutive k of one
// row); every thread first issues the loads of its kUnroll chunks, then transforms them, so that
// kUnroll*32 bytes per thread are in flight.

constexpr int kUnrollAbsmax = 4;
constexpr int kUnrollQuant = 2;

// chunk index -> (row, first k). 64-bit division is ~100 instructions, i.e. more than the whole
// transform of the chunk, so it is kept for huge tensors only.
struct ChunkMap {
  int64_t chunks_per_row;
  bool small;   // every chunk index fits 32 bits
};
__device__ __forceinline__ void chunk_to_row_k(const ChunkMap& m, int64_t c, int64_t& r, int64_t& k0) {
  if (m.small) {
    const uint32_t rr = (uint32_t)c / (uint32_t)m.chunks_per_row;
    r = rr;
    k0 = (int64_t)((uint32_t)c - rr * (uint32_t)m.chunks_per_row) << 3;
  } else {
    r = c / m.chunks_per_row;
    k0 = (c - r * m.chunks_per_row) << 3;
  }
}

__global__ void __launch_bounds__(kThreads)
absmax_kc_kernel(const float* __restrict__ src, int64_t rows, int64_t K, int64_t ld_row, int64_t K_pad,
                 int had_block, bool vec, float* amax_out, int32_t* dev_status) {
  const int64_t chunks_per_row = K_pad >> 3;
  const int64_t total = rows * chunks_per_row;
  const ChunkMap cmap{chunks_per_row, total < (int64_t(1) << 31)};
  const bool dense = (K == K_pad) && (ld_row == K);
  const int lane = threadIdx.x & 31;
  uint32_t mx = 0u;
  for (int64_t base = (int64_t)blockIdx.x * (kThreads * kUnrollAbsmax); base < total;
       base += (int64_t)gridDim.x * (kThreads * kUnrollAbsmax)) {
    float x[kUnrollAbsmax][8];
#pragma unroll
    for (int u = 0; u < kUnrollAbsmax; ++u) {
      const int64_t c = base + u * kThreads + threadIdx.x;
      if (c < total) {
        if (dense) {   // rows are back to back and unpadded: chunk c starts at element 8c
          load8_kc(src, c << 3, total << 3, vec, x[u]);
        } else {
          int64_t r, k0;
          chunk_to_row_k(cmap, c, r, k0);
          load8_kc(src + r * ld_row, k0, K, vec, x[u]);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[u][i] = 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnrollAbsmax; ++u) {
      fwht8_regs(x[u], had_block);
      fwht8_lanes(x[u], had_block, lane);
#pragma unroll
      for (int i = 0; i < 8; ++i) mx = max(mx, abs_bits(x[u][i]));
    }
  }
  block_absmax_commit(mx, amax_out, dev_status);
}

__global__ void __launch_bounds__(kThreads)
quantize_kc_kernel(const float* __restrict__ src, int64_t rows, int64_t K, int64_t ld_row, int64_t K_pad,
                   int had_block, bool vec, int bits, float clip, int mode,
                   const __grid_constant__ PhiloxKeys keys, uint32_t tag,
                   const float* __restrict__ amax_ptr, int8_t* __restrict__ codes, float* step_out,
                   uint16_t* __restrict__ row_norms, int32_t* dev_status) {
  const QuantScale qs = make_quant_scale(__ldg(amax_ptr), clip, bits);
  const QuantParams p = make_params(qs, bits, clip, mode, &keys, tag);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *step_out = qs.step;
    if (qs.bad) report_status(dev_status, HDQT_ERR_NONFINITE);
  }
  const int64_t chunks_per_row = K_pad >> 3;
  const int64_t total = rows * chunks_per_row;
  const ChunkMap cmap{chunks_per_row, total < (int64_t(1) << 31)};
  const bool dense = (K == K_pad) && (ld_row == K);
  const int lane = threadIdx.x & 31;
  for (int64_t base = (int64_t)blockIdx.x * (kThreads * kUnrollQuant); base < total;
       base += (int64_t)gridDim.x * (kThreads * kUnrollQuant)) {
    float x[kUnrollQuant][8];
#pragma unroll
    for (int u = 0; u < kUnrollQuant; ++u) {
      const int64_t c = base + u * kThreads + threadIdx.x;
      if (c < total) {
        if (dense) {   // rows are back to back and unpadded: chunk c starts at element 8c
          load8_kc(src, c << 3, total << 3, vec, x[u]);
        } else {
          int64_t r, k0;
          chunk_to_row_k(cmap, c, r, k0);
          load8_kc(src + r * ld_row, k0, K, vec, x[u]);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[u][i] = 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnrollQuant; ++u) {
      const int64_t c = base + u * kThreads + threadIdx.x;
      const bool valid = c < total;
      fwht8_regs(x[u], had_block);
      fwht8_lanes(x[u], had_block, lane);
      int q[8];
      quantize8(x[u], p, (uint64_t)c, q);  // linear index of the chunk's first element is 8*c
      // codes are dense [rows, K_pad]: chunk c is bytes [8c, 8c+8) and tile c/4 of the row-norm array
      uint2 out;
      out.x = pack4(q[0], q[1], q[2], q[3]);
      out.y = pack4(q[4], q[5], q[6], q[7]);
      if (row_norms != nullptr) {
        int ss = __dp4a((int)out.x, (int)out.x, 0);
        ss = __dp4a((int)out.y, (int)out.y, ss);
        ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
        ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
        if (valid && (lane & 3) == 0) row_norms[c >> 2] = (uint16_t)ss;
      }
      if (valid) *reinterpret_cast<uint2*>(codes + (c << 3)) = out;
    }
  }
}

// max over each block of 128 rows of the per-row tile norms: a thread block covers 64 K tiles of one
// row block, its 4 thread rows take 32 rows each, shared memory combines them
__global__ void __launch_bounds__(256)
block_norms_kernel(const uint16_t* __restrict__ row_norms, int64_t rows, int64_t T,
                   int32_t* __restrict__ tile_norms) {
  __shared__ int s_part[4][64];
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
  const int64_t t = (int64_t)blockIdx.x * 64 + tx;
  const int64_t rb = blockIdx.y;
  const int64_t r0 = rb * 128 + ty * 32;
  int mx = 0;
  if (t < T) {
    const uint16_t* p = row_norms + r0 * T + t;
    if (r0 + 32 <= rows) {
      // whole group in range: no per-row test, so the 32 independent loads can all be in flight
      int v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = (int)__ldg(p + i * T);
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = max(mx, v[i]);
    } else {
      for (int i = 0; i < 32 && r0 + i < rows; ++i) mx = max(mx, (int)__ldg(p + i * T));
    }
  }
  s_part[ty][tx] = mx;
  __syncthreads();
  if (ty == 0 && t < T) {
    tile_norms[rb * T + t] = max(max(s_part[0][tx], s_part[1][tx]), max(s_part[2][tx], s_part[3][tx]));
  }
}

// ---- K-strided kernels ------------------------------------------------------------------------
// element (r, k) = src[k*ld_k + r]; thread = (row r, 32-block kb); r is the fast thread index.

__device__ __forceinline__ void load32_ks(const float* __restrict__ src, int64_t r, int64_t kb, int64_t K,
                                          int64_t ld_k, float (&x)[32]) {
  const float* p = src + (kb << 5) * ld_k + r;
  const int64_t k_left = K - (kb << 5);
  if (k_left >= 32) {
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = __ldg(p + i * ld_k);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = (i < k_left) ? __ldg(p + i * ld_k) : 0.0f;
  }
}

__global__ void __launch_bounds__(kThreads, 3)
absmax_ks_kernel(const float* __restrict__ src, int64_t rows, int64_t K, int64_t ld_k, int64_t K_pad,
                 int had_block, float* amax_out, int32_t* dev_status) {
  // work item = (32-block of K, group of kThreads rows); the host guarantees that their number fits 31 bits
  const uint32_t row_groups = (uint32_t)((rows + kThreads - 1) / kThreads);
  const uint32_t items = row_groups * (uint32_t)(K_pad >> 5);
  uint32_t mx = 0u;
  for (uint32_t w = blockIdx.x; w < items; w += gridDim.x) {
    const uint32_t kbu = w / row_groups;
    const int64_t kb = kbu;
    const int64_t r = (int64_t)(w - kbu * row_groups) * kThreads + threadIdx.x;
    if (r < rows) {
      float x[32];
      load32_ks(src, r, kb, K, ld_k, x);
      fwht32_regs(x, had_block);
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = max(mx, abs_bits(x[i]));
    }
  }
  block_absmax_commit(mx, amax_out, dev_status);
}

__global__ void __launch_bounds__(kThreads, 3)
quantize_ks_kernel(const float* __restrict__ src, int64_t rows, int64_t K, int64_t ld_k, int64_t K_pad,
                   int had_block, int bits, float clip, int mode,
                   const __grid_constant__ PhiloxKeys keys, uint32_t tag,
                   const float* __restrict__ amax_ptr, int8_t* __restrict__ codes, float* step_out,
                   int32_t* __restrict__ tile_norms, int32_t* dev_status) {
  __shared__ int s_norm[kThreads / 32];
  const QuantScale qs = make_quant_scale(__ldg(amax_ptr), clip, bits);
  const QuantParams p = make_params(qs, bits, clip, mode, &keys, tag);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *step_out = qs.step;
    if (qs.bad) report_status(dev_status, HDQT_ERR_NONFINITE);
  }
  // rows are padded to a multiple of the block size so that one thread block never straddles
  // two 32-blocks of K and always covers whole 128-row groups (needed for the tile norms)
  const int64_t T = K_pad >> 5;
  const uint32_t row_groups = (uint32_t)((rows + kThreads - 1) / kThreads);
  const uint32_t items = row_groups * (uint32_t)T;   // the host guarantees that this fits 31 bits
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t item = blockIdx.x; item < items; item += gridDim.x) {
    const uint32_t kbu = item / row_groups;     // uniform over the block
    const int64_t kb = kbu;
    const int64_t r_group0 = (int64_t)(item - kbu * row_groups) * kThreads;
    const int64_t r = r_group0 + threadIdx.x;
    int ss = 0;
    if (r < rows) {
      float x[32];
      load32_ks(src, r, kb, K, ld_k, x);
      fwht32_regs(x, had_block);
      uint32_t w[8];
      const uint64_t g0 = (uint64_t)(r * K_pad + (kb << 5)) >> 3;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float x8[8];
        int q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x8[i] = x[8 * j + i];
        quantize8(x8, p, g0 + j, q);
        w[2 * j] = pack4(q[0], q[1], q[2], q[3]);
        w[2 * j + 1] = pack4(q[4], q[5], q[6], q[7]);
        ss = __dp4a((int)w[2 * j], (int)w[2 * j], ss);
        ss = __dp4a((int)w[2 * j + 1], (int)w[2 * j + 1], ss);
      }
      uint4* dst = reinterpret_cast<uint4*>(codes + r * K_pad + (kb << 5));
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
    if (tile_norms != nullptr) {  // uniform branch
      ss = __reduce_max_sync(0xFFFFFFFFu, ss);
      __syncthreads();
      if (lane == 0) s_norm[warp] = ss;
      __syncthreads();
      if (threadIdx.x < kThreads / 128) {
        const int64_t r_base = r_group0 + threadIdx.x * 128;
        if (r_base < rows) {
          int mx = 0;
#pragma unroll
          for (int i = 0; i < 4; ++i) mx = max(mx, s_norm[threadIdx.x * 4 + i]);
          tile_norms[(r_base >> 7) * T + kb] = mx;
        }
      }
    }
  }
}

int g_sm_count = 0;

}  // namespace

int sm_count() {
  if (g_sm_count == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      n = kNumSMsHint;
    }
    g_sm_count = n;
  }
  return g_sm_count;
}

static int grid_for(int64_t work_items, int per_block, int blocks_per_sm) {
  const int64_t need = (work_items + per_block - 1) / per_block;
  const int64_t cap = (int64_t)sm_count() * blocks_per_sm;
  return (int)(need < 1 ? 1 : (need < cap ? need : cap));
}

hdqt_status_t launch_absmax(const float* src, int64_t rows, int64_t K, int64_t ld_row, int64_t ld_k,
                            int32_t had_block, float* amax_out, int32_t* dev_status, cudaStream_t s,
                            bool zero_first) {
  const int64_t K_pad = hdqt_padded_k(K, had_block);
  if (zero_first && cudaMemsetAsync(amax_out, 0, sizeof(float), s) != cudaSuccess) return HDQT_ERR_CUDA;
  if (ld_k == 1) {
    const bool vec = (ld_row % 4 == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0);
    const int64_t total = rows * (K_pad >> 3);
    absmax_kc_kernel<<<grid_for(total, kThreads * kUnrollAbsmax, 4), kThreads, 0, s>>>(
        src, rows, K, ld_row, K_pad, had_block, vec, amax_out, dev_status);
  } else {
    const int64_t items = ((rows + kThreads - 1) / kThreads) * (K_pad >> 5);
    if (items >= (int64_t(1) << 31)) return HDQT_ERR_UNSUPPORTED;
    absmax_ks_kernel<<<grid_for(items, 1, 3), kThreads, 0, s>>>(src, rows, K, ld_k, K_pad, had_block, amax_out,
                                                              dev_status);
  }
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}

hdqt_status_t launch_quantize(const float* src, int64_t rows, int64_t K, int64_t ld_row, int64_t ld_k,
                              int32_t had_block, int32_t bits, float clip, int32_t mode, uint64_t seed,
                              uint32_t tag, const float* amax, int8_t* codes, float* step_out,
                              int32_t* tile_norms, uint16_t* row_norms_scratch, int32_t* dev_status,
                              cudaStream_t s) {
  const int64_t K_pad = hdqt_padded_k(K, had_block);
  const int64_t T = K_pad >> 5;
  const PhiloxKeys keys = make_philox_keys(seed);
  if (ld_k == 1) {
    const bool vec = (ld_row % 4 == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0);
    const int64_t total = rows * (K_pad >> 3);
    uint16_t* rn = tile_norms ? row_norms_scratch : nullptr;
    quantize_kc_kernel<<<grid_for(total, kThreads * kUnrollQuant, 4), kThreads, 0, s>>>(
        src, rows, K, ld_row, K_pad, had_block, vec, bits, clip, mode, keys, tag, amax, codes, step_out, rn,
        dev_status);
    if (tile_norms) {
      dim3 grid((unsigned)((T + 63) / 64), (unsigned)((rows + 127) / 128));
      block_norms_kernel<<<grid, 256, 0, s>>>(rn, rows, T, tile_norms);
    }
  } else {
    const int64_t items = ((rows + kThreads - 1) / kThreads) * T;
    if (items >= (int64_t(1) << 31)) return HDQT_ERR_UNSUPPORTED;
    quantize_ks_kernel<<<grid_for(items, 1, 3), kThreads, 0, s>>>(
        src, rows, K, ld_k, K_pad, had_block, bits, clip, mode, keys, tag, amax, codes, step_out, tile_norms,
        dev_status);
  }
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}

}  // namespace hdqt

// ---- allocation-free variant of the transform + quantize call ----------------------------------
//
// Scratch for hdqt_quantize_hadamard_static lives in this fixed device array instead of a caller
// workspace: [0, 256) holds the calibration maximum, the rest holds the per-row tile norms.
// Every GPU that loads the library carries these HDQT_STATIC_SCRATCH_BYTES until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HDQT_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code the name g_static_scratch is only a handle for the runtime, not a device address;
// the address a kernel can use must be asked for, once per device, with that device current.
hdqt_status_t static_scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return hdqt::cuda_failure(e, "cudaGetDevice(static scratch)");
  if (dev < 0 || dev >= kMaxDevices) return HDQT_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || ptr == nullptr) return hdqt::cuda_failure(e, "cudaGetSymbolAddress(static scratch)");
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = static_cast<unsigned char*>(g_static_scratch_ptr[dev]);
  return HDQT_OK;
}

}  // namespace

extern "C" hdqt_status_t hdqt_quantize_hadamard_static(const float* src, int64_t rows, int64_t K, int64_t ld_row,
                                                       int64_t ld_k, int32_t had_block, int32_t bits, float clip,
                                                       int32_t mode, uint64_t seed, uint32_t tag, int8_t* codes,
                                                       float* step_out, int32_t* tile_norms, int32_t* dev_status,
                                                       void* stream) {
  // same argument rules as hdqt_quantize_hadamard
  if (!src || !codes || !step_out || rows <= 0 || K <= 0) return HDQT_ERR_INVALID_ARG;
  if (had_block < 1 || (had_block & (had_block - 1)) != 0) return HDQT_ERR_INVALID_ARG;
  if (had_block > 32) return HDQT_ERR_UNSUPPORTED;
  if (!((ld_k == 1 && ld_row >= K) || (ld_row == 1 && ld_k >= rows))) return HDQT_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return HDQT_ERR_INVALID_ARG;
  if (!(clip >= 1.0f / 64.0f && clip <= 1.0f)) return HDQT_ERR_INVALID_ARG;
  if (mode != HDQT_ROUND_NEAREST && mode != HDQT_ROUND_STOCHASTIC) return HDQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(src) & 3) || (reinterpret_cast<uintptr_t>(codes) & 127)) return HDQT_ERR_ALIGNMENT;
  // the fixed array bounds the operand: 256 bytes + 2 bytes per (row, 32-wide K tile)
  const int64_t tiles = hdqt_padded_k(K, had_block) / 32;
  if (rows > (int64_t)(HDQT_STATIC_SCRATCH_BYTES - 256) / 2 / tiles) return HDQT_ERR_STATIC_SCRATCH;

  unsigned char* scratch = nullptr;
  hdqt_status_t st = static_scratch_for_current_device(&scratch);
  if (st != HDQT_OK) return st;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  float* amax = reinterpret_cast<float*>(scratch);
  uint16_t* row_norms = reinterpret_cast<uint16_t*>(scratch + 256);
  // the array keeps whatever the previous call left: launch_absmax zeroes the maximum before it
  // accumulates into it, and every row-norm entry that is read is written first by this call
  st = hdqt::launch_absmax(src, rows, K, ld_row, ld_k, had_block, amax, dev_status, s);
  if (st != HDQT_OK) return st;
  return hdqt::launch_quantize(src, rows, K, ld_row, ld_k, had_block, bits, clip, mode, seed, tag, amax, codes,
                               step_out, tile_norms, row_norms, dev_status, s);
}
