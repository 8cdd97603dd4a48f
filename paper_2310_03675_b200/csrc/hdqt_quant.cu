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
//
// One launch serves up to two operands (the two operands of a GEMM): thread blocks
// [first_block, first_block + num_blocks) of the grid belong to operand i.  The calibration
// launch leaves one partial maximum per thread block; every block of the quantize launch
// reduces those (a few hundred values) itself, so no memset, atomic or extra launch sits
// between the two passes.
#include <mutex>

#include "hdqt_common.cuh"

namespace hdqt {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// ---- butterflies ------------------------------------------------------------------------

// strides 1, 2, 4 on 8 register values (only those below had_block)
template <bool kHad32 = false>
__device__ __forceinline__ void fwht8_regs(float (&x)[8], int had_block) {
  if (kHad32) had_block = 32;
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
template <bool kHad32 = false>
__device__ __forceinline__ void fwht8_lanes(float (&x)[8], int had_block, int lane) {
  if (kHad32) had_block = 32;
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
template <bool kHad32 = false>
__device__ __forceinline__ void fwht32_regs(float (&x)[32], int had_block) {
  if (kHad32) had_block = 32;
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

// ---- loads through the implicit im2col view ---------------------------------------------------

// Address of the 8 consecutive patch elements k0..k0+7 of output position n (they lie inside one input pixel,
// since C % 8 == 0), or nullptr if that pixel is padding.
__device__ __forceinline__ const float* conv_chunk_ptr(const ConvGeom& g, const float* __restrict__ x, int64_t n,
                                                       int64_t k0) {
  uint32_t tap, c0, kh, kw, t, wo, b, ho;
  fastdivmod((uint32_t)k0, g.div_c, tap, c0);
  fastdivmod(tap, g.div_kw, kh, kw);
  fastdivmod((uint32_t)n, g.div_wo, t, wo);
  fastdivmod(t, g.div_ho, b, ho);
  const int hi = (int)(ho * g.stride + kh) - g.pad, wi = (int)(wo * g.stride + kw) - g.pad;
  if ((unsigned)hi >= (unsigned)g.H || (unsigned)wi >= (unsigned)g.W) return nullptr;
  return x + (((int64_t)b * g.H + hi) * g.W + wi) * g.C + c0;
}

__device__ __forceinline__ void load8_conv(const ConvGeom& g, const float* __restrict__ x, int64_t n, int64_t k0,
                                           bool vec, float (&v)[8]) {
  const float* p = conv_chunk_ptr(g, x, n, k0);
  if (p == nullptr) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.0f;
  } else if (vec) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p + 4));
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(p + i);
  }
}

// 32 consecutive output positions (32-block kb of the contraction) of patch element d: the positions are uniform
// over the thread block and advance by one per element (no division inside the loop), the patch element
// (tap, channel) is this thread's.
__device__ __forceinline__ void load32_conv(const ConvGeom& g, const float* __restrict__ x, int64_t d, int64_t kb,
                                            int64_t n_positions, float (&v)[32]) {
  uint32_t tap, c, kh, kw, t, wo, b, ho;
  fastdivmod((uint32_t)d, g.div_c, tap, c);
  fastdivmod(tap, g.div_kw, kh, kw);
  fastdivmod((uint32_t)(kb << 5), g.div_wo, t, wo);
  fastdivmod(t, g.div_ho, b, ho);
  const int dh = (int)kh - g.pad, dw = (int)kw - g.pad;
  const int64_t left = n_positions - (kb << 5);
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float val = 0.0f;
    const int hi = (int)(ho * g.stride) + dh, wi = (int)(wo * g.stride) + dw;
    if (i < left && (unsigned)hi < (unsigned)g.H && (unsigned)wi < (unsigned)g.W)
      val = __ldg(x + (((int64_t)b * g.H + hi) * g.W + wi) * g.C + c);
    v[i] = val;
    if (++wo == (uint32_t)g.Wo) {
      wo = 0;
      if (++ho == (uint32_t)g.Ho) { ho = 0; ++b; }
    }
  }
}

// ---- quantizer --------------------------------------------------------------------------
// Codes are produced with the offset 2^(bits-1) added (so that they are unsigned and one
// min-with-relu instruction clamps both sides), packed four to a word, and the offset is taken out
// of all four bytes at once: (w + addc) ^ 0x80808080 with addc = (0x80 - offset) in every byte
// (no byte can carry into its neighbour).

struct QuantParams {
  float m;
  int mode;          // hdqt_round_t
  int rng;           // 2^bits - 1: the largest offset code
  int nearest_bias;  // offset - bit pattern of the fp32 rounding constant
  int sr_bias;       // (offset << 16) - bit pattern of 192.0f
  int off16;         // offset << 16
  uint32_t addc;
  bool sr_magic;     // |v| < 64 guaranteed: fixed-point conversion through the fp32 adder
  bool zero_all;     // degenerate scale (all-zero or non-finite tensor): every code is 0
  uint32_t tag;
  uint32_t stream;          // fourth Philox counter word (0, or the caller's device-side stream offset)
  const PhiloxKeys* keys;   // the launch's round keys (a kernel parameter)
};

__device__ __forceinline__ uint32_t pack4_offset(const int (&t)[8], int base, uint32_t addc) {
  const uint32_t w = (uint32_t)t[base] | ((uint32_t)t[base + 1] << 8) | ((uint32_t)t[base + 2] << 16) |
                     ((uint32_t)t[base + 3] << 24);
  return (w + addc) ^ 0x80808080u;
}

// codes of 8 consecutive elements as two packed words; `g` = (linear index of the first element) / 8.
// kMode: 0 = nearest, 1 = stochastic with the fixed-point conversion through the fp32 adder (|v| < 64
// guaranteed), 2 = stochastic with a float-to-int conversion (any v; a quarter of the arithmetic rate).
// kPerm (stochastic modes): clamp the fixed-point sum itself and gather byte 2 of four sums with byte permutes
// instead of shifting every sum down (one instruction per element less; used by the K-contiguous kernels - in the
// K-strided kernel, which runs at its register limit, it made the nearest body 13 % slower).
template <int kMode, bool kPerm = false>
__device__ __forceinline__ void quantize8(const float (&x)[8], const QuantParams& p, uint64_t g, uint32_t& w0,
                                          uint32_t& w1) {
  int t[8];
  if (kMode == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float v = __fmul_rn(x[i], p.m);
      // rint through the fp32 adder (exact for |v| < 2^22), plus the code offset
      const int q = __float_as_int(__fadd_rn(v, 12582912.0f)) + p.nearest_bias;
      t[i] = __vimin_s32_relu(q, p.rng);
    }
  } else {
    const Philox4 rnd = philox4x32_10((uint32_t)g, (uint32_t)(g >> 32), p.tag, p.stream, *p.keys);
    // s = rint(v * 2^16) + u16 + (offset << 16), a Q.16 fixed-point integer; code + offset = floor(s / 2^16), clamped
    const int rng16 = (p.rng << 16) | 0xFFFF;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float v = __fmul_rn(x[i], p.m);
      const uint32_t word = rnd.w[i >> 1];
      const int u16 = (i & 1) ? (int)(word >> 16) : (int)(word & 0xFFFFu);
      int s;
      if (kMode == 1) {
        // for v in [-64, 64): v + 192 lies in [128, 256) where one ulp is 2^-16
        s = __float_as_int(__fadd_rn(v, 192.0f)) + u16 + p.sr_bias;
      } else {
        s = __float2int_rn(__fmul_rn(v, 65536.0f)) + u16 + p.off16;
      }
      // kPerm: s clamped to [0, rng * 2^16 + 0xFFFF], its byte 2 is code + offset
      t[i] = kPerm ? __vimin_s32_relu(s, rng16) : __vimin_s32_relu(s >> 16, p.rng);
    }
  }
  if (kMode != 0 && kPerm) {
    const uint32_t a01 = __byte_perm((uint32_t)t[0], (uint32_t)t[1], 0x0062), a23 = __byte_perm((uint32_t)t[2], (uint32_t)t[3], 0x0062);
    const uint32_t a45 = __byte_perm((uint32_t)t[4], (uint32_t)t[5], 0x0062), a67 = __byte_perm((uint32_t)t[6], (uint32_t)t[7], 0x0062);
    w0 = (__byte_perm(a01, a23, 0x5410) + p.addc) ^ 0x80808080u;
    w1 = (__byte_perm(a45, a67, 0x5410) + p.addc) ^ 0x80808080u;
  } else {
    w0 = pack4_offset(t, 0, p.addc);
    w1 = pack4_offset(t, 4, p.addc);
  }
  if (p.zero_all) { w0 = 0u; w1 = 0u; }
}

// Runs `body.template operator()<kMode, kHad32>()` for the operand's rounding mode and Hadamard block: the
// per-chunk code is then free of mode and block-size tests (they cost more than a tenth of its instructions).
// kClass: 0 = every rounding mode is compiled in, 1 = nearest only, 2 = the stochastic modes only (a kernel that
// holds fewer bodies gets registers allotted for those alone)
template <bool kTrack, int kClass, typename Body>
__device__ __forceinline__ void dispatch_mode2(const QuantParams& p, int had_block, Body& body) {
  const int mode = (p.mode == HDQT_ROUND_NEAREST) ? 0 : (p.sr_magic ? 1 : 2);
  if (had_block == 32) {
    if (kClass != 2 && mode == 0) body.template operator()<0, true, kTrack>();
    else if (kClass != 1 && mode == 1) body.template operator()<1, true, kTrack>();
    else if (kClass != 1 && mode == 2) body.template operator()<2, true, kTrack>();
  } else {
    if (kClass != 2 && mode == 0) body.template operator()<0, false, kTrack>();
    else if (kClass != 1 && mode == 1) body.template operator()<1, false, kTrack>();
    else if (kClass != 1 && mode == 2) body.template operator()<2, false, kTrack>();
  }
}
// kTrack: the body also keeps the maximum magnitude of the transformed values it sees (delayed scaling)
template <int kClass = 0, typename Body>
__device__ __forceinline__ void dispatch_mode(const QuantParams& p, int had_block, bool track, Body body) {
  if (track) dispatch_mode2<true, kClass>(p, had_block, body);
  else dispatch_mode2<false, kClass>(p, had_block, body);
}

__device__ __forceinline__ QuantParams make_params(const QuantScale& qs, int bits, float clip, int mode,
                                                   const PhiloxKeys* keys, uint32_t tag, uint32_t stream) {
  QuantParams p;
  const int off = 1 << (bits - 1);
  p.m = qs.m;
  p.mode = mode;
  p.rng = (1 << bits) - 1;
  p.nearest_bias = off - 0x4B400000;
  p.sr_bias = (off << 16) - 0x43400000;
  p.off16 = off << 16;
  p.addc = (uint32_t)(0x80 - off) * 0x01010101u;
  p.sr_magic = ((float)off <= 32.0f * clip);  // |v| <= 32 (1 + eps)
  p.zero_all = qs.zero || qs.bad;
  p.keys = keys;
  p.stream = stream;
  p.tag = tag;
  return p;
}

// ---- one operand of a (batched) launch ------------------------------------------------------

constexpr int kMaxOps = 2;

struct QuantOp {
  const float* src;
  int64_t rows, K, K_pad;
  int64_t ld;               // row stride (K contiguous) or K stride (K strided)
  float clip;
  int32_t mode;
  uint32_t tag;
  int32_t vec;              // K contiguous: 128-bit loads allowed
  int32_t seg_log2;         // K contiguous, blocked mapping: log2 of the K segment a thread block covers
  int32_t rt_log2;          // K strided: log2 of the rows a thread block covers (32..256; the rest of its 256
                            // threads take further 32-blocks of K, so that operands with few rows fill the block)
  const float* amax_in;     // quantize: supplied maximum, or nullptr = reduce `partials`
  uint32_t* partials;       // calibration: one partial maximum (bit pattern) per thread block of this operand
  int32_t n_partials;
  const uint32_t* hist_in;  // quantize: kMaxPartials partial maxima of an earlier tensor, used when amax_in is null
  uint32_t* hist_out;       // quantize: partial maxima of this tensor (kMaxPartials entries, unused ones zeroed)
  float* amax_atomic;       // calibration through the public call: atomic maximum into one float instead
  float* amax_slot;         // quantize: where the maximum that was used is published (may be null)
  int8_t* codes;
  float* step_out;
  int32_t* tile_norms;
  int32_t first_block, num_blocks;
  ConvGeom conv;            // enabled: src is an NHWC tensor viewed as its im2col matrix
};

struct QuantBatch {
  QuantOp op[kMaxOps];
  int32_t n_ops;
  int32_t had_block;
  int32_t bits;
  const uint32_t* stream;   // optional device word: fourth Philox counter word of the stochastic roundings
};

// which operand this thread block works on, and its block index within that operand
__device__ __forceinline__ const QuantOp& my_operand(const QuantBatch& b, int& local_block) {
  const int second = (b.n_ops > 1 && (int)blockIdx.x >= b.op[1].first_block) ? 1 : 0;
  local_block = (int)blockIdx.x - b.op[second].first_block;
  return b.op[second];
}

// ---- block-wide max -----------------------------------------------------------------------

__device__ __forceinline__ uint32_t block_max_u32(uint32_t mx) {
  __shared__ uint32_t smax[kThreads / 32];
  __shared__ uint32_t sres;
  mx = __reduce_max_sync(0xFFFFFFFFu, mx);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) smax[warp] = mx;
  __syncthreads();
  if (warp == 0) {
    uint32_t v = (lane < kThreads / 32) ? smax[lane] : 0u;
    v = __reduce_max_sync(0xFFFFFFFFu, v);
    if (lane == 0) sres = v;
  }
  __syncthreads();
  return sres;
}

__device__ __forceinline__ void commit_partial_max(const QuantOp& op, int local_block, uint32_t mx,
                                                   int32_t* dev_status) {
  const uint32_t v = block_max_u32(mx);
  if (threadIdx.x == 0) {
    // non-negative floats order like their bit patterns
    if (op.amax_atomic != nullptr) atomicMax(reinterpret_cast<uint32_t*>(op.amax_atomic), v);
    else op.partials[local_block] = v;
    if (v >= 0x7F800000u) report_status(dev_status, HDQT_ERR_NONFINITE);
  }
}

// Delayed scaling: the quantize pass leaves the partial maxima of the tensor it has just transformed, so that the
// next call on the same tensor (the next training step) needs no calibration pass.  All kMaxPartials entries are
// defined afterwards (the operand's first block zeroes the unused ones).
__device__ __forceinline__ void commit_history(const QuantOp& op, int local_block, uint32_t mx, int32_t* dev_status) {
  const uint32_t v = block_max_u32(mx);
  if (threadIdx.x == 0) {
    op.hist_out[local_block] = v;
    if (v >= 0x7F800000u) report_status(dev_status, HDQT_ERR_NONFINITE);
  }
  if (local_block == 0) {
    for (int i = op.num_blocks + threadIdx.x; i < kMaxPartials; i += kThreads) op.hist_out[i] = 0u;
  }
}

// The calibration maximum a quantize block works with: the supplied one, or the maximum of the partial
// maxima the calibration launch left behind.  Block 0 of the operand publishes scale and maximum.
__device__ __forceinline__ QuantScale resolve_scale(const QuantOp& op, int local_block, int bits,
                                                    int32_t* dev_status) {
  float amax;
  if (op.amax_in != nullptr) {
    amax = __ldg(op.amax_in);
  } else {
    // partial maxima of this call's calibration pass, or those an earlier call's quantize pass left behind
    const uint32_t* part = op.hist_in != nullptr ? op.hist_in : op.partials;
    const int n = op.hist_in != nullptr ? kMaxPartials : op.n_partials;
    uint32_t mx = 0u;
    for (int i = threadIdx.x; i < n; i += kThreads) mx = max(mx, __ldcg(part + i));
    amax = __uint_as_float(block_max_u32(mx));
  }
  const QuantScale qs = make_quant_scale(amax, op.clip, bits);
  if (local_block == 0 && threadIdx.x == 0) {
    *op.step_out = qs.step;
    if (op.amax_slot != nullptr && op.amax_in == nullptr) *op.amax_slot = amax;
    if (qs.bad) report_status(dev_status, HDQT_ERR_NONFINITE);
  }
  return qs;
}

// ---- K-contiguous kernels -------------------------------------------------------------------
// "linear" mapping: a thread block walks the tensor in slabs of kUnroll*kThreads chunks (a chunk = 8
// consecutive k of one row); every thread first issues the loads of its kUnroll chunks, then transforms
// them, so that kUnroll*32 bytes per thread are in flight.

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
absmax_kc_kernel(const __grid_constant__ QuantBatch b, int32_t* dev_status) {
  int local_block;
  const QuantOp& op = my_operand(b, local_block);
  const float* __restrict__ src = op.src;
  const int64_t K = op.K, ld_row = op.ld;
  const bool vec = op.vec != 0;
  const int had_block = b.had_block;
  const int64_t chunks_per_row = op.K_pad >> 3;
  const int64_t total = op.rows * chunks_per_row;
  const ChunkMap cmap{chunks_per_row, total < (int64_t(1) << 31)};
  const bool dense = (K == op.K_pad) && (ld_row == K) && !op.conv.enabled;
  const int lane = threadIdx.x & 31;
  uint32_t mx = 0u;
  for (int64_t base = (int64_t)local_block * (kThreads * kUnrollAbsmax); base < total;
       base += (int64_t)op.num_blocks * (kThreads * kUnrollAbsmax)) {
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
          if (op.conv.enabled) load8_conv(op.conv, src, r, k0, vec, x[u]);
          else load8_kc(src + r * ld_row, k0, K, vec, x[u]);
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
  commit_partial_max(op, local_block, mx, dev_status);
}

// quantize, linear mapping (no tile norms)
__global__ void __launch_bounds__(kThreads, 4)
quantize_kc_kernel(const __grid_constant__ QuantBatch b, const __grid_constant__ PhiloxKeys keys,
                   int32_t* dev_status) {
  int local_block;
  const QuantOp& op = my_operand(b, local_block);
  const QuantScale qs = resolve_scale(op, local_block, b.bits, dev_status);
  const QuantParams p = make_params(qs, b.bits, op.clip, op.mode, &keys, op.tag, b.stream ? __ldg(b.stream) : 0u);
  const float* __restrict__ src = op.src;
  int8_t* __restrict__ codes = op.codes;
  const int64_t K = op.K, ld_row = op.ld;
  const bool vec = op.vec != 0;
  const int had_block = b.had_block;
  const int64_t chunks_per_row = op.K_pad >> 3;
  const int64_t total = op.rows * chunks_per_row;
  const ChunkMap cmap{chunks_per_row, total < (int64_t(1) << 31)};
  const bool dense = (K == op.K_pad) && (ld_row == K) && !op.conv.enabled;
  const int lane = threadIdx.x & 31;
  uint32_t seen = 0u;   // maximum |x H| this thread has seen (tracked only for delayed scaling)
  auto body = [&]<int kMode, bool kHad32, bool kTrack>() {
  for (int64_t base = (int64_t)local_block * (kThreads * kUnrollQuant); base < total;
       base += (int64_t)op.num_blocks * (kThreads * kUnrollQuant)) {
    float x[kUnrollQuant][8];
#pragma unroll
    for (int u = 0; u < kUnrollQuant; ++u) {
      const int64_t c = base + u * kThreads + threadIdx.x;
      if (c < total) {
        if (dense) {
          load8_kc(src, c << 3, total << 3, vec, x[u]);
        } else {
          int64_t r, k0;
          chunk_to_row_k(cmap, c, r, k0);
          if (op.conv.enabled) load8_conv(op.conv, src, r, k0, vec, x[u]);
          else load8_kc(src + r * ld_row, k0, K, vec, x[u]);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[u][i] = 0.0f;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnrollQuant; ++u) {
      const int64_t c = base + u * kThreads + threadIdx.x;
      fwht8_regs<kHad32>(x[u], had_block);
      fwht8_lanes<kHad32>(x[u], had_block, lane);
      if (kTrack) {
#pragma unroll
        for (int i = 0; i < 8; ++i) seen = max(seen, abs_bits(x[u][i]));
      }
      uint2 out;
      quantize8<kMode, true>(x[u], p, (uint64_t)c, out.x, out.y);  // linear index of the chunk's first element is 8*c
      // codes are dense [rows, K_pad]: chunk c is bytes [8c, 8c+8)
      if (c < total) *reinterpret_cast<uint2*>(codes + (c << 3)) = out;
    }
  }
  };
  dispatch_mode(p, had_block, op.hist_out != nullptr, body);
  if (op.hist_out != nullptr) commit_history(op, local_block, seen, dev_status);
}

// quantize, blocked mapping, with the tile norms: a work item is 128 rows x one K segment of 2^seg_log2
// elements (32..256), so that the maximum over the 128 rows of every tile's sum(code^2) is formed inside
// the thread block and written once.  A row's segment is covered by seg/8 neighbouring lanes; a warp
// covers 32/(seg/8) rows per pass, the block's 8 warps cover consecutive rows.
__global__ void __launch_bounds__(kThreads, 4)
quantize_kc_norms_kernel(const __grid_constant__ QuantBatch b, const __grid_constant__ PhiloxKeys keys,
                         int32_t* dev_status) {
  __shared__ int s_norm[kThreads / 32][32];
  int local_block;
  const QuantOp& op = my_operand(b, local_block);
  const QuantScale qs = resolve_scale(op, local_block, b.bits, dev_status);
  const QuantParams p = make_params(qs, b.bits, op.clip, op.mode, &keys, op.tag, b.stream ? __ldg(b.stream) : 0u);
  const float* __restrict__ src = op.src;
  int8_t* __restrict__ codes = op.codes;
  const int64_t K = op.K, K_pad = op.K_pad, ld_row = op.ld, rows = op.rows;
  const bool vec = op.vec != 0;
  const int had_block = b.had_block;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int lpr_log2 = op.seg_log2 - 3;          // lanes per row segment
  const int rpw = 32 >> lpr_log2;                // rows per warp pass
  const int row_sub = lane >> lpr_log2;
  const int kc = lane & ((1 << lpr_log2) - 1);
  const int passes = 16 / rpw;                   // 128 rows / (8 warps x rpw rows)
  const int64_t nseg = (K_pad + (int64_t(1) << op.seg_log2) - 1) >> op.seg_log2;
  const int64_t T = K_pad >> 5;
  const int64_t cpr = K_pad >> 3;                // chunks per code row
  const int64_t n_items = ((rows + 127) >> 7) * nseg;
  uint32_t seen = 0u;   // maximum |x H| this thread has seen (tracked only for delayed scaling)
  auto body = [&]<int kMode, bool kHad32, bool kTrack>() {
  for (int64_t item = local_block; item < n_items; item += op.num_blocks) {
    const int64_t rb = item / nseg, kseg = item - rb * nseg;
    const int64_t k0 = (kseg << op.seg_log2) + (kc << 3);
    const bool k_ok = k0 < K_pad;
    int nmax = 0;
    const int64_t row0 = (rb << 7) + warp * rpw + row_sub;    // this thread's row in pass 0; a pass adds 8 * rpw rows
    const bool whole = vec && !op.conv.enabled && ((rb << 7) + 128 <= rows) && (((kseg + 1) << op.seg_log2) <= K);
    if (whole) {
      // whole 128-row block, whole segment inside K, vector loads: nothing to test per chunk, running pointers
      const float* __restrict__ sp = src + row0 * ld_row + k0;
      int8_t* __restrict__ cp = codes + row0 * K_pad + k0;
      uint64_t g = (uint64_t)row0 * (uint64_t)cpr + (uint64_t)(k0 >> 3);
      const int64_t s_step = 8 * (int64_t)rpw * ld_row, c_step = 8 * (int64_t)rpw * K_pad;
      const uint64_t g_step = 8ull * (uint64_t)rpw * (uint64_t)cpr;
      for (int pass = 0; pass < passes; pass += kUnrollQuant) {
        float x[kUnrollQuant][8];
#pragma unroll
        for (int u = 0; u < kUnrollQuant; ++u) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(sp + u * s_step));
          const float4 c = __ldg(reinterpret_cast<const float4*>(sp + u * s_step + 4));
          x[u][0] = a.x; x[u][1] = a.y; x[u][2] = a.z; x[u][3] = a.w;
          x[u][4] = c.x; x[u][5] = c.y; x[u][6] = c.z; x[u][7] = c.w;
        }
#pragma unroll
        for (int u = 0; u < kUnrollQuant; ++u) {
          fwht8_regs<kHad32>(x[u], had_block);
          fwht8_lanes<kHad32>(x[u], had_block, lane);
          if (kTrack) {
#pragma unroll
            for (int i = 0; i < 8; ++i) seen = max(seen, abs_bits(x[u][i]));
          }
          uint2 out;
          quantize8<kMode, true>(x[u], p, g + u * g_step, out.x, out.y);
          int ss = __dp4a((int)out.x, (int)out.x, 0);
          ss = __dp4a((int)out.y, (int)out.y, ss);
          ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
          ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
          nmax = max(nmax, ss);
          *reinterpret_cast<uint2*>(cp + u * c_step) = out;
        }
        sp += kUnrollQuant * s_step;
        cp += kUnrollQuant * c_step;
        g += kUnrollQuant * g_step;
      }
    } else {
      for (int pass = 0; pass < passes; pass += kUnrollQuant) {
        float x[kUnrollQuant][8];
        int64_t r[kUnrollQuant];
#pragma unroll
        for (int u = 0; u < kUnrollQuant; ++u) {
          r[u] = row0 + (int64_t)(pass + u) * 8 * rpw;
          if (k_ok && r[u] < rows) {
            if (op.conv.enabled) load8_conv(op.conv, src, r[u], k0, vec, x[u]);
            else load8_kc(src + r[u] * ld_row, k0, K, vec, x[u]);
          } else {
            r[u] = -1;
#pragma unroll
            for (int i = 0; i < 8; ++i) x[u][i] = 0.0f;
          }
        }
#pragma unroll
        for (int u = 0; u < kUnrollQuant; ++u) {
          fwht8_regs<kHad32>(x[u], had_block);
          fwht8_lanes<kHad32>(x[u], had_block, lane);
          if (kTrack) {
#pragma unroll
            for (int i = 0; i < 8; ++i) seen = max(seen, abs_bits(x[u][i]));
          }
          const bool valid = r[u] >= 0;
          const uint64_t g = valid ? (uint64_t)r[u] * (uint64_t)cpr + (uint64_t)(k0 >> 3) : 0u;
          uint2 out;
          quantize8<kMode, true>(x[u], p, g, out.x, out.y);
          int ss = __dp4a((int)out.x, (int)out.x, 0);
          ss = __dp4a((int)out.y, (int)out.y, ss);
          ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
          ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
          if (valid) {
            nmax = max(nmax, ss);
            *reinterpret_cast<uint2*>(codes + r[u] * K_pad + k0) = out;
          }
        }
      }
    }
    s_norm[warp][lane] = nmax;
    __syncthreads();
    if ((int)threadIdx.x < (1 << (op.seg_log2 - 5))) {
      const int64_t t = (kseg << (op.seg_log2 - 5)) + threadIdx.x;
      if (t < T) {
        int mx = 0;
        for (int w = 0; w < kThreads / 32; ++w)
          for (int rs = 0; rs < rpw; ++rs) mx = max(mx, s_norm[w][(rs << lpr_log2) + 4 * (int)threadIdx.x]);
        op.tile_norms[rb * T + t] = mx;
      }
    }
    __syncthreads();
  }
  };
  dispatch_mode(p, had_block, op.hist_out != nullptr, body);
  if (op.hist_out != nullptr) commit_history(op, local_block, seen, dev_status);
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
absmax_ks_kernel(const __grid_constant__ QuantBatch b, int32_t* dev_status) {
  int local_block;
  const QuantOp& op = my_operand(b, local_block);
  const float* __restrict__ src = op.src;
  const int64_t rows = op.rows, K = op.K, ld_k = op.ld;
  const int had_block = b.had_block;
  // work item = (group of 2^rt_log2 rows, group of 256 >> rt_log2 32-blocks of K); the host guarantees that
  // their number fits 31 bits
  const int rt_log2 = op.rt_log2;
  const int64_t T = op.K_pad >> 5;
  const uint32_t row_groups = (uint32_t)((rows + (int64_t(1) << rt_log2) - 1) >> rt_log2);
  const uint32_t kpc = (uint32_t)kThreads >> rt_log2;
  const uint32_t items = row_groups * (uint32_t)((T + kpc - 1) / kpc);
  const uint32_t r_local = threadIdx.x & ((1u << rt_log2) - 1u), kbs = threadIdx.x >> rt_log2;
  uint32_t mx = 0u;
  for (uint32_t w = (uint32_t)local_block; w < items; w += (uint32_t)op.num_blocks) {
    const uint32_t kg = w / row_groups;
    const int64_t kb = (int64_t)kg * kpc + kbs;
    const int64_t r = ((int64_t)(w - kg * row_groups) << rt_log2) + r_local;
    if (r < rows && kb < T) {
      float x[32];
      if (op.conv.enabled) load32_conv(op.conv, src, r, kb, K, x);
      else load32_ks(src, r, kb, K, ld_k, x);
      fwht32_regs(x, had_block);
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = max(mx, abs_bits(x[i]));
    }
  }
  commit_partial_max(op, local_block, mx, dev_status);
}

// kClass: 1 = operands rounded to nearest, 2 = stochastically rounded operands (two kernels: this one runs at its
// register limit, and the stochastic bodies would otherwise set the nearest body's register allotment)
template <int kClass>
__global__ void __launch_bounds__(kThreads, 3)
quantize_ks_kernel(const __grid_constant__ QuantBatch b, const __grid_constant__ PhiloxKeys keys,
                   int32_t* dev_status) {
  __shared__ int s_norm[kThreads / 32];
  int local_block;
  const QuantOp& op = my_operand(b, local_block);
  const QuantScale qs = resolve_scale(op, local_block, b.bits, dev_status);
  const QuantParams p = make_params(qs, b.bits, op.clip, op.mode, &keys, op.tag, b.stream ? __ldg(b.stream) : 0u);
  const float* __restrict__ src = op.src;
  int8_t* __restrict__ codes = op.codes;
  int32_t* __restrict__ tile_norms = op.tile_norms;
  const int64_t rows = op.rows, K = op.K, K_pad = op.K_pad, ld_k = op.ld;
  const int had_block = b.had_block;
  // rows are padded to a multiple of the block size so that one thread block never straddles
  // two 32-blocks of K and always covers whole 128-row groups (needed for the tile norms)
  const int64_t T = K_pad >> 5;
  const int rt_log2 = op.rt_log2;
  const uint32_t row_groups = (uint32_t)((rows + (int64_t(1) << rt_log2) - 1) >> rt_log2);
  const uint32_t kpc = (uint32_t)kThreads >> rt_log2;            // 32-blocks of K per work item
  const uint32_t items = row_groups * (uint32_t)((T + kpc - 1) / kpc);   // the host guarantees that this fits 31 bits
  const uint32_t r_local = threadIdx.x & ((1u << rt_log2) - 1u), kbs = threadIdx.x >> rt_log2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t seen = 0u;   // maximum |x H| this thread has seen (tracked only for delayed scaling)
  auto body = [&]<int kMode, bool kHad32, bool kTrack>() {
  for (uint32_t item = (uint32_t)local_block; item < items; item += (uint32_t)op.num_blocks) {
    const uint32_t kg = item / row_groups;      // uniform over the block
    const int64_t kb = (int64_t)kg * kpc + kbs;
    const int64_t r_group0 = (int64_t)(item - kg * row_groups) << rt_log2;
    const int64_t r = r_group0 + r_local;
    int ss = 0;
    if (r < rows && kb < T) {
      float x[32];
      if (op.conv.enabled) load32_conv(op.conv, src, r, kb, K, x);
      else load32_ks(src, r, kb, K, ld_k, x);
      fwht32_regs<kHad32>(x, had_block);
      if (kTrack) {
#pragma unroll
        for (int i = 0; i < 32; ++i) seen = max(seen, abs_bits(x[i]));
      }
      uint32_t w[8];
      const uint64_t g0 = (uint64_t)(r * K_pad + (kb << 5)) >> 3;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float x8[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x8[i] = x[8 * j + i];
        quantize8<kMode, true>(x8, p, g0 + j, w[2 * j], w[2 * j + 1]);
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
      // one writer per (128-row block, 32-block of K) pair of the item: its warps are consecutive
      const uint32_t rb_per_item = max(1u, (1u << rt_log2) >> 7), wpp = min(4u, (1u << rt_log2) >> 5);
      if (threadIdx.x < kpc * rb_per_item) {
        const uint32_t pk = threadIdx.x / rb_per_item, prb = threadIdx.x - pk * rb_per_item;
        const int64_t r_base = r_group0 + (int64_t)prb * 128, pkb = (int64_t)kg * kpc + pk;
        if (r_base < rows && pkb < T) {
          const uint32_t w0 = ((pk << rt_log2) + (prb << 7)) >> 5;
          int mx = 0;
          for (uint32_t i = 0; i < wpp; ++i) mx = max(mx, s_norm[w0 + i]);
          tile_norms[(r_base >> 7) * T + pkb] = mx;
        }
      }
    }
  }
  };
  dispatch_mode<kClass>(p, had_block, op.hist_out != nullptr, body);
  if (op.hist_out != nullptr) commit_history(op, local_block, seen, dev_status);
}

constexpr int kMaxDevices = 64;

int grid_for(int64_t work_items, int per_block, int blocks_per_sm) {
  const int64_t need = (work_items + per_block - 1) / per_block;
  const int64_t cap = (int64_t)sm_count() * blocks_per_sm;
  const int64_t g = need < 1 ? 1 : (need < cap ? need : cap);
  return (int)(g < kMaxPartials ? g : kMaxPartials);
}

// K segment of the blocked mapping: the widest of 256/128/64/32 that wastes at most 1/8 of its lanes
int pick_seg_log2(int64_t K_pad) {
  for (int s = 8; s > 5; --s) {
    const int64_t seg = int64_t(1) << s;
    const int64_t covered = (K_pad + seg - 1) / seg * seg;
    if (covered * 8 <= K_pad * 9) return s;
  }
  return 5;
}

// work items of the K-strided kernels: (group of 2^rt_log2 rows) x (group of 256 >> rt_log2 32-blocks of K)
int64_t ks_items(int64_t rows, int64_t K_pad, int rt_log2) {
  const int64_t rt = int64_t(1) << rt_log2, kpc = kThreads >> rt_log2;
  return ((rows + rt - 1) / rt) * (((K_pad >> 5) + kpc - 1) / kpc);
}

QuantOp make_op(const QuantOperand& a, int32_t had_block, uint32_t* partials) {
  QuantOp o;
  o.src = a.src;
  o.rows = a.rows;
  o.K = a.K;
  o.K_pad = hdqt_padded_k(a.K, had_block);
  const bool kc = (a.ld_k == 1);
  o.ld = kc ? a.ld_row : a.ld_k;
  o.clip = a.clip;
  o.mode = a.mode;
  o.tag = a.tag;
  o.vec = (kc && (a.ld_row % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.src) & 15) == 0)) ? 1 : 0;
  o.seg_log2 = pick_seg_log2(o.K_pad);
  o.rt_log2 = 8;
  while (o.rt_log2 > 5 && (int64_t(1) << (o.rt_log2 - 1)) >= a.rows) --o.rt_log2;
  o.amax_in = a.amax_in;
  o.partials = partials;
  o.n_partials = 0;
  o.hist_in = a.hist_in;
  o.hist_out = a.hist_out;
  o.amax_atomic = nullptr;
  o.amax_slot = a.amax_slot;
  o.codes = a.codes;
  o.step_out = a.step_out;
  o.tile_norms = a.tile_norms;
  o.first_block = 0;
  o.num_blocks = 0;
  o.conv = a.conv;
  if (a.conv.enabled) o.vec = ((reinterpret_cast<uintptr_t>(a.src) & 15) == 0) ? 1 : 0;
  return o;
}

}  // namespace

int sm_count() {
  static int cache[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return kNumSMsHint;
  if (cache[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = kNumSMsHint;
    cache[dev] = n;
  }
  return cache[dev];
}

hdqt_status_t launch_absmax(const float* src, int64_t rows, int64_t K, int64_t ld_row, int64_t ld_k,
                            int32_t had_block, float* amax_out, int32_t* dev_status, cudaStream_t s) {
  if (cudaMemsetAsync(amax_out, 0, sizeof(float), s) != cudaSuccess) return HDQT_ERR_CUDA;
  QuantOperand a{};
  a.src = src; a.rows = rows; a.K = K; a.ld_row = ld_row; a.ld_k = ld_k;
  QuantBatch b{};
  b.n_ops = 1;
  b.had_block = had_block;
  b.bits = 4;
  b.op[0] = make_op(a, had_block, nullptr);
  b.op[0].amax_atomic = amax_out;
  if (ld_k == 1) {
    b.op[0].num_blocks = grid_for(rows * (b.op[0].K_pad >> 3), kThreads * kUnrollAbsmax, 4);
    absmax_kc_kernel<<<b.op[0].num_blocks, kThreads, 0, s>>>(b, dev_status);
  } else {
    const int64_t items = ks_items(rows, b.op[0].K_pad, b.op[0].rt_log2);
    if (items >= (int64_t(1) << 31)) return HDQT_ERR_UNSUPPORTED;
    b.op[0].num_blocks = grid_for(items, 1, 3);
    absmax_ks_kernel<<<b.op[0].num_blocks, kThreads, 0, s>>>(b, dev_status);
  }
  return cudaGetLastError() == cudaSuccess ? HDQT_OK : HDQT_ERR_CUDA;
}

hdqt_status_t launch_calibrate_quantize(const QuantOperand* ops, int n_ops, int32_t had_block, int32_t bits,
                                        uint64_t seed, const uint32_t* philox_offset, uint32_t* partials,
                                        int32_t* dev_status, cudaStream_t s) {
  if (n_ops < 1 || n_ops > kMaxOps) return HDQT_ERR_INVALID_ARG;
  QuantOp op[kMaxOps];
  for (int i = 0; i < n_ops; ++i) {
    op[i] = make_op(ops[i], had_block, partials + (size_t)i * kMaxPartials);
    if (ops[i].ld_k != 1) {
      const int64_t items = ks_items(ops[i].rows, op[i].K_pad, op[i].rt_log2);
      if (items >= (int64_t(1) << 31)) return HDQT_ERR_UNSUPPORTED;
    }
  }
  // ---- calibration pass: operands without a supplied maximum, one launch per memory layout
  for (int layout = 0; layout < 2; ++layout) {   // 0 = K contiguous, 1 = K strided
    QuantBatch b{};
    b.had_block = had_block;
    b.bits = bits;
    int grid = 0;
    for (int i = 0; i < n_ops; ++i) {
      if ((ops[i].ld_k != 1) != (layout == 1) || ops[i].amax_in != nullptr || ops[i].hist_in != nullptr) continue;
      int g;
      QuantOp cal = op[i];
      if (layout == 0) {
        // Patch view of a convolution whose patches cover every input pixel: its 32-channel blocks are exactly the
        // blocks of the activation tensor (each kh*kw times, plus all-zero padding blocks), so the maximum is taken
        // over the tensor itself, [batch*H*W, C]: kh*kw times less to read, the same value bit for bit.
        const ConvGeom& cg = ops[i].conv;
        if (cg.enabled && cg.C % 32 == 0 && had_block == 32) {
          const int64_t kh = ops[i].K / ((int64_t)cg.KW * cg.C);
          const bool covered = cg.stride <= cg.KW && cg.stride <= kh &&
                               (int64_t)(cg.Ho - 1) * cg.stride + kh - 1 - cg.pad >= cg.H - 1 &&
                               (int64_t)(cg.Wo - 1) * cg.stride + cg.KW - 1 - cg.pad >= cg.W - 1;
          if (covered) {
            const int64_t batch = ops[i].rows / ((int64_t)cg.Ho * cg.Wo);
            cal.conv.enabled = 0;
            cal.rows = batch * cg.H * cg.W;
            cal.K = cal.K_pad = cal.ld = cg.C;
          }
        }
        g = grid_for(cal.rows * (cal.K_pad >> 3), kThreads * kUnrollAbsmax, 4);
      } else {
        g = grid_for(ks_items(op[i].rows, op[i].K_pad, op[i].rt_log2), 1, 3);
      }
      op[i].n_partials = g;
      cal.n_partials = g;
      QuantOp& o = b.op[b.n_ops++];
      o = cal;
      o.first_block = grid;
      o.num_blocks = g;
      grid += g;
    }
    if (b.n_ops == 0) continue;
    if (layout == 0) absmax_kc_kernel<<<grid, kThreads, 0, s>>>(b, dev_status);
    else absmax_ks_kernel<<<grid, kThreads, 0, s>>>(b, dev_status);
    if (cudaGetLastError() != cudaSuccess) return HDQT_ERR_CUDA;
  }
  // ---- quantize pass: one launch per kernel variant
  const PhiloxKeys keys = make_philox_keys(seed);
  for (int variant = 0; variant < 4; ++variant) {   // 0 = K contiguous, 1 = K contiguous + tile norms, 2 / 3 = K strided, nearest / stochastic
    QuantBatch b{};
    b.had_block = had_block;
    b.bits = bits;
    b.stream = philox_offset;
    int grid = 0;
    for (int i = 0; i < n_ops; ++i) {
      const int v = (ops[i].ld_k != 1) ? (ops[i].mode == HDQT_ROUND_NEAREST ? 2 : 3) : (ops[i].tile_norms != nullptr ? 1 : 0);
      if (v != variant) continue;
      int g;
      if (variant == 0) {
        g = grid_for(op[i].rows * (op[i].K_pad >> 3), kThreads * kUnrollQuant, 4);
      } else if (variant == 1) {
        const int64_t seg = int64_t(1) << op[i].seg_log2;
        g = grid_for(((op[i].rows + 127) / 128) * ((op[i].K_pad + seg - 1) / seg), 1, 4);
      } else {
        g = grid_for(ks_items(op[i].rows, op[i].K_pad, op[i].rt_log2), 1, 3);
      }
      QuantOp& o = b.op[b.n_ops++];
      o = op[i];
      o.first_block = grid;
      o.num_blocks = g;
      grid += g;
    }
    if (b.n_ops == 0) continue;
    if (variant == 0) quantize_kc_kernel<<<grid, kThreads, 0, s>>>(b, keys, dev_status);
    else if (variant == 1) quantize_kc_norms_kernel<<<grid, kThreads, 0, s>>>(b, keys, dev_status);
    else if (variant == 2) quantize_ks_kernel<1><<<grid, kThreads, 0, s>>>(b, keys, dev_status);
    else quantize_ks_kernel<2><<<grid, kThreads, 0, s>>>(b, keys, dev_status);
    if (cudaGetLastError() != cudaSuccess) return HDQT_ERR_CUDA;
  }
  return HDQT_OK;
}

}  // namespace hdqt

// ---- allocation-free variant of the transform + quantize call ----------------------------------
//
// Scratch for hdqt_quantize_hadamard_static lives in this fixed device array instead of a caller
// workspace: the partial maxima that the calibration pass hands to the quantize pass.
// Every GPU that loads the library carries these HDQT_STATIC_SCRATCH_BYTES until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HDQT_STATIC_SCRATCH_BYTES];

namespace {

std::mutex g_static_mutex;
void* g_static_scratch_ptr[hdqt::kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code the name g_static_scratch is only a handle for the runtime, not a device address;
// the address a kernel can use must be asked for, once per device, with that device current.
hdqt_status_t static_scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return hdqt::cuda_failure(e, "cudaGetDevice(static scratch)");
  if (dev < 0 || dev >= hdqt::kMaxDevices) return HDQT_ERR_UNSUPPORTED;
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
  // the stated maximum of this entry point: rows * (K_pad / 32) <= HDQT_STATIC_MAX_ROW_TILES
  const int64_t tiles = hdqt_padded_k(K, had_block) / 32;
  if (rows > (int64_t)HDQT_STATIC_MAX_ROW_TILES / tiles) return HDQT_ERR_STATIC_SCRATCH;

  unsigned char* scratch = nullptr;
  hdqt_status_t st = static_scratch_for_current_device(&scratch);
  if (st != HDQT_OK) return st;
  // the array keeps whatever the previous call left: the calibration pass overwrites every partial
  // maximum that the quantize pass of this call reads, so nothing needs clearing
  hdqt::QuantOperand a{};
  a.src = src; a.rows = rows; a.K = K; a.ld_row = ld_row; a.ld_k = ld_k;
  a.clip = clip; a.mode = mode; a.tag = tag;
  a.amax_in = nullptr;
  a.amax_slot = reinterpret_cast<float*>(scratch);
  a.codes = codes; a.step_out = step_out; a.tile_norms = tile_norms;
  return hdqt::launch_calibrate_quantize(&a, 1, had_block, bits, seed, nullptr, reinterpret_cast<uint32_t*>(scratch + 256),
                                         dev_status, reinterpret_cast<cudaStream_t>(stream));
}
