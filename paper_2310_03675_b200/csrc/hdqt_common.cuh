// Shared declarations of the HDQT CUDA library (device helpers + internal launchers).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "hdqt.h"

namespace hdqt {

constexpr int kNumSMsHint = 148;  // B200; grids are sized from the queried SM count at run time

// Sticky maximum into the caller's device status word (may be null).
__device__ __forceinline__ void report_status(int32_t* dev_status, int32_t code) {
  if (dev_status != nullptr) atomicMax(dev_status, code);
}

// ---- Philox4x32-10 (Salmon et al., SC'11): counter-based generator for stochastic rounding ----
struct Philox4 {
  uint32_t w[4];
};

// The ten round keys of Philox4x32-10 depend on the seed only: the host computes them once per launch and
// passes them as a kernel parameter, so the kernels spend no instructions on the key schedule.
struct PhiloxKeys {
  uint32_t k[10][2];
};

inline PhiloxKeys make_philox_keys(uint64_t seed) {
  PhiloxKeys keys;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    keys.k[r][0] = k0;
    keys.k[r][1] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return keys;
}

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                 const PhiloxKeys& keys) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    c0 = hi1 ^ c1 ^ keys.k[r][0];
    c1 = lo1;
    c2 = hi0 ^ c3 ^ keys.k[r][1];
    c3 = lo0;
  }
  Philox4 o;
  o.w[0] = c0; o.w[1] = c1; o.w[2] = c2; o.w[3] = c3;
  return o;
}

// Parameters of the quantizer derived from the calibration maximum (all fp32, one rounding each).
struct QuantScale {
  float m;     // 2^(bits-1) / (clip*amax): multiplier from H-domain value to code units
  float step;  // clip*amax*2^-(bits-1): value of one code unit
  bool zero;   // amax == 0 (all codes are 0)
  bool bad;    // amax or m not finite
};

__device__ __forceinline__ QuantScale make_quant_scale(float amax, float clip, int bits) {
  QuantScale q;
  const float half_range = (float)(1 << (bits - 1));
  const float t = __fmul_rn(clip, amax);
  q.m = __fdiv_rn(half_range, t);
  q.step = __fmul_rn(t, __fdiv_rn(1.0f, half_range));
  q.zero = (amax == 0.0f);
  q.bad = !(isfinite(amax)) || (!q.zero && !isfinite(q.m));
  if (q.zero || q.bad) { q.m = 0.0f; q.step = 0.0f; }
  return q;
}

// A failed CUDA call: HDQT_ERR_CUDA, with the runtime's message on stderr when HDQT_DEBUG is set.
inline hdqt_status_t cuda_failure(cudaError_t e, const char* what) {
  if (getenv("HDQT_DEBUG") != nullptr) fprintf(stderr, "[hdqt] %s: %s\n", what, cudaGetErrorString(e));
  return HDQT_ERR_CUDA;
}

// ---- internal launchers (defined in the .cu files) ----

constexpr int kMaxPartials = 1024;   // partial calibration maxima per operand (>= thread blocks of a calibration launch)

// Implicit im2col view of an NHWC activation tensor x[B, H, W, C] (paper Section 3: the transform and the
// quantizer act along the contraction dimension of the matmul a convolution lowers to): the logical matrix has
// one row per output position (b, ho, wo) and the column index runs over (kh, kw, c) with c fastest; element
// (n, k) is x[b, ho*stride + kh - pad, wo*stride + kw - pad, c], or 0 outside the image.  C must be a multiple
// of 32, so that every 32-wide block of the column index is 32 consecutive channels of one input pixel.
// Exact unsigned division by a run-time constant without a divide: q = (umulhi(n, m) + n) >> l with
// l = ceil(log2 d), m = floor(2^32 (2^l - d) / d) + 1 (round-up method; exact for every n < 2^31, where the sum
// cannot overflow).  The host fills m and l once per launch.
struct FastDiv {
  uint32_t d, m, l;
};
inline FastDiv make_fastdiv(uint32_t d) {
  FastDiv f;
  f.d = d;
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;
  f.l = l;
  f.m = (uint32_t)((((1ull << l) - d) << 32) / d + 1);
  return f;
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, const FastDiv& f) { return (__umulhi(n, f.m) + n) >> f.l; }
__device__ __forceinline__ void fastdivmod(uint32_t n, const FastDiv& f, uint32_t& q, uint32_t& r) {
  q = fastdiv(n, f);
  r = n - q * f.d;
}

struct ConvGeom {
  int32_t enabled;        // 0 = plain matrix operand
  int32_t H, W, C;        // input height, width, channels
  int32_t KW;             // kernel width (the kernel height follows from the column count)
  int32_t stride, pad;
  int32_t Ho, Wo;         // output height, width
  FastDiv div_c, div_kw, div_wo, div_ho;
};

// One operand of a transform + quantize call: logical [rows, K], element (r, k) = src[r*ld_row + k*ld_k]
// (or the implicit im2col view above: ld_k == 1 then means "the contraction runs over the patch index", anything
// else "the contraction runs over the output positions").
struct QuantOperand {
  const float* src;
  int64_t rows, K, ld_row, ld_k;
  ConvGeom conv;
  float clip;
  int32_t mode;          // hdqt_round_t
  uint32_t tag;
  const float* amax_in;  // supplied calibration maximum (device) or nullptr = measure
  const uint32_t* hist_in;  // or: kMaxPartials partial maxima left by an earlier call's quantize pass (delayed scaling)
  uint32_t* hist_out;       // optional: this call's quantize pass leaves the partial maxima of ITS tensor here
  float* amax_slot;      // optional: where the measured maximum is published
  int8_t* codes;
  float* step_out;
  int32_t* tile_norms;   // optional
};

// amax_out[0] = max |src H| (zeroes amax_out first, then one launch)
hdqt_status_t launch_absmax(const float* src, int64_t rows, int64_t K, int64_t ld_row, int64_t ld_k,
                            int32_t had_block, float* amax_out, int32_t* dev_status, cudaStream_t s);

// Calibration (for operands without a supplied maximum) and quantize passes for one or two operands that
// share had_block, bits and seed: at most one launch per pass and memory layout.
// partials: scratch of n_ops * kMaxPartials uint32.
hdqt_status_t launch_calibrate_quantize(const QuantOperand* ops, int n_ops, int32_t had_block, int32_t bits,
                                        uint64_t seed, const uint32_t* philox_offset, uint32_t* partials,
                                        int32_t* dev_status, cudaStream_t s);

// hdqt_gemm_i8_tiled plus an optional output-column bias (fp32 [N]); HDQT_FLAG_RELU in `flags` clamps at zero
hdqt_status_t gemm_i8_tiled_impl(const int8_t* Aq, const int8_t* Bq, const float* step_a, const float* step_b,
                                 int64_t M, int64_t N, int64_t K_pad, int32_t code_bits, int32_t acc_bits,
                                 int32_t acc_tile, int32_t acc_shift, int32_t had_block, float* out, int64_t ld_out,
                                 int32_t* S_out, void* tiles_out, int32_t tiles_elem_bytes, const int32_t* norms_a,
                                 const int32_t* norms_b, uint32_t flags, const float* bias, void* workspace,
                                 size_t workspace_bytes, int32_t* dev_status, void* stream);

int sm_count();   // of the current device

}  // namespace hdqt
