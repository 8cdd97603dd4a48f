// Host side of the C ABI: argument checks, workspace carving and the three training GEMMs
// composed from the transform/quantize kernels and the tiled integer GEMM (paper Section 3).
#include <string.h>

#include "hdqt_common.cuh"

using namespace hdqt;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline bool pow2_le32(int32_t n) { return n >= 1 && n <= 32 && (n & (n - 1)) == 0; }

hdqt_status_t check_quant_args(const float* src, int64_t rows, int64_t K, int64_t ld_row, int64_t ld_k,
                               int32_t had_block) {
  if (!src || rows <= 0 || K <= 0) return HDQT_ERR_INVALID_ARG;
  if (had_block < 1 || (had_block & (had_block - 1)) != 0) return HDQT_ERR_INVALID_ARG;
  if (!pow2_le32(had_block)) return HDQT_ERR_UNSUPPORTED;
  if (!((ld_k == 1 && ld_row >= K) || (ld_row == 1 && ld_k >= rows))) return HDQT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(src) & 3) return HDQT_ERR_ALIGNMENT;
  return HDQT_OK;
}

constexpr int64_t kMinBlocksForNorms = 32;
constexpr int64_t kMinHarmonicForNorms = 512;   // M N / (M + N), see run_gemm

struct OperandView {  // logical [rows, K] view of an operand with the contraction index as "K"
  const float* src;
  int64_t rows, ld_row, ld_k;
  ConvGeom conv{};    // enabled: src is an NHWC tensor and the view is its implicit im2col matrix (or its transpose)
};

}  // namespace

extern "C" const char* hdqt_status_string(hdqt_status_t s) {
  switch (s) {
    case HDQT_OK: return "ok";
    case HDQT_ERR_INVALID_ARG: return "invalid argument";
    case HDQT_ERR_UNSUPPORTED: return "unsupported parameter";
    case HDQT_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case HDQT_ERR_WORKSPACE: return "workspace too small";
    case HDQT_ERR_NONFINITE: return "non-finite value in an operand";
    case HDQT_ERR_TIMEOUT: return "bounded device wait ran out";
    case HDQT_ERR_CUDA: return "CUDA call failed";
    case HDQT_ERR_STATIC_SCRATCH: return "operand too large for the built-in scratch array";
  }
  return "unknown status";
}

extern "C" int64_t hdqt_padded_k(int64_t K, int32_t had_block) {
  const int64_t q = had_block > 32 ? had_block : 32;
  return (K + q - 1) / q * q;
}

extern "C" void hdqt_default_desc(hdqt_gemm_desc_t* d, int kind) {
  memset(d, 0, sizeof(*d));
  d->in_bits = 4;
  d->acc_bits = 8;
  d->acc_tile = 32;
  d->acc_shift = 0;
  d->had_block = 32;
  d->seed = 0;
  if (kind == 0) {         // forward: nearest rounding, clip 0.975 on activations and weights
    d->clip_a = d->clip_b = 0.975f;
    d->round_a = d->round_b = HDQT_ROUND_NEAREST;
  } else if (kind == 1) {  // dgrad: SR on the gradient, nearest on the weight
    d->clip_a = d->clip_b = 1.0f;
    d->round_a = HDQT_ROUND_STOCHASTIC;
    d->round_b = HDQT_ROUND_NEAREST;
  } else {                 // wgrad: SR on the activation and on the gradient
    d->clip_a = d->clip_b = 1.0f;
    d->round_a = d->round_b = HDQT_ROUND_STOCHASTIC;
  }
  d->tag_a = 2u * (uint32_t)kind;
  d->tag_b = 2u * (uint32_t)kind + 1u;
}

extern "C" hdqt_status_t hdqt_absmax_hadamard(const float* src, int64_t rows, int64_t K, int64_t ld_row,
                                              int64_t ld_k, int32_t had_block, float* amax_out,
                                              int32_t* dev_status, void* stream) {
  hdqt_status_t st = check_quant_args(src, rows, K, ld_row, ld_k, had_block);
  if (st != HDQT_OK) return st;
  if (!amax_out) return HDQT_ERR_INVALID_ARG;
  return launch_absmax(src, rows, K, ld_row, ld_k, had_block, amax_out, dev_status,
                       reinterpret_cast<cudaStream_t>(stream));
}

// workspace of hdqt_quantize_hadamard: [measured maximum fp32 | pad to 256 | partial maxima u32[kMaxPartials]]
extern "C" size_t hdqt_quantize_workspace_bytes(int64_t rows, int64_t K, int32_t had_block) {
  if (rows <= 0 || K <= 0 || had_block < 1) return 0;
  return 256 + sizeof(uint32_t) * (size_t)kMaxPartials;
}

extern "C" hdqt_status_t hdqt_quantize_hadamard(const float* src, int64_t rows, int64_t K, int64_t ld_row,
                                                int64_t ld_k, int32_t had_block, int32_t bits, float clip,
                                                int32_t mode, uint64_t seed, uint32_t tag, const float* amax_in,
                                                int8_t* codes, float* step_out, int32_t* tile_norms,
                                                void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                                void* stream) {
  hdqt_status_t st = check_quant_args(src, rows, K, ld_row, ld_k, had_block);
  if (st != HDQT_OK) return st;
  if (!codes || !step_out || !workspace) return HDQT_ERR_INVALID_ARG;
  if (bits < 2 || bits > 8) return HDQT_ERR_INVALID_ARG;
  if (!(clip >= 1.0f / 64.0f && clip <= 1.0f)) return HDQT_ERR_INVALID_ARG;
  if (mode != HDQT_ROUND_NEAREST && mode != HDQT_ROUND_STOCHASTIC) return HDQT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(codes) & 127) || (reinterpret_cast<uintptr_t>(workspace) & 127))
    return HDQT_ERR_ALIGNMENT;
  if (workspace_bytes < hdqt_quantize_workspace_bytes(rows, K, had_block)) return HDQT_ERR_WORKSPACE;
  QuantOperand a{};
  a.src = src; a.rows = rows; a.K = K; a.ld_row = ld_row; a.ld_k = ld_k;
  a.clip = clip; a.mode = mode; a.tag = tag;
  a.amax_in = amax_in;
  a.amax_slot = reinterpret_cast<float*>(workspace);
  a.codes = codes; a.step_out = step_out; a.tile_norms = tile_norms;
  return launch_calibrate_quantize(&a, 1, had_block, bits, seed, nullptr,
                                   reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(workspace) + 256),
                                   dev_status, reinterpret_cast<cudaStream_t>(stream));
}

// ---- the three training GEMMs -----------------------------------------------------------------

extern "C" hdqt_status_t hdqt_workspace_layout(const hdqt_gemm_desc_t* d, int64_t M, int64_t N, int64_t K,
                                               hdqt_ws_layout_t* out) {
  if (!d || !out || M <= 0 || N <= 0 || K <= 0) return HDQT_ERR_INVALID_ARG;
  if (!pow2_le32(d->had_block)) return HDQT_ERR_UNSUPPORTED;
  const int64_t K_pad = hdqt_padded_k(K, d->had_block);
  const int64_t T = K_pad / 32;
  size_t off = 0;
  out->k_pad = K_pad;
  out->step_a = off; off += 64;
  out->step_b = off; off += 64;
  out->amax_a = off; off += 64;
  out->amax_b = off; off += 64;
  out->codes_a = off; off += align_up((size_t)M * K_pad, 256);
  out->codes_b = off; off += align_up((size_t)N * K_pad, 256);
  out->norms_a = off; off += align_up((size_t)((M + 127) / 128) * T * sizeof(int32_t), 256);
  out->norms_b = off; off += align_up((size_t)((N + 127) / 128) * T * sizeof(int32_t), 256);
  out->gemm_ws = off;
  const size_t quant_ws = 2 * sizeof(uint32_t) * (size_t)kMaxPartials;   // partial maxima of both operands
  const size_t gemm_ws = hdqt_gemm_i8_workspace_bytes(M, N, K_pad);
  off += align_up(quant_ws > gemm_ws ? quant_ws : gemm_ws, 256);
  out->total = off;
  return HDQT_OK;
}

extern "C" size_t hdqt_workspace_bytes(const hdqt_gemm_desc_t* d, int64_t M, int64_t N, int64_t K) {
  hdqt_ws_layout_t l;
  if (hdqt_workspace_layout(d, M, N, K, &l) != HDQT_OK) return 0;
  return l.total;
}

namespace {

// Out[M,N] (row-major, ld_out) = A[M,K] B[K,N] with operand "a" of the descriptor feeding GEMM
// operand A unless `swap` (then descriptor operand a is the GEMM's B operand).
hdqt_status_t run_gemm(const hdqt_gemm_desc_t* d, OperandView va, OperandView vb, bool swap, int64_t K,
                       float* out, int64_t ld_out, void* workspace, size_t workspace_bytes,
                       int32_t* dev_status, void* stream) {
  if (!d || !out || !workspace) return HDQT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return HDQT_ERR_ALIGNMENT;
  // descriptor operand a -> GEMM rows M unless swapped
  const int64_t M = swap ? vb.rows : va.rows;
  const int64_t N = swap ? va.rows : vb.rows;
  hdqt_ws_layout_t L;
  hdqt_status_t st = hdqt_workspace_layout(d, M, N, K, &L);
  if (st != HDQT_OK) return st;
  if (workspace_bytes < L.total) return HDQT_ERR_WORKSPACE;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  // codes_a / step_a / norms_a always hold the GEMM's A operand (rows M)
  const OperandView& gA = swap ? vb : va;
  const OperandView& gB = swap ? va : vb;
  const float clipA = swap ? d->clip_b : d->clip_a, clipB = swap ? d->clip_a : d->clip_b;
  const int32_t roundA = swap ? d->round_b : d->round_a, roundB = swap ? d->round_a : d->round_b;
  const uint32_t tagA = swap ? d->tag_b : d->tag_a, tagB = swap ? d->tag_a : d->tag_b;
  const float* amaxA = swap ? d->amax_b : d->amax_a;
  const float* amaxB = swap ? d->amax_a : d->amax_b;
  // Tile norms are worth producing only where the GEMM can use them: merging allowed, a tile sum that can
  // exceed the accumulator at all, and enough output blocks for the merged path to pay for the blocked
  // quantize mapping (small products are bound by launch latency, not by the accumulator epilogue).
  bool merge = !(d->flags & HDQT_FLAG_NO_MERGE) && d->acc_shift == 0 && d->acc_bits >= 2 && d->acc_bits < 32 &&
               d->in_bits >= 2 && d->in_bits <= 8 && d->acc_tile >= 0;
  if (merge) {
    const int64_t tiles32 = L.k_pad / 32;
    const int64_t tpa = d->acc_tile == 0 ? tiles32 : d->acc_tile / 32;
    const int64_t code_max = int64_t(1) << (d->in_bits - 1);
    const int64_t p_max = tpa * 32 * code_max * code_max;
    const int64_t hi = (int64_t(1) << (d->acc_bits - 1)) - 1;
    const int64_t blocks = ((M + 127) / 128) * ((N + 255) / 256);
    // Tile norms (and with them the merging of clamp-free tiles) only where the GEMM outweighs the transform:
    // its work grows with M N K, the quantize passes' with (M + N) K, so the ratio is M N / (M + N).  The norm
    // output makes the quantize pass ~10 % slower and the GEMM carries the certificate bookkeeping; on the
    // convolution layers of the CNN workload (N = 64 .. 512 output channels) that cost 8 % of a training step
    // whatever the share of certified tiles, while the large square products gain up to 4x from merging.
    merge = (p_max > hi) && (blocks >= kMinBlocksForNorms) && (M * N >= kMinHarmonicForNorms * (M + N));
  }
  int32_t* normsA = merge ? reinterpret_cast<int32_t*>(ws + L.norms_a) : nullptr;
  int32_t* normsB = merge ? reinterpret_cast<int32_t*>(ws + L.norms_b) : nullptr;
  const size_t scratch_bytes = L.total - L.gemm_ws;

  // argument rules of hdqt_quantize_hadamard, checked once for both operands
  if ((st = check_quant_args(gA.src, gA.rows, K, gA.ld_row, gA.ld_k, d->had_block)) != HDQT_OK) return st;
  if ((st = check_quant_args(gB.src, gB.rows, K, gB.ld_row, gB.ld_k, d->had_block)) != HDQT_OK) return st;
  if ((gA.conv.enabled || gB.conv.enabled) && d->had_block != 32) return HDQT_ERR_UNSUPPORTED;
  if (d->in_bits < 2 || d->in_bits > 8) return HDQT_ERR_INVALID_ARG;
  if (!(clipA >= 1.0f / 64.0f && clipA <= 1.0f) || !(clipB >= 1.0f / 64.0f && clipB <= 1.0f))
    return HDQT_ERR_INVALID_ARG;
  if ((roundA != HDQT_ROUND_NEAREST && roundA != HDQT_ROUND_STOCHASTIC) ||
      (roundB != HDQT_ROUND_NEAREST && roundB != HDQT_ROUND_STOCHASTIC))
    return HDQT_ERR_INVALID_ARG;

  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (scratch_bytes < 2 * sizeof(uint32_t) * (size_t)kMaxPartials) return HDQT_ERR_WORKSPACE;
  // both operands in one calibration and one quantize launch (per memory layout); measured maxima are
  // published where the layout says (harnesses read them back)
  QuantOperand ops[2];
  const uint32_t* histInA = swap ? d->amax_hist_in_b : d->amax_hist_in_a;
  const uint32_t* histInB = swap ? d->amax_hist_in_a : d->amax_hist_in_b;
  uint32_t* histOutA = swap ? d->amax_hist_out_b : d->amax_hist_out_a;
  uint32_t* histOutB = swap ? d->amax_hist_out_a : d->amax_hist_out_b;
  ops[0] = QuantOperand{gA.src, gA.rows, K, gA.ld_row, gA.ld_k, gA.conv, clipA, roundA, tagA, amaxA, histInA, histOutA,
                        reinterpret_cast<float*>(ws + L.amax_a), reinterpret_cast<int8_t*>(ws + L.codes_a),
                        reinterpret_cast<float*>(ws + L.step_a), normsA};
  ops[1] = QuantOperand{gB.src, gB.rows, K, gB.ld_row, gB.ld_k, gB.conv, clipB, roundB, tagB, amaxB, histInB, histOutB,
                        reinterpret_cast<float*>(ws + L.amax_b), reinterpret_cast<int8_t*>(ws + L.codes_b),
                        reinterpret_cast<float*>(ws + L.step_b), normsB};
  st = launch_calibrate_quantize(ops, 2, d->had_block, d->in_bits, d->seed, d->philox_offset,
                                 reinterpret_cast<uint32_t*>(ws + L.gemm_ws), dev_status, s);
  if (st != HDQT_OK) return st;
  return gemm_i8_tiled_impl(reinterpret_cast<int8_t*>(ws + L.codes_a), reinterpret_cast<int8_t*>(ws + L.codes_b),
                            reinterpret_cast<float*>(ws + L.step_a), reinterpret_cast<float*>(ws + L.step_b), M, N,
                            L.k_pad, d->in_bits, d->acc_bits, d->acc_tile, d->acc_shift, d->had_block, out, ld_out, nullptr,
                            nullptr, 0, normsA, normsB, d->flags, d->bias, ws + L.gemm_ws, scratch_bytes, dev_status,
                            stream);
}

}  // namespace

extern "C" hdqt_status_t hdqt_gemm_fwd(const hdqt_gemm_desc_t* d, const float* X, const float* W, float* Y,
                                       int64_t Nb, int64_t D, int64_t C, int32_t w_is_cd, void* workspace,
                                       size_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!X || !W || !Y || Nb <= 0 || D <= 0 || C <= 0) return HDQT_ERR_INVALID_ARG;
  // A = X [Nb, D] (K = D contiguous); B as [C, D]: W[D,C] is K-strided, W[C,D] is K-contiguous
  OperandView a{X, Nb, D, 1};
  OperandView b = w_is_cd ? OperandView{W, C, D, 1} : OperandView{W, C, 1, C};
  return run_gemm(d, a, b, false, D, Y, C, workspace, workspace_bytes, dev_status, stream);
}

extern "C" hdqt_status_t hdqt_gemm_dgrad(const hdqt_gemm_desc_t* d, const float* G, const float* W, float* dX,
                                         int64_t Nb, int64_t D, int64_t C, int32_t w_is_cd, void* workspace,
                                         size_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!G || !W || !dX || Nb <= 0 || D <= 0 || C <= 0) return HDQT_ERR_INVALID_ARG;
  // A = G [Nb, C] (K = C contiguous); B as [D, C]: W[D,C] is K-contiguous, W[C,D] is K-strided
  OperandView a{G, Nb, C, 1};
  OperandView b = w_is_cd ? OperandView{W, D, 1, D} : OperandView{W, D, C, 1};
  return run_gemm(d, a, b, false, C, dX, D, workspace, workspace_bytes, dev_status, stream);
}

extern "C" hdqt_status_t hdqt_gemm_wgrad(const hdqt_gemm_desc_t* d, const float* X, const float* G, float* dW,
                                         int64_t Nb, int64_t D, int64_t C, int32_t w_is_cd, void* workspace,
                                         size_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!X || !G || !dW || Nb <= 0 || D <= 0 || C <= 0) return HDQT_ERR_INVALID_ARG;
  // contraction over the batch: X^T as [D, Nb] and G^T as [C, Nb], both K-strided
  OperandView a{X, D, 1, D};
  OperandView b{G, C, 1, C};
  // dW[D,C] = (X^T)(G); for the [C,D] layout the operands trade places: dW^T[C,D] = (G^T)(X)
  if (w_is_cd) return run_gemm(d, a, b, true, Nb, dW, D, workspace, workspace_bytes, dev_status, stream);
  return run_gemm(d, a, b, false, Nb, dW, C, workspace, workspace_bytes, dev_status, stream);
}

// ---- convolution as an implicit im2col GEMM ----------------------------------------------------

namespace {

hdqt_status_t conv_geom(const hdqt_conv2d_geom_t* g, ConvGeom* out, int64_t* positions, int64_t* patch) {
  if (!g || g->batch <= 0 || g->height <= 0 || g->width <= 0 || g->channels <= 0) return HDQT_ERR_INVALID_ARG;
  if (g->kernel_h <= 0 || g->kernel_w <= 0 || g->stride <= 0 || g->padding < 0) return HDQT_ERR_INVALID_ARG;
  if (g->channels % 32 != 0) return HDQT_ERR_UNSUPPORTED;     // a 32-wide K block must stay inside one input pixel
  const int64_t Ho = (g->height + 2 * g->padding - g->kernel_h) / g->stride + 1;
  const int64_t Wo = (g->width + 2 * g->padding - g->kernel_w) / g->stride + 1;
  if (Ho <= 0 || Wo <= 0) return HDQT_ERR_INVALID_ARG;
  const int64_t n = g->batch * Ho * Wo, k = (int64_t)g->kernel_h * g->kernel_w * g->channels;
  if (n >= (int64_t(1) << 31) || k >= (int64_t(1) << 31) || g->height >= (1 << 30) || g->width >= (1 << 30))
    return HDQT_ERR_UNSUPPORTED;
  out->enabled = 1;
  out->H = (int32_t)g->height; out->W = (int32_t)g->width; out->C = (int32_t)g->channels;
  out->KW = g->kernel_w; out->stride = g->stride; out->pad = g->padding;
  out->Ho = (int32_t)Ho; out->Wo = (int32_t)Wo;
  out->div_c = make_fastdiv((uint32_t)g->channels);
  out->div_kw = make_fastdiv((uint32_t)g->kernel_w);
  out->div_wo = make_fastdiv((uint32_t)Wo);
  out->div_ho = make_fastdiv((uint32_t)Ho);
  *positions = n;
  *patch = k;
  return HDQT_OK;
}

}  // namespace

extern "C" hdqt_status_t hdqt_conv2d_fwd(const hdqt_gemm_desc_t* d, const hdqt_conv2d_geom_t* g, const float* X,
                                         const float* W, float* Y, int64_t Cout, void* workspace,
                                         size_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!X || !W || !Y || Cout <= 0) return HDQT_ERR_INVALID_ARG;
  ConvGeom cg{};
  int64_t n = 0, k = 0;
  hdqt_status_t st = conv_geom(g, &cg, &n, &k);
  if (st != HDQT_OK) return st;
  // A = patches [positions, kh*kw*Cin] (contraction contiguous, gathered on the fly); B = W as [Cout, kh*kw*Cin]
  OperandView a{X, n, k, 1, cg};
  OperandView b{W, Cout, k, 1};
  return run_gemm(d, a, b, false, k, Y, Cout, workspace, workspace_bytes, dev_status, stream);
}

extern "C" hdqt_status_t hdqt_conv2d_wgrad(const hdqt_gemm_desc_t* d, const hdqt_conv2d_geom_t* g, const float* X,
                                           const float* G, float* dW, int64_t Cout, void* workspace,
                                           size_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!X || !G || !dW || Cout <= 0) return HDQT_ERR_INVALID_ARG;
  ConvGeom cg{};
  int64_t n = 0, k = 0;
  hdqt_status_t st = conv_geom(g, &cg, &n, &k);
  if (st != HDQT_OK) return st;
  // contraction over the output positions: descriptor operand a = patches^T [kh*kw*Cin, positions], operand
  // b = G^T [Cout, positions]; dW is written as [Cout, kh*kw*Cin], so the operands trade places in the GEMM
  OperandView a{X, k, 1, k, cg};
  OperandView b{G, Cout, 1, Cout};
  return run_gemm(d, a, b, true, n, dW, k, workspace, workspace_bytes, dev_status, stream);
}
