/*
 * hdqt.h - C ABI of the B200 (sm_100a) HDQT quantized training GEMM library.
 *
 * HDQT = Hadamard Domain Quantized Training (arXiv 2310.03675).  The library
 * implements the paper's quantized matrix multiply Z = X W (Section 3) for the
 * forward product and the two backward products:
 *
 *   1. block-diagonal Sylvester Hadamard transform along the contraction
 *      dimension of both operands (Section 3, "BlockDiag(H_k, ..., H_k)");
 *   2. max-calibrated uniform integer quantizer Q (Section 3, definition of Q),
 *      with stochastic rounding on the tensors the paper singles out
 *      (Section 3, sensitivity paragraph) and the 0.975 clip on the forward
 *      operands (Section 4, hyper-parameters);
 *   3. integer matrix multiply whose contraction is cut into tiles of s terms,
 *      each tile sum held in a low-bit accumulator (Section 3, "tiled
 *      quantization ... tiles of size s"; Section 4, "block-size for
 *      accumulators (32)"; Section 4.2, "8-bit integer accumulators in forward
 *      and backward-pass");
 *   4. wide sum of the tile results and a dequantising scale; no inverse
 *      transform is needed because H H^T = n I (Section 3).
 *
 * Conventions that hold for every entry point
 *   - Every pointer is a DEVICE pointer owned by the caller unless it is
 *     marked "host".  The library allocates no device memory, keeps no pointer
 *     after the call returns, and never synchronises the host: all work is
 *     enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy
 *     default stream).
 *   - Return value: HDQT_OK, or an error detected on the host before anything
 *     was launched (nothing is launched in that case).
 *   - Errors only the device can see (a non-finite input, a bounded wait that
 *     ran out) are recorded in *dev_status (device int32, sticky maximum of
 *     hdqt_status_t values; the caller zeroes it and reads it after a
 *     synchronise).  dev_status may be NULL (such errors are then dropped).
 *   - Alignment: fp32 sources and outputs 4 bytes (16 bytes, with leading
 *     dimensions that are multiples of 4, select the vector paths); code
 *     buffers and workspaces 128 bytes (256 for the three-GEMM calls).
 *   - Code layout: int8 lanes, row-major [rows, K_pad] with the contraction
 *     index contiguous, K_pad = hdqt_padded_k(K, had_block); padded entries are
 *     codes of zero-padded source entries.
 *   - Floating point: every step is IEEE binary32, round-to-nearest-even, no
 *     fused multiply-add; integer results are exact and reproducible bit for
 *     bit for a given (seed, tag).
 */
#ifndef HDQT_H_
#define HDQT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HDQT_OK = 0,
  HDQT_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, bad enum      */
  HDQT_ERR_UNSUPPORTED = 2,  /* valid in the paper's terms, not built here     */
  HDQT_ERR_ALIGNMENT = 3,    /* pointer or leading dimension not aligned       */
  HDQT_ERR_WORKSPACE = 4,    /* workspace smaller than hdqt_*_workspace_bytes  */
  HDQT_ERR_NONFINITE = 5,    /* (device) NaN/Inf in a transformed operand      */
  HDQT_ERR_TIMEOUT = 6,      /* (device) a bounded wait inside a kernel ran out*/
  HDQT_ERR_CUDA = 7,         /* a CUDA runtime / driver call failed            */
  HDQT_ERR_STATIC_SCRATCH = 8 /* operand too large for the library's built-in scratch array */
} hdqt_status_t;

typedef enum {
  HDQT_ROUND_NEAREST = 0,    /* ties to even                                   */
  HDQT_ROUND_STOCHASTIC = 1  /* Philox4x32-10 stream keyed by (seed, tag, idx) */
} hdqt_round_t;

/* flags for the GEMM entry points */
#define HDQT_FLAG_NO_MERGE 1u   /* never merge provably clamp-free tiles (see hdqt_gemm_i8_tiled) */
#define HDQT_FLAG_NO_SPLIT_K 2u /* never cut a long contraction with few output blocks into several work items */
#define HDQT_FLAG_RELU 4u       /* the three-GEMM / convolution calls: max(., 0) after the scale (and the bias)      */

/*
 * Parameters of one HDQT GEMM Out[M,N] = A[M,K] B[K,N] (Section 3).
 * Defaults of the paper: in_bits 4, acc_bits 8, acc_tile 32, had_block 32,
 * acc_shift 0; clip 0.975 forward, 1.0 backward (Section 4).
 */
typedef struct hdqt_gemm_desc {
  int32_t in_bits;    /* b   : 2..8, bit width of the operand codes                    */
  int32_t acc_bits;   /* b_a : 2..32, bit width of a tile accumulator; 32 = unquantised */
  int32_t acc_tile;   /* s   : tile length along K, a multiple of 32; 0 = whole K      */
  int32_t acc_shift;  /* r   : tile sums are divided by 2^r (round-half-even) before the
                               clamp to b_a bits; 0 = plain saturating accumulator      */
  int32_t had_block;  /* n_h : Hadamard block, power of two in 1..32; 1 = no transform  */
  float clip_a;       /* rho : operand A is scaled so that rho*max|x| maps to 2^(b-1)   */
  float clip_b;
  int32_t round_a;    /* hdqt_round_t for operand A                                    */
  int32_t round_b;
  uint64_t seed;      /* Philox key                                                    */
  uint32_t tag_a;     /* Philox stream tag per operand: counter word 2                 */
  uint32_t tag_b;
  const float* amax_a; /* optional device scalar: max|H-domain A| supplied by the caller
                          (skips the calibration pass); NULL = measure                 */
  const float* amax_b;
  uint32_t flags;     /* HDQT_FLAG_*                                                   */
  const float* bias;  /* optional device fp32 [N], N = columns of the call's output: Out = fp32(S)*scale + bias[n],
                         one fp32 multiply and one fp32 add per element, then the optional ReLU.  Bias and
                         activation are outside the quantized path (Section 3 quantizes the matmul's inputs and
                         accumulators only); fusing them saves the output's round trip.  NULL = none      */
  /* Delayed scaling (optional; Section 3 calibrates alpha from the tensor's maximum and leaves open when it
     is measured).  amax_hist_out_*: device uint32[HDQT_AMAX_HISTORY_WORDS]; the call's quantize pass leaves the
     partial maxima (fp32 bit patterns) of max|x H| of the operand it has just transformed there, at no extra
     pass.  amax_hist_in_*: such an array from an EARLIER call (the same tensor one training step before); its
     maximum replaces this call's calibration pass (4 of the 9 bytes per element), and values that have grown
     beyond it saturate at the largest code.  amax_* (the scalar) takes precedence; in and out must be
     different arrays.  NULL = not used.                                                                     */
  const uint32_t* amax_hist_in_a;
  const uint32_t* amax_hist_in_b;
  uint32_t* amax_hist_out_a;
  uint32_t* amax_hist_out_b;
  /* Optional device uint32: its value at the time the kernels run is the fourth Philox counter word of both
     operands' stochastic roundings (0 when NULL).  `seed` is fixed when a call is recorded into a CUDA graph;
     a caller who replays the graph advances this word on the device instead (one increment per training
     step), so that no two steps round with the same random numbers.                                          */
  const uint32_t* philox_offset;
} hdqt_gemm_desc_t;

#define HDQT_AMAX_HISTORY_WORDS 1024

/* Fills *d with the paper's defaults for kind 0 = forward, 1 = dgrad, 2 = wgrad
 * (rounding modes and clip per Section 3 / Section 4). `d` is a host pointer. */
void hdqt_default_desc(hdqt_gemm_desc_t* d, int kind);

/* K rounded up to whole Hadamard blocks and 32-wide tiles (zero padding leaves
 * X W unchanged; Section 3 defines H only for whole blocks). */
int64_t hdqt_padded_k(int64_t K, int32_t had_block);

const char* hdqt_status_string(hdqt_status_t s);

/* ------------------------------------------------------------------------ */
/* Transform + quantize (Section 3: Hadamard paragraph and definition of Q)   */
/* ------------------------------------------------------------------------ */

/*
 * amax_out[0] = max |x H| over the zero-padded tensor, x H being the block-
 * diagonal transform of `src` along K (the calibration maximum of Section 3).
 *
 * src: fp32, logical shape [rows, K]; element (r, k) is src[r*ld_row + k*ld_k].
 *      Exactly one of ld_row, ld_k must be 1 (K contiguous, or K strided with
 *      the row index contiguous); the other must cover the contiguous extent
 *      (ld_row >= K, resp. ld_k >= rows).  With K contiguous, a 16-byte aligned
 *      src and ld_row % 4 == 0 select 128-bit loads; anything else still works
 *      through scalar loads.
 * Non-finite values set HDQT_ERR_NONFINITE in *dev_status.
 */
hdqt_status_t hdqt_absmax_hadamard(const float* src, int64_t rows, int64_t K,
                                   int64_t ld_row, int64_t ld_k, int32_t had_block,
                                   float* amax_out, int32_t* dev_status, void* stream);

/*
 * codes[rows, K_pad] = Q(src H) with `bits`-bit two's-complement codes in int8
 * lanes; step_out[0] = value of one code unit (codes*step ~ src H).
 *
 *   t = clip*amax, v = (src H) * (2^(bits-1) / t)
 *   nearest   : code = clamp(rint(v))
 *   stochastic: code = clamp(floor((rint(v*2^16) + u16) / 2^16)), u16 = 16 bits of
 *               Philox4x32-10(counter = (g lo, g hi, tag, 0), key = seed), g = idx/8 (the GEMM calls put
 *               the descriptor's philox_offset word in place of the 0),
 *               idx = r*K_pad + k; element idx%8 takes half (idx&1) of word (idx%8)/2
 *   clamp to [-2^(bits-1), 2^(bits-1)-1]; all-zero tensor -> zero codes, step 0.
 *
 * amax_in : optional device scalar max|src H|; NULL = measure it first (one more
 *           read pass over src) into the workspace.
 * tile_norms: optional int32 [ceil(rows/128), K_pad/32]: for every block of 128
 *           rows and every 32-wide K tile, max over the rows of sum(code^2); lets
 *           the GEMM prove that a tile cannot clamp.  NULL = not produced.
 * workspace: at least hdqt_quantize_workspace_bytes(rows, K, had_block) bytes (holds the
 *           measured maximum and the partial maxima the calibration pass hands to the
 *           quantize pass).
 */
hdqt_status_t hdqt_quantize_hadamard(const float* src, int64_t rows, int64_t K,
                                     int64_t ld_row, int64_t ld_k, int32_t had_block,
                                     int32_t bits, float clip, int32_t mode,
                                     uint64_t seed, uint32_t tag, const float* amax_in,
                                     int8_t* codes, float* step_out, int32_t* tile_norms,
                                     void* workspace, size_t workspace_bytes,
                                     int32_t* dev_status, void* stream);

size_t hdqt_quantize_workspace_bytes(int64_t rows, int64_t K, int32_t had_block);

/*
 * hdqt_quantize_hadamard for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a deployment convenience, not part of the method.)
 *
 * Some callers cannot provide the workspace the call above needs, because they are not allowed
 * to call cudaMalloc (or any allocating library routine) at the point where they quantize: code
 * that runs after the application has handed all device memory to its own pool, plug-ins whose
 * host forbids allocation, or latency-critical loops that cannot afford the device-wide
 * synchronisation an allocation implies.  For them this entry point computes exactly what
 * hdqt_quantize_hadamard computes with amax_in == NULL (same codes, step and tile norms, bit for
 * bit) but takes its scratch from a fixed device array built into the library, so the call performs
 * no cudaMalloc / cudaFree and needs no workspace argument.  Inputs and outputs are still the
 * caller's buffers.
 *
 * Limits and rules
 *   - The array is HDQT_STATIC_SCRATCH_BYTES and exists once per GPU for as long as the library
 *     stays loaded.  It holds the measured maximum and the partial maxima that the calibration
 *     pass leaves for the quantize pass (one per thread block of that pass).
 *   - Stated maximum operand size: rows * (K_pad / 32) <= HDQT_STATIC_MAX_ROW_TILES (2 097 152,
 *     e.g. 8192 x 8192).  Larger operands are refused with HDQT_ERR_STATIC_SCRATCH and nothing is
 *     launched; use hdqt_quantize_hadamard then.
 *   - The first call on each device looks up the array's device address (a cheap runtime query,
 *     made with that device current); make that first call during set-up, before any stream
 *     capture you may do.
 *   - All calls on a device share the one array, and it keeps what the previous call left in it.
 *     Every entry a call reads is written by that same call first, so back-to-back calls on one
 *     stream are fine; calls that can overlap on the GPU (different streams, no ordering between
 *     them) race on the array and corrupt each other's results.
 */
#define HDQT_STATIC_SCRATCH_BYTES (256u + 4096u)
#define HDQT_STATIC_MAX_ROW_TILES 2097152

hdqt_status_t hdqt_quantize_hadamard_static(const float* src, int64_t rows, int64_t K,
                                            int64_t ld_row, int64_t ld_k, int32_t had_block,
                                            int32_t bits, float clip, int32_t mode,
                                            uint64_t seed, uint32_t tag, int8_t* codes,
                                            float* step_out, int32_t* tile_norms,
                                            int32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------ */
/* Tiled integer GEMM with low-bit tile accumulators (Section 3, last para.)  */
/* ------------------------------------------------------------------------ */

/*
 * out[m, n] = fp32(S[m, n]) * fp32(step_a*step_b*2^r / had_block),
 *   S = sum over tiles t of clamp(rne(P_t / 2^r), -2^(b_a-1), 2^(b_a-1)-1),
 *   P_t[m, n] = sum over the tile's k of Aq[m, k]*Bq[n, k]          (exact).
 *
 * Aq [M, K_pad], Bq [N, K_pad]: int8 codes, K contiguous, K_pad % 32 == 0.
 * code_bits: the caller's promise that every |code| <= 2^(code_bits-1) (2..8; 8 is always
 *     true).  It bounds the tile sums and selects the narrowest exact epilogue; codes that
 *     break the promise give undefined results.
 * step_a, step_b: device scalars written by hdqt_quantize_hadamard.
 * out   : fp32 [M, ld_out] row-major, ld_out >= N.  While the call runs, `out` may hold
 *     intermediate integer partial sums (long contractions widen their 16-bit lane sums
 *     through it); it holds the fp32 result when the kernel has finished.
 * S_out : optional int32 [M, N] (dense): the integer sums S.
 * tiles_out: optional int8/int16 debug output, see `tiles_elem_bytes`: [T, M, N]
 *     per-tile accumulator contents c_t; forces every tile through the clamp path.
 * tiles_elem_bytes: 1 (acc_bits <= 8) or 2 (acc_bits <= 16); ignored if tiles_out NULL.
 * norms_a [ceil(M/128), K_pad/32], norms_b [ceil(N/128), K_pad/32]: optional
 *     tile_norms from the quantizer.  When both are given, acc_shift == 0 and
 *     HDQT_FLAG_NO_MERGE is clear, consecutive tiles for which the Cauchy-Schwarz
 *     bound proves |P_t| <= 2^(b_a-1)-1 for a whole 128x256 output block are
 *     accumulated together on the tensor core; the clamp is the identity on such
 *     tiles, so the result is bit-identical to the tile-by-tile path.
 * workspace: at least hdqt_gemm_i8_workspace_bytes(M, N, K_pad) bytes.
 */
hdqt_status_t hdqt_gemm_i8_tiled(const int8_t* Aq, const int8_t* Bq, const float* step_a,
                                 const float* step_b, int64_t M, int64_t N, int64_t K_pad,
                                 int32_t code_bits, int32_t acc_bits, int32_t acc_tile, int32_t acc_shift,
                                 int32_t had_block, float* out, int64_t ld_out,
                                 int32_t* S_out, void* tiles_out, int32_t tiles_elem_bytes,
                                 const int32_t* norms_a, const int32_t* norms_b,
                                 uint32_t flags, void* workspace, size_t workspace_bytes,
                                 int32_t* dev_status, void* stream);

size_t hdqt_gemm_i8_workspace_bytes(int64_t M, int64_t N, int64_t K_pad);

/*
 * shift_out[0] (device int32) = smallest r >= 0 for which no tile of the given
 * operands clamps: max calibration (Section 3) of the accumulator restricted to
 * powers of two.  Operand layout as in hdqt_gemm_i8_tiled.
 */
hdqt_status_t hdqt_calibrate_acc_shift(const int8_t* Aq, const int8_t* Bq, int64_t M,
                                       int64_t N, int64_t K_pad, int32_t acc_bits,
                                       int32_t acc_tile, int32_t* shift_out,
                                       void* workspace, size_t workspace_bytes,
                                       int32_t* dev_status, void* stream);

/*
 * Diagnostic: runs the two bounded barrier waits that the GEMM kernels use (Section 3's tiled matmul is
 * a producer/consumer pipeline here) on a barrier nothing arrives at, with a budget of about a
 * millisecond, in a one-block kernel with no copy or tensor-core operation in flight.  Every waiting
 * thread must give up and the block must end normally: afterwards *dev_status holds HDQT_ERR_TIMEOUT
 * (sticky maximum, as for the GEMM kernels) and *gave_up (optional device int32, the caller zeroes it)
 * the number of threads whose wait ran out (1 spinning thread + 32 suspending ones).
 */
hdqt_status_t hdqt_selftest_bounded_wait(int32_t* dev_status, int32_t* gave_up, void* stream);

/*
 * Yardstick for the tiled matmul of Section 3 on this chip: every SM issues `iters` back-to-back
 * tcgen05.mma.kind::i8 operations of the shape the GEMM kernels use (M128 N256 K32) on operands resident in
 * shared memory - no loads, no epilogue.  The caller times the call with events; *ops_out (host, optional)
 * receives the integer operations of the launch (2*128*256*32 per MMA and SM), so that ops / time is the
 * integer tensor rate reached at the current clocks.
 */
hdqt_status_t hdqt_selftest_mma_rate(int32_t iters, int64_t* ops_out /*host*/, int32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------ */
/* The three training GEMMs of one linear layer (Section 3: Z = X W and the    */
/* backward products; X [Nb, D] activations, W weights, G = dL/dY [Nb, C])     */
/* ------------------------------------------------------------------------ */

/* W storage: w_is_cd == 0: W[D, C] row-major (the paper's W in R^{DxC});
 *            w_is_cd != 0: W[C, D] row-major (the transposed, "linear layer" layout). */

/* Y[Nb, C] = X[Nb, D] W : contraction over D. */
hdqt_status_t hdqt_gemm_fwd(const hdqt_gemm_desc_t* desc /*host*/, const float* X,
                            const float* W, float* Y, int64_t Nb, int64_t D, int64_t C,
                            int32_t w_is_cd, void* workspace, size_t workspace_bytes,
                            int32_t* dev_status, void* stream);

/* dX[Nb, D] = G[Nb, C] W^T : contraction over C. */
hdqt_status_t hdqt_gemm_dgrad(const hdqt_gemm_desc_t* desc /*host*/, const float* G,
                              const float* W, float* dX, int64_t Nb, int64_t D, int64_t C,
                              int32_t w_is_cd, void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* stream);

/* dW = X^T G : contraction over the batch Nb; dW is written in W's layout
 * ([D, C] or, if w_is_cd, [C, D]). */
hdqt_status_t hdqt_gemm_wgrad(const hdqt_gemm_desc_t* desc /*host*/, const float* X,
                              const float* G, float* dW, int64_t Nb, int64_t D, int64_t C,
                              int32_t w_is_cd, void* workspace, size_t workspace_bytes,
                              int32_t* dev_status, void* stream);

/*
 * Convolution layers without a materialised im2col matrix (Section 3: the quantized matmul Z = X W is the
 * product every layer lowers to; for a convolution X is the patch matrix of the input).  The transform and
 * quantize kernels gather the patches straight from the NHWC activation tensor.
 *
 *   X : [batch, height, width, channels] fp32, contiguous, channels % 32 == 0 (else HDQT_ERR_UNSUPPORTED:
 *       lower such a layer to hdqt_gemm_* on an explicit patch matrix)
 *   W, dW : [Cout, kernel_h, kernel_w, channels] fp32, contiguous
 *   Y, G  : [batch, Ho, Wo, Cout] fp32, contiguous, Ho = (height + 2 padding - kernel_h) / stride + 1
 * The patch matrix has one row per output position (b, ho, wo) and its column index runs over
 * (kh, kw, channel) with the channel fastest; padding pixels read as zero.  The results equal
 * hdqt_gemm_fwd / hdqt_gemm_wgrad (w_is_cd = 1) on that matrix bit for bit; only hdqt_had_block = 32 is served.
 * The data gradient of a convolution is hdqt_gemm_dgrad on G and W followed by the caller's scatter-add of the
 * patch-matrix gradient (no implicit form is provided).
 * Workspace: hdqt_workspace_bytes(desc, positions, Cout, kernel_h*kernel_w*channels) for the forward call,
 * hdqt_workspace_bytes(desc, Cout, kernel_h*kernel_w*channels, positions) for the weight gradient.
 */
typedef struct hdqt_conv2d_geom {
  int64_t batch, height, width, channels;
  int32_t kernel_h, kernel_w, stride, padding;
} hdqt_conv2d_geom_t;

hdqt_status_t hdqt_conv2d_fwd(const hdqt_gemm_desc_t* desc /*host*/, const hdqt_conv2d_geom_t* geom /*host*/,
                              const float* X, const float* W, float* Y, int64_t Cout, void* workspace,
                              size_t workspace_bytes, int32_t* dev_status, void* stream);

hdqt_status_t hdqt_conv2d_wgrad(const hdqt_gemm_desc_t* desc /*host*/, const hdqt_conv2d_geom_t* geom /*host*/,
                                const float* X, const float* G, float* dW, int64_t Cout, void* workspace,
                                size_t workspace_bytes, int32_t* dev_status, void* stream);

/* Workspace for any of the three calls on a GEMM of the given size
 * (codes of both operands, scales, tile norms, GEMM scratch). */
size_t hdqt_workspace_bytes(const hdqt_gemm_desc_t* desc /*host*/, int64_t M, int64_t N,
                            int64_t K);

/*
 * Host-side view of the workspace layout used by the three calls above, so a
 * test harness can read the intermediate codes and scales back after a call.
 * All offsets are in bytes from `workspace`.
 */
typedef struct hdqt_ws_layout {
  size_t codes_a, codes_b;   /* int8 [M, K_pad], [N, K_pad]          */
  size_t step_a, step_b;     /* fp32 scalars                         */
  size_t amax_a, amax_b;     /* fp32 scalars                         */
  size_t norms_a, norms_b;   /* int32 tile norms                     */
  size_t gemm_ws;            /* scratch of hdqt_gemm_i8_tiled        */
  size_t total;
  int64_t k_pad;
} hdqt_ws_layout_t;

hdqt_status_t hdqt_workspace_layout(const hdqt_gemm_desc_t* desc /*host*/, int64_t M,
                                    int64_t N, int64_t K, hdqt_ws_layout_t* out /*host*/);

#ifdef __cplusplus
}
#endif
#endif /* HDQT_H_ */
