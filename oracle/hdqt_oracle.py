"""CPU oracle for the HDQT quantized training GEMM (test infrastructure only).

This module is a plain, slow restatement of what the paper's method computes,
written step by step in the paper's order.  It exists so that the CUDA path can
be checked element by element; it is NOT part of the product.  Only the tests,
the smoke check and the benchmark's CPU-baseline / reference arm may import it.
It shares no code with the CUDA path and imports nothing from the package.

Method (paper Section 3):
  * quantizer  Q(x) = round(clip(alpha x) 2^(b-1)) 2^-(b-1) / alpha with alpha
    calibrated from the tensor's maximum magnitude  (Section 3, definition of Q);
  * Sylvester Hadamard matrices H_0=[1], H_k=[[H,H],[H,-H]] applied as a
    block-diagonal transform along the contraction dimension of both operands;
    because H H^T = n I the product of the transformed operands is n X W and
    no inverse transform is needed  (Section 3, Hadamard paragraph);
  * stochastic rounding on the two gradient operands and on the activation
    operand of the backward pass  (Section 3, sensitivity paragraph);
  * tiled accumulation: the contraction is cut into tiles of s (=32) terms,
    each tile's partial sum lives in a low-bit (8-bit) accumulator and the tile
    results are then summed  (Section 3, last paragraph; Section 4,
    hyper-parameters "block-size for accumulators (32)" and clip 0.975).

Arithmetic conventions (the readings this build takes where the paper is silent
are listed in the repository's design notes):
  * every floating-point step is IEEE binary32, round-to-nearest-even, one
    rounding per operation, no fused multiply-add;
  * butterflies run in ascending stride order h = 1, 2, 4, ...;
  * integer work is exact (int64 here).

Parity pins: every function below is pinned by tests/test_oracle_*.py against
facts that do not come from this file (explicit Sylvester matrices, scipy's
Hadamard routine, closed-form cases, Random123's published Philox known-answer
vectors, brute-force loops, statistical unbiasedness).  Training-level accuracy
is not covered here at all.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32

ROUND_NEAREST = 0
ROUND_STOCHASTIC = 1


# --------------------------------------------------------------------------
# Padding and the block-diagonal Hadamard transform (Section 3)
# --------------------------------------------------------------------------

def padded_k(K: int, had_block: int) -> int:
    """Length of the contraction dimension after zero padding.

    Padding with zeros up to a whole number of Hadamard blocks (and of 32-wide
    accumulator tiles) leaves X W unchanged, since padded coordinates
    contribute nothing to the product (Section 3: the block-diagonal H is only
    defined for whole blocks)."""
    q = max(32, int(had_block))
    return ((int(K) + q - 1) // q) * q


def pad_contraction(x: np.ndarray, had_block: int) -> np.ndarray:
    """x[rows, K] -> fp32 [rows, K_pad] with zeros appended along K."""
    x = np.asarray(x, dtype=F32)
    rows, K = x.shape
    Kp = padded_k(K, had_block)
    out = np.zeros((rows, Kp), dtype=F32)
    out[:, :K] = x
    return out


def fwht_blockdiag(x: np.ndarray, had_block: int) -> np.ndarray:
    """x . BlockDiag(H_n, ..., H_n) along axis 1, n = had_block, unnormalised.

    Fast Walsh-Hadamard butterflies (n log n additions, Section 3) in fp32:
    for h = 1, 2, 4, ..., n/2 every pair (i, i+h) with bit h of i clear becomes
    (x_i + x_{i+h}, x_i - x_{i+h}).  Each element is rounded once per stage."""
    x = np.array(x, dtype=F32, copy=True)
    n = int(had_block)
    assert n >= 1 and (n & (n - 1)) == 0, "Hadamard block must be a power of two"
    rows, Kp = x.shape
    assert Kp % n == 0
    blocks = x.reshape(rows, Kp // n, n)
    h = 1
    while h < n:
        nxt = np.empty_like(blocks)
        for i in range(n):
            if (i & h) == 0:
                a = blocks[:, :, i]
                b = blocks[:, :, i + h]
                nxt[:, :, i] = a + b          # fp32 add, one rounding
                nxt[:, :, i + h] = a - b      # fp32 sub, one rounding
        blocks = nxt
        h *= 2
    return blocks.reshape(rows, Kp)


# --------------------------------------------------------------------------
# Philox4x32-10 counter-based generator (Salmon et al., SC'11) for SR
# --------------------------------------------------------------------------

_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of Philox-4x32.  c0..c3: uint32 arrays (counter words),
    k0, k1: the two key words.  Returns four uint32 arrays."""
    c0 = np.asarray(c0, dtype=np.uint64)
    c1 = np.asarray(c1, dtype=np.uint64)
    c2 = np.asarray(c2, dtype=np.uint64)
    c3 = np.asarray(c3, dtype=np.uint64)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _PHILOX_M0 * c0            # 32x32 -> 64 bit products
        p1 = _PHILOX_M1 * c2
        n0 = (p1 >> np.uint64(32)) ^ c1 ^ np.uint64(k0)
        n1 = p1 & _MASK32
        n2 = (p0 >> np.uint64(32)) ^ c3 ^ np.uint64(k1)
        n3 = p0 & _MASK32
        c0, c1, c2, c3 = n0, n1, n2, n3
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return (c0.astype(np.uint32), c1.astype(np.uint32),
            c2.astype(np.uint32), c3.astype(np.uint32))


def sr_random_u16(seed: int, tag: int, idx: np.ndarray, stream: int = 0) -> np.ndarray:
    """The 16 random bits that stochastic rounding uses for element `idx`.

    idx is the element's linear index in the code layout [rows, K_pad].  Eight
    consecutive elements share one Philox call: counter = (g_lo, g_hi, tag, stream)
    with g = idx // 8, key = (seed_lo, seed_hi); element e = idx % 8 takes the
    low (e even) or high (e odd) half of output word e // 2.  `stream` (32 bits,
    0 unless the caller advances it, e.g. once per training step) selects one of
    2^32 independent streams under the same key."""
    idx = np.asarray(idx, dtype=np.uint64)
    g = idx >> np.uint64(3)
    e = (idx & np.uint64(7)).astype(np.int64)
    w = philox4x32_10(g & _MASK32, g >> np.uint64(32),
                      np.full(g.shape, int(tag) & 0xFFFFFFFF, dtype=np.uint64),
                      np.full(g.shape, int(stream) & 0xFFFFFFFF, dtype=np.uint64),
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    words = np.stack(w, axis=0).astype(np.uint64)          # [4, ...]
    word = np.take_along_axis(words, (e >> 1)[None, ...], axis=0)[0]
    half = (word >> (np.uint64(16) * (e & 1).astype(np.uint64))) & np.uint64(0xFFFF)
    return half.astype(np.int64)


def sr_random_u16_tensor(seed: int, tag: int, rows: int, K_pad: int, stream: int = 0) -> np.ndarray:
    """sr_random_u16 for every element of a [rows, K_pad] code tensor, with one
    Philox call per group of eight elements instead of one per element."""
    n = rows * K_pad
    assert n % 8 == 0
    g = np.arange(n // 8, dtype=np.uint64)
    w = philox4x32_10(g & _MASK32, g >> np.uint64(32),
                      np.full(g.shape, int(tag) & 0xFFFFFFFF, dtype=np.uint64),
                      np.full(g.shape, int(stream) & 0xFFFFFFFF, dtype=np.uint64),
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    out = np.empty((n // 8, 8), dtype=np.int64)
    for j in range(4):
        out[:, 2 * j] = w[j] & np.uint32(0xFFFF)       # even element: low half of word j
        out[:, 2 * j + 1] = w[j] >> np.uint32(16)      # odd element: high half
    return out.reshape(rows, K_pad)


# --------------------------------------------------------------------------
# Quantizer (Section 3, definition of Q; Section 4, clip factor 0.975)
# --------------------------------------------------------------------------

def quantize_transformed(xh: np.ndarray, bits: int, clip: float, mode: int,
                         seed: int = 0, tag: int = 0, amax=None, stream: int = 0):
    """Quantize an already transformed (and padded) fp32 tensor xh[rows, K_pad].

    Returns (codes int8 [rows, K_pad], step fp32, amax fp32).

      amax = max |xh| over the whole tensor          (max calibration)
      t    = clip * amax                              (fp32 multiply)
      m    = 2^(b-1) / t                              (fp32 divide) = alpha 2^(b-1)
      v    = xh * m                                   (fp32 multiply)
      nearest   : q = rint(v), ties to even
      stochastic: v_fx = rint(v * 2^16) (a Q.16 fixed-point integer),
                  q = floor((v_fx + u16) / 2^16), u16 = 16 Philox bits
                  => P(round up) = frac(v_fx / 2^16), integers never move
      code = clamp(q, -2^(b-1), 2^(b-1) - 1)          (b-bit two's complement)
      step = t * 2^-(b-1): the value of one code unit (codes * step ~ xh)
    """
    xh = np.asarray(xh, dtype=F32)
    b = int(bits)
    assert 2 <= b <= 8
    if amax is None:
        amax = F32(np.max(np.abs(xh))) if xh.size else F32(0.0)
    amax = F32(amax)
    if not np.isfinite(amax):
        raise FloatingPointError("non-finite value in the transformed tensor")
    lo, hi = -(1 << (b - 1)), (1 << (b - 1)) - 1
    if amax == 0:
        return np.zeros(xh.shape, dtype=np.int8), F32(0.0), amax
    t = F32(F32(clip) * amax)
    m = F32(F32(1 << (b - 1)) / t)
    if not np.isfinite(m):
        raise FloatingPointError("scale 2^(b-1)/t overflows fp32")
    step = F32(t * F32(2.0 ** -(b - 1)))
    v = (xh * m).astype(F32)
    if mode == ROUND_NEAREST:
        q = np.rint(v).astype(np.int64)
    elif mode == ROUND_STOCHASTIC:
        v_fx = np.rint((v * F32(65536.0)).astype(F32)).astype(np.int64)
        rows, Kp = xh.shape
        u16 = sr_random_u16_tensor(seed, tag, rows, Kp, stream)
        q = (v_fx + u16) >> 16          # arithmetic shift = floor division
    else:
        raise ValueError("unknown rounding mode")
    codes = np.clip(q, lo, hi).astype(np.int8)
    return codes, step, amax


def quantize_hadamard(src: np.ndarray, had_block: int = 32, bits: int = 4,
                      clip: float = 1.0, mode: int = ROUND_NEAREST,
                      seed: int = 0, tag: int = 0, amax=None, stream: int = 0):
    """src[rows, K] (K = contraction dim) -> (codes [rows, K_pad], step, amax).

    pad -> block-diagonal FWHT along K -> max calibration -> quantize."""
    xh = fwht_blockdiag(pad_contraction(src, had_block), had_block)
    return quantize_transformed(xh, bits, clip, mode, seed, tag, amax, stream)


# --------------------------------------------------------------------------
# Tiled integer matmul with low-bit per-tile accumulators (Section 3)
# --------------------------------------------------------------------------

def rne_shift(P: np.ndarray, r: int) -> np.ndarray:
    """Round P / 2^r to the nearest integer, ties to even (r >= 0)."""
    P = np.asarray(P, dtype=np.int64)
    r = int(r)
    if r == 0:
        return P.copy()
    fl = P >> r                              # floor(P / 2^r)
    rem = P - (fl << r)                      # 0 <= rem < 2^r
    half = 1 << (r - 1)
    up = (rem > half) | ((rem == half) & ((fl & 1) == 1))
    return fl + up.astype(np.int64)


def accumulator_quantize(P: np.ndarray, acc_bits: int, acc_shift: int) -> np.ndarray:
    """What a b_a-bit accumulator holds for the exact tile sum P:
    c = clamp(rne(P / 2^r), -2^(b_a-1), 2^(b_a-1)-1)."""
    ba = int(acc_bits)
    lo, hi = -(1 << (ba - 1)), (1 << (ba - 1)) - 1
    return np.clip(rne_shift(P, acc_shift), lo, hi)


def num_tiles(K_pad: int, acc_tile: int) -> int:
    s = int(acc_tile) if acc_tile else int(K_pad)
    return (int(K_pad) + s - 1) // s


def gemm_i8_tiled(Aq: np.ndarray, Bq: np.ndarray, step_a, step_b,
                  acc_bits: int = 8, acc_tile: int = 32, acc_shift: int = 0,
                  had_block: int = 32, want_tiles: bool = False, bias=None, relu: bool = False):
    """Out[M,N] from codes Aq[M,K_pad], Bq[N,K_pad] (both K contiguous).

    For every tile t of s consecutive k:   P_t = sum_k a[m,k] b[n,k]   (exact)
                                           c_t = accumulator_quantize(P_t)
    then S = sum_t c_t (wide integer) and
    Out = fp32(S) * fp32(step_a * step_b * 2^r / n_h)  (the 1/n_h undoes H H^T = n I).

    Returns (out fp32 [M,N], S int64 [M,N], tiles int64 [T,M,N] or None)."""
    Aq = np.asarray(Aq)
    Bq = np.asarray(Bq)
    M, Kp = Aq.shape
    N, Kp2 = Bq.shape
    assert Kp == Kp2
    s = int(acc_tile) if acc_tile else Kp
    T = num_tiles(Kp, acc_tile)
    S = np.zeros((M, N), dtype=np.int64)
    tiles = np.zeros((T, M, N), dtype=np.int64) if want_tiles else None
    for t in range(T):
        a = Aq[:, t * s:(t + 1) * s].astype(np.float64)
        b = Bq[:, t * s:(t + 1) * s].astype(np.float64)
        # products of small integers summed in fp64 are exact (|P| << 2^53)
        P = np.rint(a @ b.T).astype(np.int64)
        c = accumulator_quantize(P, acc_bits, acc_shift)
        if want_tiles:
            tiles[t] = c
        S += c
    scale = F32(np.float64(F32(step_a)) * np.float64(F32(step_b))
                * (2.0 ** int(acc_shift)) / float(had_block))
    out = (S.astype(F32) * scale).astype(F32)
    # fp32 tail outside the quantized path (only the matmul's inputs and accumulators are quantized, Section 3):
    # bias of the output column (one fp32 add), then ReLU
    if bias is not None:
        out = (out + np.asarray(bias, dtype=F32)[None, :]).astype(F32)
    if relu:
        out = np.maximum(out, F32(0.0))
    return out, S, tiles


# --------------------------------------------------------------------------
# The three training GEMMs (Section 3: Z = X W "for both forward- and
# backward-pass"; SR on both gradient operands and on the backward activation)
# --------------------------------------------------------------------------

class GemmDesc:
    """Parameters of one HDQT GEMM, defaults = the paper's 4-bit inputs,
    8-bit accumulators, tile 32 (Section 4), Hadamard block 32."""

    def __init__(self, in_bits=4, acc_bits=8, acc_tile=32, acc_shift=0,
                 had_block=32, clip_a=1.0, clip_b=1.0,
                 round_a=ROUND_NEAREST, round_b=ROUND_NEAREST,
                 seed=0, tag_a=0, tag_b=1, bias=None, relu=False, philox_offset=0):
        self.in_bits, self.acc_bits, self.acc_tile = in_bits, acc_bits, acc_tile
        self.acc_shift, self.had_block = acc_shift, had_block
        self.clip_a, self.clip_b = clip_a, clip_b
        self.round_a, self.round_b = round_a, round_b
        self.seed, self.tag_a, self.tag_b = seed, tag_a, tag_b
        self.bias, self.relu = bias, relu
        self.philox_offset = philox_offset    # fourth Philox counter word of both operands' streams


def hdqt_gemm(A_mk: np.ndarray, B_nk: np.ndarray, d: GemmDesc, want_tiles=False):
    """Out[M,N] = A[M,K] . B[N,K]^T through the whole path.  Both operands are
    given with the contraction dimension last.  Returns a dict with every
    intermediate the GPU path is compared on."""
    Aq, sa, amax_a = quantize_hadamard(A_mk, d.had_block, d.in_bits, d.clip_a,
                                       d.round_a, d.seed, d.tag_a, stream=d.philox_offset)
    Bq, sb, amax_b = quantize_hadamard(B_nk, d.had_block, d.in_bits, d.clip_b,
                                       d.round_b, d.seed, d.tag_b, stream=d.philox_offset)
    out, S, tiles = gemm_i8_tiled(Aq, Bq, sa, sb, d.acc_bits, d.acc_tile,
                                  d.acc_shift, d.had_block, want_tiles, d.bias, d.relu)
    return dict(out=out, S=S, tiles=tiles, Aq=Aq, Bq=Bq, step_a=sa, step_b=sb,
                amax_a=amax_a, amax_b=amax_b)


def fwd_desc(**kw) -> GemmDesc:
    """Forward Y = X W: nearest rounding, clip 0.975 on both (Section 4)."""
    base = dict(clip_a=0.975, clip_b=0.975, round_a=ROUND_NEAREST, round_b=ROUND_NEAREST)
    base.update(kw)
    return GemmDesc(**base)


def dgrad_desc(**kw) -> GemmDesc:
    """dX = G W^T: SR on the gradient, nearest on the weight."""
    base = dict(round_a=ROUND_STOCHASTIC, round_b=ROUND_NEAREST)
    base.update(kw)
    return GemmDesc(**base)


def wgrad_desc(**kw) -> GemmDesc:
    """dW = X^T G: SR on the activation and on the gradient."""
    base = dict(round_a=ROUND_STOCHASTIC, round_b=ROUND_STOCHASTIC)
    base.update(kw)
    return GemmDesc(**base)


def gemm_fwd(X: np.ndarray, W_dc: np.ndarray, d: GemmDesc, want_tiles=False):
    """Y[Nb,C] = X[Nb,D] W[D,C]; contraction over D."""
    return hdqt_gemm(np.asarray(X, F32), np.asarray(W_dc, F32).T, d, want_tiles)


def gemm_dgrad(G: np.ndarray, W_dc: np.ndarray, d: GemmDesc, want_tiles=False):
    """dX[Nb,D] = G[Nb,C] W[D,C]^T; contraction over C."""
    return hdqt_gemm(np.asarray(G, F32), np.asarray(W_dc, F32), d, want_tiles)


def gemm_wgrad(X: np.ndarray, G: np.ndarray, d: GemmDesc, want_tiles=False):
    """dW[D,C] = X[Nb,D]^T G[Nb,C]; contraction over the batch Nb."""
    return hdqt_gemm(np.asarray(X, F32).T, np.asarray(G, F32).T, d, want_tiles)


def calibrate_acc_shift(Aq: np.ndarray, Bq: np.ndarray, acc_bits: int = 8,
                        acc_tile: int = 32) -> int:
    """Smallest shift r >= 0 for which no tile sum clamps: the power-of-two
    form of max calibration applied to the accumulator."""
    Aq = np.asarray(Aq)
    Bq = np.asarray(Bq)
    Kp = Aq.shape[1]
    s = int(acc_tile) if acc_tile else Kp
    lo, hi = -(1 << (acc_bits - 1)), (1 << (acc_bits - 1)) - 1
    r = 0
    for t in range(num_tiles(Kp, acc_tile)):
        a = Aq[:, t * s:(t + 1) * s].astype(np.float64)
        b = Bq[:, t * s:(t + 1) * s].astype(np.float64)
        P = np.rint(a @ b.T).astype(np.int64)
        while True:
            c = rne_shift(P, r)
            if c.min() >= lo and c.max() <= hi:
                break
            r += 1
    return r
