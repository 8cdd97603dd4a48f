"""Pins for the CPU oracle: every check here compares the oracle with a fact that
does not come from the oracle itself (explicit matrices, library routines,
closed forms, published known-answer vectors, brute-force loops, statistics)."""
import os

import numpy as np
import pytest
import scipy.linalg

from oracle import hdqt_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def sylvester(n):
    """H_0 = [1], H_k = [[H, H], [H, -H]] (paper Section 3), built by recursion."""
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


# ---------------------------------------------------------------- FWHT ------

@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 32, 64])
def test_fwht_equals_explicit_sylvester_matrix(n):
    rng = np.random.default_rng(n)
    K = 2 * max(n, 32)
    x = rng.integers(-50, 50, size=(5, K)).astype(np.float32)   # exact in fp32
    got = O.fwht_blockdiag(x, n).astype(np.float64)
    H = sylvester(n)
    want = np.concatenate([x[:, b:b + n].astype(np.float64) @ H for b in range(0, K, n)], axis=1)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("n", [2, 8, 32])
def test_fwht_matches_scipy_hadamard(n):
    eye = np.eye(n, dtype=np.float32)
    assert np.array_equal(O.fwht_blockdiag(eye, n), scipy.linalg.hadamard(n).astype(np.float32))


def test_hadamard_facts():
    n = 32
    H = O.fwht_blockdiag(np.eye(n, dtype=np.float32), n).astype(np.float64)
    assert np.array_equal(H, H.T)                       # symmetric
    assert np.array_equal(H @ H.T, n * np.eye(n))       # H H^T = n I
    rng = np.random.default_rng(0)
    x = rng.integers(-100, 100, size=(7, 96)).astype(np.float32)
    twice = O.fwht_blockdiag(O.fwht_blockdiag(x, n), n)
    assert np.array_equal(twice, n * x)                 # involution up to n
    xh = O.fwht_blockdiag(x, n).astype(np.float64)
    # Parseval per block and "first output is the block sum"
    for b in range(0, 96, n):
        assert np.allclose((xh[:, b:b + n] ** 2).sum(1), n * (x[:, b:b + n].astype(np.float64) ** 2).sum(1))
        assert np.array_equal(xh[:, b], x[:, b:b + n].astype(np.float64).sum(1))


def test_fwht_blocks_are_independent():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 64)).astype(np.float32)
    y = x.copy()
    y[:, 32:] = 0
    assert np.array_equal(O.fwht_blockdiag(x, 32)[:, :32], O.fwht_blockdiag(y, 32)[:, :32])


@pytest.mark.parametrize("K", [128, 27, 100, 561])
def test_hadamard_domain_gemm_identity(K):
    """(X H)(H^T W) / n = X W to 1e-5 relative (paper Section 3), also with zero-padded K."""
    rng = np.random.default_rng(K)
    X = rng.standard_normal((16, K)).astype(np.float32)
    W = (rng.standard_normal((K, 24)) * 0.05).astype(np.float32)
    Xh = O.fwht_blockdiag(O.pad_contraction(X, 32), 32).astype(np.float64)
    Wh = O.fwht_blockdiag(O.pad_contraction(W.T.copy(), 32), 32).astype(np.float64)
    got = Xh @ Wh.T / 32.0
    want = X.astype(np.float64) @ W.astype(np.float64)
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 1e-5


def test_padding():
    assert O.padded_k(128, 32) == 128
    assert O.padded_k(27, 32) == 32
    assert O.padded_k(12, 1) == 32
    assert O.padded_k(100, 64) == 128
    p = O.pad_contraction(np.ones((2, 5), np.float32), 32)
    assert p.shape == (2, 32) and p[:, :5].sum() == 10 and p[:, 5:].sum() == 0


# ---------------------------------------------------------- Philox ----------

def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = O.philox4x32_10(*[np.array([c], dtype=np.uint32) for c in v[0:4]], v[4], v[5])
        assert [int(o[0]) for o in out] == v[6:10]


def test_sr_bits_layout_and_uniformity():
    idx = np.arange(8 * 4096, dtype=np.uint64)
    u = O.sr_random_u16(123, 5, idx)
    assert u.min() >= 0 and u.max() <= 0xFFFF
    # element e of a group takes half (e & 1) of word e >> 1 of ONE Philox call on counter (g, 0, tag, 0)
    g = 77
    w = O.philox4x32_10(np.array([g], np.uint32), np.array([0], np.uint32),
                        np.array([5], np.uint32), np.array([0], np.uint32), 123, 0)
    want = []
    for word in w:
        want += [int(word[0]) & 0xFFFF, int(word[0]) >> 16]
    assert list(u[8 * g:8 * g + 8]) == want
    # the whole-tensor form draws the same bits as the per-index form
    assert np.array_equal(O.sr_random_u16_tensor(123, 5, 64, 512).ravel(), u)
    # chi-square over 16 equal bins: 15 dof, 99.99 % quantile ~ 44.3
    counts = np.bincount(u >> 12, minlength=16)
    chi2 = ((counts - len(u) / 16) ** 2 / (len(u) / 16)).sum()
    assert chi2 < 44.3
    # other seed / tag -> another stream
    assert not np.array_equal(u, O.sr_random_u16(124, 5, idx))
    assert not np.array_equal(u, O.sr_random_u16(123, 6, idx))
    # 64-bit seeds and indices reach the high key / counter words
    assert not np.array_equal(O.sr_random_u16(1, 0, idx), O.sr_random_u16(1 + (1 << 32), 0, idx))
    assert not np.array_equal(O.sr_random_u16(1, 0, idx), O.sr_random_u16(1, 0, idx + np.uint64(1 << 35)))


# ---------------------------------------------------------- quantizer -------

def test_nearest_closed_cases():
    # amax = 8 and b = 4, clip 1  =>  t = 8, m = 1, v = x
    x = np.array([[8.0, -8.0, 0.0, 0.5, 1.5, 2.5, -0.5, -1.5, 7.49, 7.5, 7.51, -7.5, 3.2, -3.7, 0.49, -8.0]],
                 dtype=np.float32)
    x = np.concatenate([x, np.zeros((1, 16), np.float32)], axis=1)
    codes, step, amax = O.quantize_transformed(x, 4, 1.0, O.ROUND_NEAREST)
    assert amax == 8 and step == 1.0
    want = [7, -8, 0, 0, 2, 2, 0, -2, 7, 7, 7, -8, 3, -4, 0, -8]   # ties to even; +8 saturates at 7
    assert list(codes[0, :16]) == want
    assert codes.dtype == np.int8


def test_nearest_error_bound_monotone_idempotent():
    rng = np.random.default_rng(3)
    xh = rng.standard_normal((8, 64)).astype(np.float32)
    codes, step, amax = O.quantize_transformed(xh, 4, 1.0, O.ROUND_NEAREST)
    v = xh.astype(np.float64) * 8.0 / float(amax)
    inside = (v >= -8.5) & (v <= 7.5)
    err = np.abs(codes.astype(np.float64) * float(step) - xh.astype(np.float64))
    assert np.all(err[inside] <= float(step) / 2 * (1 + 1e-5))
    order = np.argsort(xh.ravel(), kind="stable")
    assert np.all(np.diff(codes.ravel()[order].astype(int)) >= 0)            # monotone
    # re-quantising the dequantised codes with the same amax gives the same codes
    again, _, _ = O.quantize_transformed((codes.astype(np.float32) * step), 4, 1.0, O.ROUND_NEAREST, amax=amax)
    assert np.array_equal(again, codes)


def test_clip_factor():
    x = np.zeros((1, 32), np.float32)
    x[0, :6] = [10.0, 9.75, 9.7, -9.9, 5.0, -10.0]
    codes, step, amax = O.quantize_transformed(x, 4, 0.975, O.ROUND_NEAREST)
    assert amax == 10.0
    assert np.isclose(float(step), 0.975 * 10 / 8)
    # everything at or above 0.975 amax * (7.5/8) saturates at 7 / below -(...) at -8
    assert list(codes[0, :6]) == [7, 7, 7, -8, 4, -8]


def test_zero_and_nonfinite():
    codes, step, amax = O.quantize_transformed(np.zeros((2, 32), np.float32), 4, 1.0, O.ROUND_NEAREST)
    assert not codes.any() and step == 0 and amax == 0
    bad = np.zeros((1, 32), np.float32)
    bad[0, 3] = np.inf
    with pytest.raises(FloatingPointError):
        O.quantize_transformed(bad, 4, 1.0, O.ROUND_NEAREST)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 8])
def test_code_range(bits):
    rng = np.random.default_rng(bits)
    x = rng.standard_normal((4, 64)).astype(np.float32)
    for mode in (O.ROUND_NEAREST, O.ROUND_STOCHASTIC):
        codes, _, _ = O.quantize_hadamard(x, 32, bits, 1.0, mode, seed=1, tag=2)
        assert codes.min() >= -(1 << (bits - 1)) and codes.max() <= (1 << (bits - 1)) - 1
        assert codes.min() == -(1 << (bits - 1)) or codes.max() == (1 << (bits - 1)) - 1   # max-calibrated


# ---------------------------------------------------------- stochastic ------

def _sr_draws(v_values, n_draws, seed):
    """Quantize a tensor holding n_draws copies of each v (plus an 8.0 that fixes amax => m = 1)."""
    cols = 32
    rows = (n_draws + cols - 1) // cols + 1
    out = {}
    for j, v in enumerate(v_values):
        x = np.full((rows, cols), v, dtype=np.float32)
        x[0, :] = 8.0
        codes, step, amax = O.quantize_transformed(x, 4, 1.0, O.ROUND_STOCHASTIC, seed=seed, tag=j)
        assert step == 1.0
        out[v] = codes[1:].ravel()[:n_draws].astype(np.int64)
    return out


def test_sr_unbiased_and_adjacent():
    """Mean of 10^4 draws within 3 sigma of the input; every draw is floor or floor + 1."""
    vs = [0.1, 0.25, 0.5, 0.75, 0.9, -0.3, -2.6, 3.375, 6.9]
    n = 10_000
    draws = _sr_draws(vs, n, seed=2024)
    for v, c in draws.items():
        f = np.floor(v)
        assert set(np.unique(c)) <= {int(f), int(f) + 1}
        frac = np.float32(v) - f
        sigma = np.sqrt(frac * (1 - frac) / n)
        assert abs(c.mean() - float(np.float32(v))) <= 3 * sigma + 2.0 ** -16


def test_sr_integers_never_move_and_top_saturates():
    vs = [0.0, 1.0, -1.0, 7.0, -8.0, 5.0]
    draws = _sr_draws(vs, 2000, seed=7)
    for v, c in draws.items():
        assert np.all(c == int(v))
    top = _sr_draws([7.5, 7.999], 2000, seed=8)
    for c in top.values():
        assert np.all(c == 7)             # code 8 is not representable in 4-bit two's complement


def test_sr_probability_is_fraction_of_fixed_point_value():
    """P(up) = frac(rint(v 2^16) / 2^16): the oracle's up-count over 2^17 independent draws of one value
    against that probability (a wrong half-word, a shifted fraction or a biased draw fails the 4-sigma gate),
    and the degenerate fractions 0 and 1 - 2^-16 exactly."""
    n = 1 << 17
    for j, v in enumerate([0.3, -1.7, 2.000031, 5.75, -0.0001]):
        draws = _sr_draws([v], n, seed=99 + j)[v]
        v_fx = int(np.rint(np.float64(np.float32(v)) * 65536.0))
        p_up = (v_fx & 0xFFFF) / 65536.0
        ups = int((draws - (v_fx >> 16)).sum())
        assert set(np.unique(draws - (v_fx >> 16))) <= {0, 1}
        assert abs(ups - n * p_up) <= 4.0 * np.sqrt(n * p_up * (1 - p_up)) + 1
    # fraction exactly 0: never up; fraction 65535/65536: up unless the draw is 0 (expected ~2 misses in 2^17)
    assert np.all(_sr_draws([3.0], 4096, seed=5)[3.0] == 3)
    top = np.float32(2.0 + 65535.0 / 65536.0)
    d = _sr_draws([float(top)], n, seed=6)[float(top)]
    assert 0 <= int((d == 2).sum()) <= 12 and np.all((d == 2) | (d == 3))


def test_sr_deterministic_and_seed_sensitive():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((16, 64)).astype(np.float32)
    a, _, _ = O.quantize_hadamard(x, 32, 4, 1.0, O.ROUND_STOCHASTIC, seed=11, tag=3)
    b, _, _ = O.quantize_hadamard(x, 32, 4, 1.0, O.ROUND_STOCHASTIC, seed=11, tag=3)
    c, _, _ = O.quantize_hadamard(x, 32, 4, 1.0, O.ROUND_STOCHASTIC, seed=12, tag=3)
    d, _, _ = O.quantize_hadamard(x, 32, 4, 1.0, O.ROUND_STOCHASTIC, seed=11, tag=4)
    n, _, _ = O.quantize_hadamard(x, 32, 4, 1.0, O.ROUND_NEAREST)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, c) and not np.array_equal(a, d)
    assert np.max(np.abs(a.astype(int) - n.astype(int))) <= 1


# ---------------------------------------------------------- tiled matmul ----

def brute_force_tiled(Aq, Bq, s, acc_bits, r):
    """Independent scalar-loop statement of the tiled low-bit accumulation."""
    M, K = Aq.shape
    N = Bq.shape[0]
    lo, hi = -(2 ** (acc_bits - 1)), 2 ** (acc_bits - 1) - 1
    S = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            total = 0
            for t0 in range(0, K, s):
                P = 0
                for k in range(t0, min(K, t0 + s)):
                    P += int(Aq[m, k]) * int(Bq[n, k])
                # round-half-even of P / 2^r with exact rational arithmetic
                q, rem = divmod(P, 2 ** r)
                if 2 * rem > 2 ** r or (2 * rem == 2 ** r and q % 2 == 1):
                    q += 1
                total += max(lo, min(hi, q))
            S[m][n] = total
    return np.array(S, dtype=np.int64)


@pytest.mark.parametrize("s,acc_bits,r", [(32, 8, 0), (32, 8, 2), (32, 4, 0), (64, 8, 1), (32, 6, 3), (0, 8, 0), (32, 12, 0)])
def test_tiled_matmul_vs_brute_force(s, acc_bits, r):
    rng = np.random.default_rng(s * 100 + acc_bits * 10 + r)
    Aq = rng.integers(-8, 8, size=(6, 128)).astype(np.int8)
    Bq = rng.integers(-8, 8, size=(5, 128)).astype(np.int8)
    out, S, tiles = O.gemm_i8_tiled(Aq, Bq, 0.5, 0.25, acc_bits, s, r, 32, want_tiles=True)
    want = brute_force_tiled(Aq, Bq, s if s else 128, acc_bits, r)
    assert np.array_equal(S, want)
    assert np.array_equal(tiles.sum(0), S)
    assert np.abs(tiles).max() <= 2 ** (acc_bits - 1)
    scale = np.float32(0.5 * 0.25 * 2 ** r / 32)
    assert np.array_equal(out, S.astype(np.float32) * scale)


def test_tiled_matmul_reduces_to_plain_matmul():
    rng = np.random.default_rng(9)
    Aq = rng.integers(-2, 3, size=(9, 96)).astype(np.int8)     # |P| <= 32*4 = 128 ... keep small
    Bq = rng.integers(-1, 2, size=(7, 96)).astype(np.int8)     # |P| <= 64: never clamps
    plain = Aq.astype(np.int64) @ Bq.astype(np.int64).T
    _, S, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, 8, 32, 0, 32)
    assert np.array_equal(S, plain)
    big_a = rng.integers(-8, 8, size=(9, 96)).astype(np.int8)
    big_b = rng.integers(-8, 8, size=(7, 96)).astype(np.int8)
    _, S32, _ = O.gemm_i8_tiled(big_a, big_b, 1.0, 1.0, 32, 32, 0, 32)
    assert np.array_equal(S32, big_a.astype(np.int64) @ big_b.astype(np.int64).T)


def test_saturating_cases():
    A = np.full((1, 64), 7, np.int8)
    B = np.full((1, 64), 7, np.int8)
    _, S, tiles = O.gemm_i8_tiled(A, B, 1.0, 1.0, 8, 32, 0, 32, want_tiles=True)
    assert tiles[:, 0, 0].tolist() == [127, 127] and S[0, 0] == 254      # 7*7*32 = 1568 -> 127
    An = np.full((1, 32), -8, np.int8)
    _, S, _ = O.gemm_i8_tiled(An, B[:, :32], 1.0, 1.0, 8, 32, 0, 32)
    assert S[0, 0] == -128
    # r = 4: only the (-8)(-8)*32 = 2048 corner (-> 128) clamps
    _, S, _ = O.gemm_i8_tiled(An, An, 1.0, 1.0, 8, 32, 4, 32)
    assert S[0, 0] == 127
    _, S, _ = O.gemm_i8_tiled(A[:, :32], B[:, :32], 1.0, 1.0, 8, 32, 4, 32)
    assert S[0, 0] == 98                                                  # 1568 / 16 = 98 exactly


def test_rne_shift_ties():
    P = np.array([8, 24, 40, -8, -24, 7, 9, -9, 0, 23, 25])
    assert O.rne_shift(P, 4).tolist() == [0, 2, 2, 0, -2, 0, 1, -1, 0, 1, 2]
    assert O.rne_shift(P, 0).tolist() == P.tolist()


def test_permutation_within_tile_only():
    rng = np.random.default_rng(10)
    Aq = rng.integers(-8, 8, size=(4, 64)).astype(np.int8)
    Bq = rng.integers(-8, 8, size=(4, 64)).astype(np.int8)
    _, S, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, 6, 32, 0, 32)
    perm = np.concatenate([rng.permutation(32), 32 + rng.permutation(32)])
    _, Sp, _ = O.gemm_i8_tiled(Aq[:, perm], Bq[:, perm], 1.0, 1.0, 6, 32, 0, 32)
    assert np.array_equal(S, Sp)
    cross = rng.permutation(64)
    _, Sc, _ = O.gemm_i8_tiled(Aq[:, cross], Bq[:, cross], 1.0, 1.0, 6, 32, 0, 32)
    assert not np.array_equal(S, Sc)       # 6-bit accumulators clamp often: tiles matter


def test_calibrate_acc_shift():
    A = np.full((2, 32), 7, np.int8)
    assert O.calibrate_acc_shift(A, A, 8, 32) == 4          # 1568 -> needs /16 (98)
    small = np.ones((2, 32), np.int8)
    assert O.calibrate_acc_shift(small, small, 8, 32) == 0
    An = np.full((2, 32), -8, np.int8)
    assert O.calibrate_acc_shift(An, An, 8, 32) == 5        # 2048/16 = 128 clamps, /32 = 64 fits


# ---------------------------------------------------------- end to end ------

# What the paper fixes per product (Section 3, sensitivity paragraph: stochastic rounding on the two gradient
# operands and on the activation of the backward pass; Section 4: clip 0.975 on the forward operands), written
# out once more here as literals and compared with the oracle's descriptor tables.
ROLE_TABLE = {
    #          round_a  round_b  clip_a  clip_b
    "fwd":   (0,       0,       0.975,  0.975),    # X nearest, W nearest
    "dgrad": (1,       0,       1.0,    1.0),      # G stochastic, W nearest
    "wgrad": (1,       1,       1.0,    1.0),      # X stochastic, G stochastic
}


def test_role_tables_follow_the_paper():
    for kind, make in (("fwd", O.fwd_desc), ("dgrad", O.dgrad_desc), ("wgrad", O.wgrad_desc)):
        d = make()
        assert (d.round_a, d.round_b, d.clip_a, d.clip_b) == ROLE_TABLE[kind], kind
        assert (d.in_bits, d.acc_bits, d.acc_tile, d.acc_shift, d.had_block) == (4, 8, 32, 0, 32), kind
    assert (O.ROUND_NEAREST, O.ROUND_STOCHASTIC) == (0, 1)


def test_three_gemms_shapes_roles_and_behaviour():
    """Shapes, which operand is transposed, and the behaviour each role implies: a nearest-rounded operand does
    not depend on the seed, a stochastically rounded one does; the forward scale carries the 0.975 clip."""
    from paper_2310_03675_b200 import inputs
    X, W, G = inputs.single_layer(0)
    runs = {}
    for seed in (0, 1):
        runs[seed] = (O.gemm_fwd(X, W, O.fwd_desc(seed=seed)), O.gemm_dgrad(G, W, O.dgrad_desc(seed=seed)),
                      O.gemm_wgrad(X, G, O.wgrad_desc(seed=seed)))
    f, d, w = runs[0]
    assert f["out"].shape == (32, 64) and f["Aq"].shape == (32, 128) and f["Bq"].shape == (64, 128)
    assert d["out"].shape == (32, 128) and d["Aq"].shape == (32, 64) and d["Bq"].shape == (128, 64)
    assert w["out"].shape == (128, 64) and w["Aq"].shape == (128, 32) and w["Bq"].shape == (64, 32)
    # operands and their transposes: each code matrix equals the quantizer run on the stated view
    for res, a_view, b_view in ((f, X, W.T), (d, G, W), (w, X.T, G.T)):
        d0 = O.GemmDesc()
        for name, view, rnd, clip, tag in (("Aq", a_view, res is not f, 0.975 if res is f else 1.0, d0.tag_a),
                                           ("Bq", b_view, res is w, 0.975 if res is f else 1.0, d0.tag_b)):
            want, _, _ = O.quantize_hadamard(np.ascontiguousarray(view), 32, 4, clip, int(rnd), seed=0, tag=tag)
            assert np.array_equal(res[name], want), name
    # seed dependence follows the rounding mode of each operand
    f1, d1, w1 = runs[1]
    assert np.array_equal(f["Aq"], f1["Aq"]) and np.array_equal(f["Bq"], f1["Bq"])          # fwd: both nearest
    assert not np.array_equal(d["Aq"], d1["Aq"]) and np.array_equal(d["Bq"], d1["Bq"])      # dgrad: G stochastic
    assert not np.array_equal(w["Aq"], w1["Aq"]) and not np.array_equal(w["Bq"], w1["Bq"])  # wgrad: both
    # the forward scale is 0.975 * max|xH| / 8 (one fp32 multiply, then an exact power of two); backward: max / 8
    xh = O.fwht_blockdiag(O.pad_contraction(X, 32), 32)
    gh = O.fwht_blockdiag(O.pad_contraction(G, 32), 32)
    amax_x, amax_g = np.float32(np.abs(xh).max()), np.float32(np.abs(gh).max())
    assert f["step_a"] == np.float32(np.float32(0.975) * amax_x) * np.float32(0.125)
    assert d["step_a"] == amax_g * np.float32(0.125)
    # with the clip, every transformed element above 0.975 max saturates at +7 / -8 (Section 4)
    v = xh / np.float32(np.float32(0.975) * amax_x) * 8
    assert np.all(f["Aq"][v >= 7.5] == 7) and np.all(f["Aq"][v <= -8.0] == -8) and (v >= 7.5).any()
    # quantised results track the exact products (4-bit operands: loose bound)
    for res, exact in ((f, X @ W), (d, G @ W.T), (w, X.T @ G)):
        rel = np.linalg.norm(res["out"] - exact) / np.linalg.norm(exact)
        assert rel < 0.6


def test_wide_accumulator_nearest_error_bound():
    """b_a = 32, nearest: |Out - X W| is bounded by the quantisation noise of the operands."""
    rng = np.random.default_rng(12)
    X = rng.standard_normal((16, 64)).astype(np.float32)
    W = rng.standard_normal((64, 8)).astype(np.float32)
    res = O.gemm_fwd(X, W, O.fwd_desc(acc_bits=32, clip_a=1.0, clip_b=1.0))
    Xh = O.fwht_blockdiag(X, 32).astype(np.float64)
    Wh = O.fwht_blockdiag(W.T.copy(), 32).astype(np.float64)
    sa, sb = float(res["step_a"]), float(res["step_b"])
    # |a_q s_a - a| <= s_a/2 except the clamped top code (<= s_a): use s_a for safety
    bound = (np.abs(Xh).sum(1)[:, None] * sb + np.abs(Wh).sum(1)[None, :] * sa + 64 * sa * sb) / 32.0
    exact = X.astype(np.float64) @ W.astype(np.float64)
    assert np.all(np.abs(res["out"] - exact) <= bound)


def test_sr_gemm_is_unbiased_on_average():
    rng = np.random.default_rng(13)
    G = (rng.standard_t(3, size=(8, 32)) * 1e-3).astype(np.float32)
    W = (rng.standard_normal((16, 32)) * 0.05).astype(np.float32)
    exact = G.astype(np.float64) @ W.astype(np.float64).T
    errs = []
    acc = np.zeros_like(exact)
    R = 256
    for seed in range(R):
        res = O.gemm_dgrad(G, W, O.dgrad_desc(acc_bits=32, round_b=O.ROUND_STOCHASTIC, seed=seed))
        acc += res["out"]
        if seed + 1 in (16, 256):
            errs.append(np.linalg.norm(acc / (seed + 1) - exact) / np.linalg.norm(exact))
    # 16x more samples -> about 4x less error; allow slack
    assert errs[1] < errs[0] / 2.5


def test_bias_and_relu_tail_is_plain_fp32_arithmetic():
    """The optional fp32 tail of the epilogue equals bias add and ReLU applied to the unfused result."""
    rng = np.random.default_rng(21)
    Aq = rng.integers(-8, 8, size=(9, 64)).astype(np.int8)
    Bq = rng.integers(-8, 8, size=(5, 64)).astype(np.int8)
    bias = rng.standard_normal(5).astype(np.float32)
    plain, S, _ = O.gemm_i8_tiled(Aq, Bq, 0.01, 0.5)
    fused, S2, _ = O.gemm_i8_tiled(Aq, Bq, 0.01, 0.5, bias=bias, relu=True)
    assert np.array_equal(S, S2)
    want = np.maximum((plain + bias[None, :]).astype(np.float32), np.float32(0))
    assert np.array_equal(fused, want) and (fused == 0).any() and (fused > 0).any()
    only_bias, _, _ = O.gemm_i8_tiled(Aq, Bq, 0.01, 0.5, bias=bias)
    assert np.array_equal(only_bias, (plain + bias[None, :]).astype(np.float32))
    X = rng.standard_normal((6, 40)).astype(np.float32)
    W = rng.standard_normal((40, 5)).astype(np.float32)
    a = O.gemm_fwd(X, W, O.fwd_desc())["out"]
    b = O.gemm_fwd(X, W, O.fwd_desc(bias=bias, relu=True))["out"]
    assert np.array_equal(b, np.maximum((a + bias).astype(np.float32), 0))


def test_sr_stream_word_is_the_fourth_philox_counter_word():
    """`stream` selects the fourth counter word of the Philox call behind the 16 rounding bits: stream 0 is the
    plain generator, any other value gives different bits for the same (seed, tag, index), and the choice reaches
    the codes of a stochastic quantization but not those of a nearest one."""
    idx = np.arange(64, dtype=np.uint64) + 8 * 12345
    base = O.sr_random_u16(3, 9, idx)
    assert np.array_equal(base, O.sr_random_u16(3, 9, idx, stream=0))
    other = O.sr_random_u16(3, 9, idx, stream=2)
    assert (base != other).mean() > 0.9
    g = int(idx[8] >> 3)
    w = O.philox4x32_10(np.array([g], np.uint32), np.array([0], np.uint32), np.array([9], np.uint32),
                        np.array([2], np.uint32), 3, 0)
    assert other[8] == int(w[0][0]) & 0xFFFF and other[11] == int(w[1][0]) >> 16
    assert np.array_equal(O.sr_random_u16_tensor(3, 9, 4, 32, stream=2).ravel()[:64], O.sr_random_u16(3, 9, np.arange(64), stream=2))
    x = np.random.default_rng(0).standard_normal((8, 64)).astype(np.float32)
    q0 = O.quantize_hadamard(x, mode=O.ROUND_STOCHASTIC, seed=1, tag=2)[0]
    q1 = O.quantize_hadamard(x, mode=O.ROUND_STOCHASTIC, seed=1, tag=2, stream=1)[0]
    assert not np.array_equal(q0, q1) and np.abs(q0.astype(int) - q1.astype(int)).max() <= 1
    n0 = O.quantize_hadamard(x, mode=O.ROUND_NEAREST, seed=1, tag=2)[0]
    assert np.array_equal(n0, O.quantize_hadamard(x, mode=O.ROUND_NEAREST, seed=1, tag=2, stream=1)[0])
