"""GPU parity: tiled integer GEMM and the three training GEMMs against the CPU oracle.
Integers (codes, per-tile accumulators, sums) bit-exact; fp32 outputs within 1e-5 relative."""
import numpy as np
import pytest
import torch

from oracle import hdqt_oracle as O
from paper_2310_03675_b200 import inputs

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5   # fp32 output tolerance stated for this path (in practice the outputs are identical)


@pytest.fixture(scope="module")
def hdqt():
    from paper_2310_03675_b200 import hdqt as mod
    return mod


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _assert_close(got, want):
    got = got.astype(np.float64)
    want = want.astype(np.float64)
    denom = max(np.abs(want).max(), 1e-30)
    assert np.abs(got - want).max() / denom <= REL_TOL


def _codes(rng, rows, K, lo=-8, hi=8):
    return rng.integers(lo, hi, size=(rows, K)).astype(np.int8)


GEMM_SHAPES = [(32, 64, 128), (1, 1, 32), (128, 256, 32), (129, 257, 160), (300, 520, 416), (64, 12, 256), (260, 100, 96)]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
def test_i8_tiled_default_parameters(hdqt, M, N, K):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
    sa, sb = np.float32(0.0123), np.float32(3.5e-4)
    want_out, want_S, want_tiles = O.gemm_i8_tiled(Aq, Bq, sa, sb, 8, 32, 0, 32, want_tiles=True)
    status = hdqt.new_status("cuda")
    out, S, tiles = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), torch.tensor([sa], device="cuda"),
                                       torch.tensor([sb], device="cuda"), want_S=True, want_tiles=True,
                                       dev_status=status)
    hdqt.check_device_status(status)
    assert np.array_equal(tiles.cpu().numpy().astype(np.int64), want_tiles)
    assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)
    _assert_close(out.cpu().numpy(), want_out)
    # and without the debug output (the production kernel variant)
    out2, S2, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), torch.tensor([sa], device="cuda"),
                                     torch.tensor([sb], device="cuda"), want_S=True, dev_status=status)
    hdqt.check_device_status(status)
    assert np.array_equal(S2.cpu().numpy().astype(np.int64), want_S)
    assert np.array_equal(out2.cpu().numpy(), out.cpu().numpy())


@pytest.mark.parametrize("acc_bits,acc_tile,acc_shift", [(8, 32, 2), (8, 32, 4), (4, 32, 0), (6, 32, 3), (12, 32, 0),
                                                         (16, 64, 0), (8, 64, 1), (8, 128, 3), (8, 0, 0), (32, 0, 0),
                                                         (32, 32, 0), (8, 96, 0)])
def test_i8_tiled_parameter_family(hdqt, acc_bits, acc_tile, acc_shift):
    rng = np.random.default_rng(acc_bits * 100 + acc_tile + acc_shift)
    M, N, K = 140, 270, 448
    Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
    sa, sb = np.float32(0.5), np.float32(0.25)
    want_tiles_flag = acc_bits <= 16
    want_out, want_S, want_tiles = O.gemm_i8_tiled(Aq, Bq, sa, sb, acc_bits, acc_tile, acc_shift, 32,
                                                   want_tiles=want_tiles_flag)
    status = hdqt.new_status("cuda")
    out, S, tiles = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), torch.tensor([sa], device="cuda"),
                                       torch.tensor([sb], device="cuda"), acc_bits, acc_tile, acc_shift, 32,
                                       want_S=True, want_tiles=want_tiles_flag, dev_status=status)
    hdqt.check_device_status(status)
    if want_tiles_flag:
        assert np.array_equal(tiles.cpu().numpy().astype(np.int64), want_tiles)
    assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)
    _assert_close(out.cpu().numpy(), want_out)


def test_i8_tiled_saturating_and_8bit_codes(hdqt):
    """All-7 codes clamp every tile at 127; full-range int8 codes exercise the signed 8-bit MMA path."""
    A = np.full((130, 96), 7, np.int8)
    B = np.full((20, 96), 7, np.int8)
    one = torch.ones(1, device="cuda")
    _, S, _ = hdqt.gemm_i8_tiled(_dev(A), _dev(B), one, one, want_S=True)
    assert (S == 3 * 127).all().item()
    _, S, _ = hdqt.gemm_i8_tiled(_dev(-A - 1), _dev(B), one, one, want_S=True)      # -8 * 7 * 32 -> -128
    assert (S == 3 * -128).all().item()
    rng = np.random.default_rng(3)
    A8, B8 = _codes(rng, 64, 128, -128, 128), _codes(rng, 48, 128, -128, 128)
    _, want_S, _ = O.gemm_i8_tiled(A8, B8, 1.0, 1.0, 32, 0, 0, 32)
    _, S, _ = hdqt.gemm_i8_tiled(_dev(A8), _dev(B8), one, one, 32, 0, 0, 32, code_bits=8, want_S=True)
    assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)


def test_i8_tiled_strided_output_and_canaries(hdqt):
    rng = np.random.default_rng(5)
    M, N, K = 70, 33, 64
    Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
    want_out, _, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0)
    big = torch.full((M + 2, N + 7), -777.0, device="cuda")
    view = big[1:M + 1, 3:3 + N]
    one = torch.ones(1, device="cuda")
    hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, out=view)
    torch.cuda.synchronize()
    assert np.array_equal(view.cpu().numpy(), want_out)
    mask = torch.ones_like(big, dtype=torch.bool)
    mask[1:M + 1, 3:3 + N] = False
    assert (big[mask] == -777.0).all().item()


def test_calibrate_acc_shift(hdqt):
    rng = np.random.default_rng(6)
    for lo, hi, bits in ((-8, 8, 8), (-2, 3, 8), (-8, 8, 6), (-8, 8, 12)):
        Aq, Bq = _codes(rng, 40, 96, lo, hi), _codes(rng, 24, 96, lo, hi)
        want = O.calibrate_acc_shift(Aq, Bq, bits, 32)
        got = hdqt.calibrate_acc_shift(_dev(Aq), _dev(Bq), bits, 32).item()
        assert got == want


# ---- the three training GEMMs ----------------------------------------------------------------------

def _run_three(hdqt, X, W, G, w_is_cd=False, **over):
    """Runs fwd/dgrad/wgrad on the GPU and through the oracle; compares every intermediate."""
    Xd, Gd = _dev(X), _dev(G)
    Wd = _dev(W.T) if w_is_cd else _dev(W)
    status = hdqt.new_status("cuda")
    cases = [
        ("fwd", hdqt.gemm_fwd, (Xd, Wd), O.gemm_fwd(X, W, O.fwd_desc(tag_a=0, tag_b=1, **over)), False),
        ("dgrad", hdqt.gemm_dgrad, (Gd, Wd), O.gemm_dgrad(G, W, O.dgrad_desc(tag_a=2, tag_b=3, **over)), False),
        ("wgrad", hdqt.gemm_wgrad, (Xd, Gd), O.gemm_wgrad(X, G, O.wgrad_desc(tag_a=4, tag_b=5, **over)), True),
    ]
    for kind, fn, args, want, is_wgrad in cases:
        desc = hdqt.default_desc(kind, **over)
        out, ws = fn(*args, desc=desc, w_is_cd=w_is_cd, dev_status=status)
        hdqt.check_device_status(status, kind)
        swapped = is_wgrad and w_is_cd
        got_a, got_b = ws.codes_a().cpu().numpy(), ws.codes_b().cpu().numpy()
        sa, sb = ws.scalar("step_a").item(), ws.scalar("step_b").item()
        if swapped:
            got_a, got_b, sa, sb = got_b, got_a, sb, sa
        assert np.array_equal(got_a, want["Aq"]), kind
        assert np.array_equal(got_b, want["Bq"]), kind
        assert sa == float(want["step_a"]) and sb == float(want["step_b"]), kind
        want_out = want["out"].T if swapped else want["out"]
        _assert_close(out.cpu().numpy(), want_out)
        # integer sums: re-run the integer GEMM on the codes the library produced
        _, S, tiles = hdqt.gemm_i8_tiled(ws.codes_a(), ws.codes_b(), ws.scalar("step_a"), ws.scalar("step_b"),
                                         desc.acc_bits, desc.acc_tile, desc.acc_shift, desc.had_block,
                                         code_bits=desc.in_bits, want_S=True, want_tiles=desc.acc_bits <= 16)
        # the production variants (no per-tile debug output; with and without clamp-free tile merging)
        for flags in (0, hdqt.FLAG_NO_MERGE):
            _, S2, _ = hdqt.gemm_i8_tiled(ws.codes_a(), ws.codes_b(), ws.scalar("step_a"), ws.scalar("step_b"),
                                          desc.acc_bits, desc.acc_tile, desc.acc_shift, desc.had_block,
                                          code_bits=desc.in_bits, want_S=True, flags=flags)
            assert torch.equal(S2, S), (kind, flags)
        want_S = want["S"].T if swapped else want["S"]
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), kind
        if tiles is not None:
            _, _, want_tiles = O.gemm_i8_tiled(want["Aq"], want["Bq"], 1, 1, desc.acc_bits, desc.acc_tile,
                                               desc.acc_shift, desc.had_block, want_tiles=True)
            if swapped:
                want_tiles = want_tiles.transpose(0, 2, 1)
            assert np.array_equal(tiles.cpu().numpy().astype(np.int64), want_tiles), kind


@pytest.mark.parametrize("w_is_cd", [False, True])
def test_single_linear_layer(hdqt, w_is_cd):
    """X [32,128] ~ N(0,1), W [128,64] ~ N(0,0.05^2), G [32,64] ~ 1e-3 t(3); seed 0."""
    X, W, G = inputs.single_layer(0)
    _run_three(hdqt, X, W, G, w_is_cd=w_is_cd, seed=0)


@pytest.mark.parametrize("Nb,D,C", [(256, 1152, 512), (256, 512, 256), (256, 256, 12), (128, 561, 561), (128, 27, 64),
                                    (130, 100, 7)])
def test_mlp_and_ragged_layers(hdqt, Nb, D, C):
    X = np.maximum(inputs.activations(Nb, D, seed=D), 0)        # post-ReLU activations
    W = inputs.weights(D, C, seed=C)
    G = inputs.gradients(Nb, C, seed=Nb + C)
    _run_three(hdqt, X, W, G, seed=42)


@pytest.mark.parametrize("over", [dict(acc_bits=12), dict(acc_bits=4), dict(in_bits=3, acc_bits=6), dict(in_bits=8, acc_bits=16),
                                  dict(acc_tile=0), dict(had_block=1), dict(acc_shift=2), dict(acc_tile=64, acc_shift=1)])
def test_bit_width_family_and_paper_arrangement(hdqt, over):
    X, W, G = inputs.single_layer(1, Nb=96, D=160, C=72)
    _run_three(hdqt, X, W, G, seed=7, **over)


def test_im2col_like_wgrad_long_contraction(hdqt):
    """wgrad with a long batch contraction (many tiles) and a narrow output."""
    X = np.maximum(inputs.activations(4096, 576, seed=11), 0)
    G = inputs.gradients(4096, 64, seed=12)
    W = inputs.weights(576, 64, seed=13)
    _run_three(hdqt, X, W, G, seed=3)


def test_runs_are_bitwise_reproducible(hdqt):
    X, W, G = inputs.single_layer(2, Nb=200, D=300, C=150)
    Xd, Gd = _dev(X), _dev(G)
    a, _ = hdqt.gemm_wgrad(Xd, Gd)
    b, _ = hdqt.gemm_wgrad(Xd, Gd)
    assert torch.equal(a, b)
    c, _ = hdqt.gemm_wgrad(Xd, Gd, desc=hdqt.default_desc("wgrad", seed=1))
    assert not torch.equal(a, c)


@pytest.mark.parametrize("size", [4096, 8192, 16384])
def test_sampled_parity_at_sweep_size(hdqt, size):
    """Sweep-size dgrad-layout GEMM on heavy-tailed operands (16384 = the shape and launch configuration the
    benchmark's headline times): codes in full, outputs on sampled rows and columns."""
    M = N = K = size
    A = inputs.heavy_tailed_torch(M, K, seed=100, device="cuda")
    B = inputs.heavy_tailed_torch(N, K, seed=101, device="cuda")
    desc = hdqt.default_desc("dgrad", seed=9)
    status = hdqt.new_status("cuda")
    out, ws = hdqt.gemm_dgrad(A, B, desc=desc, dev_status=status)
    hdqt.check_device_status(status)
    want_a, sa, _ = O.quantize_hadamard(A.cpu().numpy(), 32, 4, 1.0, 1, seed=9, tag=desc.tag_a)
    want_b, sb, _ = O.quantize_hadamard(B.cpu().numpy(), 32, 4, 1.0, 0, seed=9, tag=desc.tag_b)
    assert np.array_equal(ws.codes_a().cpu().numpy(), want_a)
    assert np.array_equal(ws.codes_b().cpu().numpy(), want_b)
    assert ws.scalar("step_a").item() == float(sa) and ws.scalar("step_b").item() == float(sb)
    rng = np.random.default_rng(0)
    rows = np.sort(rng.choice(M, 64, replace=False))
    cols = np.sort(rng.choice(N, 64, replace=False))
    got = out.cpu().numpy()
    want_rows, _, _ = O.gemm_i8_tiled(want_a[rows], want_b, sa, sb)
    want_cols, _, _ = O.gemm_i8_tiled(want_a, want_b[cols], sa, sb)
    _assert_close(got[rows], want_rows)
    _assert_close(got[:, cols], want_cols)
    assert np.array_equal(got[rows], want_rows) and np.array_equal(got[:, cols], want_cols)


# ---- clamp-free tile merging and the 16-bit-lane epilogue --------------------------------------------

def _tile_norms(codes):
    rows, Kp = codes.shape
    sq = (codes.astype(np.int64) ** 2).reshape(rows, Kp // 32, 32).sum(2)
    nb = (rows + 127) // 128
    return np.stack([sq[b * 128:(b + 1) * 128].max(0) for b in range(nb)]).astype(np.int32)


def _sparse_codes(rng, rows, K, density):
    c = rng.integers(-8, 8, size=(rows, K))
    return (c * (rng.random((rows, K)) < density)).astype(np.int8)


@pytest.mark.parametrize("density_a,density_b", [(0.05, 0.05), (0.3, 0.1), (1.0, 0.02), (1.0, 1.0)])
@pytest.mark.parametrize("acc_bits,acc_tile", [(8, 32), (8, 64), (6, 32)])
def test_merging_is_bit_identical(hdqt, density_a, density_b, acc_bits, acc_tile):
    """Mixed certified / uncertified tiles: merged, unmerged and oracle sums agree exactly."""
    rng = np.random.default_rng(int(density_a * 100) * 7 + int(density_b * 100) + acc_bits + acc_tile)
    M, N, K = 200, 300, 1024
    Aq, Bq = _sparse_codes(rng, M, K, density_a), _sparse_codes(rng, N, K, density_b)
    # make certification vary along K: a dense stripe of tiles
    Aq[:, 256:384] = rng.integers(-8, 8, size=(M, 128))
    Bq[:, 320:448] = rng.integers(-8, 8, size=(N, 128))
    _, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, acc_bits, acc_tile, 0, 32)
    one = torch.ones(1, device="cuda")
    na, nb = _dev(_tile_norms(Aq)), _dev(_tile_norms(Bq))
    status = hdqt.new_status("cuda")
    for flags in (0, hdqt.FLAG_NO_MERGE):
        _, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, acc_bits, acc_tile, 0, 32, want_S=True,
                                     norms_a=na, norms_b=nb, flags=flags, dev_status=status)
        hdqt.check_device_status(status)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), flags


def test_merging_with_norms_from_the_quantizer(hdqt):
    """Heavy-tailed operands: most tiles certify; the composite call (merging on) equals the oracle."""
    A = inputs.heavy_tailed(300, 2048, seed=21)
    B = inputs.heavy_tailed(520, 2048, seed=22)
    want = O.gemm_dgrad(A, B, O.dgrad_desc(seed=3, tag_a=2, tag_b=3))
    status = hdqt.new_status("cuda")
    out, ws = hdqt.gemm_dgrad(_dev(A), _dev(B), desc=hdqt.default_desc("dgrad", seed=3), dev_status=status)
    hdqt.check_device_status(status)
    assert np.array_equal(out.cpu().numpy(), want["out"])
    out2, _ = hdqt.gemm_dgrad(_dev(A), _dev(B), desc=hdqt.default_desc("dgrad", seed=3, flags=hdqt.FLAG_NO_MERGE))
    assert torch.equal(out, out2)
    # the certified fraction is what makes merging worthwhile on such data: check it is large
    na = _tile_norms(want["Aq"]).astype(np.int64)
    nb = _tile_norms(want["Bq"]).astype(np.int64)
    nb256 = np.stack([nb[2 * j:2 * j + 2].max(0) for j in range((nb.shape[0] + 1) // 2)])
    cert = (na[:, None, :] * nb256[None, :, :]) <= 127 * 127
    assert cert.mean() > 0.9


def test_long_contraction_widens_packed_sums(hdqt):
    """More than 256 clamp tiles: the 16-bit lane sums are widened through the output buffer."""
    rng = np.random.default_rng(31)
    M, N, K = 130, 70, 32 * 700
    Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
    Aq[:, :] = np.where(rng.random((M, K)) < 0.5, 7, Aq)       # push many tiles into saturation
    want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 0.5, 0.125)
    half, eighth = torch.tensor([0.5], device="cuda"), torch.tensor([0.125], device="cuda")
    # odd leading dimension: exercises the scalar store path of the widening too
    big = torch.zeros((M, N + 3), device="cuda")
    for view in (None, big[:, 1:N + 1]):
        # split-K off: one work item walks all 700 tiles and widens its 16-bit lane sums twice
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), half, eighth, want_S=True, out=view,
                                       flags=hdqt.FLAG_NO_SPLIT_K)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)
        assert np.array_equal(out.cpu().numpy(), want_out)
        # split-K on (the default for so few output blocks): same integers, same fp32 values
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), half, eighth, want_S=True, out=view)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)
        assert np.array_equal(out.cpu().numpy(), want_out)
    assert (big[:, 0] == 0).all().item() and (big[:, N + 1:] == 0).all().item()


@pytest.mark.parametrize("acc_bits,acc_tile,acc_shift,K", [(8, 32, 0, 32 * 1001), (8, 96, 0, 32 * 999), (12, 32, 0, 32 * 515),
                                                           (8, 64, 2, 32 * 640), (6, 32, 0, 32 * 77), (16, 128, 0, 32 * 400)])
def test_split_k_matches_the_oracle(hdqt, acc_bits, acc_tile, acc_shift, K):
    """Long contraction, one or two output blocks: the contraction is cut into work items whose integer sums are
    added up atomically (exact, order-free).  Ragged last item, accumulator tiles of 1, 2, 3 and 4 K tiles, the
    16-bit-lane and the 32-bit epilogue, with and without a rounding shift, ragged M and N."""
    rng = np.random.default_rng(K + acc_bits)
    M, N = 70, 300
    Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
    want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 0.5, 0.25, acc_bits, acc_tile, acc_shift, 32)
    half, quarter = torch.tensor([0.5], device="cuda"), torch.tensor([0.25], device="cuda")
    status = hdqt.new_status("cuda")
    for flags in (0, hdqt.FLAG_NO_SPLIT_K):
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), half, quarter, acc_bits, acc_tile, acc_shift, 32,
                                       want_S=True, flags=flags, dev_status=status)
        hdqt.check_device_status(status)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), flags
        assert np.array_equal(out.cpu().numpy(), want_out), flags


def test_wide_accumulators_merge_without_norms(hdqt):
    """b_a >= 13 with 4-bit codes: no tile can clamp, every tile is merged; equals the plain int matmul."""
    rng = np.random.default_rng(32)
    Aq, Bq = _codes(rng, 150, 480), _codes(rng, 260, 480)
    plain = Aq.astype(np.int64) @ Bq.astype(np.int64).T
    one = torch.ones(1, device="cuda")
    for acc_bits in (13, 16, 32):
        _, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, acc_bits, 32, 0, 32, want_S=True)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), plain)


@pytest.mark.parametrize("size", [4096, 8192])
def test_sampled_parity_wgrad_layout_at_sweep_size(hdqt, size):
    """Sweep-size wgrad layout (both operands K-strided, both stochastic): codes in full, outputs sampled."""
    M = N = K = size
    X = inputs.heavy_tailed_torch(K, M, seed=200, device="cuda")     # stored [Nb, D]: contraction index first
    G = inputs.heavy_tailed_torch(K, N, seed=201, device="cuda")
    desc = hdqt.default_desc("wgrad", seed=5)
    status = hdqt.new_status("cuda")
    out, ws = hdqt.gemm_wgrad(X, G, desc=desc, dev_status=status)
    hdqt.check_device_status(status)
    want_a, sa, _ = O.quantize_hadamard(X.cpu().numpy().T, 32, 4, 1.0, 1, seed=5, tag=desc.tag_a)
    want_b, sb, _ = O.quantize_hadamard(G.cpu().numpy().T, 32, 4, 1.0, 1, seed=5, tag=desc.tag_b)
    assert np.array_equal(ws.codes_a().cpu().numpy(), want_a)
    assert np.array_equal(ws.codes_b().cpu().numpy(), want_b)
    rng = np.random.default_rng(1)
    rows = np.sort(rng.choice(M, 48, replace=False))
    cols = np.sort(rng.choice(N, 48, replace=False))
    got = out.cpu().numpy()
    want_rows, _, _ = O.gemm_i8_tiled(want_a[rows], want_b, sa, sb)
    want_cols, _, _ = O.gemm_i8_tiled(want_a, want_b[cols], sa, sb)
    assert np.array_equal(got[rows], want_rows) and np.array_equal(got[:, cols], want_cols)


def test_tall_skinny_conv_like_shapes(hdqt):
    """im2col-like layer: 32768 x 576 activations, 64 output channels (many row blocks, one column block)."""
    Nb, D, C = 32768, 576, 64
    X = np.maximum(inputs.activations(Nb, D, seed=31), 0)
    W = inputs.weights(D, C, seed=32)
    G = inputs.gradients(Nb, C, seed=33)
    status = hdqt.new_status("cuda")
    Xd, Wd, Gd = _dev(X), _dev(W), _dev(G)
    for kind, fn, args, want in (
            ("fwd", hdqt.gemm_fwd, (Xd, Wd), O.gemm_fwd(X, W, O.fwd_desc(tag_a=0, tag_b=1, seed=2))),
            ("dgrad", hdqt.gemm_dgrad, (Gd, Wd), O.gemm_dgrad(G, W, O.dgrad_desc(tag_a=2, tag_b=3, seed=2))),
            ("wgrad", hdqt.gemm_wgrad, (Xd, Gd), O.gemm_wgrad(X, G, O.wgrad_desc(tag_a=4, tag_b=5, seed=2)))):
        out, ws = fn(*args, desc=hdqt.default_desc(kind, seed=2), dev_status=status)
        hdqt.check_device_status(status, kind)
        assert np.array_equal(ws.codes_a().cpu().numpy(), want["Aq"]), kind
        assert np.array_equal(ws.codes_b().cpu().numpy(), want["Bq"]), kind
        _assert_close(out.cpu().numpy(), want["out"])


def test_persistent_ctas_mix_merged_and_clamped_blocks(hdqt):
    """More output blocks than SMs, with certified, partly certified and uncertifiable blocks interleaved, so
    that one persistent CTA walks through blocks of different kinds (accumulator hand-over state carries over)."""
    rng = np.random.default_rng(77)
    M, N, K = 128 * 21, 256 * 9 + 40, 1024            # 22 x 10 = 220 blocks (incl. ragged edges) on 148 SMs
    Aq = _sparse_codes(rng, M, K, 0.03)
    Bq = _sparse_codes(rng, N, K, 0.03)
    for rb in range(0, M // 128, 3):                   # every third row block: dense codes -> nothing certifies
        Aq[rb * 128:(rb + 1) * 128] = rng.integers(-8, 8, size=(128, K))
    for rb in range(1, M // 128, 3):                   # next: one dense stripe of K tiles -> a few clamp tiles
        Aq[rb * 128:(rb + 1) * 128, 96:160] = rng.integers(-8, 8, size=(128, 64))
    Bq[:, 96:160] = rng.integers(-8, 8, size=(N, 64))
    want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 0.25, 0.5)
    na, nb = _dev(_tile_norms(Aq)), _dev(_tile_norms(Bq))
    qa, qb = torch.tensor([0.25], device="cuda"), torch.tensor([0.5], device="cuda")
    status = hdqt.new_status("cuda")
    for flags in (0, hdqt.FLAG_NO_MERGE):
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), qa, qb, want_S=True, norms_a=na, norms_b=nb, flags=flags,
                                       dev_status=status)
        hdqt.check_device_status(status)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), flags
        assert np.array_equal(out.cpu().numpy(), want_out), flags


@pytest.mark.parametrize("acc_bits,acc_tile", [(8, 32), (8, 64), (6, 32)])
def test_work_split_pure_fixup_and_general_blocks(hdqt, acc_bits, acc_tile):
    """Large enough for the work split (>= 8 blocks per SM): pair blocks that are fully certified, that have a
    few uncertified tiles (fix-up pass) and that have many (general kernel), with ragged edges."""
    rng = np.random.default_rng(88)
    M, N, K = 128 * 37 + 50, 256 * 33 + 24, 2048            # 38 x 34 = 1292 single blocks >= 8 x 148
    Aq = (rng.integers(-1, 2, size=(M, K)) * (rng.random((M, K)) < 0.05)).astype(np.int8)   # tiny norms: certifiable
    Bq = (rng.integers(-1, 2, size=(N, K)) * (rng.random((N, K)) < 0.05)).astype(np.int8)
    for rb in range(0, M // 128, 5):                         # dense row blocks: nothing certifies there
        Aq[rb * 128:(rb + 1) * 128] = rng.integers(-8, 8, size=(128, K))
    Bq[:, ::3] = np.where(Bq[:, ::3] == 0, 3, Bq[:, ::3])    # enough weight in B for the dense A blocks to fail
    for rb in range(2, M // 128, 5):                         # one dense 32-wide K tile: a single uncertified tile
        Aq[rb * 128:(rb + 1) * 128, 320:352] = rng.integers(-8, 8, size=(128, 32))
    Bq[:, 320:352] = rng.integers(-8, 8, size=(N, 32))
    Bq[:, 1024:1056] = rng.integers(6, 8, size=(N, 32))      # large codes: these tiles really clamp
    Aq[2 * 128:3 * 128, 1024:1056] = rng.integers(6, 8, size=(128, 32))
    # the oracle on sampled rows (all columns) and sampled columns (all rows) keeps this test affordable
    rows = np.sort(rng.choice(M, 96, replace=False))
    cols = np.sort(rng.choice(N, 96, replace=False))
    rows[:4] = [0, 2 * 128 + 5, M - 1, 128 * 5 + 7]          # incl. the really clamping block and the ragged edge
    want_r, want_Sr, _ = O.gemm_i8_tiled(Aq[rows], Bq, 0.25, 0.5, acc_bits, acc_tile)
    want_c, want_Sc, _ = O.gemm_i8_tiled(Aq, Bq[cols], 0.25, 0.5, acc_bits, acc_tile)
    na, nb = _dev(_tile_norms(Aq)), _dev(_tile_norms(Bq))
    qa, qb = torch.tensor([0.25], device="cuda"), torch.tensor([0.5], device="cuda")
    status = hdqt.new_status("cuda")
    out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), qa, qb, acc_bits, acc_tile, want_S=True, norms_a=na,
                                   norms_b=nb, dev_status=status)
    hdqt.check_device_status(status)
    Sn, outn = S.cpu().numpy().astype(np.int64), out.cpu().numpy()
    assert np.array_equal(Sn[rows], want_Sr) and np.array_equal(Sn[:, cols], want_Sc)
    assert np.array_equal(outn[rows], want_r) and np.array_equal(outn[:, cols], want_c)
    # the unsplit kernel (merging off) must give the same matrix everywhere
    out2, S2, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), qa, qb, acc_bits, acc_tile, want_S=True, norms_a=na,
                                     norms_b=nb, flags=hdqt.FLAG_NO_MERGE, dev_status=status)
    hdqt.check_device_status(status)
    assert torch.equal(S2, S) and torch.equal(out2, out)
    if (acc_bits, acc_tile) != (8, 32):
        return
    # the classes really occur: a fully certified pair block, one with a few uncertified tiles, one with many
    na64, nb64 = _tile_norms(Aq).astype(np.int64), _tile_norms(Bq).astype(np.int64)
    def uncert(tm, tn):
        a = na64[2 * tm:2 * tm + 2].max(0)
        b = nb64[2 * tn:2 * tn + 2].max(0)
        return int((a * b > 127 * 127).sum())
    counts = sorted({min(uncert(tm, 0), 3) for tm in range(M // 256)})
    assert counts[0] == 0 and 1 in counts + [2] and counts[-1] == 3
    # wide accumulators: every block goes to the pair kernel without certificates
    out16, S16, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), qa, qb, acc_bits=16, want_S=True, dev_status=status)
    hdqt.check_device_status(status)
    plain = np.rint(Aq.astype(np.float64) @ Bq.astype(np.float64).T).astype(np.int64)     # exact: small integers in fp64
    assert np.array_equal(S16.cpu().numpy().astype(np.int64), plain)


def test_work_split_ragged_shapes_and_unaligned_output(hdqt):
    """Split path with a single, half-empty row of pair blocks, a ragged last column block, a K that ends inside
    a shared-memory stage, and an output whose leading dimension rules out vector stores."""
    rng = np.random.default_rng(99)
    M, N, K = 200, 256 * 1200 + 8, 96                        # 2 x 1201 single blocks >= 8 x 148
    Aq = (rng.integers(-1, 2, size=(M, K)) * (rng.random((M, K)) < 0.2)).astype(np.int8)
    Bq = (rng.integers(-1, 2, size=(N, K)) * (rng.random((N, K)) < 0.2)).astype(np.int8)
    Bq[256 * 7:256 * 9, 32:64] = rng.integers(6, 8, size=(512, 32))      # a few blocks with one clamping tile
    Aq[:, 32:64] = rng.integers(5, 8, size=(M, 32))
    Bq[256 * 40:256 * 41] = rng.integers(-8, 8, size=(256, K))          # one block where nothing certifies
    Aq[:, 64:96] = np.where(Aq[:, 64:96] == 0, 2, Aq[:, 64:96])
    want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 0.5, 0.5)
    na, nb = _dev(_tile_norms(Aq)), _dev(_tile_norms(Bq))
    half = torch.tensor([0.5], device="cuda")
    status = hdqt.new_status("cuda")
    big = torch.full((M, N + 3), -7.0, device="cuda")
    for view in (None, big[:, 1:N + 1]):
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), half, half, want_S=True, norms_a=na, norms_b=nb,
                                       dev_status=status, out=view)
        hdqt.check_device_status(status)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S)
        assert np.array_equal(out.cpu().numpy(), want_out)
    assert (big[:, 0] == -7.0).all().item() and (big[:, N + 1:] == -7.0).all().item()


@pytest.mark.parametrize("in_bits,acc_bits", [(7, 8), (8, 8), (7, 16), (8, 16)])
def test_merging_with_wide_codes_uses_exact_tile_norms(hdqt, in_bits, acc_bits):
    """7/8-bit codes: a tile's sum(code^2) exceeds 16 bits, so a truncated norm would certify tiles that clamp.
    Composite call with merging on (enough output blocks for the norms to be produced) against the oracle."""
    Nb, D, C = 128 * 8 + 40, 256 * 4 + 24, 192            # dgrad: M = Nb, N = D: 9 x 5 = 45 output blocks
    G = inputs.gradients(Nb, C, seed=in_bits)
    G[5, :] *= 40.0                                       # one loud row: most other codes are small, some tiles certify
    W = inputs.weights(D, C, seed=acc_bits)
    over = dict(in_bits=in_bits, acc_bits=acc_bits, clip_a=0.25, clip_b=0.25, seed=3)
    want = O.gemm_dgrad(G, W, O.dgrad_desc(tag_a=2, tag_b=3, **over))
    status = hdqt.new_status("cuda")
    out, ws = hdqt.gemm_dgrad(_dev(G), _dev(W), desc=hdqt.default_desc("dgrad", **over), dev_status=status)
    hdqt.check_device_status(status)
    assert np.array_equal(ws.codes_a().cpu().numpy(), want["Aq"])
    assert np.array_equal(ws.codes_b().cpu().numpy(), want["Bq"])
    assert np.array_equal(out.cpu().numpy(), want["out"])


def test_packed_epilogue_limit_with_two_bit_codes(hdqt):
    """code_bits = 2, acc_tile = 8160: a tile sum reaches 32640, and 32640 + 128 no longer fits the signed
    16-bit lanes of the packed epilogue, so the 32-bit epilogue must be chosen."""
    K = 8160
    A = np.full((40, K), -2, np.int8)
    B = np.full((24, K), -2, np.int8)
    one = torch.ones(1, device="cuda")
    _, S, _ = hdqt.gemm_i8_tiled(_dev(A), _dev(B), one, one, 8, 8160, 0, 32, code_bits=2, want_S=True)
    assert (S == 127).all().item()                        # +32640 saturates at +127
    _, S, _ = hdqt.gemm_i8_tiled(_dev(A), _dev(-B), one, one, 8, 8160, 0, 32, code_bits=2, want_S=True)
    assert (S == -128).all().item()


def test_clamp_path_rare_and_frequent_saturation(hdqt):
    """The 16-bit-lane epilogue adds a register batch unclamped when an OR-reduction proves it in range and
    clamps it otherwise: operands where no tile, a few tiles, and most tiles leave the 8-bit range, merging off."""
    rng = np.random.default_rng(123)
    M, N, K = 260, 520, 32 * 40
    one = torch.ones(1, device="cuda")
    for scale_a, scale_b in ((1.0, 1.0), (2.2, 2.2), (8.0, 8.0)):
        Aq = np.clip(np.rint(rng.standard_normal((M, K)) * scale_a), -8, 7).astype(np.int8)
        Bq = np.clip(np.rint(rng.standard_normal((N, K)) * scale_b), -8, 7).astype(np.int8)
        want_out, want_S, want_tiles = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, want_tiles=True)
        clamped = float(np.mean((want_tiles == 127) | (want_tiles == -128)))
        _, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, want_S=True, flags=hdqt.FLAG_NO_MERGE)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), (scale_a, clamped)
    assert clamped > 0.2                                   # the last case really saturates often
    for acc_bits in (6, 4, 2):                             # narrower accumulators through the same epilogue
        want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, acc_bits)
        _, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, acc_bits, want_S=True, flags=hdqt.FLAG_NO_MERGE)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), acc_bits


def test_bounded_waits_run_out_and_report_timeout(hdqt):
    """A wait on a barrier nothing arrives at gives up, the block ends normally and the status word holds
    HDQT_ERR_TIMEOUT; the status word is a sticky maximum; the context stays usable."""
    status = hdqt.new_status("cuda")
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert hdqt.lib.hdqt_selftest_bounded_wait(status.data_ptr(), gave_up.data_ptr(), stream) == 0
    torch.cuda.synchronize()
    assert status.item() == 6 and hdqt.STATUS_NAMES[6] == "TIMEOUT"
    assert gave_up.item() == 33                            # the spinning thread and the 32 suspending ones
    with pytest.raises(hdqt.HdqtError) as err:
        hdqt.check_device_status(status, "selftest")
    assert err.value.status == 6
    # sticky maximum: a smaller code (non-finite operand = 5) does not overwrite it, a larger one would
    z = torch.full((4, 32), float("nan"), device="cuda")
    hdqt.quantize_hadamard(z, dev_status=status)
    assert status.item() == 6
    status.zero_()
    hdqt.quantize_hadamard(z, dev_status=status)
    assert status.item() == 5
    # the device is still fine: a real GEMM afterwards gives the right answer
    A = np.full((8, 32), 1, np.int8)
    one = torch.ones(1, device="cuda")
    _, S, _ = hdqt.gemm_i8_tiled(_dev(A), _dev(A), one, one, want_S=True)
    assert (S == 32).all().item()


@pytest.mark.parametrize("Nb,D,C,heavy", [(64, 96, 40, False), (300, 561, 130, False), (128 * 37 + 50, 1024, 256 * 33 + 24, True),
                                          (70, 32 * 300, 50, False), (200, 160, 144, False), (700, 4608, 512, False)])
def test_fused_bias_and_relu(hdqt, Nb, D, C, heavy):
    """Forward product with the bias and ReLU folded into the dequantising epilogue: small blocks, the work split of
    large problems (pair kernel, fix-up pass, general kernel) and split-K all apply the same fp32 tail."""
    if heavy:
        X, W = inputs.heavy_tailed(Nb, D, seed=5), inputs.heavy_tailed(D, C, seed=6)
    else:
        X, W = inputs.activations(Nb, D, seed=Nb), inputs.weights(D, C, seed=C)
    bias = inputs.activations(1, C, seed=7)[0] * np.float32(np.abs(X).mean() * np.abs(W).mean() * 4)
    want = O.gemm_fwd(X, W, O.fwd_desc(tag_a=0, tag_b=1, bias=bias, relu=True))
    status = hdqt.new_status("cuda")
    bd = _dev(bias)
    desc = hdqt.default_desc("fwd", bias=bd, flags=hdqt.FLAG_RELU)
    out, ws = hdqt.gemm_fwd(_dev(X), _dev(W), desc=desc, dev_status=status)
    hdqt.check_device_status(status)
    assert np.array_equal(ws.codes_a().cpu().numpy(), want["Aq"])
    got = out.cpu().numpy()
    assert np.array_equal(got, want["out"])
    assert (got == 0).mean() > 0.05 and (got > 0).mean() > 0.05      # the ReLU really cuts, the bias really shifts
    # bias only
    want_b = O.gemm_fwd(X, W, O.fwd_desc(tag_a=0, tag_b=1, bias=bias))
    out_b, _ = hdqt.gemm_fwd(_dev(X), _dev(W), desc=hdqt.default_desc("fwd", bias=bd), dev_status=status)
    assert np.array_equal(out_b.cpu().numpy(), want_b["out"])


def test_mma_rate_yardstick_runs_and_is_plausible(hdqt):
    """The MMA-only loop finishes within its bounded wait and reports a rate of the order of the chip's dense
    int8 figure (a few POP/s)."""
    status = hdqt.new_status("cuda")
    rate = hdqt.mma_rate_tops(iters=4000, repeats=2, dev_status=status)
    hdqt.check_device_status(status)
    assert 1000.0 < rate < 6000.0
    assert hdqt.lib.hdqt_selftest_mma_rate(0, None, None, None) == 1      # invalid argument, nothing launched


@pytest.mark.parametrize("kind,shape", [("dgrad", (70, 96, 200)), ("wgrad", (64, 300, 40)), ("wgrad", (2048, 160, 4100))])
def test_device_side_philox_offset(hdqt, kind, shape):
    """The descriptor's device word is the fourth Philox counter word of every stochastic rounding of the call:
    both operand layouts (and the tile-norm variant of the large weight-gradient case) agree with the oracle's
    `philox_offset`, the word is read when the kernels run (not when the call is made), and offset 0 is the
    plain stream."""
    Nb, D, Cc = shape
    X, W, G = inputs.activations(Nb, D, seed=1), inputs.weights(D, Cc, seed=2), inputs.gradients(Nb, Cc, seed=3)
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = hdqt.new_status("cuda")
    codes = {}
    for off in (0, 7, 0x80000001):
        word.fill_(off - (1 << 32) if off >= (1 << 31) else off)
        d = hdqt.default_desc(kind, seed=5, philox_offset=word)
        if kind == "dgrad":
            out, ws = hdqt.gemm_dgrad(_dev(G), _dev(W), desc=d, dev_status=status)
            want = O.gemm_dgrad(G, W, O.dgrad_desc(seed=5, tag_a=2, tag_b=3, philox_offset=off))
        else:
            out, ws = hdqt.gemm_wgrad(_dev(X), _dev(G), desc=d, dev_status=status)
            want = O.gemm_wgrad(X, G, O.wgrad_desc(seed=5, tag_a=4, tag_b=5, philox_offset=off))
        hdqt.check_device_status(status)
        assert np.array_equal(ws.codes_a().cpu().numpy(), want["Aq"])
        assert np.array_equal(ws.codes_b().cpu().numpy(), want["Bq"])
        assert np.array_equal(out.cpu().numpy(), want["out"])
        codes[off] = ws.codes_a().cpu().numpy().copy()
    assert not np.array_equal(codes[0], codes[7])
    # stream-ordered: the word is changed after the call was enqueued behind a change, not at call time
    word.fill_(7)
    d = hdqt.default_desc(kind, seed=5, philox_offset=word)
    if kind == "dgrad":
        _, ws = hdqt.gemm_dgrad(_dev(G), _dev(W), desc=d, dev_status=status)
    else:
        _, ws = hdqt.gemm_wgrad(_dev(X), _dev(G), desc=d, dev_status=status)
    got = ws.codes_a().clone()
    word.fill_(0)
    assert np.array_equal(got.cpu().numpy(), codes[7])


@pytest.mark.parametrize("K,acc_bits", [(32 * 260, 8), (32 * 700, 8), (32 * 1100, 5)])
def test_long_contraction_keeps_lane_sums_in_registers(hdqt, K, acc_bits):
    """More clamp-path tiles per output block than the 16-bit lane sums hold (256 at b_a = 8): the variant with
    a second set of lanes (low byte / high bytes) must give the same integers as the oracle, for operands that
    never clamp, that clamp often (sums of a lane run close to the lane limit) and for all-saturated tiles,
    with split-K switched off so that a work item really spans the whole contraction."""
    rng = np.random.default_rng(K)
    M, N = 200, 300
    one = torch.ones(1, device="cuda")
    flags = hdqt.FLAG_NO_MERGE | hdqt.FLAG_NO_SPLIT_K
    status = hdqt.new_status("cuda")
    for kind in ("calm", "wild", "saturated"):
        if kind == "calm":
            Aq = np.clip(np.rint(rng.standard_normal((M, K)) * 1.2), -8, 7).astype(np.int8)
            Bq = np.clip(np.rint(rng.standard_normal((N, K)) * 1.2), -8, 7).astype(np.int8)
        elif kind == "wild":
            Aq, Bq = _codes(rng, M, K), _codes(rng, N, K)
        else:
            Aq, Bq = np.full((M, K), 7, np.int8), np.full((N, K), 7, np.int8)     # every tile sum clamps to the top
            Bq[::2] = -8                                                          # ... or to the bottom
        want_out, want_S, _ = O.gemm_i8_tiled(Aq, Bq, 1.0, 1.0, acc_bits)
        out, S, _ = hdqt.gemm_i8_tiled(_dev(Aq), _dev(Bq), one, one, acc_bits, want_S=True, flags=flags,
                                       dev_status=status)
        hdqt.check_device_status(status)
        assert np.array_equal(S.cpu().numpy().astype(np.int64), want_S), kind
        assert np.array_equal(out.cpu().numpy(), want_out), kind
    if acc_bits == 8:
        assert int(np.abs(want_S).max()) == 128 * (K // 32)       # the saturated case reaches the largest sum there is
