"""GPU parity: FWHT + calibration maximum + quantizer against the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import hdqt_oracle as O
from paper_2310_03675_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hdqt():
    from paper_2310_03675_b200 import hdqt as mod
    return mod


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def _expected_norms(codes):
    rows, Kp = codes.shape
    sq = (codes.astype(np.int64) ** 2).reshape(rows, Kp // 32, 32).sum(2)
    nb = (rows + 127) // 128
    out = np.zeros((nb, Kp // 32), dtype=np.int64)
    for b in range(nb):
        out[b] = sq[b * 128:(b + 1) * 128].max(0)
    return out


SHAPES = [(32, 128), (32, 64), (1, 32), (7, 27), (129, 100), (300, 561), (256, 1152), (1000, 96), (5, 8)]


@pytest.mark.parametrize("rows,K", SHAPES)
@pytest.mark.parametrize("layout", ["k_contiguous", "k_strided"])
@pytest.mark.parametrize("mode", [0, 1])
def test_quantize_matches_oracle(hdqt, rows, K, layout, mode):
    x = inputs.gradients(rows, K, seed=rows * 1000 + K, scale=1.0)
    want_codes, want_step, want_amax = O.quantize_hadamard(x, 32, 4, 1.0, mode, seed=5, tag=9)
    if layout == "k_contiguous":
        src = _dev(x)
    else:
        src = _dev(x.T).t()            # same logical [rows, K], rows contiguous in memory
    status = hdqt.new_status("cuda")
    amax = hdqt.absmax_hadamard(src, 32, status)
    codes, step, norms = hdqt.quantize_hadamard(src, 32, 4, 1.0, mode, seed=5, tag=9, want_norms=True,
                                                dev_status=status)
    hdqt.check_device_status(status)
    assert amax.item() == float(want_amax)
    assert step.item() == float(want_step)
    got = codes.cpu().numpy()
    assert got.shape == want_codes.shape
    assert np.array_equal(got, want_codes)
    assert np.array_equal(norms.cpu().numpy().astype(np.int64), _expected_norms(want_codes))


@pytest.mark.parametrize("bits,clip,had", [(2, 1.0, 32), (3, 0.975, 32), (5, 1.0, 16), (6, 0.5, 8), (8, 0.975, 32),
                                           (8, 0.25, 4), (4, 0.975, 1), (4, 1.0, 2)])
@pytest.mark.parametrize("mode", [0, 1])
def test_bit_widths_clip_and_block_sizes(hdqt, bits, clip, had, mode):
    x = inputs.activations(70, 200, seed=bits * 10 + had)
    want_codes, want_step, _ = O.quantize_hadamard(x, had, bits, clip, mode, seed=77, tag=3)
    for src in (_dev(x), _dev(x.T).t()):
        codes, step, _ = hdqt.quantize_hadamard(src, had, bits, clip, mode, seed=77, tag=3)
        assert step.item() == float(want_step)
        assert np.array_equal(codes.cpu().numpy(), want_codes)


def test_unaligned_row_stride_and_views(hdqt):
    base = inputs.activations(64, 203, seed=1)
    x = base[:, 3:130]                       # K = 127, row stride 203 (not a multiple of 4), offset pointer
    want, step_w, _ = O.quantize_hadamard(x, 32, 4, 1.0, 1, seed=1, tag=1)
    src = _dev(base)[:, 3:130]
    codes, step, _ = hdqt.quantize_hadamard(src, 32, 4, 1.0, 1, seed=1, tag=1)
    assert step.item() == float(step_w)
    assert np.array_equal(codes.cpu().numpy(), want)


def test_supplied_amax_skips_calibration(hdqt):
    x = inputs.activations(40, 96, seed=2)
    amax = np.float32(123.5)
    xh = O.fwht_blockdiag(O.pad_contraction(x, 32), 32)
    want, want_step, _ = O.quantize_transformed(xh, 4, 0.975, 0, amax=amax)
    codes, step, _ = hdqt.quantize_hadamard(_dev(x), 32, 4, 0.975, 0, amax=torch.tensor([amax], device="cuda"))
    assert step.item() == float(want_step)
    assert np.array_equal(codes.cpu().numpy(), want)


def test_seed_high_word_and_determinism(hdqt):
    x = _dev(inputs.gradients(64, 64, seed=3))
    a, _, _ = hdqt.quantize_hadamard(x, mode=1, seed=(5 << 32) + 1, tag=2)
    b, _, _ = hdqt.quantize_hadamard(x, mode=1, seed=(5 << 32) + 1, tag=2)
    c, _, _ = hdqt.quantize_hadamard(x, mode=1, seed=1, tag=2)
    assert torch.equal(a, b) and not torch.equal(a, c)
    want, _, _ = O.quantize_hadamard(x.cpu().numpy(), 32, 4, 1.0, 1, seed=(5 << 32) + 1, tag=2)
    assert np.array_equal(a.cpu().numpy(), want)


def test_all_zero_and_nonfinite(hdqt):
    status = hdqt.new_status("cuda")
    z = torch.zeros(16, 64, device="cuda")
    codes, step, _ = hdqt.quantize_hadamard(z, dev_status=status)
    assert not codes.any().item() and step.item() == 0.0 and status.item() == 0
    z[3, 5] = float("inf")
    for src in (z, z.t().contiguous().t()):
        for mode in (0, 1):
            status.zero_()
            codes, step, _ = hdqt.quantize_hadamard(src, mode=mode, dev_status=status)
            assert status.item() == 5      # HDQT_ERR_NONFINITE, reported through the device status word
            # a contaminated operand yields all-zero codes and a zero scale, never saturated garbage
            assert not codes.any().item() and step.item() == 0.0
    status.zero_()
    z[3, 5] = float("nan")
    hdqt.absmax_hadamard(z.t().contiguous().t(), dev_status=status)
    assert status.item() == 5


def test_output_canaries(hdqt):
    """Nothing is written outside [rows, K_pad]."""
    rows, K = 37, 70
    Kp = hdqt.padded_k(K)
    buf = torch.full((rows * Kp + 512,), 0x5A, dtype=torch.int8, device="cuda")
    codes = buf[256:256 + rows * Kp].view(rows, Kp)
    step = torch.empty(1, device="cuda")
    ws = torch.empty(hdqt.lib.hdqt_quantize_workspace_bytes(rows, K, 32), dtype=torch.uint8, device="cuda")
    x = _dev(inputs.activations(rows, K, seed=4))
    for src in (x, x.t().contiguous().t()):
        hdqt.quantize_hadamard(src, mode=1, out=(codes, step, None, ws))
        torch.cuda.synchronize()
        assert (buf[:256] == 0x5A).all().item() and (buf[256 + rows * Kp:] == 0x5A).all().item()


def test_large_tensor_multiple_waves(hdqt):
    """Larger than one grid wave, ragged tail; codes compared in full."""
    rows, K = 3001, 2080
    x = inputs.heavy_tailed(rows, K, seed=8)
    for mode in (0, 1):
        want, step_w, _ = O.quantize_hadamard(x, 32, 4, 1.0, mode, seed=2, tag=4)
        for src in (_dev(x), _dev(x.T).t()):
            codes, step, _ = hdqt.quantize_hadamard(src, mode=mode, seed=2, tag=4)
            assert step.item() == float(step_w)
            assert np.array_equal(codes.cpu().numpy(), want)


@pytest.mark.parametrize("bits,clip", [(8, 0.25), (8, 1.0), (7, 0.05), (4, 1.0 / 64)])
def test_tile_norms_of_wide_and_saturated_codes(hdqt, bits, clip):
    """Tile norms of 7/8-bit codes reach 32 * 128^2 (far beyond 16 bits); a small clip saturates most codes.
    Both layouts, several 128-row blocks, a ragged last block and K segments of every width."""
    for rows, K in ((300, 561), (130, 8192), (257, 96)):
        x = inputs.activations(rows, K, seed=bits + rows)
        want_codes, _, _ = O.quantize_hadamard(x, 32, bits, clip, 0)
        for src in (_dev(x), _dev(x.T).t()):
            codes, _, norms = hdqt.quantize_hadamard(src, 32, bits, clip, 0, want_norms=True)
            assert np.array_equal(codes.cpu().numpy(), want_codes)
            assert np.array_equal(norms.cpu().numpy().astype(np.int64), _expected_norms(want_codes))


@pytest.mark.parametrize("kind", ["dgrad", "wgrad", "fwd"])
def test_delayed_scaling_uses_the_previous_tensors_maximum(hdqt, kind):
    """Step 1 measures its maxima and leaves their partial maxima behind; step 2 quantizes DIFFERENT tensors with
    step 1's maxima (no calibration pass) and leaves its own.  Codes, scales and outputs against the oracle run with
    the same maxima; the history always holds exactly the maximum of the tensor just transformed."""
    Nb, D, C = 300, 160, 200
    X1, W1, G1 = inputs.single_layer(3, Nb=Nb, D=D, C=C)
    X2, W2, G2 = inputs.single_layer(4, Nb=Nb, D=D, C=C)
    X2, G2 = X2 * np.float32(1.7), G2 * np.float32(0.4)       # one operand grows (saturates), one shrinks
    make = {"dgrad": (hdqt.gemm_dgrad, O.dgrad_desc, lambda X, W, G: (G, W), lambda X, W, G: (G, W)),
            "wgrad": (hdqt.gemm_wgrad, O.wgrad_desc, lambda X, W, G: (X, G), lambda X, W, G: (X.T, G.T)),
            "fwd": (hdqt.gemm_fwd, O.fwd_desc, lambda X, W, G: (X, W), lambda X, W, G: (X, W.T))}[kind]
    call, odesc, pick, views = make
    d0 = hdqt.default_desc(kind)
    od = odesc(tag_a=d0.tag_a, tag_b=d0.tag_b, seed=3)
    hist = [[torch.full((hdqt.AMAX_HISTORY_WORDS,), 0xFFFFFFFF, dtype=torch.int64, device="cuda").to(torch.int32)
             for _ in range(2)] for _ in range(2)]          # [step parity][operand], pre-filled with garbage
    status = hdqt.new_status("cuda")

    def amax_h(v):
        return np.float32(np.abs(O.fwht_blockdiag(O.pad_contraction(np.ascontiguousarray(v), 32), 32)).max())

    def hist_max(t):
        return float(t.view(torch.float32).max().item())

    # step 1: measured maxima, history written
    a1, b1 = pick(X1, W1, G1)
    desc = hdqt.default_desc(kind, seed=3, amax_hist_out_a=hist[0][0], amax_hist_out_b=hist[0][1])
    out1, ws = call(_dev(a1), _dev(b1), desc=desc, dev_status=status)
    hdqt.check_device_status(status)
    va, vb = views(X1, W1, G1)
    want1 = O.hdqt_gemm(np.ascontiguousarray(va), np.ascontiguousarray(vb), od)
    assert np.array_equal(out1.cpu().numpy(), want1["out"])
    assert hist_max(hist[0][0]) == float(amax_h(va)) and hist_max(hist[0][1]) == float(amax_h(vb))
    assert (hist[0][0] >= 0).all().item()                     # every entry defined: no garbage left (sign bit clear)
    # step 2: other tensors, step 1's maxima, new history
    a2, b2 = pick(X2, W2, G2)
    desc = hdqt.default_desc(kind, seed=3, amax_hist_in_a=hist[0][0], amax_hist_in_b=hist[0][1],
                             amax_hist_out_a=hist[1][0], amax_hist_out_b=hist[1][1])
    out2, ws = call(_dev(a2), _dev(b2), desc=desc, dev_status=status)
    hdqt.check_device_status(status)
    va2, vb2 = views(X2, W2, G2)
    Aq, sa, _ = O.quantize_hadamard(np.ascontiguousarray(va2), 32, 4, od.clip_a, od.round_a, 3, od.tag_a, amax=amax_h(va))
    Bq, sb, _ = O.quantize_hadamard(np.ascontiguousarray(vb2), 32, 4, od.clip_b, od.round_b, 3, od.tag_b, amax=amax_h(vb))
    assert np.array_equal(ws.codes_a().cpu().numpy(), Aq) and np.array_equal(ws.codes_b().cpu().numpy(), Bq)
    assert ws.scalar("step_a").item() == float(sa) and ws.scalar("step_b").item() == float(sb)
    want2, _, _ = O.gemm_i8_tiled(Aq, Bq, sa, sb)
    assert np.array_equal(out2.cpu().numpy(), want2)
    assert hist_max(hist[1][0]) == float(amax_h(va2)) and hist_max(hist[1][1]) == float(amax_h(vb2))
    fresh, _, _ = O.quantize_hadamard(np.ascontiguousarray(va2), 32, 4, od.clip_a, od.round_a, 3, od.tag_a)
    assert not np.array_equal(fresh, Aq)                       # the carried scale really differs from a fresh one
