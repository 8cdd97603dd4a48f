"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and rejects bad arguments on the host before touching a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hdqt():
    from paper_2310_03675_b200 import hdqt as mod
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hdqt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hdqt_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(hdqt):
    names = declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(hdqt.lib, n), n
    assert sorted(hdqt.EXPORTED) == names


def test_status_strings(hdqt):
    seen = set()
    for code in range(9):
        s = hdqt.lib.hdqt_status_string(code).decode()
        assert s and s not in seen
        seen.add(s)
    assert hdqt.lib.hdqt_status_string(0).decode() == "ok"


def test_padded_k(hdqt):
    assert hdqt.padded_k(128) == 128
    assert hdqt.padded_k(27) == 32
    assert hdqt.padded_k(12, 1) == 32
    assert hdqt.padded_k(561) == 576
    assert hdqt.padded_k(1) == 32


def test_default_descs_follow_the_paper(hdqt):
    f, d, w = (hdqt.default_desc(k) for k in ("fwd", "dgrad", "wgrad"))
    for x in (f, d, w):
        assert (x.in_bits, x.acc_bits, x.acc_tile, x.had_block, x.acc_shift) == (4, 8, 32, 32, 0)
    assert abs(f.clip_a - 0.975) < 1e-7 and abs(f.clip_b - 0.975) < 1e-7
    assert (f.round_a, f.round_b) == (0, 0)          # forward: nearest
    assert (d.round_a, d.round_b) == (1, 0)          # dgrad: SR on G only
    assert (w.round_a, w.round_b) == (1, 1)          # wgrad: SR on X and G
    assert d.clip_a == 1.0 and w.clip_b == 1.0
    tags = [f.tag_a, f.tag_b, d.tag_a, d.tag_b, w.tag_a, w.tag_b]
    assert len(set(tags)) == 6


def test_workspace_layout_is_disjoint_and_aligned(hdqt):
    d = hdqt.default_desc("fwd")
    L = hdqt.workspace_layout(d, 300, 520, 561)
    assert L.k_pad == 576
    offs = [("step_a", 4), ("step_b", 4), ("amax_a", 4), ("amax_b", 4), ("codes_a", 300 * 576),
            ("codes_b", 520 * 576), ("norms_a", 3 * 18 * 4), ("norms_b", 5 * 18 * 4), ("gemm_ws", 1)]
    spans = sorted((getattr(L, n), getattr(L, n) + sz) for n, sz in offs)
    for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
        assert a1 <= b0
    assert spans[-1][1] <= L.total == hdqt.workspace_bytes(d, 300, 520, 561)
    for n in ("codes_a", "codes_b", "norms_a", "norms_b", "gemm_ws"):
        assert getattr(L, n) % 256 == 0


def test_host_side_rejections(hdqt):
    lib = hdqt.lib
    d = hdqt.default_desc("fwd")
    INVALID, UNSUPPORTED, ALIGN, WS = 1, 2, 3, 4
    # null pointers / bad sizes never reach a launch
    assert lib.hdqt_gemm_fwd(C.byref(d), None, None, None, 4, 4, 4, 0, None, 0, None, None) == INVALID
    assert lib.hdqt_gemm_dgrad(C.byref(d), 256, 256, 256, 0, 4, 4, 0, 256, 0, None, None) == INVALID
    assert lib.hdqt_gemm_wgrad(C.byref(d), 256, 256, 256, 4, 4, -1, 0, 256, 0, None, None) == INVALID
    # workspace too small / misaligned
    assert lib.hdqt_gemm_fwd(C.byref(d), 256, 256, 256, 4, 4, 4, 0, 256, 16, None, None) == WS
    assert lib.hdqt_gemm_fwd(C.byref(d), 256, 256, 256, 4, 4, 4, 0, 264, 1 << 20, None, None) == ALIGN
    # unsupported Hadamard block (valid in the paper's terms, not built)
    d64 = hdqt.default_desc("fwd", had_block=64)
    assert lib.hdqt_gemm_fwd(C.byref(d64), 256, 256, 256, 4, 64, 4, 0, 256, 1 << 20, None, None) == UNSUPPORTED
    # quantizer argument checks
    q = lib.hdqt_quantize_hadamard
    assert q(None, 4, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 32, 1, 32, 9, 1.0, 0, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 32, 1, 32, 4, 2.0, 0, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 32, 1, 32, 4, 1.0, 7, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 33, 2, 32, 4, 1.0, 0, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 32, 1, 24, 4, 1.0, 0, 0, 0, None, 256, 256, None, 256, 1 << 20, None, None) == INVALID
    assert q(256, 4, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, None, 260, 256, None, 256, 1 << 20, None, None) == ALIGN
    assert q(256, 4, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, None, 256, 256, None, 256, 8, None, None) == WS
    # integer GEMM argument checks
    g = lib.hdqt_gemm_i8_tiled
    assert g(256, 256, 256, 256, 8, 8, 48, 4, 8, 32, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == INVALID
    assert g(256, 256, 256, 256, 8, 8, 64, 4, 40, 32, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == INVALID
    assert g(256, 256, 256, 256, 8, 8, 64, 4, 8, 48, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == INVALID
    assert g(256, 256, 256, 256, 8, 8, 64, 4, 8, 32, 0, 32, 256, 4, None, None, 0, None, None, 0, 256, 4096, None, None) == INVALID
    assert g(264, 256, 256, 256, 8, 8, 64, 4, 8, 32, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == ALIGN
    # per-tile debug output in int8 cannot hold 12-bit accumulators
    assert g(256, 256, 256, 256, 8, 8, 64, 4, 12, 32, 0, 32, 256, 8, None, 256, 1, None, None, 0, 256, 4096, None, None) == INVALID
    # code_bits outside 2..8
    assert g(256, 256, 256, 256, 8, 8, 64, 9, 8, 32, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == INVALID
    # a wide sum that could overflow int32 is refused
    assert g(256, 256, 256, 256, 8, 8, 1 << 22, 8, 32, 0, 0, 32, 256, 8, None, None, 0, None, None, 0, 256, 4096, None, None) == UNSUPPORTED
