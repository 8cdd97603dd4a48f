"""ctypes binding over the HDQT C-ABI library (include/hdqt.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch supplies device memory and the current stream.  There is no
CPU fallback: if the library cannot be loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

ROUND_NEAREST = 0
ROUND_STOCHASTIC = 1
FLAG_NO_MERGE = 1
FLAG_NO_SPLIT_K = 2
FLAG_RELU = 4
AMAX_HISTORY_WORDS = 1024

STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "ALIGNMENT", "WORKSPACE", "NONFINITE", "TIMEOUT", "CUDA",
                "STATIC_SCRATCH"]

EXPORTED = [
    "hdqt_default_desc", "hdqt_padded_k", "hdqt_status_string", "hdqt_absmax_hadamard",
    "hdqt_quantize_hadamard", "hdqt_quantize_workspace_bytes", "hdqt_gemm_i8_tiled",
    "hdqt_gemm_i8_workspace_bytes", "hdqt_calibrate_acc_shift", "hdqt_gemm_fwd", "hdqt_gemm_dgrad",
    "hdqt_gemm_wgrad", "hdqt_workspace_bytes", "hdqt_workspace_layout", "hdqt_quantize_hadamard_static",
    "hdqt_selftest_bounded_wait", "hdqt_conv2d_fwd", "hdqt_conv2d_wgrad", "hdqt_selftest_mma_rate",
]


class GemmDesc(C.Structure):
    """Mirror of hdqt_gemm_desc_t."""
    _fields_ = [
        ("in_bits", C.c_int32), ("acc_bits", C.c_int32), ("acc_tile", C.c_int32), ("acc_shift", C.c_int32),
        ("had_block", C.c_int32), ("clip_a", C.c_float), ("clip_b", C.c_float),
        ("round_a", C.c_int32), ("round_b", C.c_int32), ("seed", C.c_uint64),
        ("tag_a", C.c_uint32), ("tag_b", C.c_uint32), ("amax_a", C.c_void_p), ("amax_b", C.c_void_p),
        ("flags", C.c_uint32), ("bias", C.c_void_p),
        ("amax_hist_in_a", C.c_void_p), ("amax_hist_in_b", C.c_void_p),
        ("amax_hist_out_a", C.c_void_p), ("amax_hist_out_b", C.c_void_p),
        ("philox_offset", C.c_void_p),
    ]


class Conv2dGeom(C.Structure):
    """Mirror of hdqt_conv2d_geom_t."""
    _fields_ = [("batch", C.c_int64), ("height", C.c_int64), ("width", C.c_int64), ("channels", C.c_int64),
                ("kernel_h", C.c_int32), ("kernel_w", C.c_int32), ("stride", C.c_int32), ("padding", C.c_int32)]


class WsLayout(C.Structure):
    """Mirror of hdqt_ws_layout_t."""
    _fields_ = [(n, C.c_size_t) for n in ("codes_a", "codes_b", "step_a", "step_b", "amax_a", "amax_b",
                                          "norms_a", "norms_b", "gemm_ws", "total")] + [("k_pad", C.c_int64)]


def _load() -> C.CDLL:
    path = _build.LIB_PATH
    if not os.path.exists(path) or _build.needs_rebuild():
        try:
            _build.build()
        except Exception as e:
            # No silent fallback: neither to a CPU path nor to a library older than the sources beside it.
            # A box without the CUDA toolkit may still load a library that was built elsewhere from these
            # very sources (the build stamps their digest next to it).
            if not (os.path.exists(path) and _build.stamp_matches_sources()):
                raise ImportError(f"HDQT CUDA library is missing or older than its sources and could not be "
                                  f"rebuilt: {e}") from e
    lib = C.CDLL(path)
    i32, i64, u32, u64, f32, vp, sz = C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_float, C.c_void_p, C.c_size_t
    lib.hdqt_default_desc.argtypes = [C.POINTER(GemmDesc), C.c_int]
    lib.hdqt_default_desc.restype = None
    lib.hdqt_padded_k.argtypes = [i64, i32]
    lib.hdqt_padded_k.restype = i64
    lib.hdqt_status_string.argtypes = [C.c_int]
    lib.hdqt_status_string.restype = C.c_char_p
    lib.hdqt_absmax_hadamard.argtypes = [vp, i64, i64, i64, i64, i32, vp, vp, vp]
    lib.hdqt_quantize_hadamard.argtypes = [vp, i64, i64, i64, i64, i32, i32, f32, i32, u64, u32, vp, vp, vp, vp,
                                           vp, sz, vp, vp]
    lib.hdqt_quantize_hadamard_static.argtypes = [vp, i64, i64, i64, i64, i32, i32, f32, i32, u64, u32, vp, vp, vp,
                                                  vp, vp]
    lib.hdqt_quantize_hadamard_static.restype = C.c_int
    lib.hdqt_quantize_workspace_bytes.argtypes = [i64, i64, i32]
    lib.hdqt_quantize_workspace_bytes.restype = sz
    lib.hdqt_gemm_i8_tiled.argtypes = [vp, vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, i32, vp, i64, vp, vp, i32,
                                       vp, vp, u32, vp, sz, vp, vp]
    lib.hdqt_gemm_i8_workspace_bytes.argtypes = [i64, i64, i64]
    lib.hdqt_gemm_i8_workspace_bytes.restype = sz
    lib.hdqt_calibrate_acc_shift.argtypes = [vp, vp, i64, i64, i64, i32, i32, vp, vp, sz, vp, vp]
    for name in ("hdqt_gemm_fwd", "hdqt_gemm_dgrad", "hdqt_gemm_wgrad"):
        getattr(lib, name).argtypes = [C.POINTER(GemmDesc), vp, vp, vp, i64, i64, i64, i32, vp, sz, vp, vp]
    lib.hdqt_selftest_mma_rate.argtypes = [i32, C.POINTER(C.c_int64), vp, vp]
    lib.hdqt_selftest_mma_rate.restype = C.c_int
    lib.hdqt_selftest_bounded_wait.argtypes = [vp, vp, vp]
    lib.hdqt_selftest_bounded_wait.restype = C.c_int
    for name in ("hdqt_conv2d_fwd", "hdqt_conv2d_wgrad"):
        getattr(lib, name).argtypes = [C.POINTER(GemmDesc), C.POINTER(Conv2dGeom), vp, vp, vp, i64, vp, sz, vp, vp]
        getattr(lib, name).restype = C.c_int
    lib.hdqt_workspace_bytes.argtypes = [C.POINTER(GemmDesc), i64, i64, i64]
    lib.hdqt_workspace_bytes.restype = sz
    lib.hdqt_workspace_layout.argtypes = [C.POINTER(GemmDesc), i64, i64, i64, C.POINTER(WsLayout)]
    for name in ("hdqt_absmax_hadamard", "hdqt_quantize_hadamard", "hdqt_gemm_i8_tiled", "hdqt_calibrate_acc_shift",
                 "hdqt_gemm_fwd", "hdqt_gemm_dgrad", "hdqt_gemm_wgrad", "hdqt_workspace_layout"):
        getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


class HdqtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.hdqt_status_string(status).decode()} (status {status})")


def _check(status: int, where: str) -> None:
    if status != 0:
        raise HdqtError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def new_status(device) -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def check_device_status(dev_status: torch.Tensor, where: str = "hdqt") -> None:
    """Synchronises and raises if a kernel recorded an error."""
    code = int(dev_status.item())
    if code != 0:
        raise HdqtError(code, where)


def default_desc(kind: str, **overrides) -> GemmDesc:
    d = GemmDesc()
    lib.hdqt_default_desc(C.byref(d), {"fwd": 0, "dgrad": 1, "wgrad": 2}[kind])
    for k, v in overrides.items():
        if k in ("amax_a", "amax_b", "bias", "amax_hist_in_a", "amax_hist_in_b", "amax_hist_out_a", "amax_hist_out_b",
                 "philox_offset"):
            v = _ptr(v)
        setattr(d, k, v)
    return d


def padded_k(K: int, had_block: int = 32) -> int:
    return int(lib.hdqt_padded_k(K, had_block))


def _view_2d(src: torch.Tensor):
    """(rows, K, ld_row, ld_k) of a 2-D fp32 CUDA tensor whose dim 1 is the contraction index."""
    if src.dim() != 2 or src.dtype != torch.float32 or not src.is_cuda:
        raise ValueError("expected a 2-D fp32 CUDA tensor")
    rows, K = src.shape
    ld_row, ld_k = src.stride()
    if K == 1 and ld_k != 1:
        ld_k = 1
    if rows == 1 and ld_row != 1 and ld_k != 1:
        ld_row = 1
    return rows, K, ld_row, ld_k


def absmax_hadamard(src: torch.Tensor, had_block: int = 32, dev_status: Optional[torch.Tensor] = None):
    rows, K, ld_row, ld_k = _view_2d(src)
    out = torch.empty(1, dtype=torch.float32, device=src.device)
    _check(lib.hdqt_absmax_hadamard(src.data_ptr(), rows, K, ld_row, ld_k, had_block, out.data_ptr(),
                                    _ptr(dev_status), _stream()), "hdqt_absmax_hadamard")
    return out


def quantize_hadamard(src: torch.Tensor, had_block: int = 32, bits: int = 4, clip: float = 1.0,
                      mode: int = ROUND_NEAREST, seed: int = 0, tag: int = 0,
                      amax: Optional[torch.Tensor] = None, want_norms: bool = False,
                      dev_status: Optional[torch.Tensor] = None, out=None):
    """src[rows, K] (dim 1 = contraction; either dim may be the contiguous one).
    Returns (codes int8 [rows, K_pad], step fp32 [1], tile_norms int32 or None)."""
    rows, K, ld_row, ld_k = _view_2d(src)
    Kp = padded_k(K, had_block)
    if out is None:
        codes = torch.empty((rows, Kp), dtype=torch.int8, device=src.device)
        step = torch.empty(1, dtype=torch.float32, device=src.device)
        norms = torch.empty(((rows + 127) // 128, Kp // 32), dtype=torch.int32, device=src.device) if want_norms else None
        ws = torch.empty(lib.hdqt_quantize_workspace_bytes(rows, K, had_block), dtype=torch.uint8, device=src.device)
    else:
        codes, step, norms, ws = out
    _check(lib.hdqt_quantize_hadamard(src.data_ptr(), rows, K, ld_row, ld_k, had_block, bits, clip, mode, seed, tag,
                                      _ptr(amax), codes.data_ptr(), step.data_ptr(), _ptr(norms), ws.data_ptr(),
                                      ws.numel(), _ptr(dev_status), _stream()), "hdqt_quantize_hadamard")
    return codes, step, norms


STATIC_SCRATCH_BYTES = 256 + 4096
STATIC_MAX_ROW_TILES = 2097152


def quantize_hadamard_static(src: torch.Tensor, codes: torch.Tensor, step: torch.Tensor,
                             norms: Optional[torch.Tensor] = None, had_block: int = 32, bits: int = 4,
                             clip: float = 1.0, mode: int = ROUND_NEAREST, seed: int = 0, tag: int = 0,
                             dev_status: Optional[torch.Tensor] = None):
    """Same result as quantize_hadamard (measured maximum), written into buffers the caller already
    owns, for callers that cannot allocate device memory at this point: the library's built-in
    scratch array replaces the workspace, so neither this wrapper nor the C call allocates anything.
    Operands are limited to rows * K_pad / 32 <= 2 097 152; calls on different streams must not
    overlap (they share the one array)."""
    rows, K, ld_row, ld_k = _view_2d(src)
    _check(lib.hdqt_quantize_hadamard_static(src.data_ptr(), rows, K, ld_row, ld_k, had_block, bits, clip, mode,
                                             seed, tag, codes.data_ptr(), step.data_ptr(), _ptr(norms),
                                             _ptr(dev_status), _stream()), "hdqt_quantize_hadamard_static")
    return codes, step, norms


def gemm_i8_tiled(Aq: torch.Tensor, Bq: torch.Tensor, step_a: torch.Tensor, step_b: torch.Tensor,
                  acc_bits: int = 8, acc_tile: int = 32, acc_shift: int = 0, had_block: int = 32,
                  code_bits: int = 4, want_S: bool = False, want_tiles: bool = False, norms_a=None, norms_b=None, flags: int = 0,
                  dev_status: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None):
    """Out[M,N] from codes Aq[M,K_pad], Bq[N,K_pad]. Returns (out, S or None, tiles or None)."""
    M, Kp = Aq.shape
    N, Kp2 = Bq.shape
    if Kp != Kp2 or Aq.dtype != torch.int8 or Bq.dtype != torch.int8:
        raise ValueError("code matrices must be int8 with equal K_pad")
    if not (Aq.is_contiguous() and Bq.is_contiguous()):
        raise ValueError("code matrices must be contiguous")
    dev = Aq.device
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=dev)
    S = torch.empty((M, N), dtype=torch.int32, device=dev) if want_S else None
    tiles, elem = None, 0
    if want_tiles:
        s = acc_tile if acc_tile else Kp
        T = (Kp + s - 1) // s
        elem = 1 if acc_bits <= 8 else 2
        tiles = torch.empty((T, M, N), dtype=torch.int8 if elem == 1 else torch.int16, device=dev)
    ws = torch.empty(max(256, lib.hdqt_gemm_i8_workspace_bytes(M, N, Kp)), dtype=torch.uint8, device=dev)
    _check(lib.hdqt_gemm_i8_tiled(Aq.data_ptr(), Bq.data_ptr(), step_a.data_ptr(), step_b.data_ptr(), M, N, Kp,
                                  code_bits, acc_bits, acc_tile, acc_shift, had_block, out.data_ptr(), out.stride(0),
                                  _ptr(S), _ptr(tiles), elem, _ptr(norms_a), _ptr(norms_b), flags, ws.data_ptr(),
                                  ws.numel(), _ptr(dev_status), _stream()), "hdqt_gemm_i8_tiled")
    return out, S, tiles


def calibrate_acc_shift(Aq: torch.Tensor, Bq: torch.Tensor, acc_bits: int = 8, acc_tile: int = 32) -> torch.Tensor:
    M, Kp = Aq.shape
    N = Bq.shape[0]
    out = torch.empty(1, dtype=torch.int32, device=Aq.device)
    _check(lib.hdqt_calibrate_acc_shift(Aq.data_ptr(), Bq.data_ptr(), M, N, Kp, acc_bits, acc_tile, out.data_ptr(),
                                        None, 0, None, _stream()), "hdqt_calibrate_acc_shift")
    return out


# ---- the three training GEMMs ---------------------------------------------------------------------

def workspace_layout(desc: GemmDesc, M: int, N: int, K: int) -> WsLayout:
    L = WsLayout()
    _check(lib.hdqt_workspace_layout(C.byref(desc), M, N, K, C.byref(L)), "hdqt_workspace_layout")
    return L


def workspace_bytes(desc: GemmDesc, M: int, N: int, K: int) -> int:
    return int(lib.hdqt_workspace_bytes(C.byref(desc), M, N, K))


class Workspace:
    """A device buffer plus the layout the library carves it into (to read intermediates back)."""

    def __init__(self, desc: GemmDesc, M: int, N: int, K: int, device):
        self.layout = workspace_layout(desc, M, N, K)
        self.M, self.N = M, N
        self.buf = torch.empty(self.layout.total, dtype=torch.uint8, device=device)

    def codes_a(self):
        L = self.layout
        return self.buf[L.codes_a:L.codes_a + self.M * L.k_pad].view(torch.int8).view(self.M, L.k_pad)

    def codes_b(self):
        L = self.layout
        return self.buf[L.codes_b:L.codes_b + self.N * L.k_pad].view(torch.int8).view(self.N, L.k_pad)

    def scalar(self, name: str) -> torch.Tensor:
        off = getattr(self.layout, name)
        return self.buf[off:off + 4].view(torch.float32)


def _w_dims(W: torch.Tensor, w_is_cd: bool):
    return (W.shape[1], W.shape[0]) if w_is_cd else (W.shape[0], W.shape[1])


def _run(fn_name, desc, a, b, out, Nb, D, C_, w_is_cd, M, N, K, workspace, dev_status):
    if workspace is None:
        workspace = Workspace(desc, M, N, K, a.device)
    _check(getattr(lib, fn_name)(C.byref(desc), a.data_ptr(), b.data_ptr(), out.data_ptr(), Nb, D, C_,
                                 1 if w_is_cd else 0, workspace.buf.data_ptr(), workspace.buf.numel(),
                                 _ptr(dev_status), _stream()), fn_name)
    return out, workspace


def _req(t: torch.Tensor, name: str):
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous fp32 CUDA tensor")


def gemm_fwd(X, W, desc: Optional[GemmDesc] = None, w_is_cd: bool = False, workspace=None, dev_status=None,
             out=None):
    """Y[Nb,C] = X[Nb,D] W. W is [D,C], or [C,D] when w_is_cd. Returns (Y, workspace)."""
    _req(X, "X"); _req(W, "W")
    desc = desc or default_desc("fwd")
    Nb, D = X.shape
    Dw, Cw = _w_dims(W, w_is_cd)
    if Dw != D:
        raise ValueError("shape mismatch")
    if out is None:
        out = torch.empty((Nb, Cw), dtype=torch.float32, device=X.device)
    return _run("hdqt_gemm_fwd", desc, X, W, out, Nb, D, Cw, w_is_cd, Nb, Cw, D, workspace, dev_status)


def gemm_dgrad(G, W, desc: Optional[GemmDesc] = None, w_is_cd: bool = False, workspace=None, dev_status=None,
               out=None):
    """dX[Nb,D] = G[Nb,C] W^T. Returns (dX, workspace)."""
    _req(G, "G"); _req(W, "W")
    desc = desc or default_desc("dgrad")
    Nb, Cg = G.shape
    Dw, Cw = _w_dims(W, w_is_cd)
    if Cw != Cg:
        raise ValueError("shape mismatch")
    if out is None:
        out = torch.empty((Nb, Dw), dtype=torch.float32, device=G.device)
    return _run("hdqt_gemm_dgrad", desc, G, W, out, Nb, Dw, Cg, w_is_cd, Nb, Dw, Cg, workspace, dev_status)


def gemm_wgrad(X, G, desc: Optional[GemmDesc] = None, w_is_cd: bool = False, workspace=None, dev_status=None,
               out=None):
    """dW = X^T G in W's layout ([D,C], or [C,D] when w_is_cd). Returns (dW, workspace)."""
    _req(X, "X"); _req(G, "G")
    desc = desc or default_desc("wgrad")
    Nb, D = X.shape
    Nb2, Cg = G.shape
    if Nb != Nb2:
        raise ValueError("shape mismatch")
    M, N = (Cg, D) if w_is_cd else (D, Cg)
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=X.device)
    return _run("hdqt_gemm_wgrad", desc, X, G, out, Nb, D, Cg, w_is_cd, M, N, Nb, workspace, dev_status)


# ---- convolution without a materialised patch matrix ------------------------------------------------

def conv2d_out_size(H: int, W: int, kernel, stride: int, padding: int):
    """Output height and width; `kernel` is an int (square) or a (kh, kw) pair."""
    kh, kw = (kernel, kernel) if isinstance(kernel, int) else kernel
    return (H + 2 * padding - kh) // stride + 1, (W + 2 * padding - kw) // stride + 1


def conv2d_fwd(X, W, stride: int = 1, padding: int = 0, desc: Optional[GemmDesc] = None, workspace=None,
               dev_status=None, out=None):
    """Y[B,Ho,Wo,Cout] from X[B,H,W,Cin] (NHWC, Cin % 32 == 0) and W[Cout,kh,kw,Cin]. Returns (Y, workspace)."""
    _req(X, "X"); _req(W, "W")
    desc = desc or default_desc("fwd")
    B, H, Wd, Cin = X.shape
    Cout, kh, kw, Cin2 = W.shape
    if Cin2 != Cin:
        raise ValueError("shape mismatch")
    Ho, Wo = conv2d_out_size(H, Wd, (kh, kw), stride, padding)
    g = Conv2dGeom(B, H, Wd, Cin, kh, kw, stride, padding)
    M, N, K = B * Ho * Wo, Cout, kh * kw * Cin
    if workspace is None:
        workspace = Workspace(desc, M, N, K, X.device)
    if out is None:
        out = torch.empty((B, Ho, Wo, Cout), dtype=torch.float32, device=X.device)
    _check(lib.hdqt_conv2d_fwd(C.byref(desc), C.byref(g), X.data_ptr(), W.data_ptr(), out.data_ptr(), Cout,
                               workspace.buf.data_ptr(), workspace.buf.numel(), _ptr(dev_status), _stream()),
           "hdqt_conv2d_fwd")
    return out, workspace


def conv2d_dgrad(G, W, padding: int = 0, desc: Optional[GemmDesc] = None, workspace=None, dev_status=None, out=None):
    """dX[B,H,W,Cin] of a stride-1 convolution from G[B,Ho,Wo,Cout] (NHWC, Cout % 32 == 0) and W[Cout,kh,kw,Cin]:
    the input gradient is itself a convolution, of G with the kernel rotated by 180 degrees and padding
    k-1-padding, so it runs through hdqt_conv2d_fwd with the dgrad roles (stochastic rounding on G, nearest on
    W): contraction over (kh, kw, cout), no patch-matrix gradient and no scatter-add.  Returns (dX, workspace)."""
    _req(G, "G"); _req(W, "W")
    desc = desc or default_desc("dgrad")
    Cout, kh, kw, Cin = W.shape
    if G.shape[3] != Cout or kh - 1 - padding != kw - 1 - padding or kh - 1 - padding < 0:
        raise ValueError("shape mismatch")
    w_rot = W.flip(1, 2).permute(3, 1, 2, 0).contiguous()          # [Cin, kh, kw, Cout]
    return conv2d_fwd(G, w_rot, 1, kh - 1 - padding, desc=desc, workspace=workspace, dev_status=dev_status, out=out)


def conv2d_wgrad(X, G, kernel, stride: int = 1, padding: int = 0, desc: Optional[GemmDesc] = None,
                 workspace=None, dev_status=None, out=None):
    """dW[Cout,kh,kw,Cin] from X[B,H,W,Cin] and G[B,Ho,Wo,Cout] (both NHWC); `kernel` is an int or (kh, kw).
    Returns (dW, workspace)."""
    _req(X, "X"); _req(G, "G")
    desc = desc or default_desc("wgrad")
    B, H, Wd, Cin = X.shape
    Cout = G.shape[3]
    kh, kw = (kernel, kernel) if isinstance(kernel, int) else kernel
    Ho, Wo = conv2d_out_size(H, Wd, (kh, kw), stride, padding)
    if tuple(G.shape[:3]) != (B, Ho, Wo):
        raise ValueError("shape mismatch")
    g = Conv2dGeom(B, H, Wd, Cin, kh, kw, stride, padding)
    M, N, K = Cout, kh * kw * Cin, B * Ho * Wo
    if workspace is None:
        workspace = Workspace(desc, M, N, K, X.device)
    if out is None:
        out = torch.empty((Cout, kh, kw, Cin), dtype=torch.float32, device=X.device)
    _check(lib.hdqt_conv2d_wgrad(C.byref(desc), C.byref(g), X.data_ptr(), G.data_ptr(), out.data_ptr(), Cout,
                                 workspace.buf.data_ptr(), workspace.buf.numel(), _ptr(dev_status), _stream()),
           "hdqt_conv2d_wgrad")
    return out, workspace


def mma_rate_tops(iters: int = 20000, repeats: int = 3, dev_status=None) -> float:
    """Integer tensor rate (TOP/s) of back-to-back M128 N256 K32 kind::i8 MMAs on all SMs (no loads, no epilogue),
    best of `repeats` timed launches: the ceiling of the tiled GEMM at the current clocks."""
    ops = C.c_int64(0)
    best = 0.0
    for _ in range(repeats + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        _check(lib.hdqt_selftest_mma_rate(iters, C.byref(ops), _ptr(dev_status), _stream()), "hdqt_selftest_mma_rate")
        e1.record()
        torch.cuda.synchronize()
        best = max(best, ops.value / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return best
