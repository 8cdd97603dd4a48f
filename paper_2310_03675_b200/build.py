"""Builds the C-ABI CUDA library in-tree: paper_2310_03675_b200/libhdqt.so (sm_100a only)."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libhdqt.so")
SOURCES = ["hdqt_api.cu", "hdqt_quant.cu", "hdqt_gemm.cu"]


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found; the HDQT library needs the CUDA toolkit to build")
    return cand


STAMP_PATH = LIB_PATH + ".stamp"


def _deps():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC)) + [os.path.join(ROOT, "include", "hdqt.h")]


def sources_digest() -> str:
    """Digest of every file the library is compiled from (contents, not time stamps)."""
    h = hashlib.sha256()
    for d in _deps():
        h.update(os.path.basename(d).encode())
        with open(d, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def stamp_matches_sources() -> bool:
    """True if the library beside the sources was built from exactly these sources."""
    try:
        with open(STAMP_PATH) as f:
            return f.read().strip() == sources_digest()
    except OSError:
        return False


def needs_rebuild() -> bool:
    return not os.path.exists(LIB_PATH) or not stamp_matches_sources()


def _compile(out_path: str, defines=(), verbose: bool = False) -> None:
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++20", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    cmd += [f"-D{d}" for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    tmp = out_path + ".tmp"
    cmd += ["-o", tmp]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    os.replace(tmp, out_path)


def build_timeline() -> str:
    """Tuning build with the GEMM kernels' event timeline compiled in (libhdqt_tl.so, exports
    hdqt_debug_timeline besides the regular entry points).  Not loaded by the binding."""
    out = os.path.join(PKG_DIR, "libhdqt_tl.so")
    _compile(out, defines=("HDQT_TIMELINE",))
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu into one shared library for sm_100a. Returns the library path."""
    if not force and not needs_rebuild():
        return LIB_PATH
    _compile(LIB_PATH, verbose=verbose)
    with open(STAMP_PATH, "w") as f:
        f.write(sources_digest() + "\n")
    return LIB_PATH


if __name__ == "__main__":
    if "--timeline" in sys.argv:
        print(build_timeline())
    else:
        print(build(force=True, verbose="-v" in sys.argv))
