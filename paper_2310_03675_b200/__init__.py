"""B200-native HDQT quantized training GEMM (Hadamard transform -> int4
quantize -> tiled int8 tensor-core GEMM with 8-bit per-tile accumulators).

`hdqt` (the ctypes binding over the C-ABI library) is imported lazily so that
the seeded input generators in `inputs` can be used without the CUDA library.
"""

__all__ = ["hdqt", "inputs"]


def __getattr__(name):
    if name == "hdqt":
        import importlib
        return importlib.import_module(__name__ + ".hdqt")
    raise AttributeError(name)
