"""The allocation-free quantize entry point (hdqt_quantize_hadamard_static) against the regular one.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The entry point serves callers that may not allocate device memory when they
quantize (all memory already handed to the application's pool, a host that forbids allocation, a
loop that cannot afford an allocation's device-wide synchronisation): its scratch is a fixed array
inside the library, shared by all calls, so the second call in a row must not see the first one's
leftovers."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2310_03675_b200 import inputs


@pytest.fixture(scope="module")
def hdqt():
    from paper_2310_03675_b200 import hdqt as mod
    return mod


def test_oversized_operand_is_refused_on_the_host(hdqt):
    """rows * K_pad/32 beyond the built-in array: a clear error, nothing launched (no GPU needed)."""
    q = hdqt.lib.hdqt_quantize_hadamard_static
    TOO_LARGE = 8
    assert q(256, 8193, 8192, 8192, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == TOO_LARGE
    assert q(256, 1 << 22, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == TOO_LARGE
    assert hdqt.lib.hdqt_status_string(TOO_LARGE).decode() == "operand too large for the built-in scratch array"
    assert q(None, 4, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == 1   # invalid argument
    assert hdqt.STATIC_SCRATCH_BYTES == 4 * 1024 * 1024 + 256


@pytest.mark.gpu
def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row(hdqt):
    dev = torch.device("cuda")
    status = hdqt.new_status(dev)
    # two different operands back to back: the second has a much smaller maximum and fewer rows, so any
    # leftover of the first call in the shared array (stale maximum, stale row norms) would show
    cases = [
        (inputs.heavy_tailed(1000, 2080, seed=41), False, hdqt.ROUND_STOCHASTIC),
        ((inputs.activations(300, 561, seed=42) * 1e-3).astype(np.float32), True, hdqt.ROUND_NEAREST),
    ]
    for x, strided, mode in cases:
        src = torch.from_numpy(np.ascontiguousarray(x.T)).to(dev).t() if strided else torch.from_numpy(x).to(dev)
        rows, K = x.shape
        Kp = hdqt.padded_k(K)
        want_codes, want_step, want_norms = hdqt.quantize_hadamard(src, 32, 4, 0.975, mode, seed=11, tag=5,
                                                                   want_norms=True, dev_status=status)
        codes = torch.full((rows, Kp), 0x55, dtype=torch.int8, device=dev)
        step = torch.full((1,), -1.0, device=dev)
        norms = torch.full(((rows + 127) // 128, Kp // 32), -1, dtype=torch.int32, device=dev)
        ld_row, ld_k = src.stride()
        rc = hdqt.lib.hdqt_quantize_hadamard_static(src.data_ptr(), rows, K, ld_row, ld_k, 32, 4, 0.975, mode, 11, 5,
                                                    codes.data_ptr(), step.data_ptr(), norms.data_ptr(),
                                                    status.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        hdqt.check_device_status(status)
        # integer outputs are compared exactly, the fp32 scale within the 1e-5 the other tests use
        assert torch.equal(codes, want_codes)
        assert torch.equal(norms, want_norms)
        assert abs(step.item() - want_step.item()) <= 1e-5 * abs(want_step.item())
