"""The allocation-free quantize entry point (hdqt_quantize_hadamard_static) against the regular one and
against the CPU oracle.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The entry point serves callers that may not allocate device memory when they
quantize (all memory already handed to the application's pool, a host that forbids allocation, a
loop that cannot afford an allocation's device-wide synchronisation): its scratch is a fixed array
inside the library, shared by all calls, so the second call in a row must not see the first one's
leftovers, and the call itself must leave the amount of free device memory unchanged."""
import numpy as np
import pytest
import torch

from oracle import hdqt_oracle as O
from paper_2310_03675_b200 import inputs


@pytest.fixture(scope="module")
def hdqt():
    from paper_2310_03675_b200 import hdqt as mod
    return mod


def test_oversized_operand_is_refused_on_the_host(hdqt):
    """rows * K_pad/32 beyond the stated maximum: a clear error, nothing launched (no GPU needed)."""
    q = hdqt.lib.hdqt_quantize_hadamard_static
    TOO_LARGE = 8
    assert q(256, 8193, 8192, 8192, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == TOO_LARGE
    assert q(256, 1 << 22, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == TOO_LARGE
    assert hdqt.lib.hdqt_status_string(TOO_LARGE).decode() == "operand too large for the built-in scratch array"
    assert q(None, 4, 32, 32, 1, 32, 4, 1.0, 0, 0, 0, 256, 256, None, None, None) == 1   # invalid argument
    assert hdqt.STATIC_MAX_ROW_TILES == 2097152 and hdqt.STATIC_SCRATCH_BYTES == 256 + 4096
    assert hdqt.STATUS_NAMES[TOO_LARGE] == "STATIC_SCRATCH"


def _expected_norms(codes):
    rows, Kp = codes.shape
    sq = (codes.astype(np.int64) ** 2).reshape(rows, Kp // 32, 32).sum(2)
    return np.stack([sq[b * 128:(b + 1) * 128].max(0) for b in range((rows + 127) // 128)])


@pytest.mark.gpu
def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row(hdqt):
    dev = torch.device("cuda")
    status = hdqt.new_status(dev)
    # two different operands back to back: the second has a much smaller maximum and fewer rows, so any
    # leftover of the first call in the shared array (stale maximum, stale partial maxima) would show
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
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        rc = hdqt.lib.hdqt_quantize_hadamard_static(src.data_ptr(), rows, K, ld_row, ld_k, 32, 4, 0.975, mode, 11, 5,
                                                    codes.data_ptr(), step.data_ptr(), norms.data_ptr(),
                                                    status.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert rc == 0
        assert free_after == free_before          # nothing was allocated (or freed) on the device by the call
        hdqt.check_device_status(status)
        # every output is an exact function of the input: codes, tile norms and the fp32 scale all compare equal
        assert torch.equal(codes, want_codes)
        assert torch.equal(norms, want_norms)
        assert step.item() == want_step.item()
        # ... and equal to what the CPU oracle computes from the same operand
        o_codes, o_step, _ = O.quantize_hadamard(x, 32, 4, 0.975, mode, seed=11, tag=5)
        assert np.array_equal(codes.cpu().numpy(), o_codes)
        assert step.item() == float(o_step)
        assert np.array_equal(norms.cpu().numpy().astype(np.int64), _expected_norms(o_codes))
