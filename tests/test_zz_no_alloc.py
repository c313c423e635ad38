"""gemm_s4_static: the INT4 GEMM for callers that must not allocate on the device.

A serving process that has handed all device memory to its own pool, or a loop that must not
run into an allocator call, cannot use gemm_s4 (it leases scratch that is allocated on first
use) and may have no buffer to lend to gemm_s4_ws.  gemm_s4_static unpacks into a fixed array
inside the library instead.  These tests call it through the C-ABI twice in a row, compare
every result with the CPU oracle (integer path: exact equality) and with what gemm_s4 gives,
and watch the device's free memory across the calls.  The file is collected last so that a
failure here cannot hide any other test; it also passes on its own in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def test_static_scratch_matches_the_oracle_on_two_calls_in_a_row():
    L = binding.lib()
    stream = torch.cuda.current_stream()
    handle = int(stream.cuda_stream)
    # two different problems back to back: the second must not see the first one's leftovers
    cases = [(1500, 1100, 2048, 41), (640, 2304, 1056, 42)]
    inputs = []
    for M, N, K, seed in cases:
        assert binding.gemm_s4_workspace_bytes(M, N, K) <= binding.gemm_s4_static_capacity()
        A, B = synth.s4_uniform(M, N, K, seed)
        inputs.append((A, B, _dev(A), _dev(B),
                       torch.full((M, N), -5, dtype=torch.int32, device="cuda"),
                       torch.full((M, N), -3, dtype=torch.int32, device="cuda")))
    # the first call on a device looks the array's address up (and loads the module that
    # holds it): do that before watching the allocator
    A, B, dA, dB, got, _ = inputs[0]
    M, N, K = cases[0][:3]
    assert L.gemm_s4_static(M, N, K, dA.data_ptr(), dB.data_ptr(), got.data_ptr(), handle) == 0
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for (M, N, K, seed), (A, B, dA, dB, got, other) in zip(cases, inputs):
        got.fill_(-5)
        assert L.gemm_s4_static(M, N, K, dA.data_ptr(), dB.data_ptr(), got.data_ptr(), handle) == 0
    stream.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "gemm_s4_static changed the free device memory"
    for (M, N, K, seed), (A, B, dA, dB, got, other) in zip(cases, inputs):
        want = oracle.gemm_s4(A, B, K)
        assert np.array_equal(got.cpu().numpy(), want), \
            "gemm_s4_static differs from the oracle (M=%d N=%d K=%d)" % (M, N, K)
        # and the allocating entry point, by whichever route it takes, agrees
        assert L.gemm_s4(M, N, K, dA.data_ptr(), dB.data_ptr(), other.data_ptr(), handle) == 0
        stream.synchronize()
        assert torch.equal(got, other)
    assert binding.gemm_last_device_status() == 0


def test_static_scratch_at_capacity_and_beyond():
    L = binding.lib()
    cap = binding.gemm_s4_static_capacity()
    assert cap == 32 << 20
    M = N = K = 4096                                  # exactly at the limit: accepted
    assert binding.gemm_s4_workspace_bytes(M, N, K) == cap
    A, B = synth.s4_uniform(M, N, K, seed=43)         # random operands: the last bytes of the
    dA, dB = _dev(A), _dev(B)                         # array are read for real
    C = torch.full((M, N), 9, dtype=torch.int32, device="cuda")
    assert L.gemm_s4_static(M, N, K, dA.data_ptr(), dB.data_ptr(), C.data_ptr(), None) == 0
    torch.cuda.synchronize()
    got = C.cpu().numpy()
    rows = np.array([0, 1, 2047, 2048, 4094, 4095], dtype=np.int32)
    cols = np.array([0, 255, 256, 4095], dtype=np.int32)
    assert np.array_equal(got[rows], oracle.gemm_s4(A, B, K, rows=rows))
    assert np.array_equal(got[:, cols], oracle.gemm_s4(A, B, K, cols=cols))
    C.fill_(9)
    # one more row of A no longer fits: refused, nothing enqueued
    assert L.gemm_s4_static(M + 1, N, K, dA.data_ptr(), dB.data_ptr(), C.data_ptr(), None) == -7
    assert L.gemm_s4_static(M, N, 48, dA.data_ptr(), dB.data_ptr(), C.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert int((C != 9).sum()) == 0
    with pytest.raises(binding.GemmError) as e:
        binding.gemm_s4_static(torch.zeros((8192, 4096), dtype=torch.uint8, device="cuda"),
                               torch.zeros((64, 4096), dtype=torch.uint8, device="cuda"))
    assert e.value.code == -7
