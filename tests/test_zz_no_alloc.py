"""gemm_s4_static: the INT4 GEMM for callers that must not allocate on the device.

A serving process that has given all device memory to its own pool, or a
latency-critical loop that cannot take cudaMalloc's device-wide synchronisation,
cannot use gemm_s4 (it allocates its workspace on first use) and may have no
buffer to pass to gemm_s4_ws.  gemm_s4_static unpacks into a fixed array inside
the library instead.  This test calls it through the C-ABI twice in a row and
requires bit-identical results to gemm_s4 (integer path: the tolerance of the
INT4 parity tests is exact equality).  It runs last so that a failure here
cannot hide any other test, and it passes on its own in a fresh process too.
"""
import numpy as np
import pytest
import torch

from paper_2608_10103_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def test_static_scratch_matches_gemm_s4_on_two_calls_in_a_row():
    L = binding.lib()
    stream = torch.cuda.current_stream()
    handle = int(stream.cuda_stream)
    # two different problems back to back: the second must not see the first one's leftovers
    cases = [(1500, 1100, 2048, 41), (640, 2304, 1056, 42)]
    for M, N, K, seed in cases:
        assert binding.gemm_s4_workspace_bytes(M, N, K) <= binding.gemm_s4_static_capacity()
        A, B = synth.s4_uniform(M, N, K, seed)
        dA, dB = _dev(A), _dev(B)
        want = torch.full((M, N), -3, dtype=torch.int32, device="cuda")
        got = torch.full((M, N), -5, dtype=torch.int32, device="cuda")
        assert L.gemm_s4(M, N, K, dA.data_ptr(), dB.data_ptr(), want.data_ptr(), handle) == 0
        assert L.gemm_s4_static(M, N, K, dA.data_ptr(), dB.data_ptr(), got.data_ptr(), handle) == 0
        stream.synchronize()
        assert torch.equal(got, want), "gemm_s4_static differs from gemm_s4 (M=%d N=%d K=%d)" % (M, N, K)
    assert binding.gemm_last_device_status() == 0


def test_static_scratch_refuses_what_does_not_fit():
    L = binding.lib()
    cap = binding.gemm_s4_static_capacity()
    assert cap == 32 << 20
    M = N = K = 4096                                  # exactly at the limit: accepted
    assert binding.gemm_s4_workspace_bytes(M, N, K) == cap
    A = torch.zeros((M, K // 2), dtype=torch.uint8, device="cuda")
    C = torch.full((M, N), 9, dtype=torch.int32, device="cuda")
    assert L.gemm_s4_static(M, N, K, A.data_ptr(), A.data_ptr(), C.data_ptr(), None) == 0
    torch.cuda.synchronize()
    assert int(C.abs().max()) == 0
    C.fill_(9)
    # one more row of A no longer fits: refused, nothing enqueued
    assert L.gemm_s4_static(M + 1, N, K, A.data_ptr(), A.data_ptr(), C.data_ptr(), None) == -7
    assert L.gemm_s4_static(M, N, 48, A.data_ptr(), A.data_ptr(), C.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert int((C != 9).sum()) == 0
    with pytest.raises(binding.GemmError) as e:
        binding.gemm_s4_static(torch.zeros((8192, 4096), dtype=torch.uint8, device="cuda"),
                               torch.zeros((64, 4096), dtype=torch.uint8, device="cuda"))
    assert e.value.code == -7
