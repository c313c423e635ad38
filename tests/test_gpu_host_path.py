"""gemm_host: operands and result in host memory, blocked and overlapped transfers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import assert_block, oracle_block

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("prec", synth.PRECISIONS)
def test_host_path_multi_block(prec, pinned):
    M, N, K = 2500, 4200, 512                    # 2 x 3 blocks of 2048 rows, ragged last blocks
    A, B = synth.make(prec, M, N, K, seed=77)
    hA, hB = torch.from_numpy(A), torch.from_numpy(B)
    if pinned:
        hA, hB = hA.pin_memory(), hB.pin_memory()
    hC = torch.full((M, N), -7, dtype=torch.float32 if prec == "fp16" else torch.int32)
    if pinned:
        hC = hC.pin_memory()
    out = binding.gemm_host(prec, hA, hB, hC)
    torch.cuda.synchronize()
    assert out is hC
    ref, S = oracle_block(prec, A, B)
    assert_block(prec, hC.numpy(), ref, S, "host path")
    # a second call reuses the device buffers
    hC.fill_(-9)
    binding.gemm_host(prec, hA, hB, hC)
    torch.cuda.synchronize()
    assert_block(prec, hC.numpy(), ref, S, "host path, second call")
    assert binding.gemm_last_device_status() == 0


def test_host_path_small_and_odd_shapes():
    for prec, (M, N, K) in (("fp16", (1, 3, 8)), ("s8", (130, 70, 16)), ("s4", (33, 2049, 64))):
        A, B = synth.make(prec, M, N, K, seed=5)
        hC = binding.gemm_host(prec, torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory())
        torch.cuda.synchronize()
        ref, S = oracle_block(prec, A, B)
        assert_block(prec, hC.numpy(), ref, S, "host path %s" % prec)


def test_host_path_argument_errors_and_release():
    L = binding.lib()
    a = torch.zeros(64, 64, dtype=torch.int8).pin_memory()
    c = torch.zeros(64, 64, dtype=torch.int32).pin_memory()
    assert L.gemm_host(1, 64, 64, 64, None, a.data_ptr(), c.data_ptr(), None) == -1
    assert L.gemm_host(7, 64, 64, 64, a.data_ptr(), a.data_ptr(), c.data_ptr(), None) == -1
    assert L.gemm_host(1, 64, 64, 24, a.data_ptr(), a.data_ptr(), c.data_ptr(), None) == -2
    assert L.gemm_host(2, 64, 64, 48, a.data_ptr(), a.data_ptr(), c.data_ptr(), None) == -2
    with pytest.raises(TypeError):
        binding.gemm_host("s8", a.cuda(), a)
    binding.gemm_host_release()
    A, B = synth.s8_uniform(300, 200, 128, seed=3)
    hC = binding.gemm_host("s8", torch.from_numpy(A), torch.from_numpy(B))
    torch.cuda.synchronize()
    assert np.array_equal(hC.numpy(), oracle.gemm_s8(A, B))


def test_host_path_few_rows_after_other_precisions():
    """INT4 through the host entry point expands its operands into a scratch right in front of the
    GEMM; with a few rows that GEMM is the kernel that starts early and must not read the scratch
    before the expansion has finished (it once did, and returned sums of the call before)."""
    import numpy as np
    for rep in range(2):
        for prec in synth.PRECISIONS:
            for M, N, K in [(8, 4096, 2048), (3000, 12, 1056), (16, 5000, 4128)]:
                A, B = synth.make(prec, M, N, K, seed=5 + rep)
                hA, hB = torch.from_numpy(A).pin_memory(), torch.from_numpy(B).pin_memory()
                C = binding.gemm_host(prec, hA, hB)
                torch.cuda.synchronize()
                got = C.numpy()
                if prec == "fp16":
                    ref, S = oracle.gemm_fp16(A, B)
                    assert oracle.fp16_check(got, ref, S)[0], (prec, M, N, K)
                else:
                    ref = oracle.gemm_s8(A, B) if prec == "s8" else oracle.gemm_s4(A, B, K)
                    assert np.array_equal(got, ref), (prec, M, N, K, int((got != ref).sum()))
