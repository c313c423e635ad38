"""The kernels never wait without a limit.  This drill makes one operand slot stay empty
(a host-requested switch; nothing faults, traps or spins forever): the waits must run out
after their 2 s limit, the kernel must record a status code, drain and return, and the
next call on the same context must work."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cta_group", [1, 2])
def test_expired_wait_is_reported_and_the_context_survives(cta_group):
    M, N, K = 256, 256, 1024                      # one tile, 16 k-blocks (> ring depth)
    A, B = synth.s8_uniform(M, N, K, seed=9)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    assert binding.gemm_last_device_status() == 0
    binding.gemm_set_config_override(256, 0, cta_group)
    try:
        binding.gemm_trace_enable(16)
        t0 = time.time()
        binding.gemm_s8(dA, dB, C)
        torch.cuda.synchronize()                  # returns: the kernel gave up by itself
        took = time.time() - t0
        binding.gemm_trace_enable(0)
        status = binding.gemm_last_device_status()
        assert status in (1, 2, 3), "expected a recorded wait expiry, got %d" % status
        assert 1.5 < took < 30.0
        assert binding.gemm_last_device_status() == 0        # reading clears it
        # the context is intact: the same call now gives the right answer
        binding.gemm_s8(dA, dB, C)
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B))
        assert binding.gemm_last_device_status() == 0
    finally:
        binding.gemm_trace_enable(0)
        binding.gemm_set_config_override(0, 0, 0)


@pytest.mark.parametrize("variant", ["pair tile", "one-CTA tile, exchanged operands"])
def test_expired_wait_in_the_fused_int4_kernels(variant):
    """Same drill through the kernel variants with the extra nibble-expansion warps and the
    second (packed) ring: a packed slot of CTA 0 is never filled."""
    if variant.startswith("pair"):
        M, N, K = 256, 256, 2048                  # one tile, 8 packed slots (> ring depth 2)
        override, swap, tag = (256, 0, 2, 1), 1, "fused_unpack"
    else:
        M, N, K = 16, 128, 4096                   # one tile, 16 packed slots (> ring depth 5)
        override, swap, tag = (32, 0, 1, 1), 2, "swap_ab"
    A, B = synth.s4_uniform(M, N, K, seed=10)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    assert binding.gemm_last_device_status() == 0
    binding.gemm_set_config_override(*override)
    binding.gemm_set_s4_scheme(2)
    binding.gemm_set_swap_ab(swap)
    try:
        assert tag in binding.gemm_query_config("s4", M, N, K)
        binding.gemm_trace_enable(16)
        t0 = time.time()
        binding.gemm_s4(dA, dB, C)
        torch.cuda.synchronize()
        took = time.time() - t0
        binding.gemm_trace_enable(0)
        status = binding.gemm_last_device_status()
        assert status in (1, 2, 3, 5), "expected a recorded wait expiry, got %d" % status
        assert 1.5 < took < 30.0
        binding.gemm_s4(dA, dB, C)
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), oracle.gemm_s4(A, B, K))
        assert binding.gemm_last_device_status() == 0
    finally:
        binding.gemm_trace_enable(0)
        binding.gemm_set_s4_scheme(0)
        binding.gemm_set_swap_ab(0)
        binding.gemm_set_config_override(0, 0, 0)


def test_expired_wait_in_the_cluster_split_k_kernel():
    """Same drill where four CTAs of a cluster share a tile and hand partial sums to rank 0
    through shared memory: rank 0 of the first cluster never gets one operand slot, gives up,
    and the other three (whose copies have long landed) leave with it."""
    M, N, K = 16, 1536, 8192
    A, B = synth.s8_uniform(M, N, K, seed=11)
    g = np.random.Generator(np.random.PCG64(11))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    d_rs, d_cs = torch.from_numpy(rs).cuda(), torch.from_numpy(cs).cuda()
    C = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    assert binding.gemm_last_device_status() == 0
    binding.gemm_set_config_override(32, 0, 1, 4)
    binding.gemm_set_swap_ab(2)
    try:
        binding.gemm_trace_enable(17)              # drill + cycle records
        t0 = time.time()
        binding.gemm_s8_dequant(dA, dB, d_rs, d_cs, C, torch.float16)
        torch.cuda.synchronize()
        took = time.time() - t0
        ctas = sum(1 for t in binding.gemm_trace_read(160) if t["cycles"] > 0)
        binding.gemm_trace_enable(0)
        assert ctas == 48, ctas                    # 12 tiles x 4 CTAs: the cluster split-K kernel ran
        status = binding.gemm_last_device_status()
        assert status in (1, 2, 3), "expected a recorded wait expiry, got %d" % status
        assert 1.5 < took < 30.0
        binding.gemm_s8_dequant(dA, dB, d_rs, d_cs, C, torch.float16)
        torch.cuda.synchronize()
        ref = oracle.dequant_ref(oracle.gemm_s8_i64(A, B), rs, cs)
        assert oracle.dequant_check(C.cpu().numpy(), ref, True)[0]
        assert binding.gemm_last_device_status() == 0
    finally:
        binding.gemm_trace_enable(0)
        binding.gemm_set_swap_ab(0)
        binding.gemm_set_config_override(0, 0, 0)
