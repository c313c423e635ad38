"""GPU parity of the 512 x 256 CTA-pair kernel (two accumulators per CTA fill tensor memory;
the MMA issuer restarts on the first one while the second is still being read out), forced for
every shape here through gemm_set_kernel_family(2), against the oracle through the C-ABI."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, freivalds, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _wide_family():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_kernel_family(2)
    yield
    binding.gemm_set_kernel_family(0)
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_trace_enable(0)
    assert binding.gemm_last_device_status() == 0


def is_wide(prec, M, N, K):
    return "BM=512 BN=256" in binding.gemm_query_config(prec, M, N, K)


# one tile; ragged in M, N and K; one k-block (shorter than the ring); K longer than the ring
# by one; more tiles than CTA pairs with a short mainloop (tile hand-over dominates)
SHAPES = [(512, 256, 512), (1000, 700, 328), (513, 257, 64), (300, 100, 640), (77, 3, 64),
          (1536, 1280, 1088), (5000, 4000, 128), (2048, 2048, 2048)]


@pytest.mark.parametrize("prec", ["fp16", "s8"])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_wide_matches_the_oracle(prec, M, N, K):
    if prec == "s8":
        K = (K + 15) // 16 * 16
    assert is_wide(prec, M, N, K)
    A, B = synth.make(prec, M, N, K, seed=M + N + K)
    C = run_gpu(prec, A, B, fill=-7)
    check_against_oracle(prec, A, B, C, seed=M)
    if max(M, N) > 2048:
        freivalds(prec, A, B, C, seed=M, vectors=4)


@pytest.mark.parametrize("prec", ["fp16", "s8"])
def test_wide_rows_that_are_not_16_byte_multiples(prec):
    M, N, K = 700, 1030 + 1, 256          # N % 4 != 0: plain predicated stores
    assert is_wide(prec, M, N, K)
    A, B = synth.make(prec, M, N, K, seed=5)
    check_against_oracle(prec, A, B, run_gpu(prec, A, B, fill=-7), seed=5)


@pytest.mark.parametrize("prec", ["fp16", "s8"])
def test_wide_index_mapping_product_table(prec):
    """a(i,0) = i mod 97 - 48, b(j,0) = j mod 89 - 44, rest 0: C[i][j] is their product, so a
    row, column, accumulator half or CTA half that lands in the wrong place shows up."""
    M, N, K = 2100, 1300, 192
    if prec == "fp16":
        A, B = np.zeros((M, K), np.float16), np.zeros((N, K), np.float16)
    else:
        A, B = np.zeros((M, K), np.int8), np.zeros((N, K), np.int8)
    A[:, 0] = (np.arange(M) % 97) - 48
    B[:, 0] = (np.arange(N) % 89) - 44
    want = np.outer(A[:, 0].astype(np.int64), B[:, 0].astype(np.int64))
    got = run_gpu(prec, A, B, fill=-7)
    assert np.array_equal(got.astype(np.int64), want)


def test_wide_config_8192_fp16_sampled_and_repeatable():
    N = 8192
    assert is_wide("fp16", N, N, N)
    A, B = synth.fp16_normal_clipped(N, N, N, seed=3)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.empty((N, N), dtype=torch.float32, device="cuda")
    for rep in range(3):                  # back-to-back launches chained by early start
        binding.gemm_fp16(dA, dB, C)
    torch.cuda.synchronize()
    got = C.cpu().numpy()
    check_against_oracle("fp16", A, B, got, seed=3)
    freivalds("fp16", A, B, got, seed=3)


def test_wide_s8_4096_exact_and_band_heights():
    N = 4096
    A, B = synth.s8_uniform(N, N, N, seed=synth.sweep_seed("s8", N))
    want_rows = None
    for g in (0, 1, 3, 8):
        binding.gemm_set_config_override(0, g, 0, 0)
        C = run_gpu("s8", A, B)
        check_against_oracle("s8", A, B, C, seed=g)
        freivalds("s8", A, B, C, seed=g, vectors=2)


def test_wide_fp16_output_and_dequant():
    M, N, K = 1100, 1544, 704
    A, B = synth.fp16_normal_clipped(M, N, K, seed=11)
    ref, S = oracle.gemm_fp16(A, B)
    C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    ok, worst = oracle.fp16_out_check(C.cpu().numpy(), ref, S)
    assert ok, "error %.3g x bound" % worst
    A8, B8 = synth.s8_uniform(M, N, K, seed=12)
    g = np.random.Generator(np.random.PCG64(13))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * g.choice([-1.0, 1.0], N) * 1e-1).astype(np.float32)
    ref = oracle.dequant_ref(oracle.gemm_s8_i64(A8, B8), rs, cs)
    for dt in (torch.float32, torch.float16):
        C = torch.full((M, N), float("nan"), dtype=dt, device="cuda")
        binding.gemm_s8_dequant(to_dev(A8), to_dev(B8), to_dev(rs), to_dev(cs), C, dt)
        torch.cuda.synchronize()
        ok, worst = oracle.dequant_check(C.cpu().numpy(), ref, dt == torch.float16)
        assert ok, "error %.3g x bound" % worst


def test_wide_fp16_output_ragged_columns():
    M, N, K = 600, 516, 128               # N % 8 != 0: 16-bit rows are not 16-byte multiples
    A, B = synth.fp16_uniform(M, N, K, seed=14)
    ref, S = oracle.gemm_fp16(A, B)
    C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    assert oracle.fp16_out_check(C.cpu().numpy(), ref, S)[0]


def test_wide_expired_wait_is_reported_and_the_context_survives():
    """Failure drill without a fault: a host switch makes the producer leave one ring slot
    unfilled, the bounded waits run out, the kernel records a code, drains and returns."""
    M, N, K = 512, 256, 1024
    A, B = synth.s8_uniform(M, N, K, seed=9)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    assert binding.gemm_last_device_status() == 0
    try:
        binding.gemm_trace_enable(16)
        t0 = time.time()
        binding.gemm_s8(dA, dB, C)
        torch.cuda.synchronize()
        took = time.time() - t0
        binding.gemm_trace_enable(0)
        status = binding.gemm_last_device_status()
        assert status in (1, 2, 3), "expected a recorded wait expiry, got %d" % status
        assert 1.5 < took < 30.0
        binding.gemm_s8(dA, dB, C)
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B))
    finally:
        binding.gemm_trace_enable(0)


def test_wide_cycle_accounting_reports_both_accumulator_waits():
    N = 2048
    A, B = synth.s8_uniform(N, N, N, seed=2)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.empty((N, N), dtype=torch.int32, device="cuda")
    binding.gemm_trace_enable(1)
    binding.gemm_s8(dA, dB, C)
    tr = binding.gemm_trace_read(148)
    binding.gemm_trace_enable(0)
    busy = [t for t in tr if t["cycles"]]
    assert len(busy) == 2 * 32                      # 4 x 8 tiles, one CTA pair each
    assert sum(t["tiles"] for t in busy) == 2 * 32
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B))
