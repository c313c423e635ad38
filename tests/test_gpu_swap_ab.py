"""GPU parity with the operands exchanged inside the library (the kernel's rows are the
caller's N side, C written along N by plain stores): every precision and output mode, with
and without split-K, and the automatic choice for INT4 problems with few rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _state():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_swap_ab(2)
    yield
    binding.gemm_set_swap_ab(0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_config_override(0, 0, 0, 0)
    assert binding.gemm_last_device_status() == 0


@pytest.mark.parametrize("prec", synth.PRECISIONS)
@pytest.mark.parametrize("M,N,K", [(16, 2048, 1056), (1, 777, 512), (64, 4096, 4096), (33, 130, 96),
                                   (300, 500, 640), (5, 3, 64)])
def test_swapped_full_compare(prec, M, N, K):
    assert "swap_ab" in binding.gemm_query_config(prec, M, N, K)
    A, B = synth.make(prec, M, N, K, seed=M + N)
    for rep in range(2):
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        check_against_oracle(prec, A, B, C, force_full=True)


@pytest.mark.parametrize("scheme", [1, 2])
@pytest.mark.parametrize("bn,split_k", [(32, 1), (32, 4), (64, 3), (128, 2), (256, 1)])
def test_swapped_int4_routes_tiles_and_split_k(bn, split_k, scheme):
    M, N, K = 24, 1300, 2048
    binding.gemm_set_s4_scheme(scheme)
    binding.gemm_set_config_override(bn, 0, 1, split_k)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "swap_ab" in cfg and ("fused_unpack" in cfg) == (scheme == 2)
    A, B = synth.s4_uniform(M, N, K, seed=bn + split_k)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


def test_swapped_output_variants():
    M, N, K = 40, 1096, 1184
    A, B = synth.fp16_normal_clipped(M, N, K, seed=3)
    ref, S = oracle.gemm_fp16(A, B)
    C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    ok, worst = oracle.fp16_out_check(C.cpu().numpy(), ref, S)
    assert ok, "fp16 out: %.3g x bound" % worst
    g = np.random.Generator(np.random.PCG64(4))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    for prec in ("s8", "s4"):
        A, B = synth.make(prec, M, N, K, seed=5)
        exact = oracle.gemm_s8_i64(A, B) if prec == "s8" else oracle.gemm_s4_i64(A, B, K)
        ref = oracle.dequant_ref(exact, rs, cs)
        fn = binding.gemm_s8_dequant if prec == "s8" else binding.gemm_s4_dequant
        for out_dtype in (torch.float32, torch.float16):
            C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
            fn(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
            torch.cuda.synchronize()
            ok, worst = oracle.dequant_check(C.cpu().numpy(), ref, out_dtype == torch.float16)
            assert ok, "%s %s: %.3g x bound" % (prec, out_dtype, worst)


def test_automatic_choice_for_few_rows():
    binding.gemm_set_swap_ab(0)
    cfg = binding.gemm_query_config("s4", 48, 8192, 8192)
    assert "fused_unpack" in cfg and "swap_ab" in cfg
    assert binding.gemm_query_config("s4", 16, 8192, 8192).startswith("few_rows")
    assert "swap_ab" in binding.gemm_query_config("s4", 64, 8192, 8192)
    assert "swap_ab" not in binding.gemm_query_config("s4", 128, 8192, 8192)
    assert "swap_ab" in binding.gemm_query_config("s8", 64, 8192, 8192)
    assert "swap_ab" not in binding.gemm_query_config("s8", 80, 8192, 8192)
    assert "swap_ab" not in binding.gemm_query_config("fp16", 64, 8192, 8192)
    assert "swap_ab" in binding.gemm_query_config("s8", 24, 8192, 8192)
    assert "swap_ab" in binding.gemm_query_config("fp16", 16, 8192, 8192)
    assert "swap_ab" not in binding.gemm_query_config("fp16", 128, 8192, 8192)
    assert "swap_ab" not in binding.gemm_query_config("s8", 16, 512, 8192)
    assert "swap_ab" not in binding.gemm_query_config("s8", 2048, 2048, 2048)
    M, N, K = 24, 8192, 4096
    for prec in synth.PRECISIONS:
        A, B = synth.make(prec, M, N, K, seed=12)
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        check_against_oracle(prec, A, B, C, force_full=True)
    binding.gemm_set_swap_ab(1)
    assert "swap_ab" not in binding.gemm_query_config("s8", 16, 8192, 8192)


@pytest.mark.parametrize("split_k", [1, 2])
def test_swapped_16_bit_outputs_on_the_32_wide_tile(split_k):
    """With exchanged operands C goes out by plain stores, so the 32-wide tile, which has no
    64-column staging block, serves the binary16 outputs too (with and without the split of K
    inside a cluster)."""
    M, N, K = 24, 1300, 2080
    binding.gemm_set_config_override(32, 0, 1, split_k)
    A, B = synth.fp16_normal_clipped(M, N, K, seed=8)
    ref, S = oracle.gemm_fp16(A, B)
    C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    ok, worst = oracle.fp16_out_check(C.cpu().numpy(), ref, S)
    assert ok, "fp16 out: %.3g x bound" % worst
    g = np.random.Generator(np.random.PCG64(8))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    for prec, scheme in (("s8", 0), ("s4", 1), ("s4", 2)):
        binding.gemm_set_s4_scheme(scheme)
        A, B = synth.make(prec, M, N, K, seed=9)
        exact = oracle.gemm_s8_i64(A, B) if prec == "s8" else oracle.gemm_s4_i64(A, B, K)
        ref = oracle.dequant_ref(exact, rs, cs)
        fn = binding.gemm_s8_dequant if prec == "s8" else binding.gemm_s4_dequant
        C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        fn(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, torch.float16)
        torch.cuda.synchronize()
        ok, worst = oracle.dequant_check(C.cpu().numpy(), ref, True)
        assert ok, "%s scheme %d: %.3g x bound" % (prec, scheme, worst)
