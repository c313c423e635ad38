"""GPU parity of the fused INT4 route (nibbles expanded inside the GEMM kernel) against the
oracle, and bit-equality with the default pre-pass route."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _fused_route():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(2)
    yield
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_config_override(0, 0, 0, 0)
    assert binding.gemm_last_device_status() == 0


def _force_pair_tile(bn=256):
    binding.gemm_set_config_override(bn, 0, 2, 1)    # the pair tiles of the fused variant: 256, 128 wide


# K = 32: a single 16-byte chunk per row; 96/160: partly filled packed slots; 256/512: whole
# slots; 1056, 4128: ragged tails; M, N not tile multiples
@pytest.mark.parametrize("M,N,K", [(256, 256, 32), (256, 256, 256), (130, 70, 96), (300, 500, 160),
                                   (512, 768, 512), (640, 1100, 1056), (1, 8, 64), (1000, 1000, 4128)])
@pytest.mark.parametrize("bn", [256, 128])
def test_fused_full_compare(M, N, K, bn):
    _force_pair_tile(bn)
    assert "fused_unpack" in binding.gemm_query_config("s4", M, N, K)
    A, B = synth.s4_uniform(M, N, K, seed=M + K)
    for rep in range(2):
        check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


def test_fused_is_what_the_selector_reports_and_runs_at_2048():
    M = N = K = 2048
    assert "fused_unpack" in binding.gemm_query_config("s4", M, N, K)
    A, B = synth.s4_uniform(M, N, K, seed=5)
    C = run_gpu("s4", A, B, fill=-7)
    check_against_oracle("s4", A, B, C, force_full=True)
    binding.gemm_set_s4_scheme(1)
    assert "prepass" in binding.gemm_query_config("s4", M, N, K)
    assert np.array_equal(C, run_gpu("s4", A, B, fill=-7))


def test_fused_falls_back_where_the_variant_does_not_apply():
    M, N, K = 640, 512, 1056
    binding.gemm_set_config_override(64, 0, 2, 1)       # no fused variant for this pair tile
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "prepass" in cfg and "fused" not in cfg
    A, B = synth.s4_uniform(M, N, K, seed=6)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


@pytest.mark.parametrize("split_k", [1, 3])
@pytest.mark.parametrize("bn", [256, 128, 64, 32])
@pytest.mark.parametrize("M,N,K", [(16, 520, 1056), (130, 300, 2048), (1, 64, 96), (400, 700, 512)])
def test_fused_one_cta_tiles_with_split_k(M, N, K, bn, split_k):
    """Every one-CTA fused variant, with K split over several CTAs (each partial holds a
    multiple of 256 and is shifted before it is added into C) and with tiles whose rows beyond
    M or N are not expanded at all."""
    binding.gemm_set_config_override(bn, 0, 1, split_k)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "fused_unpack" in cfg and ("BN=%d " % bn) in cfg
    A, B = synth.s4_uniform(M, N, K, seed=bn + split_k)
    for rep in range(2):
        check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


@pytest.mark.parametrize("split_k", [2, 3, 5])
@pytest.mark.parametrize("bn", [256, 128])
@pytest.mark.parametrize("M,N,K", [(300, 500, 1056), (512, 768, 2048), (256, 2048, 8192), (1000, 1000, 4128)])
def test_fused_pair_tiles_with_split_k(M, N, K, bn, split_k):
    """K divided in whole packed slots between CTA pairs that add into a zeroed C."""
    binding.gemm_set_config_override(bn, 0, 2, split_k)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "fused_unpack" in cfg and "cta_group=2" in cfg
    A, B = synth.s4_uniform(M, N, K, seed=M + split_k)
    for rep in range(2):
        check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


def test_automatic_route_by_shape():
    binding.gemm_set_s4_scheme(0)
    assert "fused_unpack" in binding.gemm_query_config("s4", 48, 8192, 8192)      # few rows
    assert binding.gemm_query_config("s4", 16, 8192, 8192).startswith("few_rows")  # up to 16: no tiles
    assert "fused_unpack" in binding.gemm_query_config("s4", 8192, 64, 4096)
    assert "fused_unpack" in binding.gemm_query_config("s4", 512, 512, 512)       # small
    assert "fused_unpack" in binding.gemm_query_config("s4", 2048, 2048, 2048)    # one wave of pair tiles
    # large in both dimensions (at least a wave of pair tiles, K >= 2048): the fused pair kernel,
    # with A as an int8 image where that pays
    big = binding.gemm_query_config("s4", 8192, 8192, 8192)
    assert "fused_unpack" in big and "a=int8_image" in big
    mid = binding.gemm_query_config("s4", 4096, 4096, 4096)
    assert "fused_unpack" in mid and "a=int8_image" not in mid
    assert "fused_unpack" in binding.gemm_query_config("s4", 2048, 8192, 8192)
    assert "prepass" in binding.gemm_query_config("s4", 8192, 8192, 1024)       # short K
    assert "prepass" in binding.gemm_query_config("s4", 1536, 1536, 8192)       # less than a wave
    assert "prepass" in binding.gemm_query_config("s4", 512, 4096, 4096)
    # a short side against a large N K: M N / (M + N) <= 384, or <= 1024 rows on well-filled pair tiles
    assert "fused_unpack" in binding.gemm_query_config("s4", 256, 28672, 8192)
    assert "fused_unpack" in binding.gemm_query_config("s4", 28672, 256, 8192)
    assert "fused_unpack" in binding.gemm_query_config("s4", 384, 4096, 16384)
    assert "fused_unpack" in binding.gemm_query_config("s4", 1024, 8192, 8192)
    # 96 pair tiles on 74 pairs: the last 22 are split in two along K, which fills the waves to 80 %
    assert "fused_unpack" in binding.gemm_query_config("s4", 640, 8192, 8192)
    assert "prepass" in binding.gemm_query_config("s4", 896, 2048, 8192)
    binding.gemm_set_s4_scheme(1)
    assert "prepass" in binding.gemm_query_config("s4", 16, 8192, 8192)
    binding.gemm_set_s4_scheme(0)
    M, N, K = 48, 4096, 8192
    A, B = synth.s4_uniform(M, N, K, seed=11)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)
    for M, N, K in [(200, 20000, 2080), (300, 5000, 1056)]:   # two waves of pair tiles; one-CTA tiles
        assert "fused_unpack" in binding.gemm_query_config("s4", M, N, K)
        A, B = synth.s4_uniform(M, N, K, seed=M)
        check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), seed=M)


def test_fused_extreme_values_and_nibble_positions():
    """-8 * -8 over the longest K the INT4 path allows for its tile (the 256 * C accumulators
    peak at 16384 * K), -8 * 7, and one-hot K positions across chunk and slot boundaries."""
    _force_pair_tile()
    M, N, K = 256, 256, 8192
    lo = np.full((M, K // 2), 0x88, dtype=np.uint8)       # every nibble -8
    hi = np.full((N, K // 2), 0x77, dtype=np.uint8)       # every nibble 7
    assert np.array_equal(run_gpu("s4", lo, lo, fill=-7), np.full((M, N), 64 * K, dtype=np.int32))
    assert np.array_equal(run_gpu("s4", lo, hi, fill=-7), np.full((M, N), -56 * K, dtype=np.int32))
    K = 1024
    ks = [0, 1, 2, 7, 8, 31, 32, 33, 63, 64, 127, 128, 255, 256, 257, 511, 512, 1023]
    A = np.zeros((len(ks), K // 2), dtype=np.uint8)
    B = np.zeros((len(ks), K // 2), dtype=np.uint8)
    for r, k in enumerate(ks):
        A[r, k // 2] = (3 & 15) << (4 * (k & 1))           # a(r, k) = 3
        B[r, k // 2] = (-5 & 15) << (4 * (k & 1))          # b(r, k) = -5
    want = np.where(np.eye(len(ks), dtype=bool), -15, 0).astype(np.int32)
    assert np.array_equal(run_gpu("s4", A, B, fill=-7), want)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.float16])
def test_fused_dequant(out_dtype):
    _force_pair_tile()
    M, N, K = 650, 1096, 1184
    A, B = synth.s4_uniform(M, N, K, seed=9)
    g = np.random.Generator(np.random.PCG64(9))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    ref = oracle.dequant_ref(oracle.gemm_s4_i64(A, B, K), rs, cs)
    C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    binding.gemm_s4_dequant(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
    torch.cuda.synchronize()
    ok, worst = oracle.dequant_check(C.cpu().numpy(), ref, out_dtype == torch.float16)
    assert ok, "error %.3g x bound" % worst


def test_fused_many_tiles_per_cta_sampled_4096():
    M = N = K = 4096
    A, B = synth.s4_uniform(M, N, K, seed=2)
    assert "fused_unpack" in binding.gemm_query_config("s4", M, N, K)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), seed=2)
