"""GPU parity of the output variants: FP16-rounded C and fused dequantisation.
References come from the oracle's exact sums pushed through the definition in fp64."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import to_dev

pytestmark = pytest.mark.gpu

SHAPES16 = [(64, 1), (128, 1), (256, 1), (64, 2), (128, 2), (256, 2)]


@pytest.fixture(autouse=True)
def _clean_state():
    binding.gemm_set_config_override(0, 0, 0)
    yield
    binding.gemm_set_config_override(0, 0, 0)
    assert binding.gemm_last_device_status() == 0


def scales(M, N, seed):
    g = np.random.Generator(np.random.PCG64(seed))
    rs = (g.uniform(0.5, 2.0, M) * g.choice([-1.0, 1.0], M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * g.choice([-1.0, 1.0], N) * 1e-1).astype(np.float32)
    return rs, cs


def run_f16out(A, B):
    C = torch.full((A.shape[0], B.shape[0]), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    return C.cpu().numpy()


@pytest.mark.parametrize("M,N,K", [(512, 512, 512), (300, 520, 320), (129, 1032, 4128),
                                   (200, 100, 128), (77, 3, 64), (1, 8, 8)])
def test_fp16_out_full(M, N, K):
    A, B = synth.fp16_uniform(M, N, K, seed=M + N)
    ref, S = oracle.gemm_fp16(A, B)
    ok, worst = oracle.fp16_out_check(run_f16out(A, B), ref, S)
    assert ok, "error %.3g x bound" % worst


@pytest.mark.parametrize("bn,cta_group", SHAPES16)
def test_fp16_out_every_tile_shape(bn, cta_group):
    M, N, K = 650, 1096, 1184
    A, B = synth.fp16_normal_clipped(M, N, K, seed=bn + cta_group)
    ref, S = oracle.gemm_fp16(A, B)
    binding.gemm_set_config_override(bn, 0, cta_group)
    ok, worst = oracle.fp16_out_check(run_f16out(A, B), ref, S)
    assert ok, "error %.3g x bound" % worst



@pytest.mark.parametrize("bn,cta_group", SHAPES16)
def test_fp16_out_many_short_tiles_per_cta(bn, cta_group):
    """Short mainloop, several tiles per CTA: consecutive tiles' stores overlap (the 64-wide
    tile has a single 16-bit store block per tile)."""
    M, N, K = 3000, 1000, 32
    A, B = synth.fp16_normal_clipped(M, N, K, seed=bn)
    ref, S = oracle.gemm_fp16(A, B)
    binding.gemm_set_config_override(bn, 0, cta_group, 1)
    for rep in range(3):
        ok, worst = oracle.fp16_out_check(run_f16out(A, B), ref, S)
        assert ok, "repeat %d: error %.3g x bound" % (rep, worst)


def test_fp16_out_rejects_the_32_wide_tile():
    A, B = synth.fp16_uniform(64, 64, 64, seed=1)
    binding.gemm_set_config_override(32, 0, 1)
    with pytest.raises(binding.GemmError):
        run_f16out(A, B)


def test_fp16_out_sampled_4096_and_exact_small_integers():
    N = 4096
    A, B = synth.fp16_normal_clipped(N, N, N, seed=3)
    got = run_f16out(A, B)
    rows, cols = synth.sample_rows_cols(N, N, seed=3)
    ref, S = oracle.gemm_fp16(A, B, rows=rows)
    assert oracle.fp16_out_check(got[rows], ref, S)[0]
    ref, S = oracle.gemm_fp16(A, B, cols=cols)
    assert oracle.fp16_out_check(got[:, cols], ref, S)[0]
    # sums that are small integers are exact in binary16
    a = np.zeros((256, 64), np.float16)
    a[:, 0] = (np.arange(256) % 31) - 15
    b = np.zeros((256, 64), np.float16)
    b[:, 0] = (np.arange(256) % 29) - 14
    want = np.outer(a[:, 0].astype(np.float64), b[:, 0].astype(np.float64))
    assert np.array_equal(run_f16out(a, b).astype(np.float64), want)


def run_dequant(prec, A, B, rs, cs, out_dtype):
    fn = binding.gemm_s8_dequant if prec == "s8" else binding.gemm_s4_dequant
    C = torch.full((A.shape[0], B.shape[0]), float("nan"), dtype=out_dtype, device="cuda")
    fn(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
    torch.cuda.synchronize()
    return C.cpu().numpy()


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.float16])
@pytest.mark.parametrize("prec", ["s8", "s4"])
@pytest.mark.parametrize("M,N,K", [(512, 512, 512), (300, 520, 320), (129, 1030, 4128),
                                   (200, 100, 128), (77, 3, 64)])
def test_dequant_full(prec, M, N, K, out_dtype):
    A, B = synth.make(prec, M, N, K, seed=M + K)
    rs, cs = scales(M, N, seed=N)
    exact = oracle.gemm_s8_i64(A, B) if prec == "s8" else oracle.gemm_s4_i64(A, B, K)
    ref = oracle.dequant_ref(exact, rs, cs)
    ok, worst = oracle.dequant_check(run_dequant(prec, A, B, rs, cs, out_dtype), ref,
                                     out_dtype == torch.float16)
    assert ok, "error %.3g x bound" % worst


@pytest.mark.parametrize("bn,cta_group", [(32, 1)] + SHAPES16)
def test_dequant_every_tile_shape(bn, cta_group):
    M, N, K = 650, 1096, 1184
    A, B = synth.s8_uniform(M, N, K, seed=bn)
    rs, cs = scales(M, N, seed=bn)
    ref = oracle.dequant_ref(oracle.gemm_s8_i64(A, B), rs, cs)
    binding.gemm_set_config_override(bn, 0, cta_group)
    assert oracle.dequant_check(run_dequant("s8", A, B, rs, cs, torch.float32), ref, False)[0]
    if bn >= 64:
        assert oracle.dequant_check(run_dequant("s8", A, B, rs, cs, torch.float16), ref, True)[0]



@pytest.mark.parametrize("bn,cta_group", [(32, 1), (64, 1), (64, 2), (256, 2)])
def test_dequant_many_short_tiles_per_cta(bn, cta_group):
    M, N, K = 1024, 4096, 32
    A, B = synth.s8_uniform(M, N, K, seed=bn)
    rs, cs = scales(M, N, seed=bn)
    ref = oracle.dequant_ref(oracle.gemm_s8_i64(A, B), rs, cs)
    binding.gemm_set_config_override(bn, 0, cta_group, 1)
    for rep in range(2):
        assert oracle.dequant_check(run_dequant("s8", A, B, rs, cs, torch.float32), ref, False)[0]
        if bn >= 64:
            assert oracle.dequant_check(run_dequant("s8", A, B, rs, cs, torch.float16), ref, True)[0]


def test_dequant_with_unit_scales_is_the_exact_integer():
    M, N, K = 384, 640, 256                      # |sum| <= 128*128*256 = 2^22: exact in float32
    A, B = synth.s8_uniform(M, N, K, seed=5)
    ones_r, ones_c = np.ones(M, np.float32), np.ones(N, np.float32)
    got = run_dequant("s8", A, B, ones_r, ones_c, torch.float32)
    assert np.array_equal(got.astype(np.int64), oracle.gemm_s8_i64(A, B))
    # row / column scale really index rows / columns
    rs = np.arange(1, M + 1, dtype=np.float32)
    cs = np.ones(N, np.float32)
    a = np.ones((M, K), np.int8)
    b = np.ones((N, K), np.int8)
    got = run_dequant("s8", a, b, rs, cs, torch.float32)
    assert np.array_equal(got, np.repeat((K * rs)[:, None], N, axis=1))
    got = run_dequant("s8", b, a, cs, rs, torch.float32)
    assert np.array_equal(got, np.repeat((K * rs)[None, :], N, axis=0))


def test_dequant_argument_errors():
    L = binding.lib()
    A = torch.zeros(64, 64, dtype=torch.int8, device="cuda")
    C = torch.zeros(64, 64, dtype=torch.float32, device="cuda")
    sc = torch.ones(64, dtype=torch.float32, device="cuda")
    p, c, s = A.data_ptr(), C.data_ptr(), sc.data_ptr()
    assert L.gemm_s8_dequant(64, 64, 64, p, p, None, s, c, 0, None) == -1
    assert L.gemm_s8_dequant(64, 64, 64, p, p, s, s, c, 2, None) == -1
    assert L.gemm_s8_dequant(64, 64, 64, p, p, s + 2, s, c, 0, None) == -2
    assert L.gemm_s8_dequant(64, 64, 24, p, p, s, s, c, 0, None) == -2
    assert L.gemm_s4_dequant(64, 64, 48, p, p, s, s, c, 0, None) == -2
    assert L.gemm_fp16_f16out(64, 64, 12, p, p, c, None) == -2


# ------------------------------------------------ split-K inside a cluster of two CTAs
def _ctas_of_last_launch():
    return sum(1 for t in binding.gemm_trace_read(160) if t["cycles"] > 0)


@pytest.mark.parametrize("swap", [1, 2])
@pytest.mark.parametrize("M,N,K,bn,tiles", [(16, 2048, 4096, 64, 16), (1, 1030, 2080, 64, 9),
                                            (40, 12800, 1056, 64, 100), (24, 640, 8192, 32, 5)])
def test_cluster_split_k_for_16_bit_and_scaled_outputs(M, N, K, bn, tiles, swap):
    """The outputs that cannot be split through C (binary16, dequantised) split K between the
    two CTAs of a cluster, which exchange partial sums through shared memory: twice as many
    CTAs as tiles work on the problem (checked through the cycle-accounting records), also when
    a cluster has several tiles in a row (100 tiles on 74 clusters) and the hand-over buffer is
    reused."""
    binding.gemm_set_swap_ab(swap)
    try:
        kernel_tiles = tiles if swap == 2 else -(-M // 128) * -(-N // bn)
        binding.gemm_set_config_override(bn, 0, 1, 2)
        g = np.random.Generator(np.random.PCG64(M + N))
        rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
        cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
        A, B = synth.s8_uniform(M, N, K, seed=M)
        ref = oracle.dequant_ref(oracle.gemm_s8_i64(A, B), rs, cs)
        for out_dtype in ((torch.float32, torch.float16) if bn == 64 else (torch.float32,)):
            binding.gemm_trace_enable(1)
            got = run_dequant("s8", A, B, rs, cs, out_dtype)
            ctas = _ctas_of_last_launch()
            binding.gemm_trace_enable(0)
            assert ctas == min(2 * kernel_tiles, 148), (ctas, kernel_tiles)
            ok, worst = oracle.dequant_check(got, ref, out_dtype == torch.float16)
            assert ok, "%s: %.3g x bound" % (out_dtype, worst)
        if bn == 64:
            A, B = synth.fp16_normal_clipped(M, N, K, seed=N)
            ref, S = oracle.gemm_fp16(A, B)
            for rep in range(2):
                ok, worst = oracle.fp16_out_check(run_f16out(A, B), ref, S)
                assert ok, "fp16 out: %.3g x bound" % worst
    finally:
        binding.gemm_set_swap_ab(0)
        binding.gemm_trace_enable(0)


def test_cluster_split_k_is_the_automatic_choice_for_few_rows():
    M, N, K = 16, 4096, 8192                      # 32 kernel tiles for 148 SMs
    A, B = synth.s8_uniform(M, N, K, seed=77)
    g = np.random.Generator(np.random.PCG64(77))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    ref = oracle.dequant_ref(oracle.gemm_s8_i64(A, B), rs, cs)
    binding.gemm_trace_enable(1)
    got = run_dequant("s8", A, B, rs, cs, torch.float16)
    ctas = _ctas_of_last_launch()
    binding.gemm_trace_enable(0)
    assert ctas in (64, 128), ctas              # 32 tiles x 2 or 4 CTAs
    assert oracle.dequant_check(got, ref, True)[0]


@pytest.mark.parametrize("prec", ["s8", "s4", "s4 fused", "fp16"])
@pytest.mark.parametrize("M,N,K", [(16, 1536, 16384),    # 12 tiles x 4 CTAs
                                   (24, 5000, 4128),     # clusters take several tiles in a row
                                   (8, 128, 640)])       # fewer ring slots than would fill the ranks
def test_cluster_split_k_four_ways(prec, M, N, K):
    """Few tiles and a long K: four CTAs of a cluster share a 32-wide tile (exchanged
    operands), ranks 1..3 each hand their partial sums to rank 0 in a buffer of their own."""
    g = np.random.Generator(np.random.PCG64(M + N))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    # packed INT4 through the pre-pass (the INT8 kernel) or expanded inside the kernel
    binding.gemm_set_s4_scheme(2 if prec == "s4 fused" else 1)
    prec = prec.split()[0]
    binding.gemm_set_config_override(32, 0, 1, 4)
    binding.gemm_set_swap_ab(2)
    try:
        if prec == "fp16":
            A, B = synth.fp16_normal_clipped(M, N, K, seed=N)
            ref, S = oracle.gemm_fp16(A, B)
        else:
            A, B = synth.make(prec, M, N, K, seed=M)
            exact = oracle.gemm_s8_i64(A, B) if prec == "s8" else oracle.gemm_s4_i64(A, B, K)
            ref = oracle.dequant_ref(exact, rs, cs)
        for rep in range(2):
            binding.gemm_trace_enable(1)
            if prec == "fp16":
                got = run_f16out(A, B)
            else:
                got = run_dequant(prec, A, B, rs, cs, torch.float16)
            ctas = _ctas_of_last_launch()
            binding.gemm_trace_enable(0)
            if M == 16:
                assert ctas == 48, ctas
            if prec == "fp16":
                ok, worst = oracle.fp16_out_check(got, ref, S)
            else:
                ok, worst = oracle.dequant_check(got, ref, True)
            assert ok, "%s: %.3g x bound" % (prec, worst)
    finally:
        binding.gemm_set_s4_scheme(0)
        binding.gemm_set_swap_ab(0)
        binding.gemm_trace_enable(0)


@pytest.mark.parametrize("scheme", [1, 2])
@pytest.mark.parametrize("M,N,K,bn", [(16, 2048, 4096, 64), (24, 640, 8192, 32), (40, 12800, 1056, 64)])
def test_cluster_split_k_dequantised_int4(M, N, K, bn, scheme):
    """The same for packed INT4 operands, on the pre-pass route (INT8 kernel) and on the fused
    route (nibbles expanded inside the kernel, K divided in whole packed slots)."""
    binding.gemm_set_swap_ab(2)
    binding.gemm_set_s4_scheme(scheme)
    try:
        binding.gemm_set_config_override(bn, 0, 1, 2)
        g = np.random.Generator(np.random.PCG64(M + N))
        rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
        cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
        A, B = synth.s4_uniform(M, N, K, seed=M)
        ref = oracle.dequant_ref(oracle.gemm_s4_i64(A, B, K), rs, cs)
        kernel_tiles = -(-N // 128)
        for out_dtype in ((torch.float32, torch.float16) if bn == 64 else (torch.float32,)):
            binding.gemm_trace_enable(1)
            got = run_dequant("s4", A, B, rs, cs, out_dtype)
            ctas = _ctas_of_last_launch()
            binding.gemm_trace_enable(0)
            assert ctas == min(2 * kernel_tiles, 148), (ctas, kernel_tiles)
            ok, worst = oracle.dequant_check(got, ref, out_dtype == torch.float16)
            assert ok, "%s: %.3g x bound" % (out_dtype, worst)
    finally:
        binding.gemm_set_swap_ab(0)
        binding.gemm_set_s4_scheme(0)
        binding.gemm_trace_enable(0)


def test_cluster_split_k_and_fused_int4_share_the_gpu_from_two_streams():
    """Clusters of four (INT8 dequantised to FP16) and the fused few-row INT4 kernel, enqueued
    alternately on two streams without any synchronisation in between, so that CTAs of both are
    resident at once: every result of both must be right."""
    M, N, K = 16, 4096, 8192
    g = np.random.Generator(np.random.PCG64(5))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-1).astype(np.float32)
    A8, B8 = synth.s8_uniform(M, N, K, seed=51)
    A4, B4 = synth.s4_uniform(M, N, K, seed=52)
    ref8 = oracle.dequant_ref(oracle.gemm_s8_i64(A8, B8), rs, cs)
    ref4 = oracle.gemm_s4(A4, B4, K)
    dA8, dB8, dA4, dB4, d_rs, d_cs = (to_dev(x) for x in (A8, B8, A4, B4, rs, cs))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs8, outs4 = [], []
    for rep in range(12):
        C8 = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
        C4 = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
        s1.wait_stream(torch.cuda.current_stream())
        s2.wait_stream(torch.cuda.current_stream())
        binding.gemm_s8_dequant(dA8, dB8, d_rs, d_cs, C8, torch.float16, stream=s1)
        binding.gemm_s4(dA4, dB4, C4, stream=s2)
        outs8.append(C8)
        outs4.append(C4)
    s1.synchronize()
    s2.synchronize()
    for C8, C4 in zip(outs8, outs4):
        assert oracle.dequant_check(C8.cpu().numpy(), ref8, True)[0]
        assert np.array_equal(C4.cpu().numpy(), ref4)


@pytest.mark.parametrize("prec", ["fp16", "s8"])
@pytest.mark.parametrize("cta_group", [1, 2])
def test_sector_store_epilogue_switch_gives_the_same_results(prec, cta_group):
    """Measurement switch 64: accumulators read in the 16x256b shape and stored as whole 32-byte
    sectors, no staging.  Ragged in M, N a multiple of 8 (rows of whole sectors), several tiles."""
    M, N, K = 700, 1032, 512
    A, B = synth.make(prec, M, N, K, seed=5)
    binding.gemm_set_config_override(256, 0, cta_group, 1)
    try:
        binding.gemm_trace_enable(64)
        C = torch.full((M, N), -7, dtype=torch.float32 if prec == "fp16" else torch.int32, device="cuda")
        binding.gemm(prec, to_dev(A), to_dev(B), C)
        torch.cuda.synchronize()
    finally:
        binding.gemm_trace_enable(0)
    got = C.cpu().numpy()
    if prec == "s8":
        assert np.array_equal(got, oracle.gemm_s8(A, B))
    else:
        ref, S = oracle.gemm_fp16(A, B)
        assert oracle.fp16_check(got, ref, S)[0]
