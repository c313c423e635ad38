"""GPU parity of the hybrid fused INT4 route -- B packed and expanded inside the GEMM kernel, A as
an int8 image made by a small kernel in front -- against the oracle, and bit-equality with the
form that keeps both operands packed.  Scheme 6 forces the hybrid form wherever it exists (the
CTA-pair tiles in plain operand order), scheme 5 forbids it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _hybrid_route():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(6)
    yield
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_config_override(0, 0, 0, 0)
    assert binding.gemm_last_device_status() == 0


# K = 32: a single 16-byte chunk per row (the image's row is padded to 256); 96/160: partly
# filled packed slots; 1056, 4128: ragged tails; M, N not tile multiples; several tiles per CTA
@pytest.mark.parametrize("M,N,K", [(256, 256, 32), (130, 70, 96), (300, 500, 160), (512, 768, 512),
                                   (640, 1100, 1056), (1, 8, 64), (1000, 1000, 4128),
                                   (700, 5000, 256)])
@pytest.mark.parametrize("bn", [256, 128])
def test_hybrid_full_compare(M, N, K, bn):
    binding.gemm_set_config_override(bn, 0, 2, 1)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "fused_unpack" in cfg and "a=int8_image" in cfg
    A, B = synth.s4_uniform(M, N, K, seed=M + K)
    for rep in range(2):
        check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


@pytest.mark.parametrize("split_k", [2, 3])
@pytest.mark.parametrize("M,N,K", [(300, 520, 2048), (512, 512, 4128)])
def test_hybrid_with_k_split_through_c(M, N, K, split_k):
    """Each unit fetches the atoms of the A image that belong to its own K range."""
    binding.gemm_set_config_override(256, 0, 2, split_k)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "a=int8_image" in cfg and ("split_k=%d" % split_k) in cfg
    A, B = synth.s4_uniform(M, N, K, seed=split_k)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


def test_hybrid_equals_the_form_with_both_operands_packed_and_the_prepass():
    M, N, K = 900, 2100, 1056
    A, B = synth.s4_uniform(M, N, K, seed=3)
    binding.gemm_set_config_override(256, 0, 2, 1)
    got = run_gpu("s4", A, B, fill=-7)
    check_against_oracle("s4", A, B, got, force_full=True)
    for scheme in (5, 1):
        binding.gemm_set_s4_scheme(scheme)
        cfg = binding.gemm_query_config("s4", M, N, K)
        assert "a=int8_image" not in cfg
        assert np.array_equal(got, run_gpu("s4", A, B, fill=-7))


def test_hybrid_extreme_values_and_one_hot_positions():
    """-8 x -8 over a ragged K (every product 64, the image holds -128 everywhere), and one-hot
    rows whose single 1 sits at every position of a packed slot: the order of K inside the image
    must be the order the expansion warps give B."""
    M, N, K = 256, 256, 544
    binding.gemm_set_config_override(256, 0, 2, 1)
    A = np.full((M, K // 2), 0x88, dtype=np.uint8)
    B = np.full((N, K // 2), 0x88, dtype=np.uint8)
    C = run_gpu("s4", A, B, fill=-7)
    assert np.all(C == 64 * K)
    K = 512
    vals_a = np.zeros((M, K), dtype=np.int8)
    vals_b = np.zeros((N, K), dtype=np.int8)
    for i in range(M):
        vals_a[i, i % K] = 1 + (i % 7)
        vals_a[i, (i + 256) % K] = -8
    for j in range(N):
        vals_b[j, j % K] = -3
        vals_b[j, (j + 256) % K] = 7
    A, B = synth.pack_s4(vals_a), synth.pack_s4(vals_b)
    C = run_gpu("s4", A, B, fill=-7)
    assert np.array_equal(C, oracle.gemm_s4(A, B, K))


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.float16])
def test_hybrid_dequantised_outputs(out_dtype):
    M, N, K = 520, 1300, 1056
    binding.gemm_set_config_override(256, 0, 2, 1)
    A, B = synth.s4_uniform(M, N, K, seed=8)
    g = np.random.Generator(np.random.PCG64(8))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-2).astype(np.float32)
    C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    binding.gemm_s4_dequant(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
    torch.cuda.synchronize()
    ref = oracle.dequant_ref(oracle.gemm_s4_i64(A, B, K), rs, cs)
    ok, worst = oracle.dequant_check(C.cpu().numpy(), ref, out_dtype == torch.float16)
    assert ok, worst


def test_hybrid_in_a_cuda_graph_and_on_two_streams():
    """The image lives in pooled scratch: replays of a captured call, eager calls of another
    shape in between, and a second stream with its own buffer all stay exact."""
    binding.gemm_set_config_override(256, 0, 2, 1)
    shapes = [(300, 800, 1056), (600, 520, 2048)]
    data = [synth.s4_uniform(M, N, K, seed=M) for M, N, K in shapes]
    dev = [(to_dev(A), to_dev(B)) for A, B in data]
    outs = [torch.full((M, N), -7, dtype=torch.int32, device="cuda") for M, N, K in shapes]
    ref = [oracle.gemm_s4(A, B, K) for (A, B), (M, N, K) in zip(data, shapes)]
    binding.gemm_s4(dev[0][0], dev[0][1], outs[0])      # first use outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.gemm_s4(dev[0][0], dev[0][1], outs[0], stream=side)
    for rep in range(3):
        outs[0].fill_(-7)
        g.replay()
        binding.gemm_s4(dev[1][0], dev[1][1], outs[1])
        torch.cuda.synchronize()
        assert np.array_equal(outs[0].cpu().numpy(), ref[0])
        assert np.array_equal(outs[1].cpu().numpy(), ref[1])


def test_automatic_rule_takes_the_hybrid_form_for_a_short_m_against_a_large_n_k():
    binding.gemm_set_s4_scheme(0)
    assert "a=int8_image" in binding.gemm_query_config("s4", 256, 28672, 8192)
    assert "a=int8_image" in binding.gemm_query_config("s4", 512, 28672, 8192)
    assert "a=int8_image" in binding.gemm_query_config("s4", 1024, 8192, 8192)
    assert "a=int8_image" in binding.gemm_query_config("s4", 8192, 8192, 8192)
    assert "a=int8_image" not in binding.gemm_query_config("s4", 8192, 2048, 8192)   # a tall A, few tile columns
    assert "a=int8_image" not in binding.gemm_query_config("s4", 4096, 4096, 4096)
    assert "a=int8_image" not in binding.gemm_query_config("s4", 256, 8192, 8192)
    assert "a=int8_image" not in binding.gemm_query_config("s4", 2048, 2048, 2048)
    assert "a=int8_image" not in binding.gemm_query_config("s4", 16, 8192, 8192)   # exchanged operands
    M, N, K = 256, 28672, 1056          # the rule's shape in M and N, a short K to keep the oracle quick
    binding.gemm_set_s4_scheme(6)
    A, B = synth.s4_uniform(M, N, K, seed=2)
    C = run_gpu("s4", A, B, fill=-7)
    check_against_oracle("s4", A, B, C)


def test_hybrid_captured_without_an_earlier_call_falls_back_to_the_form_without_scratch():
    """Nothing can be allocated while a stream is captured: with no pooled buffer from an earlier
    call the captured call keeps both operands packed (no scratch at all) and is still exact."""
    binding.gemm_release_workspaces()
    binding.gemm_set_config_override(256, 0, 2, 1)
    M, N, K = 300, 900, 1056
    A, B = synth.s4_uniform(M, N, K, seed=21)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.gemm_s4(dA, dB, C, stream=side)
    assert binding.gemm_debug_counters()["pool_buffers"] == 0
    g.replay()
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s4(A, B, K))


def test_hybrid_long_k_many_laps_of_the_rings():
    """K = 65568: 257 packed slots per tile, i.e. dozens of laps of the A ring, the packed ring and
    the int8 ring, ending in a partly filled slot."""
    M, N, K = 200, 520, 65568
    binding.gemm_set_config_override(256, 0, 2, 1)
    assert "a=int8_image" in binding.gemm_query_config("s4", M, N, K)
    A, B = synth.s4_uniform(M, N, K, seed=65)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)
