"""GPU parity of the overlapped INT4 pre-pass (gemm_set_s4_scheme(4), a measured alternative to
the separate pre-pass launch): four extra warps per CTA of the INT8 kernel expand the packed
operands into the int8 scratch, chunk by chunk, just ahead of the tiles that read them (ready flags,
dynamic claims, an epoch per call).  Everything through the C-ABI (gemm_s4 / gemm_s4_dequant)
against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, freivalds, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _clean_state():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(4)
    binding.gemm_set_swap_ab(0)
    binding.gemm_set_kernel_family(0)
    yield
    binding.gemm_set_s4_scheme(0)
    assert binding.gemm_last_device_status() == 0


def run_s4(A, B, stream=None, fill=-7):
    C = torch.full((A.shape[0], B.shape[0]), fill, dtype=torch.int32, device="cuda")
    binding.gemm_s4(to_dev(A), to_dev(B), C, stream=stream)
    return C


def test_config_s4_4096_runs_overlapped_and_is_exact():
    N = 4096
    A, B = synth.s4_uniform(N, N, N, seed=2)
    C = run_s4(A, B)
    assert binding.gemm_debug_counters()["s4_overlapped"] == 1
    torch.cuda.synchronize()
    got = C.cpu().numpy()
    check_against_oracle("s4", A, B, got, seed=2)
    freivalds("s4", A, B, got, seed=2)


# ragged rows and columns, K that ends inside a 512-column chunk, K shorter than one chunk,
# a long K with few tiles per CTA pair
@pytest.mark.parametrize("M,N,K", [(3000, 3400, 1056), (2400, 4700, 8224), (5000, 2500, 96),
                                   (2304, 4224, 16416), (4097, 4095, 544)])
def test_overlapped_shapes_match_the_oracle(M, N, K):
    A, B = synth.s4_uniform(M, N, K, seed=M + K)
    C = run_s4(A, B)
    if K >= 512:     # (with a single k-block per tile the selector prefers narrower tiles)
        assert binding.gemm_debug_counters()["s4_overlapped"] == 1, "expected the overlapped route"
    torch.cuda.synchronize()
    got = C.cpu().numpy()
    check_against_oracle("s4", A, B, got, seed=K)
    freivalds("s4", A, B, got, seed=K, vectors=3)


def test_back_to_back_calls_of_different_shapes_share_the_scratch():
    """Each call works under a new epoch: flags and int8 rows that an earlier, differently
    shaped call left in the buffer must never be taken for this call's."""
    shapes = [(4096, 4096, 2048, 1), (3000, 5000, 1024, 2), (4096, 4096, 2048, 3), (2560, 3840, 4096, 4)]
    ops = [(M, N, K, synth.s4_uniform(M, N, K, seed)) for M, N, K, seed in shapes]
    dev = [(to_dev(a), to_dev(b)) for _, _, _, (a, b) in ops]
    outs = [torch.full((M, N), -7, dtype=torch.int32, device="cuda") for M, N, K, _ in ops]
    for rep in range(2):
        for (dA, dB), C in zip(dev, outs):
            binding.gemm_s4(dA, dB, C)          # no synchronisation in between
    torch.cuda.synchronize()
    assert binding.gemm_debug_counters()["pool_buffers"] >= 1
    for (M, N, K, (A, B)), C in zip(ops, outs):
        rows = np.array([0, 1, 31, 32, 255, 256, M // 2, M - 1], dtype=np.int32)
        assert np.array_equal(C.cpu().numpy()[rows], oracle.gemm_s4(A, B, K, rows=rows)), (M, N, K)


def test_replayed_graph_and_eager_calls_interleaved():
    """A captured call bakes no epoch in: the kernel reads it from the buffer, so replays give
    the right answer every time, also with eager calls in between."""
    M, N, K = 4096, 4096, 1024
    A, B = synth.s4_uniform(M, N, K, seed=77)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        binding.gemm_s4(dA, dB, C, stream=side)          # allocates this stream's scratch
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.gemm_s4(dA, dB, C, stream=side)
            binding.gemm_s4(dA, dB, C, stream=side)
    want = oracle.gemm_s4(A, B, K, rows=np.arange(0, M, 97, dtype=np.int32))
    for rep in range(3):
        C.zero_()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy()[::97], want), "replay %d" % rep
        with torch.cuda.stream(side):
            binding.gemm_s4(dA, dB, C, stream=side)
        side.synchronize()
        assert np.array_equal(C.cpu().numpy()[::97], want), "eager call after replay %d" % rep


def test_two_streams_get_scratch_of_their_own():
    M, N, K = 4096, 4096, 1024
    A1, B1 = synth.s4_uniform(M, N, K, seed=5)
    A2, B2 = synth.s4_uniform(M, N, K, seed=6)
    d = [to_dev(x) for x in (A1, B1, A2, B2)]
    C1 = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    C2 = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for rep in range(3):
        binding.gemm_s4(d[0], d[1], C1, stream=s1)
        binding.gemm_s4(d[2], d[3], C2, stream=s2)
    torch.cuda.synchronize()
    assert binding.gemm_debug_counters()["pool_buffers"] >= 2
    rows = np.arange(0, M, 131, dtype=np.int32)
    assert np.array_equal(C1.cpu().numpy()[rows], oracle.gemm_s4(A1, B1, K, rows=rows))
    assert np.array_equal(C2.cpu().numpy()[rows], oracle.gemm_s4(A2, B2, K, rows=rows))


def test_separate_prepass_launch_gives_the_same_bits():
    M, N, K = 3072, 4096, 2048
    A, B = synth.s4_uniform(M, N, K, seed=9)
    over = run_s4(A, B)
    assert binding.gemm_debug_counters()["s4_overlapped"] == 1
    binding.gemm_set_s4_scheme(1)
    plain = run_s4(A, B)
    assert binding.gemm_debug_counters()["s4_overlapped"] == 0
    torch.cuda.synchronize()
    assert torch.equal(over, plain)
    rows = np.arange(0, M, 61, dtype=np.int32)
    assert np.array_equal(over.cpu().numpy()[rows], oracle.gemm_s4(A, B, K, rows=rows))


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.float16])
def test_overlapped_dequant(out_dtype):
    M, N, K = 2600, 3900, 1120
    A, B = synth.s4_uniform(M, N, K, seed=21)
    g = np.random.Generator(np.random.PCG64(21))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * g.choice([-1.0, 1.0], N) * 1e-1).astype(np.float32)
    C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    binding.gemm_s4_dequant(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
    assert binding.gemm_debug_counters()["s4_overlapped"] == 1
    torch.cuda.synchronize()
    rows = np.arange(0, M, 13, dtype=np.int32)
    ref = oracle.dequant_ref(oracle.gemm_s4_i64(A, B, K, rows=rows), rs[rows], cs)
    ok, worst = oracle.dequant_check(C.cpu().numpy()[rows], ref, out_dtype == torch.float16)
    assert ok, "error %.3g x bound" % worst

