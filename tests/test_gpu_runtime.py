"""GPU checks of the host-side runtime behind the entry points: the per-thread tensor-map cache,
the stream-ordered status read-back, calls from several host threads at once, and the scratch
pool's behaviour across streams (all through the C-ABI; results against the oracle)."""
import threading

import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import to_dev

pytestmark = pytest.mark.gpu


def test_repeated_calls_on_the_same_buffers_encode_no_new_tensor_maps():
    M, N, K = 640, 768, 512
    A, B = synth.s8_uniform(M, N, K, seed=1)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.empty((M, N), dtype=torch.int32, device="cuda")
    binding.gemm_s8(dA, dB, C)
    before = binding.gemm_debug_counters()["map_encodes"]
    for _ in range(20):
        binding.gemm_s8(dA, dB, C)
    assert binding.gemm_debug_counters()["map_encodes"] == before
    C2 = torch.empty((M, N), dtype=torch.int32, device="cuda")     # another C: one new map (C's)
    binding.gemm_s8(dA, dB, C2)
    assert 1 <= binding.gemm_debug_counters()["map_encodes"] - before <= 3
    torch.cuda.synchronize()
    want = oracle.gemm_s8(A, B)
    assert np.array_equal(C.cpu().numpy(), want) and np.array_equal(C2.cpu().numpy(), want)


def test_a_cached_map_is_not_reused_for_a_different_shape_at_the_same_address():
    buf = torch.zeros(1 << 20, dtype=torch.int8, device="cuda")
    g = np.random.Generator(np.random.PCG64(3))
    for (M, N, K) in [(256, 128, 1024), (128, 256, 1024), (256, 128, 512), (64, 512, 256)]:
        A = g.integers(-128, 128, size=(M, K), dtype=np.int8)
        B = g.integers(-128, 128, size=(N, K), dtype=np.int8)
        dA = buf[: M * K].view(M, K)
        dB = buf[M * K: M * K + N * K].view(N, K)        # same base addresses, new extents
        dA.copy_(torch.from_numpy(A)); dB.copy_(torch.from_numpy(B))
        C = binding.gemm_s8(dA, dB)
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B)), (M, N, K)


def test_status_word_can_be_read_in_stream_order():
    M, N, K = 512, 512, 256
    A, B = synth.fp16_uniform(M, N, K, seed=2)
    dA, dB = to_dev(A), to_dev(B)
    s = torch.cuda.Stream()
    word = torch.full((1,), 77, dtype=torch.int32).pin_memory()
    with torch.cuda.stream(s):
        C = binding.gemm_fp16(dA, dB, stream=s)
        binding.gemm_read_device_status(word, stream=s)
    s.synchronize()
    assert int(word[0]) == 0
    ref, S = oracle.gemm_fp16(A, B)
    assert oracle.fp16_check(C.cpu().numpy(), ref, S)[0]


def test_calls_from_several_host_threads_on_their_own_streams():
    """No global lock on the call path; each thread's INT4 calls lease scratch for its stream."""
    shapes = [(1536, 1280, 1024), (1280, 1792, 512), (2048, 1024, 2048), (1100, 1300, 768)]
    results, errors = {}, []

    def worker(idx):
        try:
            torch.cuda.set_device(0)
            M, N, K = shapes[idx]
            A, B = synth.s4_uniform(M, N, K, seed=100 + idx)
            A8, B8 = synth.s8_uniform(M, N, K, seed=200 + idx)
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                dA, dB, dA8, dB8 = to_dev(A), to_dev(B), to_dev(A8), to_dev(B8)
                outs = []
                for rep in range(6):
                    outs.append((binding.gemm_s4(dA, dB, stream=s), binding.gemm_s8(dA8, dB8, stream=s)))
            s.synchronize()
            results[idx] = (A, B, A8, B8, K, [(a.cpu().numpy(), b.cpu().numpy()) for a, b in outs])
        except Exception as e:            # surfaced by the main thread
            errors.append((idx, repr(e)))

    binding.gemm_set_s4_scheme(1)          # the route with scratch
    try:
        threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(shapes))]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
    finally:
        binding.gemm_set_s4_scheme(0)
    assert not errors, errors
    for idx, (A, B, A8, B8, K, outs) in results.items():
        want4, want8 = oracle.gemm_s4(A, B, K), oracle.gemm_s8(A8, B8)
        for got4, got8 in outs:
            assert np.array_equal(got4, want4) and np.array_equal(got8, want8), idx
    assert binding.gemm_debug_counters()["pool_buffers"] >= 2
    assert binding.gemm_last_device_status() == 0


def test_release_workspaces_empties_the_pool_and_calls_still_work():
    M, N, K = 1536, 1536, 512
    A, B = synth.s4_uniform(M, N, K, seed=8)
    dA, dB = to_dev(A), to_dev(B)
    binding.gemm_set_s4_scheme(1)
    try:
        binding.gemm_s4(dA, dB)
        assert binding.gemm_debug_counters()["pool_buffers"] >= 1
        binding.gemm_release_workspaces()
        assert binding.gemm_debug_counters()["pool_buffers"] == 0
        C = binding.gemm_s4(dA, dB)
        torch.cuda.synchronize()
    finally:
        binding.gemm_set_s4_scheme(0)
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s4(A, B, K))


def test_host_cost_probe_runs_real_calls_and_rejects_bad_arguments():
    """gemm_debug_host_cost loops the product entry point: C holds the result afterwards, the
    figure is a plausible enqueue time, and counts outside 1..512 are refused."""
    M, N, K = 256, 384, 512
    A, B = synth.make("s8", M, N, K, seed=11)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    C = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    ns = binding.gemm_debug_host_cost("s8", dA, dB, C, calls=50)
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B))
    assert 200.0 < ns < 200000.0
    for calls in (0, 513):
        with pytest.raises(binding.GemmError) as e:
            binding.gemm_debug_host_cost("s8", dA, dB, C, calls=calls)
        assert e.value.code == -1


def test_read_probe_reads_and_writes_nothing():
    """The read-only probe takes any 16-byte multiple, leaves the data and the status word alone,
    and rejects sizes and addresses that are not 16-byte multiples."""
    data = torch.arange(1 << 20, dtype=torch.int32, device="cuda")
    before = data.clone()
    for n in (4, 4 * 37, 1 << 20):
        binding.gemm_debug_read_probe(data[:n])
    torch.cuda.synchronize()
    assert torch.equal(data, before) and binding.gemm_last_device_status() == 0
    with pytest.raises(binding.GemmError):
        binding.gemm_debug_read_probe(data[:3])
    with pytest.raises(binding.GemmError):
        binding.gemm_debug_read_probe(data[1:5])


def test_reset_l2_is_harmless_between_calls():
    A, B = synth.make("s8", 300, 500, 512, seed=4)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.empty((300, 500), dtype=torch.int32, device="cuda")
    binding.gemm_s8(dA, dB, C)
    binding.gemm_debug_reset_l2()
    binding.gemm_s8(dA, dB, C)
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s8(A, B))
