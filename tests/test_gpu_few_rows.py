"""GPU parity of the kernel for problems with a few rows on one side (the long operand goes
from global memory into warp-level MMA fragments; no tile, no split-K through C) against the
oracle: every precision, either operand as the short one, every output mode,
ragged sizes, many row blocks per CTA, and bit-equality with the tile kernels.
gemm_set_kernel_family(3) takes the kernel wherever it exists (a short side of up to 32 rows),
family 1 never."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _few_rows_route():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_kernel_family(3)
    yield
    binding.gemm_set_kernel_family(0)
    assert binding.gemm_last_device_status() == 0


def _make(prec, M, N, K, seed):
    return synth.s4_uniform(M, N, K, seed=seed) if prec == "s4" else synth.make(prec, M, N, K, seed=seed)


# short side 1..32 (one, two and four groups of eight rows; 3, 12, 20 leave a group partly
# filled), the long side ragged against the 16- and 32-row blocks, K from a single 16-byte piece
# per row (32 packed values) over ragged steps (96, 160, 1056, 4128) to many steps per warp
SHAPES = [(1, 1, 32), (1, 777, 512), (3, 100, 96), (8, 1000, 4128), (9, 530, 160), (12, 2049, 1056),
          (16, 4100, 2048), (16, 31, 64), (20, 600, 1056), (32, 1500, 512),
          (777, 1, 512), (1000, 8, 4128), (2049, 12, 1056), (530, 16, 160), (600, 29, 96),
          # few row blocks against a long K: sixteen warps per CTA (eight with 17-32 short rows,
          # whose sums take the room of a ring slot)
          (20, 2048, 8192), (32, 1024, 16384), (16, 2000, 8192), (5, 1500, 16384)]


@pytest.mark.parametrize("prec", ["fp16", "s8", "s4"])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_few_rows_full_compare(prec, M, N, K):
    assert binding.gemm_query_config(prec, M, N, K).startswith("few_rows")
    A, B = _make(prec, M, N, K, seed=M + N + K)
    for rep in range(2):
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        check_against_oracle(prec, A, B, C, force_full=True)


@pytest.mark.parametrize("prec", ["fp16", "s8", "s4"])
@pytest.mark.parametrize("M,N,K", [(8, 80000, 1056), (16, 160001, 256), (5, 200000, 64), (160000, 16, 512)])
def test_few_rows_more_row_blocks_than_ctas(prec, M, N, K):
    """More row blocks than CTAs fit the SMs: a CTA walks several, its copies running ahead
    across the block boundaries."""
    cfg = binding.gemm_query_config(prec, M, N, K)
    ctas = int(cfg.split("ctas=")[1].split()[0])
    blocks = int(cfg.split("blocks=")[1].split()[0])
    assert cfg.startswith("few_rows") and ctas < blocks
    A, B = _make(prec, M, N, K, seed=N)
    check_against_oracle(prec, A, B, run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7))


@pytest.mark.parametrize("prec", ["s8", "s4"])
def test_few_rows_equals_the_tile_kernels(prec):
    for M, N, K in [(16, 3000, 4128), (7, 2500, 1056), (1500, 11, 2048)]:
        A, B = _make(prec, M, N, K, seed=K)
        got = run_gpu(prec, A, B, fill=-7)
        binding.gemm_set_kernel_family(1)
        assert not binding.gemm_query_config(prec, M, N, K).startswith("few_rows")
        tiles = run_gpu(prec, A, B, fill=-7)
        binding.gemm_set_kernel_family(3)
        assert np.array_equal(got, tiles)


def test_few_rows_extreme_values_at_the_longest_k():
    """-8 x -8 over K = 131040 (the scaled products reach 16384 K = 2^31 - 524288 summed over the
    warps of a CTA: each warp's partial sum is brought back to scale before they are added), and
    -128 x -128 in INT8."""
    M, N, K = 2, 40, 131040
    A = np.full((M, K // 2), 0x88, dtype=np.uint8)
    B = np.full((N, K // 2), 0x88, dtype=np.uint8)
    assert np.all(run_gpu("s4", A, B, fill=-7) == 64 * K)
    A8 = np.full((M, K), -128, dtype=np.int8)
    B8 = np.full((N, K), -128, dtype=np.int8)
    assert np.all(run_gpu("s8", A8, B8, fill=-7) == 16384 * K)


def test_few_rows_one_hot_positions():
    """Rows with a single non-zero value at every position of a 64-byte step: the order of K
    inside the fragments must be the same on both sides."""
    M, N, K = 16, 256, 512
    vals_a = np.zeros((M, K), dtype=np.int8)
    vals_b = np.zeros((N, K), dtype=np.int8)
    for i in range(M):
        vals_a[i, (37 * i) % K] = 1 + (i % 7)
        vals_a[i, (37 * i + 129) % K] = -8
    for j in range(N):
        vals_b[j, j % K] = -3
        vals_b[j, (j + 129) % K] = 7
        if vals_b[j, (2 * j + 1) % K] == 0:
            vals_b[j, (2 * j + 1) % K] = 2
    A, B = synth.pack_s4(vals_a), synth.pack_s4(vals_b)
    assert np.array_equal(run_gpu("s4", A, B, fill=-7), oracle.gemm_s4(A, B, K))
    assert np.array_equal(run_gpu("s8", vals_a, vals_b, fill=-7), oracle.gemm_s8(vals_a, vals_b))


@pytest.mark.parametrize("prec", ["s8", "s4"])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.float16])
@pytest.mark.parametrize("M,N,K", [(12, 1300, 1056), (900, 5, 512)])
def test_few_rows_dequantised_outputs(prec, out_dtype, M, N, K):
    A, B = _make(prec, M, N, K, seed=8)
    g = np.random.Generator(np.random.PCG64(8))
    rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
    cs = (g.uniform(0.5, 2.0, N) * 1e-2).astype(np.float32)
    C = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    fn = binding.gemm_s4_dequant if prec == "s4" else binding.gemm_s8_dequant
    fn(to_dev(A), to_dev(B), to_dev(rs), to_dev(cs), C, out_dtype)
    torch.cuda.synchronize()
    acc = oracle.gemm_s4_i64(A, B, K) if prec == "s4" else oracle.gemm_s8(A, B).astype(np.int64)
    ok, worst = oracle.dequant_check(C.cpu().numpy(), oracle.dequant_ref(acc, rs, cs),
                                     out_dtype == torch.float16)
    assert ok, worst


def test_few_rows_fp16_output_and_special_values():
    """FP16 result rounded once from the FP32 sums; infinities and NaNs of the operands reach
    the rows and columns they belong to and no others."""
    M, N, K = 12, 1300, 1056
    A, B = synth.fp16_normal_clipped(M, N, K, seed=3)
    ref, S = oracle.gemm_fp16(A, B)
    C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    binding.gemm_fp16_f16out(to_dev(A), to_dev(B), C)
    torch.cuda.synchronize()
    ok, worst = oracle.fp16_out_check(C.cpu().numpy(), ref, S)
    assert ok, "fp16 out: %.3g x bound" % worst
    A = A.copy()
    B = B.copy()
    A[3, 700] = np.float16(np.inf)
    B[77, 5] = np.float16(np.nan)
    got = run_gpu("fp16", A, B, fill=0.0)
    assert np.all(np.isnan(got[:, 77])) and np.all(np.isinf(got[3, :77]) | np.isnan(got[3, :77]))
    clean = np.ones((M, N), dtype=bool)
    clean[3, :] = False
    clean[:, 77] = False
    assert np.all(np.isfinite(got[clean]))


def test_few_rows_automatic_rule():
    binding.gemm_set_kernel_family(0)
    few = lambda prec, M, N, K: binding.gemm_query_config(prec, M, N, K).startswith("few_rows")
    assert few("s4", 16, 8192, 8192) and few("s4", 1, 28672, 8192) and few("s4", 4096, 9, 1024)
    assert few("s4", 17, 8192, 8192) and few("s4", 32, 4096, 4096)       # 17-32 rows: up to 8192
    assert not few("s4", 17, 16384, 8192) and not few("s4", 33, 8192, 8192) and not few("s4", 16, 500, 8192)
    assert few("s8", 8, 2048, 4096) and few("s8", 16, 4096, 8192) and few("s8", 16, 8192, 8192)
    assert few("s4", 16, 512, 8192)
    assert few("s8", 8, 28672, 8192)
    assert not few("s8", 16, 12288, 8192) and not few("s8", 17, 2048, 4096)
    assert few("fp16", 1, 4096, 8192) and few("fp16", 16, 8192, 4096) and few("fp16", 3000, 7, 512)
    assert not few("fp16", 16, 8192, 8192) and not few("fp16", 17, 4096, 4096)
    assert not few("fp16", 16, 1024, 8192) and not few("s8", 16, 512, 8192)   # few blocks, long rows
    binding.gemm_set_s4_scheme(2)          # a forced INT4 scheme means the tile kernels
    assert not few("s4", 16, 8192, 8192)
    binding.gemm_set_s4_scheme(0)
    M, N, K = 16, 4096, 1056
    A, B = synth.s4_uniform(M, N, K, seed=2)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7))


def test_few_rows_in_a_cuda_graph():
    """No scratch, no zeroing launch: a captured call is one kernel node and replays exactly."""
    M, N, K = 16, 2100, 2048
    A, B = synth.s4_uniform(M, N, K, seed=5)
    dA, dB = to_dev(A), to_dev(B)
    C = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.gemm_s4(dA, dB, C, stream=side)
    ref = oracle.gemm_s4(A, B, K)
    for rep in range(3):
        C.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(C.cpu().numpy(), ref)


def test_few_rows_seeded_walk_of_shapes():
    """Random short sides (1..32), long sides, K and orientations through every launch shape the
    host picks (warps 1..16, ring depths 2..8),
    each checked against the oracle on sampled rows."""
    g = np.random.Generator(np.random.PCG64(4321))
    shapes_met = set()
    cases = 0
    while cases < 80:
        M = int(g.integers(1, 33))
        kind = int(g.integers(4))
        N = (int(g.integers(1, 600)) if kind == 0 else int(g.integers(600, 9000)) if kind == 1
             else int(g.integers(9000, 40000)) if kind == 2 else int(g.choice([512, 2048, 4096, 8192])))
        K = (int(g.integers(1, 40)) * 32 if g.integers(3) == 0 else int(g.integers(1, 300)) * 32
             if g.integers(2) == 0 else int(g.choice([4096, 8192, 16384, 32768])))
        prec = str(g.choice(["fp16", "s8", "s4"]))
        if (M + N) * K > 150e6:
            continue
        if g.integers(3) == 0:
            M, N = N, M
        cases += 1
        cfg = binding.gemm_query_config(prec, M, N, K)
        assert cfg.startswith("few_rows"), cfg
        shapes_met.add(tuple(cfg.split(k)[1].split()[0] for k in ("warps=", "depth=")))
        A, B = synth.make(prec, M, N, K, seed=int(g.integers(1 << 30)))
        rows = np.unique(np.concatenate([g.choice(M, size=min(10, M), replace=False), [0, M - 1]])).astype(np.int32)
        got = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)[rows]
        what = "%s %d x %d x %d: %s" % (prec, M, N, K, cfg)
        if prec == "fp16":
            ref, S = oracle.gemm_fp16(A, B, rows=rows)
            assert oracle.fp16_check(got, ref, S)[0], what
        else:
            exact = oracle.gemm_s8_i64(A, B, rows=rows) if prec == "s8" else oracle.gemm_s4_i64(A, B, K, rows=rows)
            assert np.array_equal(got.astype(np.int64), exact), what
    assert len(shapes_met) >= 10, shapes_met


def test_few_rows_operands_written_by_the_launch_in_front():
    """The kernel may start while the kernel in front of it in the stream still runs and must read
    nothing before that one has finished: operands and scale factors rewritten right in front of
    every call (a device-to-device copy kernel, then the GEMM, no synchronisation in between), the
    result of every call checked afterwards.  (Loads through the non-coherent path were once
    placed above the wait for the grid in front and read the values of the call before.)"""
    M, N, K = 8, 4096, 2048
    rounds = 6
    g = np.random.Generator(np.random.PCG64(11))
    for prec in ("s8", "s4", "fp16"):
        data = [_make(prec, M, N, K, seed=100 + r) for r in range(rounds)]
        src = [(to_dev(A), to_dev(B)) for A, B in data]
        dA, dB = torch.empty_like(src[0][0]), torch.empty_like(src[0][1])
        outs = [torch.empty((M, N), dtype=torch.float32 if prec == "fp16" else torch.int32, device="cuda")
                for _ in range(rounds)]
        for rep in range(3):
            for r in range(rounds):
                dA.copy_(src[r][0])
                dB.copy_(src[r][1])
                binding.gemm(prec, dA, dB, outs[r])
            torch.cuda.synchronize()
            for r in range(rounds):
                check_against_oracle(prec, data[r][0], data[r][1], outs[r].cpu().numpy(), force_full=(rep == 0 and r < 2))
    # scale factors written in front of a dequantising call
    A, B = _make("s8", M, N, K, seed=7)
    dA, dB = to_dev(A), to_dev(B)
    acc = oracle.gemm_s8(A, B).astype(np.int64)
    rs_d, cs_d = torch.empty(M, device="cuda"), torch.empty(N, device="cuda")
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    for r in range(rounds):
        rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
        cs = (g.uniform(0.5, 2.0, N) * 1e-2).astype(np.float32)
        rs_src, cs_src = to_dev(rs), to_dev(cs)
        rs_d.copy_(rs_src)
        cs_d.copy_(cs_src)
        binding.gemm_s8_dequant(dA, dB, rs_d, cs_d, C, torch.float32)
        torch.cuda.synchronize()
        ok, worst = oracle.dequant_check(C.cpu().numpy(), oracle.dequant_ref(acc, rs, cs), False)
        assert ok, worst
