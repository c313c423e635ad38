"""GPU parity: the CUDA library, called through its C-ABI, against the CPU
oracle on the same seeded inputs.  Integer paths must match bit for bit; FP16
must satisfy |C_gpu - C_ref| <= 1e-4 * sum_k|a*b| + 1e-6 element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import (assert_block, check_against_oracle, decode_s4, freivalds, oracle_block,
                      run_gpu, to_dev)

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _clean_state():
    binding.gemm_set_config_override(0, 0, 0)
    yield
    binding.gemm_set_config_override(0, 0, 0)
    assert binding.gemm_last_device_status() == 0


# ------------------------------------------------------------ the named configs
def test_config_fp16_512_seed0():
    A, B = synth.fp16_uniform(512, 512, 512, seed=0)
    C = run_gpu("fp16", A, B, fill=float("nan"))
    assert check_against_oracle("fp16", A, B, C) == 512 * 512


def test_config_s8_2048_seed1():
    A, B = synth.s8_uniform(2048, 2048, 2048, seed=1)
    C = run_gpu("s8", A, B, fill=-1)
    assert check_against_oracle("s8", A, B, C) == 2048 * 2048


def test_config_s4_4096_seed2():
    A, B = synth.s4_uniform(4096, 4096, 4096, seed=2)
    C = run_gpu("s4", A, B, fill=-1)
    check_against_oracle("s4", A, B, C, seed=2)
    freivalds("s4", A, B, C, seed=2)


def test_config_fp16_8192_seed3_normal():
    A, B = synth.fp16_normal_clipped(8192, 8192, 8192, seed=3)
    C = run_gpu("fp16", A, B, fill=float("nan"))
    assert np.isfinite(C).all()
    check_against_oracle("fp16", A, B, C, seed=3)
    freivalds("fp16", A, B, C, seed=3)


@pytest.mark.parametrize("N", synth.SWEEP_SIZES)
@pytest.mark.parametrize("prec", synth.PRECISIONS)
def test_sweep(prec, N):
    seed = synth.sweep_seed(prec, N)
    A, B = synth.make(prec, N, N, N, seed)
    C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
    check_against_oracle(prec, A, B, C, seed=seed)
    if N > 2048:
        freivalds(prec, A, B, C, seed=seed)


# --------------------------------------------------- ragged and degenerate shapes
RAGGED = [
    # (M, N, K): K obeys the alignment rule of each precision (multiple of 32 works for all)
    (1, 1, 32), (1, 300, 64), (300, 1, 96), (127, 129, 160), (130, 70, 224),
    (257, 513, 288), (300, 520, 320), (640, 33, 1056), (129, 1030, 4128),
]


@pytest.mark.parametrize("prec", synth.PRECISIONS)
@pytest.mark.parametrize("M,N,K", RAGGED)
def test_ragged_shapes(prec, M, N, K):
    A, B = synth.make(prec, M, N, K, seed=1000 + M + N + K)
    ref, S = oracle_block(prec, A, B)
    for cta_group in (0, 1, 2):
        binding.gemm_set_config_override(0, 0, cta_group)
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        assert_block(prec, C, ref, S, "cta_group=%d" % cta_group)


@pytest.mark.parametrize("N", [1, 2, 3, 5, 30, 66, 131])
def test_n_not_multiple_of_four(N):
    """Rows of C that are not 16-byte multiples take the scalar store path."""
    M, K = 200, 128
    for prec in synth.PRECISIONS:
        A, B = synth.make(prec, M, N, K, seed=N)
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        check_against_oracle(prec, A, B, C, force_full=True)


def test_minimal_k():
    A, B = synth.fp16_uniform(140, 260, 8, seed=5)
    check_against_oracle("fp16", A, B, run_gpu("fp16", A, B, fill=float("nan")), force_full=True)
    A, B = synth.s8_uniform(140, 260, 16, seed=6)
    check_against_oracle("s8", A, B, run_gpu("s8", A, B, fill=-7), force_full=True)
    A, B = synth.s4_uniform(140, 260, 32, seed=7)
    check_against_oracle("s4", A, B, run_gpu("s4", A, B, fill=-7), force_full=True)


# ------------------------------------------------ every tile width the selector has
SHAPES = [(32, 1), (64, 1), (128, 1), (256, 1), (64, 2), (128, 2), (256, 2)]   # (BN, CTAs per tile)


@pytest.mark.parametrize("bn,cta_group", SHAPES)
@pytest.mark.parametrize("prec", synth.PRECISIONS)
def test_every_tile_shape(prec, bn, cta_group):
    M, N, K = 650, 1100, 1184           # several tiles in both directions + ragged tails
    A, B = synth.make(prec, M, N, K, seed=bn + cta_group)
    binding.gemm_set_config_override(bn, 0, cta_group)
    cfg = binding.gemm_query_config(prec, M, N, K)
    assert ("BN=%d " % bn) in cfg and ("cta_group=%d " % cta_group) in cfg
    C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
    check_against_oracle(prec, A, B, C, force_full=True)


@pytest.mark.parametrize("bn,cta_group", SHAPES)
@pytest.mark.parametrize("prec,M,N,K", [("fp16", 3000, 1000, 32), ("s8", 1024, 4096, 32),
                                        ("s4", 1500, 2304, 32), ("s8", 1500, 4096, 512)])
def test_many_short_tiles_per_cta(prec, M, N, K, bn, cta_group):
    """Several tiles per CTA with a mainloop far shorter than the epilogue: the stores of
    consecutive tiles overlap, so a staging buffer reused too early shows as wrong values
    (a tile whose epilogue has an odd number of store blocks is the critical case).
    Repeated calls, compared in full."""
    A, B = synth.make(prec, M, N, K, seed=K + bn)
    binding.gemm_set_config_override(bn, 0, cta_group, 1)
    ref, S = oracle_block(prec, A, B)
    for rep in range(3):
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        assert_block(prec, C, ref, S, "repeat %d" % rep)


@pytest.mark.parametrize("group_m", [1, 2, 3, 7, 64])
def test_raster_band_heights(group_m):
    M, N, K = 1300, 1500, 256
    A, B = synth.s8_uniform(M, N, K, seed=group_m)
    for cta_group in (1, 2):
        binding.gemm_set_config_override(64, group_m, cta_group)
        check_against_oracle("s8", A, B, run_gpu("s8", A, B, fill=-7), force_full=True)


# --------------------------------------------------------------- structured cases
def test_index_mapping_product_table():
    """a(i,0) = i mod 97 - 48, b(j,0) = j mod 89 - 44, rest 0: any row, column,
    lane-quarter or tile mix-up shows as a structured difference."""
    M, N, K = 1024, 1024, 128
    a = np.zeros((M, K), np.int8)
    b = np.zeros((N, K), np.int8)
    a[:, 0] = (np.arange(M) % 97) - 48
    b[:, 0] = (np.arange(N) % 89) - 44
    want = np.outer(a[:, 0].astype(np.int32), b[:, 0].astype(np.int32))
    for bn, cta_group in [(0, 0)] + SHAPES:
        binding.gemm_set_config_override(bn, 0, cta_group)
        assert np.array_equal(run_gpu("s8", a, b, fill=-7), want)
        got = run_gpu("fp16", a.astype(np.float16), b.astype(np.float16), fill=float("nan"))
        assert np.array_equal(got, want.astype(np.float32))
        a4, b4 = np.clip(a, -8, 7), np.clip(b, -8, 7)
        want4 = np.outer(a4[:, 0].astype(np.int32), b4[:, 0].astype(np.int32))
        assert np.array_equal(run_gpu("s4", synth.pack_s4(a4), synth.pack_s4(b4), fill=-7), want4)


def test_one_hot_k_positions():
    """C = [k0 == k1] for one-hot rows: pins the K order through swizzle, the
    32-byte MMA steps, the k-block ring and (int4) the nibble order."""
    K = 512
    ks = [0, 1, 2, 15, 16, 31, 32, 63, 64, 65, 127, 128, 129, 255, 256, 383, 384, K - 1]
    a = np.zeros((len(ks), K), np.int8)
    for r, k in enumerate(ks):
        a[r, k] = 1
    eye = np.eye(len(ks), dtype=np.int32)
    for cta_group in (1, 2):
        binding.gemm_set_config_override(0, 0, cta_group)
        assert np.array_equal(run_gpu("s8", a, a, fill=-7), eye)
        assert np.array_equal(run_gpu("s4", synth.pack_s4(a), synth.pack_s4(a), fill=-7), eye)
        assert np.array_equal(run_gpu("fp16", a.astype(np.float16), a.astype(np.float16)),
                              eye.astype(np.float32))


def test_all_ones_and_identity():
    K = 2048
    ones8 = np.ones((256, K), np.int8)
    assert np.all(run_gpu("s8", ones8, ones8) == K)
    assert np.all(run_gpu("fp16", ones8.astype(np.float16), ones8.astype(np.float16)) == K)
    assert np.all(run_gpu("s4", synth.pack_s4(ones8), synth.pack_s4(ones8)) == K)
    A, _ = synth.s8_uniform(300, 8, 256, seed=3)
    eye = np.eye(256, dtype=np.int8)
    assert np.array_equal(run_gpu("s8", A, eye), A.astype(np.int32))          # B = I -> C = A
    assert np.array_equal(run_gpu("s8", eye, A), A.T.astype(np.int32))        # A = I -> C = B^T


def test_int32_extremes():
    K = 8192
    lo8 = np.full((130, K), -128, np.int8)
    hi8 = np.full((70, K), 127, np.int8)
    assert np.all(run_gpu("s8", lo8, lo8) == 2 ** 27)
    assert np.all(run_gpu("s8", lo8, hi8) == -133169152)
    lo4 = synth.pack_s4(np.full((130, K), -8))
    hi4 = synth.pack_s4(np.full((70, K), 7))
    assert np.all(run_gpu("s4", lo4, lo4) == 524288)
    assert np.all(run_gpu("s4", lo4, hi4) == -458752)


def test_largest_k_for_int8():
    """K = 131056 (largest multiple of 16 <= 131071): 16384*K < 2^31 holds exactly."""
    K = 131056
    lo8 = np.full((3, K), -128, np.int8)
    assert np.all(run_gpu("s8", lo8, lo8) == 16384 * K)
    A, B = synth.s8_uniform(5, 7, K, seed=8)
    check_against_oracle("s8", A, B, run_gpu("s8", A, B), force_full=True)


def test_fp16_subnormals_and_large_values():
    g = np.random.Generator(np.random.PCG64(9))
    M, N, K = 150, 140, 256
    A = (g.integers(0, 0x0400, size=(M, K)).astype(np.uint16)
         | (g.integers(0, 2, size=(M, K)).astype(np.uint16) << 15)).view(np.float16)  # subnormals
    B = g.uniform(-60000, 60000, size=(N, K)).astype(np.float16)
    C = run_gpu("fp16", A, B, fill=float("nan"))
    check_against_oracle("fp16", A, B, C, force_full=True)


# ------------------------------------------------------------------ the pre-pass
def test_unpack_s4_matches_decoder():
    g = np.random.Generator(np.random.PCG64(10))
    P = g.integers(0, 256, size=(333, 480), dtype=np.uint8)
    out = binding.gemm_unpack_s4(to_dev(P))
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().astype(np.int16), decode_s4(P))
    # every byte value, in every position of a 16-byte group
    P = np.tile(np.arange(256, dtype=np.uint8), (16, 1))
    P = np.stack([np.roll(P[i], i) for i in range(16)])
    out = binding.gemm_unpack_s4(to_dev(P)).cpu().numpy()
    assert np.array_equal(out.astype(np.int16), decode_s4(P))


def test_s4_with_caller_workspace():
    M, N, K = 300, 200, 512
    A, B = synth.s4_uniform(M, N, K, seed=11)
    need = binding.gemm_s4_workspace_bytes(M, N, K)
    assert need >= (M + N) * K
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    C = binding.gemm_s4_ws(to_dev(A), to_dev(B), ws)
    torch.cuda.synchronize()
    assert np.array_equal(C.cpu().numpy(), oracle.gemm_s4(A, B, K))
    with pytest.raises(binding.GemmError) as e:
        binding.gemm_s4_ws(to_dev(A), to_dev(B), ws[: need - 256])
    assert e.value.code == -6


# ------------------------------------------------------------- API behaviour
def test_non_default_stream_and_repeat_calls():
    A, B = synth.s8_uniform(512, 384, 1024, seed=12)
    dA, dB = to_dev(A), to_dev(B)
    ref = oracle.gemm_s8(A, B)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        outs = [binding.gemm_s8(dA, dB) for _ in range(5)]
    st.synchronize()
    for C in outs:
        assert np.array_equal(C.cpu().numpy(), ref)


def test_argument_errors_enqueue_nothing():
    L = binding.lib()
    A = torch.zeros(64, 64, dtype=torch.int8, device="cuda")
    C = torch.full((64, 64), 5, dtype=torch.int32, device="cuda")
    p, c = A.data_ptr(), C.data_ptr()
    assert L.gemm_s8(64, 64, 64, None, p, c, None) == -1
    assert L.gemm_s8(0, 64, 64, p, p, c, None) == -1
    assert L.gemm_s8(64, -1, 64, p, p, c, None) == -1
    assert L.gemm_s8(64, 64, 24, p, p, c, None) == -2          # K % 16
    assert L.gemm_s8(64, 64, 64, p + 1, p, c, None) == -2      # pointer alignment
    assert L.gemm_s8(2, 2, 131072, p, p, c, None) == -3
    assert L.gemm_fp16(64, 64, 12, p, p, c, None) == -2        # K % 8
    assert L.gemm_s4(64, 64, 48, p, p, c, None) == -2          # K % 32
    assert L.gemm_s4(2, 2, 131072, p, p, c, None) == -3
    assert L.gemm_unpack_s4(4, 32, p, None, 32, None) == -1
    torch.cuda.synchronize()
    assert int((C != 5).sum()) == 0
    assert L.gemm_status_string(-3).decode().startswith("K too large")


# ----------------------------------------------------------------------- split-K
@pytest.mark.parametrize("splits", [2, 3, 5, 8])
@pytest.mark.parametrize("prec", synth.PRECISIONS)
def test_split_k_forced(prec, splits):
    M, N, K = 300, 520, 2080                      # 65 resp. 33 k-blocks: uneven K ranges
    A, B = synth.make(prec, M, N, K, seed=splits)
    ref, S = oracle_block(prec, A, B)
    for bn, cta_group in [(256, 2), (256, 1), (64, 1)]:
        binding.gemm_set_config_override(bn, 0, cta_group, splits)
        cfg = binding.gemm_query_config(prec, M, N, K)
        got = int(cfg.split("split_k=")[1].split()[0])
        assert 2 <= got <= splits, cfg            # capped so that no K range is empty
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        assert_block(prec, C, ref, S, "bn=%d cta_group=%d" % (bn, cta_group))


@pytest.mark.parametrize("M,N,K", [(1, 4096, 4096), (16, 8192, 8192), (64, 4096, 16384),
                                   (128, 1030, 4128), (40, 70, 8192), (8, 33, 1024)])
def test_small_m_shapes_pick_split_k(M, N, K):
    """Decode-like shapes: few C tiles, long K.  The selector splits K on its own; rows of C
    that are not 16-byte multiples take the atomic-add path."""
    for prec in synth.PRECISIONS:
        A, B = synth.make(prec, M, N, K, seed=M + N)
        if K >= 4096:
            assert "split_k=1 " not in binding.gemm_query_config(prec, M, N, K)
        C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        check_against_oracle(prec, A, B, C, force_full=True)


def test_split_k_more_ranges_than_blocks_is_capped():
    A, B = synth.s8_uniform(130, 260, 256, seed=1)      # 2 k-blocks
    for bn in (0, 256, 64):
        binding.gemm_set_config_override(bn, 0, 0, 8)
        cfg = binding.gemm_query_config("s8", 130, 260, 256)
        assert int(cfg.split("split_k=")[1].split()[0]) <= 2, cfg     # never more ranges than slots
        check_against_oracle("s8", A, B, run_gpu("s8", A, B, fill=-7), force_full=True)


# ------------------------------------------------------------ size and host-side edges
def test_large_m_and_n_small_k():
    """Many tiles (157 x 79 of the 128 x 256 shape), ragged both ways, C = 1.6 GB."""
    M, N, K = 20001, 20004, 64
    for prec in ("s8", "fp16"):
        A, B = synth.make(prec, M, N, K, seed=123)
        C = run_gpu(prec, A, B)
        check_against_oracle(prec, A, B, C, seed=123)          # 256 rows + 256 columns + edges
        if prec == "s8":
            freivalds(prec, A, B, C, seed=123, vectors=2)
        del C


def test_two_host_threads_on_two_streams():
    import threading
    A, B = synth.s8_uniform(1024, 768, 2048, seed=31)
    ref = oracle.gemm_s8(A, B)
    dA, dB = to_dev(A), to_dev(B)
    results, errors = {}, []

    def worker(tag):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                outs = [binding.gemm_s8(dA, dB, stream=st) for _ in range(20)]
            st.synchronize()
            results[tag] = [o.cpu().numpy() for o in outs[-3:]]
        except Exception as e:          # noqa: BLE001 - reported below
            errors.append(e)

    torch.cuda.synchronize()
    threads = [threading.Thread(target=worker, args=(t,)) for t in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for tag in range(2):
        for C in results[tag]:
            assert np.array_equal(C, ref)


def test_transpose_symmetry_on_gpu():
    """gemm(A, B) == gemm(B, A)^T exactly for the integer paths (different tiles, same sums)."""
    A, B = synth.s8_uniform(700, 300, 1024, seed=41)
    assert np.array_equal(run_gpu("s8", A, B), run_gpu("s8", B, A).T)
    A4, B4 = synth.s4_uniform(700, 300, 1024, seed=42)
    assert np.array_equal(run_gpu("s4", A4, B4), run_gpu("s4", B4, A4).T)


def test_tail_wave_split():
    """4096^2 x 8192 FP16: 256 tiles on 74 SM pairs leave a last wave of 34 tiles, which the
    selector splits in two along K (adds into a zeroed rectangle of C); ragged variant too."""
    for M, N, K in ((4096, 4096, 8192), (4000, 3900, 8200)):
        cfg = binding.gemm_query_config("fp16", M, N, K)
        assert "split_k=2 " in cfg and "split_tiles=0 " not in cfg, cfg
        A, B = synth.fp16_uniform(M, N, K, seed=77)
        C = run_gpu("fp16", A, B, fill=float("nan"))
        check_against_oracle("fp16", A, B, C, seed=77)
        freivalds("fp16", A, B, C, seed=77, vectors=4)
    # the integer kernel takes the same path when K is long enough
    M, N, K = 4096, 4096, 8192
    assert "split_k=2 " in binding.gemm_query_config("s8", M, N, K)
    A, B = synth.s8_uniform(M, N, K, seed=78)
    C = run_gpu("s8", A, B, fill=-7)
    check_against_oracle("s8", A, B, C, seed=78)
    freivalds("s8", A, B, C, seed=78, vectors=4)


@pytest.mark.parametrize("prec", ["fp16", "s8", "s4"])
def test_tail_wave_of_a_few_tiles_is_split_deep(prec):
    """76 (ragged: 19 x 4) tiles of 256 x 256 on 74 SM pairs leave a last wave of two tiles: the
    selector splits those as deep as the idle pairs allow (>= 8 k-blocks per unit) instead of
    paying a whole tile time for them.  INT4 through the fused CTA-pair kernel in both forms."""
    M, N, K = 1000, 4864, 8192 if prec != "fp16" else 4096
    schemes = [0] if prec != "s4" else [5, 6]
    A, B = synth.make(prec, M, N, K, seed=79)
    for scheme in schemes:
        binding.gemm_set_s4_scheme(scheme)
        try:
            cfg = binding.gemm_query_config(prec, M, N, K)
            assert "split_k=8 " in cfg and "split_tiles=2 " in cfg and "tiles=76 " in cfg, cfg
            C = run_gpu(prec, A, B, fill=float("nan") if prec == "fp16" else -7)
        finally:
            binding.gemm_set_s4_scheme(0)
        check_against_oracle(prec, A, B, C, seed=79)
        freivalds(prec, A, B, C, seed=79, vectors=4)
