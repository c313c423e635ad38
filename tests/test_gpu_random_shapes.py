"""Seeded random walk over shapes x forced tile configurations x entry points x streams,
each result checked against the oracle on a random subset of rows (all columns).

The fixed-shape parity tests pin the cases one can think of; this one exists for the
interactions nobody listed (tile count per CTA x K length x output mode x split-K)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import to_dev

pytestmark = pytest.mark.gpu

# (bn, group_m, cta_group, split_k); 0 = let the selector decide
CONFIGS = [(0, 0, 0, 0), (0, 0, 0, 1), (256, 0, 2, 0), (256, 0, 1, 1), (128, 0, 2, 1), (64, 0, 1, 1),
           (32, 0, 1, 1), (128, 0, 1, 0), (64, 0, 2, 0), (256, 3, 2, 2), (0, 0, 0, 3), (128, 1, 2, 4),
           (64, 5, 1, 2), (256, 0, 2, 8), (32, 0, 1, 5), (32, 0, 1, 4)]
MS = [1, 2, 17, 127, 128, 129, 255, 256, 300, 511, 777, 1024, 1500, 2048, 3000]
NS = [1, 3, 8, 64, 100, 256, 260, 512, 1000, 1024, 2304, 4096]
KS = [32, 64, 96, 128, 160, 256, 512, 1056, 2048, 4128]
ROWS = 24


@pytest.fixture(autouse=True)
def _clean_state():
    binding.gemm_set_config_override(0, 0, 0, 0)
    yield
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_swap_ab(0)
    assert binding.gemm_last_device_status() == 0


def _exact_rows(prec, A, B, K, rows):
    if prec == "fp16":
        return oracle.gemm_fp16(A, B, rows=rows)
    if prec == "s8":
        return oracle.gemm_s8_i64(A, B, rows=rows), None
    return oracle.gemm_s4_i64(A, B, K, rows=rows), None


def _modes(prec):
    if prec == "fp16":
        return ["raw", "raw", "out16"]
    if prec == "s8":
        return ["raw", "raw", "deq32", "deq16"]
    return ["raw", "deq32", "deq16", "ws", "static"]


@pytest.mark.parametrize("seed", range(30))
def test_random_shapes_configs_and_entry_points(seed):
    g = np.random.Generator(np.random.PCG64(9000 + seed))
    side = torch.cuda.Stream()
    checked = 0
    for case in range(14):
        M, N, K = int(g.choice(MS)), int(g.choice(NS)), int(g.choice(KS))
        prec = str(g.choice(synth.PRECISIONS))
        A, B = synth.make(prec, M, N, K, seed=int(g.integers(1 << 30)))
        rows = np.unique(np.concatenate([g.choice(M, size=min(ROWS, M), replace=False), [0, M - 1]])).astype(np.int32)
        exact, S = _exact_rows(prec, A, B, K, rows)
        dA, dB = to_dev(A), to_dev(B)
        rs = (g.uniform(0.5, 2.0, M) * 1e-2).astype(np.float32)
        cs = (g.uniform(0.5, 2.0, N) * 1e-2).astype(np.float32)
        d_rs, d_cs = to_dev(rs), to_dev(cs)
        for trial in range(3):
            cfg = CONFIGS[int(g.integers(len(CONFIGS)))]
            mode = str(g.choice(_modes(prec)))
            if mode == "static" and binding.gemm_s4_workspace_bytes(M, N, K) > binding.gemm_s4_static_capacity():
                mode = "raw"
            stream = side if g.integers(2) else None
            what = "%s %s M=%d N=%d K=%d cfg=%s side_stream=%s" % (prec, mode, M, N, K, cfg, stream is not None)
            binding.gemm_set_config_override(*cfg)
            binding.gemm_set_s4_scheme(int(g.integers(3)))   # automatic / pre-pass / fused
            binding.gemm_set_swap_ab(int(g.integers(3)))     # automatic / never / always
            out_dtype = {"raw": torch.float32 if prec == "fp16" else torch.int32, "ws": torch.int32,
                         "static": torch.int32, "out16": torch.float16, "deq32": torch.float32,
                         "deq16": torch.float16}[mode]
            fill = float("nan") if out_dtype.is_floating_point else -7
            outs = []        # every output stays alive until the side stream has drained
            try:
                for rep in range(int(g.integers(1, 3))):
                    C = torch.full((M, N), fill, dtype=out_dtype, device="cuda")
                    outs.append(C)
                    if stream is not None:
                        stream.wait_stream(torch.cuda.current_stream())
                    if mode == "raw":
                        binding.gemm(prec, dA, dB, C, stream=stream)
                    elif mode == "out16":
                        binding.gemm_fp16_f16out(dA, dB, C, stream=stream)
                    elif mode in ("deq32", "deq16"):
                        fn = binding.gemm_s8_dequant if prec == "s8" else binding.gemm_s4_dequant
                        fn(dA, dB, d_rs, d_cs, C, out_dtype, stream=stream)
                    elif mode == "ws":
                        ws = torch.empty(binding.gemm_s4_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
                        outs.append(ws)
                        binding.gemm_s4_ws(dA, dB, ws, C, stream=stream)
                    else:
                        binding.gemm_s4_static(dA, dB, C, stream=stream)
            except binding.GemmError as e:
                # a forced tile shape the output mode does not have is refused, nothing enqueued
                assert e.code == -1, what
                torch.cuda.synchronize()
                continue
            torch.cuda.synchronize()
            got = C.cpu().numpy()[rows]
            if mode in ("raw", "ws", "static"):
                if prec == "fp16":
                    ok, worst = oracle.fp16_check(got, exact, S)
                    assert ok, "%s: %.3g x bound" % (what, worst)
                else:
                    assert np.array_equal(got, oracle.narrow_int32(exact)), what
            elif mode == "out16":
                ok, worst = oracle.fp16_out_check(got, exact, S)
                assert ok, "%s: %.3g x bound" % (what, worst)
            else:
                ref = oracle.dequant_ref(exact, rs[rows], cs)
                ok, worst = oracle.dequant_check(got, ref, mode == "deq16")
                assert ok, "%s: %.3g x bound" % (what, worst)
            checked += 1
    assert checked >= 20
