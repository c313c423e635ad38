"""Seeded walk over shapes of the kind that trigger the selector's special cases in the automatic
mode -- a sparsely filled last wave split along K, even shares, the hybrid INT4 form, exchanged
operands, the pre-pass, the kernel for a few rows -- each result checked against the oracle on a sample of rows, and the
walk as a whole checked to have met every one of those cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _shape(g):
    kind = int(g.integers(6))
    if kind == 5:      # INT4, a short M against a large N K: the hybrid form of the fused pair kernel
        return (int(g.choice([256, 384, 512])), int(g.integers(24000, 29000)), 8192), "s4"
    if kind == 4:      # INT4, few rows, 1.3 ... 1.9 tiles of 128 rows per SM: even shares
        return (int(g.choice([24, 32, 32])), int(g.integers(24000, 30000)), int(g.choice([4096, 4128, 8192]))), "s4"
    if kind == 0:      # few rows against a wide N
        return (int(g.choice([1, 3, 8, 16, 24, 32, 48, 64, 100, 128])), int(g.integers(8000, 30000)),
                int(g.choice([1024, 2048, 4096, 4128, 8192]))), None
    if kind == 1:      # a short M against a wide N
        return (int(g.choice([192, 256, 300, 384, 512, 640, 1000, 1024])), int(g.integers(6000, 29000)),
                int(g.choice([1056, 2048, 4096, 8192]))), None
    if kind == 2:      # tile counts just above a multiple of the 74 SM pairs
        tm = int(g.integers(1, 12))
        tiles = int(g.choice([74, 148, 222])) + int(g.integers(1, 9))
        tn = max(1, tiles // tm)
        return (tm * 256 - int(g.integers(0, 200)), tn * 256 - int(g.integers(0, 200)),
                int(g.choice([2048, 4096, 8192]))), None
    return (int(g.integers(1, 3000)), int(g.integers(1, 5000)), int(g.integers(1, 130)) * 32), None


def test_automatic_paths_over_a_seeded_walk_of_shapes():
    g = np.random.Generator(np.random.PCG64(777))
    met = set()
    cases = 0
    while cases < 70:
        (M, N, K), forced = _shape(g)
        prec = forced or str(g.choice(["fp16", "s8", "s4", "s4"]))
        if M * N > 30e6 or (M + N) * K > 300e6:
            continue
        if forced is None and g.integers(3) == 0:
            M, N = N, M
        cases += 1
        A, B = synth.make(prec, M, N, K, seed=int(g.integers(1 << 30)))
        rows = np.unique(np.concatenate([g.choice(M, size=min(10, M), replace=False), [0, M - 1]])).astype(np.int32)
        cfg = binding.gemm_query_config(prec, M, N, K)
        m = dict(kv.split("=") for kv in cfg.split() if "=" in kv)
        for f in ("even_share", "a=int8_image", "fused_unpack", "prepass", "swap_ab", "few_rows"):
            if f in cfg:
                met.add(f)
        if "few_rows" not in cfg and int(m["split_k"]) > 1 and m["split_tiles"] != m["tiles"]:
            met.add("tail_split_deep" if int(m["split_k"]) > 4 else "tail_split")
        C = torch.full((M, N), float("nan") if prec == "fp16" else -7,
                       dtype=torch.float32 if prec == "fp16" else torch.int32, device="cuda")
        dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
        for rep in range(2):
            binding.gemm(prec, dA, dB, C)
        torch.cuda.synchronize()
        got = C.cpu().numpy()[rows]
        what = "%s %d x %d x %d: %s" % (prec, M, N, K, cfg)
        if prec == "fp16":
            ref, S = oracle.gemm_fp16(A, B, rows=rows)
            assert oracle.fp16_check(got, ref, S)[0], what
        else:
            exact = oracle.gemm_s8_i64(A, B, rows=rows) if prec == "s8" else oracle.gemm_s4_i64(A, B, K, rows=rows)
            assert np.array_equal(got.astype(np.int64), exact), what
    assert binding.gemm_last_device_status() == 0
    assert met >= {"even_share", "a=int8_image", "fused_unpack", "prepass", "swap_ab", "tail_split",
                   "tail_split_deep", "few_rows"}, met
