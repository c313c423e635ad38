"""CPU-only checks of the boundary: the shared library loads, exports every
symbol the header declares, and rejects bad arguments without a GPU."""
import ctypes
import os
import re

import pytest

from paper_2608_10103_b200 import binding, build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADERS = [os.path.join(ROOT, "include", "b200gemm.h"),
           os.path.join(ROOT, "include", "b200gemm_debug.h")]


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return binding.lib()


def declared_functions():
    text = "".join(open(h).read() for h in HEADERS)
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(gemm_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_header_and_binding_agree():
    assert declared_functions() == sorted(binding.EXPORTS)


def test_every_declared_symbol_is_exported(lib):
    for name in declared_functions():
        assert getattr(lib, name) is not None


def test_status_strings_and_version(lib):
    assert binding.gemm_version() >= 1000
    assert binding.gemm_status_string(0) == "ok"
    for code in range(-7, 0):
        assert binding.gemm_status_string(code) != "unknown status"
    assert binding.gemm_status_string(-99) == "unknown status"


def test_argument_validation_needs_no_gpu(lib):
    # these are rejected before any CUDA call is made
    assert lib.gemm_fp16(0, 8, 8, 16, 16, 16, None) == -1
    assert lib.gemm_fp16(8, 8, 8, None, 16, 16, None) == -1
    assert lib.gemm_fp16(8, 8, 12, 16, 16, 16, None) == -2
    assert lib.gemm_fp16(8, 8, 8, 24, 16, 16, None) == -2
    assert lib.gemm_s8(8, 8, 8, 16, 16, 16, None) == -2          # K % 16
    assert lib.gemm_s8(8, 8, 131072, 16, 16, 16, None) == -3
    assert lib.gemm_s4(8, 8, 16, 16, 16, 16, None) == -2         # K % 32
    assert lib.gemm_s4(8, 8, 131104, 16, 16, 16, None) == -3
    assert lib.gemm_s4_ws(8, 8, 32, 16, 16, 16, None, 0, None) == -1
    assert lib.gemm_s4_ws(8, 8, 32, 16, 16, 16, 256, 16, None) == -6
    assert lib.gemm_unpack_s4(4, 48, 16, 16, 48, None) == -2
    assert lib.gemm_mma_peak_probe(2, 10, 256, 0, ctypes.pointer(ctypes.c_double(0)), None) == -1
    assert lib.gemm_mma_peak_probe(0, 10, 24, 0, ctypes.pointer(ctypes.c_double(0)), None) == -1
    assert lib.gemm_set_config_override(48, 0, 0, 0) == -1
    assert lib.gemm_set_config_override(32, 0, 2, 0) == -1          # no 32-wide pair tile
    assert lib.gemm_set_config_override(0, 0, 3, 0) == -1
    assert lib.gemm_set_config_override(0, 0, 0, 0) == 0
    assert lib.gemm_set_config_override(0, 0, 0, 65) == -1


def test_workspace_size(lib):
    assert binding.gemm_s4_workspace_bytes(0, 8, 32) == 0
    assert binding.gemm_s4_workspace_bytes(8192, 8192, 8192) == 2 * 8192 * 8192
    assert binding.gemm_s4_workspace_bytes(3, 5, 32) == 512      # each half rounded up to 256


def test_selector_descriptions(lib):
    cfg = binding.gemm_query_config("fp16", 8192, 8192, 8192)
    assert "BN=256" in cfg and "cta_group=2" in cfg and "kind=f16" in cfg
    assert "prepass=unpack_s4" in binding.gemm_query_config("s4", 1536, 1536, 8192)
    assert "s4=fused_unpack" in binding.gemm_query_config("s4", 4096, 4096, 4096)
    binding.gemm_set_config_override(64, 3, 1)
    try:
        cfg = binding.gemm_query_config("s8", 1000, 1000, 1024)
        assert "BM=128 BN=64 " in cfg and "group_m=3" in cfg and "tiles=%d" % (8 * 16) in cfg
    finally:
        binding.gemm_set_config_override(0, 0, 0)


def test_binding_rejects_cpu_tensors(lib):
    import torch
    a = torch.zeros(8, 8, dtype=torch.float16)
    with pytest.raises(TypeError):
        binding.gemm_fp16(a, a, torch.zeros(8, 8))


def test_product_path_never_touches_the_oracle():
    """The library, its binding and its build script must not import or link the checker."""
    pkg = os.path.join(ROOT, "paper_2608_10103_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "gemm_oracle" not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2608_10103_b200" not in text and "b200gemm" not in text, f


def _parse(cfg):
    out = {}
    for tok in cfg.split():
        if "=" in tok:
            k, v = tok.split("=", 1)
            out[k] = int(v) if v.lstrip("-").isdigit() else v
    return out


def test_selector_invariants_over_many_shapes(lib):
    """Host logic only: whatever the selector picks must be a built shape, its split-K
    factor must leave no K range empty, and the CTA count must fit the machine."""
    import itertools
    dims = [1, 7, 128, 129, 256, 300, 512, 1000, 2048, 2560, 4096, 5120, 8192, 20001]
    ks = [32, 64, 160, 512, 1056, 4096, 8192, 16384, 131040]
    built = {(1, 256), (1, 128), (1, 64), (1, 32), (2, 256), (2, 128), (2, 64)}
    for prec, elem in (("fp16", 2), ("s8", 1), ("s4", 1)):
        for M, N, K in itertools.product(dims, dims, ks):
            text = binding.gemm_query_config(prec, M, N, K)
            c = _parse(text)
            if text.startswith("few_rows"):   # the kernel for a short side of up to 16 rows
                short, long_ = min(M, N), max(M, N)
                assert (short <= 16 or (prec == "s4" and short <= 32 and long_ <= 8192)) and long_ >= 512
                assert c["short_rows"] == short
                if prec == "s8":
                    assert short <= 8 or long_ * K <= 64 << 20
                if prec == "fp16":
                    assert long_ * K <= 32 << 20
                if prec != "s4":       # enough row blocks for the length of a row
                    assert -(-long_ // 32) >= 6 * -(-(K * (2 if prec == "fp16" else 1)) // 1024)
                rows = c["rows_per_block"]
                assert rows == 32 and c["blocks"] == -(-long_ // rows)
                row_bytes = K // 2 if prec == "s4" else 2 * K if prec == "fp16" else K
                w, d = c["warps"], c["depth"]
                assert w in (1, 2, 4, 8, 16) and 2 <= d <= 8
                assert w == 1 or -(-row_bytes // 64) >= 2 * w      # two 64-byte steps per warp
                nt, mt = (1 if short <= 8 else 2 if short <= 16 else 4), rows // 16
                smem = d * (2 * mt + nt) * w * 512 + w * 8 * nt * (16 * mt + 4) * 4
                per_sm = min((227 * 1024) // (smem + 1024), 64 // w, 32)
                assert per_sm >= 1 and 1 <= c["ctas"] <= min(c["blocks"], per_sm * 148)
                assert c["ctas"] == c["blocks"] or c["ctas"] % 148 == 0
                continue
            if "swap_ab" in text:        # the tile is described in the kernel's orientation
                assert N >= 1024 and M <= (32 if prec == "fp16" and N < 16384 else 64)
                M, N = N, M
            cg, bn, sp = c["cta_group"], c["BN"], c["split_k"]
            wide = c["BM"] == 512            # the 512 x 256 CTA-pair kernel for large problems
            assert (cg, bn) in built and (c["BM"] == 128 * cg or (wide and (cg, bn) == (2, 256)))
            if wide:
                assert sp == 1 and "swap_ab" not in text and "fused_unpack" not in text
                assert -(-M // 512) * -(-N // 256) >= 2 * 74 and c["stages"] == 4
                assert K >= (6144 if prec == "fp16" else 8192)
            atoms = c["BK"] * elem // 128
            assert atoms in (1, 2)
            if "fused_unpack" in text:   # K is split in packed slots of 256 values
                # a problem with a short side, or a single wave of pair tiles
                tiles2 = -(-M // 256) * -(-N // bn)
                units2 = tiles2 + c["split_tiles"] * (sp - 1)
                # ... or large in both dimensions: at least a wave of pair tiles, K >= 2048
                assert (M * N <= 512 * (M + N) or (cg == 2 and bn == 256 and tiles2 <= 74) or
                        (cg == 2 and bn == 256 and min(M, N) <= 1024 and
                         4 * units2 >= 3 * 74 * -(-units2 // 74)) or
                        (cg == 2 and bn == 256 and min(M, N) > 1024 and tiles2 >= 74 and K >= 2048))
                if cg == 2:
                    assert bn in (256, 128)
                atoms = 2
            slots = -(-(-(-K * elem // 128)) // atoms)
            tiles = -(-M // c["BM"]) * -(-N // bn)
            assert c["tiles"] == tiles
            assert 1 <= sp <= 32 and sp <= slots
            assert (sp - 1) * -(-slots // sp) < slots, (prec, M, N, K, c)
            if sp > 1:
                assert 0 < c["split_tiles"] <= tiles
                units = tiles + c["split_tiles"] * (sp - 1)
            else:
                assert c["split_tiles"] == 0
                units = tiles
            if "even_share" in text:     # fused INT4, one-CTA tiles: equal contiguous shares of K
                share = int(text.split("even_share=")[1].split()[0])
                slots = -(-K // 256)
                assert "fused_unpack" in text and cg == 1 and share >= 16
                assert c["ctas"] == -(-tiles * slots // share) <= 148
                assert share == -(-tiles * slots // 148)
            else:
                assert c["ctas"] == min(units, 148 // cg) * cg
            assert 1 <= c["group_m"] <= -(-M // c["BM"])


def test_few_rows_shapes_when_forced(lib):
    """gemm_set_kernel_family(3) takes the few-rows kernel up to 32 short rows, whatever the other
    sizes: its launch shape must fit an SM (ring of at least two slots plus the warps' sums)."""
    binding.gemm_set_kernel_family(3)
    try:
        for prec in ("fp16", "s8", "s4"):
            for short in (1, 8, 9, 16, 17, 24, 32):
                for long_ in (33, 512, 2048, 4096, 20001):
                    for K in (32, 512, 4096, 8192, 16384, 131040):
                        c = _parse(binding.gemm_query_config(prec, short, long_, K))
                        assert "rows_per_block" in c, (prec, short, long_, K)
                        nt = 1 if short <= 8 else 2 if short <= 16 else 4
                        w, d = c["warps"], c["depth"]
                        smem = d * (4 + nt) * w * 512 + w * 8 * nt * 36 * 4
                        assert w in (1, 2, 4, 8, 16) and 2 <= d <= 8 and smem + 1024 <= 227 * 1024
    finally:
        binding.gemm_set_kernel_family(0)


def test_selector_headline_choices(lib):
    big = _parse(binding.gemm_query_config("fp16", 8192, 8192, 8192))
    assert (big["BM"], big["BN"], big["cta_group"], big["split_k"], big["stages"]) == (512, 256, 2, 1, 4)
    binding.gemm_set_kernel_family(1)
    try:
        classic = _parse(binding.gemm_query_config("fp16", 8192, 8192, 8192))
        assert (classic["BM"], classic["BN"], classic["cta_group"], classic["stages"]) == (256, 256, 2, 6)
    finally:
        binding.gemm_set_kernel_family(0)
    dec = _parse(binding.gemm_query_config("fp16", 16, 8192, 8192))
    assert dec["split_k"] > 1 and dec["split_tiles"] == dec["tiles"]
    assert binding.gemm_query_config("fp16", 16, 4096, 8192).startswith("few_rows")
    assert not binding.gemm_query_config("fp16", 16, 8192, 8192).startswith("few_rows")
    assert not binding.gemm_query_config("fp16", 16, 1024, 8192).startswith("few_rows")
    few = binding.gemm_query_config("s4", 16, 8192, 8192)
    assert few.startswith("few_rows") and "s4=in_registers" in few
    assert binding.gemm_query_config("s8", 8, 4096, 4096).startswith("few_rows")
    assert binding.gemm_query_config("s8", 16, 8192, 8192).startswith("few_rows")
    assert not binding.gemm_query_config("s8", 16, 28672, 8192).startswith("few_rows")
    assert binding.gemm_query_config("s8", 8, 28672, 8192).startswith("few_rows")
    assert binding.gemm_query_config("s4", 17, 8192, 8192).startswith("few_rows")
    assert not binding.gemm_query_config("s4", 17, 8200, 8192).startswith("few_rows")
    assert not binding.gemm_query_config("s4", 33, 8192, 8192).startswith("few_rows")
    tail = _parse(binding.gemm_query_config("fp16", 4096, 4096, 8192))
    assert tail["split_k"] == 2 and tail["split_tiles"] == 256 % 74
    binding.gemm_set_config_override(0, 0, 0, 1)
    try:
        assert _parse(binding.gemm_query_config("fp16", 4096, 4096, 8192))["split_k"] == 1
    finally:
        binding.gemm_set_config_override(0, 0, 0, 0)
