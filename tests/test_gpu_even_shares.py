"""GPU parity of the "even shares" form of split-K in the one-CTA fused INT4 kernels: the tiles' K
ranges, laid end to end, are cut into equal contiguous shares, one per SM, so a CTA works on the
end of one tile, whole tiles and the beginning of another, and every piece is added into a
zeroed C.  Exact against the oracle, equal to the plain forms, switchable by policy bit 128."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_10103_b200 import binding, synth
from gpu_util import check_against_oracle, run_gpu, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _clean():
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_l2_policy(11)
    yield
    binding.gemm_set_config_override(0, 0, 0, 0)
    binding.gemm_set_s4_scheme(0)
    binding.gemm_set_l2_policy(11)
    binding.gemm_set_swap_ab(0)
    binding.gemm_set_kernel_family(0)
    assert binding.gemm_last_device_status() == 0


def _share(cfg):
    return int(cfg.split("even_share=")[1].split()[0]) if "even_share=" in cfg else 0


# 224 tiles on 148 SMs, unsplit (some SMs two, the average 1.5), with a ragged K whose last packed
# slot is partly filled; 165 64-wide, 188 and 230 32-wide tiles; a long K; shares that start and
# end inside tiles in every combination
@pytest.mark.parametrize("M,N,K", [(32, 28672, 4128), (64, 28000, 4096), (16, 24000, 4128), (8, 29440, 8192)])
def test_even_shares_exact(M, N, K):
    if M <= 16:       # the automatic route there is the kernel for a few rows: ask for the tiles
        binding.gemm_set_kernel_family(1)
    cfg = binding.gemm_query_config("s4", M, N, K)
    assert "fused_unpack" in cfg and _share(cfg) >= 16, cfg
    A, B = synth.s4_uniform(M, N, K, seed=M + K)
    for rep in range(2):
        C = run_gpu("s4", A, B, fill=-7)
        check_against_oracle("s4", A, B, C, force_full=M * N <= 1 << 20)
    binding.gemm_set_l2_policy(11 + 128)     # the plain form: same numbers, bit for bit
    assert _share(binding.gemm_query_config("s4", M, N, K)) == 0
    assert np.array_equal(C, run_gpu("s4", A, B, fill=-7))


def test_even_shares_with_operands_not_exchanged_and_forced_widths():
    """The 64- and 128-wide one-CTA fused tiles take the same path (forced here)."""
    for bn, (M, N, K) in ((64, (48, 9000, 2048)), (128, (100, 24000, 1056)), (32, (16, 8192, 4096))):
        binding.gemm_set_s4_scheme(2)
        binding.gemm_set_swap_ab(2 if bn == 32 else 1)
        binding.gemm_set_config_override(bn, 0, 1, 0)
        cfg = binding.gemm_query_config("s4", M, N, K)
        A, B = synth.s4_uniform(M, N, K, seed=bn)
        C = run_gpu("s4", A, B, fill=-7)
        check_against_oracle("s4", A, B, C, force_full=M * N <= 1 << 20)
        if _share(cfg) == 0:
            continue
        binding.gemm_set_l2_policy(11 + 128)
        assert np.array_equal(C, run_gpu("s4", A, B, fill=-7))
        binding.gemm_set_l2_policy(11)


def test_even_shares_not_taken_where_they_do_not_pay():
    assert _share(binding.gemm_query_config("s4", 256, 256, 8192)) == 0      # one tile, no split chosen
    binding.gemm_set_kernel_family(1)
    assert _share(binding.gemm_query_config("s4", 16, 8192, 8192)) == 0      # 16 -> 14 slots per SM: not worth a second piece
    binding.gemm_set_kernel_family(0)
    assert _share(binding.gemm_query_config("s4", 64, 21000, 1056)) == 0     # shares of 6 slots: measured slower
    assert _share(binding.gemm_query_config("s4", 8192, 8192, 8192)) == 0    # pre-pass route
    assert _share(binding.gemm_query_config("s4", 256, 28672, 8192)) == 0    # CTA-pair tiles
    assert _share(binding.gemm_query_config("s8", 16, 8192, 8192)) == 0      # INT8: bound by HBM, not by the SM
