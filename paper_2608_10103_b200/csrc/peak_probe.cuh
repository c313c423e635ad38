// MMA-issue-only peak probe: how fast one SM's tensor core retires tcgen05.mma
// when nothing else is in the way (operands resident in shared memory, no
// loads, no epilogue).  Its throughput is the "measured peak" that the GEMM's
// achieved rate is reported against, next to the spec-sheet figure.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace b200gemm {

constexpr int PROBE_BN = 256;
constexpr int PROBE_SLOTS = 4;  // operand slots cycled through, as the GEMM's ring does
constexpr int PROBE_SMEM = PROBE_SLOTS * (BM + PROBE_BN) * BK_BYTES + 1024 + 64;  // ring + align + barriers

// n_cols: N of each MMA (multiple of 16, <= 256).  iters is rounded down to a
// multiple of 4.  commit_every: 0 = one commit at the end; c > 0 = also a
// tcgen05.commit after every c groups of 4 MMAs (to a barrier nobody waits on);
// a pipelined GEMM commits once per k-block, i.e. c = 1.
// trace: optional, TRACE_SLOTS words per CTA ([0] cycles, [1] ns of the MMA loop).
template <int KIND>
__global__ void __launch_bounds__(128, 1)
mma_peak_probe_kernel(int iters, int n_cols, int commit_every, int* status,
                      unsigned long long* trace) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_addr(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  constexpr int RING = PROBE_SLOTS * (BM + PROBE_BN) * BK_BYTES;
  const uint32_t bar = base + RING;
  const uint32_t side_bar = base + RING + 8;
  volatile uint32_t* holder = reinterpret_cast<volatile uint32_t*>(base_ptr + RING + 16);

  // Operand bits: pseudo-random, finite (fp16 magnitudes in [2^-3, 2)), so that
  // data toggling -- and with it power and clocks -- resembles a real GEMM.
  uint32_t x = 0x9E3779B9u * (blockIdx.x * blockDim.x + threadIdx.x + 1);
  for (int i = threadIdx.x; i < RING / 4; i += blockDim.x) {
    x ^= x << 13; x ^= x >> 17; x ^= x << 5;
    uint32_t v = x;
    if (KIND == ptx::KIND_F16) v = (x & 0x8FFF8FFFu) | 0x30003000u;
    reinterpret_cast<uint32_t*>(base_ptr)[i] = v;
  }
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);
    ptx::mbar_init(side_bar, 1);
    ptx::fence_mbar_init();
  }
  ptx::fence_proxy_async_smem();
  if (threadIdx.x < 32) {
    ptx::tmem_alloc<1>(ptx::smem_addr(const_cast<uint32_t*>(holder)), 512);
    ptx::tmem_relinquish<1>();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *holder;

  if (threadIdx.x < 32) {  // whole warp runs the loop; one elected lane issues
    const uint32_t idesc = ptx::make_idesc<KIND>(BM, n_cols);
    const long long c0 = clock64();
    const uint64_t t_begin = ptx::globaltimer_ns();
    // Groups of 4 MMAs = one k-block of the GEMM kernels (4 x 32 bytes of K in one slot).
    const int groups = iters / 4;
    for (int g = 0; g < groups; ++g) {
      const int slot = g % PROBE_SLOTS;
      const uint32_t a_src = base + slot * (BM + PROBE_BN) * BK_BYTES;
      const uint64_t a_desc = ptx::smem_desc_sw128(a_src);
      const uint64_t b_desc = ptx::smem_desc_sw128(a_src + BM * BK_BYTES);
      const uint32_t d = tmem_base + ((g >> 4) & 1) * PROBE_BN;  // switch accumulator every 64 MMAs
      const bool commit = commit_every > 0 && (g + 1) % commit_every == 0;
      if (ptx::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const uint64_t step = static_cast<uint64_t>((kk * MMA_K_BYTES) >> 4);
          ptx::mma_ss<KIND, 1>(d, a_desc + step, b_desc + step, idesc,
                               ((g & 15) | kk) ? 1u : 0u);
        }
        if (commit) ptx::mma_commit<1>(side_bar);
      }
      __syncwarp();
    }
    if (ptx::elect_one()) ptx::mma_commit<1>(bar);
    __syncwarp();
    uint64_t t0 = ptx::globaltimer_ns();
    while (!ptx::mbar_try_wait(bar, 0)) {
      if (ptx::globaltimer_ns() - t0 > 4 * WAIT_LIMIT_NS) {
        atomicCAS(status, 0, DEV_TIMEOUT_DRAIN);
        break;
      }
    }
    if (trace && threadIdx.x == 0) {
      trace[static_cast<size_t>(blockIdx.x) * TRACE_SLOTS + TRACE_CYCLES] =
          static_cast<unsigned long long>(clock64() - c0);
      trace[static_cast<size_t>(blockIdx.x) * TRACE_SLOTS + TRACE_NANOS] =
          ptx::globaltimer_ns() - t_begin;
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x < 32) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<1>(tmem_base, 512);
  }
}

}  // namespace b200gemm
