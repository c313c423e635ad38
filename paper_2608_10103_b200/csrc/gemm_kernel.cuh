// Persistent, warp-specialised GEMM kernel for sm_100a:  C = A * B^T.
//
// Roles of the paper's double/triple-buffered cp.async -> ldmatrix -> mma.sync
// loop (Sec. III-A, Listings 1 and 3), re-cast for Blackwell:
//
//   warp 0, one lane   : TMA producer.  One tensor copy per operand per
//                        k-block lands a 128 x 128-byte A tile and a
//                        B_ROWS x 128-byte B tile (128-byte swizzle) in a ring
//                        of STAGES shared-memory slots; completion is counted
//                        in bytes on the slot's `full` mbarrier.
//   warp 1, one lane   : MMA issuer.  Waits `full`, issues 4 tcgen05.mma
//                        (each consumes 32 bytes of K) accumulating into one of
//                        two TMEM accumulator buffers, then commits to the
//                        slot's `empty` barrier so the producer may refill it.
//   warps 2..5         : epilogue.  Wait for the accumulator buffer, read it
//                        with tcgen05.ld (one TMEM lane = one C row per
//                        thread), write C, hand the buffer back.  This overlaps
//                        the next tile's mainloop.
//
// CTA_GROUP = 1: one CTA owns a 128 x BN tile of C.
// CTA_GROUP = 2: a cluster of two CTAs owns a 256 x BN tile.  Each CTA loads its
//   own 128 rows of A and HALF of the B tile (BN/2 rows); the leader CTA (cluster
//   rank 0) issues tcgen05.mma.cta_group::2, which feeds both tensor cores from
//   both halves, and each CTA ends up with its 128 rows of the accumulator in its
//   own TMEM.  Per SM this halves the B bytes fetched from L2 per unit of math.
//   Both producers count their bytes on the leader's `full` barrier; the leader's
//   commits signal `empty` / `acc_full` in both CTAs; both epilogues report to the
//   leader's `acc_empty`.
//
// A is M x K row-major, B is N x K with K contiguous (the paper's ".row.col"
// operand layout, Listing 2c); C is M x N row-major, 32-bit, overwritten.
// Tiles outside M, N or K are zero-filled by the TMA loads and clipped by the
// stores, so no dimension needs to be a tile multiple.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace b200gemm {

constexpr int BM = 128;           // C rows per CTA (= TMEM lanes)
constexpr int BK_BYTES = 128;     // K extent of one pipeline slot, in bytes (one swizzle row)
constexpr int MMA_K_BYTES = 32;   // K extent of one tcgen05.mma, in bytes
constexpr int NUM_THREADS = 192;  // 6 warps: producer, MMA, 4 x epilogue
constexpr int EPI_WARPS = 4;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // every barrier wait gives up after 2 s

// Device status codes written to the status word when a wait gives up.
enum DeviceStatus {
  DEV_OK = 0,
  DEV_TIMEOUT_PRODUCER = 1,
  DEV_TIMEOUT_MMA = 2,
  DEV_TIMEOUT_EPILOGUE = 3,
  DEV_TIMEOUT_DRAIN = 4,
};

struct GemmParams {
  int M, N, K;
  int tiles_m, tiles_n;  // number of C tiles (128*CTA_GROUP x BN) along M and N
  int group_m;           // raster: tiles are walked in bands of `group_m` tile rows
  int k_blocks;          // ceil(K bytes / BK_BYTES)
  int c_vec_ok;          // 1 if C rows allow 16-byte vector stores (N % 4 == 0, base aligned)
  uint32_t* C;
  int* status;           // device status word (0 = ok)
};

template <int BN, int STAGES, int CTA_GROUP>
struct SmemLayout {
  static constexpr int B_ROWS = BN / CTA_GROUP;  // B rows each CTA loads
  static constexpr int A_BYTES = BM * BK_BYTES;
  static constexpr int B_BYTES = B_ROWS * BK_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int RING_BYTES = STAGES * STAGE_BYTES;
  static constexpr int BAR_OFFSET = RING_BYTES;
  // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain
  static constexpr int NUM_BARS = 2 * STAGES + 5;
  static constexpr int MISC_OFFSET = BAR_OFFSET + NUM_BARS * 8;
  static constexpr int TOTAL = MISC_OFFSET + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack to align the ring to 1024 bytes
  static_assert(B_BYTES % 1024 == 0, "B tile must keep the next slot 1024-byte aligned");
  static_assert(DYN_BYTES <= 232448, "exceeds the 227 KB shared-memory limit per CTA");
};

// Bounded wait: polls the barrier; after the limit (or once another role has
// given up) records `code` and returns false.  The caller then leaves its loop.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity,
                                             volatile uint32_t* abort_flag, int* status, int code) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  uint64_t t0 = 0;
  uint32_t spins = 0;
  while (true) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return false;
      uint64_t now = ptx::globaltimer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}

// Tile index -> (tile row, tile column).  Tiles are numbered down bands of
// `group_m` tile rows so that the CTAs running at the same time share A rows
// and B rows in L2.
__device__ __forceinline__ void tile_coords(const GemmParams& p, int t, int& tm, int& tn) {
  const int band_tiles = p.group_m * p.tiles_n;
  const int band = t / band_tiles;
  const int first_m = band * p.group_m;
  const int rows_in_band = min(p.group_m, p.tiles_m - first_m);
  const int r = t - band * band_tiles;
  tm = first_m + r % rows_in_band;
  tn = r / rows_in_band;
}

template <int KIND, int BN, int STAGES, int CTA_GROUP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const GemmParams p) {
  using L = SmemLayout<BN, STAGES, CTA_GROUP>;
  constexpr int ELEM_BYTES = (KIND == ptx::KIND_F16) ? 2 : 1;
  constexpr int BK_ELEMS = BK_BYTES / ELEM_BYTES;
  constexpr int TILE_M = BM * CTA_GROUP;
  constexpr uint32_t TMEM_COLS = (2 * BN <= 32) ? 32 : 2 * BN;  // two accumulator buffers
  static_assert(CTA_GROUP == 1 || CTA_GROUP == 2, "CTA_GROUP is 1 or 2");
  static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "BN must be a multiple of 32 up to 256");
  static_assert((TMEM_COLS & (TMEM_COLS - 1)) == 0 && TMEM_COLS <= 512, "TMEM columns: power of 2");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_addr(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);

  const uint32_t bar0 = base + L::BAR_OFFSET;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto acc_empty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * STAGES + 4);
  volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(base_ptr + L::MISC_OFFSET);
  volatile uint32_t* abort_flag = tmem_holder + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (CTA_GROUP == 2) ? ptx::cluster_ctarank() : 0u;
  const bool leader = (cta_rank == 0);
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int first_tile = static_cast<int>(blockIdx.x) / CTA_GROUP;
  const int tile_stride = static_cast<int>(gridDim.x) / CTA_GROUP;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(acc_full_bar(a), 1);
      ptx::mbar_init(acc_empty_bar(a), EPI_WARPS * CTA_GROUP);
    }
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc<CTA_GROUP>(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), TMEM_COLS);
    ptx::tmem_relinquish<CTA_GROUP>();
  }
  ptx::tc_fence_before_sync();
  if constexpr (CTA_GROUP == 2) {
    ptx::cluster_sync();  // the peer's barriers must exist before anything signals them
  } else {
    __syncthreads();
  }
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        int tm, tn;
        tile_coords(p, t, tm, tn);
        const int a_row = tm * TILE_M + static_cast<int>(cta_rank) * BM;
        const int b_row = tn * BN + static_cast<int>(cta_rank) * L::B_ROWS;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status,
                            DEV_TIMEOUT_PRODUCER);
          if (!ok) break;
          const uint32_t a_dst = base + stage * L::STAGE_BYTES;
          const uint32_t b_dst = a_dst + L::A_BYTES;
          if constexpr (CTA_GROUP == 1) {
            ptx::mbar_arrive_expect_tx(full_bar(stage), L::STAGE_BYTES);
            ptx::tma_load_2d(a_dst, &tmap_a, kb * BK_ELEMS, a_row, full_bar(stage));
            ptx::tma_load_2d(b_dst, &tmap_b, kb * BK_ELEMS, b_row, full_bar(stage));
          } else {
            // Bytes of both CTAs are counted on the leader's barrier.
            if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), 2 * L::STAGE_BYTES);
            const uint32_t lead_full = ptx::map_to_cta(full_bar(stage), 0);
            ptx::tma_load_2d_pair(a_dst, &tmap_a, kb * BK_ELEMS, a_row, lead_full);
            ptx::tma_load_2d_pair(b_dst, &tmap_b, kb * BK_ELEMS, b_row, lead_full);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && (CTA_GROUP == 1 || leader)) {
        // Gave up: let the copies already in flight land before the CTA exits.
        int n = issued < STAGES ? issued : STAGES;
        for (int i = 0; i < n; ++i) {
          if (--stage < 0) { stage = STAGES - 1; phase ^= 1u; }
          uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(full_bar(stage), phase) &&
                 ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = ptx::make_idesc<KIND>(TILE_M, BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        ok = wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status,
                          DEV_TIMEOUT_MMA);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t a_src = base + stage * L::STAGE_BYTES;
          const uint64_t a_desc = ptx::smem_desc_sw128(a_src);
          const uint64_t b_desc = ptx::smem_desc_sw128(a_src + L::A_BYTES);
#pragma unroll
          for (int kk = 0; kk < BK_BYTES / MMA_K_BYTES; ++kk) {
            const uint64_t step = static_cast<uint64_t>((kk * MMA_K_BYTES) >> 4);
            ptx::mma_ss<KIND, CTA_GROUP>(d_tmem, a_desc + step, b_desc + step, idesc,
                                         (kb > 0 || kk > 0) ? 1u : 0u);
          }
          if constexpr (CTA_GROUP == 1) {
            ptx::mma_commit<1>(empty_bar(stage));
          } else {
            ptx::mma_commit_pair(empty_bar(stage), 0x3);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if constexpr (CTA_GROUP == 1) {
          ptx::mma_commit<1>(acc_full_bar(acc));
        } else {
          ptx::mma_commit_pair(acc_full_bar(acc), 0x3);
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (!ok) {
        // Gave up: wait for the MMAs already issued before TMEM is released.
        ptx::mma_commit<CTA_GROUP>(drain_bar);
        uint64_t t0 = ptx::globaltimer_ns();
        while (!ptx::mbar_try_wait(drain_bar, 0) && ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;  // TMEM lane quarter this warp may read
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
      int tm, tn;
      tile_coords(p, t, tm, tn);
      ok = wait_bounded(acc_full_bar(acc), acc_phase, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const int row = tm * TILE_M + static_cast<int>(cta_rank) * BM + quarter * 32 + lane;
      const int col0 = tn * BN;
      uint32_t* crow = p.C + static_cast<size_t>(row) * p.N;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        ptx::tmem_ld_32x32b_x32(tmem_base + lane_base + static_cast<uint32_t>(acc * BN + c * 32),
                                r);
        ptx::tmem_wait_ld();
        const int col = col0 + c * 32;
        if (row < p.M) {
          if (p.c_vec_ok && col + 32 <= p.N) {
            uint4* dst = reinterpret_cast<uint4*>(crow + col);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              dst[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          } else {
#pragma unroll
            for (int v = 0; v < 32; ++v)
              if (col + v < p.N) crow[col + v] = r[v];
          }
        }
      }
      // Hand the accumulator buffer back to the (leader's) MMA issuer.
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if constexpr (CTA_GROUP == 1) {
          ptx::mbar_arrive(acc_empty_bar(acc));
        } else {
          ptx::mbar_arrive_cluster(ptx::map_to_cta(acc_empty_bar(acc), 0));
        }
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  // Teardown: every role gets here (all waits are bounded).  In a pair neither
  // CTA may release TMEM or exit while the other can still touch its memory.
  ptx::tc_fence_before_sync();
  if constexpr (CTA_GROUP == 2) {
    __syncwarp();
    ptx::cluster_sync();
  } else {
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<CTA_GROUP>(tmem_base, TMEM_COLS);
  }
}

}  // namespace b200gemm
