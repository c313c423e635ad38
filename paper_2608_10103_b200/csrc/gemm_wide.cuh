// The large-problem GEMM kernel:  C = A * B^T  with a 512 x 256 tile of C per CTA pair.
//
// Same roles as gemm_kernel (the paper's staged-load -> tensor-core-MMA loop, Sec. III-A,
// Listings 1 and 3, re-cast for Blackwell), different tile: each CTA owns 256 rows of C --
// two 128-row halves -- against the pair's 256 columns, so its two accumulators (128 lanes x
// 256 columns of 32 bits each) fill all of the SM's tensor memory.  Per k-block (128 bytes of
// K) a CTA fetches 256 rows of A and 128 rows of B = 48 KB for 8 MMAs of 256 x 256 x (32 B),
// where the 256 x 256 pair tile fetches 32 KB for 4: a quarter fewer operand bytes per unit
// of math through L2 and the SM's port, which on a power-capped part is what sets the clock
// (measured at N = 8192, FP16: 6.4 instead of 8.6 GB from L2 into the SMs per GEMM).
//
// The price is that no second accumulator is left for the epilogue to overlap with, so the
// hand-over between tiles is made short instead:
//   * the two accumulators are released separately; as soon as the rows of the first one have
//     been read out of tensor memory the MMA issuer starts the next tile on it and runs up to
//     STAGES k-blocks ahead there, and catches up on the second one when that is free;
//   * eight epilogue warps (two per TMEM lane quarter, 128 columns each) read 32 x 32 blocks
//     with tcgen05.ld, turn them through a small swizzled staging buffer of their own and
//     write C with plain 16-byte stores, each warp instruction covering four whole 128-byte
//     pieces of rows -- nothing asynchronous to wait for, so a buffer is reusable at once;
//   * the producer keeps running ahead across the tile boundary, so the ring is full when the
//     MMAs restart.
//
// warp 0: TMA producer; warp 1: MMA issuer (leader CTA) and owner of tensor memory;
// warps 2..9: epilogue.  A: M x K row-major, B: N x K K-major (Listing 2c's ".row.col"),
// C: M x N row-major; tiles outside M, N, K are zero-filled by TMA and clipped by the stores.
#pragma once

#include "gemm_kernel.cuh"

namespace b200gemm {

constexpr int WIDE_STAGES = 4;
constexpr int WIDE_EPI_WARPS = 8;
constexpr int WIDE_THREADS = 64 + 32 * WIDE_EPI_WARPS;
constexpr int WIDE_BN = 256;                 // C columns per tile
constexpr int WIDE_CTA_ROWS = 2 * BM;        // C rows per CTA
constexpr int WIDE_TILE_M = 2 * WIDE_CTA_ROWS;  // C rows per tile (CTA pair)

struct WideSmem {
  static constexpr int A_BYTES = WIDE_CTA_ROWS * BK_BYTES;   // both 128-row halves, 32 KB
  static constexpr int B_BYTES = (WIDE_BN / 2) * BK_BYTES;   // this CTA's half of the B tile
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int RING_BYTES = WIDE_STAGES * STAGE_BYTES;
  static constexpr int EPI_BUF_BYTES = 32 * 128;             // one per epilogue warp
  static constexpr int EPI_OFFSET = RING_BYTES;
  static constexpr int EPI_BYTES = WIDE_EPI_WARPS * EPI_BUF_BYTES;
  static constexpr int BAR_OFFSET = EPI_OFFSET + EPI_BYTES;
  // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain
  static constexpr int NUM_BARS = 2 * WIDE_STAGES + 5;
  static constexpr int MISC_OFFSET = BAR_OFFSET + NUM_BARS * 8;
  static constexpr int TOTAL = MISC_OFFSET + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
  static_assert(DYN_BYTES <= 232448, "exceeds the 227 KB shared-memory limit per CTA");
};

// Writes one staged block (32 rows x 128 bytes at `buf`; 16-byte chunk j of row r sits at
// position j ^ (r & 7)) to global memory at `dst` (row pitch `pitch` bytes): per lane eight
// 16-byte stores, each warp instruction covering four rows x 128 contiguous bytes.
__device__ __forceinline__ void wide_store_block(uint32_t buf, uint8_t* dst, size_t pitch,
                                                 int rows_valid, int bytes_valid, int lane,
                                                 uint64_t policy) {
  const int ch = lane & 7;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 4 + (lane >> 3);
    uint32_t a, b, c, d;
    ptx::ld_shared_v4(buf + static_cast<uint32_t>(r * 128 + ((ch ^ (r & 7)) << 4)), a, b, c, d);
    if (r < rows_valid && ch * 16 < bytes_valid)
      ptx::st_global_v4_hint(dst + static_cast<size_t>(r) * pitch + ch * 16, a, b, c, d, policy);
  }
}

// DBG: the measurement and drill switches of GemmParams::ablate are compiled in.
template <int KIND, int EPI, bool DBG>
__global__ void __launch_bounds__(WIDE_THREADS, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap tmap_a,
                 const __grid_constant__ CUtensorMap tmap_b, const GemmParams p) {
  using L = WideSmem;
  constexpr int STAGES = WIDE_STAGES;
  constexpr int ELEM_BYTES = (KIND == ptx::KIND_F16) ? 2 : 1;
  constexpr int BK_ELEMS = BK_BYTES / ELEM_BYTES;
  constexpr uint32_t TMEM_COLS = 512;
  const int ablate = DBG ? p.ablate : 0;

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
  const uint32_t cta_rank = ptx::cluster_ctarank();
  const bool leader = (cta_rank == 0);
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int k_slots = p.k_blocks;
  const int first_tile = static_cast<int>(blockIdx.x) / 2;
  const int tile_stride = static_cast<int>(gridDim.x) / 2;
  unsigned long long* const trace =
      p.trace ? p.trace + static_cast<size_t>(blockIdx.x) * TRACE_SLOTS : nullptr;
  if (trace && threadIdx.x < TRACE_SLOTS) trace[threadIdx.x] = 0;
  if (threadIdx.x == 0) ptx::grid_dep_launch_dependents();
  const long long clk_start = trace ? clock64() : 0;
  const uint64_t ns_start = trace ? ptx::globaltimer_ns() : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(acc_full_bar(0), 1);
    ptx::mbar_init(acc_full_bar(1), 1);
    ptx::mbar_init(acc_empty_bar(0), 2 * WIDE_EPI_WARPS);
    ptx::mbar_init(acc_empty_bar(1), 2 * WIDE_EPI_WARPS);
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc<2>(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), TMEM_COLS);
    ptx::tmem_relinquish<2>();
  }
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();  // the peer's barriers must exist before anything signals them
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  if (trace && threadIdx.x == 0)
    trace[TRACE_SETUP] = static_cast<unsigned long long>(clock64() - clk_start);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // All lanes walk the loops (warp-uniform state), the lane elected once issues.
    const bool elected = ptx::elect_one();
    if (p.wait_prior_grid) ptx::grid_dep_wait();  // the operands may come from a grid in front
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    long long waited = 0, prod_issue = 0;
    const uint64_t pol_a = p.l2_policy == 0 ? ptx::policy_evict_normal() : ptx::policy_evict_last();
    const uint64_t pol_b = (p.l2_policy == 0 || p.l2_policy == 3) ? ptx::policy_evict_normal()
                           : p.l2_policy == 1                      ? ptx::policy_evict_first()
                                                                   : ptx::policy_evict_last();
    bool backward = false;
    for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
      int tm, tn;
      tile_coords(p, t, tm, tn);
      const int a_row = tm * WIDE_TILE_M + static_cast<int>(cta_rank) * WIDE_CTA_ROWS;
      const int b_row = tn * WIDE_BN + static_cast<int>(cta_rank) * (WIDE_BN / 2);
      for (int ks = 0; ks < k_slots; ++ks) {
        const long long w0 = trace ? clock64() : 0;
        ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
        const long long w9 = trace ? clock64() : 0;
        if (trace) waited += w9 - w0;
        if (!ok) break;
        const uint32_t a_dst = base + stage * L::STAGE_BYTES;
        const uint32_t b_dst = a_dst + L::A_BYTES;
        if (!elected) {
          // nothing to issue in this lane
        } else if (DBG && (ablate & 8) && blockIdx.x == 0 && t == first_tile && ks == 2) {
          // failure drill: this slot is never filled
        } else if (DBG && (ablate & 2)) {
          if (leader) ptx::mbar_arrive(full_bar(stage));
        } else {
          // the bytes of both CTAs are counted on the leader's barrier
          if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), 2 * L::STAGE_BYTES);
          const uint32_t lead_full = ptx::map_to_cta(full_bar(stage), 0);
          const int k0 = (backward ? k_slots - 1 - ks : ks) * BK_ELEMS;
          ptx::tma_load_2d_pair(a_dst, &tmap_a, k0, a_row, lead_full, pol_a);
          ptx::tma_load_2d_pair(b_dst, &tmap_b, k0, b_row, lead_full, pol_b);
        }
        ++issued;
        if (trace) prod_issue += clock64() - w9;
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (p.serpentine_k) backward = !backward;
    }
    if (trace && elected) {
      trace[TRACE_PROD_WAIT] = static_cast<unsigned long long>(waited);
      trace[TRACE_PROD_ISSUE] = static_cast<unsigned long long>(prod_issue);
    }
    if (!ok && elected && leader) {
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
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (p.wait_prior_grid) ptx::grid_dep_wait();  // wait limits count from the predecessor's end
    if (leader) {
      const bool elected = ptx::elect_one();
      constexpr uint32_t idesc = ptx::make_idesc<KIND>(2 * BM, WIDE_BN);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      long long wait_full = 0, wait_acc0 = 0, wait_acc1 = 0, t_issue = 0, t_commit = 0;
      // The four MMAs of one k-block into accumulator `a` (rows a * 128 .. of this CTA's 256).
      auto issue_half = [&](int s, int a, bool first_kblock) {
        const uint32_t a_src = base + s * L::STAGE_BYTES + a * (BM * BK_BYTES);
        const uint64_t a_desc = ptx::smem_desc_sw128(a_src);
        const uint64_t b_desc = ptx::smem_desc_sw128(base + s * L::STAGE_BYTES + L::A_BYTES);
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(a * WIDE_BN);
        if (elected && !(DBG && (ablate & 1))) {
#pragma unroll
          for (int kk = 0; kk < BK_BYTES / MMA_K_BYTES; ++kk) {
            const uint64_t step = static_cast<uint64_t>((kk * MMA_K_BYTES) >> 4);
            ptx::mma_ss<KIND, 2>(d_tmem, a_desc + step, b_desc + step, idesc,
                                 (!first_kblock || kk > 0) ? 1u : 0u);
          }
        }
      };
      auto advance = [&](int& s, uint32_t& ph) {
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      };
      // One pass over `n` consecutive ring slots for accumulator 0 (waiting for their operands),
      // then a second pass over the same slots for accumulator 1, which also frees them.
      // Used at both ends of a tile: at its start accumulator 0 is handed back first and the
      // tensor pipe gets going on it while accumulator 1 is still being read out; at its end
      // accumulator 0 finishes n k-blocks' worth of MMA time before accumulator 1, so its
      // rows are on their way out while the pipe is still busy.
      auto two_pass = [&](int n, bool first_of_tile, bool last_of_tile) {
        int s = stage;
        uint32_t ph = phase;
        for (int i = 0; i < n && ok; ++i) {
          const long long w1 = trace ? clock64() : 0;
          ok = wait_bounded(full_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA);
          const long long w2 = trace ? clock64() : 0;
          if (trace) wait_full += w2 - w1;
          if (!ok) return;
          ptx::tc_fence_after_sync();
          issue_half(s, 0, first_of_tile && i == 0);
          if (trace) t_issue += clock64() - w2;
          advance(s, ph);
        }
        if (last_of_tile && elected) ptx::mma_commit_pair(acc_full_bar(0), 0x3);
        if (first_of_tile) {
          const long long w0 = trace ? clock64() : 0;
          ok = wait_bounded(acc_empty_bar(1), acc_phase ^ 1u, abort_flag, p.status, DEV_TIMEOUT_MMA);
          if (trace) wait_acc1 += clock64() - w0;
          if (!ok) return;
          ptx::tc_fence_after_sync();
        }
        for (int i = 0; i < n; ++i) {
          const long long w2 = trace ? clock64() : 0;
          issue_half(stage, 1, first_of_tile && i == 0);
          const long long w4 = trace ? clock64() : 0;
          if (elected) ptx::mma_commit_pair(empty_bar(stage), 0x3);
          if (trace) {
            t_issue += w4 - w2;
            t_commit += clock64() - w4;
          }
          advance(stage, phase);
        }
        if (last_of_tile && elected) ptx::mma_commit_pair(acc_full_bar(1), 0x3);
      };
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        const long long w0 = trace ? clock64() : 0;
        ok = wait_bounded(acc_empty_bar(0), acc_phase ^ 1u, abort_flag, p.status, DEV_TIMEOUT_MMA);
        if (trace) wait_acc0 += clock64() - w0;
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const int head = k_slots < STAGES ? k_slots : STAGES;
        const int tail = (k_slots - head) < STAGES ? (k_slots - head) : STAGES;
        two_pass(head, true, tail == 0);
        if (!ok) break;
        for (int ks = head; ks < k_slots - tail; ++ks) {
          const long long w1 = trace ? clock64() : 0;
          ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
          const long long w2 = trace ? clock64() : 0;
          if (trace) wait_full += w2 - w1;
          if (!ok) break;
          ptx::tc_fence_after_sync();
          issue_half(stage, 0, false);
          issue_half(stage, 1, false);
          const long long w4 = trace ? clock64() : 0;
          if (elected) ptx::mma_commit_pair(empty_bar(stage), 0x3);
          if (trace) {
            t_issue += w4 - w2;
            t_commit += clock64() - w4;
          }
          advance(stage, phase);
        }
        if (!ok) break;
        if (tail > 0) two_pass(tail, false, true);
        if (!ok) break;
        acc_phase ^= 1u;
      }
      if (trace && elected) {
        trace[TRACE_MMA_WAIT_FULL] = static_cast<unsigned long long>(wait_full);
        trace[TRACE_MMA_WAIT_ACC] = static_cast<unsigned long long>(wait_acc0);
        trace[TRACE_MMA_WAIT_ACC1] = static_cast<unsigned long long>(wait_acc1);
        trace[TRACE_MMA_ISSUE] = static_cast<unsigned long long>(t_issue);
        trace[TRACE_MMA_COMMIT] = static_cast<unsigned long long>(t_commit);
      }
      if (!ok && elected) {
        // Gave up: wait for the MMAs already issued before tensor memory is released.
        ptx::mma_commit<2>(drain_bar);
        uint64_t t0 = ptx::globaltimer_ns();
        while (!ptx::mbar_try_wait(drain_bar, 0) && ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 2;
    const int quarter = warp & 3;   // TMEM lane quarter this warp may read
    const int half = ew >> 2;       // which 128 columns of the tile this warp writes
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t buf = base + L::EPI_OFFSET + static_cast<uint32_t>(ew * L::EPI_BUF_BYTES);
    const uint64_t pol_c = p.c_evict_first ? ptx::policy_evict_first() : ptx::policy_evict_normal();
    constexpr int C_ELEM = (EPI == EPI_OUT16) ? 2 : 4;
    constexpr int BLOCK_COLS = 128 / C_ELEM;  // columns of C in one staged block (128-byte rows)
    constexpr int BLOCKS = 128 / BLOCK_COLS;  // blocks per accumulator for this warp
    const size_t pitch = static_cast<size_t>(p.ldc) * C_ELEM;
    uint32_t acc_phase = 0;
    bool ok = true;
    // wait limits count from the end of the grid in front, which may also still use C and the
    // scale factors
    if (p.wait_prior_grid) ptx::grid_dep_wait();
    bool prior_grid_done = true;
    long long epi_wait = 0, epi_busy = 0, tiles_done = 0;
    for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
      int tm, tn;
      tile_coords(p, t, tm, tn);
      const int cta_row0 = tm * WIDE_TILE_M + static_cast<int>(cta_rank) * WIDE_CTA_ROWS;
      const int col_base = tn * WIDE_BN + half * 128;
      float rs[2] = {1.0f, 1.0f};
      if constexpr (EPI != EPI_RAW32) {
        // scale factors are fetched while the mainloop still runs (they may come from the grid
        // in front, whose end the producer awaits as well before its first load)
        if (p.row_scale || p.col_scale) {
          if (p.wait_prior_grid && !prior_grid_done) {
            ptx::grid_dep_wait();
            prior_grid_done = true;
          }
#pragma unroll
          for (int a = 0; a < 2; ++a) {
            const int row = cta_row0 + a * BM + quarter * 32 + lane;
            if (p.row_scale && row < p.M) rs[a] = ptx::ld_global_f32(p.row_scale + row);
          }
          if (p.col_scale && lane < 4 && col_base + lane * 32 < p.N)
            ptx::prefetch_l1(p.col_scale + col_base + lane * 32);
        }
      }
      long long w1 = 0;
#pragma unroll 1
      for (int a = 0; a < 2; ++a) {
        const int row0 = cta_row0 + a * BM + quarter * 32;
        const int row = row0 + lane;
        const float rs_a = a ? rs[1] : rs[0];
        const uint32_t t_acc = tmem_base + lane_base + static_cast<uint32_t>(a * WIDE_BN + half * 128);
        const long long w0 = trace ? clock64() : 0;
        ok = wait_bounded<true>(acc_full_bar(a), acc_phase, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE,
                                (DBG && (ablate & 4)) ? 500u : 0u);
        ok = __all_sync(0xffffffffu, ok);
        if (trace) {
          const long long now = clock64();
          epi_wait += now - w0;
          if (a == 0) w1 = now;
        }
        if (!ok) break;
        ptx::tc_fence_after_sync();
        if (p.wait_prior_grid && !prior_grid_done) {  // C may still be in use by the grid in front
          ptx::grid_dep_wait();
          prior_grid_done = true;
        }
        // This warp's whole share of the accumulator (its row x 128 columns) goes to registers
        // at once and the accumulator is handed back to the (leader's) MMA issuer before
        // anything is written out: with every CTA of the grid storing its tile at the same
        // moment the stores run at the chip's L2 write rate, several thousand cycles for the
        // tile, and the tensor pipe should not wait for them.
        uint32_t v[4][32];
#pragma unroll
        for (int b = 0; b < 4; ++b) ptx::tmem_ld_32x32b_x32(t_acc + static_cast<uint32_t>(b * 32), v[b]);
        ptx::tmem_wait_ld();
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_remote(ptx::map_to_cta(acc_empty_bar(a), 0));
#pragma unroll
        for (int c = 0; c < BLOCKS; ++c) {
          const int col = col_base + c * BLOCK_COLS;
          uint32_t w[32];  // this thread's 128 bytes of output
          if constexpr (EPI == EPI_RAW32) {
#pragma unroll
            for (int i = 0; i < 32; ++i) w[i] = v[c][i];
          } else if constexpr (EPI == EPI_F32_SCALED) {
            const float cs_mine = (col + lane < p.N) ? ptx::ld_global_f32(p.col_scale + col + lane) : 0.0f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float cs = __shfl_sync(0xffffffffu, cs_mine, i);
              w[i] = __float_as_uint(acc_to_float<KIND>(v[c][i]) * rs_a * cs);
            }
          } else {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int cc = col + h * 32 + lane;
              const float cs_mine = (p.col_scale && cc < p.N) ? ptx::ld_global_f32(p.col_scale + cc) : 0.0f;
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                float x0 = acc_to_float<KIND>(v[2 * c + h][i]);
                float x1 = acc_to_float<KIND>(v[2 * c + h][i + 1]);
                if (p.col_scale) {  // same for the whole warp
                  x0 *= rs_a * __shfl_sync(0xffffffffu, cs_mine, i);
                  x1 *= rs_a * __shfl_sync(0xffffffffu, cs_mine, i + 1);
                }
                w[h * 16 + i / 2] = pack_half2(x0, x1);
              }
            }
          }
          if (p.c_vec_ok) {
            // registers -> swizzled staging -> 16-byte stores, four 128-byte row pieces per
            // warp instruction
#pragma unroll
            for (int j = 0; j < 8; ++j)
              ptx::st_shared_v4(buf + static_cast<uint32_t>(lane * 128 + ((j ^ (lane & 7)) * 16)),
                                w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            __syncwarp();
            if (row0 < p.M && col < p.N) {
              const int bytes_valid = (p.N - col) * C_ELEM;
              wide_store_block(buf, reinterpret_cast<uint8_t*>(p.C) +
                                        (static_cast<size_t>(row0) * p.ldc + col) * C_ELEM,
                               pitch, p.M - row0, bytes_valid, lane, pol_c);
            }
            __syncwarp();  // the buffer is rewritten by the next block
          } else if (row < p.M) {
            // rows of C are not 16-byte multiples: plain predicated stores, one row per thread
            if constexpr (EPI == EPI_OUT16) {
              uint16_t* crow = reinterpret_cast<uint16_t*>(p.C) + static_cast<size_t>(row) * p.ldc;
#pragma unroll
              for (int i = 0; i < BLOCK_COLS; ++i)
                if (col + i < p.N) crow[col + i] = static_cast<uint16_t>(w[i / 2] >> (16 * (i & 1)));
            } else {
              uint32_t* crow = p.C + static_cast<size_t>(row) * p.ldc;
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (col + i < p.N) crow[col + i] = w[i];
            }
          }
        }
      }
      if (!ok) break;
      if (trace) epi_busy += clock64() - w1;
      ++tiles_done;
      acc_phase ^= 1u;
    }
    if (trace && warp == 2 && lane == 0) {
      trace[TRACE_EPI_WAIT] = static_cast<unsigned long long>(epi_wait);
      trace[TRACE_EPI_BUSY] = static_cast<unsigned long long>(epi_busy);
      trace[TRACE_TILES] = static_cast<unsigned long long>(tiles_done);
    }
  }

  // Teardown: every role gets here (all waits are bounded); neither CTA may release tensor
  // memory or exit while the other can still touch its shared memory.
  ptx::tc_fence_before_sync();
  __syncwarp();
  ptx::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<2>(tmem_base, TMEM_COLS);
  }
  if (trace && threadIdx.x == 0) {
    trace[TRACE_CYCLES] = static_cast<unsigned long long>(clock64() - clk_start);
    trace[TRACE_NANOS] = ptx::globaltimer_ns() - ns_start;
  }
}

}  // namespace b200gemm
