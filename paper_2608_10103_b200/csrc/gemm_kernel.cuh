// Persistent, warp-specialised GEMM kernel for sm_100a:  C = A * B^T.
//
// Roles of the paper's double/triple-buffered cp.async -> ldmatrix -> mma.sync
// loop (Sec. III-A, Listings 1 and 3), re-cast for Blackwell:
//
//   warp 0             : TMA producer (all lanes walk the loops, one elected lane
//                        issues).  One tensor copy per operand per k-block lands a
//                        128 x 128-byte A tile and a B_ROWS x 128-byte B tile
//                        (128-byte swizzle) in a ring of STAGES shared-memory
//                        slots; completion is counted in bytes on the slot's
//                        `full` mbarrier.
//   warp 1             : MMA issuer (likewise).  Waits `full`, issues 4 tcgen05.mma
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
// PSTAGES > 0 (fused INT4): A and B hold packed signed 4-bit values (Listing 2c's s4
//   operands).  The producer lands PACKED tiles (rows x 128 bytes = 256 nibbles of K) in a
//   second ring of PSTAGES slots; warps 6..13 expand each packed slot into two int8 slots of
//   the ring the MMA issuer reads, every value multiplied by 16 (nibble moved to the high
//   half of its byte, low half zero), so the accumulators hold 256 * C and the epilogue
//   shifts them right by 8, exactly.  The order in which K values land in the int8 slots
//   differs from their order in memory, identically for A and B, which leaves every dot
//   product unchanged.
//   A8 (fused INT4, hybrid): only B arrives packed.  A is an int8 image made beforehand by a
//   small pre-pass in exactly the form the expansion produces (16 * value, the same order of
//   K inside a packed slot).  Its 128-byte atoms have a ring of their own, filled by a warp of
//   its own (warp 14) as soon as the MMAs release a slot, so that the loads run a full ring
//   ahead of the MMAs; the int8 ring the expansion warps fill then holds B only.  The short
//   operand of a problem with M << N is otherwise expanded again for every tile column; this
//   halves the expansion work and takes a sixth off the shared-memory traffic that bounds
//   the fused kernel.
//
// A is M x K row-major, B is N x K with K contiguous (the paper's ".row.col"
// operand layout, Listing 2c); C is M x N row-major, 32-bit, overwritten.
// Tiles outside M, N or K are zero-filled by the TMA loads and clipped by the
// stores, so no dimension needs to be a tile multiple.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"
#include "s4_ahead.cuh"

namespace b200gemm {

constexpr int BM = 128;           // C rows per CTA (= TMEM lanes)
constexpr int BK_BYTES = 128;     // K extent of one pipeline slot, in bytes (one swizzle row)
constexpr int MMA_K_BYTES = 32;   // K extent of one tcgen05.mma, in bytes
constexpr int NUM_THREADS = 192;  // 6 warps: producer, MMA, 4 x epilogue
constexpr int EPI_WARPS = 4;
constexpr int UNPACK_WARPS = 8;   // fused INT4 only: warps 6..13
constexpr int NUM_THREADS_FUSED = NUM_THREADS + 32 * UNPACK_WARPS;
constexpr int NUM_THREADS_FUSED_A8 = NUM_THREADS_FUSED + 32;  // hybrid: warp 14 fetches the A image
constexpr int AHEAD_WARPS = 4;    // overlapped INT4 pre-pass only: warps 6..9
constexpr int NUM_THREADS_AHEAD = NUM_THREADS + 32 * AHEAD_WARPS;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;  // every barrier wait gives up after 2 s

// Device status codes written to the status word when a wait gives up.
enum DeviceStatus {
  DEV_OK = 0,
  DEV_TIMEOUT_PRODUCER = 1,
  DEV_TIMEOUT_MMA = 2,
  DEV_TIMEOUT_EPILOGUE = 3,
  DEV_TIMEOUT_DRAIN = 4,
  DEV_TIMEOUT_UNPACK = 5,
};

// What the epilogue writes.
enum EpiMode {
  EPI_RAW32 = 0,       // the 32-bit accumulators as they are (FP32 resp. INT32)
  EPI_OUT16 = 1,       // binary16: FP32 accumulators rounded once (RNE); INT32 accumulators
                       // converted to float and multiplied by row_scale[i] * col_scale[j] first
  EPI_F32_SCALED = 2,  // float(INT32 accumulator) * row_scale[i] * col_scale[j]
};

struct GemmParams {
  int M, N, K;
  int tiles_m, tiles_n;  // number of C tiles (128*CTA_GROUP x BN) along M and N
  int group_m;           // raster: tiles are walked in bands of `group_m` tile rows
  int k_blocks;          // ceil(K bytes / BK_BYTES): 128-byte K atoms to cover K
  int splits;            // split-K: each C tile from `split_from` on is computed by `splits` work
                         // units over disjoint K ranges and ADDED into a zeroed C (EPI_RAW32
                         // only); 1 = off
  int split_from;        // first split tile in raster order: 0 splits every tile (few tiles, long
                         // K); tiles - r splits only the last, partly filled wave of tiles
  int c_vec_ok;          // 1 if C rows allow 16-byte accesses (N % 4 == 0, base 16-byte aligned):
                         // the epilogue then stages C in shared memory and stores it by TMA
  uint32_t* C;           // element size 4 bytes, or 2 with EPI_OUT16
  long long ldc;         // row pitch of C in elements (N for a dense C)
  // Even shares (0 = off; split-K through C only): the tiles' K ranges, laid end to end and
  // counted in granules of one ring slot (fused INT4: one packed slot = two), are cut into
  // contiguous shares of sk_share granules, one per CTA; a share covers the end of one tile,
  // whole tiles, and the beginning of another, and every piece is ADDED into the zeroed C.
  // Fills all SMs with equal work whatever the tile count (64 tiles x 2 halves occupy 128 of
  // 148 SMs; 224 tiles make the busiest SM do two where the average is 1.5).
  int sk_share;
  long long sk_total;
  // 1: the caller's A and B have changed places (the kernel's rows are the caller's columns), so
  // element (row, col) of the kernel's result belongs at C[col * ldc + row].  Used for problems
  // with few rows: the long operand then fills the 128-row side of the tile, and a warp's 32
  // lanes (32 consecutive kernel rows) store 32 consecutive elements of a row of C.  Always
  // with c_vec_ok = 0 (plain stores).
  int transpose_c;
  // 1: this grid was launched to start before the grid in front of it in the stream has
  // drained (programmatic dependent launch): its set-up overlaps that grid's tail, and whoever
  // touches global memory (the producer before its first load, the epilogue before its first
  // store) waits for that grid first.  In front may be another GEMM of this library or the
  // kernel that zeroes C for split-K, both of which let their successor start as soon as they
  // run themselves (and wait for their own predecessor in the same way).
  int wait_prior_grid;
  const float* row_scale;  // EPI_OUT16 (integer kinds) / EPI_F32_SCALED: M per-row factors
  const float* col_scale;  // and N per-column factors; both null = no scaling (FP16 kind)
  int* status;           // device status word (0 = ok)
  // Optional per-CTA cycle accounting (TRACE_SLOTS 64-bit words per CTA), or null.
  unsigned long long* trace;
  // L2 eviction priority of the operand loads: 0 = normal for both; 1 = keep A (evict last),
  // stream B (evict first); 2 = keep both; 3 = keep A, B normal.
  int l2_policy;
  int c_evict_first;     // 1: C stores are marked evict-first (written once, never re-read)
  // 1: successive tiles of a CTA walk K in opposite directions, so a tile starts on the
  // K range its predecessor (same A rows) touched last and finds it still in L2.
  int serpentine_k;
  // Ablation switches for cycle accounting runs (results are then meaningless):
  // bit 0 = issue no MMAs (loads + barriers only), bit 1 = issue no loads (MMAs + barriers only),
  // bit 4 = epilogue stores C straight from registers (no staging, no TMA store), bit 5 = the
  // same from the 16x256b TMEM load shape, whole 32-byte sectors per four threads,
  // bit 2 = epilogue waits back off with nanosleep, bit 3 = host-requested failure drill: the
  // producer of CTA 0 leaves out the 3rd ring slot of its first tile, so the consumers' bounded
  // waits must expire, record a status code and let the kernel drain and return.
  int ablate;
  // Overlapped INT4 pre-pass (kernel variants built with AHEAD): the int8 operands this GEMM
  // reads are produced by four extra warps of its own CTAs from the packed ones named here.
  S4Ahead ahead;
};

// Trace slots written per CTA when GemmParams::trace is set.
enum TraceSlot {
  TRACE_CYCLES = 0,         // SM cycles from kernel start to teardown
  TRACE_NANOS = 1,          // the same interval in ns of %globaltimer
  TRACE_PROD_WAIT = 2,      // producer: cycles waiting for a free slot
  TRACE_MMA_WAIT_FULL = 3,  // MMA issuer: cycles waiting for operands
  TRACE_MMA_WAIT_ACC = 4,   // MMA issuer: cycles waiting for a free accumulator buffer
  TRACE_EPI_WAIT = 5,       // epilogue warp 2: cycles waiting for a finished accumulator
  TRACE_EPI_BUSY = 6,       // epilogue warp 2: cycles draining accumulators
  TRACE_TILES = 7,          // tiles this CTA worked on
  TRACE_MMA_ISSUE = 8,      // MMA issuer: cycles inside the tcgen05.mma issue instructions
  TRACE_MMA_COMMIT = 9,     // MMA issuer: cycles inside tcgen05.commit
  TRACE_SETUP = 10,         // cycles from kernel start until barriers and TMEM are set up
  TRACE_PROD_ISSUE = 11,    // producer: cycles issuing expect_tx + TMA loads
  TRACE_UNPACK_WAIT_IN = 12,   // fused INT4, unpack warp 6: cycles waiting for packed operands
  TRACE_UNPACK_WAIT_OUT = 13,  // ... waiting for a free int8 slot
  TRACE_UNPACK_BUSY = 14,      // ... expanding nibbles
  TRACE_MMA_WAIT_ACC1 = 15,    // wide kernel: MMA issuer waiting for the tile's second accumulator;
                               // hybrid fused INT4: the part of [3] spent waiting for the A atom
  TRACE_SLOTS = 16
};

// One ring slot holds KB "atoms" per operand; an atom is a tile of rows x 128
// bytes of K in the 128-byte-swizzle layout (the widest a swizzled TMA box can
// be).  KB = 2 halves the per-slot barrier work (one wait, one commit per 8 MMAs)
// of the single issuing thread, whose instruction time is the scarce resource.
template <int BN, int STAGES, int CTA_GROUP, int KB, int PSTAGES = 0, int CSPLIT = 1, bool A8 = false>
struct SmemLayout {
  static constexpr int B_ROWS = BN / CTA_GROUP;  // B rows each CTA loads
  static constexpr int A_BYTES = BM * BK_BYTES;       // one A atom
  static constexpr int B_BYTES = B_ROWS * BK_BYTES;   // one B atom
  // (hybrid fused INT4, A8: the slots of this ring hold B only; A has the ring below)
  static constexpr int STAGE_BYTES = A8 ? B_BYTES : KB * (A_BYTES + B_BYTES);
  // Fused INT4: PSTAGES more slots, each one packed atom per operand (256 nibbles of K per row).
  // (hybrid: only B is packed, see A8 in the kernel's head comment)
  static constexpr int P_STAGE_BYTES = (A8 ? 0 : A_BYTES) + B_BYTES;
  static constexpr int P_OFFSET = STAGES * STAGE_BYTES;
  // hybrid: ring of A atoms (int8 image), as many as fit beside the other two rings
  static constexpr int A8_STAGES = A8 ? (BN >= 256 ? 4 : 6) : 0;
  static constexpr int A8_OFFSET = P_OFFSET + PSTAGES * P_STAGE_BYTES;
  static constexpr int RING_BYTES = STAGES * STAGE_BYTES + PSTAGES * P_STAGE_BYTES + A8_STAGES * A_BYTES;
  // Epilogue staging: per epilogue warp two buffers of 32 rows x 128 bytes (32 x 32 C values).
  static constexpr int EPI_BUF_BYTES = 32 * 128;
  static constexpr int EPI_OFFSET = RING_BYTES;
  static constexpr int EPI_BYTES = EPI_WARPS * 2 * EPI_BUF_BYTES;
  // Cluster split-K: the CTA of cluster rank 0 receives the other CTAs' 128 x BN partial
  // accumulators (32-bit) here, one buffer per sender.
  static constexpr int X_OFFSET = EPI_OFFSET + EPI_BYTES;
  static constexpr int X_PEER_BYTES = BM * BN * 4;  // one buffer per contributing CTA
  static constexpr int X_BYTES = CSPLIT > 1 ? (CSPLIT - 1) * X_PEER_BYTES : 0;
  static constexpr int BAR_OFFSET = X_OFFSET + X_BYTES;
  // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], drain, p_full[PSTAGES], p_empty[PSTAGES]
  // fused INT4 adds ready[STAGES], its hybrid form a_full[A8_STAGES], a_empty[A8_STAGES];
  // cluster split-K adds part_full, part_free (last two)
  static constexpr int NUM_BARS = 2 * STAGES + 5 + 2 * PSTAGES + (PSTAGES > 0 ? STAGES : 0) +
                                  2 * A8_STAGES + (CSPLIT > 1 ? 2 : 0);
  static constexpr int MISC_OFFSET = BAR_OFFSET + NUM_BARS * 8;
  static constexpr int TOTAL = MISC_OFFSET + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack to align the ring to 1024 bytes
  static_assert(B_BYTES % 1024 == 0, "B tile must keep the next slot 1024-byte aligned");
  static_assert(DYN_BYTES <= 232448, "exceeds the 227 KB shared-memory limit per CTA");
};

// Bounded wait: polls the barrier; after the limit (or once another role has
// given up) records `code` and returns false.  The caller then leaves its loop.
template <bool BACKOFF = false>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity,
                                             volatile uint32_t* abort_flag, int* status, int code,
                                             uint32_t backoff_ns = 0) {
  auto done = [&]() { return ptx::mbar_try_wait(bar, parity); };
  if (done()) return true;
  uint64_t t0 = 0;
  uint32_t spins = 0;
  while (true) {
    if (done()) return true;
    if (BACKOFF && backoff_ns) __nanosleep(backoff_ns);
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

// Accumulator bits -> output value as float (identity for raw mode is handled by the caller).
template <int KIND>
__device__ __forceinline__ float acc_to_float(uint32_t bits) {
  if constexpr (KIND == ptx::KIND_F16) return __uint_as_float(bits);
  return static_cast<float>(static_cast<int32_t>(bits));
}

__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// DBG: the measurement and drill switches of GemmParams::ablate are compiled in (the product
// instantiations leave them out of their loops).
template <int KIND, int BN, int STAGES, int CTA_GROUP, int KB, int EPI = EPI_RAW32, int PSTAGES = 0,
          int CSPLIT = 1, bool DBG = false, bool AHEAD = false, bool A8 = false>
__global__ void __launch_bounds__(A8 ? NUM_THREADS_FUSED_A8
                                     : PSTAGES > 0 ? NUM_THREADS_FUSED : (AHEAD ? NUM_THREADS_AHEAD : NUM_THREADS), 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
  using L = SmemLayout<BN, STAGES, CTA_GROUP, KB, PSTAGES, CSPLIT, A8>;
  constexpr bool FUSED = PSTAGES > 0;  // packed INT4 operands, expanded on the way to the MMAs
  static_assert(!A8 || (PSTAGES > 0 && CSPLIT == 1 && !DBG), "hybrid: a fused INT4 variant");
  const int ablate = DBG ? p.ablate : 0;
  // fused INT4: the expansion warps work as one group of eight, or -- where both rings are at
  // least four slots deep -- as two groups of four on alternate packed slots
  constexpr int UNPACK_GROUPS = (STAGES >= 4 && PSTAGES >= 4) ? 2 : 1;
  constexpr int GROUP_WARPS = UNPACK_WARPS / UNPACK_GROUPS;
  // CSPLIT = 2 or 4 (cluster split-K): a cluster of CSPLIT single CTAs owns every tile; each
  // takes its share of K into its own accumulator, the CTAs of rank 1.. hand their 128 x BN
  // partial sums to rank 0 through the cluster's shared-memory window (one buffer each), and
  // rank 0 adds them to its own on the way out.  Unlike split-K through C this needs no zeroed C and no adds in global memory, so it
  // also serves the 16-bit and scaled outputs, and a call is a single launch.
  static_assert(CSPLIT == 1 || ((CSPLIT == 2 || CSPLIT == 4) && CTA_GROUP == 1 && BN <= 64),
                "cluster split-K: two or four single CTAs, narrow tile");
  static_assert(!AHEAD || (KIND == ptx::KIND_I8 && !FUSED && KB == 1 && CSPLIT == 1),
                "overlapped INT4 pre-pass: the plain int8 kernel, one atom per slot");
  static_assert(!FUSED || (KIND == ptx::KIND_I8 && KB == 1 && STAGES >= 2),
                "fused INT4: int8 MMAs, one atom per slot, a packed slot fills two int8 slots at once");
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
  auto p_full_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 5 + s); };
  auto p_empty_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 5 + PSTAGES + s); };
  // fused INT4: int8 slot s of THIS CTA has been written by all its unpack warps.  The leader's
  // MMA issuer waits for its own `ready` and, in a pair, for `full`, on which the peer's
  // otherwise idle warp 1 relays the peer's `ready` (one remote arrive per slot: a remote
  // arrive with release semantics straight from the writing warps costs each of them
  // hundreds of cycles).
  auto ready_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 5 + 2 * PSTAGES + s); };
  // hybrid: slot s of the A ring holds its atom (both CTAs' bytes are counted on the leader's) /
  // the MMAs that read it have retired
  auto a_full_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 5 + 2 * PSTAGES + STAGES + s); };
  auto a_empty_bar = [&](int s) {
    return bar0 + 8u * (2 * STAGES + 5 + 2 * PSTAGES + STAGES + L::A8_STAGES + s);
  };
  // cluster split-K: `part_full` lives in rank 0 (the other ranks' partial sums of a tile have
  // all landed), `part_free` in every other rank (rank 0 has consumed them, the buffer may be
  // overwritten)
  const uint32_t part_full_bar = bar0 + 8u * (L::NUM_BARS - 2);
  const uint32_t part_free_bar = bar0 + 8u * (L::NUM_BARS - 1);
  volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(base_ptr + L::MISC_OFFSET);
  volatile uint32_t* abort_flag = tmem_holder + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (CTA_GROUP == 2) ? ptx::cluster_ctarank() : 0u;
  const bool leader = (cta_rank == 0);
  const uint32_t krank = (CSPLIT > 1) ? ptx::cluster_ctarank() : 0u;  // which part of K this CTA takes
  // Work units (`num_tiles` counts units): unit u < split_from is the whole tile u; the
  // remaining tiles are each covered by `splits` units, one per K range.
  const int real_tiles = p.tiles_m * p.tiles_n;
  const int split_tiles = real_tiles - p.split_from;
  const int k_slots_all = (p.k_blocks + KB - 1) / KB;  // ring slots per tile; a K tail is zero-filled
  // even shares: this CTA's (CTA pair's) contiguous range of granules and the pieces it is cut into
  constexpr int SK_GRAN = FUSED ? 2 : 1;          // ring slots per granule
  const int sk_tile = k_slots_all / SK_GRAN;      // granules per tile (fused INT4: k_slots_all is even)
  const bool sk_on = CSPLIT == 1 && p.sk_share > 0;
  const long long sk_begin =
      sk_on ? static_cast<long long>(blockIdx.x / CTA_GROUP) * p.sk_share : 0;
  const long long sk_end =
      sk_on ? (sk_begin + p.sk_share < p.sk_total ? sk_begin + p.sk_share : p.sk_total) : 0;
  const int sk_pieces =
      sk_begin < sk_end ? static_cast<int>((sk_end - 1) / sk_tile - sk_begin / sk_tile) + 1 : 0;
  const int num_tiles = sk_on ? sk_pieces : p.split_from + split_tiles * p.splits;
  // (fused INT4: K is split in whole packed slots = pairs of int8 slots)
  const int k_per_split = FUSED ? 2 * ((k_slots_all / 2 + p.splits - 1) / p.splits)
                                : (k_slots_all + p.splits - 1) / p.splits;
  // unit -> tile, K range (in ring slots) and whether its result is added into C
  auto decode_unit = [&](int u, int& tile, int& k_begin, int& k_end, bool& add) {
    if constexpr (CSPLIT > 1) {  // every unit is a whole tile; K is divided inside the cluster
      // (fused INT4: in whole packed slots = pairs of int8 slots)
      const int per = FUSED ? 2 * ((k_slots_all / 2 + CSPLIT - 1) / CSPLIT)
                            : (k_slots_all + CSPLIT - 1) / CSPLIT;
      tile = u;
      k_begin = static_cast<int>(krank) * per;
      k_end = min(k_begin + per, k_slots_all);
      add = false;
    } else if (sk_on) {
      const int first = static_cast<int>(sk_begin / sk_tile), last = static_cast<int>((sk_end - 1) / sk_tile);
      tile = first + u;
      k_begin = (u == 0 ? static_cast<int>(sk_begin - static_cast<long long>(first) * sk_tile) : 0) * SK_GRAN;
      k_end = (tile == last ? static_cast<int>(sk_end - static_cast<long long>(last) * sk_tile) : sk_tile) * SK_GRAN;
      add = true;
    } else if (u < p.split_from) {
      tile = u;
      k_begin = 0;
      k_end = k_slots_all;
      add = false;
    } else {
      const int r = u - p.split_from;
      tile = p.split_from + r % split_tiles;
      k_begin = (r / split_tiles) * k_per_split;
      k_end = min(k_begin + k_per_split, k_slots_all);
      add = p.splits > 1;
    }
  };
  const int first_tile = sk_on ? 0 : static_cast<int>(blockIdx.x) / (CTA_GROUP * CSPLIT);
  const int tile_stride = sk_on ? 1 : static_cast<int>(gridDim.x) / (CTA_GROUP * CSPLIT);
  unsigned long long* const trace =
      p.trace ? p.trace + static_cast<size_t>(blockIdx.x) * TRACE_SLOTS : nullptr;
  if (trace && threadIdx.x < TRACE_SLOTS) trace[threadIdx.x] = 0;  // roles that do not run leave 0
  if (threadIdx.x == 0) ptx::grid_dep_launch_dependents();  // a following GEMM may set up now
  const long long clk_start = trace ? clock64() : 0;
  const uint64_t ns_start = trace ? ptx::globaltimer_ns() : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
      if constexpr (FUSED) ptx::mbar_init(ready_bar(s), GROUP_WARPS);
    }
    for (int s = 0; s < L::A8_STAGES; ++s) {
      ptx::mbar_init(a_full_bar(s), 1);
      ptx::mbar_init(a_empty_bar(s), 1);
    }
    for (int s = 0; s < PSTAGES; ++s) {
      ptx::mbar_init(p_full_bar(s), 1);
      ptx::mbar_init(p_empty_bar(s), GROUP_WARPS);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(acc_full_bar(a), 1);
      ptx::mbar_init(acc_empty_bar(a), EPI_WARPS * CTA_GROUP);
    }
    ptx::mbar_init(drain_bar, 1);
    if constexpr (CSPLIT > 1) {
      ptx::mbar_init(part_full_bar, 1);  // rank 0's own announcement; the rest is a byte count
      ptx::mbar_init(part_free_bar, EPI_WARPS);
    }
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
    ptx::prefetch_tensormap(&tmap_c);
  }
  if (warp == 1) {
    ptx::tmem_alloc<CTA_GROUP>(ptx::smem_addr(const_cast<uint32_t*>(tmem_holder)), TMEM_COLS);
    ptx::tmem_relinquish<CTA_GROUP>();
  }
  ptx::tc_fence_before_sync();
  if constexpr (CTA_GROUP == 2 || CSPLIT > 1) {
    ptx::cluster_sync();  // the peer's barriers must exist before anything signals them
  } else {
    __syncthreads();
  }
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  if (trace && threadIdx.x == 0)
    trace[TRACE_SETUP] = static_cast<unsigned long long>(clock64() - clk_start);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    {
      // The whole warp walks the loops and polls the barriers (so loop state stays
      // warp-uniform and cheap to turn into TMA operands); the lane elected here, once,
      // issues the copies.  Nothing inside the loops is warp-collective, so a lane whose
      // wait gives up can leave on its own.
      const bool elected = ptx::elect_one();
      if (p.wait_prior_grid) ptx::grid_dep_wait();  // the operands may come from a grid in front
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      long long waited = 0, prod_issue = 0, flag_wait = 0;
      const uint64_t pol_a = p.l2_policy == 0 ? ptx::policy_evict_normal() : ptx::policy_evict_last();
      const uint64_t pol_b = (p.l2_policy == 0 || p.l2_policy == 3) ? ptx::policy_evict_normal()
                             : p.l2_policy == 1                      ? ptx::policy_evict_first()
                                                                     : ptx::policy_evict_last();
      bool backward = false;
      constexpr int RING = FUSED ? PSTAGES : STAGES;  // slots of the ring this role fills
      for (int t = first_tile; FUSED && t < num_tiles && ok; t += tile_stride) {
        // Fused INT4: every CTA fills its own ring of packed slots and counts its own bytes;
        // one packed slot (128 bytes = 256 values of K per row) feeds two int8 slots.
        int tm, tn, tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        tile_coords(p, tile, tm, tn);
        const int a_row = tm * TILE_M + static_cast<int>(cta_rank) * BM;
        const int b_row = tn * BN + static_cast<int>(cta_rank) * L::B_ROWS;
        const int ps_begin = k_begin / 2, ps_end = k_end / 2;
        for (int ps = ps_begin; ps < ps_end; ++ps) {
          const long long w0 = trace ? clock64() : 0;
          ok = wait_bounded(p_empty_bar(stage), phase ^ 1u, abort_flag, p.status,
                            DEV_TIMEOUT_PRODUCER);
          const long long w9 = trace ? clock64() : 0;
          if (trace) waited += w9 - w0;
          if (!ok) break;
          const uint32_t a_dst = base + L::P_OFFSET + stage * L::P_STAGE_BYTES;
          const uint32_t b_dst = a_dst + (A8 ? 0 : L::A_BYTES);
          if (!elected) {
            // nothing to issue in this lane
          } else if ((ablate & 8) && blockIdx.x == 0 && t == first_tile && ps == ps_begin + 2) {
            // failure drill: this slot is never filled
          } else if (ablate & 2) {
            ptx::mbar_arrive(p_full_bar(stage));
          } else {
            const int k0 = (backward ? ps_begin + ps_end - 1 - ps : ps) * BK_BYTES;  // packed bytes
            ptx::mbar_arrive_expect_tx(p_full_bar(stage), L::P_STAGE_BYTES);
            if constexpr (!A8) ptx::tma_load_2d(a_dst, &tmap_a, k0, a_row, p_full_bar(stage), pol_a);
            ptx::tma_load_2d(b_dst, &tmap_b, k0, b_row, p_full_bar(stage), pol_b);
          }
          ++issued;
          if (trace) prod_issue += clock64() - w9;
          if (++stage == RING) { stage = 0; phase ^= 1u; }
        }
        if (p.serpentine_k) backward = !backward;
      }
      // overlapped INT4 pre-pass: the int8 rows behind a box must have been produced
      const uint32_t ahead_epoch = AHEAD ? s4a_epoch(p.ahead) : 0u;
      bool ahead_all = !AHEAD;
      for (int t = first_tile; !FUSED && t < num_tiles && ok; t += tile_stride) {
        int tm, tn, tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        tile_coords(p, tile, tm, tn);
        const int a_row = tm * TILE_M + static_cast<int>(cta_rank) * BM;
        const int b_row = tn * BN + static_cast<int>(cta_rank) * L::B_ROWS;
        int ahead_kc = -1;
        for (int ks = k_begin; ks < k_end; ++ks) {
          const long long w0 = trace ? clock64() : 0;
          ok = wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, p.status,
                            DEV_TIMEOUT_PRODUCER);
          if constexpr (AHEAD) {
            const int kc = (backward ? k_begin + k_end - 1 - ks : ks) * BK_BYTES / S4A_CHUNK_COLS;
            const long long f0 = trace ? clock64() : 0;
            if (ok && !ahead_all && kc != ahead_kc) {
              ahead_kc = kc;
              if (ld_acquire_u32(p.ahead.sync + S4A_ALL_DONE) == ahead_epoch) {
                ahead_all = true;
              } else {
                ok = s4a_wait_ready(p.ahead, ahead_epoch, a_row, BM / S4A_CHUNK_ROWS, b_row,
                                    L::B_ROWS / S4A_CHUNK_ROWS, kc, lane, abort_flag, WAIT_LIMIT_NS);
                if (!ok) {
                  *abort_flag = 1;
                  atomicCAS(p.status, 0, DEV_TIMEOUT_PRODUCER);
                }
              }
            }
            if (trace) flag_wait += clock64() - f0;
          }
          const long long w9 = trace ? clock64() : 0;
          if (trace) waited += w9 - w0;
          if (!ok) break;
          const uint32_t a_dst = base + stage * L::STAGE_BYTES;
          const uint32_t b_dst = a_dst + KB * L::A_BYTES;
          if (!elected) {
            // nothing to issue in this lane
          } else if ((ablate & 8) && blockIdx.x == 0 && t == first_tile && ks == k_begin + 2) {
            // failure drill: this slot is never filled
          } else if (ablate & 2) {
            if (leader) ptx::mbar_arrive(full_bar(stage));
          } else if constexpr (CTA_GROUP == 1) {
            ptx::mbar_arrive_expect_tx(full_bar(stage), L::STAGE_BYTES);
#pragma unroll
            for (int a = 0; a < KB; ++a) {
              const int k0 = ((backward ? k_begin + k_end - 1 - ks : ks) * KB + a) * BK_ELEMS;
              ptx::tma_load_2d(a_dst + a * L::A_BYTES, &tmap_a, k0, a_row, full_bar(stage), pol_a);
              ptx::tma_load_2d(b_dst + a * L::B_BYTES, &tmap_b, k0, b_row, full_bar(stage), pol_b);
            }
          } else {
            // Bytes of both CTAs are counted on the leader's barrier.
            if (leader) ptx::mbar_arrive_expect_tx(full_bar(stage), 2 * L::STAGE_BYTES);
            const uint32_t lead_full = ptx::map_to_cta(full_bar(stage), 0);
#pragma unroll
            for (int a = 0; a < KB; ++a) {
              const int k0 = ((backward ? k_begin + k_end - 1 - ks : ks) * KB + a) * BK_ELEMS;
              ptx::tma_load_2d_pair(a_dst + a * L::A_BYTES, &tmap_a, k0, a_row, lead_full, pol_a);
              ptx::tma_load_2d_pair(b_dst + a * L::B_BYTES, &tmap_b, k0, b_row, lead_full, pol_b);
            }
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
        if (AHEAD) trace[TRACE_UNPACK_WAIT_IN] = static_cast<unsigned long long>(flag_wait);
      }
      if (!ok && elected && (FUSED || CTA_GROUP == 1 || leader)) {
        // Gave up: let the copies already in flight land before the CTA exits.
        int n = issued < RING ? issued : RING;
        for (int i = 0; i < n; ++i) {
          if (--stage < 0) { stage = RING - 1; phase ^= 1u; }
          uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(FUSED ? p_full_bar(stage) : full_bar(stage), phase) &&
                 ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    // A grid launched to start early counts its 2 s wait limits only from the moment the grid
    // in front has completed: no operand can arrive before the producer has passed the same
    // point, and the time spent behind a long predecessor must not look like a stuck barrier.
    if (p.wait_prior_grid) ptx::grid_dep_wait();
    if (leader) {  // whole warp walks the loops, the lane elected once issues (see producer)
      const bool elected = ptx::elect_one();
      constexpr uint32_t idesc = ptx::make_idesc<KIND>(TILE_M, BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      int astage = 0;          // hybrid fused INT4: the ring of A atoms
      uint32_t aphase = 0;
      bool ok = true;
      long long wait_full = 0, wait_acc = 0, t_issue = 0, t_commit = 0, wait_a = 0;
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        const long long w0 = trace ? clock64() : 0;
        ok = wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status,
                          DEV_TIMEOUT_MMA);
        if (trace) wait_acc += clock64() - w0;
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(acc * BN);
        int tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        for (int ks = k_begin; ks < k_end; ++ks) {
          const long long w1 = trace ? clock64() : 0;
          if constexpr (FUSED) {
            ok = wait_bounded(ready_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
            if (ok && CTA_GROUP == 2)
              ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
            if constexpr (A8) {
              const long long wa = trace ? clock64() : 0;
              if (ok) ok = wait_bounded(a_full_bar(astage), aphase, abort_flag, p.status, DEV_TIMEOUT_MMA);
              if (trace) wait_a += clock64() - wa;
            }
          } else {
            ok = wait_bounded(full_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_MMA);
          }
          const long long w2 = trace ? clock64() : 0;
          if (trace) wait_full += w2 - w1;
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const uint32_t a_src = A8 ? base + L::A8_OFFSET + astage * L::A_BYTES : base + stage * L::STAGE_BYTES;
          const uint64_t a_desc = ptx::smem_desc_sw128(a_src);
          const uint64_t b_desc =
              ptx::smem_desc_sw128(A8 ? base + stage * L::STAGE_BYTES : a_src + KB * L::A_BYTES);
          if (elected && !(ablate & 1)) {
#pragma unroll
            for (int a = 0; a < KB; ++a) {
#pragma unroll
              for (int kk = 0; kk < BK_BYTES / MMA_K_BYTES; ++kk) {
                // descriptor addresses are in 16-byte units
                const uint64_t a_step =
                    static_cast<uint64_t>((a * L::A_BYTES + kk * MMA_K_BYTES) >> 4);
                const uint64_t b_step =
                    static_cast<uint64_t>((a * L::B_BYTES + kk * MMA_K_BYTES) >> 4);
                ptx::mma_ss<KIND, CTA_GROUP>(d_tmem, a_desc + a_step, b_desc + b_step, idesc,
                                             (ks > k_begin || a > 0 || kk > 0) ? 1u : 0u);
              }
            }
          }
          if (trace) t_issue += clock64() - w2;
          const long long w4 = trace ? clock64() : 0;
          if (elected) {
            if constexpr (CTA_GROUP == 1) {
              ptx::mma_commit<1>(empty_bar(stage));
              if constexpr (A8) ptx::mma_commit<1>(a_empty_bar(astage));
            } else {
              ptx::mma_commit_pair(empty_bar(stage), 0x3);
              if constexpr (A8) ptx::mma_commit_pair(a_empty_bar(astage), 0x3);
            }
          }
          if (trace) t_commit += clock64() - w4;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          if constexpr (A8) {
            if (++astage == L::A8_STAGES) { astage = 0; aphase ^= 1u; }
          }
        }
        if (!ok) break;
        if (elected) {
          if constexpr (CTA_GROUP == 1) {
            ptx::mma_commit<1>(acc_full_bar(acc));
          } else {
            ptx::mma_commit_pair(acc_full_bar(acc), 0x3);
          }
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (trace && elected) {
        trace[TRACE_MMA_WAIT_FULL] = static_cast<unsigned long long>(wait_full);
        trace[TRACE_MMA_WAIT_ACC] = static_cast<unsigned long long>(wait_acc);
        trace[TRACE_MMA_ISSUE] = static_cast<unsigned long long>(t_issue);
        trace[TRACE_MMA_COMMIT] = static_cast<unsigned long long>(t_commit);
        if (A8) trace[TRACE_MMA_WAIT_ACC1] = static_cast<unsigned long long>(wait_a);  // of wait_full: for the A atom
      }
      if (!ok && elected) {
        // Gave up: wait for the MMAs already issued before TMEM is released.
        ptx::mma_commit<CTA_GROUP>(drain_bar);
        uint64_t t0 = ptx::globaltimer_ns();
        while (!ptx::mbar_try_wait(drain_bar, 0) && ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
        }
      }
    } else if constexpr (FUSED && CTA_GROUP == 2) {
      // Peer CTA, fused INT4: relay "my int8 slot is written" to the leader's `full` barrier.
      const bool elected = ptx::elect_one();
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        int tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        for (int ks = k_begin; ks < k_end; ++ks) {
          ok = wait_bounded(ready_bar(stage), phase, abort_flag, p.status, DEV_TIMEOUT_UNPACK);
          if (!ok) break;
          // The leader does not read this CTA's shared memory itself: the MMAs it issues make
          // this SM's tensor core read it, after the writers' proxy fences.
          if (elected) ptx::mbar_arrive_remote(ptx::map_to_cta(full_bar(stage), 0));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (AHEAD && warp >= 2 + EPI_WARPS) {
    // ------------------------------------- overlapped INT4 pre-pass: int8 chunks for the tiles to come
    // Warps of their own: a chunk takes thousands of cycles inside a busy GEMM (its loads and
    // stores queue behind the operand tiles), and a warp with another duty -- an epilogue that
    // became due meanwhile -- would be late for it by that much.
    if constexpr (AHEAD) {
      if (p.wait_prior_grid) ptx::grid_dep_wait();  // the scratch may be in use by the grid in front
      const uint32_t epoch = s4a_epoch(p.ahead);
      const long long u0 = trace ? clock64() : 0;
      s4a_work(p.ahead, epoch, lane, [&]() { return *abort_flag != 0; });
      if (trace && warp == 2 + EPI_WARPS && lane == 0)
        trace[TRACE_UNPACK_BUSY] = static_cast<unsigned long long>(clock64() - u0);
    }
    __syncwarp();
  } else if (A8 && warp == 2 + EPI_WARPS + UNPACK_WARPS) {
    // ------------------------------------------ hybrid fused INT4: producer of the A image
    // One 128-byte atom of the int8 image of A per k-block of the MMA issuer, into a ring of
    // its own, in the order the packed B slots are sent (slot ps of a unit feeds k-blocks 2 ps
    // and 2 ps + 1; with the serpentine order every other tile walks its slots backwards).
    if constexpr (A8) {
      const bool elected = ptx::elect_one();
      if (p.wait_prior_grid) ptx::grid_dep_wait();  // the image comes from the grid in front
      int astage = 0, issued = 0;
      uint32_t aphase = 0;
      bool ok = true, backward = false;
      const uint64_t pol = ptx::policy_evict_last();  // every tile column re-reads A
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        int tm, tn, tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        tile_coords(p, tile, tm, tn);
        const int a_row = tm * TILE_M + static_cast<int>(cta_rank) * BM;
        const int ps_begin = k_begin / 2, ps_end = k_end / 2;
        for (int ks = k_begin; ks < k_end; ++ks) {
          ok = wait_bounded(a_empty_bar(astage), aphase ^ 1u, abort_flag, p.status, DEV_TIMEOUT_PRODUCER);
          if (!ok) break;
          if (elected) {
            const int ps = ks / 2;
            const int atom = 2 * (backward ? ps_begin + ps_end - 1 - ps : ps) + (ks & 1);
            const uint32_t dst = base + L::A8_OFFSET + astage * L::A_BYTES;
            if constexpr (CTA_GROUP == 1) {
              ptx::mbar_arrive_expect_tx(a_full_bar(astage), L::A_BYTES);
              ptx::tma_load_2d(dst, &tmap_a, atom * BK_BYTES, a_row, a_full_bar(astage), pol);
            } else {
              // bytes of both CTAs are counted on the leader's barrier
              if (leader) ptx::mbar_arrive_expect_tx(a_full_bar(astage), 2 * L::A_BYTES);
              ptx::tma_load_2d_pair(dst, &tmap_a, atom * BK_BYTES, a_row,
                                    ptx::map_to_cta(a_full_bar(astage), 0), pol);
            }
          }
          ++issued;
          if (++astage == L::A8_STAGES) { astage = 0; aphase ^= 1u; }
        }
        if (p.serpentine_k) backward = !backward;
      }
      if (!ok && elected && (CTA_GROUP == 1 || leader)) {
        // Gave up: let the copies already in flight land before the CTA exits.
        int n = issued < L::A8_STAGES ? issued : L::A8_STAGES;
        for (int i = 0; i < n; ++i) {
          if (--astage < 0) { astage = L::A8_STAGES - 1; aphase ^= 1u; }
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(a_full_bar(astage), aphase) &&
                 ptx::globaltimer_ns() - t0 < WAIT_LIMIT_NS) {
          }
        }
      }
    }
    __syncwarp();
  } else if (FUSED && warp >= 2 + EPI_WARPS) {
    // ------------------------------------------------- fused INT4: nibble expansion
    // One packed slot holds, per operand row, 128 bytes = 8 chunks of 16 bytes (32 values of K
    // each), chunk c stored at position c ^ (row & 7) by the 128-byte swizzle.  Chunks 0..3 feed
    // int8 slot "h = 0", chunks 4..7 slot "h = 1".  A chunk's even-k values (low nibbles) become
    // int8 chunk c & 3 of the row, its odd-k values chunk (c & 3) + 4, both in the same swizzle;
    // in byte offsets inside the operand tile that is x ^ (h * 64) resp. x ^ (h * 64) ^ 64 for a
    // chunk read at offset x.  Lane -> (row, chunk) is chosen so that each quarter-warp reads
    // and writes all 32 banks once.
    if constexpr (FUSED) {
      if (p.wait_prior_grid) ptx::grid_dep_wait();  // wait limits count from the predecessor's end
      // With deep rings (the narrow tiles of problems with few rows) the eight warps work as
      // two groups on alternate packed slots: a slot's fixed costs -- three barrier waits, the
      // proxy fence, the arrives: ~700 of the ~1300 cycles a slot took -- then overlap.
      const int uw = (warp - (2 + EPI_WARPS)) % GROUP_WARPS;  // warp within its group
      const int ugroup = (warp - (2 + EPI_WARPS)) / GROUP_WARPS;
      int pcount = 0;                                          // packed slots so far, all tiles
      const int c = lane & 3;
      const int row_in_8 = (lane >> 3) + 4 * ((lane >> 2) & 1);
      constexpr uint32_t HI = 0xF0F0F0F0u;
      int pstage = 0, ustage = 0;
      uint32_t pphase = 0, uphase = 0;
      bool ok = true;
      long long wait_in = 0, wait_out = 0, busy = 0;
      // Rows this role expands: the whole packed slot (A rows, then B rows), or -- hybrid --
      // only the B rows, which then start at row 0 of both the packed slot and the int8 slot
      // (ROW0: what to add to a row of the slot to get its place in the A-then-B numbering
      // that the validity test uses).
      constexpr int ROW0 = A8 ? BM : 0;
      constexpr int ROWS = A8 ? L::B_ROWS : BM + L::B_ROWS;
      for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
        int tm, tn, tile, k_begin, k_end;
        bool add;
        decode_unit(t, tile, k_begin, k_end, add);
        tile_coords(p, tile, tm, tn);
        // Rows of the tile beyond M resp. N are not expanded: the accumulator rows and columns
        // they feed are never stored, so whatever the int8 slot holds there does no harm, and a
        // problem with few rows (M = 16) skips most of the A tile.
        const int a_row = tm * TILE_M + static_cast<int>(cta_rank) * BM;
        const int a_valid = p.M - a_row;
        const int b_valid = p.N - (tn * BN + static_cast<int>(cta_rank) * L::B_ROWS);
        constexpr int TASKS = (ROWS + 8 * GROUP_WARPS - 1) / (8 * GROUP_WARPS);
        bool active[TASKS];
#pragma unroll
        for (int i = 0; i < TASKS; ++i) {
          const int row8 = ROW0 + (i * GROUP_WARPS + uw) * 8;  // first row of this lane's group of 8
          active[i] = row8 < BM ? row8 < a_valid : (row8 < BM + L::B_ROWS && row8 - BM < b_valid);
        }
        for (int ps = k_begin / 2; ps < k_end / 2 && ok; ++ps, ++pcount) {
          if (UNPACK_GROUPS > 1 && pcount % UNPACK_GROUPS != ugroup) {
            // the other group's slot: only keep the ring positions in step
            ustage += 2;
            if (ustage >= STAGES) { ustage -= STAGES; uphase ^= 1u; }
            if (++pstage == PSTAGES) { pstage = 0; pphase ^= 1u; }
            continue;
          }
          const long long w0 = trace ? clock64() : 0;
          ok = wait_bounded(p_full_bar(pstage), pphase, abort_flag, p.status, DEV_TIMEOUT_UNPACK);
          ok = __all_sync(0xffffffffu, ok);
          if (trace) wait_in += clock64() - w0;
          if (!ok) break;
          const uint32_t src = base + L::P_OFFSET + pstage * L::P_STAGE_BYTES;
          // Both int8 slots this packed slot feeds are taken at once, so that one proxy fence
          // (a few hundred cycles per warp) covers both.
          const int u0 = ustage, u1 = (ustage + 1 == STAGES) ? 0 : ustage + 1;
          const uint32_t ph0 = uphase, ph1 = (ustage + 1 == STAGES) ? (uphase ^ 1u) : uphase;
          const long long w1 = trace ? clock64() : 0;
          ok = wait_bounded(empty_bar(u0), ph0 ^ 1u, abort_flag, p.status, DEV_TIMEOUT_UNPACK);
          if (ok) ok = wait_bounded(empty_bar(u1), ph1 ^ 1u, abort_flag, p.status, DEV_TIMEOUT_UNPACK);
          ok = __all_sync(0xffffffffu, ok);
          const long long w2 = trace ? clock64() : 0;
          if (trace) wait_out += w2 - w1;
          if (!ok) break;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t dst = base + (h ? u1 : u0) * L::STAGE_BYTES;
            const uint32_t x0 = static_cast<uint32_t>(row_in_8 * 128 + (((4 * h + c) ^ row_in_8) << 4));
            const uint32_t flip = static_cast<uint32_t>(h) << 6;
            // A rows first, then the B rows (the B tile follows the A tile in both rings); all
            // loads are issued before the first store so that their latencies overlap
            uint32_t wv[TASKS][4];
#pragma unroll
            for (int i = 0; i < TASKS; ++i)
              if (active[i])
                ptx::ld_shared_v4(src + x0 + static_cast<uint32_t>((i * GROUP_WARPS + uw) * 8 * 128),
                                  wv[i][0], wv[i][1], wv[i][2], wv[i][3]);
#pragma unroll
            for (int i = 0; i < TASKS; ++i) {
              if (!active[i]) continue;
              const uint32_t x = x0 + static_cast<uint32_t>((i * GROUP_WARPS + uw) * 8 * 128);
              ptx::st_shared_v4(dst + (x ^ flip), (wv[i][0] << 4) & HI, (wv[i][1] << 4) & HI,
                                (wv[i][2] << 4) & HI, (wv[i][3] << 4) & HI);
              ptx::st_shared_v4(dst + (x ^ flip ^ 64u), wv[i][0] & HI, wv[i][1] & HI, wv[i][2] & HI,
                                wv[i][3] & HI);
            }
          }
          // the tensor cores read shared memory through the async proxy
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::mbar_arrive(ready_bar(u0));
            ptx::mbar_arrive(ready_bar(u1));
          }
          if (trace) busy += clock64() - w2;
          ustage += 2;
          if (ustage >= STAGES) { ustage -= STAGES; uphase ^= 1u; }
          if (!ok) break;
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(p_empty_bar(pstage));  // every lane has read its chunks
          if (++pstage == PSTAGES) { pstage = 0; pphase ^= 1u; }
        }
      }
      if (trace && uw == 0 && ugroup == 0 && lane == 0) {
        trace[TRACE_UNPACK_WAIT_IN] = static_cast<unsigned long long>(wait_in);
        trace[TRACE_UNPACK_WAIT_OUT] = static_cast<unsigned long long>(wait_out);
        trace[TRACE_UNPACK_BUSY] = static_cast<unsigned long long>(busy);
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue
    // Fused INT4 accumulators hold 256 * C: an arithmetic shift restores C exactly.
    auto fix = [](uint32_t bits) -> uint32_t {
      if constexpr (FUSED) return static_cast<uint32_t>(static_cast<int32_t>(bits) >> 8);
      return bits;
    };
    const int quarter = warp & 3;  // TMEM lane quarter this warp may read
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t epi_base =
        base + L::EPI_OFFSET + static_cast<uint32_t>((warp - 2) * 2 * L::EPI_BUF_BYTES);
    const uint64_t pol_c = p.c_evict_first ? ptx::policy_evict_first() : ptx::policy_evict_normal();
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    long long epi_wait = 0, epi_busy = 0, tiles_done = 0;
    uint32_t staged_blocks = 0;  // blocks sent through the staging buffers so far
    // (see the MMA issuer: wait limits count from the end of the grid in front; also C, the
    // scale factors and the INT4 scratch may still be in use by it)
    if (p.wait_prior_grid) ptx::grid_dep_wait();
    bool prior_grid_done = true;
    uint32_t xphase = 0;         // cluster split-K: parity of the partial-sum hand-over
    const bool xpeer = CSPLIT > 1 && krank != 0;  // this CTA only contributes partial sums
    // Cluster split-K, rank 0: adds the other CTAs' partial sums for accumulator columns
    // [32 * b32, 32 * b32 + 32) of this thread's row to the 32 raw accumulators in r.
    auto add_partial = [&](uint32_t (&r)[32], int b32) {
      if constexpr (CSPLIT > 1) {
#pragma unroll
        for (int peer = 0; peer < CSPLIT - 1; ++peer) {
        const uint32_t xsrc = base + L::X_OFFSET +
                              static_cast<uint32_t>(peer * L::X_PEER_BYTES + quarter * (32 * BN * 4) +
                                                    b32 * 4096 + lane * 128);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t t0, t1, t2, t3;
          ptx::ld_shared_v4(xsrc + static_cast<uint32_t>(((j ^ (lane & 7)) * 16)), t0, t1, t2, t3);
          if constexpr (KIND == ptx::KIND_F16) {
            r[4 * j + 0] = __float_as_uint(__uint_as_float(r[4 * j + 0]) + __uint_as_float(t0));
            r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + __uint_as_float(t1));
            r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + __uint_as_float(t2));
            r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + __uint_as_float(t3));
          } else {
            r[4 * j + 0] += t0;
            r[4 * j + 1] += t1;
            r[4 * j + 2] += t2;
            r[4 * j + 3] += t3;
          }
        }
        }
      }
    };
    for (int t = first_tile; t < num_tiles && ok; t += tile_stride) {
      int tm, tn, tile, k_begin, k_end;
      bool add;
      decode_unit(t, tile, k_begin, k_end, add);
      tile_coords(p, tile, tm, tn);
      const int row0 = tm * TILE_M + static_cast<int>(cta_rank) * BM + quarter * 32;
      const int row = row0 + lane;
      const int col0 = tn * BN;
      float rs = 1.0f;
      if constexpr (EPI != EPI_RAW32) {
        // The scale factors are fetched while the mainloop still runs: this thread's row
        // factor into a register, the tile's column factors into L1 (one line per lane).
        // They may come from the grid in front, so its end is awaited first -- the producer
        // waits for the same before its first load, so no accumulator could be ready earlier.
        if (p.row_scale || p.col_scale) {
          if (p.wait_prior_grid && !prior_grid_done) {
            ptx::grid_dep_wait();
            prior_grid_done = true;
          }
          if (p.row_scale && row < p.M) rs = ptx::ld_global_f32(p.row_scale + row);
          if (p.col_scale && lane * 32 < BN && col0 + lane * 32 < p.N)
            ptx::prefetch_l1(p.col_scale + col0 + lane * 32);
        }
      }
      const long long w0 = trace ? clock64() : 0;
      ok = wait_bounded<true>(acc_full_bar(acc), acc_phase, abort_flag, p.status,
                              DEV_TIMEOUT_EPILOGUE, (ablate & 4) ? 500u : 0u);
      ok = __all_sync(0xffffffffu, ok);
      const long long w1 = trace ? clock64() : 0;
      epi_wait += w1 - w0;
      if (!ok) break;
      ptx::tc_fence_after_sync();
      if constexpr (CSPLIT > 1) {
        if (xpeer) {
          // Ranks 1..: write this tile's raw 32-bit accumulators (one 128-byte row piece per
          // thread and 32 columns, swizzled like the staging buffers) into this CTA's own
          // hand-over buffer, then -- once rank 0 has consumed the previous tile's partial
          // sums -- send the warp's 32 rows to rank 0's buffer for this rank as one bulk copy,
          // whose bytes are counted on rank 0's `part_full`.  (No cluster-scope fence or
          // release: the copy engine orders the data before the byte count.)
          if (lane == 0) ptx::bulk_wait_group_read<0>();  // the previous copy has read the buffer
          __syncwarp();
          const uint32_t xown = base + L::X_OFFSET + static_cast<uint32_t>(quarter * (32 * BN * 4));
#pragma unroll 1
          for (int b = 0; b < BN / 32; ++b) {
            uint32_t r[32];
            ptx::tmem_ld_32x32b_x32(tmem_base + lane_base + static_cast<uint32_t>(acc * BN + b * 32), r);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              ptx::st_shared_v4(xown + static_cast<uint32_t>(b * 4096 + lane * 128 + ((j ^ (lane & 7)) * 16)),
                                r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
          }
          ptx::fence_proxy_async_smem();
          ok = wait_bounded(part_free_bar, xphase ^ 1u, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) {
            ptx::bulk_copy_to_cluster(
                ptx::map_to_cta(base + L::X_OFFSET, 0) +
                    static_cast<uint32_t>((krank - 1) * L::X_PEER_BYTES + quarter * (32 * BN * 4)),
                xown, 32 * BN * 4, ptx::map_to_cta(part_full_bar, 0));
            ptx::bulk_commit_group();
          }
        } else {
          // rank 0: one thread announces the bytes the other ranks will send for this tile
          if (warp == 2 && lane == 0)
            ptx::mbar_arrive_expect_tx(part_full_bar, (CSPLIT - 1) * L::X_PEER_BYTES);
          ok = wait_bounded(part_full_bar, xphase, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        xphase ^= 1u;
      }
      // A split-K unit whose K range is empty (the host never creates one) contributes nothing.
      const bool empty_range = k_begin >= k_end;
      if (p.wait_prior_grid && !prior_grid_done) {  // C may be read, written or zeroed by the grid in front
        ptx::grid_dep_wait();
        prior_grid_done = true;
      }
      // One staging block = 32 rows x 128 bytes = 32 columns of 32-bit or 64 columns of
      // 16-bit results.  Thread `lane` owns row `lane`; 16-byte chunk j of the row goes to
      // chunk j ^ (lane & 7), the 128-byte swizzle the C tensor map expects, which also
      // spreads the warp's 16-byte stores over all banks.
      // (The 32-wide tile with 16-bit output has no staging form -- a block would be 64 bytes
      // wide -- and only ever runs with plain stores: c_vec_ok = 0, set by the host.)
      constexpr int BLOCK_COLS = (EPI == EPI_OUT16 && BN >= 64) ? 64 : 32;
      static_assert(BN % BLOCK_COLS == 0, "tile width must be a multiple of the store block");
#pragma unroll 1
      for (int c = 0; c < BN / BLOCK_COLS && !xpeer; ++c) {
        const int col = col0 + c * BLOCK_COLS;
        uint32_t w[32];  // the thread's 128 bytes of output
        if constexpr (EPI == EPI_RAW32 && CSPLIT == 1) {
          if (DBG && (ablate & 32) && p.c_vec_ok && p.ldc % 8 == 0 && !add) {
            // ablation: no staging at all -- read the block in the 16x256b shape, in which four
            // neighbouring threads hold 32 contiguous bytes of a row, and store those straight
            // to C: whole 32-byte sectors, no shared-memory traffic beside the mainloop's
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              uint32_t r16[16];
              ptx::tmem_ld_16x256b_x4(tmem_base + lane_base + (static_cast<uint32_t>(h * 16) << 16) +
                                          static_cast<uint32_t>(acc * BN + c * 32),
                                      r16);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int cj = col + 8 * j + 2 * (lane & 3);
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                  const int rr = row0 + 16 * h + 8 * u + (lane >> 2);
                  if (rr < p.M && cj < p.N && !empty_range)
                    ptx::st_global_v2_hint(p.C + static_cast<size_t>(rr) * p.ldc + cj,
                                           fix(r16[4 * j + 2 * u]), fix(r16[4 * j + 2 * u + 1]), pol_c);
                }
              }
            }
            continue;
          }
        }
        if constexpr (EPI == EPI_RAW32) {
          ptx::tmem_ld_32x32b_x32(
              tmem_base + lane_base + static_cast<uint32_t>(acc * BN + c * 32), w);
          ptx::tmem_wait_ld();
          add_partial(w, c);
          if constexpr (FUSED) {
#pragma unroll
            for (int v = 0; v < 32; ++v) w[v] = fix(w[v]);
          }
        } else if constexpr (EPI == EPI_F32_SCALED) {
          // Column factors: one coalesced load per 32 columns (lane v fetches column v's),
          // handed round by shuffles -- a load per element, even from L1, made this loop
          // wait ~25 cycles per column.
          const float cs_mine = (col + lane < p.N) ? ptx::ld_global_f32(p.col_scale + col + lane) : 0.0f;
          ptx::tmem_ld_32x32b_x32(
              tmem_base + lane_base + static_cast<uint32_t>(acc * BN + c * 32), w);
          ptx::tmem_wait_ld();
          add_partial(w, c);
#pragma unroll
          for (int v = 0; v < 32; ++v) {
            const float cs = __shfl_sync(0xffffffffu, cs_mine, v);
            w[v] = __float_as_uint(acc_to_float<KIND>(fix(w[v])) * rs * cs);
          }
        } else {
#pragma unroll
          for (int h = 0; h < BLOCK_COLS / 32; ++h) {
            const int cc = col + h * 32 + lane;
            const float cs_mine = (p.col_scale && cc < p.N) ? ptx::ld_global_f32(p.col_scale + cc) : 0.0f;
            uint32_t r[32];
            ptx::tmem_ld_32x32b_x32(
                tmem_base + lane_base + static_cast<uint32_t>(acc * BN + c * BLOCK_COLS + h * 32), r);
            ptx::tmem_wait_ld();
            add_partial(r, c * (BLOCK_COLS / 32) + h);
#pragma unroll
            for (int v = 0; v < 32; v += 2) {
              float x0 = acc_to_float<KIND>(fix(r[v])), x1 = acc_to_float<KIND>(fix(r[v + 1]));
              if (p.col_scale) {  // same for the whole warp
                x0 *= rs * __shfl_sync(0xffffffffu, cs_mine, v);
                x1 *= rs * __shfl_sync(0xffffffffu, cs_mine, v + 1);
              }
              w[h * 16 + v / 2] = pack_half2(x0, x1);
            }
          }
        }
        if (EPI == EPI_RAW32 && (ablate & 16) && p.c_vec_ok && !add) {
          // ablation: straight from registers, 8 x 16 bytes per thread into its own C row
          if (row < p.M) {
            uint32_t* crow = p.C + static_cast<size_t>(row) * p.ldc;
            if (col + 32 <= p.N) {
              uint4* dst = reinterpret_cast<uint4*>(crow + col);
#pragma unroll
              for (int v = 0; v < 8; ++v)
                dst[v] = make_uint4(w[4 * v], w[4 * v + 1], w[4 * v + 2], w[4 * v + 3]);
            } else {
#pragma unroll
              for (int v = 0; v < 32; ++v)
                if (col + v < p.N) crow[col + v] = w[v];
            }
          }
        } else if (p.c_vec_ok) {
          // registers -> swizzled shared memory -> one TMA store per block
          // The two staging buffers alternate per BLOCK, counted across tiles (a tile may
          // have an odd number of blocks): the store issued from this buffer two blocks ago
          // must have read it
          const uint32_t buf = epi_base + static_cast<uint32_t>((staged_blocks & 1) * L::EPI_BUF_BYTES);
          ++staged_blocks;
          if (lane == 0) ptx::bulk_wait_group_read<1>();
          __syncwarp();
          const uint32_t row_addr = buf + static_cast<uint32_t>(lane * 128);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            ptx::st_shared_v4(row_addr + static_cast<uint32_t>(((j ^ (lane & 7)) * 16)), w[4 * j],
                              w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          // Partly outside C: the hardware clips.  Wholly outside: issue no store, but still
          // close a (then empty) group so that "one group per block" keeps the buffer
          // reuse rule above exact.
          if (lane == 0) {
            if (row0 < p.M && col < p.N && !empty_range) {
              if (EPI == EPI_RAW32 && add)
                ptx::tma_reduce_add_2d(&tmap_c, col, row0, buf);
              else
                ptx::tma_store_2d(&tmap_c, col, row0, buf, pol_c);
            }
            ptx::bulk_commit_group();
          }
        } else if (row < p.M && !empty_range) {
          // C rows are not 16-byte multiples: plain predicated stores.
          // element (row, col + v) sits at row * rstep + (col + v) * cstep
          const size_t rstep = p.transpose_c ? 1 : static_cast<size_t>(p.ldc);
          const size_t cstep = p.transpose_c ? static_cast<size_t>(p.ldc) : 1;
          if constexpr (EPI == EPI_OUT16) {
            uint16_t* crow = reinterpret_cast<uint16_t*>(p.C) + static_cast<size_t>(row) * rstep;
#pragma unroll
            for (int v = 0; v < BLOCK_COLS; ++v)
              if (col + v < p.N)
                crow[(col + v) * cstep] = static_cast<uint16_t>(w[v / 2] >> (16 * (v & 1)));
          } else {
            uint32_t* crow = p.C + static_cast<size_t>(row) * rstep;
            if (EPI == EPI_RAW32 && add) {
#pragma unroll
              for (int v = 0; v < 32; ++v) {
                if (col + v >= p.N) continue;
                if constexpr (KIND == ptx::KIND_F16)
                  atomicAdd(reinterpret_cast<float*>(crow + (col + v) * cstep), __uint_as_float(w[v]));
                else
                  atomicAdd(reinterpret_cast<int*>(crow + (col + v) * cstep), static_cast<int>(w[v]));
              }
            } else {
#pragma unroll
              for (int v = 0; v < 32; ++v)
                if (col + v < p.N) crow[(col + v) * cstep] = w[v];
            }
          }
        }
      }
      if constexpr (CSPLIT > 1) {
        if (!xpeer) {  // the partial sums have been read: the others may send the next tile's
          // (a plain arrive: the receiver reads nothing this CTA wrote, and this warp's loads
          // from the buffer have returned their values)
          __syncwarp();
          if (lane == 0) {
#pragma unroll
            for (int peer = 1; peer < CSPLIT; ++peer)
              ptx::mbar_arrive_remote(ptx::map_to_cta(part_free_bar, peer));
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
          // CTA-scope release on the leader's barrier: the accumulator reads above are complete
          // (tcgen05.wait::ld) and ordered by the tcgen05 fence; nothing else has to be made
          // visible cluster-wide, and a cluster-scope release would stall this lane for
          // hundreds of cycles per tile.
          ptx::mbar_arrive_remote(ptx::map_to_cta(acc_empty_bar(acc), 0));
        }
      }
      if (trace) epi_busy += clock64() - w1;
      ++tiles_done;
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    // C stores still in flight read this CTA's shared memory: wait until they have read it
    // (their global writes complete on their own before the grid counts as finished).  A
    // hand-over copy into rank 0's shared memory has to have landed as well.
    if (lane == 0) {
      if (xpeer) ptx::bulk_wait_group_all();
      else ptx::bulk_wait_group_read<0>();
    }
    __syncwarp();
    if (trace && warp == 2 && lane == 0) {
      trace[TRACE_EPI_WAIT] = static_cast<unsigned long long>(epi_wait);
      trace[TRACE_EPI_BUSY] = static_cast<unsigned long long>(epi_busy);
      trace[TRACE_TILES] = static_cast<unsigned long long>(tiles_done);
    }
  }

  // Teardown: every role gets here (all waits are bounded).  In a pair neither
  // CTA may release TMEM or exit while the other can still touch its memory.
  ptx::tc_fence_before_sync();
  if constexpr (CTA_GROUP == 2 || CSPLIT > 1) {
    __syncwarp();
    ptx::cluster_sync();
  } else {
    __syncthreads();
  }
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc<CTA_GROUP>(tmem_base, TMEM_COLS);
  }
  if constexpr (AHEAD) {
    if (threadIdx.x == 0) s4a_cta_exit(p.ahead);  // every claim of this CTA lies before the barrier above
  }
  if (trace && threadIdx.x == 0) {
    trace[TRACE_CYCLES] = static_cast<unsigned long long>(clock64() - clk_start);
    trace[TRACE_NANOS] = ptx::globaltimer_ns() - ns_start;
  }
}

}  // namespace b200gemm
