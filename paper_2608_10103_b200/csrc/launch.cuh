// Launch plumbing: one kernel variant per (kind, tile shape, output mode), argument checks
// shared by the entry points, the INT4 pre-pass and its workspaces.
#pragma once

#include <utility>

#include "few_rows.cuh"
#include "gemm_wide.cuh"
#include "runtime.cuh"
#include "selector.cuh"
#include "unpack_s4.cuh"

namespace b200gemm {
namespace {

// Zeroes C ahead of a split-K GEMM.  Like the GEMMs it is launched to start early and lets its
// successor start early: the launch latencies of the zeroing and of the GEMM behind it overlap
// the tail of whatever runs in front, and each waits for its predecessor to complete before
// it touches global memory -- which takes two launch gaps off the critical path of the small,
// latency-bound problems that split K.
__global__ void zero_c_kernel(uint4* c16, size_t n16, uint32_t* tail, int tail_words, int chained) {
  ptx::grid_dep_launch_dependents();
  if (chained) ptx::grid_dep_wait();  // launched early itself: the grid in front may still use C
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n16; i += stride)
    c16[i] = make_uint4(0, 0, 0, 0);
  if (blockIdx.x == 0 && static_cast<int>(threadIdx.x) < tail_words) tail[threadIdx.x] = 0;
}

// Kernel variants that also exist with the measurement / drill switches compiled in, and the
// attr_set bit of that twin (208..): the two 256-wide tiles of the raw outputs, two of the
// fused INT4 kernels and the 4-way cluster split-K kernel -- the ones the ablation runs and
// the failure drills use.
template <int KIND, int BN, int STAGES, int CTA_GROUP, int KB, int EPI, int PSTAGES, int CSPLIT>
constexpr int dbg_twin_bit() {
  if (EPI == EPI_RAW32 && CSPLIT == 1 && PSTAGES == 0 && BN == 256 &&
      ((CTA_GROUP == 1 && STAGES == 4) || (CTA_GROUP == 2 && STAGES == 6)))
    return 208 + (KIND == ptx::KIND_F16 ? 0 : 2) + (CTA_GROUP - 1);
  if (KIND == ptx::KIND_I8 && EPI == EPI_RAW32 && CSPLIT == 1 && PSTAGES > 0 && BN == 256 &&
      CTA_GROUP == 2)
    return 212;
  if (KIND == ptx::KIND_I8 && EPI == EPI_RAW32 && CSPLIT == 1 && PSTAGES > 0 && BN == 32) return 213;
  if (KIND == ptx::KIND_I8 && EPI == EPI_OUT16 && CSPLIT == 4 && PSTAGES == 0) return 214;
  return -1;
}

template <class Kernel>
int launch_kernel(DeviceState* s, Kernel kernel, int variant, int dyn_bytes, int threads,
                  int cluster, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc,
                  const GemmParams& p, cudaStream_t stream) {
  if (!(s->attr_set[variant >> 6].load(std::memory_order_relaxed) & (1ull << (variant & 63)))) {
    cudaError_t e =
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn_bytes);
    if (e != cudaSuccess) return cuda_fail(e);
    s->attr_set[variant >> 6].fetch_or(1ull << (variant & 63), std::memory_order_relaxed);
  }
  const long long all_tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
  const long long tiles = p.split_from + (all_tiles - p.split_from) * p.splits;  // work units
  const long long units = s->num_sms / cluster;
  int grid = static_cast<int>((tiles < units ? tiles : units) * cluster);
  if (p.sk_share > 0)  // even shares: one CTA (pair) per share
    grid = static_cast<int>((p.sk_total + p.sk_share - 1) / p.sk_share) * cluster;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(threads, 1, 1);
  cfg.dynamicSmemBytes = dyn_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.wait_prior_grid ? 2 : 1;  // may start while the grid in front still runs
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, ta, tb, tc, p);
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

template <int KIND, int BN, int STAGES, int CTA_GROUP, int KB, int EPI, int PSTAGES = 0,
          int CSPLIT = 1>
int launch_variant(DeviceState* s, int variant, const CUtensorMap& ta, const CUtensorMap& tb,
                   const CUtensorMap& tc, const GemmParams& p, cudaStream_t stream) {
  using L = SmemLayout<BN, STAGES, CTA_GROUP, KB, PSTAGES, CSPLIT>;
  constexpr int THREADS = PSTAGES > 0 ? NUM_THREADS_FUSED : NUM_THREADS;
  constexpr int CLUSTER = CTA_GROUP * CSPLIT;  // CTAs that work on one unit together
  if (p.ablate) {
    constexpr int twin = dbg_twin_bit<KIND, BN, STAGES, CTA_GROUP, KB, EPI, PSTAGES, CSPLIT>();
    if constexpr (twin >= 0) {
      return launch_kernel(s, gemm_kernel<KIND, BN, STAGES, CTA_GROUP, KB, EPI, PSTAGES, CSPLIT, true>,
                           twin, L::DYN_BYTES, THREADS, CLUSTER, ta, tb, tc, p, stream);
    } else {
      return GEMM_ERR_INVALID_ARG;  // this variant is not built with the switches
    }
  }
  return launch_kernel(s, gemm_kernel<KIND, BN, STAGES, CTA_GROUP, KB, EPI, PSTAGES, CSPLIT>,
                       variant, L::DYN_BYTES, THREADS, CLUSTER, ta, tb, tc, p, stream);
}

// The 512 x 256 CTA-pair kernel for large problems (gemm_wide.cuh).  attr_set bits 160..
template <int KIND, int EPI>
int launch_wide(DeviceState* s, const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p,
                cudaStream_t stream) {
  const bool dbg = p.ablate != 0;
  if (dbg && EPI != EPI_RAW32) return GEMM_ERR_INVALID_ARG;  // switches exist for the raw outputs
  const int variant = 160 + ((KIND == ptx::KIND_F16) ? 0 : 8) + EPI * 2 + (dbg ? 1 : 0);
  void (*kernel)(CUtensorMap, CUtensorMap, GemmParams) = gemm_wide_kernel<KIND, EPI, false>;
  if constexpr (EPI == EPI_RAW32) {
    if (dbg) kernel = gemm_wide_kernel<KIND, EPI, true>;
  }
  if (!(s->attr_set[variant >> 6].load(std::memory_order_relaxed) & (1ull << (variant & 63)))) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         WideSmem::DYN_BYTES);
    if (e != cudaSuccess) return cuda_fail(e);
    s->attr_set[variant >> 6].fetch_or(1ull << (variant & 63), std::memory_order_relaxed);
  }
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
  const long long pairs = s->num_sms / 2;
  const int grid = static_cast<int>((tiles < pairs ? tiles : pairs) * 2);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(WIDE_THREADS, 1, 1);
  cfg.dynamicSmemBytes = WideSmem::DYN_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.wait_prior_grid ? 2 : 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, ta, tb, p);
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

// Band height (in tiles) of the raster for a tile of `rows_per_tile` x `bn`: one wave of tiles
// about twice as tall as wide in operand bytes, then evened out over the bands so that no
// short last band streams the other operand for little work.
int band_height(int M, int rows_per_tile, int bn, int units) {
  int g = 1;
  while ((g + 1) * (g + 1) * rows_per_tile <= 2 * units * bn) ++g;
  if (g_override_group_m) g = g_override_group_m;
  const int tiles_m = ceil_div(M, rows_per_tile);
  if (g > tiles_m) g = tiles_m;
  if (g < 1) g = 1;
  if (!g_override_group_m) g = ceil_div(tiles_m, ceil_div(tiles_m, g));
  return g;
}

// Whether a problem goes to the 512 x 256 kernel.  It needs the same number of SM cycles as the
// 256 x 256 pair tile but a quarter fewer operand bytes from L2, which buys clock on a
// power-capped part; its tiles are twice as large, so it needs enough of them to fill its waves.
bool wide_wanted(const TileConfig& cfg, int M, int N, int k_blocks, int num_sms, bool swap,
                 bool csplit, bool packed_s4, bool fp16_kind) {
  if (swap || csplit || packed_s4 || g_family == 1) return false;
  if (g_family == 2) return !(g_override_bn && g_override_bn != 256) && g_override_cta_group != 1 &&
                            g_override_splits <= 1;
  if (cfg.bn != 256 || cfg.cta_group != 2 || cfg.splits != 1) return false;
  const long long tiles = static_cast<long long>(ceil_div(M, WIDE_TILE_M)) * ceil_div(N, WIDE_BN);
  const long long pairs = num_sms / 2;
  const long long waves = (tiles + pairs - 1) / pairs;
  // At least two waves, at least 90 % full, and tiles long enough that the hand-over between
  // them (~4.5 k cycles per tile that the 256 x 256 kernel does not have) stays small.  Measured
  // in alternating sustained loops, FP16 with 8192 x 8192 outputs: +3 % at K = 8192, +2 % at
  // 6144, even at 4096, -2 % at 2048.  The integer kinds' tiles take half as long for the same
  // C bytes, so the hand-over weighs twice as much: the kernel needs more SM cycles there
  // (N = 8192: 525 k against 496 k) and still wins on the power-capped part from K = 8192 on
  // (8192^3 +1.8 %, 16384 x 8192 x 8192 +2.4 %, 8192 x 8192 x 16384 +5 %; 6144^3 -1 %).
  return tiles >= 2 * pairs && 10 * tiles >= 9 * waves * pairs && k_blocks >= (fp16_kind ? 96 : 64);
}

// Output options of one GEMM call.
struct OutputSpec {
  int epi = EPI_RAW32;
  const float* row_scale = nullptr;
  const float* col_scale = nullptr;
  long long ldc = 0;        // row pitch of C in elements; 0 = dense (N)
  bool no_split = false;    // C is a block of a larger matrix: never zero / add into it
  bool tiles_only = false;  // the GEMM of the INT4 pre-pass route: always a tile kernel
};

// Overlapped INT4 pre-pass: A and B of the call are the (not yet written) int8 images in a
// scratch buffer, these are the packed operands they are to be made from inside the GEMM
// kernel, and `sync` its bookkeeping words (see s4_ahead.cuh).
struct S4AheadReq {
  const uint8_t* packed_a;
  const uint8_t* packed_b;
  uint32_t* sync;
};

// Returned (never to the caller of the library) when a call with an S4AheadReq is not one the
// overlapped kernel takes: nothing has been enqueued, the caller runs the pre-pass launch.
constexpr int GEMM_NOT_AHEAD = 2;

thread_local int t_last_s4_overlapped = 0;

// Hybrid fused INT4 (CTA-pair tiles, plain orientation): B stays packed and is expanded inside
// the kernel, A comes as the int8 image expand_s4_slots_kernel makes (rows of a8_pitch bytes,
// K rounded up to 256).  A call that would take this form but was given no image enqueues
// nothing and returns GEMM_WANT_A8; the caller makes the image and calls again.
struct S4HybridReq {
  const int8_t* a8;
  size_t a8_pitch;
};
constexpr int GEMM_WANT_A8 = 3;

// Index in attr_set of the unfused cluster split-K variants: 96.., by kind, output mode, width.
template <int KIND, int EPI>
constexpr int csplit_variant_base() {
  return 96 + ((KIND == ptx::KIND_F16) ? 0 : 16) + EPI * 2;
}

// How many clusters of four CTAs of the 4-way cluster split-K kernel the device holds at once.
// (Clusters are placed inside one GPC, so this is less than SMs / 4 when a GPC's SM count is
// not a multiple of four: a tile more than that would wait for a second wave.)
template <int KIND, int EPI>
int quad_clusters_resident(DeviceState* s, int variant) {
  std::atomic<int>& cached = s->quad_clusters[KIND == ptx::KIND_F16 ? 0 : 1][EPI];
  if (cached.load()) return cached.load();
  using L = SmemLayout<32, 3, 1, 2, 0, 4>;
  auto kernel = gemm_kernel<KIND, 32, 3, 1, 2, EPI, 0, 4>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES) !=
      cudaSuccess)
    return 0;
  s->attr_set[variant >> 6].fetch_or(1ull << (variant & 63), std::memory_order_relaxed);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(s->num_sms / 4 * 4), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = L::DYN_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 4;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    n = s->num_sms / 8;  // unknown: assume half
  }
  cached.store(n);
  return n;
}

// Whether the selector's choice can run as split-K inside a cluster of two or four CTAs
// (four only for the 32-wide tile, where the buffers fit).
bool cluster_split_ok(const TileConfig& c, int M, int N) {
  const long long tiles = static_cast<long long>(ceil_div(M, BM * c.cta_group)) * ceil_div(N, c.bn);
  if (c.cta_group != 1 || c.bn > 64 || c.split_tiles != tiles) return false;
  return c.splits == 2 || (c.splits == 4 && c.bn == 32);
}

// Whether the packed route is taken for the tile the selector picked.  Scheme 2 forces it
// wherever a variant exists; scheme 0 (automatic) takes it where a pre-pass over the operands
// does not pay: problems with few rows on one side (LLM decoding), which are bound by the
// bytes of the other operand, and small problems, whose time is launches and latencies and
// which save one launch (measured: 10-26 % faster up to 1024^2 outputs, 8 % for a single wave
// of pair tiles such as 2048^3, even or slower beyond).
bool s4_fused_wanted(int M, int N, const TileConfig& cfg, int num_sms) {
  if (s4_fused_forced()) return true;
  if (s4_prepass_forced()) return false;
  if (cfg.cta_group == 2) {  // (the 128-wide pair tile only comes in through select_fused_s4)
    const long long tiles = static_cast<long long>(ceil_div(M, 2 * BM)) * ceil_div(N, cfg.bn);
    return cfg.bn == 256 && tiles <= num_sms / 2;
  }
  return M <= 128 || N <= 128 || (M <= 1024 && N <= 1024);
}

// The INT4 route of a problem (M, N: the kernel's, user_m/user_n: the caller's): true, with
// the tile in *out, when the nibbles are expanded inside the GEMM kernel.  First the selector's
// free choice, taken if the fused kernel has that shape and s4_fused_wanted agrees.  Then
// problems with a short side: the pre-pass costs the bytes of BOTH operands, (M + N) K, the
// expansion inside the kernel costs shared-memory time that grows with the work, M N K, so
// what decides is M N / (M + N).  Up to 384 the selector's best choice among all the shapes
// the fused kernel has is taken; up to 1024 rows or columns its 256-wide CTA-pair shape, the
// efficient one, where the work units fill their waves to 75 %.  A pair tile that would have
// to split K where the INT8 kernel behind the pre-pass (`int8_choice`) would not is left to
// the pre-pass (1024 x 2048 x 8192: 24.1 against 22.5 us).  Measured, packed B from HBM:
// 256 x 28672 x 8192 119 -> 67 us, 512 x 16384 x 4096 44 -> 35 us, 256 x 8192 x 8192 35 -> 28 us,
// 512 x 4096 x 16384 49 -> 38 us, 1024 x 8192 x 8192 63 -> 60 us; the one-CTA shapes at
// 640-1024 x 2048 x 8192 would lose 15-35 %, and from 1280 rows on the pre-pass is even or ahead.
bool select_fused_s4(int M, int N, int user_m, int user_n, int num_sms, int k_blocks, int min_bn,
                     bool allow_split, const TileConfig& int8_choice, TileConfig* out) {
  if (s4_prepass_forced()) return false;
  const TileConfig c = select_config(M, N, num_sms, k_blocks, min_bn, allow_split, 2);
  const auto pair_split_only_here = [&](const TileConfig& f) {
    return g_s4_scheme == 0 && f.cta_group == 2 && f.splits > 1 && int8_choice.splits == 1;
  };
  if (c.bn != 0 && fused_s4_variant_exists(c.bn, c.cta_group, c.splits) &&
      s4_fused_wanted(user_m, user_n, c, num_sms) && !pair_split_only_here(c)) {
    *out = c;
    return true;
  }
  const long long mn = static_cast<long long>(user_m) * user_n;
  if (s4_fused_forced() || mn <= 384ll * (user_m + user_n)) {
    const TileConfig f = select_config(M, N, num_sms, k_blocks, min_bn, allow_split, 2, 0, 1);
    if (f.bn != 0) {
      *out = f;
      return true;
    }
  }
  if (user_m <= 1024 || user_n <= 1024) {
    const TileConfig f = select_config(M, N, num_sms, k_blocks, min_bn, allow_split, 2, 0, 2);
    if (f.bn != 0) {
      // work units: tiles, those of a split-K part counted once per K range
      const long long tiles = static_cast<long long>(ceil_div(M, 2 * BM)) * ceil_div(N, f.bn) +
                              static_cast<long long>(f.split_tiles) * (f.splits - 1);
      const long long pairs = num_sms / 2;
      const long long waves = (tiles + pairs - 1) / pairs;
      if (4 * tiles >= 3 * waves * pairs && !pair_split_only_here(f)) {
        *out = f;
        return true;
      }
    }
  }
  if (user_m > 1024 && user_n > 1024) {
    // Large in both dimensions: the fused 256-wide CTA-pair kernel again, usually in its hybrid
    // form.  Its mainloop needs more SM cycles than the INT8 kernel behind a pre-pass (N = 8192:
    // 591 k against 528 k) but no pre-pass over both operands, and it draws less power, which on
    // this power-capped part is clock: measured 20-launch / 0.4 s loops, pre-pass route ->
    // fused, 8192^3 359 / 409 -> 337 / 379 us (INT8 on int8 operands: 342 / 385), 6144^3
    // 165 / 187 -> 154 / 170, 4096^3 57.5 / 64.3 -> 57.7 / 56.9, 2048 x 8192 x 8192 110 / 124 ->
    // 97 / 101, 8192 x 2048 x 8192 112 / 126 -> 101 / 101, 3072^3 28.4 / 29.3 -> 27.0 / 26.1;
    // of fifteen shapes between 2048 and 16384 the pre-pass was ahead on none by more than 0.5 %.
    // (at least one wave of pair tiles and K >= 2048: what was measured)
    const TileConfig f = select_config(M, N, num_sms, k_blocks, min_bn, allow_split, 2, 0, 2);
    const long long tiles = static_cast<long long>(ceil_div(M, 2 * BM)) * ceil_div(N, 256);
    if (f.bn != 0 && tiles >= num_sms / 2 && k_blocks >= 16 && !pair_split_only_here(f)) {
      *out = f;
      return true;
    }
  }
  return false;
}

// Even shares for the one-CTA fused INT4 tiles with split-K through C (problems with few rows,
// bound by the shared-memory time of the expansion, i.e. by the busiest SM): returns the share
// in packed slots per CTA, or 0 where whole tiles or equal tile parts do as well.  Taken when
// the busiest SM's work falls by a fifth or more -- 150 or 224 tiles on 148 SMs make some SMs do
// two tiles where the average is 1.0 or 1.5 (M = 32, N = 28672, K = 8192: 39.4 -> 35.5 us) --
// and a share is at least 16 packed slots.  Smaller gains on paper are eaten by the second
// piece a CTA then has (M = 16, N = K = 8192, 16 -> 14 slots per CTA: 15.2 -> 15.4 us).
int s4_even_share(long long tiles, int k_blocks, int splits, long long split_tiles, int num_sms) {
  if (g_l2_policy & 128) return 0;
  const long long per_tile = k_blocks / 2;  // packed slots
  const long long total = tiles * per_tile;
  const long long cur_units = (splits > 1 && split_tiles == tiles) ? tiles * splits : tiles;
  const long long cur = ((cur_units + num_sms - 1) / num_sms) *
                        ((splits > 1 && split_tiles == tiles) ? (per_tile + splits - 1) / splits : per_tile);
  const long long share = (total + num_sms - 1) / num_sms;
  // short shares lose to the second piece (epilogue, adds, pipeline refill) a CTA then has:
  // measured 16 x 24000 x 4096 (share 21) 23.0 -> 19.9 us, 8 x 29440 x 4096 (25) 23.1 -> 21.4,
  // 24 x 26000 x 2048 (12) even, 64 x 21000 x 1056 (6) 13.8 -> 15.5 us
  if (share < 16) return 0;
  if (splits > 1 && split_tiles != tiles) return 0;  // a split of the last wave only stays as it is
  if (splits == 1 && tiles <= num_sms) return 0;     // the selector found no split worth its cost
  return share * 100 <= cur * 80 ? static_cast<int>(share) : 0;
}

// Whether a fused INT4 call on a CTA-pair tile takes A as an int8 image made beforehand (the
// hybrid form).  Measured, the kernel gains 14-20 % from not expanding A again for every tile
// column; the image costs a launch in the chain (~2.5 us) plus its bytes (1/2 read + 1 written
// per element at ~5 TB/s).  256 / 512 / 1024 x 28672 x 8192: 66.5 -> 55.2, 102.0 -> 83.8,
// 177.3 -> 149.1 us (the INT8 kernel on pre-expanded operands: 56.3, 86.9, 158.9);
// 1024 x 8192 x 8192 59.7 -> 55.0, 512 x 16384 x 4096 35.4 -> 33.4; 256 x 8192 x 8192 and
// 384 x 12288 x 4096 even, 2048^3 14.5 -> 16.5 are the other side of the rule; so are a
// tall A against few tile columns (8192 x 2048 x 8192: 101 -> 112 us) and mid-sized squares
// (4096^3 57.7 -> 59.6, 3072^3 27.0 -> 29.7), where the image costs more than it saves, while
// 8192^3 gains 377 -> 337 us and 2048 x 8192 x 8192 108 -> 97.  Scheme 5 never, scheme 6 always
// (tests, ablation).
bool s4_hybrid_wanted(int M, int N, int K) {
  if (g_s4_scheme == 5) return false;
  if (g_s4_scheme == 6) return true;
  const double gain = 0.14 * 2.0 * M * static_cast<double>(N) * K / 1.9e15;
  const double cost = 2.5e-6 + 1.5 * M * static_cast<double>(K) / 5.0e12;
  return gain > 1.1 * cost + 2.0e-6;
}

// Whether the kernel runs on exchanged operands (its rows = the caller's N side).  The 128-row
// side of a tile is then filled by the long operand of a problem with few rows (LLM decoding:
// M = 1..64), instead of 128 - M rows of zero fill taking shared memory, ring depth and, on
// the fused INT4 route, expansion work; C goes out by plain stores that are contiguous along
// the caller's N.  Automatic when N >= 1024 and M <= 32 (FP16 with FP32 output) or M <= 64 (the
// integer kinds, both INT4 routes, and FP16 with FP16 output): measured 2-12 % faster there
// (INT8, M = 48-64: 3-8 %; FP16 -> FP16, M = 40-64: 1-13 %; FP16 -> FP32 even; from M = 80 on,
// where the narrow side needs the 128-wide tile, 4-20 % slower).
bool swap_ab_wanted(int M, int N, bool integer_kind, const OutputSpec& out) {
  if (out.no_split || out.ldc) return false;  // C is a block of a larger matrix
  if (g_swap_ab == 1) return false;
  if (g_swap_ab == 2) return true;
  // (FP16 -> FP32 at M = 33..64: 3-4 % faster from N = 16384 on, 2-4 % slower at N = 8192)
  return N >= 1024 && M <= ((integer_kind || out.epi == EPI_OUT16 || N >= 16384) ? 64 : 32);
}

// Returned (never to the caller of the library) when the fused INT4 kernel does not cover the
// shape the selector picked: the entry point then takes the pre-pass route.
constexpr int GEMM_NOT_FUSED = 1;

// A, B in the element type of KIND (fp16 or int8), pitches in bytes.  packed_s4 (KIND_I8
// only): A and B hold packed signed 4-bit values, K/2 bytes per row, and go to the kernel
// variant that expands them on the way to the MMAs; where select_fused_s4 leaves the problem
// to the pre-pass GEMM_NOT_FUSED comes back and nothing has been enqueued.
template <int KIND, int EPI>
int launch_gemm_epi(int M, int N, int K, const void* A, size_t a_pitch, const void* B,
                    size_t b_pitch, void* C, const OutputSpec& out, cudaStream_t stream,
                    bool packed_s4 = false, const S4AheadReq* req = nullptr,
                    const S4HybridReq* hyb = nullptr) {
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  constexpr int ELEM = (KIND == ptx::KIND_F16) ? 2 : 1;
  constexpr int C_ELEM = (EPI == EPI_OUT16) ? 2 : 4;
  const long long ldc = out.ldc ? out.ldc : N;
  const int user_m = M, user_n = N;
  const bool swap = swap_ab_wanted(M, N, KIND == ptx::KIND_I8, out);
  if (swap) {  // from here on M, N, A, B are the kernel's
    std::swap(M, N);
    std::swap(A, B);
    std::swap(a_pitch, b_pitch);
  }
  const CUtensorMapDataType type =
      (KIND == ptx::KIND_F16) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  // the selector sees the int8 problem either way, so both INT4 routes get the same tile
  int k_blocks = ceil_div(static_cast<long long>(K) * ELEM, BK_BYTES);
  // 16-bit outputs are staged 64 columns at a time; with exchanged operands C goes out by
  // plain stores and the 32-wide tile serves them too
  const int min_bn = (EPI == EPI_OUT16 && !swap) ? 64 : 32;
  const bool split_through_c = EPI == EPI_RAW32 && !out.no_split;
  TileConfig cfg = select_config(M, N, s->num_sms, k_blocks, min_bn, split_through_c);
  bool fused_cfg = false;
  if (packed_s4)
    fused_cfg = select_fused_s4(M, N, user_m, user_n, s->num_sms, k_blocks, min_bn,
                                split_through_c, TileConfig(cfg), &cfg);
  if (cfg.bn == 0) return GEMM_ERR_INVALID_ARG;  // override asks for a shape this mode lacks
  // Outputs that cannot be split through C (16-bit, scaled, blocks of a larger C): split-K
  // inside a cluster of two or four CTAs where the kernel has that variant (one-CTA tiles up
  // to 64 wide, every tile split the same way) -- no zeroing of C, no adds in global memory.  Where the
  // raw 32-bit output can split through C that stays the choice: with the launches chained it
  // measured ~1 us faster per call than the hand-over inside the cluster.
  bool csplit = false;
  if (!split_through_c && !(g_l2_policy & 64)) {
    // try up to four CTAs per tile (all clusters at once, unless the split is forced), then two
    for (int cap = 4; cap >= 2 && !csplit; cap -= 2) {
      const TileConfig c2 =
          select_config(M, N, s->num_sms, k_blocks, min_bn, true, packed_s4 ? 2 : 0, cap);
      if (c2.bn == 0 || !cluster_split_ok(c2, M, N)) continue;
      if (c2.splits == 4 && (EPI != EPI_OUT16 || swap)) {
        if (!g_override_splits &&
            c2.split_tiles > quad_clusters_resident<KIND, EPI>(s, csplit_variant_base<KIND, EPI>() + 8))
          continue;
      } else if (c2.splits == 4) {
        continue;  // 16-bit outputs take the 32-wide tile only with exchanged operands
      }
      cfg = c2;
      csplit = true;
    }
  }
  if (packed_s4) {
    if (KIND != ptx::KIND_I8) return GEMM_NOT_FUSED;
    if (csplit ? !s4_fused_wanted(user_m, user_n, cfg, s->num_sms) : !fused_cfg)
      return GEMM_NOT_FUSED;
    k_blocks = 2 * ceil_div(K, 2 * BK_BYTES);  // one packed slot (256 values of K) = two int8 slots
  }
  // The CTA-pair fused tiles serve problems with a short M against a large N K (and single
  // waves): every tile column would expand the same rows of A again, so A is expanded once,
  // beforehand (scheme 5 keeps both operands packed; so do the runs with measurement switches).
  bool hybrid = packed_s4 && !swap && !csplit && cfg.cta_group == 2 && (g_trace_on >> 1) == 0 &&
                s4_hybrid_wanted(M, N, K);
  if (hybrid && !hyb) return GEMM_WANT_A8;
  if (hybrid && !hyb->a8) hybrid = false;  // the caller has no scratch for the image: both packed
  int even_share = 0;
  if (packed_s4 && !hybrid && !csplit && cfg.cta_group == 1 && split_through_c && (g_trace_on >> 1) == 0) {
    const long long tiles = static_cast<long long>(ceil_div(M, BM)) * ceil_div(N, cfg.bn);
    even_share = s4_even_share(tiles, k_blocks, cfg.splits, cfg.split_tiles, s->num_sms);
    if (even_share) {  // every piece is added into a zeroed C
      if (cfg.splits < 2) cfg.splits = 2;
      cfg.split_tiles = static_cast<int>(tiles);
    }
  }

  // (a call that asks for the overlapped INT4 pre-pass stays on the kernel that has that role)
  const bool wide = !req && wide_wanted(cfg, M, N, k_blocks, s->num_sms, swap, csplit, packed_s4,
                                        KIND == ptx::KIND_F16);
  if (wide) {
    cfg.bn = WIDE_BN;
    cfg.cta_group = 2;
    cfg.splits = 1;
    cfg.split_tiles = 0;
    cfg.group_m = band_height(M, WIDE_TILE_M, WIDE_BN, s->num_sms / 2);
  }
  bool ahead = false;
  const int rows_per_cta = wide ? WIDE_CTA_ROWS : BM;
  if (req) {
    // The overlapped pre-pass rides on the 256 x 256 pair-tile kernel of large problems: at
    // least two waves of tiles, so that the expansion is done long before the GEMM is.  Only on
    // request (scheme 4): measured, it loses to the separate launch.  While the four pre-pass
    // warps per CTA are at work (the first ~130 k cycles at N = 8192) the GEMM's mainloop runs at
    // ~60 % of its speed -- that kernel keeps the SM's L2 port and shared-memory pipe full with
    // operand tiles already -- and the first wave starts a batch of chunks late: 573 k SM cycles
    // against 495 k + a 36 us (~50 k cycle) pre-pass.  The same role inside the 512 x 256 kernel,
    // whose L2 port has a quarter to spare, measured no better (596 k against ~520 k).
    const long long tiles = static_cast<long long>(ceil_div(M, 2 * BM)) * ceil_div(N, 256);
    ahead = KIND == ptx::KIND_I8 && !wide && !swap && !csplit && !packed_s4 && cfg.bn == 256 &&
            cfg.cta_group == 2 && cfg.stages == 6 && g_s4_scheme == 4 && (g_trace_on >> 1) == 0 &&
            tiles >= 2 * (s->num_sms / 2);
    if (!ahead) return GEMM_NOT_AHEAD;
  }
  CUtensorMap ta, tb;
  const bool promote = !(g_l2_policy & 16);
  // packed: the tensor is K/2 bytes wide; boxes stay 128 bytes
  const uint64_t k_cols = packed_s4 ? static_cast<uint64_t>(K) / 2 : static_cast<uint64_t>(K);
  if (hybrid) {
    rc = encode_operand_map(&ta, type, ELEM, hyb->a8, M, static_cast<uint64_t>(k_blocks) * BK_BYTES,
                            hyb->a8_pitch, rows_per_cta, promote);
  } else {
    rc = encode_operand_map(&ta, type, ELEM, A, M, k_cols, a_pitch, rows_per_cta, promote);
  }
  if (rc != GEMM_OK) return rc;
  rc = encode_operand_map(&tb, type, ELEM, B, N, k_cols, b_pitch, cfg.bn / cfg.cta_group, promote);
  if (rc != GEMM_OK) return rc;

  GemmParams p;
  p.M = M;
  p.N = N;
  p.K = K;
  p.tiles_m = ceil_div(M, rows_per_cta * cfg.cta_group);
  p.tiles_n = ceil_div(N, cfg.bn);
  p.group_m = cfg.group_m;
  p.k_blocks = k_blocks;
  p.splits = csplit ? 1 : cfg.splits;
  p.split_from = p.tiles_m * p.tiles_n - ((cfg.splits > 1 && !csplit) ? cfg.split_tiles : 0);
  p.ldc = ldc;
  p.transpose_c = swap ? 1 : 0;
  // policy bit 32: plain stream order; so are traced launches, whose cycle counts would
  // otherwise include the time spent waiting for the predecessor's tail
  p.wait_prior_grid = ((g_l2_policy & 32) || (g_trace_on & 1)) ? 0 : 1;
  p.c_vec_ok = !swap && (ldc % (16 / C_ELEM) == 0) && (reinterpret_cast<uintptr_t>(C) % 16 == 0);
  if (wide && N % (16 / C_ELEM)) p.c_vec_ok = 0;  // its 16-byte stores must end on a row's end
  CUtensorMap tc;
  if (wide) {
    tc = ta;  // the wide kernel writes C with plain stores
  } else if (p.c_vec_ok) {
    // split-K adds into C by TMA reduction, which takes the element type from the map
    rc = encode_c_map(&tc, C, M, N, ldc, C_ELEM,
                      cfg.splits == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT32
                      : KIND == ptx::KIND_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                              : CU_TENSOR_MAP_DATA_TYPE_INT32);
    if (rc != GEMM_OK) return rc;
  } else {
    tc = ta;  // unused by the kernel on the plain-store path
  }
  p.C = static_cast<uint32_t*>(C);
  p.row_scale = swap ? out.col_scale : out.row_scale;  // indexed by the kernel's rows
  p.col_scale = swap ? out.row_scale : out.col_scale;
  p.status = s->status_ptr;
  p.trace = (g_trace_on & 1) ? s->trace_ptr : nullptr;
  p.ablate = (g_trace_on >> 1) & 63;
  p.l2_policy = g_l2_policy & 3;
  // Default policy, one tile column or one tile row (problems with few rows on one side): the
  // short operand, which every CTA re-reads, gets the same priority in L2 as the long one that
  // streams past it once ("normal" let it be pushed out: INT8 M = 1, N = K = 8192 15.4 -> 11.9 us;
  // marking the long operand "evict first" instead costs more than it saves, because each
  // 256-byte L2 fetch serves two consecutive k-blocks)
  if (p.l2_policy == 3 && (p.tiles_n == 1 || p.tiles_m == 1)) p.l2_policy = 2;
  p.serpentine_k = (g_l2_policy & 4) ? 0 : 1;
  p.c_evict_first = (g_l2_policy & 8) ? 1 : 0;
  p.sk_share = even_share;
  p.sk_total = even_share ? static_cast<long long>(p.tiles_m) * p.tiles_n * (k_blocks / 2) : 0;
  p.ahead = S4Ahead();
  if (ahead) {
    p.ahead.packed_a = reinterpret_cast<const uint4*>(req->packed_a);
    p.ahead.packed_b = reinterpret_cast<const uint4*>(req->packed_b);
    p.ahead.a8 = static_cast<int8_t*>(const_cast<void*>(A));
    p.ahead.b8 = static_cast<int8_t*>(const_cast<void*>(B));
    p.ahead.sync = req->sync;
    p.ahead.M = M;
    p.ahead.N = N;
    p.ahead.K = K;
    S4AheadPlan& pl = p.ahead.plan;
    pl.ra = ceil_div(M, S4A_CHUNK_ROWS);
    pl.rb = ceil_div(N, S4A_CHUNK_ROWS);
    pl.kc = ceil_div(K, S4A_CHUNK_COLS);
    pl.ga = 2 * BM / S4A_CHUNK_ROWS;
    pl.gb = 256 / S4A_CHUNK_ROWS;
    // what the first wave of tiles reads: the first band's rows of A, and as many tile columns
    // of B as one wave of CTA pairs covers in that band
    const int band = p.group_m < p.tiles_m ? p.group_m : p.tiles_m;
    const int first_cols = ceil_div(s->num_sms / 2, band);
    pl.ra1 = band * pl.ga < pl.ra ? band * pl.ga : pl.ra;
    pl.rb1 = first_cols * pl.gb < pl.rb ? first_cols * pl.gb : pl.rb;
  }

  if (wide) return launch_wide<KIND, EPI>(s, ta, tb, p, stream);
  if (cfg.splits > 1 && !csplit) {  // only with a dense C (no_split is set for blocks of a larger matrix)
    // Split tiles add into C: zero them first.  All tiles: one memset.  The last wave only:
    // the bounding rectangle of those tiles (other tiles inside it are overwritten later).
    cudaError_t e;
    if (p.split_from == 0 || swap) {
      const size_t bytes = static_cast<size_t>(M) * N * C_ELEM;  // a multiple of 4 (32-bit C only)
      const size_t n16 = bytes / 16;
      size_t blocks = (n16 + 255) / 256;
      if (blocks > static_cast<size_t>(s->num_sms) * 4) blocks = static_cast<size_t>(s->num_sms) * 4;
      if (blocks < 1) blocks = 1;
      cudaLaunchConfig_t zc = {};
      zc.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
      zc.blockDim = dim3(256, 1, 1);
      zc.stream = stream;
      cudaLaunchAttribute za[1];
      za[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      za[0].val.programmaticStreamSerializationAllowed = 1;
      zc.attrs = za;
      zc.numAttrs = p.wait_prior_grid ? 1 : 0;
      e = cudaLaunchKernelEx(&zc, zero_c_kernel, static_cast<uint4*>(C), n16,
                             reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(C) + n16 * 16),
                             static_cast<int>((bytes % 16) / 4), p.wait_prior_grid);
    } else {
      int tm_lo = p.tiles_m, tm_hi = -1, tn_lo = p.tiles_n, tn_hi = -1;
      for (int t = p.split_from; t < p.tiles_m * p.tiles_n; ++t) {
        // the kernel's raster (tile_coords), on the host
        const int band_tiles = p.group_m * p.tiles_n;
        const int band = t / band_tiles;
        const int first_m = band * p.group_m;
        const int rows_in_band =
            p.group_m < p.tiles_m - first_m ? p.group_m : p.tiles_m - first_m;
        const int r = t - band * band_tiles;
        const int tm = first_m + r % rows_in_band, tn = r / rows_in_band;
        tm_lo = tm < tm_lo ? tm : tm_lo;
        tm_hi = tm > tm_hi ? tm : tm_hi;
        tn_lo = tn < tn_lo ? tn : tn_lo;
        tn_hi = tn > tn_hi ? tn : tn_hi;
      }
      const long long row_lo = static_cast<long long>(tm_lo) * BM * cfg.cta_group;
      long long row_hi = static_cast<long long>(tm_hi + 1) * BM * cfg.cta_group;
      const long long col_lo = static_cast<long long>(tn_lo) * cfg.bn;
      long long col_hi = static_cast<long long>(tn_hi + 1) * cfg.bn;
      if (row_hi > M) row_hi = M;
      if (col_hi > N) col_hi = N;
      e = cudaMemset2DAsync(static_cast<uint8_t*>(C) + (row_lo * ldc + col_lo) * C_ELEM,
                            static_cast<size_t>(ldc) * C_ELEM, 0,
                            static_cast<size_t>(col_hi - col_lo) * C_ELEM,
                            static_cast<size_t>(row_hi - row_lo), stream);
    }
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (csplit && packed_s4) {  // attr_set bits 128..
    if constexpr (KIND == ptx::KIND_I8) {
      const int cb = 128 + EPI * 2;
      if (cfg.bn == 64)
        return launch_variant<KIND, 64, 4, 1, 1, EPI, 2, 2>(s, cb + 1, ta, tb, tc, p, stream);
      if (EPI != EPI_OUT16 || swap) {
        if (cfg.splits == 4)
          return launch_variant<KIND, 32, 4, 1, 1, EPI, 3, 4>(s, 136 + EPI, ta, tb, tc, p, stream);
        return launch_variant<KIND, 32, 4, 1, 1, EPI, 4, 2>(s, cb, ta, tb, tc, p, stream);
      }
    }
    return GEMM_ERR_INVALID_ARG;
  }
  if (csplit) {  // attr_set bits 96..: kind, output mode, width
    const int cb = csplit_variant_base<KIND, EPI>();
    if (cfg.bn == 64)
      return launch_variant<KIND, 64, 3, 1, 2, EPI, 0, 2>(s, cb + 1, ta, tb, tc, p, stream);
    if (EPI != EPI_OUT16 || swap) {
      if (cfg.splits == 4)
        return launch_variant<KIND, 32, 3, 1, 2, EPI, 0, 4>(s, cb + 8, ta, tb, tc, p, stream);
      return launch_variant<KIND, 32, 4, 1, 2, EPI, 0, 2>(s, cb, ta, tb, tc, p, stream);
    }
    return GEMM_ERR_INVALID_ARG;
  }
  const int vbase = ((KIND == ptx::KIND_F16) ? 0 : 32) + EPI * 8;  // bit index in attr_set
  if (packed_s4) {
    // fused INT4 variants: (int8 slots, packed slots) sized to fill shared memory; attr_set
    // bits 64.. (one per tile shape and output mode)
    if constexpr (KIND == ptx::KIND_I8) {
      const int fb = 64 + EPI * 8;
      if (hybrid) {  // (int8 slots, packed B slots) = (4, 4): two groups of expansion warps
        if (cfg.bn == 128) {
          using L = SmemLayout<128, 4, 2, 1, 4, 1, true>;
          return launch_kernel(s, gemm_kernel<KIND, 128, 4, 2, 1, EPI, 4, 1, false, false, true>, fb + 7,
                               L::DYN_BYTES, NUM_THREADS_FUSED_A8, 2, ta, tb, tc, p, stream);
        }
        using L = SmemLayout<256, 4, 2, 1, 4, 1, true>;
        return launch_kernel(s, gemm_kernel<KIND, 256, 4, 2, 1, EPI, 4, 1, false, false, true>, fb + 6,
                             L::DYN_BYTES, NUM_THREADS_FUSED_A8, 2, ta, tb, tc, p, stream);
      }
      if (cfg.cta_group == 2) {
        if (cfg.bn == 128)
          return launch_variant<KIND, 128, 4, 2, 1, EPI, 3>(s, fb + 5, ta, tb, tc, p, stream);
        return launch_variant<KIND, 256, 4, 2, 1, EPI, 2>(s, fb + 0, ta, tb, tc, p, stream);
      }
      switch (cfg.bn) {
        case 256: return launch_variant<KIND, 256, 2, 1, 1, EPI, 2>(s, fb + 1, ta, tb, tc, p, stream);
        case 128: return launch_variant<KIND, 128, 4, 1, 1, EPI, 2>(s, fb + 2, ta, tb, tc, p, stream);
        case 64: return launch_variant<KIND, 64, 4, 1, 1, EPI, 4>(s, fb + 3, ta, tb, tc, p, stream);
        case 32:
          if (EPI != EPI_OUT16 || swap)
            return launch_variant<KIND, 32, 4, 1, 1, EPI, 5>(s, fb + 4, ta, tb, tc, p, stream);
          return GEMM_ERR_INVALID_ARG;
        default: return GEMM_ERR_INVALID_ARG;
      }
    }
    return GEMM_ERR_INVALID_ARG;
  }
  if (cfg.cta_group == 2) {
    switch (cfg.bn) {
      case 256:
        if constexpr (KIND == ptx::KIND_I8) {
          if (ahead) {  // attr_set bits 224..
            t_last_s4_overlapped = 1;
            using L = SmemLayout<256, 6, 2, 1, 0, 1>;
            return launch_kernel(s, gemm_kernel<KIND, 256, 6, 2, 1, EPI, 0, 1, false, true>, 224 + EPI,
                                 L::DYN_BYTES, NUM_THREADS_AHEAD, 2, ta, tb, tc, p, stream);
          }
        }
        if constexpr (EPI == EPI_RAW32) {
          // ring depth as an ablation variable (gemm_set_stages_override); attr_set bits 216..
          const int sb = 216 + (KIND == ptx::KIND_F16 ? 0 : 4);
          if (cfg.stages == 3) return launch_variant<KIND, 256, 3, 2, 1, EPI>(s, sb + 0, ta, tb, tc, p, stream);
          if (cfg.stages == 4) return launch_variant<KIND, 256, 4, 2, 1, EPI>(s, sb + 1, ta, tb, tc, p, stream);
          if (cfg.stages == 5) return launch_variant<KIND, 256, 5, 2, 1, EPI>(s, sb + 2, ta, tb, tc, p, stream);
        }
        return launch_variant<KIND, 256, 6, 2, 1, EPI>(s, vbase + 4, ta, tb, tc, p, stream);
      case 128: return launch_variant<KIND, 128, 4, 2, 2, EPI>(s, vbase + 5, ta, tb, tc, p, stream);
      case 64: return launch_variant<KIND, 64, 4, 2, 2, EPI>(s, vbase + 6, ta, tb, tc, p, stream);
      default: return GEMM_ERR_INVALID_ARG;
    }
  }
  switch (cfg.bn) {
    case 256: return launch_variant<KIND, 256, 4, 1, 1, EPI>(s, vbase + 0, ta, tb, tc, p, stream);
    case 128: return launch_variant<KIND, 128, 3, 1, 2, EPI>(s, vbase + 1, ta, tb, tc, p, stream);
    case 64: return launch_variant<KIND, 64, 4, 1, 2, EPI>(s, vbase + 2, ta, tb, tc, p, stream);
    case 32:
      if (EPI != EPI_OUT16 || swap)
        return launch_variant<KIND, 32, 4, 1, 2, EPI>(s, vbase + 3, ta, tb, tc, p, stream);
      return GEMM_ERR_INVALID_ARG;
    default: return GEMM_ERR_INVALID_ARG;
  }
}

// Shape of a few-rows launch.  Two groups of 16 long rows per CTA (32-row blocks): the short
// operand's requests are then at most half the long operand's, and 9-16 short rows measured
// 10 %, up to 8 short rows 2-9 % faster than with 16-row blocks.
constexpr int FEW_ROWS_MT = 2;

// Problems with a few rows on one side go to few_rows_kernel (the long operand from
// global memory to MMA fragments without a pass through a shared tile, one launch, nothing
// zeroed).  Automatic for a short side of up to 16 rows (INT4: 32 against at most 8192) against
// 512 or more: INT4 always (it
// measured 0.45-0.98 of the tile kernels' time for 2048 <= N <= 28672, K = 4096 / 8192: there the
// tile kernels are bound by expanding the nibbles in shared memory); INT8 with up to 8 short
// rows always too (0.65-0.93 of the tile kernels' time, 0.94 of the HBM bandwidth at
// 1 x 28672 x 8192), with 9-16 while the long operand has at most 64 MB (0.8-0.9; level at
// 128 MB, 5-15 % slower at 96 and 235 MB, where the tile kernels' bulk copies reach 0.86-0.88 of
// the HBM bandwidth); FP16 while the long operand has at most 32 M elements (64 MB: 0.82-0.95
// of the tile kernels' time; level at 128 MB, 4-17 % slower beyond); INT8 and FP16 only with
// at least six 32-row blocks per KB of a row (16 x 1024 x 8192 FP16 has 32 blocks of 16 KB rows
// and ran 12.3 against 8.5 us: too few CTAs for rows that long).
// gemm_set_kernel_family(3) takes it wherever it exists (a short side of up to 32 rows),
// families 1 and 2, forced tile shapes, forced operand orders, every forced INT4 scheme and the
// traced runs never.
constexpr int FEW_ROWS_AUTO = 16;
constexpr int FEW_ROWS_MAX = 32;
bool few_rows_wanted(int M, int N, int K, bool packed_s4, const OutputSpec& out,
                     bool fp16 = false) {
  if (out.tiles_only || g_override_bn || g_override_cta_group || g_override_splits) return false;
  if ((g_trace_on & 1) || (g_l2_policy & 64)) return false;  // measurement runs mean the tile kernels
  if (g_swap_ab) return false;                                // so does a forced operand order
  if (packed_s4 && g_s4_scheme != 0) return false;
  const int fam = g_family;
  const int shorter = M < N ? M : N, longer = M < N ? N : M;
  if (fam == 3) return shorter <= FEW_ROWS_MAX;
  if (fam != 0 || longer < 512) return false;
  // INT4 with 17-32 rows (four groups of short rows per warp) against up to 8192: 3-33 % ahead of
  // the tile kernels (32 x 4096 x 4096 9.9 -> 6.7 us, 32 x 8192 x 8192 16.4 -> 16.0); behind from
  // 16384 rows on (32 x 28672 x 8192: 46.3 against 35.7 us)
  if (packed_s4 && shorter > FEW_ROWS_AUTO) return shorter <= FEW_ROWS_MAX && longer <= 8192;
  if (shorter > FEW_ROWS_AUTO) return false;
  if (packed_s4) return true;
  // A CTA's time grows with the length of a row (its 16 warps share it), the tile kernels
  // split K over as many CTAs as it takes: few row blocks against long rows stay on tiles.
  const long long row_bytes = fp16 ? 2LL * K : K;
  if (ceil_div(longer, 16 * FEW_ROWS_MT) < 6 * ceil_div(row_bytes, 1024)) return false;
  if (fp16) return static_cast<long long>(longer) * K <= (32LL << 20);
  return shorter <= 8 || static_cast<long long>(longer) * K <= (64LL << 20);
}

struct FewRowsShape {
  int mt, depth, warps, grid, smem;
};

constexpr int FEW_ROWS_SMEM_SM = 227 * 1024;  // shared memory of an SM; each CTA reserves 1 KB more
// What the CTAs of an SM take of it between them: the rest of the 256 KB stays L1, where the
// short operand, which every CTA reads again, finds room (with all 227 KB given to deeper rings
// up to 8 short rows ran 9.9 us instead of 9.2-9.4 at N = K = 8192, INT4; with 160 KB the
// problems whose blocks outnumber the resident CTAs lost 15-20 %).
constexpr int FEW_ROWS_SMEM_RING = 192 * 1024;

// Warps per CTA share K (64 bytes per step): eight, fewer for a short K (two steps each at
// least), sixteen while the SMs would have fewer than twelve warps each and K is long enough.
// CTAs per SM: as many as hold every row block at once if the ring can still be two steps deep;
// else fewer, with a ring of at least three steps, and a CTA walks the blocks c, c + grid, ...
// The ring takes what is left of the SM's allotment (FEW_ROWS_SMEM_RING, up to eight steps).
FewRowsShape few_rows_shape(int rows_l, int rows_s, int row_bytes, int num_sms) {
  const int nt = rows_s <= 8 ? 1 : rows_s <= 16 ? 2 : 4;
  FewRowsShape f;
  f.mt = FEW_ROWS_MT;
  const int steps = ceil_div(row_bytes, 64);
  const long long blocks = ceil_div(rows_l, 16 * f.mt);
  f.warps = 8;
  while (f.warps > 1 && steps < 2 * f.warps) f.warps /= 2;
  if (f.warps == 8 && blocks * 8 < 12LL * num_sms && steps >= 64) f.warps = 16;
  // (17-32 short rows: sixteen warps' sums and two ring slots do not fit the allotment)
  while (f.warps > 1 && few_rows_ring_bytes(f.mt, nt, 2, f.warps) + few_rows_red_bytes(f.mt, nt, f.warps) +
                                1024 > FEW_ROWS_SMEM_RING)
    f.warps /= 2;
  const int red = few_rows_red_bytes(f.mt, nt, f.warps);
  const int slot = few_rows_ring_bytes(f.mt, nt, 1, f.warps);
  int per_sm = static_cast<int>((blocks + num_sms - 1) / num_sms);
  if (per_sm * f.warps > 64) per_sm = 64 / f.warps;  // warp slots of an SM
  if (per_sm > 32) per_sm = 32;                      // and its CTA slots
  for (;; --per_sm) {
    f.depth = (FEW_ROWS_SMEM_RING / per_sm - 1024 - red) / slot;
    const bool all_at_once = blocks <= static_cast<long long>(per_sm) * num_sms;
    if (f.depth >= (all_at_once ? 2 : 3) || per_sm == 1) break;
  }
  if (f.depth > FEW_ROWS_MAX_DEPTH) f.depth = FEW_ROWS_MAX_DEPTH;
  if (f.depth < 2) f.depth = 2;  // (cannot happen after the loop above; the kernel needs two)
  f.smem = few_rows_ring_bytes(f.mt, nt, f.depth, f.warps) + red;
  const long long resident = static_cast<long long>(per_sm) * num_sms;
  f.grid = static_cast<int>(blocks < resident ? blocks : resident);
  return f;
}

template <int FKIND, int NT, int EPI>
int launch_few_rows_nt(DeviceState* s, FewRowsParams& p, const FewRowsShape& f,
                       cudaStream_t stream) {
  // attr_set bits 256..282: by operand kind, short-row groups, output mode
  constexpr int variant = 256 + (FKIND * 3 + (NT == 1 ? 0 : NT == 2 ? 1 : 2)) * 3 + EPI;
  auto kernel = few_rows_kernel<FKIND, FEW_ROWS_MT, NT, EPI>;
  if (!(s->attr_set[variant >> 6].load(std::memory_order_relaxed) & (1ull << (variant & 63)))) {
    const cudaError_t e = cudaFuncSetAttribute(
        kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FEW_ROWS_SMEM_SM);
    if (e != cudaSuccess) return cuda_fail(e);
    s->attr_set[variant >> 6].fetch_or(1ull << (variant & 63), std::memory_order_relaxed);
  }
  p.depth = f.depth;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(f.grid), 1, 1);
  cfg.blockDim = dim3(static_cast<unsigned>(f.warps * 32), 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(f.smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.wait_prior_grid ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, p);
  return e == cudaSuccess ? GEMM_OK : cuda_fail(e);
}

// A, B: int8, packed INT4 or FP16 rows, pitches in bytes.
template <int FKIND, int EPI>
int launch_few_rows(int M, int N, int K, const void* A, size_t a_pitch, const void* B,
                    size_t b_pitch, void* C, const OutputSpec& out, cudaStream_t stream) {
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  const long long ldc = out.ldc ? out.ldc : N;
  const bool a_short = M <= N;
  FewRowsParams p;
  p.L = static_cast<const uint8_t*>(a_short ? B : A);
  p.S = static_cast<const uint8_t*>(a_short ? A : B);
  p.l_pitch = static_cast<long long>(a_short ? b_pitch : a_pitch);
  p.s_pitch = static_cast<long long>(a_short ? a_pitch : b_pitch);
  p.rows_l = a_short ? N : M;
  p.rows_s = a_short ? M : N;
  p.row_bytes = FKIND == FEW_ROWS_S4 ? K / 2 : FKIND == FEW_ROWS_F16 ? 2 * K : K;
  p.C = C;
  p.c_stride_s = a_short ? ldc : 1;
  p.c_stride_l = a_short ? 1 : ldc;
  p.scale_s = a_short ? out.row_scale : out.col_scale;
  p.scale_l = a_short ? out.col_scale : out.row_scale;
  p.scale_s_first = a_short ? 1 : 0;
  p.wait_prior_grid = (g_l2_policy & 32) ? 0 : 1;
  const FewRowsShape f = few_rows_shape(p.rows_l, p.rows_s, p.row_bytes, s->num_sms);
  switch (ceil_div(p.rows_s, 8)) {
    case 1: return launch_few_rows_nt<FKIND, 1, EPI>(s, p, f, stream);
    case 2: return launch_few_rows_nt<FKIND, 2, EPI>(s, p, f, stream);
    case 3:
    case 4: return launch_few_rows_nt<FKIND, 4, EPI>(s, p, f, stream);
    default: return GEMM_ERR_INVALID_ARG;
  }
}

template <int KIND>
int launch_gemm(int M, int N, int K, const void* A, size_t a_pitch, const void* B, size_t b_pitch,
                void* C, cudaStream_t stream, const OutputSpec& out = OutputSpec(),
                bool packed_s4 = false, const S4AheadReq* req = nullptr,
                const S4HybridReq* hyb = nullptr) {
  if constexpr (KIND == ptx::KIND_I8) {
    if (!req && !hyb && few_rows_wanted(M, N, K, packed_s4, out)) {
      switch (out.epi) {
        case EPI_RAW32:
          return packed_s4 ? launch_few_rows<FEW_ROWS_S4, EPI_RAW32>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream)
                           : launch_few_rows<FEW_ROWS_S8, EPI_RAW32>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
        case EPI_OUT16:
          return packed_s4 ? launch_few_rows<FEW_ROWS_S4, EPI_OUT16>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream)
                           : launch_few_rows<FEW_ROWS_S8, EPI_OUT16>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
        case EPI_F32_SCALED:
          return packed_s4 ? launch_few_rows<FEW_ROWS_S4, EPI_F32_SCALED>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream)
                           : launch_few_rows<FEW_ROWS_S8, EPI_F32_SCALED>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
        default: return GEMM_ERR_INVALID_ARG;
      }
    }
  } else {
    if (!req && !hyb && !packed_s4 && few_rows_wanted(M, N, K, false, out, true)) {
      if (out.epi == EPI_RAW32)
        return launch_few_rows<FEW_ROWS_F16, EPI_RAW32>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
      if (out.epi == EPI_OUT16)
        return launch_few_rows<FEW_ROWS_F16, EPI_OUT16>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream);
    }
  }
  switch (out.epi) {
    case EPI_RAW32:
      return launch_gemm_epi<KIND, EPI_RAW32>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream,
                                              packed_s4, req, hyb);
    case EPI_OUT16:
      return launch_gemm_epi<KIND, EPI_OUT16>(M, N, K, A, a_pitch, B, b_pitch, C, out, stream,
                                              packed_s4, req, hyb);
    case EPI_F32_SCALED:
      if constexpr (KIND == ptx::KIND_I8)
        return launch_gemm_epi<KIND, EPI_F32_SCALED>(M, N, K, A, a_pitch, B, b_pitch, C, out,
                                                     stream, packed_s4, req, hyb);
      return GEMM_ERR_INVALID_ARG;
    default: return GEMM_ERR_INVALID_ARG;
  }
}

int check_common(int M, int N, int K, const void* A, const void* B, const void* C) {
  if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !C) return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) |
       reinterpret_cast<uintptr_t>(C)) & 15)
    return GEMM_ERR_MISALIGNED;
  return GEMM_OK;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Unpacks one or two packed matrices (rows_b may be 0) with the same K and output pitch.
int launch_unpack(long long rows_a, const uint8_t* packed_a, int8_t* out_a, long long rows_b,
                  const uint8_t* packed_b, int8_t* out_b, int K, size_t out_pitch,
                  cudaStream_t stream) {
  UnpackJob a{reinterpret_cast<const uint4*>(packed_a), out_a, rows_a * (K / 32)};
  UnpackJob b{reinterpret_cast<const uint4*>(packed_b), out_b, rows_b * (K / 32)};
  DeviceState* s = nullptr;
  int rc = device_state(&s);
  if (rc != GEMM_OK) return rc;
  const long long chunks = a.chunks + b.chunks;
  long long blocks = (chunks + 255) / 256;
  if (blocks > static_cast<long long>(s->num_sms) * 32) blocks = static_cast<long long>(s->num_sms) * 32;
  if (blocks < 1) blocks = 1;
  // policy bit 32 and traced launches: plain stream order, as for the GEMMs
  const int chained = ((g_l2_policy & 32) || (g_trace_on & 1)) ? 0 : 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, unpack_s4_kernel, a, b, K / 32,
                                     static_cast<long long>(out_pitch), chained);
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

// The int8 image of one packed operand for the hybrid fused kernel (expand_s4_slots_kernel).
int launch_expand_slots(long long rows, const uint8_t* packed, int8_t* out, int K, size_t out_pitch,
                        int num_sms, cudaStream_t stream) {
  const long long chunks = rows * static_cast<long long>(out_pitch / 32);
  long long blocks = (chunks + 255) / 256;
  if (blocks > static_cast<long long>(num_sms) * 32) blocks = static_cast<long long>(num_sms) * 32;
  if (blocks < 1) blocks = 1;
  const int chained = ((g_l2_policy & 32) || (g_trace_on & 1)) ? 0 : 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, expand_s4_slots_kernel, packed, out, rows, K / 2,
                                     static_cast<long long>(out_pitch), chained);
  if (e != cudaSuccess) return cuda_fail(e);
  return GEMM_OK;
}

int check_s4(int M, int N, int K, const void* A, const void* B, const void* C) {
  int rc = check_common(M, N, K, A, B, C);
  if (rc != GEMM_OK) return rc;
  if (K % 32) return GEMM_ERR_MISALIGNED;
  if (K > K_LIMIT_INT) return GEMM_ERR_K_TOO_LARGE;
  return GEMM_OK;
}

size_t s4_workspace_need(int M, int N, int K) {
  return align_up(static_cast<size_t>(M) * K, 256) + align_up(static_cast<size_t>(N) * K, 256);
}

// INT4 GEMM through caller-visible scratch: unpack A and B to int8, then the INT8 kernel.
// `sync`: bookkeeping words of the overlapped pre-pass in front of a pool buffer, or null
// (caller-supplied scratch, whose surroundings the library knows nothing about).
int s4_with_workspace(int M, int N, int K, const uint8_t* A, const uint8_t* B, void* C,
                      void* workspace, size_t workspace_bytes, const OutputSpec& out_in,
                      cudaStream_t st, uint32_t* sync = nullptr) {
  if (!workspace) return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < s4_workspace_need(M, N, K))
    return GEMM_ERR_WORKSPACE;
  int8_t* a8 = static_cast<int8_t*>(workspace);
  int8_t* b8 = a8 + align_up(static_cast<size_t>(M) * K, 256);
  OutputSpec out = out_in;
  out.tiles_only = true;
  int rc;
  if (sync) {
    const S4AheadReq req{A, B, sync};
    rc = launch_gemm<ptx::KIND_I8>(M, N, K, a8, static_cast<size_t>(K), b8, static_cast<size_t>(K),
                                   C, st, out, false, &req);
    if (rc != GEMM_NOT_AHEAD) return rc;
  }
  rc = launch_unpack(M, A, a8, N, B, b8, K, static_cast<size_t>(K), st);
  if (rc != GEMM_OK) return rc;
  return launch_gemm<ptx::KIND_I8>(M, N, K, a8, static_cast<size_t>(K), b8, static_cast<size_t>(K),
                                   C, st, out);
}

// Zero-initialised bookkeeping bytes in front of a pool buffer of `need` data bytes (ready
// flags of the overlapped pre-pass: one word per 32 rows x 512 columns of int8, both operands).
size_t s4_head_bytes(int M, int N, int K) {
  const size_t flags = (static_cast<size_t>(ceil_div(M, 32)) + ceil_div(N, 32)) * ceil_div(K, 512);
  return align_up(4 * (S4A_SYNC_WORDS + flags), 256);
}

// INT4 GEMM by the route gemm_set_s4_scheme selected: the fused kernel if asked for and
// applicable, else the pre-pass through a scratch buffer leased from the device's pool for
// this stream (allocated stream-ordered on first use or growth: no device-wide
// synchronisation, and calls on different streams never share a buffer).
int s4_auto(int M, int N, int K, const uint8_t* A, const uint8_t* B, void* C, const OutputSpec& out,
            cudaStream_t st) {
  t_last_s4_overlapped = 0;
  DeviceState* s = nullptr;
  int dev = 0;
  int rc = device_state(&s, &dev);
  if (rc != GEMM_OK) return rc;
  if (!s4_prepass_forced()) {
    rc = launch_gemm<ptx::KIND_I8>(M, N, K, A, static_cast<size_t>(K) / 2, B,
                                   static_cast<size_t>(K) / 2, C, st, out, true);
    if (rc == GEMM_WANT_A8) {
      // hybrid: the int8 image of A (M rows of K rounded up to 256) in leased scratch, then the
      // fused kernel on it and the packed B
      const size_t pitch = align_up(static_cast<size_t>(K), 256);
      ScratchPool::Lease lease;
      const int prc = g_pool[dev].acquire(st, align_up(static_cast<size_t>(M) * pitch, 256),
                                          s4_head_bytes(M, N, K), &lease);
      if (prc == ScratchPool::kNoAllocInCapture) {
        // a stream being captured with no buffer from an earlier call: the form that needs none
        const S4HybridReq none{nullptr, 0};
        return launch_gemm<ptx::KIND_I8>(M, N, K, A, static_cast<size_t>(K) / 2, B,
                                         static_cast<size_t>(K) / 2, C, st, out, true, nullptr, &none);
      }
      if (prc != 0) return pool_fail(prc);
      int8_t* a8 = reinterpret_cast<int8_t*>(static_cast<uint8_t*>(lease.ptr) + lease.head_bytes);
      rc = launch_expand_slots(M, A, a8, K, pitch, s->num_sms, st);
      if (rc == GEMM_OK) {
        const S4HybridReq hyb{a8, pitch};
        rc = launch_gemm<ptx::KIND_I8>(M, N, K, A, static_cast<size_t>(K) / 2, B,
                                       static_cast<size_t>(K) / 2, C, st, out, true, nullptr, &hyb);
      }
      const int qrc = g_pool[dev].release(lease, st);
      if (rc == GEMM_OK && qrc != 0) rc = pool_fail(qrc);
      return rc;
    }
    if (rc != GEMM_NOT_FUSED) return rc;
  }
  ScratchPool::Lease lease;
  const int prc = g_pool[dev].acquire(st, s4_workspace_need(M, N, K), s4_head_bytes(M, N, K), &lease);
  if (prc != 0) return pool_fail(prc);
  rc = s4_with_workspace(M, N, K, A, B, C, static_cast<uint8_t*>(lease.ptr) + lease.head_bytes,
                         lease.bytes, out, st, static_cast<uint32_t*>(lease.ptr));
  const int qrc = g_pool[dev].release(lease, st);
  if (rc == GEMM_OK && qrc != 0) rc = pool_fail(qrc);
  return rc;
}

int check_scales(const float* row_scale, const float* col_scale, const void* C, int c_is_fp16,
                 OutputSpec* out) {
  if (!row_scale || !col_scale || !C || (c_is_fp16 != 0 && c_is_fp16 != 1))
    return GEMM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(row_scale) | reinterpret_cast<uintptr_t>(col_scale)) & 3)
    return GEMM_ERR_MISALIGNED;
  out->epi = c_is_fp16 ? EPI_OUT16 : EPI_F32_SCALED;
  out->row_scale = row_scale;
  out->col_scale = col_scale;
  return GEMM_OK;
}
}  // namespace
}  // namespace b200gemm
