// Tile-shape, raster and split-K selection.
#pragma once

#include "runtime.cuh"

namespace b200gemm {
namespace {

// ------------------------------------------------------------------ selector
struct TileConfig {
  int bn;
  int cta_group;  // 1: one CTA per 128 x bn tile; 2: a CTA pair per 256 x bn tile
  int stages;
  int group_m;
  int splits;     // split-K factor (1 = off)
  int split_tiles;  // how many tiles, counted from the end of the raster, are split
                    // (all of them, or only the last partly filled wave)
};

constexpr int kWidths[] = {256, 128, 64, 32};

// Ring depth and 128-byte K atoms per slot of each built shape.
int stages_for(int bn, int cta_group) {
  if (cta_group == 2 && bn == 256) {
    const int o = g_override_stages;
    return (o >= 3 && o <= 6) ? o : 6;
  }
  if (cta_group == 2) return 4;
  switch (bn) {
    case 256: return 4;
    case 128: return 3;
    default: return 4;
  }
}

// 256-wide tiles are bound by the tensor pipe and want many small slots; narrower tiles are
// bound by the issuing thread and get two K atoms per slot (one wait + one commit per 8 MMAs).
int atoms_for(int bn, int) { return bn == 256 ? 1 : 2; }

bool variant_exists(int bn, int cta_group) {
  if (cta_group == 1) return bn == 256 || bn == 128 || bn == 64 || bn == 32;
  if (cta_group == 2) return bn == 256 || bn == 128 || bn == 64;
  return false;
}

// Kernel variants that take packed INT4 operands and expand them on the way to the MMAs.
bool fused_s4_variant_exists(int bn, int cta_group, int splits) {
  if (cta_group == 2) return bn == 256 || bn == 128;
  return bn == 256 || bn == 128 || bn == 64 || bn == 32;
}

int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

// Picks the C-tile shape and the split-K factor.  The paper fixes one tiling for all
// sizes (Sec. III-A) and lists non-square shapes as future work (Sec. VI); on 148 SMs small
// problems need more work units than they have tiles, and large ones want the CTA-pair
// tile, which halves the B bytes each SM pulls from L2.
// Cost model, in SM cycles, fitted to the cycle accounting of the kernel: a k-block (128
// bytes of K) costs the slowest of the tensor pipe (2*bn: a 128-row MMA of width bn occupies
// it bn/2 cycles, 4 per k-block), the issuing thread (~450) and the SM's L2 port
// ((128 + bn/cta_group) rows x 128 bytes at ~66 bytes/cycle); units run in waves over the SMs
// (or SM pairs); the last epilogue (~16 cycles per column), set-up (~3000) and a pair's
// cluster launch (~2500) are paid once; split-K adds zeroing C and adding into it.
// force_atoms: K atoms per split unit whatever the tile (the fused INT4 kernel splits K in
// packed slots = 2 int8 k-blocks); 0 = the tile's own ring slot.
// split_cap: upper limit of the split-K factor (0 = none).
// fused_only: 1 = only shapes the fused INT4 kernel is built for, 2 = only its 256-wide
// CTA-pair shape.
TileConfig select_config(int M, int N, int num_sms, int k_blocks, int min_bn = 32,
                         bool allow_split = false, int force_atoms = 0, int split_cap = 0,
                         int fused_only = 0) {
  TileConfig best{256, 2, 6, 8, 1, 0};
  long long best_cost = -1;
  // the ablation overrides, read once
  const int o_bn = g_override_bn, o_cta_group = g_override_cta_group;
  const int o_splits = g_override_splits, o_group_m = g_override_group_m;
  for (int cg = 2; cg >= 1; --cg) {
    if (o_cta_group && cg != o_cta_group) continue;
    if (fused_only == 2 && cg != 2) continue;
    for (int bn : kWidths) {
      if (o_bn && bn != o_bn) continue;
      if (!variant_exists(bn, cg) || bn < min_bn) continue;
      if (fused_only == 2 && bn != 256) continue;
      const long long tiles = static_cast<long long>(ceil_div(M, BM * cg)) * ceil_div(N, bn);
      const long long units = num_sms / cg;
      const int atoms = force_atoms ? force_atoms : atoms_for(bn, cg);
      const int slots = ceil_div(k_blocks, atoms);  // K is split in whole ring slots
      int max_split = 1;
      if (allow_split) {
        max_split = static_cast<int>(units / tiles);
        if (max_split > k_blocks / 2) max_split = k_blocks / 2;  // at least 2 k-blocks each
        if (max_split > 32) max_split = 32;
        if (split_cap && max_split > split_cap) max_split = split_cap;
        if (max_split < 1) max_split = 1;
      }
      if (o_splits) {
        // forced: the largest factor <= the request that leaves no K range empty
        max_split = o_splits < slots ? o_splits : slots;
        while (max_split > 1 &&
               static_cast<long long>(max_split - 1) * ceil_div(slots, max_split) >= slots)
          --max_split;
        if (!allow_split) max_split = 1;
      }
      if (max_split > slots) max_split = slots;
      for (int sp = o_splits ? max_split : 1; sp <= max_split; ++sp) {
        if (static_cast<long long>(sp - 1) * ceil_div(slots, sp) >= slots) continue;  // empty range
        if (fused_only && !fused_s4_variant_exists(bn, cg, sp)) continue;
        const int per = ceil_div(slots, sp) * atoms;  // k-blocks per unit
        const long long waves = (tiles * sp + units - 1) / units;
        long long per_kb = 2 * bn;
        if (per_kb < 450) per_kb = 450;
        const long long port = (128 + bn / cg) * 128 / 66;
        if (per_kb < port) per_kb = port;
        // measured: with a short K (up to 48 k-blocks) the 256 x 128 pair tile runs ahead of
        // the port figure (2304^3 FP16: 24.4 us against 27.6 on the 256-wide tile, INT8 15.1 / 16.3;
        // not so the fused INT4 kernel: 256 x 12288 x 1536 14.0 against 12.4 us)
        if (cg == 2 && bn == 128 && k_blocks <= 48 && force_atoms == 0) per_kb = 320;
        long long cost = waves * per * per_kb + 3000 + 16 * bn + (cg == 2 ? 2500 : 0);
        if (sp > 1) cost += 6000 + static_cast<long long>(M) * N / 250;  // zeroing C + adding into it
        if (best_cost < 0 || cost < best_cost) {
          best_cost = cost;
          best.bn = bn;
          best.cta_group = cg;
          best.splits = sp;
        }
      }
    }
  }
  if (best_cost < 0) {  // the override names a shape this output mode does not have
    best.bn = 0;
    return best;
  }
  {
    // Split-K of every tile, or -- when the tiles fill at least one wave and the last wave
    // is at most half full -- of the last wave only: its r tiles become r * s units over
    // disjoint K ranges, so the tail costs 1/s of a tile time instead of a whole one.
    const long long tiles =
        static_cast<long long>(ceil_div(M, BM * best.cta_group)) * ceil_div(N, best.bn);
    const long long units = num_sms / best.cta_group;
    const int slots =
        ceil_div(k_blocks, force_atoms ? force_atoms : atoms_for(best.bn, best.cta_group));
    best.split_tiles = best.splits > 1 ? static_cast<int>(tiles) : 0;
    const long long r = tiles % units;
    const int atoms = force_atoms ? force_atoms : atoms_for(best.bn, best.cta_group);
    if (allow_split && best.splits == 1 && o_splits == 0 && tiles > units && r > 0 &&
        2 * r <= units && slots * atoms >= (units / r >= 5 ? 32 : 64)) {  // measured: a fuller last
      // wave pays off (+2-3 %) only for long K
      int sp = static_cast<int>(units / r);
      // A last wave of a few tiles only (224 tiles on 74 pairs leave 2) would cost a whole tile
      // time: there the split goes as deep as the idle units allow, down to 8 k-blocks per
      // unit.  Fuller last waves keep the measured rule: up to 4 ways, 32 k-blocks each.
      const bool few = sp >= 5;
      const int cap = few ? 16 : 4, min_kb = few ? 8 : 32;
      if (sp > cap) sp = cap;
      while (sp > 1 && (slots * atoms / sp < min_kb ||
                        static_cast<long long>(sp - 1) * ceil_div(slots, sp) >= slots))
        --sp;
      if (sp > 1) {
        best.splits = sp;
        best.split_tiles = static_cast<int>(r);
      }
    }
  }
  best.stages = stages_for(best.bn, best.cta_group);
  // Band height: one wave of tiles about twice as tall as wide in operand bytes (measured
  // DRAM traffic at N = 8192 is lowest there: the A band is what later waves re-read).
  int rows_per_tile = BM * best.cta_group;
  int units = num_sms / best.cta_group;
  int g = 1;
  while ((g + 1) * (g + 1) * rows_per_tile <= 2 * units * best.bn) ++g;
  if (o_group_m) g = o_group_m;
  int tiles_m = ceil_div(M, rows_per_tile);
  if (g > tiles_m) g = tiles_m;
  if (g < 1) g = 1;
  best.group_m = g;
  return best;
}
}  // namespace
}  // namespace b200gemm
