// Work list of the overlapped INT4 pre-pass: in which order the 32-row x 512-column chunks of
// the int8 images of A and B are produced while the GEMM that consumes them is already running
// in the same kernel.  Plain C++ (host and device), no CUDA types, so the order can be checked
// on a CPU: every chunk appears exactly once, and what the first wave of tiles needs comes
// first, k-chunk by k-chunk.
//
// The paper's INT4 kernels feed packed nibbles straight to mma.sync (Listing 2c); tcgen05 has
// no 4-bit integer kind, so the operands pass through an int8 image.  Producing that image
// inside the GEMM kernel, just ahead of the tiles that read it, takes the pre-pass off the
// critical path.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define S4A_HD __host__ __device__ __forceinline__
#else
#define S4A_HD inline
#endif

namespace b200gemm {

constexpr int S4A_CHUNK_ROWS = 32;
constexpr int S4A_CHUNK_COLS = 512;  // int8 columns (= 256 packed bytes per row)
constexpr int S4A_SYNC_WORDS = 64;   // words in front of the flags: epoch, counters

struct S4AheadPlan {
  int ra, rb;    // row chunks of A and of B: ceil(M / 32), ceil(N / 32)
  int kc;        // k-chunks: ceil(K / 512)
  int ra1, rb1;  // row chunks of A / B that the first wave of tiles reads (made first)
  int ga, gb;    // row chunks per tile row of A (16) / tile column of B (8)
};

S4A_HD int s4a_total(const S4AheadPlan& p) { return (p.ra + p.rb) * p.kc; }

// Flag word of a chunk (operand 0 = A, 1 = B).
S4A_HD int s4a_flag_index(const S4AheadPlan& p, int operand, int row_chunk, int k_chunk) {
  return (operand ? p.ra * p.kc : 0) + row_chunk * p.kc + k_chunk;
}

// Rows [first, first + count) of one operand, all k-chunks, in groups of `group` row chunks:
// group after group, inside a group k-chunk after k-chunk (a tile reads all rows of its group
// at one k before it moves on).
S4A_HD void s4a_decode_grouped(int j, int first, int count, int group, int kc, int* row_chunk,
                               int* k_chunk) {
  const int per_group = group * kc;
  const int g = j / per_group;
  const int rows_here = (count - g * group) < group ? (count - g * group) : group;
  const int within = j - g * per_group;
  *k_chunk = within / rows_here;
  *row_chunk = first + g * group + within % rows_here;
}

// i-th chunk of the work list, 0 <= i < s4a_total(p).
S4A_HD void s4a_decode(const S4AheadPlan& p, int i, int* operand, int* row_chunk, int* k_chunk) {
  const int first_rows = p.ra1 + p.rb1;
  const int n1 = first_rows * p.kc;
  if (i < n1) {  // what the first wave reads, one k-chunk of all its rows after the other
    *k_chunk = i / first_rows;
    const int r = i - *k_chunk * first_rows;
    *operand = r < p.ra1 ? 0 : 1;
    *row_chunk = r < p.ra1 ? r : r - p.ra1;
    return;
  }
  i -= n1;
  const int n2 = (p.rb - p.rb1) * p.kc;
  if (i < n2) {  // the rest of B, in the order the raster walks its tile columns
    *operand = 1;
    s4a_decode_grouped(i, p.rb1, p.rb - p.rb1, p.gb, p.kc, row_chunk, k_chunk);
    return;
  }
  i -= n2;  // the rest of A, band after band
  *operand = 0;
  s4a_decode_grouped(i, p.ra1, p.ra - p.ra1, p.ga, p.kc, row_chunk, k_chunk);
}

}  // namespace b200gemm
