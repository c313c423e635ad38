// CPU check of the overlapped INT4 pre-pass work list: a bijection onto the chunks, flags
// distinct, the first wave's rows first and k-chunk-major.  Prints "ok" or the first failure.
#include <stdio.h>

#include <set>
#include <vector>

#include "../../paper_2608_10103_b200/csrc/s4_ahead.h"

using namespace b200gemm;

#define EXPECT(cond)                                             \
  do {                                                           \
    if (!(cond)) {                                               \
      printf("FAILED line %d: %s (plan %d %d %d %d %d)\n", __LINE__, #cond, p.ra, p.rb, p.kc, p.ra1, p.rb1); \
      return 1;                                                  \
    }                                                            \
  } while (0)

int check(const S4AheadPlan& p) {
  const int total = s4a_total(p);
  std::set<int> flags;
  std::vector<int> pos(total, -1);
  for (int i = 0; i < total; ++i) {
    int op = -1, r = -1, k = -1;
    s4a_decode(p, i, &op, &r, &k);
    EXPECT(op == 0 || op == 1);
    EXPECT(r >= 0 && r < (op ? p.rb : p.ra));
    EXPECT(k >= 0 && k < p.kc);
    const int f = s4a_flag_index(p, op, r, k);
    EXPECT(f >= 0 && f < total);
    EXPECT(flags.insert(f).second);  // no chunk twice
    pos[f] = i;
    if (i < (p.ra1 + p.rb1) * p.kc) {  // first wave: its rows only, k-chunk-major
      EXPECT(r < (op ? p.rb1 : p.ra1));
      EXPECT(k == i / (p.ra1 + p.rb1));
    }
  }
  EXPECT(static_cast<int>(flags.size()) == total);
  // inside a group of the later phases a smaller k-chunk never comes after a larger one
  for (int r = p.rb1; r < p.rb; ++r)
    for (int k = 1; k < p.kc; ++k)
      EXPECT(pos[s4a_flag_index(p, 1, r, k - 1)] < pos[s4a_flag_index(p, 1, r, k)]);
  // B's remaining tile columns come in raster order
  for (int r = p.rb1 + p.gb; r < p.rb; ++r)
    EXPECT(pos[s4a_flag_index(p, 1, r - p.gb, p.kc - 1)] < pos[s4a_flag_index(p, 1, r, 0)]);
  return 0;
}

int main() {
  const int shapes[][5] = {  // ra, rb, kc, ra1, rb1
      {256, 256, 16, 96, 56}, {256, 256, 16, 256, 256}, {1, 1, 1, 1, 1}, {33, 70, 3, 16, 8},
      {157, 126, 9, 112, 48}, {16, 8, 1, 16, 8}, {625, 641, 2, 80, 120}, {40, 40, 5, 0, 0}};
  for (const auto& s : shapes) {
    S4AheadPlan p{s[0], s[1], s[2], s[3], s[4], 16, 8};
    if (check(p)) return 1;
  }
  printf("ok\n");
  return 0;
}
