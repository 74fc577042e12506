// Host-side check of the attention kernel's static schedule (csrc/attn_schedule.h): over a sweep of shapes every
// query tile is handed out exactly once and the items are well formed; at the model shapes the load of the CTAs is
// even and no CTA holds more than one pair that straddles two heads.  Prints "ok ..." and exits 0, or names the
// first violation and exits 1.
#include <algorithm>
#include <cstdio>
#include <utility>
#include <vector>

#include "attn_schedule.h"

int main() {
  long checked = 0;
  for (int ctas : {1, 2, 3, 7, 9, 18, 37, 74, 132, 148, 160})
    for (int heads = 1; heads <= 164; heads += (heads < 48 ? 1 : 29))
      for (int tiles = 1; tiles <= 80; ++tiles) {
        const int tokens = tiles * 128 - 17, total = tiles * heads;
        const int g = total < ctas ? total : ctas;           // the launch's grid rule
        const WsSchedule s(tokens, heads, g, 128);
        std::vector<int> seen(total, 0);
        double lo = 1e9, hi = 0;
        for (int b = 0; b < g; ++b) {
          WsItem it;
          double load = 0;
          for (int n = 0; s.get(b, n, 10, it); ++n) {
            if (n > total) return std::printf("runaway loop: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            const bool pair = it.lanes == 2 && !it.split;
            for (int l = 0; l < 2; ++l)
              if (it.head[l] < 0 || it.head[l] >= heads || it.tile[l] < 0 || it.tile[l] >= tiles)
                return std::printf("out of range: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            const int g0 = it.head[0] * tiles + it.tile[0], g1 = it.head[1] * tiles + it.tile[1];
            if (pair && (g1 != g0 + 1 || it.dual != (it.head[0] != it.head[1]) || it.nk[0] != 10 || it.nk[1] != 10))
              return std::printf("bad pair: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            if (!pair && (g1 != g0 || !it.dual || it.nk[0] + it.nk[1] != 10))
              return std::printf("bad single: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            ++seen[g0];
            if (pair) ++seen[g1];
            load += pair ? 1.0 : 0.5;
          }
          lo = std::min(lo, load), hi = std::max(hi, load);
        }
        for (int x : seen)
          if (x != 1) return std::printf("tile handed out %d times: ctas %d heads %d tiles %d\n", x, g, heads, tiles), 1;
        if (hi - lo > 0.5) return std::printf("uneven: %.1f .. %.1f: ctas %d heads %d tiles %d\n", lo, hi, g, heads, tiles), 1;
        ++checked;
      }
  // the model shapes on 148 CTAs (4680 tokens = 37 tiles): target, drafter, and their guidance pairs
  for (auto sh : {std::pair<int, double>{40, 5.0}, {12, 1.5}, {80, 10.0}, {24, 3.0}}) {
    const WsSchedule s(4680, sh.first, 148, 128);
    for (int b = 0; b < 148; ++b) {
      double load = 0;
      int straddling = 0;
      WsItem it;
      for (int n = 0; s.get(b, n, 256, it); ++n) {
        load += it.split ? 0.5 : 1.0;
        straddling += !it.split && it.dual;
      }
      if (load != sh.second) return std::printf("uneven load %.1f on CTA %d with %d heads\n", load, b, sh.first), 1;
      if (straddling > 1 + (sh.first > 40)) return std::printf("%d straddling pairs on CTA %d with %d heads\n", straddling, b, sh.first), 1;
    }
  }
  std::printf("ok %ld shapes\n", checked);
  return 0;
}
