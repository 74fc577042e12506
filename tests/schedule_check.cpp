// Host-side check of the attention kernel's static schedule (csrc/attn_schedule.h): over a sweep of shapes every
// query tile is handed out exactly once, pairs never straddle two heads, and the load of the CTAs is even at
// the two model shapes.  Prints "ok ..." and exits 0, or names the first violation and exits 1.
#include <algorithm>
#include <cstdio>
#include <utility>
#include <vector>

#include "attn_schedule.h"

static double load_of(const WsItem& it) { return it.lanes == 2 && !it.split ? 1.0 : 0.5; }

int main() {
  long checked = 0;
  for (int ctas : {1, 2, 3, 7, 9, 18, 37, 74, 132, 148, 160})
    for (int heads = 1; heads <= 164; heads += (heads < 48 ? 1 : 29))
      for (int tiles = 1; tiles <= 80; ++tiles) {
        const int tokens = tiles * 128 - 17, total = tiles * heads;
        const int g = total < ctas ? total : ctas;           // the launch's grid rule
        const WsSchedule s(tokens, heads, g, 128);
        std::vector<int> seen(total, 0);
        for (int b = 0; b < g; ++b) {
          WsItem it;
          for (int n = 0; s.get(b, n, 10, it); ++n) {
            if (n > total) return std::printf("runaway loop: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            const bool pair = it.lanes == 2 && !it.split;
            if (it.head[0] < 0 || it.head[0] >= heads || it.tile[0] < 0 || it.tile[0] >= tiles || it.head[1] != it.head[0])
              return std::printf("out of range or straddling: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            if (pair && (it.tile[1] != it.tile[0] + 1 || it.tile[1] >= tiles || it.dual))
              return std::printf("bad pair: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            if (!pair && (it.tile[1] != it.tile[0] || !it.dual || it.nk[0] + it.nk[1] != 10))
              return std::printf("bad single: ctas %d heads %d tiles %d\n", g, heads, tiles), 1;
            ++seen[it.head[0] * tiles + it.tile[0]];
            if (pair) ++seen[it.head[1] * tiles + it.tile[1]];
          }
        }
        for (int x : seen)
          if (x != 1) return std::printf("tile handed out %d times: ctas %d heads %d tiles %d\n", x, g, heads, tiles), 1;
        ++checked;
      }
  // the model shapes on 148 CTAs (4680 tokens = 37 tiles): target, drafter, and their guidance pairs
  for (auto sh : {std::pair<int, double>{40, 5.0}, {12, 1.5}, {80, 10.0}, {24, 3.0}}) {
    const WsSchedule s(4680, sh.first, 148, 128);
    for (int b = 0; b < 148; ++b) {
      double l = 0;
      WsItem it;
      for (int n = 0; s.get(b, n, 256, it); ++n) l += load_of(it);
      if (l != sh.second) return std::printf("uneven load %.1f on CTA %d with %d heads\n", l, b, sh.first), 1;
    }
  }
  std::printf("ok %ld shapes\n", checked);
  return 0;
}
