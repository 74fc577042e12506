// Static schedule of the attention kernel: which query tiles a CTA works on, and in what order.
// Plain C++ (no CUDA types), so that the host can enumerate it too.
//
// A work item occupies both "lanes" of a CTA (a lane holds one 128-row query tile with its S, P and O in tensor
// memory).  The query tiles of all heads form one list (head-major); with G CTAs and U tiles, the first
// P = G floor(U / 2G) items are PAIRS of neighbouring tiles (tiles 2v and 2v+1): the same head, sharing every K/V
// tile, or, where the pair straddles a head boundary, two heads whose lanes stream their own K/V.  The remaining
// U - 2P tiles are SINGLES, whose keys are split between the two lanes (even and odd key tiles; the two partial
// results are merged when the item ends), so that a single costs about half a pair.
//
// Pairs are dealt in rounds of G: every CTA gets the same number of pairs, and CTAs that run at the same time work
// on neighbouring tiles of few heads, whose K/V tiles reach DRAM once and are shared through L2.  From round to
// round the dealing is rotated by one CTA.  A pair that straddles two heads takes about 6% longer (two K/V streams),
// and such pairs recur every t pairs for t (odd) tiles per head: with t = 37 and G = 148 = 4 x 37 an unrotated
// deal put all 20 of them on the same four CTAs, which finished 6% after all the others; rotated, no CTA holds more
// than one.  The singles are dealt round-robin after the pairs and even out the last round.
#pragma once

#if defined(__CUDACC__)
#define SDVG_HD __host__ __device__
#else
#define SDVG_HD
#endif

struct WsItem {
  int head[2], tile[2];   // per lane
  int lanes;              // 1 or 2
  bool dual;              // lanes stream their own K/V tiles (different heads, or one tile split by keys)
  bool split;             // both lanes work on ONE query tile: lane i takes key tiles i, i + 2, i + 4, ...
  int nk[2];              // key tiles per lane
  // branch-free on purpose: a loop-invariant branch on `split` makes the compiler clone whole role loops
  SDVG_HD int key_tile(int lane, int t) const { return (t << (int)split) + (lane & -(int)split); }
};

struct WsSchedule {
  int tiles, ctas, rounds, num_pairs, num_singles;

  SDVG_HD WsSchedule(int tokens, int heads, int ctas_, int tile_rows) : ctas(ctas_) {
    tiles = (tokens + tile_rows - 1) / tile_rows;
    const int total = tiles * heads;
    rounds = total / (2 * ctas);          // full rounds of pairs
    num_pairs = rounds * ctas;
    num_singles = total - 2 * num_pairs;
  }

  // The n-th item of CTA b; false when the CTA has no n-th item.  ntiles_k: key tiles of the launch.
  SDVG_HD bool get(int b, int n, int ntiles_k, WsItem& it) const {
    if (n < rounds) {
      int c = b - n % ctas;               // round n is dealt n CTAs further on
      if (c < 0) c += ctas;
      const int g0 = 2 * (n * ctas + c);
      it.head[0] = g0 / tiles;
      it.tile[0] = g0 - it.head[0] * tiles;
      it.head[1] = (g0 + 1) / tiles;
      it.tile[1] = g0 + 1 - it.head[1] * tiles;
      it.lanes = 2;
      it.dual = it.head[1] != it.head[0];
      it.split = false;
      it.nk[0] = it.nk[1] = ntiles_k;
      return true;
    }
    const int i = b + (n - rounds) * ctas;
    if (i >= num_singles) return false;
    const int g0 = 2 * num_pairs + i;
    it.head[0] = it.head[1] = g0 / tiles;
    it.tile[0] = it.tile[1] = g0 - it.head[0] * tiles;
    it.split = ntiles_k >= 2;
    it.lanes = it.split ? 2 : 1;
    it.dual = true;
    it.nk[0] = it.split ? (ntiles_k + 1) / 2 : ntiles_k;
    it.nk[1] = it.split ? ntiles_k / 2 : 0;
    return true;
  }
};
