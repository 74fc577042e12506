// Static schedule of the attention kernel: which query tiles a CTA works on, and in what order.
// Plain C++ (no CUDA types), so that the host can enumerate it too.
//
// A work item occupies both "lanes" of a CTA (a lane holds one 128-row query tile with its S, P and O in tensor
// memory).  It is either a PAIR of neighbouring query tiles of ONE head, which share every K/V tile, or a SINGLE
// tile whose keys are split between the lanes (even and odd key tiles; the two partial results are merged when
// the item ends), which costs about half a pair but streams K/V for each lane separately.  A pair never
// straddles two heads: its lanes would stream separate K/V like a single does, for a whole item, and with 37
// tiles per head and 148 = 4 x 37 CTAs every such pair landed on the same four CTAs, which then finished 6%
// after all the others.
//
// With G CTAs, H heads of t tiles each and U = H t tiles in all, the number of pairs is
//   P = min(G floor(U / 2G), H floor(t / 2)),
// taken from the heads in order: the first heads give floor(t / 2) pairs each (tiles [0, 2 floor(t / 2))), one head
// the rest, the heads after it none; what a head does not give as pairs it gives as singles.  Few heads are thus
// at work at any time, and the CTAs on one head stream the same K/V tiles at about the same time and share them
// through L2.  Pairs are numbered head by head and dealt round-robin (pair v to CTA v mod G).  Singles, numbered
// the same way, even out the rest: CTAs that got one pair less take two singles each first, what is left goes
// round-robin over all CTAs.
#pragma once

#if defined(__CUDACC__)
#define SDVG_HD __host__ __device__
#else
#define SDVG_HD
#endif

struct WsItem {
  int head[2], tile[2];   // per lane
  int lanes;              // 1 or 2
  bool dual;              // lanes stream their own K/V tiles (one tile split by keys)
  bool split;             // both lanes work on ONE query tile: lane i takes key tiles i, i + 2, i + 4, ...
  int nk[2];              // key tiles per lane
  // branch-free on purpose: a loop-invariant branch on `split` makes the compiler clone whole role loops
  SDVG_HD int key_tile(int lane, int t) const { return (t << (int)split) + (lane & -(int)split); }
};

struct WsSchedule {
  int tiles, heads, ctas;
  int pairs, singles;     // P and U - 2P
  int cap;                // pairs a head can give: floor(tiles / 2)
  int full, part;         // heads [0, full) give cap pairs, head `full` gives part (< cap), the others none
  int rem;                // CTAs [0, rem) hold one pair more than the others
  int first;              // singles dealt two at a time to the CTAs [rem, ctas) before the round-robin part

  SDVG_HD WsSchedule(int tokens, int heads_, int ctas_, int tile_rows) : heads(heads_), ctas(ctas_) {
    tiles = (tokens + tile_rows - 1) / tile_rows;
    const int total = tiles * heads;
    cap = tiles / 2;
    const int balanced = (total / (2 * ctas)) * ctas, unstraddled = heads * cap;
    pairs = balanced < unstraddled ? balanced : unstraddled;
    singles = total - 2 * pairs;
    full = cap > 0 ? pairs / cap : 0;
    part = cap > 0 ? pairs - full * cap : 0;
    rem = pairs % ctas;
    const int fill = rem > 0 ? 2 * (ctas - rem) : 0;
    first = fill < singles ? fill : singles;
  }

  // The n-th item of CTA b; false when the CTA has no n-th item.  ntiles_k: key tiles of the launch.
  SDVG_HD bool get(int b, int n, int ntiles_k, WsItem& it) const {
    const int my_pairs = pairs / ctas + (b < rem ? 1 : 0);
    if (n < my_pairs) {
      const int v = b + n * ctas;        // pairs > 0 implies cap > 0
      const int h = v / cap;             // head `full` included: its pairs are numbered full * cap ...
      const int l = v - h * cap;
      it.head[0] = it.head[1] = h;
      it.tile[0] = 2 * l;
      it.tile[1] = 2 * l + 1;
      it.lanes = 2;
      it.dual = false;
      it.split = false;
      it.nk[0] = it.nk[1] = ntiles_k;
      return true;
    }
    const int m = n - my_pairs;           // the CTA's m-th single
    int i;
    if (rem > 0 && b >= rem) {
      i = m < 2 ? 2 * (b - rem) + m : first + b + (m - 2) * ctas;
      if (m < 2 && i >= first) return false;     // fewer singles than short CTAs: nothing is left for the round-robin part
    } else {
      i = first + b + m * ctas;
    }
    if (i >= singles) return false;
    // singles in head order: the odd last tile of every head that gave all its pairs, then what head `full` kept,
    // then the whole heads after it
    const int odd = tiles - 2 * cap;      // 0 or 1
    int h, t;
    if (i < full * odd) {
      h = i;
      t = 2 * cap;
    } else {
      int w = i - full * odd;
      const int kept = full < heads ? tiles - 2 * part : 0;
      if (w < kept) {
        h = full;
        t = 2 * part + w;
      } else {
        w -= kept;
        h = full + 1 + w / tiles;
        t = w - (h - full - 1) * tiles;
      }
    }
    it.head[0] = it.head[1] = h;
    it.tile[0] = it.tile[1] = t;
    it.split = ntiles_k >= 2;
    it.lanes = it.split ? 2 : 1;
    it.dual = true;
    it.nk[0] = it.split ? (ntiles_k + 1) / 2 : ntiles_k;
    it.nk[1] = it.split ? ntiles_k / 2 : 0;
    return true;
  }
};
