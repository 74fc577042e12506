// Warp-specialised, persistent block-attention kernel (included by attn_fwd.cu after the common
// definitions).  One CTA per SM; a work item is a pair of 128-row query tiles ("lanes").  Usually
// the two tiles belong to one head and share every K/V tile; a pair that straddles a head boundary
// has lanes that stream their own K/V, and the tiles left over after the pairs run alone.
//
//   warps 0-3   softmax of lane 0 (one thread per row)            \  S, P and O live in tensor memory:
//   warps 4-7   softmax of lane 1                                  >  S0 S1 O0 O1 = 4 x 128 columns
//   warps 8-11  helper: rescales O when a row maximum moved, and  /
//               exponentiates the last 32 key columns of both lanes
//   warp  12    TMA producer: Q tiles, then the K/V ring
//   warp  13    MMA issuer: S_i = Q_i K^T, O_i += P_i V
//   warps 14-15 idle
//
// Tensor-pipe order per key tile j:  PV_0(j) QK_0(j+1) PV_1(j) QK_1(j+1); while the pipe works for
// lane 1 the softmax warps of lane 0 turn S_0(j+1) into P_0(j+1), and vice versa.  The running row
// maximum is only raised when it grew by more than 2^8 in the exp2 domain, so O is rarely rescaled
// and that work stays off the critical path; the final 1/l normalisation and the store are done by
// the softmax warps themselves, which own the same TMEM lanes.
//
// The chain S ready -> softmax -> P ready -> PV, QK -> next S ready of one lane sets the pace, so it
// is shortened from both ends.  A softmax thread reduces its whole row of S to the maximum, hands
// the reference maximum to the helper thread of the same row, and exponentiates key columns 0-95;
// the helper thread does columns 96-127 meanwhile.  P is released to the issuer in two parts
// (columns 0-63 and 96-127 together with "O rescaled", then columns 64-95), and the issuer starts
// the PV product on the first part while the softmax thread finishes the third quarter.  The issuer
// is blocked while the tensor pipe's queue is full, so it looks at the K/V stages of its next step
// right after queueing a batch of MMAs, when that costs nothing.  The producer and issuer warps
// run their loops with all 32 lanes (warp-uniform control flow and values) and only predicate the
// TMA / MMA / commit instructions on one elected lane: descriptors and addresses then stay in
// uniform registers.  All role loops are kept small (rare paths rolled, ragged tiles masked in
// tensor memory by a cold loop): the roles share the SM's instruction cache, and the issuer, which
// runs once per key tile, pays for every line the others push out.
//
// The exponentials are the co-limiter of this kernel: a 128 x 128 tile needs 16384 of them and the
// special-function unit delivers 16 per clock per SM, the same 1024 clocks the tile's two MMAs take.
// A compile-time share of the elements can be evaluated on the FMA pipe instead (range reduction to
// [0, 1) plus a cubic, relative error 2e-4, a tenth of the bf16 rounding P gets anyway); it is off by
// default (SDVG_ATTN_POLY_PAIRS = 0) because the extra instructions cost more than the freed
// special-function slots gain once the GPU runs under its power cap.
//
// 8-bit variant (template flag F8): Q, K and V tiles are E4M3 bytes (a 128-dim row is one 128-byte panel, so a
// tile is half the size and the ring holds 8 stages), both products use the 8-bit MMA kind (K = 32 per
// instruction, half the tensor-pipe time), P is rounded to E4M3 (four per TMEM column) and the per-head
// scales enter as a factor of the logit scale and of the final 1/l.  Everything else (roles, barriers,
// schedule, lazy maximum, split tiles) is shared; the softmax, not the tensor pipe, then sets the pace.
#pragma once

#ifdef SDVG_ATTN_TRACE
__device__ long long* g_trace = nullptr;     // [6 roles][512 events][id, clock]
#define SDVG_TRACE_DECL(cond)                 \
  long long* const tr_base = g_trace;         \
  const bool tr_on = (cond) && tr_base;       \
  int tr_n = 0;
#define SDVG_TRACE(role, id)                                                                      \
  do {                                                                                            \
    if (tr_on && tr_n < 512) {                                                                    \
      longlong2 ev_;                                                                              \
      ev_.x = (id);                                                                               \
      ev_.y = clock64();                                                                          \
      reinterpret_cast<longlong2*>(tr_base)[(role)*512 + tr_n] = ev_;                             \
      ++tr_n;                                                                                     \
    }                                                                                             \
  } while (0)
#else
#define SDVG_TRACE_DECL(cond)
#define SDVG_TRACE(role, id) do { } while (0)
#endif

// F8: operands are E4M3 bytes instead of bf16 (a row of 128 dims is then one 128-byte panel).
template <int D, bool F8 = false>
struct WsCfg {
  static_assert(!F8 || D == 128, "the 8-bit variant is built for head_dim 128");
  static constexpr int kHalves = F8 ? D / 128 : D / 64;             // 128-byte panels per row
  static constexpr int kPanelBytes = 128 * 128;
  static constexpr int kTileBytes = kHalves * kPanelBytes;          // one Q, K or V tile
  static constexpr int kStages = (D == 128 && !F8) ? 5 : 8;         // K/V ring entries (K and V alternate)
  static constexpr int kPanelElems = F8 ? 128 : 64;                 // elements per panel row
  static constexpr int kQ = 0;                                      // two query tiles
  static constexpr int kKV = 2 * kTileBytes;
  static constexpr int kRowState = kKV + kStages * kTileBytes;      // float [2][128]: -m*c2 of a row, later the helper's l
  static constexpr int kMerge = kRowState + 2 * 128 * 4;            // float [128]: lane 1's -m*c2 when a split tile is merged
  static constexpr int kBars = kMerge + 128 * 4;
  static constexpr int kNumBars = 20 + 2 * kStages;
  static constexpr int kMisc = kBars + kNumBars * 8;                // tmem slot
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;
  static constexpr int kThreads = 512;
  static constexpr uint32_t kTmemCols = 512;
  static_assert(kDynamic <= 232448, "shared memory budget");
};

struct WsItem {
  int head[2], tile[2];   // per lane
  int lanes;              // 1 or 2
  bool dual;              // lanes stream their own K/V tiles (different heads, or one tile split by keys)
  bool split;             // both lanes work on ONE query tile: lane i takes key tiles i, i + 2, i + 4, ...
  int nk[2];              // key tiles per lane
  // branch-free on purpose: a loop-invariant branch on `split` makes the compiler clone whole role loops
  __device__ int key_tile(int lane, int t) const { return (t << (int)split) + (lane & -(int)split); }
};

// Static schedule.  The query tiles of all heads form one list (head-major); with G CTAs and U tiles,
// the first P = G * floor(U / 2G) items are pairs of neighbouring tiles (tiles 2v and 2v+1: the same
// head, or, where the pair straddles a head boundary, two heads whose lanes stream their own K/V),
// the remaining U - 2P tiles are items of one tile each, whose keys are split between the two lanes
// (even and odd key tiles; the two partial results are merged when the item ends), so that a single
// tile costs about half a pair.  Items are dealt round-robin, so every CTA gets the same number of
// pairs, CTAs that run at the same time work on neighbouring tiles of few heads (their K/V tiles are
// shared through L2), and the single tiles even out the last round.
struct WsSchedule {
  int tiles, num_pairs, num_items;
  __host__ __device__ WsSchedule(int tokens, int heads, int ctas) {
    tiles = (tokens + kTileM - 1) / kTileM;
    const int total = tiles * heads;
    num_pairs = (total / (2 * ctas)) * ctas;
    num_items = num_pairs + (total - 2 * num_pairs);
  }
  __device__ void get(int v, int ntiles_k, WsItem& it) const {
    const int g0 = v < num_pairs ? 2 * v : 2 * num_pairs + (v - num_pairs);
    it.head[0] = g0 / tiles;
    it.tile[0] = g0 - it.head[0] * tiles;
    if (v < num_pairs) {
      it.head[1] = (g0 + 1) / tiles;
      it.tile[1] = g0 + 1 - it.head[1] * tiles;
      it.lanes = 2;
      it.dual = it.head[1] != it.head[0];
      it.split = false;
      it.nk[0] = it.nk[1] = ntiles_k;
    } else {
      it.head[1] = it.head[0];
      it.tile[1] = it.tile[0];
      it.split = ntiles_k >= 2;
      it.lanes = it.split ? 2 : 1;
      it.dual = true;
      it.nk[0] = it.split ? (ntiles_k + 1) / 2 : ntiles_k;
      it.nk[1] = it.split ? ntiles_k / 2 : 0;
    }
  }
};

// Ring position (stage, phase parity) advanced one stage at a time.
struct RingPos {
  uint32_t stage = 0, phase = 0;
  template <int N>
  __device__ __forceinline__ void advance() {
    if (++stage == (uint32_t)N) {
      stage = 0;
      phase ^= 1;
    }
  }
  template <int N>
  __device__ __forceinline__ void skip(uint32_t n) {
    const uint32_t t = stage + n;
    stage = t % (uint32_t)N;
    phase ^= (t / (uint32_t)N) & 1;
  }
};

// ---- packed fp32 pairs (two floats in one 64-bit register) -----------------------------------
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// round-toward-minus-infinity add: with b = 1.5 * 2^23 the low mantissa bits of the sum hold floor(a)
__device__ __forceinline__ uint64_t add2_rm(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^x for x <= 127 on the FMA and integer pipes: x = n + f with n = floor(x), f in [0, 1);
// 2^f by a cubic with p(0) = 1 (fitted to minimise the relative error, 2.0e-4 at most); n is added
// into the exponent field.  Inputs below -126 give 2^-126 (their true value is zero at bf16 scale).
__device__ __forceinline__ void exp2_poly2(uint64_t x2, float& e0, float& e1) {
  constexpr float kMagic = 12582912.f;            // 1.5 * 2^23
  float x0, x1;
  unpack2(x2, x0, x1);
  x0 = fmaxf(x0, -126.f);
  x1 = fmaxf(x1, -126.f);
  const uint64_t xc = pack2(x0, x1);
  const uint64_t magic = pack2(kMagic, kMagic);
  const uint64_t t = add2_rm(xc, magic);          // bits: 0x4B400000 + floor(x)
  const uint64_t fl = sub2(t, magic);             // floor(x), exact
  const uint64_t fr = sub2(xc, fl);               // f in [0, 1), exact
  uint64_t p = fma2(pack2(0.07764089852571487f, 0.07764089852571487f), fr,
                    pack2(0.22760449349880219f, 0.22760449349880219f));
  p = fma2(p, fr, pack2(0.6946666836738586f, 0.6946666836738586f));
  p = fma2(p, fr, pack2(1.f, 1.f));
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(t, t0, t1);
  // (bits(t) << 23) keeps n mod 512 in the exponent field; adding it to bits(p) scales p by 2^n
  e0 = __uint_as_float(__float_as_uint(t0) * 0x00800000u + __float_as_uint(p0));
  e1 = __uint_as_float(__float_as_uint(t1) * 0x00800000u + __float_as_uint(p1));
}

// Out of every 4 consecutive element pairs of a row, this many take the polynomial path.
#ifndef SDVG_ATTN_POLY_PAIRS
#define SDVG_ATTN_POLY_PAIRS 0
#endif

#ifndef SDVG_ATTN_POLY_PAIRS_F8
#define SDVG_ATTN_POLY_PAIRS_F8 0
#endif

// One 32-column chunk of a row: P = 2^(c2 * S - m*c2) as bf16 pairs, returns the packed partial row sums.
__device__ __forceinline__ void exp_chunk(const uint32_t (&s)[32], uint64_t c2x2, uint64_t negx2, uint32_t (&pk)[16],
                                          uint64_t& sum_a, uint64_t& sum_b) {
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const uint64_t x2 = fma2(pack2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1])), c2x2, negx2);
    float p0, p1;
    if ((k & 3) < SDVG_ATTN_POLY_PAIRS) {
      exp2_poly2(x2, p0, p1);
    } else {
      float x0, x1;
      unpack2(x2, x0, x1);
      p0 = fast_exp2(x0);
      p1 = fast_exp2(x1);
    }
    if (k & 1) sum_b = add2(sum_b, pack2(p0, p1));
    else sum_a = add2(sum_a, pack2(p0, p1));
    __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
    pk[k] = *reinterpret_cast<uint32_t*>(&b);
  }
}

// The same chunk as E4M3 bytes (four per word); the row sums are taken before the rounding, as above.
__device__ __forceinline__ void exp_chunk_f8(const uint32_t (&s)[32], uint64_t c2x2, uint64_t negx2, uint32_t (&pk)[8],
                                             uint64_t& sum_a, uint64_t& sum_b) {
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    float e[4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const uint64_t x2 =
          fma2(pack2(__uint_as_float(s[4 * k + 2 * u]), __uint_as_float(s[4 * k + 2 * u + 1])), c2x2, negx2);
      if (((2 * k + u) & 3) < SDVG_ATTN_POLY_PAIRS_F8) {
        exp2_poly2(x2, e[2 * u], e[2 * u + 1]);
      } else {
        float x0, x1;
        unpack2(x2, x0, x1);
        e[2 * u] = fast_exp2(x0);
        e[2 * u + 1] = fast_exp2(x1);
      }
    }
    sum_a = add2(sum_a, pack2(e[0], e[1]));
    sum_b = add2(sum_b, pack2(e[2], e[3]));
    pk[k] = pack_e4m3x4(e[0], e[1], e[2], e[3]);
  }
}

// Reference-maximum policy.  P = 2^(c2 S - m_ref c2 + shift) and the reference is only raised when the row
// maximum outgrew it by more than `lazy` (in the exp2 domain), so P <= 2^(shift + lazy).  bf16 has the
// range for 2^8; E4M3 ends at 448, and its precision ends 2^-9 below 1, so there the window is moved up:
// P <= 2^8 still, and a key 2^-12 below the reference still gets a normal number.
template <bool F8>
struct RefMax {
  static constexpr float kLazy = F8 ? 4.f : 8.f;
  static constexpr float kShift = F8 ? 4.f : 0.f;
};

__device__ __forceinline__ void max_chunk(const uint32_t (&s)[32], float (&mx)[4]) {
#pragma unroll
  for (int k = 0; k < 32; k += 8)
#pragma unroll
    for (int u = 0; u < 4; ++u)
      mx[u] = fmax3(mx[u], __uint_as_float(s[k + 2 * u]), __uint_as_float(s[k + 2 * u + 1]));
}

template <int D, bool F8 = false>
__global__ void __launch_bounds__(512, 1) attn_fwd_ws_kernel(const __grid_constant__ AttnParams p) {
  using C = WsCfg<D, F8>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // [2][128]: while an item runs, -m_ref * c2 of the row (softmax -> helper); at its end the helper's
  // share of the row sum travels back through the same word
  float* s_neg = reinterpret_cast<float*>(smem + C::kRowState);
  float* s_lhelp = s_neg;
  float* s_merge = reinterpret_cast<float*>(smem + C::kMerge);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBars);
  uint64_t* q_full = bars;            // [2] TMA -> MMA
  uint64_t* q_empty = bars + 2;       // [2] MMA -> TMA
  uint64_t* s_full = bars + 4;        // [2] MMA -> softmax
  uint64_t* p_lo = bars + 6;          // [2] P columns 0-63 (softmax), 96-127 + O rescaled (helper) -> MMA, 256 arrivals
  uint64_t* p_mid = bars + 8;         // [2] P columns 64-95 stored (softmax) -> MMA, 128 arrivals
  uint64_t* row_ready = bars + 12;    // [2] softmax -> helper: -m*c2 of the row published, 128 arrivals
  uint64_t* o_full = bars + 14;       // [2] MMA -> helper / softmax epilogue
  uint64_t* l_ready = bars + 16;      // [2] helper -> softmax epilogue: its share of the row sum, 128 arrivals
  uint64_t* lane1_done = bars + 18;   // softmax of lane 1 -> softmax of lane 0: partial result of a split tile published, 128 arrivals
  uint64_t* merge_done = bars + 19;   // softmax of lane 0 -> softmax of lane 1: O_1 has been read, 128 arrivals
  uint64_t* kv_full = bars + 20;      // [kStages]
  uint64_t* kv_empty = kv_full + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kMisc);

  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&p_lo[i], 256);
      mbar_init(&p_mid[i], 128);
      mbar_init(&row_ready[i], 128);
      mbar_init(&o_full[i], 1);
      mbar_init(&l_ready[i], 128);
    }
    mbar_init(lane1_done, 128);
    mbar_init(merge_done, 128);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    fence_mbar_init();
    for (int b = 0; b < p.batch; ++b) {
      prefetch_tmap(&p.prob[b].q_map);
      for (int s = 0; s < p.nseg; ++s) {
        prefetch_tmap(&p.prob[b].k_map[s]);
        prefetch_tmap(&p.prob[b].v_map[s]);
      }
    }
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Every wait of this kernel gives up at the same absolute time; a thread that gives up records
  // the timeout and leaves its role loop, and all roles meet at the common exit below.
  const Deadline dl{globaltimer_ns() + kWaitLimitNs, p.work + 1};
  const WsSchedule sched(p.tokens, p.heads * p.batch, gridDim.x);   // it.head[] are global heads: problem * heads + head
  int ntiles_k = 0;
  for (int s = 0; s < p.nseg; ++s) ntiles_k += (p.seg_len[s] + kTileN - 1) / kTileN;

  if (warp >= 12) {
    // ================= producer / issuer warps: few registers ==================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    if (warp == 12) {
      // ---- TMA producer -------------------------------------------------------------------
      const bool leader = elect_one();
      uint32_t q_cnt[2] = {0, 0}, kv_issued = 0;
      RingPos ring;
      bool alive = true;
      SDVG_TRACE_DECL(blockIdx.x == 0 && leader)

      // one K or V tile of key tile j of `head` into the next ring stage
      auto load_kv = [&](bool is_v, int head, int j) {
        int seg = 0, kt = j;
        for (; seg < p.nseg - 1; ++seg) {
          const int nt = (p.seg_len[seg] + kTileN - 1) / kTileN;
          if (kt < nt) break;
          kt -= nt;
        }
        if (!(alive = wait_warp(&kv_empty[ring.stage], ring.phase ^ 1, dl))) return;
        SDVG_TRACE(4, kv_issued);
        if (leader) {
          mbar_expect_tx(&kv_full[ring.stage], C::kTileBytes);
          const AttnProblem& pr = p.prob[head / p.heads];
          const CUtensorMap* m = is_v ? &pr.v_map[seg] : &pr.k_map[seg];
          for (int h = 0; h < C::kHalves; ++h)
            tma_load_3d(smem + C::kKV + ring.stage * C::kTileBytes + h * C::kPanelBytes, m, &kv_full[ring.stage],
                        h * C::kPanelElems, kt * kTileN, head % p.heads);
        }
        ring.template advance<C::kStages>();
        ++kv_issued;
      };

      #pragma unroll 1
      for (int v = blockIdx.x; v < sched.num_items && alive; v += gridDim.x) {
        WsItem it;
        sched.get(v, ntiles_k, it);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= it.lanes || !alive) break;
          if (!(alive = wait_warp(&q_empty[i], (q_cnt[i] & 1) ^ 1, dl))) break;
          ++q_cnt[i];
          if (leader) {
            mbar_expect_tx(&q_full[i], C::kTileBytes);
            for (int h = 0; h < C::kHalves; ++h)
              tma_load_3d(smem + C::kQ + i * C::kTileBytes + h * C::kPanelBytes, &p.prob[it.head[i] / p.heads].q_map,
                          &q_full[i], h * C::kPanelElems, it.tile[i] * kTileM, it.head[i] % p.heads);
          }
        }
        // K/V tiles in the order the issuer consumes them: K of the first key tile of every stream, then
        // step by step and lane by lane V of this step and K of the next
        const int streams = it.dual ? it.lanes : 1;
        for (int s = 0; s < streams && alive; ++s) load_kv(false, it.head[s], it.key_tile(s, 0));
        #pragma unroll 1
        for (int t = 0; t < it.nk[0] && alive; ++t)
          for (int s = 0; s < streams && alive; ++s) {
            if (t >= it.nk[s]) continue;
            load_kv(true, it.head[s], it.key_tile(s, t));
            if (t + 1 < it.nk[s] && alive) load_kv(false, it.head[s], it.key_tile(s, t + 1));
          }
      }
      // Drain: every load issued above lands in this CTA's shared memory; do not exit under them.
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (q_cnt[i] > 0) wait_warp(&q_full[i], (q_cnt[i] - 1) & 1, dl);
      for (uint32_t n = kv_issued > (uint32_t)C::kStages ? kv_issued - C::kStages : 0; n < kv_issued; ++n)
        wait_warp(&kv_full[n % C::kStages], (n / C::kStages) & 1, dl);
    } else if (warp == 13) {
      // ---- MMA issuer ---------------------------------------------------------------------
      const bool leader = elect_one();
      constexpr uint32_t kIdescQK = F8 ? idesc_e4m3_f32(kTileM, kTileN, false) : idesc_bf16_f32(kTileM, kTileN, false);
      constexpr uint32_t kIdescPV = F8 ? idesc_e4m3_f32(kTileM, D, true) : idesc_bf16_f32(kTileM, D, true);
      const uint32_t sQ = smem_u32(smem + C::kQ), sKV = smem_u32(smem + C::kKV);
      uint32_t q_cnt[2] = {0, 0};
      uint32_t pv_par = 0;                 // bit i: phase parity of lane i's P barriers
      RingPos ring;                        // next K/V stage to consume
      bool alive = true;
      SDVG_TRACE_DECL(blockIdx.x == 0 && leader)

      // Every instruction this warp executes between "P is ready" and the MMAs lengthens the chain that
      // paces the kernel, so the issue loops are unrolled (descriptor offsets become immediates) while the
      // loop over the two lanes stays rolled to keep the code this warp has to fetch small.
      // S_i = Q_i K^T into TMEM columns [128 i, 128 i + 128)
      // Descriptors of stage 0 and of the two query tiles, built once; a stage or a 16-wide slice is then one
      // addition to the address field (all of this CTA's shared memory fits that field, so nothing carries out).
      const uint64_t descQ0 = smem_desc_sw128(sQ, 16, 1024);
      const uint64_t descK0 = smem_desc_sw128(sKV, 16, 1024);
      const uint64_t descV0 = smem_desc_sw128(sKV, C::kPanelBytes, 1024);
      auto issue_qk = [&](int i, uint32_t st) {
        const uint32_t d = tmem_base + i * 128;
        const uint64_t a = descQ0 + (uint64_t)(i * (C::kTileBytes >> 4));
        const uint64_t b = descK0 + (uint64_t)(st * (C::kTileBytes >> 4));
        uint32_t acc = 0;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          if (F8 && kk >= D / 32) break;                   // an 8-bit MMA covers 32 dims
          // one MMA reads 32 B of every row = 2 descriptor units within a 128-byte panel, panels kPanelBytes apart
          const uint64_t off = (uint64_t)((kk >> 2) * (C::kPanelBytes >> 4) + (kk & 3) * 2);
          if constexpr (F8) mma_ss_f8(d, a + off, b + off, kIdescQK, acc);
          else mma_ss(d, a + off, b + off, kIdescQK, acc);
          acc = 1;
        }
      };
      // O_i (+)= P_i[:, 16 kk .. 16 kk + 16) V[16 kk .. 16 kk + 16, :] for kk in [k0, k1); P_i is read from
      // the first 64 columns of S_i
      auto issue_pv = [&](int i, uint32_t st, int k0, int k1, uint32_t acc) {
        const uint32_t d = tmem_base + 256 + i * 128, a = tmem_base + i * 128;
        const uint64_t b = descV0 + (uint64_t)(st * (C::kTileBytes >> 4));
#pragma unroll
        for (int kk = k0; kk < k1; ++kk) {
          // slice kk of P is 8 TMEM columns (16 bf16 or 32 bytes per row); its keys are 16 or 32 rows of V
          if constexpr (F8) mma_ts_f8(d, a + kk * 8, b + (uint64_t)(kk * (4096 >> 4)), kIdescPV, acc);
          else mma_ts(d, a + kk * 8, b + (uint64_t)(kk * (2048 >> 4)), kIdescPV, acc);
          acc = 1;
        }
      };
      // slices of P per 32-column chunk of S: chunk c of the softmax is slices [c kPc, c kPc + kPc)
      constexpr int kPc = F8 ? 1 : 2;
      // Are the next `n` (1 or 2) stages of the ring filled?  Does not block (test_wait, not try_wait,
      // which may suspend the thread for microseconds when the answer is no).
      auto stages_filled = [&](int n) {
        RingPos r = ring;
        bool ok = mbar_test_wait(&kv_full[r.stage], r.phase);
        if (n > 1) {
          r.template advance<C::kStages>();
          ok = mbar_test_wait(&kv_full[r.stage], r.phase) && ok;
        }
        return __all_sync(0xffffffffu, ok);
      };

      #pragma unroll 1
      for (int v = blockIdx.x; v < sched.num_items && alive; v += gridDim.x) {
        WsItem it;
        sched.get(v, ntiles_k, it);
        const int nl = it.lanes;
        const bool dual = it.dual;
        const int nk0 = it.nk[0], nk1 = it.nk[1];      // scalars: indexing the item by the lane would put it in local memory
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= nl || !alive) break;
          alive = wait_warp(&q_full[i], q_cnt[i] & 1, dl);
          ++q_cnt[i];
        }
        if (!alive) break;
        // ---- prologue: S_i(0) ------------------------------------------------------------------
        uint32_t stK = 0;
#pragma unroll 1
        for (int i = 0; i < nl && alive; ++i) {
          const bool own = (i == 0) || dual;                 // this lane takes a stage of its own
          const bool last_user = dual || (i == nl - 1);
          if (own) {
            stK = ring.stage;
            if (!(alive = wait_warp(&kv_full[stK], ring.phase, dl))) break;
            ring.template advance<C::kStages>();
            tc_fence_after();
          }
          if (leader) {
            issue_qk(i, stK);
            mma_commit(&s_full[i]);
            if (last_user) mma_commit(&kv_empty[stK]);
          }
        }
        // ---- main loop: step t of lane i works on that lane's t-th key tile --------------------------
        // The stages of a step (V of this key tile, K of the next) are taken from the ring one step ahead, in
        // the shadow of MMAs already queued: what is left at the start of a step is a look at `nx.filled`.
        struct {
          uint32_t stV, phV, stK, phK;
          bool filled;
        } nx = {0, 0, 0, 0, false};
        auto take = [&](bool with_k) {
          nx.stV = ring.stage;
          nx.phV = ring.phase;
          nx.filled = stages_filled(with_k ? 2 : 1);
          ring.template advance<C::kStages>();
          if (with_k) {
            nx.stK = ring.stage;
            nx.phK = ring.phase;
            ring.template advance<C::kStages>();
          }
        };
        take(nk0 > 1);                                       // for step (0, lane 0)
        #pragma unroll 1
        for (int t = 0; t < nk0 && alive; ++t) {
          uint32_t stV = 0;
          SDVG_TRACE(2, 100 + t);
          // everything that depends on t alone is worked out here: each instruction inside the lane loop
          // sits between "P is ready" and the next MMA
          const int nl_t = t < nk1 ? nl : 1;                 // a split tile with an odd number of key tiles ends on lane 0
          const bool more0 = t + 1 < nk0, more1 = t + 1 < nk1;
#pragma unroll 1
          for (int i = 0; i < nl_t && alive; ++i) {
            const bool more = i == 0 ? more0 : more1;
            const bool last_user = dual || (i == nl - 1);
            if (i == 0 || dual) {                            // this lane has stages of its own
              stV = nx.stV;
              stK = nx.stK;
              if (!nx.filled) {
                if (!(alive = wait_warp(&kv_full[stV], nx.phV, dl))) break;
                if (more && !(alive = wait_warp(&kv_full[stK], nx.phK, dl))) break;
              }
            }
            SDVG_TRACE(2, 1000 + i * 1000 + t);
            const uint32_t par = (pv_par >> i) & 1;
            pv_par ^= 1u << i;
            // P_i columns 0-63 and 96-127 stored, O_i rescaled (for t = 0: O_i was read out by the
            // epilogue of the previous item before its softmax threads arrived here)
            if (!(alive = wait_warp(&p_lo[i], par, dl))) break;
            SDVG_TRACE(2, 3000 + i * 1000 + t);
            tc_fence_after();
            if (leader) {
              issue_pv(i, stV, 3 * kPc, 4 * kPc, t > 0 ? 1u : 0u);
              issue_pv(i, stV, 0, 2 * kPc, 1u);
            }
            // six MMAs are queued: take the stages of the next step that has stages of its own
            {
              const bool next_in_this_t = dual && (i + 1 < nl_t);
              if (next_in_this_t) take(more1);
              else if (more0 && (dual || i == nl_t - 1)) take(t + 2 < nk0);
            }
            if (!(alive = wait_warp(&p_mid[i], par, dl))) break;
            SDVG_TRACE(2, 5000 + i * 1000 + t);
            tc_fence_after();
            if (leader) {
              issue_pv(i, stV, 2 * kPc, 3 * kPc, 1u);
              mma_commit(&o_full[i]);
              if (last_user) mma_commit(&kv_empty[stV]);
              if (more) {
                issue_qk(i, stK);
                mma_commit(&s_full[i]);
                if (last_user) mma_commit(&kv_empty[stK]);
              } else {
                mma_commit(&q_empty[i]);
              }
            }
            SDVG_TRACE(2, 9000 + i * 1000 + t);
          }
        }
      }
    }
  } else if (warp >= 8) {
    // ================= helper warps =============================================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
    const int row = tid - 256;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS[2] = {tmem_base + lane_off, tmem_base + 128 + lane_off};
    const uint32_t tO[2] = {tmem_base + 256 + lane_off, tmem_base + 384 + lane_off};
    const float c2 = p.scale_log2e;
    const uint64_t c2x2 = pack2(c2, c2);
    uint64_t c2h[2] = {c2x2, c2x2};      // 8-bit variant: the logit scale carries the head's q and k scales
    uint32_t cnt[2] = {0, 0};            // (item, key tile) steps done per lane = phase index of its barriers
    bool alive = true;
    SDVG_TRACE_DECL(blockIdx.x == 0 && tid == 256)
    #pragma unroll 1
    for (int v = blockIdx.x; v < sched.num_items && alive; v += gridDim.x) {
      WsItem it;
      sched.get(v, ntiles_k, it);
      float l_part[2] = {0.f, 0.f}, neg_prev[2] = {0.f, 0.f};
      if constexpr (F8) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float c = c2 * __ldg(p.qk_descale + it.head[i]);
          c2h[i] = pack2(c, c);
        }
      }
      #pragma unroll 1
      for (int j = 0; j < it.nk[0] && alive; ++j) {          // step j of lane i: that lane's j-th key tile
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= it.lanes || !alive) break;
          if (j >= it.nk[i]) continue;
          const uint32_t par = cnt[i] & 1;
          if (!(alive = wait_bar(&row_ready[i], par, dl))) break;
          const float neg = s_neg[i * 128 + row];
          // the row's reference maximum moved iff -m*c2 changed; both sides derive the factor the same way
          const bool moved = (j > 0) && (neg != neg_prev[i]);
          const float alpha = moved ? fast_exp2(__fsub_rn(neg, neg_prev[i])) : 1.f;
          neg_prev[i] = neg;
          SDVG_TRACE(3, 1000 * i + j);
          if (__any_sync(0xffffffffu, moved)) {
            // PV_i(j-1) is commit number cnt[i] - 1 on o_full[i]
            if (!(alive = wait_bar(&o_full[i], (cnt[i] - 1) & 1, dl))) break;
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {          // rare path: keep its code small
              uint32_t o[32];
              tmem_ld32(tO[i] + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
              tmem_st32(tO[i] + c * 32, o);
            }
            tmem_wait_st();
            tc_fence_before();
            l_part[i] *= alpha;
          }
          SDVG_TRACE(3, 20000 + 1000 * i + j);
          // ---- this row's share of P: key columns 96-127 -------------------------------------
          tc_fence_after();
          uint32_t s3[32];
          tmem_ld32(tS[i] + 96, s3);
          tmem_wait_ld();
          uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
          if constexpr (F8) {
            uint32_t pk[8];
            exp_chunk_f8(s3, c2h[i], pack2(neg, neg), pk, sum_a, sum_b);
            tmem_st8(tS[i] + 24, pk);
          } else {
            uint32_t pk[16];
            exp_chunk(s3, c2x2, pack2(neg, neg), pk, sum_a, sum_b);
            tmem_st16(tS[i] + 48, pk);
          }
          {
            float a0, a1, b0, b1;
            unpack2(sum_a, a0, a1);
            unpack2(sum_b, b0, b1);
            l_part[i] += (a0 + a1) + (b0 + b1);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&p_lo[i]);
          SDVG_TRACE(3, 30000 + 1000 * i + j);
          ++cnt[i];
        }
      }
      if (!alive) break;
      // hand the partial row sums to the softmax threads that normalise and store the rows
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i >= it.lanes) break;
        s_lhelp[i * 128 + row] = l_part[i];
        mbar_arrive(&l_ready[i]);
      }
    }
  } else {
    // ================= softmax warps ===========================================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 176;");
    const int i = warp >> 2;                       // lane (query tile) of this warpgroup
    const int row = tid & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + i * 128 + lane_off;
    const uint32_t tO = tmem_base + 256 + i * 128 + lane_off;
    float c2 = p.scale_log2e;
    uint64_t c2x2 = pack2(c2, c2);
    uint32_t s_cnt = 0, pv_cnt = 0, item_cnt = 0, split_cnt = 0;
    bool alive = true;
    SDVG_TRACE_DECL(blockIdx.x == 0 && row == 0)
    #pragma unroll 1
    for (int v = blockIdx.x; v < sched.num_items && alive; v += gridDim.x) {
      WsItem it;
      sched.get(v, ntiles_k, it);
      if (it.lanes <= i) continue;
      // this lane's fields as scalars (indexing the item by the lane would put it in local memory)
      const int my_nk = i == 0 ? it.nk[0] : it.nk[1];
      const int my_tile = i == 0 ? it.tile[0] : it.tile[1];
      const int my_head = i == 0 ? it.head[0] : it.head[1];
      if constexpr (F8) {                                  // the logit scale carries the head's q and k scales
        c2 = p.scale_log2e * __ldg(p.qk_descale + my_head);
        c2x2 = pack2(c2, c2);
      }
      float m_ref = -INFINITY, l_run = 0.f, neg = 0.f;     // neg = -m_ref * c2 (+ the window shift)
      {
        #pragma unroll 1
        for (int j = 0; j < my_nk && alive; ++j) {        // this lane's j-th key tile
          // number of real keys in that tile: the last tile of a key segment may be ragged
          int valid = kTileN;
          {
            int kt = it.key_tile(i, j);
            for (int seg = 0; seg < p.nseg; ++seg) {
              const int nt = (p.seg_len[seg] + kTileN - 1) / kTileN;
              if (kt < nt) {
                valid = min(kTileN, p.seg_len[seg] - kt * kTileN);
                break;
              }
              kt -= nt;
            }
          }
          SDVG_TRACE(i, 0 + j);
          if (!(alive = wait_bar(&s_full[i], s_cnt & 1, dl))) break;
          SDVG_TRACE(i, 1000 + j);
          ++s_cnt;
          tc_fence_after();
          if (valid < kTileN) {
            // Ragged last tile of a key segment (TMA zero-filled the missing keys): overwrite their
            // columns of S with -inf in tensor memory, for this thread and for the helper thread of the
            // row, which reads its columns after row_ready.  Rare, so a plain column-by-column loop.
#pragma unroll 1
            for (int c = valid; c < kTileN; ++c) tmem_st1(tS + c, 0xff800000u);
            tmem_wait_st();
          }
          // ---- row maximum over all 128 columns; the second half streams in while the first is reduced
          uint32_t s[3][32];
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          {
            uint32_t s3[32];
            tmem_ld32(tS + 96, s3);
            tmem_ld32(tS, s[0]);
            tmem_wait_ld();
            tmem_ld32(tS + 32, s[1]);
            tmem_ld32(tS + 64, s[2]);
            max_chunk(s3, mx);
            max_chunk(s[0], mx);
          }
          tmem_wait_ld();
          SDVG_TRACE(i, 2000 + j);
          max_chunk(s[1], mx);
          max_chunk(s[2], mx);
          const float mxa = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          if (j == 0) {
            m_ref = mxa;
            neg = __fmul_rn(-mxa, c2) + RefMax<F8>::kShift;
          } else if ((mxa - m_ref) * c2 > RefMax<F8>::kLazy) {
            const float neg_new = __fmul_rn(-mxa, c2) + RefMax<F8>::kShift;
            l_run *= fast_exp2(__fsub_rn(neg_new, neg));      // the helper derives the same factor from the same two values
            m_ref = mxa;
            neg = neg_new;
          }
          s_neg[i * 128 + row] = neg;
          mbar_arrive(&row_ready[i]);
          SDVG_TRACE(i, 3000 + j);
          // ---- P = 2^(c2 * (S - m_ref)), bf16, written back over S: columns 0-63, then 64-95 ------
          const uint64_t negx2 = pack2(neg, neg);
          uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
          uint32_t pk[F8 ? 8 : 16];
          if constexpr (F8) {
            exp_chunk_f8(s[0], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st8(tS, pk);
            exp_chunk_f8(s[1], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st8(tS + 8, pk);
          } else {
            exp_chunk(s[0], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st16(tS, pk);
            exp_chunk(s[1], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st16(tS + 16, pk);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&p_lo[i]);
          SDVG_TRACE(i, 4000 + j);
          if constexpr (F8) {
            exp_chunk_f8(s[2], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st8(tS + 16, pk);
          } else {
            exp_chunk(s[2], c2x2, negx2, pk, sum_a, sum_b);
            tmem_st16(tS + 32, pk);
          }
          {
            float a0, a1, b0, b1;
            unpack2(sum_a, a0, a1);
            unpack2(sum_b, b0, b1);
            l_run += (a0 + a1) + (b0 + b1);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&p_mid[i]);
          SDVG_TRACE(i, 5000 + j);
        }
      }
      if (!alive) break;
      // ---- epilogue: add the helper's share of the row sum, wait for the last PV, normalise, store
      // (the next item's first arrival on p_lo comes after these TMEM reads, which is what lets the
      // issuer overwrite O_i then)
      if (!(alive = wait_bar(&l_ready[i], item_cnt & 1, dl))) break;
      ++item_cnt;
      l_run += s_lhelp[i * 128 + row];
      pv_cnt += my_nk;
      if (!(alive = wait_bar(&o_full[i], (pv_cnt - 1) & 1, dl))) break;
      tc_fence_after();
      // A split tile: both lanes hold a partial result of the SAME rows over disjoint keys, each relative to its
      // own reference maximum.  Lane 1 publishes (-m*c2, l) and waits until lane 0 has folded O_1 into its output.
      float w0 = 1.f, w1 = 0.f;                      // weights of O_0 and O_1 in the merged numerator
      if (it.split) {
        const uint32_t par = split_cnt & 1;
        ++split_cnt;
        if (i == 1) {
          s_merge[row] = neg;
          s_neg[128 + row] = l_run;
          tc_fence_before();
          mbar_arrive(lane1_done);
          alive = wait_bar(merge_done, par, dl);
          if (!alive) break;
          continue;
        }
        if (!(alive = wait_bar(lane1_done, par, dl))) break;
        tc_fence_after();
        const float neg1 = s_merge[row], l1 = s_neg[128 + row];
        const float negm = fminf(neg, neg1);         // the larger of the two reference maxima
        w0 = fast_exp2(negm - neg);                  // 2^((m_0 - m) c2) <= 1: rebases lane 0's sums to the common maximum
        w1 = fast_exp2(negm - neg1);
        l_run = l_run * w0 + l1 * w1;
        neg = negm;
      }
      const int grow = my_tile * kTileM + row;
      const AttnProblem& pr = p.prob[my_head / p.heads];
      const int head = my_head % p.heads;
      const float inv = F8 ? __ldg(p.v_descale + head) / l_run : 1.f / l_run;     // 8-bit: V's scale of this head
      w0 *= inv;
      w1 *= inv;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {                  // once per item: keep its code small
        uint32_t o[32];
        tmem_ld32(tO + c * 32, o);
        tmem_wait_ld();
        if (it.split) {
          uint32_t o1[32];
          tmem_ld32(tO + 128 + c * 32, o1);               // O_1 sits 128 columns after O_0, same TMEM lanes
          tmem_wait_ld();
#pragma unroll
          for (int k = 0; k < 32; ++k)
            o[k] = __float_as_uint(__uint_as_float(o[k]) * w0 + __uint_as_float(o1[k]) * w1);
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * w0);
        }
        if (grow < p.tokens) {
          uint4* dst = reinterpret_cast<uint4*>(pr.out + ((size_t)grow * p.heads + head) * D + c * 32);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(o[q4 * 8 + 2 * k]),
                                                       __uint_as_float(o[q4 * 8 + 2 * k + 1]));
              w[k] = *reinterpret_cast<uint32_t*>(&b);
            }
            dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      tc_fence_before();
      if (it.split) mbar_arrive(merge_done);
      if (pr.lse && grow < p.tokens)
        pr.lse[(size_t)head * p.tokens + grow] = -neg * 0.6931471805599453f + logf(l_run);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, C::kTmemCols);
}
