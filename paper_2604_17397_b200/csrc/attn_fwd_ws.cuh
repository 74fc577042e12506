// Warp-specialised, persistent block-attention kernel (included by attn_fwd.cu after the common
// definitions).  One CTA of 20 warps per SM; a work item is a pair of 128-row query tiles ("lanes").
// Usually the two tiles belong to one head and share every K/V tile; a pair that straddles a head
// boundary has lanes that stream their own K/V, and the tiles left over after the pairs run alone,
// their keys split between the two lanes (attn_schedule.h says which CTA gets which).
//
//   warps 0-3    softmax of lane 0, key columns 0-63 of every tile     \  two threads per query row: a warp
//   warps 4-7    softmax of lane 1, key columns 0-63                    \ reaches the 32 TMEM lanes of its place
//   warps 8-11   softmax of lane 0, key columns 64-127                  / in its warpgroup, so the threads of a
//   warps 12-15  softmax of lane 1, key columns 64-127                 /  row sit in warps w and w + 8
//   warp  16     TMA producer: Q tiles, then the K/V ring
//   warp  17     MMA issuer of the first product,  S = Q_i K^T
//   warp  18     MMA issuer of the second product, O_i += P_i V
//   warp  19     idle (warps come in fours: one per SM sub-partition)
//
// Tensor memory: O_0 and O_1 (128 columns each), ONE S (128 columns) that the lanes use in turn, P_0 and P_1
// (64 columns each: bf16 pairs).  S only lives from the end of its product until the softmax threads of its
// lane have read it into registers (s_free); the first product of the NEXT key tile of the other lane can
// then start, whatever the softmax of either lane is doing.  Each lane's first product therefore runs one
// key tile ahead of its softmax, and the chain "S ready -> softmax -> P ready -> second product -> next
// first product -> S ready" that would otherwise pace a lane is cut: the softmax threads find their next row
// of S waiting when they have stored P, and the second product only has to finish before the lane's NEXT P
// is stored (o_full).  What paces the kernel is then the slower of the tensor pipe and the special-function
// unit: a 128 x 128 tile needs 16384 exponentials at 16 per clock per SM, the same 1024 clocks its two
// products take.
//
// A softmax thread reads its 64 logits, reduces them to a maximum, swaps that with the row's other thread
// through shared memory (mx_ready), and both take the same decision: the reference maximum m is only
// raised when the row maximum outgrew it by more than 2^8 in the exp2 domain, so O is rarely rescaled
// (when it is, each of the two threads rescales half of the head dimension).  P = 2^(c S - c m) is
// rounded to bf16 and stored to the lane's P columns; the row sum is kept per thread and added up when the
// item ends, where the lower-half thread normalises by 1/l and stores the row.
// The two products have an issuing warp each, so that the waits and bookkeeping of one overlap the MMAs
// of the other (the tensor pipe queues only a few instructions).  The producer and issuer warps run their
// loops with all 32 lanes (warp-uniform control flow and values) and only predicate the TMA / MMA / commit
// instructions on one elected lane: descriptors and addresses then stay in uniform registers.
//
// A compile-time share of the exponentials can be evaluated on the FMA pipe instead (range reduction to
// [0, 1) plus a cubic, relative error 2e-4, a tenth of the bf16 rounding P gets anyway); it is off because
// the extra instructions cost more issue slots than the freed special-function slots gain.
//
// 8-bit variant (template flag F8): Q, K and V tiles are E4M3 bytes (a 128-dim row is one 128-byte panel, so a
// tile is half the size and the ring holds 8 stages), both products use the 8-bit MMA kind (K = 32 per
// instruction, half the tensor-pipe time), P is rounded to E4M3 (four per TMEM column) and the per-head
// scales enter as a factor of the logit scale and of the final 1/l.  Everything else is shared.
#pragma once

#include "attn_schedule.h"


// F8: operands are E4M3 bytes instead of bf16 (a row of 128 dims is then one 128-byte panel).
template <int D, bool F8 = false>
struct WsCfg {
  static_assert(!F8 || D == 128, "the 8-bit variant is built for head_dim 128");
  static constexpr int kHalves = F8 ? D / 128 : D / 64;             // 128-byte panels per row
  static constexpr int kPanelBytes = 128 * 128;
  static constexpr int kTileBytes = kHalves * kPanelBytes;          // one Q, K or V tile
  static constexpr int kStages = (D == 128 && !F8) ? 4 : 8;         // K/V ring entries (K and V alternate)
  static constexpr int kPanelElems = F8 ? 128 : 64;                 // elements per panel row
  static constexpr int kQ = 0;                                      // two query tiles
  static constexpr int kKV = 2 * kTileBytes;
  static constexpr int kRowMax = kKV + kStages * kTileBytes;        // float [2 parities][2 lanes][2 halves][128]: partial row maxima
  static constexpr int kRowSum = kRowMax + 2 * 2 * 2 * 128 * 4;     // float [2 lanes][128]: the upper half's share of the row sum
  static constexpr int kMerge = kRowSum + 2 * 128 * 4;              // float [2][128]: lane 1's -m*c2 and l when a split tile is merged, then its V scale exponent
  static constexpr int kBars = kMerge + 2 * 128 * 4 + 16;
  static constexpr int kNumBars = 20 + 2 * kStages;
  static constexpr int kMisc = kBars + kNumBars * 8;                // tmem slot
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;
  static constexpr int kSoftmaxWarps = 16;                          // 2 lanes x 2 column halves x 4 warps
  static constexpr int kThreads = (kSoftmaxWarps + 4) * 32;         // + TMA producer, the two MMA issuers, one idle warp
  static constexpr uint32_t kTmemCols = 512;
  // Registers.  Warp w runs on SM sub-partition w % 4, each of which has 16384 registers: four softmax warps and
  // one of warps 16-19 share one.  The CTA is launched with kLaunchRegs per thread; the softmax warps then grow
  // to kSoftmaxRegs out of what the fifth warp gives back (setmaxnreg).
  static constexpr int kLaunchRegs = 96, kSoftmaxRegs = 112, kIssueRegs = 32;
  static_assert(5 * 32 * kLaunchRegs <= 16384, "register file of a sub-partition");
  static_assert(4 * kSoftmaxRegs + kIssueRegs <= 5 * kLaunchRegs, "register pool of a sub-partition");
  static_assert(kDynamic <= 232448, "shared memory budget");
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

// Share of the exponentials that goes to the FMA pipe: out of every 4 consecutive element pairs of a
// 32-column chunk this many take the polynomial (4 = the whole chunk), separately for the threads that own
// key columns 0-63 and 64-127 of a row.
#ifndef SDVG_POLY_LOWER
#define SDVG_POLY_LOWER 0
#endif
#ifndef SDVG_POLY_UPPER
#define SDVG_POLY_UPPER 0
#endif
#ifndef SDVG_POLY_LOWER_F8
#define SDVG_POLY_LOWER_F8 0
#endif
#ifndef SDVG_POLY_UPPER_F8
#define SDVG_POLY_UPPER_F8 0
#endif
template <bool F8>
struct ExpMix {
  static constexpr int kLower = F8 ? SDVG_POLY_LOWER_F8 : SDVG_POLY_LOWER;     // key columns 0-63
  static constexpr int kUpper = F8 ? SDVG_POLY_UPPER_F8 : SDVG_POLY_UPPER;     // key columns 64-127
};

// One 32-column chunk of a row: P = 2^(c2 * S - m*c2) as bf16 pairs, returns the packed partial row sums.
// POLY of every 4 consecutive element pairs take the polynomial path (4: the whole chunk).
template <int POLY>
__device__ __forceinline__ void exp_chunk(const uint32_t (&s)[32], uint64_t c2x2, uint64_t negx2, uint32_t (&pk)[16],
                                          uint64_t& sum_a, uint64_t& sum_b) {
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const uint64_t x2 = fma2(pack2(__uint_as_float(s[2 * k]), __uint_as_float(s[2 * k + 1])), c2x2, negx2);
    float p0, p1;
    if ((k & 3) < POLY) {
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
template <int POLY>
__device__ __forceinline__ void exp_chunk_f8(const uint32_t (&s)[32], uint64_t c2x2, uint64_t negx2, uint32_t (&pk)[8],
                                             uint64_t& sum_a, uint64_t& sum_b) {
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    float e[4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const uint64_t x2 =
          fma2(pack2(__uint_as_float(s[4 * k + 2 * u]), __uint_as_float(s[4 * k + 2 * u + 1])), c2x2, negx2);
      if (((2 * k + u) & 3) < POLY) {
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

// Number of real keys in key tile `kt` of the concatenated key segments (the last tile of a segment may be ragged).
template <bool TS>
__device__ __forceinline__ int key_tile_valid(const AttnParams& p, int kt) {
  if constexpr (TS) return min(kTileN, p.tokens - (kt % p.ts_tiles) * kTileN);      // every ring slot is tiled on its own
  int valid = kTileN;
  for (int seg = 0; seg < p.nseg; ++seg) {
    const int nt = (p.seg_len[seg] + kTileN - 1) / kTileN;
    if (kt < nt) {
      valid = min(kTileN, p.seg_len[seg] - kt * kTileN);
      break;
    }
    kt -= nt;
  }
  return valid;
}

template <int D, bool F8 = false, bool TS = false>
__global__ void __launch_bounds__(WsCfg<D, F8>::kThreads, 1) attn_fwd_ws_kernel(const __grid_constant__ AttnParams p) {
  static_assert(!TS || F8, "tile scales belong to the 8-bit variant");
  using C = WsCfg<D, F8>;
  using Mix = ExpMix<F8>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* s_rowmax = reinterpret_cast<float*>(smem + C::kRowMax);
  float* s_rowsum = reinterpret_cast<float*>(smem + C::kRowSum);
  float* s_merge = reinterpret_cast<float*>(smem + C::kMerge);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBars);
  uint64_t* q_full = bars;            // [2] TMA -> MMA
  uint64_t* q_empty = bars + 2;       // [2] MMA -> TMA
  uint64_t* s_full = bars + 4;        // [2] MMA -> softmax: S holds lane i's logits
  uint64_t* p_ready = bars + 6;       // [2] softmax -> MMA: P_i stored (and O_i rescaled), 256 arrivals
  uint64_t* mx_ready = bars + 8;      // [2] softmax <-> softmax: both partial row maxima published, 256 arrivals
  uint64_t* s_free = bars + 10;       // softmax -> MMA: the row of S is in registers, 256 arrivals
  uint64_t* sum_ready = bars + 12;    // [2] upper half -> lower half: its share of the row sum, 128 arrivals
  uint64_t* o_full = bars + 14;       // [2] MMA -> softmax: O_i += P_i V has completed
  uint64_t* lane1_done = bars + 18;   // lane 1 -> lane 0: partial result of a split tile published, 128 arrivals
  uint64_t* merge_done = bars + 19;   // lane 0 -> lane 1: O_1 has been read, 128 arrivals
  uint64_t* kv_full = bars + 20;      // [kStages]
  uint64_t* kv_empty = kv_full + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kMisc);

  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&p_ready[i], 256);
      mbar_init(&mx_ready[i], 256);
      mbar_init(&sum_ready[i], 128);
      mbar_init(&o_full[i], 1);
    }
    mbar_init(s_free, 256);
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
  // tensor memory columns: O_0, O_1 (128 each), S (128, shared by the two lanes), P_0, P_1 (64 each)
  constexpr uint32_t kColO = 0, kColS = 256, kColP = 384;
  // Every wait of this kernel gives up at the same absolute time; a thread that gives up records
  // the timeout and leaves its role loop, and all roles meet at the common exit below.
  const Deadline dl{globaltimer_ns() + kWaitLimitNs, p.work + 1};
  const WsSchedule sched(p.tokens, p.heads * p.batch, gridDim.x, kTileM);   // it.head[] are global heads: problem * heads + head
  int ntiles_k = 0;
  if constexpr (TS) ntiles_k = p.ts_nslots * p.ts_tiles;
  else
    for (int s = 0; s < p.nseg; ++s) ntiles_k += (p.seg_len[s] + kTileN - 1) / kTileN;

  if (warp >= C::kSoftmaxWarps) {
    // ================= producer / issuer warps: few registers ==================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kIssueRegs));
    if (warp == C::kSoftmaxWarps) {
      // ---- TMA producer -------------------------------------------------------------------
      const bool leader = elect_one();
      uint32_t q_cnt[2] = {0, 0}, kv_issued = 0;
      RingPos ring;
      bool alive = true;

      // one K or V tile of key tile j of `head` into the next ring stage
      auto load_kv = [&](bool is_v, int head, int j) {
        if constexpr (TS) {
          // one 4-D map over the whole byte ring (dim, token, slot, head): tile j of the visible slots, rows past
          // the block's end read as zero
          if (!(alive = wait_warp(&kv_empty[ring.stage], ring.phase ^ 1, dl))) return;
          if (leader) {
            mbar_expect_tx(&kv_full[ring.stage], C::kTileBytes);
            const AttnProblem& pr = p.prob[0];
            tma_load_4d(smem + C::kKV + ring.stage * C::kTileBytes, is_v ? &pr.v_map[0] : &pr.k_map[0],
                        &kv_full[ring.stage], 0, (j % p.ts_tiles) * kTileN, p.ts_slot[j / p.ts_tiles], head);
          }
          ring.template advance<C::kStages>();
          ++kv_issued;
          return;
        }
        int seg = 0, kt = j;
        for (; seg < p.nseg - 1; ++seg) {
          const int nt = (p.seg_len[seg] + kTileN - 1) / kTileN;
          if (kt < nt) break;
          kt -= nt;
        }
        if (!(alive = wait_warp(&kv_empty[ring.stage], ring.phase ^ 1, dl))) return;
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

      WsItem it;
      #pragma unroll 1
      for (int n = 0; alive && sched.get(blockIdx.x, n, ntiles_k, it); ++n) {
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
        // K/V tiles in the order the issuers consume them: K of the first key tile of every stream, then
        // step by step and lane by lane K of the next step and V of this one
        const int streams = it.dual ? it.lanes : 1;
        for (int s = 0; s < streams && alive; ++s) load_kv(false, it.head[s], it.key_tile(s, 0));
        #pragma unroll 1
        for (int t = 0; t < it.nk[0] && alive; ++t)
          for (int s = 0; s < streams && alive; ++s) {
            if (t >= it.nk[s]) continue;
            if (t + 1 < it.nk[s]) load_kv(false, it.head[s], it.key_tile(s, t + 1));
            if (alive) load_kv(true, it.head[s], it.key_tile(s, t));
          }
      }
      // Drain: every load issued above lands in this CTA's shared memory; do not exit under them.
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (q_cnt[i] > 0) wait_warp(&q_full[i], (q_cnt[i] - 1) & 1, dl);
      for (uint32_t n = kv_issued > (uint32_t)C::kStages ? kv_issued - C::kStages : 0; n < kv_issued; ++n)
        wait_warp(&kv_full[n % C::kStages], (n / C::kStages) & 1, dl);
    } else if (warp == C::kSoftmaxWarps + 1) {
      // ---- MMA issuer, first product: S = Q_i K^T ------------------------------------------------
      // The two products have an issuing warp each: while one warp sits in its waits and bookkeeping the
      // other one's MMAs keep the tensor pipe fed (the pipe takes only a few instructions ahead).
      const bool leader = elect_one();
      constexpr uint32_t kIdescQK = F8 ? idesc_e4m3_f32(kTileM, kTileN, false) : idesc_bf16_f32(kTileM, kTileN, false);
      const uint32_t sQ = smem_u32(smem + C::kQ), sKV = smem_u32(smem + C::kKV);
      uint32_t q_cnt[2] = {0, 0};
      uint32_t qk_cnt = 0;                 // products written into S so far = phase index of s_free
      RingPos ring;                        // walks every entry of the K/V ring; this warp consumes the K tiles
      bool alive = true;
      // Descriptors of stage 0 and of the two query tiles, built once; a stage or a 16-wide slice is then one
      // addition to the address field (all of this CTA's shared memory fits that field, so nothing carries out).
      const uint64_t descQ0 = smem_desc_sw128(sQ, 16, 1024);
      const uint64_t descK0 = smem_desc_sw128(sKV, 16, 1024);
      // S_i(t) = Q_i K^T of the lane's t-th key tile, from the ring's next stage if the lane has one of its own
      // (else from `st`, the stage the other lane just used); the previous occupant of S must have been read
      // into registers by its softmax threads
      auto qk_step = [&](int i, bool own, uint32_t& st, bool release_stage, bool last_of_item) {
        if (own) {
          st = ring.stage;
          if (!(alive = wait_warp(&kv_full[st], ring.phase, dl))) return;
          ring.template advance<C::kStages>();
        }
        if (qk_cnt > 0 && !(alive = wait_warp(s_free, (qk_cnt - 1) & 1, dl))) return;
        ++qk_cnt;
        tc_fence_after();
        if (leader) {
          const uint32_t d = tmem_base + kColS;
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
          mma_commit(&s_full[i]);
          if (release_stage) mma_commit(&kv_empty[st]);
          if (last_of_item) mma_commit(&q_empty[i]);
        }
      };

      WsItem it;
      #pragma unroll 1
      for (int n = 0; alive && sched.get(blockIdx.x, n, ntiles_k, it); ++n) {
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
        uint32_t stK = 0;
        // ---- prologue: S_i(0) ------------------------------------------------------------------
#pragma unroll 1
        for (int i = 0; i < nl && alive; ++i)
          qk_step(i, (i == 0) || dual, stK, dual || (i == nl - 1), (i == 0 ? nk0 : nk1) == 1);
        // ---- step t of lane i: S_i(t+1), one key tile ahead of that lane's softmax -----------------
        #pragma unroll 1
        for (int t = 0; t < nk0 && alive; ++t) {
          const int nl_t = t < nk1 ? nl : 1;                 // a split tile with an odd number of key tiles ends on lane 0
#pragma unroll 1
          for (int i = 0; i < nl_t && alive; ++i) {
            const int nk_i = i == 0 ? nk0 : nk1;
            const bool own = (i == 0) || dual;               // this lane has stages of its own
            if (t + 1 < nk_i) qk_step(i, own, stK, dual || (i == nl - 1), t + 2 == nk_i);
            if (own) ring.template advance<C::kStages>();    // V of this step: the other issuing warp's tile
          }
        }
      }
    } else if (warp == C::kSoftmaxWarps + 2) {
      // ---- MMA issuer, second product: O_i += P_i V ----------------------------------------------
      const bool leader = elect_one();
      constexpr uint32_t kIdescPV = F8 ? idesc_e4m3_f32(kTileM, D, true) : idesc_bf16_f32(kTileM, D, true);
      const uint32_t sKV = smem_u32(smem + C::kKV);
      uint32_t pv_par = 0;                 // bit i: phase parity of lane i's P barrier
      RingPos ring;                        // walks every entry of the K/V ring; this warp consumes the V tiles
      bool alive = true;
      const uint64_t descV0 = smem_desc_sw128(sKV, C::kPanelBytes, 1024);
      constexpr int kSlices = F8 ? 4 : 8;  // MMAs per key tile: 32 or 16 keys each

      WsItem it;
      #pragma unroll 1
      for (int n = 0; alive && sched.get(blockIdx.x, n, ntiles_k, it); ++n) {
        const int nl = it.lanes;
        const bool dual = it.dual;
        const int nk0 = it.nk[0], nk1 = it.nk[1];
        ring.template skip<C::kStages>(dual ? nl : 1);       // the K tiles of the prologue
        uint32_t stV = 0;
        #pragma unroll 1
        for (int t = 0; t < nk0 && alive; ++t) {
          const int nl_t = t < nk1 ? nl : 1;
#pragma unroll 1
          for (int i = 0; i < nl_t && alive; ++i) {
            const int nk_i = i == 0 ? nk0 : nk1;
            const bool last_user = dual || (i == nl - 1);
            if ((i == 0) || dual) {                          // this lane has stages of its own
              if (t + 1 < nk_i) ring.template advance<C::kStages>();   // K of the next step
              stV = ring.stage;
              if (!(alive = wait_warp(&kv_full[stV], ring.phase, dl))) break;
              ring.template advance<C::kStages>();
            }
            const uint32_t par = (pv_par >> i) & 1;
            pv_par ^= 1u << i;
            // P_i stored and O_i rescaled where a row maximum moved (for t = 0: O_i was read out by the
            // epilogue of the previous item before its softmax threads arrived here)
            if (!(alive = wait_warp(&p_ready[i], par, dl))) break;
            tc_fence_after();
            if (leader) {
              // O_i (+)= P_i[:, slice kk] V[slice kk, :]; slice kk of P is 8 TMEM columns (16 bf16 or 32 bytes per
              // row), its keys are 16 or 32 rows of V
              const uint32_t d = tmem_base + kColO + i * 128, a = tmem_base + kColP + i * 64;
              const uint64_t b = descV0 + (uint64_t)(stV * (C::kTileBytes >> 4));
              uint32_t acc = t > 0 ? 1u : 0u;
#pragma unroll
              for (int kk = 0; kk < kSlices; ++kk) {
                if constexpr (F8) mma_ts_f8(d, a + kk * 8, b + (uint64_t)(kk * (4096 >> 4)), kIdescPV, acc);
                else mma_ts(d, a + kk * 8, b + (uint64_t)(kk * (2048 >> 4)), kIdescPV, acc);
                acc = 1;
              }
              mma_commit(&o_full[i]);
              if (last_user) mma_commit(&kv_empty[stV]);
            }
          }
        }
      }
    }
  } else {
    // ================= softmax warps ===========================================================
    // Two threads per query row: warps 0-7 take key columns 0-63 of their lane's rows (warps 0-3 lane 0,
    // warps 4-7 lane 1), warps 8-15 columns 64-127.  A warp reaches the 32 TMEM lanes of its position in its
    // warpgroup, so the two threads of a row sit in warps w and w + 8.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kSoftmaxRegs));
    const int i = (warp >> 2) & 1;                 // lane (query tile)
    const int half = warp >> 3;                    // 0: key columns 0-63 of every tile, 1: columns 64-127
    const int row = tid & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + kColS + lane_off + half * 64;
    const uint32_t tP = tmem_base + kColP + i * 64 + lane_off + half * (F8 ? 16 : 32);
    const uint32_t tO = tmem_base + kColO + i * 128 + lane_off;
    float* const my_max = s_rowmax + (i * 2 + half) * 128 + row;           // + parity * 512
    float* const other_max = s_rowmax + (i * 2 + (half ^ 1)) * 128 + row;
    float c2 = p.scale_log2e;
    uint64_t c2x2 = pack2(c2, c2);
    uint32_t s_cnt = 0, pv_cnt = 0, item_cnt = 0, split_cnt = 0;
    bool alive = true;
    WsItem it;
    #pragma unroll 1
    for (int n = 0; alive && sched.get(blockIdx.x, n, ntiles_k, it); ++n) {
      if (it.lanes <= i) continue;
      // this lane's fields as scalars (indexing the item by the lane would put it in local memory)
      const int my_nk = i == 0 ? it.nk[0] : it.nk[1];
      const int my_tile = i == 0 ? it.tile[0] : it.tile[1];
      const int my_head = i == 0 ? it.head[0] : it.head[1];
      float c2_item = c2;                                  // tile scales: scale * log2(e) * this query tile's scale
      if constexpr (TS) {
        c2_item = p.scale_log2e * __ldg(p.prob[0].q_tile_scale + my_head * p.ts_tiles + my_tile);
      } else if constexpr (F8) {                           // the logit scale carries the head's q and k scales
        c2 = p.scale_log2e * __ldg(p.prob[my_head / p.heads].qk_descale + my_head % p.heads);
        c2x2 = pack2(c2, c2);
      }
      float m_ref = -INFINITY, l_run = 0.f, neg = 0.f;     // neg = -m_ref * c2 (+ the window shift)
      int lv_ref = 0;                                      // tile scales: exponent of the V scale that O is relative to
      // tile scales: this lane's current key tile as (visible slot, tile of the slot), stepped along with j
      int ts_sl = 0, ts_tl = TS ? it.key_tile(i, 0) : 0;
      const int ts_step = 1 << (int)it.split;
      if constexpr (TS)
        while (ts_tl >= p.ts_tiles) ts_tl -= p.ts_tiles, ++ts_sl;
      #pragma unroll 1
      for (int j = 0; j < my_nk && alive; ++j) {          // this lane's j-th key tile
        // number of real keys in that tile: the last tile of a key segment may be ragged
        const int valid = TS ? min(kTileN, p.tokens - ts_tl * kTileN) : key_tile_valid<TS>(p, it.key_tile(i, j));
        float k_sc = 1.f, v_sc = 1.f;                      // tile scales: this key tile's K and V scales (powers of two),
        if constexpr (TS) {                                // fetched ahead of the wait for the logits
          const int idx = (my_head * p.ts_cache_slots + p.ts_slot[ts_sl]) * p.ts_tiles + ts_tl;
          k_sc = __ldg(p.prob[0].k_tile_scale + idx);
          v_sc = __ldg(p.prob[0].v_tile_scale + idx);
          ts_tl += ts_step;
          while (ts_tl >= p.ts_tiles) ts_tl -= p.ts_tiles, ++ts_sl;
        }
        const uint32_t par = s_cnt & 1;
        if (!(alive = wait_bar(&s_full[i], par, dl))) break;
        tc_fence_after();
        // ---- this thread's 64 logits of the row into registers; S is then free for the other lane's product
        uint32_t s[2][32];
        tmem_ld32(tS, s[0]);
        tmem_ld32(tS + 32, s[1]);
        tmem_wait_ld();
        tc_fence_before();
        mbar_arrive(s_free);
        if (valid < kTileN) {
          // ragged last tile of a key segment (TMA zero-filled the missing keys): their logits become -inf
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int k = 0; k < 32; ++k)
              if (half * 64 + c * 32 + k >= valid) s[c][k] = 0xff800000u;
        }
        // ---- row maximum: own half, published for the row's other thread
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        max_chunk(s[0], mx);
        max_chunk(s[1], mx);
        const float mx_own = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
        my_max[par * 512] = mx_own;
        mbar_arrive(&mx_ready[i]);
        if (!(alive = wait_bar(&mx_ready[i], par, dl))) break;
        const float mxa = fmaxf(mx_own, other_max[par * 512]);
        // both threads of the row take the same decision from the same values
        float alpha = 1.f;
        bool moved = false;
        float neg_tile = 0.f, l_gain = 1.f;                // tile scales only
        if constexpr (TS) {
          // Logits of this tile are S * c2 with the tile's own K scale, so the reference maximum is kept in
          // scaled units.  V's scale rides on P: P = 2^(x - m_ref + shift - d), d = lv_ref - lv >= 0, with lv_ref
          // the largest V exponent met so far (O is rescaled, exactly, when it rises; the row sum never carries it).
          // d stops at 64: beyond that the tile's values are below 2^-64 of what O holds and P may vanish, but
          // the row sum still gets the tile's weights, scaled back by 2^d.
          c2 = c2_item * k_sc;
          c2x2 = pack2(c2, c2);
          const int lv = (__float_as_int(v_sc) >> 23) - 127;
          const float mx_s = mxa * c2;
          if (j == 0) {
            m_ref = mx_s;
            lv_ref = lv;
          } else {
            if (mx_s - m_ref > RefMax<F8>::kLazy) {
              alpha = fast_exp2(m_ref - mx_s);
              l_run *= alpha;
              m_ref = mx_s;
              moved = true;
            }
            if (lv > lv_ref) {                             // the same for every row of the tile
              const int up = lv - lv_ref;
              alpha *= up > 126 ? 0.f : __int_as_float((127 - up) << 23);
              lv_ref = lv;
              moved = true;
            }
          }
          neg = RefMax<F8>::kShift - m_ref;
          const int d = min(lv_ref - lv, 64);
          neg_tile = neg - (float)d;
          l_gain = __int_as_float((127 + d) << 23);
        } else if (j == 0) {
          m_ref = mxa;
          neg = __fmul_rn(-mxa, c2) + RefMax<F8>::kShift;
        } else if ((mxa - m_ref) * c2 > RefMax<F8>::kLazy) {
          const float neg_new = __fmul_rn(-mxa, c2) + RefMax<F8>::kShift;
          alpha = fast_exp2(__fsub_rn(neg_new, neg));
          l_run *= alpha;
          m_ref = mxa;
          neg = neg_new;
          moved = true;
        }
        if (__any_sync(0xffffffffu, moved)) {
          // Rare: the reference maximum of a row moved, so what O_i holds of that row is rescaled before the
          // next product adds to it; each of the row's two threads takes half of the head dimension.
          // PV_i(j-1) is commit number s_cnt - 1 on o_full[i].
          if (!(alive = wait_bar(&o_full[i], (s_cnt - 1) & 1, dl))) break;
          tc_fence_after();
          if ((tid & 31) == 0) atomicAdd(p.work + 2, 1u);      // diagnostic count of warp-level rescale events
#pragma unroll 1
          for (int c = 0; c < D / 64; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + half * (D / 2) + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
            tmem_st32(tO + half * (D / 2) + c * 32, o);
          }
          tmem_wait_st();
          tc_fence_before();
        }
        // ---- P = 2^(c2 * (S - m_ref)) for this thread's 64 keys
        const uint64_t negx2 = TS ? pack2(neg_tile, neg_tile) : pack2(neg, neg);
        uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
        uint32_t pk0[F8 ? 8 : 16], pk1[F8 ? 8 : 16];
        if constexpr (F8) {
          if (half == 0) {
            exp_chunk_f8<Mix::kLower>(s[0], c2x2, negx2, pk0, sum_a, sum_b);
            exp_chunk_f8<Mix::kLower>(s[1], c2x2, negx2, pk1, sum_a, sum_b);
          } else {
            exp_chunk_f8<Mix::kUpper>(s[0], c2x2, negx2, pk0, sum_a, sum_b);
            exp_chunk_f8<Mix::kUpper>(s[1], c2x2, negx2, pk1, sum_a, sum_b);
          }
        } else {
          if (half == 0) {
            exp_chunk<Mix::kLower>(s[0], c2x2, negx2, pk0, sum_a, sum_b);
            exp_chunk<Mix::kLower>(s[1], c2x2, negx2, pk1, sum_a, sum_b);
          } else {
            exp_chunk<Mix::kUpper>(s[0], c2x2, negx2, pk0, sum_a, sum_b);
            exp_chunk<Mix::kUpper>(s[1], c2x2, negx2, pk1, sum_a, sum_b);
          }
        }
        {
          float a0, a1, b0, b1;
          unpack2(sum_a, a0, a1);
          unpack2(sum_b, b0, b1);
          if constexpr (TS) l_run += ((a0 + a1) + (b0 + b1)) * l_gain;
          else l_run += (a0 + a1) + (b0 + b1);
        }
        // the previous P of this lane must have been consumed: its product is commit number s_cnt - 1 on o_full
        if (s_cnt > 0) {
          if (!(alive = wait_bar(&o_full[i], (s_cnt - 1) & 1, dl))) break;
          tc_fence_after();
        }
        ++s_cnt;
        if constexpr (F8) {
          tmem_st8(tP, pk0);
          tmem_st8(tP + 8, pk1);
        } else {
          tmem_st16(tP, pk0);
          tmem_st16(tP + 16, pk1);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&p_ready[i]);
      }
      if (!alive) break;
      // ---- epilogue: the lower-half thread of a row adds the upper half's share of the row sum, waits for
      // the last product, normalises and stores the row (the next item's first arrival on p_ready comes
      // after these TMEM reads, which is what lets the issuer overwrite O_i then)
      if (half == 1) {
        s_rowsum[i * 128 + row] = l_run;
        mbar_arrive(&sum_ready[i]);
        if (it.split && i == 1) {                        // lane 1 of a split tile: O_1 is read by lane 0's threads
          alive = wait_bar(merge_done, split_cnt & 1, dl);
          ++split_cnt;
        }
        continue;
      }
      if (!(alive = wait_bar(&sum_ready[i], item_cnt & 1, dl))) break;
      ++item_cnt;
      l_run += s_rowsum[i * 128 + row];
      pv_cnt += my_nk;
      if (!(alive = wait_bar(&o_full[i], (pv_cnt - 1) & 1, dl))) break;
      tc_fence_after();
      // A split tile: both lanes hold a partial result of the SAME rows over disjoint keys, each relative to its
      // own reference maximum.  Lane 1 publishes (-m*c2, l) and waits until lane 0 has folded O_1 into its output.
      float w0 = 1.f, w1 = 0.f;                      // weights of O_0 and O_1 in the merged numerator
      if (it.split) {
        const uint32_t spar = split_cnt & 1;
        ++split_cnt;
        if (i == 1) {
          s_merge[row] = neg;
          s_merge[128 + row] = l_run;
          if (TS && row == 0) s_merge[256] = (float)lv_ref;
          tc_fence_before();
          mbar_arrive(lane1_done);
          alive = wait_bar(merge_done, spar, dl);
          if (!alive) break;
          continue;
        }
        if (!(alive = wait_bar(lane1_done, spar, dl))) break;
        tc_fence_after();
        const float neg1 = s_merge[row], l1 = s_merge[128 + row];
        const float negm = fminf(neg, neg1);         // the larger of the two reference maxima
        w0 = fast_exp2(negm - neg);                  // 2^((m_0 - m) c2) <= 1: rebases lane 0's sums to the common maximum
        w1 = fast_exp2(negm - neg1);
        l_run = l_run * w0 + l1 * w1;
        neg = negm;
        if constexpr (TS) {                          // the two partial numerators are relative to their own V scales
          const int lv1 = (int)s_merge[256];
          const int top = max(lv_ref, lv1);
          w0 *= lv_ref == top ? 1.f : (top - lv_ref > 126 ? 0.f : __int_as_float((127 - (top - lv_ref)) << 23));
          w1 *= lv1 == top ? 1.f : (top - lv1 > 126 ? 0.f : __int_as_float((127 - (top - lv1)) << 23));
          lv_ref = top;
        }
      }
      const int grow = my_tile * kTileM + row;
      const AttnProblem& pr = p.prob[my_head / p.heads];
      const int head = my_head % p.heads;
      // 8-bit: V's scale of this head, or, with tile scales, the scale O ended up relative to
      const float inv = TS ? __int_as_float((127 + lv_ref) << 23) / l_run
                           : (F8 ? __ldg(pr.v_descale + head) / l_run : 1.f / l_run);
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
