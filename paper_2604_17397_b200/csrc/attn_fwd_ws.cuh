// Warp-specialised, persistent block-attention kernel (included by attn_fwd.cu after the common
// definitions).  One CTA per SM; a work item is a pair of 128-row query tiles ("lanes").  Usually
// the two tiles belong to one head and share every K/V tile; when the tile count of a head is odd,
// the last tiles of two heads form an item whose lanes stream their own K/V.
//
//   warps 0-3   softmax of lane 0 (one thread per row)            \  S, P and O live in tensor memory:
//   warps 4-7   softmax of lane 1                                  >  S0 S1 O0 O1 = 4 x 128 columns
//   warps 8-11  correction: rescales O when a row maximum moved   /
//   warp  12    TMA producer: Q tiles, then the K/V ring
//   warp  13    MMA issuer: S_i = Q_i K^T, O_i += P_i V
//   warps 14-15 idle
//
// Tensor-pipe order per key tile j:  PV_0(j) QK_0(j+1) PV_1(j) QK_1(j+1); while the pipe works for
// lane 1 the softmax warps of lane 0 turn S_0(j+1) into P_0(j+1), and vice versa.  The running row
// maximum is only raised when it grew by more than 2^8 in the exp2 domain, so O is rarely rescaled
// and the correction warps stay off the critical path; the final 1/l normalisation and the store
// are done by the softmax warps themselves, which own the same TMEM lanes.
//
// The issuer sits on the critical path between "P is ready" and the next S, so it waits on as few
// barriers as possible: one barrier per lane collects both the softmax threads (P stored) and the
// correction threads (O rescaled), and the K/V stages of an iteration are checked together before
// that.  The producer and issuer warps run their loops with all 32 lanes (warp-uniform control
// flow and values) and only predicate the TMA / MMA / commit instructions on one elected lane:
// descriptors and addresses then stay in uniform registers.
//
// The exponentials are the co-limiter of this kernel: a 128 x 128 tile needs 16384 of them and the
// special-function unit delivers 16 per clock per SM, the same 1024 clocks the tile's two MMAs take.
// A compile-time share of the elements can therefore be evaluated on the FMA pipe instead (range
// reduction to [0, 1) plus a cubic, relative error 2e-4, a tenth of the bf16 rounding P gets anyway).
#pragma once

#ifdef SDVG_ATTN_TRACE
__device__ long long* g_trace = nullptr;     // [5 roles][512 events][id, clock]
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

template <int D>
struct WsCfg {
  static constexpr int kHalves = D / 64;
  static constexpr int kPanelBytes = 128 * 128;
  static constexpr int kTileBytes = kHalves * kPanelBytes;          // one Q, K or V tile
  static constexpr int kStages = (D == 128) ? 5 : 8;                // K/V ring entries (K and V alternate)
  static constexpr int kQ = 0;                                      // two query tiles
  static constexpr int kKV = 2 * kTileBytes;
  static constexpr int kAlpha = kKV + kStages * kTileBytes;         // float [2][128]
  static constexpr int kBars = kAlpha + 2 * 128 * 4;
  static constexpr int kNumBars = 16 + 2 * kStages;
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
  bool dual;              // lanes stream their own K/V (different heads)
};

// Static schedule: virtual item v < num_pairs is pair v of consecutive tiles of one head; each later
// item takes the last (unpaired) tiles of two heads.  Every item costs the same, so a round-robin
// over the CTAs is balanced.
struct WsSchedule {
  int tiles, pairs_per_head, num_pairs, num_singles, num_virtual;
  __host__ __device__ WsSchedule(int tokens, int heads) {
    tiles = (tokens + kTileM - 1) / kTileM;
    pairs_per_head = tiles / 2;
    num_pairs = pairs_per_head * heads;
    num_singles = (tiles & 1) ? heads : 0;
    num_virtual = num_pairs + (num_singles + 1) / 2;
  }
  __device__ void get(int v, WsItem& it) const {
    if (v < num_pairs) {
      const int h = v / pairs_per_head;
      it.head[0] = it.head[1] = h;
      it.tile[0] = 2 * (v - h * pairs_per_head);
      it.tile[1] = it.tile[0] + 1;
      it.lanes = 2;
      it.dual = false;
    } else {
      const int s = 2 * (v - num_pairs);
      it.head[0] = s;
      it.head[1] = s + 1;
      it.tile[0] = it.tile[1] = tiles - 1;
      it.lanes = (s + 1 < num_singles) ? 2 : 1;
      it.dual = true;
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

template <int D>
__global__ void __launch_bounds__(512, 1) attn_fwd_ws_kernel(const __grid_constant__ AttnParams p) {
  using C = WsCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* s_alpha = reinterpret_cast<float*>(smem + C::kAlpha);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kBars);
  uint64_t* q_full = bars;            // [2] TMA -> MMA
  uint64_t* q_empty = bars + 2;       // [2] MMA -> TMA
  uint64_t* s_full = bars + 4;        // [2] MMA -> softmax
  uint64_t* pv_ready = bars + 6;      // [2] softmax (P stored) + correction (O rescaled) -> MMA, 256 arrivals
  uint64_t* sm2corr = bars + 8;       // [2] softmax -> correction (128 arrivals)
  uint64_t* o_full = bars + 10;       // [2] MMA -> correction / softmax epilogue
  uint64_t* kv_full = bars + 16;      // [kStages]
  uint64_t* kv_empty = kv_full + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kMisc);

  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&pv_ready[i], 256);
      mbar_init(&sm2corr[i], 128);
      mbar_init(&o_full[i], 1);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    fence_mbar_init();
    prefetch_tmap(&p.q_map);
    for (int s = 0; s < p.nseg; ++s) {
      prefetch_tmap(&p.k_map[s]);
      prefetch_tmap(&p.v_map[s]);
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
  const WsSchedule sched(p.tokens, p.heads);
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
          const CUtensorMap* m = is_v ? &p.v_map[seg] : &p.k_map[seg];
          for (int h = 0; h < C::kHalves; ++h)
            tma_load_3d(smem + C::kKV + ring.stage * C::kTileBytes + h * C::kPanelBytes, m, &kv_full[ring.stage],
                        h * 64, kt * kTileN, head);
        }
        ring.template advance<C::kStages>();
        ++kv_issued;
      };

      for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
        WsItem it;
        sched.get(v, it);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= it.lanes || !alive) break;
          if (!(alive = wait_warp(&q_empty[i], (q_cnt[i] & 1) ^ 1, dl))) break;
          ++q_cnt[i];
          if (leader) {
            mbar_expect_tx(&q_full[i], C::kTileBytes);
            for (int h = 0; h < C::kHalves; ++h)
              tma_load_3d(smem + C::kQ + i * C::kTileBytes + h * C::kPanelBytes, &p.q_map, &q_full[i], h * 64,
                          it.tile[i] * kTileM, it.head[i]);
          }
        }
        // K/V tiles in the order the issuer consumes them
        const int streams = it.dual ? it.lanes : 1;
        for (int s = 0; s < streams && alive; ++s) load_kv(false, it.head[s], 0);
        for (int j = 0; j < ntiles_k && alive; ++j)
          for (int s = 0; s < streams && alive; ++s) {
            load_kv(true, it.head[s], j);
            if (j + 1 < ntiles_k && alive) load_kv(false, it.head[s], j + 1);
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
      constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kTileN, false);
      constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, true);
      const uint32_t sQ = smem_u32(smem + C::kQ), sKV = smem_u32(smem + C::kKV);
      uint32_t q_cnt[2] = {0, 0}, pv_cnt[2] = {0, 0};
      RingPos ring;
      bool alive = true;
      SDVG_TRACE_DECL(blockIdx.x == 0 && leader)

      // S_i = Q_i K^T into TMEM columns [128 i, 128 i + 128)
      auto issue_qk = [&](int i, uint32_t st) {
        const uint32_t a0 = sQ + i * C::kTileBytes, b0 = sKV + st * C::kTileBytes;
        const uint32_t d = tmem_base + i * 128;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * C::kPanelBytes + (kk & 3) * 32;
          mma_ss(d, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(b0 + off, 16, 1024), kIdescQK, kk > 0);
        }
      };
      // O_i (+)= P_i V with P_i read from the first 64 columns of S_i
      auto issue_pv = [&](int i, uint32_t st, bool accumulate) {
        const uint32_t b0 = sKV + st * C::kTileBytes;
        const uint32_t d = tmem_base + 256 + i * 128, a = tmem_base + i * 128;
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(d, a + kk * 8, smem_desc_sw128(b0 + kk * 2048, C::kPanelBytes, 1024), kIdescPV,
                 (accumulate || kk > 0) ? 1u : 0u);
      };

      for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
        WsItem it;
        sched.get(v, it);
        const int nl = it.lanes;
        const bool dual = it.dual;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= nl || !alive) break;
          alive = wait_warp(&q_full[i], q_cnt[i] & 1, dl);
          ++q_cnt[i];
        }
        if (!alive) break;
        // ---- prologue: S_i(0) ------------------------------------------------------------------
        uint32_t stK = 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= nl || !alive) break;
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
        // ---- main loop -------------------------------------------------------------------------
        for (int j = 0; j < ntiles_k && alive; ++j) {
          const bool more = j + 1 < ntiles_k;
          uint32_t stV = 0;
          SDVG_TRACE(2, 100 + j);
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i >= nl || !alive) break;
            const bool own = (i == 0) || dual;
            const bool last_user = dual || (i == nl - 1);
            if (own) {
              // V_j and K_(j+1) are normally in place long before they are needed: check both first
              stV = ring.stage;
              const uint32_t phV = ring.phase;
              ring.template advance<C::kStages>();
              bool ok = mbar_try_wait(&kv_full[stV], phV);
              uint32_t phK = 0;
              if (more) {
                stK = ring.stage;
                phK = ring.phase;
                ring.template advance<C::kStages>();
                ok = mbar_try_wait(&kv_full[stK], phK) && ok;
              }
              if (!__all_sync(0xffffffffu, ok)) {
                if (!(alive = wait_warp(&kv_full[stV], phV, dl))) break;
                if (more && !(alive = wait_warp(&kv_full[stK], phK, dl))) break;
              }
            }
            SDVG_TRACE(2, 1000 + i * 1000 + j);
            // P_i(j) stored and O_i rescaled (for j = 0: O_i read out by the previous epilogue)
            if (!(alive = wait_warp(&pv_ready[i], pv_cnt[i] & 1, dl))) break;
            ++pv_cnt[i];
            SDVG_TRACE(2, 3000 + i * 1000 + j);
            tc_fence_after();
            if (leader) {
              issue_pv(i, stV, j > 0);
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
            SDVG_TRACE(2, 9000 + i * 1000 + j);
          }
        }
      }
    }
  } else if (warp >= 8) {
    // ================= correction warps ========================================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
    const int row = tid - 256;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tO[2] = {tmem_base + 256 + lane_off, tmem_base + 384 + lane_off};
    uint32_t a_cnt[2] = {0, 0}, pv_cnt[2] = {0, 0};
    bool alive = true;
    SDVG_TRACE_DECL(blockIdx.x == 0 && tid == 256)
    for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
      WsItem it;
      sched.get(v, it);
      for (int j = 0; j < ntiles_k && alive; ++j) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i >= it.lanes || !alive) break;
          if (j == 0) {
            // Nothing to rescale yet.  The arrival below must not fall into the previous phase of
            // pv_ready (the last key tile of the previous item), so that phase has to be over.
            if (pv_cnt[i] > 0 && !(alive = wait_bar(&pv_ready[i], (pv_cnt[i] - 1) & 1, dl))) break;
          } else {
            if (!(alive = wait_bar(&sm2corr[i], a_cnt[i] & 1, dl))) break;
            ++a_cnt[i];
            const float alpha = s_alpha[i * 128 + row];
            SDVG_TRACE(3, 1000 * i + j);
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
              // PV_i(j-1) is MMA number pv_cnt[i] - 1 on o_full[i]
              if (!(alive = wait_bar(&o_full[i], (pv_cnt[i] - 1) & 1, dl))) break;
              tc_fence_after();
#pragma unroll
              for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tO[i] + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                tmem_st32(tO[i] + c * 32, o);
              }
              tmem_wait_st();
              tc_fence_before();
            }
          }
          SDVG_TRACE(3, 20000 + 1000 * i + j);
          mbar_arrive(&pv_ready[i]);
          ++pv_cnt[i];
        }
      }
    }
  } else {
    // ================= softmax warps ===========================================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 184;");
    const int i = warp >> 2;                       // lane (query tile) of this warpgroup
    const int row = tid & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + i * 128 + lane_off;
    const uint32_t tO = tmem_base + 256 + i * 128 + lane_off;
    const float c2 = p.scale_log2e;
    const uint64_t c2x2 = pack2(c2, c2);
    uint32_t s_cnt = 0, pv_cnt = 0;
    bool alive = true;
    SDVG_TRACE_DECL(blockIdx.x == 0 && row == 0)
    for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
      WsItem it;
      sched.get(v, it);
      if (it.lanes <= i) continue;
      float m_ref = -INFINITY, l_run = 0.f;
      int j = 0;
      for (int seg = 0; seg < p.nseg && alive; ++seg) {
        const int len = p.seg_len[seg];
        const int nt = (len + kTileN - 1) / kTileN;
        for (int kt = 0; kt < nt && alive; ++kt, ++j) {
          const int valid = min(kTileN, len - kt * kTileN);
          SDVG_TRACE(i, 0 + j);
          if (!(alive = wait_bar(&s_full[i], s_cnt & 1, dl))) break;
          SDVG_TRACE(i, 1000 + j);
          ++s_cnt;
          tc_fence_after();
          // ---- row maximum; the second half of S streams in while the first is reduced -----
          uint32_t s[4][32];
          tmem_ld32(tS, s[0]);
          tmem_ld32(tS + 32, s[1]);
          tmem_wait_ld();
          tmem_ld32(tS + 64, s[2]);
          tmem_ld32(tS + 96, s[3]);
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          if (valid < kTileN) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int k = 0; k < 32; ++k)
                if (c * 32 + k >= valid) s[c][k] = 0xff800000u;      // -inf
          }
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int k = 0; k < 32; k += 8) {
#pragma unroll
              for (int u = 0; u < 4; ++u)
                mx[u] = fmax3(mx[u], __uint_as_float(s[c][k + 2 * u]), __uint_as_float(s[c][k + 2 * u + 1]));
            }
          tmem_wait_ld();
          SDVG_TRACE(i, 2000 + j);
          if (valid < kTileN) {
#pragma unroll
            for (int c = 2; c < 4; ++c)
#pragma unroll
              for (int k = 0; k < 32; ++k)
                if (c * 32 + k >= valid) s[c][k] = 0xff800000u;
          }
#pragma unroll
          for (int c = 2; c < 4; ++c)
#pragma unroll
            for (int k = 0; k < 32; k += 8) {
#pragma unroll
              for (int u = 0; u < 4; ++u)
                mx[u] = fmax3(mx[u], __uint_as_float(s[c][k + 2 * u]), __uint_as_float(s[c][k + 2 * u + 1]));
            }
          const float mxa = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
          if (j == 0) {
            m_ref = mxa;
          } else {
            float alpha = 1.f;
            if ((mxa - m_ref) * c2 > 8.f) {
              alpha = fast_exp2((m_ref - mxa) * c2);
              m_ref = mxa;
              l_run *= alpha;
            }
            s_alpha[i * 128 + row] = alpha;
            mbar_arrive(&sm2corr[i]);
          }
          SDVG_TRACE(i, 3000 + j);
          // ---- P = 2^(c2 * (S - m_ref)), bf16, written back over S ---------------------------
          const float neg = -m_ref * c2;
          const uint64_t negx2 = pack2(neg, neg);
          uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const uint64_t x2 =
                  fma2(pack2(__uint_as_float(s[c][2 * k]), __uint_as_float(s[c][2 * k + 1])), c2x2, negx2);
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
            tmem_st16(tS + c * 16, pk);
          }
          {
            float a0, a1, b0, b1;
            unpack2(sum_a, a0, a1);
            unpack2(sum_b, b0, b1);
            l_run += (a0 + a1) + (b0 + b1);
          }
          SDVG_TRACE(i, 4000 + j);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&pv_ready[i]);
          SDVG_TRACE(i, 5000 + j);
        }
      }
      if (!alive) break;
      // ---- epilogue: wait for the last PV of this item, normalise, store ------------------
      // (the next item's first arrival on pv_ready comes after these TMEM reads, which is what
      // lets the issuer overwrite O_i then)
      pv_cnt += ntiles_k;
      if (!(alive = wait_bar(&o_full[i], (pv_cnt - 1) & 1, dl))) break;
      tc_fence_after();
      const int grow = it.tile[i] * kTileM + row;
      const int head = it.head[i];
      const float inv = 1.f / l_run;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tO + c * 32, o);
        tmem_wait_ld();
        if (grow < p.tokens) {
          uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)grow * p.heads + head) * D + c * 32);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(o[q4 * 8 + 2 * k]) * inv,
                                                       __uint_as_float(o[q4 * 8 + 2 * k + 1]) * inv);
              w[k] = *reinterpret_cast<uint32_t*>(&b);
            }
            dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      tc_fence_before();
      if (p.lse && grow < p.tokens)
        p.lse[(size_t)head * p.tokens + grow] = (m_ref * c2) * 0.6931471805599453f + logf(l_run);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, C::kTmemCols);
}
