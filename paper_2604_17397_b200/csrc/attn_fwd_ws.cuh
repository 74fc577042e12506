// Warp-specialised, persistent block-attention kernel (included by attn_fwd.cu after the common
// definitions).  One CTA per SM; a work item is a pair of 128-row query tiles of one head that
// share every K/V tile, or the single last tile of a head when the tile count is odd.
//
//   warps 0-3   softmax of query tile 0 (one thread per row)      \  S, P and O live in tensor memory:
//   warps 4-7   softmax of query tile 1                            >  S0 S1 O0 O1 = 4 x 128 columns
//   warps 8-11  correction: rescales O when a row maximum moved   /
//   warp  12    TMA producer (one lane): Q tiles, then the K/V ring
//   warp  13    MMA issuer (one lane): S_i = Q_i K^T, O_i += P_i V
//   warps 14-15 idle
//
// Tensor-pipe order per key tile j:  PV_0(j) QK_0(j+1) PV_1(j) QK_1(j+1); while the pipe works for
// tile 1 the softmax warps of tile 0 turn S_0(j+1) into P_0(j+1), and vice versa.  The running row
// maximum is only raised when it grew by more than 2^8 in the exp2 domain, so O is rarely rescaled
// and the correction warps stay off the critical path; the final 1/l normalisation and the store
// are done by the softmax warps themselves, which own the same TMEM lanes.
#pragma once

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
  static constexpr int kMisc = kBars + kNumBars * 8;                // tmem slot, abort flag
  static constexpr int kTotal = kMisc + 16;
  static constexpr int kDynamic = kTotal + 1024;
  static constexpr int kThreads = 512;
  static constexpr uint32_t kTmemCols = 512;
  static_assert(kDynamic <= 232448, "shared memory budget");
};

struct WsItem {
  int head, tile0, lanes;
};

// Static schedule: virtual item v < num_pairs is pair v; each later v holds up to two single tiles
// (a single costs about half a pair, so two of them balance one pair).
struct WsSchedule {
  int tiles, pairs_per_head, num_pairs, num_singles, num_virtual;
  __host__ __device__ WsSchedule(int tokens, int heads) {
    tiles = (tokens + kTileM - 1) / kTileM;
    pairs_per_head = tiles / 2;
    num_pairs = pairs_per_head * heads;
    num_singles = (tiles & 1) ? heads : 0;
    num_virtual = num_pairs + (num_singles + 1) / 2;
  }
  __device__ bool get(int v, int e, WsItem& it) const {
    if (v < num_pairs) {
      if (e > 0) return false;
      it.head = v / pairs_per_head;
      it.tile0 = 2 * (v - it.head * pairs_per_head);
      it.lanes = 2;
      return true;
    }
    const int s = 2 * (v - num_pairs) + e;
    if (e > 1 || s >= num_singles) return false;
    it.head = s;
    it.tile0 = tiles - 1;
    it.lanes = 1;
    return true;
  }
};

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
  uint64_t* p_full = bars + 6;        // [2] softmax -> MMA (128 arrivals)
  uint64_t* sm2corr = bars + 8;       // [2] softmax -> correction (128 arrivals)
  uint64_t* o_scaled = bars + 10;     // [2] correction -> MMA (128 arrivals)
  uint64_t* o_full = bars + 12;       // [2] MMA -> correction / softmax epilogue
  uint64_t* o_free = bars + 14;       // [2] softmax epilogue -> MMA (128 arrivals)
  uint64_t* kv_full = bars + 16;      // [kStages]
  uint64_t* kv_empty = kv_full + C::kStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::kMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1);
      mbar_init(&q_empty[i], 1);
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[i], 128);
      mbar_init(&sm2corr[i], 128);
      mbar_init(&o_scaled[i], 128);
      mbar_init(&o_full[i], 1);
      mbar_init(&o_free[i], 128);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&kv_full[s], 1);
      mbar_init(&kv_empty[s], 1);
    }
    *abort_flag = 0;
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
  WaitCtx wc{abort_flag, p.work + 1, globaltimer_ns()};
  const WsSchedule sched(p.tokens, p.heads);
  int ntiles_k = 0;
  for (int s = 0; s < p.nseg; ++s) ntiles_k += (p.seg_len[s] + kTileN - 1) / kTileN;

  if (warp >= 12) {
    // ================= producer / issuer warps: few registers ==================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;");
    if (warp == 12 && lane == 0) {
      // ---- TMA producer -------------------------------------------------------------------
      uint32_t q_cnt[2] = {0, 0}, kv_cnt = 0;
      bool alive = true;
      for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
        WsItem it;
        for (int e = 0; sched.get(v, e, it) && alive; ++e) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i >= it.lanes || !alive) break;
            if (!(alive = wait_bar(&q_empty[i], (q_cnt[i] & 1) ^ 1, wc))) break;
            ++q_cnt[i];
            mbar_expect_tx(&q_full[i], C::kTileBytes);
            for (int h = 0; h < C::kHalves; ++h)
              tma_load_3d(smem + C::kQ + i * C::kTileBytes + h * C::kPanelBytes, &p.q_map, &q_full[i], h * 64,
                          (it.tile0 + i) * kTileM, it.head);
          }
          for (int seg = 0; seg < p.nseg && alive; ++seg) {
            const int nt = (p.seg_len[seg] + kTileN - 1) / kTileN;
            for (int kt = 0; kt < nt && alive; ++kt) {
              for (int kv = 0; kv < 2; ++kv) {
                const uint32_t st = kv_cnt % C::kStages, round = kv_cnt / C::kStages;
                if (!(alive = wait_bar(&kv_empty[st], (round & 1) ^ 1, wc))) break;
                ++kv_cnt;
                mbar_expect_tx(&kv_full[st], C::kTileBytes);
                const CUtensorMap* m = kv ? &p.v_map[seg] : &p.k_map[seg];
                for (int h = 0; h < C::kHalves; ++h)
                  tma_load_3d(smem + C::kKV + st * C::kTileBytes + h * C::kPanelBytes, m, &kv_full[st], h * 64,
                              kt * kTileN, it.head);
              }
            }
          }
        }
      }
      // Drain: every load issued above lands in this CTA's shared memory; do not exit under them.
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (q_cnt[i] > 0)
          for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(&q_full[i], (q_cnt[i] - 1) & 1); ++spin) {}
      const uint32_t issued = kv_cnt;
      for (uint32_t n = issued > (uint32_t)C::kStages ? issued - C::kStages : 0; n < issued; ++n) {
        const uint32_t st = n % C::kStages, round = n / C::kStages;
        for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(&kv_full[st], round & 1); ++spin) {}
      }
    } else if (warp == 13 && lane == 0) {
      // ---- MMA issuer ---------------------------------------------------------------------
      constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kTileN, false);
      constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, D, true);
      const uint32_t sQ = smem_u32(smem + C::kQ), sKV = smem_u32(smem + C::kKV);
      const uint32_t tS[2] = {tmem_base, tmem_base + 128};
      const uint32_t tO[2] = {tmem_base + 256, tmem_base + 384};
      uint32_t q_cnt[2] = {0, 0}, kv_cnt = 0, p_cnt[2] = {0, 0}, os_cnt[2] = {0, 0}, of_cnt[2] = {0, 0};
      bool alive = true;

      auto issue_qk = [&](int i, uint32_t st) {
        const uint32_t a0 = sQ + i * C::kTileBytes, b0 = sKV + st * C::kTileBytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * C::kPanelBytes + (kk & 3) * 32;
          mma_ss(tS[i], smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(b0 + off, 16, 1024), kIdescQK, kk > 0);
        }
      };
      auto issue_pv = [&](int i, uint32_t st, bool accumulate) {
        const uint32_t b0 = sKV + st * C::kTileBytes;
#pragma unroll
        for (int kk = 0; kk < kTileN / 16; ++kk)
          mma_ts(tO[i], tS[i] + kk * 8, smem_desc_sw128(b0 + kk * 2048, C::kPanelBytes, 1024), kIdescPV,
                 (accumulate || kk > 0) ? 1u : 0u);
      };

      for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
        WsItem it;
        for (int e = 0; sched.get(v, e, it) && alive; ++e) {
          const int nl = it.lanes;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i >= nl || !alive) break;
            alive = wait_bar(&q_full[i], q_cnt[i] & 1, wc);
            ++q_cnt[i];
          }
          if (!alive) break;
          uint32_t stK = kv_cnt % C::kStages;
          if (!(alive = wait_bar(&kv_full[stK], (kv_cnt / C::kStages) & 1, wc))) break;
          ++kv_cnt;
          tc_fence_after();
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i >= nl) break;
            issue_qk(i, stK);
            mma_commit(&s_full[i]);
          }
          mma_commit(&kv_empty[stK]);
          for (int j = 0; j < ntiles_k && alive; ++j) {
            const uint32_t stV = kv_cnt % C::kStages;
            if (!(alive = wait_bar(&kv_full[stV], (kv_cnt / C::kStages) & 1, wc))) break;
            ++kv_cnt;
            const bool more = j + 1 < ntiles_k;
            uint32_t parK = 0;
            if (more) {
              stK = kv_cnt % C::kStages;
              parK = (kv_cnt / C::kStages) & 1;
              ++kv_cnt;
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              if (i >= nl || !alive) break;
              if (!(alive = wait_bar(&p_full[i], p_cnt[i] & 1, wc))) break;
              ++p_cnt[i];
              if (j == 0) {
                // O_i must have been read out by the epilogue of the previous item
                if (!(alive = wait_bar(&o_free[i], (of_cnt[i] & 1) ^ 1, wc))) break;
                ++of_cnt[i];
              } else {
                if (!(alive = wait_bar(&o_scaled[i], os_cnt[i] & 1, wc))) break;
                ++os_cnt[i];
              }
              tc_fence_after();
              issue_pv(i, stV, j > 0);
              mma_commit(&o_full[i]);
              if (i == nl - 1) mma_commit(&kv_empty[stV]);
              if (more) {
                if (i == 0 && !(alive = wait_bar(&kv_full[stK], parK, wc))) break;
                tc_fence_after();
                issue_qk(i, stK);
                mma_commit(&s_full[i]);
                if (i == nl - 1) mma_commit(&kv_empty[stK]);
              } else {
                mma_commit(&q_empty[i]);
              }
            }
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
    for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
      WsItem it;
      for (int e = 0; sched.get(v, e, it) && alive; ++e) {
        for (int j = 1; j < ntiles_k && alive; ++j) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            if (i >= it.lanes || !alive) break;
            if (!(alive = wait_bar(&sm2corr[i], a_cnt[i] & 1, wc))) break;
            ++a_cnt[i];
            const float alpha = s_alpha[i * 128 + row];
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
              // PV_i(j-1) is MMA number pv_cnt[i] + j - 1 on o_full[i]
              if (!(alive = wait_bar(&o_full[i], (pv_cnt[i] + j - 1) & 1, wc))) break;
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
            mbar_arrive(&o_scaled[i]);
          }
        }
#pragma unroll
        for (int i = 0; i < 2; ++i)
          if (i < it.lanes) pv_cnt[i] += ntiles_k;
      }
    }
  } else {
    // ================= softmax warps ===========================================================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 184;");
    const int i = warp >> 2;                       // query tile of this warpgroup
    const int row = tid & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + i * 128 + lane_off;
    const uint32_t tO = tmem_base + 256 + i * 128 + lane_off;
    const float c2 = p.scale_log2e;
    uint32_t s_cnt = 0, pv_cnt = 0;
    bool alive = true;
    for (int v = blockIdx.x; v < sched.num_virtual && alive; v += gridDim.x) {
      WsItem it;
      for (int e = 0; sched.get(v, e, it) && alive; ++e) {
        if (it.lanes <= i) continue;
        float m_ref = -INFINITY, l_run = 0.f;
        int j = 0;
        for (int seg = 0; seg < p.nseg && alive; ++seg) {
          const int len = p.seg_len[seg];
          const int nt = (len + kTileN - 1) / kTileN;
          for (int kt = 0; kt < nt && alive; ++kt, ++j) {
            const int valid = min(kTileN, len - kt * kTileN);
            if (!(alive = wait_bar(&s_full[i], s_cnt & 1, wc))) break;
            ++s_cnt;
            tc_fence_after();
            uint32_t s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s[c]);
            tmem_wait_ld();
            if (valid < kTileN) {
#pragma unroll
              for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int k = 0; k < 32; ++k)
                  if (c * 32 + k >= valid) s[c][k] = 0xff800000u;      // -inf
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
              for (int k = 0; k < 32; k += 4) {
                mx0 = fmax3(mx0, __uint_as_float(s[c][k]), __uint_as_float(s[c][k + 1]));
                mx1 = fmax3(mx1, __uint_as_float(s[c][k + 2]), __uint_as_float(s[c][k + 3]));
              }
            const float mx = fmaxf(mx0, mx1);
            if (j == 0) {
              m_ref = mx;
            } else {
              float alpha = 1.f;
              if ((mx - m_ref) * c2 > 8.f) {
                alpha = fast_exp2((m_ref - mx) * c2);
                m_ref = mx;
                l_run *= alpha;
              }
              s_alpha[i * 128 + row] = alpha;
              mbar_arrive(&sm2corr[i]);
            }
            const float neg = -m_ref * c2;
            float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t pk[16];
#pragma unroll
              for (int k = 0; k < 16; ++k) {
                const float p0 = fast_exp2(fmaf(__uint_as_float(s[c][2 * k]), c2, neg));
                const float p1 = fast_exp2(fmaf(__uint_as_float(s[c][2 * k + 1]), c2, neg));
                sum0 += p0;
                sum1 += p1;
                __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
                pk[k] = *reinterpret_cast<uint32_t*>(&b);
              }
              tmem_st16(tS + c * 16, pk);
            }
            l_run += sum0 + sum1;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&p_full[i]);
          }
        }
        if (!alive) break;
        // ---- epilogue: wait for the last PV of this item, normalise, store ------------------
        pv_cnt += ntiles_k;
        if (!(alive = wait_bar(&o_full[i], (pv_cnt - 1) & 1, wc))) break;
        tc_fence_after();
        const int grow = (it.tile0 + i) * kTileM + row;
        const float inv = 1.f / l_run;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + c * 32, o);
          tmem_wait_ld();
          if (grow < p.tokens) {
            uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)grow * p.heads + it.head) * D + c * 32);
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
        mbar_arrive(&o_free[i]);
        if (p.lse && grow < p.tokens)
          p.lse[(size_t)it.head * p.tokens + grow] = (m_ref * c2) * 0.6931471805599453f + logf(l_run);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, C::kTmemCols);
}
