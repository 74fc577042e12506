// 3D-RoPE, ring commit and their fusion: one streaming pass over HBM per tensor.
//
// Every thread owns one 16-byte column slice (8 bf16 = 4 rotary pairs) of one token and walks a
// group of heads with it, so the token's (frame, row, column) split and its (cos, sin) pairs are
// fetched once and reused for every head; loads of a head group are issued before the first use
// so that several 16-byte requests per thread are in flight.  Reads use the logical
// [tokens, heads, dim] layout; writes go to the logical layout and/or to the ring slot
// ([heads][slots][tokens][dim]).  Both sides move whole 16-byte vectors, 128/256 contiguous
// bytes per (token, head) row.
#include <cuda_bf16.h>

#include "sdvg_internal.h"
#include "sm100_ptx.cuh"

namespace {

constexpr int kMaxJobs = 3;
constexpr int kHeadGroup = 8;     // heads walked by one thread
constexpr int kThreads = 256;

struct TensorJob {
  const uint4* src;        // [tokens, heads, dim] bf16
  uint4* dst_logical;      // same layout, or nullptr
  uint4* dst_slot;         // points at (head 0, slot, token 0): head stride = slots*tokens*dim, or nullptr
  int rope;                // rotate pairs (q, k) or copy (v)
  // 8-bit variant: the (rotated, bf16-rounded) values times inv_scale[head] as E4M3 bytes, 8 per thread
  uint2* q8_logical;       // [tokens, heads, dim] bytes, or nullptr
  uint2* q8_slot;          // ring slot of a byte ring (same strides, counted in 8-byte units), or nullptr
  const float* inv_scale;  // [heads]
};

struct RopeCommitParams {
  TensorJob job[kMaxJobs];
  int njobs;
  int tokens, heads;
  int grid_hw, grid_w;     // grid_h*grid_w and grid_w of the latent grid
  int frame_offset;
  int pairs_f, pairs_h;    // pair split: [0,pf) frame, [pf,pf+ph) row, rest column
  int tab_h_off, tab_w_off;  // float offsets of the row and column sub-tables
  long long slot_head_stride_vec;  // 16-byte vectors between consecutive heads in the ring buffer
  const float2* tab;
};

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// One pair: re' = fl(fl(re*c) - fl(im*s)), im' = fl(fl(re*s) + fl(im*c)); RNE pack to bf16x2.
__device__ __forceinline__ uint32_t rotate_pair(uint32_t w, float2 cs) {
  float re = bf16_lo(w), im = bf16_hi(w);
  float r0 = __fsub_rn(__fmul_rn(re, cs.x), __fmul_rn(im, cs.y));
  float r1 = __fadd_rn(__fmul_rn(re, cs.y), __fmul_rn(im, cs.x));
  __nv_bfloat162 p = __floats2bfloat162_rn(r0, r1);
  return *reinterpret_cast<uint32_t*>(&p);
}

// two bf16 pairs -> four E4M3 bytes, element order kept
__device__ __forceinline__ uint32_t quant4(uint32_t w0, uint32_t w1, float inv) {
  return sm100::pack_e4m3x4(__fmul_rn(bf16_lo(w0), inv), __fmul_rn(bf16_hi(w0), inv), __fmul_rn(bf16_lo(w1), inv),
                            __fmul_rn(bf16_hi(w1), inv));
}

template <int D, bool Q8 = false>
__global__ void __launch_bounds__(kThreads) rope_commit_kernel(const __grid_constant__ RopeCommitParams p) {
  constexpr int VPR = D / 8;                       // 16-byte vectors per (token, head) row
  const TensorJob job = p.job[blockIdx.z];
  const int h0 = blockIdx.y * kHeadGroup;
  const int nh = min(kHeadGroup, p.heads - h0);
  const int total = p.tokens * VPR;
  for (int i = blockIdx.x * kThreads + threadIdx.x; i < total; i += gridDim.x * kThreads) {
    const int t = i / VPR;
    const int j = i - t * VPR;
    float2 cs[4];
    if (job.rope) {
      const int f = t / p.grid_hw;
      const int rem = t - f * p.grid_hw;
      const int y = rem / p.grid_w;
      const int x = rem - y * p.grid_w;
      const int pairs_w = D / 2 - p.pairs_f - p.pairs_h;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int pr = 4 * j + e;
        int idx;
        if (pr < p.pairs_f) idx = (p.frame_offset + f) * p.pairs_f + pr;
        else if (pr < p.pairs_f + p.pairs_h) idx = p.tab_h_off + y * p.pairs_h + (pr - p.pairs_f);
        else idx = p.tab_w_off + x * pairs_w + (pr - p.pairs_f - p.pairs_h);
        cs[e] = __ldg(p.tab + idx);
      }
    }
    const size_t row0 = ((size_t)t * p.heads + h0) * VPR + j;     // vector index of (t, h0, j)
    uint4 v[kHeadGroup];
#pragma unroll
    for (int g = 0; g < kHeadGroup; ++g)
      if (g < nh) v[g] = __ldcs(job.src + row0 + (size_t)g * VPR);
#pragma unroll
    for (int g = 0; g < kHeadGroup; ++g) {
      if (g < nh) {
        uint4 w = v[g];
        if (job.rope) {
          w.x = rotate_pair(w.x, cs[0]);
          w.y = rotate_pair(w.y, cs[1]);
          w.z = rotate_pair(w.z, cs[2]);
          w.w = rotate_pair(w.w, cs[3]);
        }
        if (job.dst_logical) __stcs(job.dst_logical + row0 + (size_t)g * VPR, w);
        if (job.dst_slot)
          job.dst_slot[(size_t)(h0 + g) * p.slot_head_stride_vec + (size_t)t * VPR + j] = w;
        if constexpr (Q8) {
          const float inv = __ldg(job.inv_scale + h0 + g);
          const uint2 o = make_uint2(quant4(w.x, w.y, inv), quant4(w.z, w.w, inv));
          if (job.q8_logical) job.q8_logical[row0 + (size_t)g * VPR] = o;
          if (job.q8_slot) job.q8_slot[(size_t)(h0 + g) * p.slot_head_stride_vec + (size_t)t * VPR + j] = o;
        }
      }
    }
  }
}

// Ring slot -> logical layout (accessor used to inspect the cache).
template <int D>
__global__ void __launch_bounds__(kThreads) slot_read_kernel(const uint4* __restrict__ slot_base,
                                                              uint4* __restrict__ dst, int tokens, int heads,
                                                              long long slot_head_stride_vec) {
  constexpr int VPR = D / 8;
  const long long total = (long long)tokens * heads * VPR;
  for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < total;
       i += (long long)gridDim.x * kThreads) {
    const int j = (int)(i % VPR);
    const long long row = i / VPR;
    const int h = (int)(row % heads);
    const long long t = row / heads;
    dst[i] = slot_base[(long long)h * slot_head_stride_vec + t * VPR + j];
  }
}

// ---- 8-bit ring with one power-of-two scale per tile of 128 tokens and head ---------------------------------
// A CTA owns one (tile, head) of one tensor: 128 rows of 256 bytes, 8 x 16 bytes per thread held in registers
// between the two passes a data-dependent scale needs (largest magnitude, then quantise).  The rows are rotated
// first where the tensor is q or k, rounded to bf16 exactly as the bf16 path rounds them.  HBM: 2 bytes read,
// 1 written per element.
struct TileQuantJob {
  const uint4* src;             // bf16 [tokens, heads, 128]
  uint2* dst;                   // codes; (token, head) row at dst + token * token_stride + head * head_stride (8-byte units)
  long long token_stride, head_stride;
  float* scale;                 // scale of (head, tile) at scale[head * scale_head_stride + tile]
  long long scale_head_stride;
  int rope;
};

struct TileQuantParams {
  RopeCommitParams r;           // token count, head count and the rotary fields; its own jobs are unused
  TileQuantJob job[kMaxJobs];
};

// The smallest e in [-126, 120] with amax <= 448 * 2^e (448 = 0.875 * 2^9); amax is >= 0 or +inf, never NaN.
__device__ __forceinline__ int tile_scale_exponent(float amax) {
  if (!(amax < __int_as_float(0x7f800000))) return 120;
  if (amax == 0.f) return -126;
  int x;
  const float m = frexpf(amax, &x);               // amax = m * 2^x, m in [0.5, 1)
  const int e = x - 9 + (m > 0.875f ? 1 : 0);
  return e < -126 ? -126 : (e > 120 ? 120 : e);
}

// running maximum of |x| over bf16 pairs, two at a time; the maximum drops a NaN operand, so NaN elements do not set
// the scale (an accumulator that starts at zero never becomes NaN)
__device__ __forceinline__ uint32_t abs_max2(uint32_t acc, uint32_t w) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(acc), "r"(w & 0x7fff7fffu));
  return r;
}

constexpr int kTileHeads = 4;      // heads a CTA walks with the same 128 tokens (their rotary factors stay in registers)
constexpr int kTileThreads = 512;

// ROPE: some job of the launch rotates (q, k); the thread then keeps the (cos, sin) pairs of its rows in registers
// for all heads it walks, and two CTAs per SM overlap each other's loads; without them the registers go to the
// next head's vectors, requested before the current head is reduced and stored.
template <bool ROPE>
__global__ void __launch_bounds__(kTileThreads, 2) tile_quant_kernel(const __grid_constant__ TileQuantParams p) {
  constexpr int VPR = 16;                          // 16-byte vectors per (token, head) row of 128 bf16
  constexpr int kRowStep = kTileThreads / VPR;     // 32 rows per pass
  constexpr int kRows = 128 / kRowStep;            // rows per thread: 4
  constexpr int kWarps = kTileThreads / 32;
  const TileQuantJob job = p.job[blockIdx.z];
  const int tile = blockIdx.x, h0 = blockIdx.y * kTileHeads;
  const int nh = min(kTileHeads, p.r.heads - h0);
  const int j = threadIdx.x & (VPR - 1), r0 = threadIdx.x / VPR;
  const int t0 = tile * 128 + r0;                  // this thread's rows are t0 + i * kRowStep
  __shared__ float s_max[2][kWarps];
  float2 cs[ROPE ? kRows : 1][4];
  if (ROPE && job.rope) {
    const int pairs_w = 64 - p.r.pairs_f - p.r.pairs_h;
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
      const int t = min(t0 + i * kRowStep, p.r.tokens - 1);
      const int f = t / p.r.grid_hw;
      const int rem = t - f * p.r.grid_hw;
      const int y = rem / p.r.grid_w;
      const int x = rem - y * p.r.grid_w;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int pr = 4 * j + e;
        int idx;
        if (pr < p.r.pairs_f) idx = (p.r.frame_offset + f) * p.r.pairs_f + pr;
        else if (pr < p.r.pairs_f + p.r.pairs_h) idx = p.r.tab_h_off + y * p.r.pairs_h + (pr - p.r.pairs_f);
        else idx = p.r.tab_w_off + x * pairs_w + (pr - p.r.pairs_f - p.r.pairs_h);
        cs[i][e] = __ldg(p.r.tab + idx);
      }
    }
  }
  auto load = [&](uint4 (&v)[kRows], int h) {
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
      const int t = t0 + i * kRowStep;
      v[i] = t < p.r.tokens ? __ldcs(job.src + ((size_t)t * p.r.heads + h) * VPR + j) : make_uint4(0, 0, 0, 0);
    }
  };
  uint4 v[kRows], nxt[ROPE ? 1 : kRows];
  if (!ROPE) load(v, h0);
#pragma unroll 1
  for (int g = 0; g < nh; ++g) {
    const int h = h0 + g;
    if constexpr (ROPE) load(v, h);
    else if (g + 1 < nh) load(nxt, h + 1);
    if (ROPE && job.rope) {
#pragma unroll
      for (int i = 0; i < kRows; ++i) {
        v[i].x = rotate_pair(v[i].x, cs[i][0]);
        v[i].y = rotate_pair(v[i].y, cs[i][1]);
        v[i].z = rotate_pair(v[i].z, cs[i][2]);
        v[i].w = rotate_pair(v[i].w, cs[i][3]);
      }
    }
    uint32_t am2 = 0;
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
      am2 = abs_max2(am2, v[i].x);
      am2 = abs_max2(am2, v[i].y);
      am2 = abs_max2(am2, v[i].z);
      am2 = abs_max2(am2, v[i].w);
    }
    float amax = fmaxf(bf16_lo(am2), bf16_hi(am2));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) s_max[g & 1][threadIdx.x >> 5] = amax;
    __syncthreads();                               // one barrier per head: the partial maxima alternate between two rows
    amax = s_max[g & 1][threadIdx.x & (kWarps - 1)];
#pragma unroll
    for (int o = kWarps / 2; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const int e = tile_scale_exponent(amax);
    const float inv = __int_as_float((127 - e) << 23);          // 2^-e, exact; -e is in [-120, 126]
    if (threadIdx.x == 0) job.scale[(size_t)h * job.scale_head_stride + tile] = __int_as_float((127 + e) << 23);
#pragma unroll
    for (int i = 0; i < kRows; ++i) {
      const int t = t0 + i * kRowStep;
      if (t < p.r.tokens)
        job.dst[(size_t)t * job.token_stride + (size_t)h * job.head_stride + j] =
            make_uint2(quant4(v[i].x, v[i].y, inv), quant4(v[i].z, v[i].w, inv));
    }
    if constexpr (!ROPE) {
#pragma unroll
      for (int i = 0; i < kRows; ++i) v[i] = nxt[i];
    }
  }
}

int launch_tile_quant(const TileQuantParams& p, int njobs, cudaStream_t stream) {
  const int tiles = sdvg::scale_tiles(p.r.tokens);
  const int groups = (p.r.heads + kTileHeads - 1) / kTileHeads;
  if (groups > 65535 || njobs > kMaxJobs) return SDVG_ERR_BAD_SHAPE;
  bool rope = false;
  for (int i = 0; i < njobs; ++i) rope = rope || p.job[i].rope;
  const dim3 grid(tiles, groups, njobs);
  if (rope) tile_quant_kernel<true><<<grid, kTileThreads, 0, stream>>>(p);
  else tile_quant_kernel<false><<<grid, kTileThreads, 0, stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}

// Ring jobs of a tile-scaled commit into `slot`: codes into the byte rings, scales into the cache's scale arrays.
void tile_commit_jobs(TileQuantParams& p, int& n, const sdvg_cache* c, int slot, const void* k, const void* v, int rope_k) {
  const int tiles = sdvg::scale_tiles(c->block_tokens);
  const long long head_stride = (long long)c->slots * c->block_tokens * 16;      // 8-byte units per head of the ring
  uint2* kslot = (uint2*)c->k_buf + sdvg::slot_offset(c, 0, slot) / 8;
  uint2* vslot = (uint2*)c->v_buf + sdvg::slot_offset(c, 0, slot) / 8;
  p.job[n++] = TileQuantJob{(const uint4*)k, kslot, 16, head_stride, c->k_tile_scale + (size_t)slot * tiles,
                            (long long)c->slots * tiles, rope_k};
  p.job[n++] = TileQuantJob{(const uint4*)v, vslot, 16, head_stride, c->v_tile_scale + (size_t)slot * tiles,
                            (long long)c->slots * tiles, 0};
}

struct RopeArgs {
  int frames, grid_h, grid_w, frame_offset, tab_frames;
  const float* tab;
};

int fill_rope(RopeCommitParams& p, int head_dim, int tokens, const RopeArgs& r) {
  if (r.frames <= 0 || r.grid_h <= 0 || r.grid_w <= 0) return SDVG_ERR_BAD_SHAPE;
  if ((long long)r.frames * r.grid_h * r.grid_w != tokens) return SDVG_ERR_BAD_SHAPE;
  if (!r.tab) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(r.tab)) return SDVG_ERR_MISALIGNED;
  if (r.tab_frames <= 0) return SDVG_ERR_BAD_SHAPE;
  if (r.frame_offset < 0 || (long long)r.frame_offset + r.frames > r.tab_frames) return SDVG_ERR_BAD_STATE;
  int pf, ph, pw;
  sdvg_rope3d_pairs(head_dim, &pf, &ph, &pw);
  p.grid_hw = r.grid_h * r.grid_w;
  p.grid_w = r.grid_w;
  p.frame_offset = r.frame_offset;
  p.pairs_f = pf;
  p.pairs_h = ph;
  p.tab_h_off = r.tab_frames * pf;                 // in (cos, sin) pairs
  p.tab_w_off = p.tab_h_off + r.grid_h * ph;
  p.tab = reinterpret_cast<const float2*>(r.tab);
  return SDVG_OK;
}

int launch(RopeCommitParams& p, int head_dim, cudaStream_t stream, bool q8 = false) {
  if (p.njobs == 0) return SDVG_OK;
  const int vpr = head_dim / 8;
  const long long total = (long long)p.tokens * vpr;
  if (total * p.heads >= (1ll << 31)) return SDVG_ERR_BAD_SHAPE;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int groups = (p.heads + kHeadGroup - 1) / kHeadGroup;
  long long want = (total + kThreads - 1) / kThreads;
  // Enough blocks that a thread makes one pass at the model shapes (measured 4-5% faster than 8 blocks per SM
  // with two or three passes each); the cap only bounds the grid for very large tensors.
  long long cap = (long long)sms * 32 / (groups * p.njobs);
  if (cap < 1) cap = 1;
  const long long gx = want < cap ? want : cap;
  dim3 grid((unsigned)gx, groups, p.njobs);
  if (q8) rope_commit_kernel<128, true><<<grid, kThreads, 0, stream>>>(p);      // a byte ring has head_dim 128
  else if (head_dim == 128) rope_commit_kernel<128><<<grid, kThreads, 0, stream>>>(p);
  else rope_commit_kernel<64><<<grid, kThreads, 0, stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}

}  // namespace

extern "C" {

int sdvg_rope3d_qk(const void* q, const void* k, void* q_out, void* k_out, int tokens, int heads,
                   int head_dim, int frames, int grid_h, int grid_w, int frame_offset,
                   const float* cos_sin_tab, int tab_frames, void* stream) {
  SDVG_RANGE();
  if ((q == nullptr) != (q_out == nullptr) || (k == nullptr) != (k_out == nullptr)) return SDVG_ERR_INVALID_ARG;
  if (!q && !k) return SDVG_ERR_INVALID_ARG;
  if (tokens <= 0 || heads <= 0 || !sdvg::head_dim_ok(head_dim)) return SDVG_ERR_BAD_SHAPE;
  if (!sdvg::aligned16(q) || !sdvg::aligned16(k) || !sdvg::aligned16(q_out) || !sdvg::aligned16(k_out))
    return SDVG_ERR_MISALIGNED;
  RopeCommitParams p = {};
  p.tokens = tokens;
  p.heads = heads;
  int st = fill_rope(p, head_dim, tokens, RopeArgs{frames, grid_h, grid_w, frame_offset, tab_frames, cos_sin_tab});
  if (st != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  if (q) p.job[p.njobs++] = TensorJob{(const uint4*)q, (uint4*)q_out, nullptr, 1};
  if (k) p.job[p.njobs++] = TensorJob{(const uint4*)k, (uint4*)k_out, nullptr, 1};
  return launch(p, head_dim, (cudaStream_t)stream);
}

int sdvg_kv_commit(sdvg_cache* c, const void* k_roped, const void* v, int64_t block_index, int flags,
                   int64_t* evicted_block, void* stream) {
  SDVG_RANGE();
  if (!c || !k_roped || !v) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 2) return SDVG_ERR_BAD_SHAPE;          // an 8-bit cache takes sdvg_kv_commit_e4m3
  if (!sdvg::aligned16(k_roped) || !sdvg::aligned16(v)) return SDVG_ERR_MISALIGNED;
  int slot = 0;
  int st = sdvg::ring_begin_commit(c, block_index, flags, &slot);
  if (st != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  RopeCommitParams p = {};
  p.tokens = c->block_tokens;
  p.heads = c->heads;
  p.slot_head_stride_vec = (long long)c->slots * c->block_tokens * (c->head_dim / 8);
  uint4* kslot = (uint4*)c->k_buf + sdvg::slot_offset(c, 0, slot) / 8;
  uint4* vslot = (uint4*)c->v_buf + sdvg::slot_offset(c, 0, slot) / 8;
  p.job[p.njobs++] = TensorJob{(const uint4*)k_roped, nullptr, kslot, 0};
  p.job[p.njobs++] = TensorJob{(const uint4*)v, nullptr, vslot, 0};
  st = launch(p, c->head_dim, (cudaStream_t)stream);
  if (st != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

int sdvg_rope3d_qk_commit(sdvg_cache* c, const void* q, const void* k, const void* v, void* q_out,
                          void* k_out, int frames, int grid_h, int grid_w, int frame_offset,
                          const float* cos_sin_tab, int tab_frames, int64_t block_index, int flags,
                          int64_t* evicted_block, void* stream) {
  SDVG_RANGE();
  if (!c || !k || !v) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 2) return SDVG_ERR_BAD_SHAPE;
  if ((q == nullptr) != (q_out == nullptr)) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(q) || !sdvg::aligned16(k) || !sdvg::aligned16(v) || !sdvg::aligned16(q_out) ||
      !sdvg::aligned16(k_out))
    return SDVG_ERR_MISALIGNED;
  RopeCommitParams p = {};
  p.tokens = c->block_tokens;
  p.heads = c->heads;
  int st = fill_rope(p, c->head_dim, c->block_tokens,
                     RopeArgs{frames, grid_h, grid_w, frame_offset, tab_frames, cos_sin_tab});
  if (st != SDVG_OK) return st;
  int slot = 0;
  if ((st = sdvg::ring_begin_commit(c, block_index, flags, &slot)) != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  p.slot_head_stride_vec = (long long)c->slots * c->block_tokens * (c->head_dim / 8);
  uint4* kslot = (uint4*)c->k_buf + sdvg::slot_offset(c, 0, slot) / 8;
  uint4* vslot = (uint4*)c->v_buf + sdvg::slot_offset(c, 0, slot) / 8;
  if (q) p.job[p.njobs++] = TensorJob{(const uint4*)q, (uint4*)q_out, nullptr, 1};
  p.job[p.njobs++] = TensorJob{(const uint4*)k, (uint4*)k_out, kslot, 1};
  p.job[p.njobs++] = TensorJob{(const uint4*)v, nullptr, vslot, 0};
  st = launch(p, c->head_dim, (cudaStream_t)stream);
  if (st != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

int sdvg_rope3d_qk_commit_e4m3(sdvg_cache* c, const void* q, const void* k, const void* v, void* q8_out,
                               const float* q_inv_scale, const float* k_inv_scale, const float* v_inv_scale,
                               int frames, int grid_h, int grid_w, int frame_offset, const float* cos_sin_tab,
                               int tab_frames, int64_t block_index, int flags, int64_t* evicted_block, void* stream) {
  SDVG_RANGE();
  if (!c || !k || !v || !k_inv_scale || !v_inv_scale) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1) return SDVG_ERR_BAD_SHAPE;
  if ((q == nullptr) != (q8_out == nullptr) || (q && !q_inv_scale)) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(q) || !sdvg::aligned16(k) || !sdvg::aligned16(v) || !sdvg::aligned16(q8_out) ||
      ((reinterpret_cast<uintptr_t>(q_inv_scale) | reinterpret_cast<uintptr_t>(k_inv_scale) |
        reinterpret_cast<uintptr_t>(v_inv_scale)) & 3))
    return SDVG_ERR_MISALIGNED;
  RopeCommitParams p = {};
  p.tokens = c->block_tokens;
  p.heads = c->heads;
  int st = fill_rope(p, c->head_dim, c->block_tokens,
                     RopeArgs{frames, grid_h, grid_w, frame_offset, tab_frames, cos_sin_tab});
  if (st != SDVG_OK) return st;
  int slot = 0;
  if ((st = sdvg::ring_begin_commit(c, block_index, flags, &slot)) != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  p.slot_head_stride_vec = (long long)c->slots * c->block_tokens * (c->head_dim / 8);    // in 8-byte units here
  uint2* kslot = (uint2*)c->k_buf + sdvg::slot_offset(c, 0, slot) / 8;
  uint2* vslot = (uint2*)c->v_buf + sdvg::slot_offset(c, 0, slot) / 8;
  if (q) p.job[p.njobs++] = TensorJob{(const uint4*)q, nullptr, nullptr, 1, (uint2*)q8_out, nullptr, q_inv_scale};
  p.job[p.njobs++] = TensorJob{(const uint4*)k, nullptr, nullptr, 1, nullptr, kslot, k_inv_scale};
  p.job[p.njobs++] = TensorJob{(const uint4*)v, nullptr, nullptr, 0, nullptr, vslot, v_inv_scale};
  st = launch(p, c->head_dim, (cudaStream_t)stream, true);
  if (st != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

int sdvg_quant_e4m3_tiled(const void* x, void* out8, float* tile_scale, int tokens, int heads, int head_dim,
                          void* stream) {
  SDVG_RANGE();
  if (!x || !out8 || !tile_scale) return SDVG_ERR_INVALID_ARG;
  if (tokens <= 0 || heads <= 0 || head_dim != 128) return SDVG_ERR_BAD_SHAPE;
  if (!sdvg::aligned16(x) || !sdvg::aligned16(out8) || (reinterpret_cast<uintptr_t>(tile_scale) & 3))
    return SDVG_ERR_MISALIGNED;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  TileQuantParams p = {};
  p.r.tokens = tokens;
  p.r.heads = heads;
  p.job[0] = TileQuantJob{(const uint4*)x, (uint2*)out8, (long long)heads * 16, 16, tile_scale,
                          sdvg::scale_tiles(tokens), 0};
  return launch_tile_quant(p, 1, (cudaStream_t)stream);
}

int sdvg_kv_commit_e4m3_tiled(sdvg_cache* c, const void* k_roped, const void* v, int64_t block_index, int flags,
                              int64_t* evicted_block, void* stream) {
  SDVG_RANGE();
  if (!c || !k_roped || !v) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1) return SDVG_ERR_BAD_SHAPE;
  if (!c->k_tile_scale || !c->v_tile_scale) return SDVG_ERR_BAD_STATE;
  if (!sdvg::aligned16(k_roped) || !sdvg::aligned16(v)) return SDVG_ERR_MISALIGNED;
  int slot = 0;
  int st = sdvg::ring_begin_commit(c, block_index, flags, &slot);
  if (st != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  TileQuantParams p = {};
  p.r.tokens = c->block_tokens;
  p.r.heads = c->heads;
  int n = 0;
  tile_commit_jobs(p, n, c, slot, k_roped, v, 0);
  if ((st = launch_tile_quant(p, n, (cudaStream_t)stream)) != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

int sdvg_rope3d_qk_commit_e4m3_tiled(sdvg_cache* c, const void* q, const void* k, const void* v, void* q8_out,
                                     float* q_tile_scale, int frames, int grid_h, int grid_w, int frame_offset,
                                     const float* cos_sin_tab, int tab_frames, int64_t block_index, int flags,
                                     int64_t* evicted_block, void* stream) {
  SDVG_RANGE();
  if (!c || !k || !v) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1) return SDVG_ERR_BAD_SHAPE;
  if (!c->k_tile_scale || !c->v_tile_scale) return SDVG_ERR_BAD_STATE;
  if ((q == nullptr) != (q8_out == nullptr) || (q && !q_tile_scale)) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(q) || !sdvg::aligned16(k) || !sdvg::aligned16(v) || !sdvg::aligned16(q8_out) ||
      (reinterpret_cast<uintptr_t>(q_tile_scale) & 3))
    return SDVG_ERR_MISALIGNED;
  TileQuantParams p = {};
  p.r.tokens = c->block_tokens;
  p.r.heads = c->heads;
  int st = fill_rope(p.r, c->head_dim, c->block_tokens,
                     RopeArgs{frames, grid_h, grid_w, frame_offset, tab_frames, cos_sin_tab});
  if (st != SDVG_OK) return st;
  int slot = 0;
  if ((st = sdvg::ring_begin_commit(c, block_index, flags, &slot)) != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  int n = 0;
  if (q)
    p.job[n++] = TileQuantJob{(const uint4*)q, (uint2*)q8_out, (long long)c->heads * 16, 16, q_tile_scale,
                              sdvg::scale_tiles(c->block_tokens), 1};
  tile_commit_jobs(p, n, c, slot, k, v, 1);
  if ((st = launch_tile_quant(p, n, (cudaStream_t)stream)) != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

int sdvg_cache_read_block(const sdvg_cache* c, int slot, void* k_out, void* v_out, void* stream) {
  SDVG_RANGE();
  if (!c || (!k_out && !v_out)) return SDVG_ERR_INVALID_ARG;
  if (slot < 0 || slot >= c->slots) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(k_out) || !sdvg::aligned16(v_out)) return SDVG_ERR_MISALIGNED;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  const int vpr = c->head_dim * c->elem_bytes / 16;          // 16-byte vectors per (token, head) row: 16 or 8
  const long long stride = (long long)c->slots * c->block_tokens * vpr;
  const long long total = (long long)c->block_tokens * c->heads * vpr;
  const unsigned blocks = (unsigned)((total + kThreads - 1) / kThreads < 148 * 8 ? (total + kThreads - 1) / kThreads
                                                                                  : 148 * 8);
  const void* bufs[2] = {c->k_buf, c->v_buf};
  void* outs[2] = {k_out, v_out};
  for (int i = 0; i < 2; ++i) {
    if (!outs[i]) continue;
    const uint4* base = (const uint4*)bufs[i] + sdvg::slot_offset(c, 0, slot) * c->elem_bytes / 16;
    if (vpr == 16)
      slot_read_kernel<128><<<blocks, kThreads, 0, (cudaStream_t)stream>>>(base, (uint4*)outs[i], c->block_tokens,
                                                                          c->heads, stride);
    else
      slot_read_kernel<64><<<blocks, kThreads, 0, (cudaStream_t)stream>>>(base, (uint4*)outs[i], c->block_tokens,
                                                                         c->heads, stride);
    st = sdvg::cuda_status(cudaGetLastError());
    if (st != SDVG_OK) return st;
  }
  return SDVG_OK;
}

}  // extern "C"
