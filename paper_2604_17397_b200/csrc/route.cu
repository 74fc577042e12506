// Router (Sec. 3): q_b = min over the block's frame scores (Eq. 1); accept iff q_b >= tau and the
// block is not global block 0 (forced regeneration of the first block).  The same kernel serves the
// variants of the ablation (Sec. 4.3, Table 2): mean instead of minimum, uniform draws instead of
// the reward, forcing switched off, first block of every video of a batch.
//
// A CTA owns a tile of consecutive blocks, whose scores form one contiguous range.  The range is
// brought into shared memory with coalesced 16-byte loads (scalar loads for the unaligned head and
// tail), then each thread scans the frames of one block left to right with a strict '<', which is
// exactly the sequential definition (ties, +0/-0 and NaN resolve as stated in the header).  A tile
// whose range does not fit in shared memory is scanned straight from global memory.
#include "sdvg_internal.h"

namespace {

constexpr int kThreads = 256;           // blocks per tile = threads per CTA
constexpr int kSmemFloats = 8192;       // 32 KB staging

struct RouteParams {
  const float* scores;
  const int32_t* offsets;   // nullptr -> fixed frames_per_block
  int num_blocks, frames_per_block;
  long long first_block_index;
  float tau;
  uint8_t* accept;
  float* q_min;
  int32_t* argmin;
  int agg, signal, force_first;   // SDVG_AGG_*, SDVG_SIGNAL_*, reject first blocks
  int blocks_per_video;           // 0: one stream, only global block 0 is a first block
  const float* uniforms;          // SDVG_SIGNAL_RANDOM: one draw per block
  float accept_prob;
};

// Aggregate of frames [s, e) read through `at`: left-to-right strict-'<' minimum, or the fp32 mean
// (left-to-right sum, every partial sum rounded, then one IEEE division by the frame count).
template <typename At>
__device__ __forceinline__ void aggregate(const RouteParams& p, long long s, long long e, At at, float& m, int& idx) {
  m = __int_as_float(0x7fc00000);
  idx = -1;
  if (e <= s) return;
  m = at(s);
  if (p.agg == SDVG_AGG_MEAN) {
    for (long long i = s + 1; i < e; ++i) m = __fadd_rn(m, at(i));
    m = __fdiv_rn(m, (float)(e - s));
    return;
  }
  idx = 0;
  for (long long i = s + 1; i < e && m == m; ++i) {
    const float x = at(i);
    if (x != x || x < m) { m = x; idx = (int)(i - s); }
  }
}

__device__ __forceinline__ void decide(const RouteParams& p, int b, float m, int idx, bool has_frames) {
  const long long g = p.first_block_index + b;
  const bool first = p.blocks_per_video > 0 ? (g % p.blocks_per_video == 0) : (g == 0);
  bool ok = p.signal == SDVG_SIGNAL_RANDOM ? (p.uniforms[b] < p.accept_prob) : (m >= p.tau);
  ok = ok && has_frames && !(p.force_first && first);
  p.accept[b] = ok ? 1 : 0;
  p.q_min[b] = m;
  if (p.argmin) p.argmin[b] = idx;
}

__device__ __forceinline__ long long range_begin(const RouteParams& p, int b) {
  return p.offsets ? (long long)p.offsets[b] : (long long)b * p.frames_per_block;
}

// The offsets live in device memory, so the host cannot check them.  The kernel trusts only the two ends of the
// array: every read stays inside [offsets[0], offsets[num_blocks]), and a block whose own range leaves that
// interval or runs backwards counts as a block without frames (accept 0, NaN aggregate, argmin -1).
__device__ __forceinline__ bool range_ok(long long s, long long e, long long all_lo, long long all_hi) {
  return all_lo <= s && s <= e && e <= all_hi;
}

__global__ void __launch_bounds__(kThreads) route_kernel(const __grid_constant__ RouteParams p) {
  __shared__ __align__(16) float stage[kSmemFloats + 4];   // +4: room for the alignment shift
  const int ntiles = (p.num_blocks + kThreads - 1) / kThreads;
  const long long all_lo = range_begin(p, 0), all_hi = range_begin(p, p.num_blocks);
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int b0 = tile * kThreads;
    const int b1 = min(b0 + kThreads, p.num_blocks);
    const long long lo = range_begin(p, b0);
    const long long hi = range_begin(p, b1);
    const long long n = hi - lo;
    const bool staged = n > 0 && n <= kSmemFloats && range_ok(lo, hi, all_lo, all_hi);
    if (staged) {
      // stage[i] = scores[lo + i]; vector body starts at the first 16-byte aligned element
      const float* src = p.scores + lo;
      int head = (int)(((16 - (reinterpret_cast<uintptr_t>(src) & 15)) & 15) >> 2);
      if (head > n) head = (int)n;
      const int nvec = (int)((n - head) >> 2);
      const int tail0 = head + nvec * 4;
      // shared copy keeps the same misalignment so that vector stores stay aligned
      const int shift = (4 - head) & 3;
      for (int i = threadIdx.x; i < head; i += kThreads) stage[shift + i] = src[i];
      const float4* vsrc = reinterpret_cast<const float4*>(src + head);
      float4* vdst = reinterpret_cast<float4*>(stage + shift + head);
      for (int i = threadIdx.x; i < nvec; i += kThreads) vdst[i] = __ldcs(vsrc + i);
      for (int i = tail0 + threadIdx.x; i < n; i += kThreads) stage[shift + i] = src[i];
      __syncthreads();
      const int b = b0 + threadIdx.x;
      if (b < b1) {
        long long s = range_begin(p, b), e = range_begin(p, b + 1);
        if (!range_ok(s, e, all_lo, all_hi)) e = s;          // malformed: no frames
        float m;
        int idx;
        if (lo <= s && e <= hi) {
          const int sh = shift - (int)lo;
          aggregate(p, s, e, [&](long long i) { return stage[i + sh]; }, m, idx);
        } else {
          // offsets that are not sorted can place a block outside its tile's range: read it where it is
          aggregate(p, s, e, [&](long long i) { return p.scores[i]; }, m, idx);
        }
        decide(p, b, m, idx, e > s);
      }
      __syncthreads();
    } else {
      const int b = b0 + threadIdx.x;
      if (b < b1) {
        long long s = range_begin(p, b), e = range_begin(p, b + 1);
        if (!range_ok(s, e, all_lo, all_hi)) e = s;          // malformed: no frames
        float m;
        int idx;
        aggregate(p, s, e, [&](long long i) { return p.scores[i]; }, m, idx);
        decide(p, b, m, idx, e > s);
      }
    }
  }
}

// Fixed frame count that is a multiple of four, scores 16-byte aligned: a block's frames are F / 4 aligned
// 16-byte vectors, so each thread reads its own block straight from global memory (a warp's loads cover one
// contiguous run, every sector fully used; the vectors of a block after the first hit the line the first one
// fetched) and no staging or barrier is needed.  Same left-to-right scan as above.
template <int VECS>      // F / 4 when known at compile time (0: run-time count)
__global__ void __launch_bounds__(kThreads) route_vec_kernel(const __grid_constant__ RouteParams p) {
  const int vecs = VECS ? VECS : p.frames_per_block / 4;
  for (int b = blockIdx.x * kThreads + threadIdx.x; b < p.num_blocks; b += gridDim.x * kThreads) {
    const float4* src = reinterpret_cast<const float4*>(p.scores) + (long long)b * vecs;
    float m;
    int idx = -1;
    if (p.agg == SDVG_AGG_MEAN) {
      float4 x = __ldcs(src);
      m = __fadd_rn(__fadd_rn(__fadd_rn(x.x, x.y), x.z), x.w);
#pragma unroll 4
      for (int i = 1; i < vecs; ++i) {
        x = __ldcs(src + i);
        m = __fadd_rn(__fadd_rn(__fadd_rn(__fadd_rn(m, x.x), x.y), x.z), x.w);
      }
      m = __fdiv_rn(m, (float)(4 * vecs));
    } else {
      // all vectors are requested before the scan; a NaN stops the scan where the sequential definition stops
      float4 x = __ldcs(src);
      m = x.x;
      idx = 0;
      auto step = [&](float v, int i) {
        if (m == m && (v != v || v < m)) { m = v; idx = i; }
      };
      step(x.y, 1); step(x.z, 2); step(x.w, 3);
#pragma unroll 4
      for (int i = 1; i < vecs; ++i) {
        x = __ldcs(src + i);
        step(x.x, 4 * i); step(x.y, 4 * i + 1); step(x.z, 4 * i + 2); step(x.w, 4 * i + 3);
      }
    }
    decide(p, b, m, idx, true);
  }
}

// accept-rate statistics: counts[0] += accepted, counts[1] += routable, first blocks left out of both
__global__ void __launch_bounds__(kThreads) accept_stats_kernel(const uint8_t* __restrict__ accept, int num_blocks,
                                                                 long long first_block_index, int blocks_per_video,
                                                                 unsigned long long* counts) {
  unsigned int acc = 0, routable = 0;
  for (int b = blockIdx.x * kThreads + threadIdx.x; b < num_blocks; b += gridDim.x * kThreads) {
    const long long g = first_block_index + b;
    const bool first = blocks_per_video > 0 ? (g % blocks_per_video == 0) : (g == 0);
    if (!first) {
      ++routable;
      acc += accept[b] ? 1u : 0u;
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    acc += __shfl_down_sync(0xffffffffu, acc, o);
    routable += __shfl_down_sync(0xffffffffu, routable, o);
  }
  if ((threadIdx.x & 31) == 0 && (acc | routable)) {
    atomicAdd(&counts[0], (unsigned long long)acc);
    atomicAdd(&counts[1], (unsigned long long)routable);
  }
}

}  // namespace

namespace {

int route_launch(const RouteParams& p, cudaStream_t stream) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int ntiles = (p.num_blocks + kThreads - 1) / kThreads;
  if (!p.offsets && p.frames_per_block % 4 == 0 && (reinterpret_cast<uintptr_t>(p.scores) & 15) == 0) {
    const int grid = ntiles < sms * 32 ? ntiles : sms * 32;      // one block of scores per thread up to 1.2 M blocks
    if (p.frames_per_block == 12) route_vec_kernel<3><<<grid, kThreads, 0, stream>>>(p);
    else route_vec_kernel<0><<<grid, kThreads, 0, stream>>>(p);
    return sdvg::cuda_status(cudaGetLastError());
  }
  const int grid = ntiles < sms * 4 ? ntiles : sms * 4;
  route_kernel<<<grid, kThreads, 0, stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}

int route_checks(const float* scores, const int32_t* frame_offsets, int num_blocks, int frames_per_block,
                 const uint8_t* accept, const float* q_min, const int32_t* argmin) {
  if (num_blocks < 0) return SDVG_ERR_BAD_SHAPE;
  if (!frame_offsets && frames_per_block < 1) return SDVG_ERR_BAD_SHAPE;
  if (num_blocks == 0) return SDVG_OK;
  if (!scores || !accept || !q_min) return SDVG_ERR_INVALID_ARG;
  if (!frame_offsets && (long long)num_blocks * frames_per_block >= (1ll << 40)) return SDVG_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(scores) & 3) || (reinterpret_cast<uintptr_t>(q_min) & 3) ||
      (reinterpret_cast<uintptr_t>(frame_offsets) & 3) || (reinterpret_cast<uintptr_t>(argmin) & 3))
    return SDVG_ERR_MISALIGNED;
  return SDVG_OK;
}

}  // namespace

extern "C" int sdvg_route(const float* scores, const int32_t* frame_offsets, int num_blocks,
                          int frames_per_block, int64_t first_block_index, float tau, uint8_t* accept,
                          float* q_min, int32_t* argmin, void* stream) {
  SDVG_RANGE();
  int st = route_checks(scores, frame_offsets, num_blocks, frames_per_block, accept, q_min, argmin);
  if (st != SDVG_OK || num_blocks == 0) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  RouteParams p{scores, frame_offsets, num_blocks, frames_per_block, (long long)first_block_index, tau,
                accept, q_min, argmin, SDVG_AGG_MIN, SDVG_SIGNAL_REWARD, 1, 0, nullptr, 0.f};
  return route_launch(p, (cudaStream_t)stream);
}

extern "C" int sdvg_route_policy(const float* scores, const int32_t* frame_offsets, int num_blocks,
                                 int frames_per_block, int64_t first_block_index, int blocks_per_video, float tau,
                                 int agg, int signal, int force_first, const float* uniforms, float accept_prob,
                                 uint8_t* accept, float* aggregate_out, int32_t* argmin, void* stream) {
  SDVG_RANGE();
  if ((agg != SDVG_AGG_MIN && agg != SDVG_AGG_MEAN) || (signal != SDVG_SIGNAL_REWARD && signal != SDVG_SIGNAL_RANDOM))
    return SDVG_ERR_INVALID_ARG;
  if (blocks_per_video < 0 || (blocks_per_video > 0 && first_block_index < 0)) return SDVG_ERR_INVALID_ARG;
  int st = route_checks(scores, frame_offsets, num_blocks, frames_per_block, accept, aggregate_out, argmin);
  if (st != SDVG_OK || num_blocks == 0) return st;
  if (signal == SDVG_SIGNAL_RANDOM) {
    if (!uniforms) return SDVG_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(uniforms) & 3) return SDVG_ERR_MISALIGNED;
  }
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  RouteParams p{scores, frame_offsets, num_blocks, frames_per_block, (long long)first_block_index, tau,
                accept, aggregate_out, argmin, agg, signal, force_first ? 1 : 0, blocks_per_video, uniforms, accept_prob};
  return route_launch(p, (cudaStream_t)stream);
}

extern "C" int sdvg_accept_stats(const uint8_t* accept, int num_blocks, int64_t first_block_index,
                                 int blocks_per_video, unsigned long long* counts, void* stream_) {
  SDVG_RANGE();
  if (num_blocks < 0) return SDVG_ERR_BAD_SHAPE;
  if (!counts || (num_blocks > 0 && !accept)) return SDVG_ERR_INVALID_ARG;
  if (blocks_per_video < 0 || (blocks_per_video > 0 && first_block_index < 0)) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(counts) & 7) return SDVG_ERR_MISALIGNED;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  cudaError_t e = cudaMemsetAsync(counts, 0, 2 * sizeof(unsigned long long), stream);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  if (num_blocks == 0) return SDVG_OK;
  const int want = (num_blocks + kThreads - 1) / kThreads;
  accept_stats_kernel<<<want < 592 ? want : 592, kThreads, 0, stream>>>(accept, num_blocks, (long long)first_block_index,
                                                                        blocks_per_video, counts);
  return sdvg::cuda_status(cudaGetLastError());
}
