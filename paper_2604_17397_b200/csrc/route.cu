// Router (Sec. 3): q_b = min over the block's frame scores (Eq. 1); accept iff q_b >= tau and the
// block is not global block 0 (forced regeneration of the first block).
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
};

__device__ __forceinline__ long long range_begin(const RouteParams& p, int b) {
  return p.offsets ? (long long)p.offsets[b] : (long long)b * p.frames_per_block;
}

__global__ void __launch_bounds__(kThreads) route_kernel(const __grid_constant__ RouteParams p) {
  __shared__ __align__(16) float stage[kSmemFloats + 4];   // +4: room for the alignment shift
  const int ntiles = (p.num_blocks + kThreads - 1) / kThreads;
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int b0 = tile * kThreads;
    const int b1 = min(b0 + kThreads, p.num_blocks);
    const long long lo = range_begin(p, b0);
    const long long hi = range_begin(p, b1);
    const long long n = hi - lo;
    const bool staged = n > 0 && n <= kSmemFloats;
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
        const int s = (int)(range_begin(p, b) - lo) + shift;
        const int e = (int)(range_begin(p, b + 1) - lo) + shift;
        float m = __int_as_float(0x7fc00000);
        int idx = -1;
        if (e > s) {
          m = stage[s];
          idx = 0;
          for (int i = s + 1; i < e && m == m; ++i) {
            const float x = stage[i];
            if (x != x || x < m) { m = x; idx = i - s; }
          }
        }
        const bool ok = (p.first_block_index + b != 0) && (m >= p.tau);
        p.accept[b] = ok ? 1 : 0;
        p.q_min[b] = m;
        if (p.argmin) p.argmin[b] = idx;
      }
      __syncthreads();
    } else {
      const int b = b0 + threadIdx.x;
      if (b < b1) {
        const long long s = range_begin(p, b), e = range_begin(p, b + 1);
        float m = __int_as_float(0x7fc00000);
        int idx = -1;
        if (e > s) {
          m = p.scores[s];
          idx = 0;
          for (long long i = s + 1; i < e && m == m; ++i) {
            const float x = p.scores[i];
            if (x != x || x < m) { m = x; idx = (int)(i - s); }
          }
        }
        const bool ok = (p.first_block_index + b != 0) && (m >= p.tau);
        p.accept[b] = ok ? 1 : 0;
        p.q_min[b] = m;
        if (p.argmin) p.argmin[b] = idx;
      }
    }
  }
}

}  // namespace

extern "C" int sdvg_route(const float* scores, const int32_t* frame_offsets, int num_blocks,
                          int frames_per_block, int64_t first_block_index, float tau, uint8_t* accept,
                          float* q_min, int32_t* argmin, void* stream) {
  if (num_blocks < 0) return SDVG_ERR_BAD_SHAPE;
  if (!frame_offsets && frames_per_block < 1) return SDVG_ERR_BAD_SHAPE;
  if (num_blocks == 0) return SDVG_OK;
  if (!scores || !accept || !q_min) return SDVG_ERR_INVALID_ARG;
  if (!frame_offsets && (long long)num_blocks * frames_per_block >= (1ll << 40)) return SDVG_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(scores) & 3) || (reinterpret_cast<uintptr_t>(q_min) & 3) ||
      (reinterpret_cast<uintptr_t>(frame_offsets) & 3) || (reinterpret_cast<uintptr_t>(argmin) & 3))
    return SDVG_ERR_MISALIGNED;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  RouteParams p{scores, frame_offsets, num_blocks, frames_per_block, (long long)first_block_index, tau,
                accept, q_min, argmin};
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int ntiles = (num_blocks + kThreads - 1) / kThreads;
  const int grid = ntiles < sms * 4 ? ntiles : sms * 4;
  route_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}
