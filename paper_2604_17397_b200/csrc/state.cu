// Snapshot / restore of device-resident decoder state (Sec. 3 "Inference flow": the VAE decode cache is
// cloned before a draft block is scored and restored when the block is rejected).  The state is a
// list of buffers (feature maps of the causal decoder); one launch copies all of them with 16-byte
// vectors, every CTA walking the concatenated byte range in grid-sized strides.
#include "sdvg_internal.h"

namespace {

constexpr int kMaxSegments = 64;
constexpr int kThreads = 256;

struct CopyTable {
  const uint4* src[kMaxSegments];
  uint4* dst[kMaxSegments];
  unsigned long long first_vec[kMaxSegments + 1];   // prefix sums of the segment lengths in 16-byte vectors
  int count;
};

__global__ void __launch_bounds__(kThreads) state_copy_kernel(const __grid_constant__ CopyTable t) {
  const unsigned long long total = t.first_vec[t.count];
  int seg = 0;
  for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < total;
       i += (unsigned long long)gridDim.x * kThreads) {
    while (i >= t.first_vec[seg + 1]) ++seg;        // indices only grow: the search never goes back
    const unsigned long long j = i - t.first_vec[seg];
    t.dst[seg][j] = __ldcs(t.src[seg] + j);
  }
}

}  // namespace

extern "C" int sdvg_state_copy(const void* const* src, void* const* dst, const size_t* bytes, int count,
                               void* stream) {
  SDVG_RANGE();
  if (count < 0 || count > kMaxSegments) return SDVG_ERR_BAD_SHAPE;
  if (count == 0) return SDVG_OK;
  if (!src || !dst || !bytes) return SDVG_ERR_INVALID_ARG;
  CopyTable t = {};
  unsigned long long total = 0;
  for (int i = 0; i < count; ++i) {
    if (!src[i] || !dst[i]) return SDVG_ERR_INVALID_ARG;
    if (!sdvg::aligned16(src[i]) || !sdvg::aligned16(dst[i])) return SDVG_ERR_MISALIGNED;
    if (bytes[i] % 16) return SDVG_ERR_BAD_SHAPE;
    t.src[i] = (const uint4*)src[i];
    t.dst[i] = (uint4*)dst[i];
    t.first_vec[i] = total;
    total += bytes[i] / 16;
  }
  t.first_vec[count] = total;
  t.count = count;
  if (total == 0) return SDVG_OK;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned long long want = (total + kThreads - 1) / kThreads;
  const unsigned long long cap = (unsigned long long)sms * 8;
  state_copy_kernel<<<(unsigned)(want < cap ? want : cap), kThreads, 0, (cudaStream_t)stream>>>(t);
  return sdvg::cuda_status(cudaGetLastError());
}
