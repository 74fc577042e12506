// bf16 -> E4M3 with one static scale per head (the 8-bit variant of the cache and of the attention
// operands): y = e4m3(x * inv_scale[head]), the product one fp32 multiplication, the conversion round to
// nearest even and saturating at +-448.  One streaming pass: a thread turns 16 consecutive elements of a
// (token, head) row (two 16-byte loads) into one 16-byte store, either in the logical
// [tokens, heads, dim] layout or in a ring slot ([heads][slots][tokens][dim]).
#include <cuda_bf16.h>

#include "sdvg_internal.h"
#include "sm100_ptx.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxJobs = 2;

struct QuantJob {
  const uint4* src;          // bf16 [tokens, heads, dim]
  uint4* dst;                // bytes; (token, head) row at dst + token * token_stride + head * head_stride (16-byte units)
  const float* inv_scale;    // [heads]
  long long token_stride, head_stride;
};

struct QuantParams {
  QuantJob job[kMaxJobs];
  int tokens, heads, vec_per_row;        // vec_per_row = dim / 16 output vectors per row
};

__device__ __forceinline__ uint32_t quant4(uint32_t w0, uint32_t w1, float inv) {
  // a 32-bit word holds two bf16: the low half is the element with the lower index
  return sm100::pack_e4m3x4(__fmul_rn(__uint_as_float(w0 << 16), inv), __fmul_rn(__uint_as_float(w0 & 0xffff0000u), inv),
                            __fmul_rn(__uint_as_float(w1 << 16), inv), __fmul_rn(__uint_as_float(w1 & 0xffff0000u), inv));
}

__global__ void __launch_bounds__(kThreads) quant_e4m3_kernel(const __grid_constant__ QuantParams p) {
  const QuantJob job = p.job[blockIdx.y];
  const long long total = (long long)p.tokens * p.heads * p.vec_per_row;
  for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < total; i += (long long)gridDim.x * kThreads) {
    const int j = (int)(i % p.vec_per_row);
    const long long row = i / p.vec_per_row;
    const int h = (int)(row % p.heads);
    const long long t = row / p.heads;
    const float inv = __ldg(job.inv_scale + h);
    const uint4 a = __ldcs(job.src + 2 * i), b = __ldcs(job.src + 2 * i + 1);
    uint4 o;
    o.x = quant4(a.x, a.y, inv);
    o.y = quant4(a.z, a.w, inv);
    o.z = quant4(b.x, b.y, inv);
    o.w = quant4(b.z, b.w, inv);
    job.dst[t * job.token_stride + h * job.head_stride + j] = o;
  }
}

int launch(const QuantParams& p, int njobs, cudaStream_t stream) {
  const long long total = (long long)p.tokens * p.heads * p.vec_per_row;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  long long want = (total + kThreads - 1) / kThreads;
  long long cap = (long long)sms * 32 / njobs;                // few passes per thread; bounds the grid for very large tensors
  if (cap < 1) cap = 1;
  dim3 grid((unsigned)(want < cap ? want : cap), njobs, 1);
  quant_e4m3_kernel<<<grid, kThreads, 0, stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}

}  // namespace

extern "C" {

int sdvg_quant_e4m3(const void* x, const float* inv_scale, void* out, int tokens, int heads, int head_dim,
                    void* stream) {
  SDVG_RANGE();
  if (!x || !inv_scale || !out) return SDVG_ERR_INVALID_ARG;
  if (tokens <= 0 || heads <= 0 || !sdvg::head_dim_ok(head_dim)) return SDVG_ERR_BAD_SHAPE;
  if (!sdvg::aligned16(x) || !sdvg::aligned16(out) || (reinterpret_cast<uintptr_t>(inv_scale) & 3))
    return SDVG_ERR_MISALIGNED;
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  QuantParams p = {};
  p.tokens = tokens;
  p.heads = heads;
  p.vec_per_row = head_dim / 16;
  p.job[0] = QuantJob{(const uint4*)x, (uint4*)out, inv_scale, (long long)heads * p.vec_per_row, p.vec_per_row};
  return launch(p, 1, (cudaStream_t)stream);
}

int sdvg_kv_commit_e4m3(sdvg_cache* c, const void* k_roped, const void* v, const float* k_inv_scale,
                        const float* v_inv_scale, int64_t block_index, int flags, int64_t* evicted_block,
                        void* stream) {
  SDVG_RANGE();
  if (!c || !k_roped || !v || !k_inv_scale || !v_inv_scale) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1) return SDVG_ERR_BAD_SHAPE;
  if (!sdvg::aligned16(k_roped) || !sdvg::aligned16(v) ||
      ((reinterpret_cast<uintptr_t>(k_inv_scale) | reinterpret_cast<uintptr_t>(v_inv_scale)) & 3))
    return SDVG_ERR_MISALIGNED;
  int slot = 0;
  int st = sdvg::ring_begin_commit(c, block_index, flags, &slot);
  if (st != SDVG_OK) return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;
  QuantParams p = {};
  p.tokens = c->block_tokens;
  p.heads = c->heads;
  p.vec_per_row = c->head_dim / 16;
  const long long head_stride = (long long)c->slots * c->block_tokens * p.vec_per_row;
  uint4* kslot = (uint4*)c->k_buf + sdvg::slot_offset(c, 0, slot) / 16;
  uint4* vslot = (uint4*)c->v_buf + sdvg::slot_offset(c, 0, slot) / 16;
  p.job[0] = QuantJob{(const uint4*)k_roped, kslot, k_inv_scale, p.vec_per_row, head_stride};
  p.job[1] = QuantJob{(const uint4*)v, vslot, v_inv_scale, p.vec_per_row, head_stride};
  st = launch(p, 2, (cudaStream_t)stream);
  if (st != SDVG_OK) return st;
  sdvg::ring_end_commit(c, block_index, flags, slot, evicted_block);
  return SDVG_OK;
}

}  // extern "C"
