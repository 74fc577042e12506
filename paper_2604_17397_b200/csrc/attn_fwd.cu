// Block attention forward for sm_100a: O = softmax(scale * Q K^T) V over every visible key
// (Sec. 4.1 "Models": both models attend causally over a KV cache; no key is masked inside a call because the
// block sees all of itself and all of its window).
//
// Both products run on the 5th-generation tensor cores (tcgen05.mma, bf16 in, fp32 accumulators in
// tensor memory).  Q, K and V tiles are staged in shared memory by TMA with the 128-byte swizzle;
// S = Q K^T lands in TMEM, the softmax threads (two per query row) read it with tcgen05.ld and write
// the bf16 probabilities to TMEM columns of their own, and O += P V takes P straight from TMEM
// and V from shared memory as an MN-major operand.  Keys arrive as up to three segments (runs of
// ring slots and/or the block's own K/V tensors), each with its own tensor map whose row extent
// ends at the segment so that TMA zero-fills the ragged last tile; those columns are masked to
// -inf before the row maximum.
//
// The 8-bit variant (sdvg_block_attn_fwd_e4m3) runs the same kernel template on E4M3 operands with per-head
// scales; Sec. 2 names quantised attention as an orthogonal speed-up and fixes no format.
//
// Every wait on an mbarrier is bounded: kWaitLimitNs after kernel start a waiting thread gives up
// and raises the (sticky) status word to SDVG_ERR_TIMEOUT; all roles then fall through to the common
// exit, which releases tensor memory.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

#include "sdvg_internal.h"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int kTileM = 128;            // query rows per tile
constexpr int kTileN = 128;            // keys per tile
constexpr int kMaxSegments = 3;
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s
constexpr int kWorkspaceBytes = 256;

constexpr int kMaxBatch = 4;           // independent problems of one shape per launch

// One attention problem of a launch: its tensor maps and outputs.
struct alignas(64) AttnProblem {
  CUtensorMap q_map;
  CUtensorMap k_map[kMaxSegments];
  CUtensorMap v_map[kMaxSegments];
  __nv_bfloat16* out;
  float* lse;
  const float* qk_descale;             // 8-bit variant only: per head, q scale * k scale
  const float* v_descale;              // 8-bit variant only: per head, v scale
  // 8-bit variant with tile scales only (k_map[0] and v_map[0] are then 4-D maps over the whole ring):
  const float* q_tile_scale;           // [heads][query tiles]
  const float* k_tile_scale;           // [heads][slots][tiles], the cache's arrays
  const float* v_tile_scale;
};

// All problems of a launch have the same shape and the same key segments (same ring fill, same
// staging); heads of the problems are numbered through: global head g = problem * heads + head.
struct alignas(64) AttnParams {
  AttnProblem prob[kMaxBatch];
  int batch;
  int seg_len[kMaxSegments];
  int nseg;
  int tokens, heads;
  float scale_log2e;                   // scale * log2(e): softmax is evaluated with exp2
  unsigned int* work;                  // [0] self-test result, [1] sticky status word, [2] count of accumulator rescale events
  // tile scales: the keys are the tiles of ts_nslots ring slots, every slot tiled on its own (ts_tiles tiles)
  int ts_nslots, ts_tiles, ts_cache_slots;
  unsigned char ts_slot[16];
};
static_assert(sizeof(AttnParams) <= 4096, "kernel parameter space");

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}

// Every wait on an mbarrier ends at an absolute deadline taken at kernel start.
struct Deadline {
  uint64_t t_ns;                       // globaltimer value after which waits give up
  unsigned int* status;                // global status word
};

// Slow path of the bounded wait: poll until the phase completes or the deadline passes.  Kept out
// of line of the first attempt so that the timer read never sits on the fast path.  Waiting threads
// that poll less often (a suspend-time hint on the try_wait, the timer read once per 256 polls) or that
// never suspend (test_wait) were measured 2-5% slower: how soon a waiter notices counts for more than the
// issue slots its polling takes.
__device__ __forceinline__ bool wait_bar_slow(uint32_t bar_addr, uint32_t parity, uint64_t deadline_ns,
                                           unsigned int* status) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred p, q;\n\t"
      ".reg .u64 t;\n\t"
      "SDVG_WAIT:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra SDVG_DONE;\n\t"
      "mov.u64 t, %%globaltimer;\n\t"
      "setp.lt.u64 q, t, %3;\n\t"
      "@q bra SDVG_WAIT;\n\t"
      "SDVG_DONE:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity), "l"(deadline_ns)
      : "memory");
  if (!ok) atomicMax(status, (unsigned)SDVG_ERR_TIMEOUT);      // sticky: only a reset clears it
  return ok != 0;
}

// Bounded mbarrier wait.  One try_wait (which itself suspends the thread for a hardware-chosen
// time) settles almost every wait; only if it fails does the thread enter the timed poll loop.
// Returns false (and records SDVG_ERR_TIMEOUT) once the deadline has passed.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, const Deadline& d) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_bar_slow(smem_u32(bar), parity, d.t_ns, d.status);
}

// The same wait made by all 32 lanes of a warp, with a warp-uniform result.
__device__ __forceinline__ bool wait_warp(uint64_t* bar, uint32_t parity, const Deadline& d) {
  return __all_sync(0xffffffffu, wait_bar(bar, parity, d));
}

#include "attn_fwd_ws.cuh"

// ---- host side -------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  // looked up once; the initialisation of a function-local static is thread-safe
  static const EncodeTiledFn fn = [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(ptr);
    return (EncodeTiledFn) nullptr;
  }();
  return fn;
}

// bf16 (elem_bytes 2) or byte (1) matrix seen as (dim, rows, heads) with arbitrary row and head strides;
// box = 128 bytes x 128 rows x 1, 128-byte swizzle, rows beyond `rows` read as zero.
int make_map(CUtensorMap* m, const void* base, int head_dim, long long rows, int heads, size_t row_stride_bytes,
             size_t head_stride_bytes, int elem_bytes = 2) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return SDVG_ERR_CUDA;
  cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)rows, (cuuint64_t)heads};
  cuuint64_t strides[2] = {(cuuint64_t)row_stride_bytes, (cuuint64_t)head_stride_bytes};
  cuuint32_t box[3] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)kTileN, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SDVG_OK : SDVG_ERR_CUDA;
}

// The whole byte ring [heads][slots][tokens][128] as (dim, token, slot, head): box = one 128-byte row x 128 tokens
// of one slot and head; tokens past the block's end read as zero.
int make_ring_map(CUtensorMap* m, const void* base, long long tokens, int slots, int heads) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return SDVG_ERR_CUDA;
  cuuint64_t dims[4] = {128, (cuuint64_t)tokens, (cuuint64_t)slots, (cuuint64_t)heads};
  cuuint64_t strides[3] = {128, (cuuint64_t)tokens * 128, (cuuint64_t)slots * tokens * 128};
  cuuint32_t box[4] = {128, (cuuint32_t)kTileN, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SDVG_OK : SDVG_ERR_CUDA;
}

// One-time set-up per device and kernel instance: the opt-in to the kernel's dynamic shared memory is a
// per-device attribute, and the grid is sized by that device's SM count.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mu;

template <int D, bool F8 = false, bool TS = false>
int launch_ws(const AttnParams& p, cudaStream_t stream) {
  static int sms_of_device[kMaxDevices] = {};          // 0: this device has not been set up yet
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  if (dev < 0 || dev >= kMaxDevices) return SDVG_ERR_INVALID_ARG;
  int sms;
  {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (!sms_of_device[dev]) {
      // The softmax warps grow their register count out of what the other warps of their sub-partition give
      // back; a warp that asks for more than its sub-partition holds would wait forever.  The pool is what the
      // kernel was compiled to launch with, so refuse to launch a build whose count does not cover the split.
      cudaFuncAttributes attr;
      e = cudaFuncGetAttributes(&attr, attn_fwd_ws_kernel<D, F8, TS>);
      if (e != cudaSuccess) return sdvg::cuda_status(e);
      if (5 * attr.numRegs < 4 * WsCfg<D, F8>::kSoftmaxRegs + WsCfg<D, F8>::kIssueRegs) return SDVG_ERR_BAD_STATE;
      e = cudaFuncSetAttribute(attn_fwd_ws_kernel<D, F8, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               WsCfg<D, F8>::kDynamic);
      if (e != cudaSuccess) return sdvg::cuda_status(e);
      int n = 0;
      e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess || n < 1) return sdvg::cuda_status(e != cudaSuccess ? e : cudaErrorUnknown);
      sms_of_device[dev] = n;
    }
    sms = sms_of_device[dev];
  }
  const int total_tiles = ((p.tokens + kTileM - 1) / kTileM) * p.heads * p.batch;
  const int grid = total_tiles < sms ? total_tiles : sms;
  attn_fwd_ws_kernel<D, F8, TS><<<grid, WsCfg<D, F8>::kThreads, WsCfg<D, F8>::kDynamic, stream>>>(p);
  return sdvg::cuda_status(cudaGetLastError());
}

// Argument and ring-state checks of one problem; touches no CUDA API.
int check_problem(const void* q, const void* k_self, const void* v_self, const sdvg_cache* c, int64_t block_index,
                  const void* out, const float* lse) {
  if (!q || !c || !out) return SDVG_ERR_INVALID_ARG;
  if ((k_self == nullptr) != (v_self == nullptr)) return SDVG_ERR_INVALID_ARG;
  if (!sdvg::aligned16(q) || !sdvg::aligned16(k_self) || !sdvg::aligned16(v_self) || !sdvg::aligned16(out) ||
      (reinterpret_cast<uintptr_t>(lse) & 3))
    return SDVG_ERR_MISALIGNED;
  if (block_index < 0 || block_index != c->next_block) return SDVG_ERR_BAD_STATE;
  if (!k_self && c->staged_block != block_index) return SDVG_ERR_BAD_STATE;
  return SDVG_OK;
}

// Fills the tensor maps of one checked problem; the key segments go to seg_len / nseg.
int fill_problem(AttnProblem& pr, int* seg_len, int* nseg_out, const void* q, const void* k_self, const void* v_self,
                 const sdvg_cache* c, int64_t block_index, void* out, float* lse) {
  const int T = c->block_tokens, H = c->heads, D = c->head_dim, S = c->slots;
  const int eb = c->elem_bytes;                      // q, k_self and v_self have the cache's element type
  const size_t row_bytes = (size_t)D * eb;
  const size_t ring_head_stride = (size_t)S * T * row_bytes;
  int st, nseg = 0;
  pr.out = (__nv_bfloat16*)out;
  pr.lse = lse;
  if ((st = make_map(&pr.q_map, q, D, T, H, (size_t)H * row_bytes, row_bytes, eb)) != SDVG_OK) return st;

  // Visible committed blocks: the last S-1 before block_index, living in slots (b % S).  Their slots
  // form at most two runs of consecutive slots; with the block staged, its slot joins them.
  const int64_t first = block_index - (S - 1) > 0 ? block_index - (S - 1) : 0;
  bool use[64];
  if (S > 64) return SDVG_ERR_BAD_SHAPE;
  for (int s = 0; s < S; ++s) use[s] = false;
  for (int64_t b = first; b < block_index; ++b) {
    const int s = (int)(b % S);
    if (c->slot_block[s] != b) return SDVG_ERR_BAD_STATE;
    use[s] = true;
  }
  if (!k_self) use[(int)(block_index % S)] = true;
  for (int s = 0; s < S;) {
    if (!use[s]) { ++s; continue; }
    int e = s;
    while (e < S && use[e]) ++e;
    if (nseg >= kMaxSegments) return SDVG_ERR_BAD_STATE;
    const long long rows = (long long)(e - s) * T;
    const char* kb = (const char*)c->k_buf + (size_t)s * T * row_bytes;
    const char* vb = (const char*)c->v_buf + (size_t)s * T * row_bytes;
    if ((st = make_map(&pr.k_map[nseg], kb, D, rows, H, row_bytes, ring_head_stride, eb)) != SDVG_OK) return st;
    if ((st = make_map(&pr.v_map[nseg], vb, D, rows, H, row_bytes, ring_head_stride, eb)) != SDVG_OK) return st;
    seg_len[nseg++] = (int)rows;
    s = e;
  }
  if (k_self) {
    if (nseg >= kMaxSegments) return SDVG_ERR_BAD_STATE;
    if ((st = make_map(&pr.k_map[nseg], k_self, D, T, H, (size_t)H * row_bytes, row_bytes, eb)) != SDVG_OK) return st;
    if ((st = make_map(&pr.v_map[nseg], v_self, D, T, H, (size_t)H * row_bytes, row_bytes, eb)) != SDVG_OK) return st;
    seg_len[nseg++] = T;
  }
  *nseg_out = nseg;
  return SDVG_OK;
}

// Validation, tensor maps, scratch clear and launch shared by the attention entry points: `batch`
// problems of one shape, fused into one launch when their key segments agree, else launched one by one.
int attn_forward_batch(int batch, const void* const* q, const void* const* k_self, const void* const* v_self,
                       const sdvg_cache* const* caches, const int64_t* block_index, void* const* out,
                       float* const* lse, float scale, void* workspace, size_t workspace_bytes, cudaStream_t stream,
                       int elem_bytes = 2, const float* const* qk_descale = nullptr,
                       const float* const* v_descale = nullptr) {
  if (batch < 1 || !q || !caches || !block_index || !out || !workspace) return SDVG_ERR_INVALID_ARG;
  if (elem_bytes == 1) {
    if (!qk_descale || !v_descale) return SDVG_ERR_INVALID_ARG;
    for (int b = 0; b < batch && b < kMaxBatch; ++b) {
      if (!qk_descale[b] || !v_descale[b]) return SDVG_ERR_INVALID_ARG;
      if ((reinterpret_cast<uintptr_t>(qk_descale[b]) | reinterpret_cast<uintptr_t>(v_descale[b])) & 3) return SDVG_ERR_MISALIGNED;
    }
  }
  if (batch > kMaxBatch) return SDVG_ERR_BAD_SHAPE;
  if (workspace_bytes < (size_t)kWorkspaceBytes) return SDVG_ERR_INVALID_ARG;
  if (!(scale > 0.f) || !isfinite(scale)) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SDVG_ERR_MISALIGNED;
  for (int b = 0; b < batch; ++b) {
    if (!caches[b]) return SDVG_ERR_INVALID_ARG;
    if (caches[b]->block_tokens != caches[0]->block_tokens || caches[b]->heads != caches[0]->heads ||
        caches[b]->head_dim != caches[0]->head_dim || caches[b]->elem_bytes != elem_bytes)
      return SDVG_ERR_BAD_SHAPE;
  }
  int st;
  for (int b = 0; b < batch; ++b)
    if ((st = check_problem(q[b], k_self ? k_self[b] : nullptr, v_self ? v_self[b] : nullptr, caches[b], block_index[b],
                            out[b], lse ? lse[b] : nullptr)) != SDVG_OK)
      return st;
  if ((st = sdvg::require_sm100()) != SDVG_OK) return st;

  AttnParams p = {};
  p.tokens = caches[0]->block_tokens;
  p.heads = caches[0]->heads;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.work = (unsigned int*)workspace;
  const int D = caches[0]->head_dim;
  bool same = true;
  int seg_len[kMaxBatch][kMaxSegments] = {}, nseg[kMaxBatch] = {};
  for (int b = 0; b < batch; ++b) {
    st = fill_problem(p.prob[b], seg_len[b], &nseg[b], q[b], k_self ? k_self[b] : nullptr, v_self ? v_self[b] : nullptr,
                      caches[b], block_index[b], out[b], lse ? lse[b] : nullptr);
    if (st != SDVG_OK) return st;
    p.prob[b].qk_descale = elem_bytes == 1 ? qk_descale[b] : nullptr;
    p.prob[b].v_descale = elem_bytes == 1 ? v_descale[b] : nullptr;
    same = same && nseg[b] == nseg[0];
    for (int s = 0; same && s < nseg[b]; ++s) same = seg_len[b][s] == seg_len[0][s];
  }
  auto launch = [&](const AttnParams& pp) {
    if (elem_bytes == 1) return launch_ws<128, true>(pp, stream);     // an 8-bit cache always has head_dim 128
    return D == 128 ? launch_ws<128>(pp, stream) : launch_ws<64>(pp, stream);
  };
  if (same) {
    p.batch = batch;
    p.nseg = nseg[0];
    for (int s = 0; s < nseg[0]; ++s) p.seg_len[s] = seg_len[0][s];
    return launch(p);
  }
  // different ring fill or staging per problem: one launch each, in stream order (they share the status word)
  for (int b = 0; b < batch; ++b) {
    AttnParams one = p;
    one.prob[0] = p.prob[b];
    one.batch = 1;
    one.nseg = nseg[b];
    for (int s = 0; s < kMaxSegments; ++s) one.seg_len[s] = seg_len[b][s];
    if ((st = launch(one)) != SDVG_OK) return st;
  }
  return SDVG_OK;
}

int attn_forward(const void* q, const void* k_self, const void* v_self, const sdvg_cache* c, int64_t block_index,
                 void* out, float* lse, float scale, void* workspace, size_t workspace_bytes,
                 cudaStream_t stream) {
  if (!c) return SDVG_ERR_INVALID_ARG;
  return attn_forward_batch(1, &q, k_self ? &k_self : nullptr, v_self ? &v_self : nullptr, &c, &block_index, &out,
                            &lse, scale, workspace, workspace_bytes, stream);
}

// Self-test of the bounded wait: one warp waits on an mbarrier phase that nothing ever completes, with
// the given time limit, through the same wait_bar the attention kernel uses.
__global__ void bounded_wait_selftest_kernel(unsigned int* work, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  const Deadline dl{globaltimer_ns() + limit_ns, work + 1};
  const bool ok = wait_warp(&bar, 0, dl);
  if (threadIdx.x == 0) work[0] = ok ? 1u : 2u;          // 2: the wait gave up, as it should
}

// Scratch for sdvg_block_attn_fwd_noalloc: lives in the library image, one copy per device that
// loads it.  In host code this name is only a handle for cudaGetSymbolAddress, never a pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kWorkspaceBytes];

}  // namespace

extern "C" {

size_t sdvg_block_attn_workspace_bytes(void) { return kWorkspaceBytes; }

int sdvg_block_attn_workspace_reset(void* workspace, size_t workspace_bytes, void* stream_) {
  if (!workspace || workspace_bytes < (size_t)kWorkspaceBytes) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SDVG_ERR_MISALIGNED;
  return sdvg::cuda_status(cudaMemsetAsync(workspace, 0, kWorkspaceBytes, (cudaStream_t)stream_));
}

int sdvg_block_attn_fwd(const void* q, const void* k_self, const void* v_self, const sdvg_cache* c,
                        int64_t block_index, void* out, float* lse, float scale, void* workspace,
                        size_t workspace_bytes, void* stream_) {
  SDVG_RANGE();
  return attn_forward(q, k_self, v_self, c, block_index, out, lse, scale, workspace, workspace_bytes,
                      (cudaStream_t)stream_);
}

int sdvg_block_attn_fwd_batched(int batch, const void* const* q, const void* const* k_self,
                                const void* const* v_self, const sdvg_cache* const* caches,
                                const int64_t* block_index, void* const* out, float* const* lse, float scale,
                                void* workspace, size_t workspace_bytes, void* stream_) {
  SDVG_RANGE();
  return attn_forward_batch(batch, q, k_self, v_self, caches, block_index, out, lse, scale, workspace,
                            workspace_bytes, (cudaStream_t)stream_);
}

int sdvg_block_attn_fwd_e4m3(const void* q8, const void* k_self8, const void* v_self8, const sdvg_cache* c,
                             int64_t block_index, const float* qk_descale, const float* v_descale, void* out,
                             float* lse, float scale, void* workspace, size_t workspace_bytes, void* stream_) {
  SDVG_RANGE();
  if (!c) return SDVG_ERR_INVALID_ARG;
  const void* const qs[1] = {q8};
  const void* const ks[1] = {k_self8};
  const void* const vs[1] = {v_self8};
  void* const outs[1] = {out};
  float* const lses[1] = {lse};
  const float* const qkd[1] = {qk_descale};
  const float* const vd[1] = {v_descale};
  return attn_forward_batch(1, qs, k_self8 ? ks : nullptr, v_self8 ? vs : nullptr, &c, &block_index, outs, lses, scale,
                            workspace, workspace_bytes, (cudaStream_t)stream_, 1, qkd, vd);
}

int sdvg_block_attn_fwd_e4m3_batched(int batch, const void* const* q8, const void* const* k_self8,
                                     const void* const* v_self8, const sdvg_cache* const* caches,
                                     const int64_t* block_index, const float* const* qk_descale,
                                     const float* const* v_descale, void* const* out, float* const* lse, float scale,
                                     void* workspace, size_t workspace_bytes, void* stream_) {
  SDVG_RANGE();
  return attn_forward_batch(batch, q8, k_self8, v_self8, caches, block_index, out, lse, scale, workspace,
                            workspace_bytes, (cudaStream_t)stream_, 1, qk_descale, v_descale);
}

int sdvg_block_attn_fwd_e4m3_tiled(const void* q8, const float* q_tile_scale, const sdvg_cache* c, int64_t block_index,
                                   void* out, float* lse, float scale, void* workspace, size_t workspace_bytes,
                                   void* stream_) {
  SDVG_RANGE();
  if (!q8 || !q_tile_scale || !c || !out || !workspace) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1 || c->slots > 16) return SDVG_ERR_BAD_SHAPE;
  if (!c->k_tile_scale || !c->v_tile_scale) return SDVG_ERR_BAD_STATE;
  if (workspace_bytes < (size_t)kWorkspaceBytes) return SDVG_ERR_INVALID_ARG;
  if (!(scale > 0.f) || !isfinite(scale)) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SDVG_ERR_MISALIGNED;
  if (!sdvg::aligned16(q8) || !sdvg::aligned16(out) ||
      ((reinterpret_cast<uintptr_t>(lse) | reinterpret_cast<uintptr_t>(q_tile_scale)) & 3))
    return SDVG_ERR_MISALIGNED;
  // the block's own K/V must sit staged in its slot: this variant reads keys from the ring only
  if (block_index < 0 || block_index != c->next_block || c->staged_block != block_index) return SDVG_ERR_BAD_STATE;
  const int T = c->block_tokens, H = c->heads, S = c->slots;
  AttnParams p = {};
  const int64_t first = block_index - (S - 1) > 0 ? block_index - (S - 1) : 0;
  for (int64_t b = first; b <= block_index; ++b) {
    const int s = (int)(b % S);
    if (b < block_index && c->slot_block[s] != b) return SDVG_ERR_BAD_STATE;
    p.ts_slot[p.ts_nslots++] = (unsigned char)s;
  }
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  p.batch = 1;
  p.tokens = T;
  p.heads = H;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.work = (unsigned int*)workspace;
  p.nseg = 1;                                       // one (4-D) map per tensor
  p.ts_tiles = sdvg::scale_tiles(T);
  p.ts_cache_slots = S;
  AttnProblem& pr = p.prob[0];
  pr.out = (__nv_bfloat16*)out;
  pr.lse = lse;
  pr.q_tile_scale = q_tile_scale;
  pr.k_tile_scale = c->k_tile_scale;
  pr.v_tile_scale = c->v_tile_scale;
  if ((st = make_map(&pr.q_map, q8, 128, T, H, (size_t)H * 128, 128, 1)) != SDVG_OK) return st;
  if ((st = make_ring_map(&pr.k_map[0], c->k_buf, T, S, H)) != SDVG_OK) return st;
  if ((st = make_ring_map(&pr.v_map[0], c->v_buf, T, S, H)) != SDVG_OK) return st;
  return launch_ws<128, true, true>(p, (cudaStream_t)stream_);
}

int sdvg_block_attn_fwd_noalloc(const void* q, const void* k_self, const void* v_self, const sdvg_cache* c,
                                int64_t block_index, void* out, float* lse, float scale,
                                void** scratch_device_ptr, void* stream_) {
  SDVG_RANGE();
  static std::mutex mu;
  static void* scratch_of_device[kMaxDevices] = {};
  // The built-in scratch has a fixed size; refuse rather than overrun if the kernel ever needs more.
  if (sdvg_block_attn_workspace_bytes() > sizeof(g_noalloc_scratch)) return SDVG_ERR_BAD_SHAPE;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  if (dev < 0 || dev >= kMaxDevices) return SDVG_ERR_INVALID_ARG;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!scratch_of_device[dev]) {
      // once per device, with that device current: ask the runtime where this device's copy lives
      void* ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
      if (e != cudaSuccess) return sdvg::cuda_status(e);
      scratch_of_device[dev] = ptr;
    }
    scratch = scratch_of_device[dev];
  }
  if (scratch_device_ptr) *scratch_device_ptr = scratch;
  return attn_forward(q, k_self, v_self, c, block_index, out, lse, scale, scratch, sizeof(g_noalloc_scratch),
                      (cudaStream_t)stream_);
}

int sdvg_selftest_bounded_wait(void* workspace, size_t workspace_bytes, unsigned long long limit_ns, void* stream_) {
  if (!workspace || workspace_bytes < (size_t)kWorkspaceBytes) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SDVG_ERR_MISALIGNED;
  if (limit_ns == 0 || limit_ns > 1000000000ull) return SDVG_ERR_INVALID_ARG;     // at most one second
  int st = sdvg::require_sm100();
  if (st != SDVG_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  cudaError_t e = cudaMemsetAsync(workspace, 0, kWorkspaceBytes, stream);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>((unsigned int*)workspace, limit_ns);
  return sdvg::cuda_status(cudaGetLastError());
}

int sdvg_block_attn_status(const void* workspace, void* stream_) {
  if (!workspace) return SDVG_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  unsigned int w[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(w, workspace, sizeof(w), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  return w[1] == 0 ? SDVG_OK : (int)w[1];
}

int sdvg_block_attn_rescale_events(const void* workspace, unsigned long long* events, void* stream_) {
  if (!workspace || !events) return SDVG_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  unsigned int w[3] = {0, 0, 0};
  cudaError_t e = cudaMemcpyAsync(w, workspace, sizeof(w), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return sdvg::cuda_status(e);
  *events = w[2];
  return SDVG_OK;
}

}  // extern "C"
