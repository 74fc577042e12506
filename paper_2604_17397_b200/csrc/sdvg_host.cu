// Host-side parts of libsdvg: status text, error bookkeeping, device check,
// RoPE table builder and the ring-cache handle (Sec. 3 "Inference flow").
#include <math.h>
#include <new>

#include "sdvg_internal.h"

namespace {
thread_local int g_last_cuda_error = 0;
}

namespace sdvg {

int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return SDVG_OK;
  g_last_cuda_error = (int)e;
  return SDVG_ERR_CUDA;
}

int require_sm100() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_status(e);
  static thread_local int cached_dev = -1;
  static thread_local int cached_major = 0;
  if (cached_dev != dev) {
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_status(e);
    cached_dev = dev;
    cached_major = major;
  }
  return cached_major == 10 ? SDVG_OK : SDVG_ERR_UNSUPPORTED_ARCH;
}

int ring_begin_commit(sdvg_cache* c, int64_t block_index, int flags, int* slot) {
  if (!c) return SDVG_ERR_INVALID_ARG;
  if (flags != SDVG_STAGE && flags != SDVG_FINAL) return SDVG_ERR_INVALID_ARG;
  if (block_index < 0 || block_index != c->next_block) return SDVG_ERR_BAD_STATE;
  *slot = (int)(block_index % c->slots);
  return SDVG_OK;
}

void ring_end_commit(sdvg_cache* c, int64_t block_index, int flags, int slot, int64_t* evicted) {
  if (flags == SDVG_STAGE) {
    // The slot map keeps naming the previous occupant (block_index - slots) until the FINAL
    // commit reports it as evicted; that block is already outside the window of block_index.
    c->staged_block = block_index;
    if (evicted) *evicted = -1;
    return;
  }
  if (evicted) *evicted = c->slot_block[slot];
  c->slot_block[slot] = block_index;
  c->next_block = block_index + 1;
  c->staged_block = -1;
}

}  // namespace sdvg

extern "C" {

const char* sdvg_status_string(int status) {
  switch (status) {
    case SDVG_OK: return "ok";
    case SDVG_ERR_INVALID_ARG: return "invalid argument";
    case SDVG_ERR_BAD_SHAPE: return "bad shape";
    case SDVG_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case SDVG_ERR_BAD_STATE: return "bad state";
    case SDVG_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case SDVG_ERR_CUDA: return "CUDA error";
    case SDVG_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int sdvg_last_cuda_error(void) { return g_last_cuda_error; }

const char* sdvg_last_cuda_error_string(void) {
  return cudaGetErrorString((cudaError_t)g_last_cuda_error);
}

int sdvg_rope3d_pairs(int head_dim, int* pf, int* ph, int* pw) {
  if (head_dim <= 0 || (head_dim & 1)) return SDVG_ERR_BAD_SHAPE;
  int hw = head_dim / 6;
  if (pf) *pf = head_dim / 2 - 2 * hw;
  if (ph) *ph = hw;
  if (pw) *pw = hw;
  return SDVG_OK;
}

size_t sdvg_rope3d_table_floats(int head_dim, int tab_frames, int grid_h, int grid_w) {
  int pf, ph, pw;
  if (sdvg_rope3d_pairs(head_dim, &pf, &ph, &pw) != SDVG_OK) return 0;
  if (tab_frames <= 0 || grid_h <= 0 || grid_w <= 0) return 0;
  return 2 * ((size_t)tab_frames * pf + (size_t)grid_h * ph + (size_t)grid_w * pw);
}

int sdvg_rope3d_table(float* out, int head_dim, int tab_frames, int grid_h, int grid_w) {
  if (!out) return SDVG_ERR_INVALID_ARG;
  if (sdvg_rope3d_table_floats(head_dim, tab_frames, grid_h, grid_w) == 0) return SDVG_ERR_BAD_SHAPE;
  int pairs[3];
  sdvg_rope3d_pairs(head_dim, &pairs[0], &pairs[1], &pairs[2]);
  const int npos[3] = {tab_frames, grid_h, grid_w};
  size_t o = 0;
  for (int axis = 0; axis < 3; ++axis) {
    const int P = pairs[axis];
    for (int pos = 0; pos < npos[axis]; ++pos) {
      for (int i = 0; i < P; ++i) {
        // pair i of an axis with P pairs turns by pos * 10000^(-i/P)
        double omega = pow(10000.0, -((double)i / (double)P));
        double a = (double)pos * omega;
        out[o++] = (float)cos(a);
        out[o++] = (float)sin(a);
      }
    }
  }
  return SDVG_OK;
}

size_t sdvg_cache_bytes(int slots, int heads, int block_tokens, int head_dim) {
  if (slots <= 0 || heads <= 0 || block_tokens <= 0 || !sdvg::head_dim_ok(head_dim)) return 0;
  return (size_t)slots * heads * block_tokens * head_dim * 2;
}

int sdvg_cache_create(sdvg_cache** out, void* k_buf, void* v_buf, int slots, int heads,
                      int block_tokens, int head_dim) {
  if (!out || !k_buf || !v_buf) return SDVG_ERR_INVALID_ARG;
  if (sdvg_cache_bytes(slots, heads, block_tokens, head_dim) == 0) return SDVG_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(k_buf) & 1023u) || (reinterpret_cast<uintptr_t>(v_buf) & 1023u))
    return SDVG_ERR_MISALIGNED;
  sdvg_cache* c = new (std::nothrow) sdvg_cache;
  if (!c) return SDVG_ERR_INVALID_ARG;
  c->k_buf = k_buf;
  c->v_buf = v_buf;
  c->slots = slots;
  c->heads = heads;
  c->block_tokens = block_tokens;
  c->head_dim = head_dim;
  c->elem_bytes = 2;
  c->next_block = 0;
  c->staged_block = -1;
  c->slot_block.assign(slots, -1);
  *out = c;
  return SDVG_OK;
}

size_t sdvg_cache_bytes_e4m3(int slots, int heads, int block_tokens, int head_dim) {
  if (head_dim != 128) return 0;
  return sdvg_cache_bytes(slots, heads, block_tokens, head_dim) / 2;
}

int sdvg_cache_create_e4m3(sdvg_cache** out, void* k_buf, void* v_buf, int slots, int heads, int block_tokens,
                           int head_dim) {
  if (slots > 0 && heads > 0 && block_tokens > 0 && sdvg::head_dim_ok(head_dim) && head_dim != 128)
    return SDVG_ERR_BAD_SHAPE;
  const int st = sdvg_cache_create(out, k_buf, v_buf, slots, heads, block_tokens, head_dim);
  if (st == SDVG_OK) (*out)->elem_bytes = 1;
  return st;
}

size_t sdvg_cache_tile_scale_floats(int slots, int heads, int block_tokens) {
  if (slots <= 0 || heads <= 0 || block_tokens <= 0) return 0;
  return (size_t)slots * heads * sdvg::scale_tiles(block_tokens);
}

int sdvg_cache_set_tile_scales(sdvg_cache* c, float* k_scale, float* v_scale) {
  if (!c || !k_scale || !v_scale) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != 1) return SDVG_ERR_BAD_SHAPE;
  if ((reinterpret_cast<uintptr_t>(k_scale) | reinterpret_cast<uintptr_t>(v_scale)) & 3) return SDVG_ERR_MISALIGNED;
  c->k_tile_scale = k_scale;
  c->v_tile_scale = v_scale;
  return SDVG_OK;
}

int sdvg_cache_reset(sdvg_cache* c) {
  if (!c) return SDVG_ERR_INVALID_ARG;
  c->next_block = 0;
  c->staged_block = -1;
  c->slot_block.assign(c->slots, -1);
  return SDVG_OK;
}

int sdvg_cache_destroy(sdvg_cache* c) {
  if (!c) return SDVG_ERR_INVALID_ARG;
  delete c;
  return SDVG_OK;
}

int sdvg_cache_state(const sdvg_cache* c, int64_t* next_block, int64_t* slot_block,
                     int64_t* staged_block) {
  if (!c) return SDVG_ERR_INVALID_ARG;
  if (next_block) *next_block = c->next_block;
  if (staged_block) *staged_block = c->staged_block;
  if (slot_block)
    for (int s = 0; s < c->slots; ++s) slot_block[s] = c->slot_block[s];
  return SDVG_OK;
}

}  // extern "C"
