// Internal host-side declarations shared by the translation units of libsdvg.
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include <vector>

#include "sdvg.h"

struct sdvg_cache {
  void* k_buf;
  void* v_buf;
  int slots, heads, block_tokens, head_dim;
  int elem_bytes;                       // 2: bf16 elements; 1: E4M3 codes (8-bit variant)
  int64_t next_block;
  int64_t staged_block;                 // block whose provisional K/V sit in its slot, -1 if none
  std::vector<int64_t> slot_block;      // slot -> committed block, -1 = empty
  // 8-bit ring with one power-of-two scale per (head, slot, tile of 128 tokens): device fp32 [heads][slots][tiles],
  // caller-owned like the rings; null until sdvg_cache_set_tile_scales
  float* k_tile_scale = nullptr;
  float* v_tile_scale = nullptr;
};

namespace sdvg {

// NVTX range over the host side of an entry point (argument checks, tensor maps, launch): a timeline
// tool then shows which library call enqueued which kernels.  Costs a function-pointer test when no
// tool is attached.
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
  Range(const Range&) = delete;
  Range& operator=(const Range&) = delete;
};
#define SDVG_RANGE() ::sdvg::Range sdvg_range_(__func__)

// Records a CUDA error for sdvg_last_cuda_error() and maps it to a status.
int cuda_status(cudaError_t e);

// SDVG_OK if the current device is compute capability 10.x (cached per device).
int require_sm100();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool head_dim_ok(int d) { return d == 64 || d == 128; }

constexpr int kScaleTileTokens = 128;   // tokens per scale tile of the tile-scaled 8-bit ring
inline int scale_tiles(int block_tokens) { return (block_tokens + kScaleTileTokens - 1) / kScaleTileTokens; }

// Element (not byte) offset of (head, slot, token 0, dim 0) in a cache buffer laid out [heads][slots][tokens][dim].
inline size_t slot_offset(const sdvg_cache* c, int head, int slot) {
  return ((size_t)head * c->slots + slot) * (size_t)c->block_tokens * c->head_dim;
}

// Host-side ring bookkeeping shared by the commit entry points; returns a status and,
// on success, the slot to write and (for SDVG_FINAL) the evicted block.
int ring_begin_commit(sdvg_cache* c, int64_t block_index, int flags, int* slot);
void ring_end_commit(sdvg_cache* c, int64_t block_index, int flags, int slot, int64_t* evicted);

}  // namespace sdvg
