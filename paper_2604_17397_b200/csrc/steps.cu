// The denoising steps of one block in one call (Sec. 4.1 "Models": 4 denoising steps per block; Sec. 3
// "Inference flow": every drafter and target step pays this path).  Each step is the fused prologue
// (3D-RoPE of q and k, provisional write of k', v into the block's ring slot) followed by the block
// attention against the ring.  The call only strings the library's own entry points together on the
// caller's stream, after checking every step's arguments first, so that a caller's CUDA-graph capture of a
// block (or a plain eager loop) is one call instead of 2 S.
#include "sdvg_internal.h"

namespace {

// Everything that can be refused without touching the device, for all steps, before the first launch.
int check_steps(int steps, const sdvg_cache* c, const void* const* q, const void* const* k, const void* const* v,
                void* const* q_roped, void* const* out, int64_t block_index, const void* workspace,
                size_t workspace_bytes, float scale, int want_elem_bytes) {
  if (steps < 1 || steps > 64) return SDVG_ERR_BAD_SHAPE;
  if (!c || !q || !k || !v || !q_roped || !out || !workspace) return SDVG_ERR_INVALID_ARG;
  if (c->elem_bytes != want_elem_bytes) return SDVG_ERR_BAD_SHAPE;
  if (workspace_bytes < sdvg_block_attn_workspace_bytes()) return SDVG_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SDVG_ERR_MISALIGNED;
  if (!(scale > 0.f) || scale != scale || scale > 3.0e38f) return SDVG_ERR_INVALID_ARG;
  if (block_index < 0 || block_index != c->next_block) return SDVG_ERR_BAD_STATE;
  for (int s = 0; s < steps; ++s) {
    if (!q[s] || !k[s] || !v[s] || !q_roped[s] || !out[s]) return SDVG_ERR_INVALID_ARG;
    if (!sdvg::aligned16(q[s]) || !sdvg::aligned16(k[s]) || !sdvg::aligned16(v[s]) || !sdvg::aligned16(q_roped[s]) ||
        !sdvg::aligned16(out[s]))
      return SDVG_ERR_MISALIGNED;
  }
  return SDVG_OK;
}

}  // namespace

extern "C" {

int sdvg_block_steps(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                     const void* const* v, void* const* q_roped, void* const* out, int frames, int grid_h,
                     int grid_w, int frame_offset, const float* cos_sin_tab, int tab_frames, int64_t block_index,
                     float scale, void* workspace, size_t workspace_bytes, void* stream) {
  SDVG_RANGE();
  int st = check_steps(steps, cache, q, k, v, q_roped, out, block_index, workspace, workspace_bytes, scale, 2);
  if (st != SDVG_OK) return st;
  for (int s = 0; s < steps; ++s) {
    // the first prologue also checks the grid, the table and the device; after it nothing below can be refused
    st = sdvg_rope3d_qk_commit(cache, q[s], k[s], v[s], q_roped[s], nullptr, frames, grid_h, grid_w, frame_offset,
                               cos_sin_tab, tab_frames, block_index, SDVG_STAGE, nullptr, stream);
    if (st != SDVG_OK) return st;
    st = sdvg_block_attn_fwd(q_roped[s], nullptr, nullptr, cache, block_index, out[s], nullptr, scale, workspace,
                             workspace_bytes, stream);
    if (st != SDVG_OK) return st;
  }
  return SDVG_OK;
}

int sdvg_block_steps_e4m3(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                          const void* const* v, void* const* q8_roped, void* const* out,
                          const float* q_inv_scale, const float* k_inv_scale, const float* v_inv_scale,
                          const float* qk_descale, const float* v_descale, int frames, int grid_h, int grid_w,
                          int frame_offset, const float* cos_sin_tab, int tab_frames, int64_t block_index, float scale,
                          void* workspace, size_t workspace_bytes, void* stream) {
  SDVG_RANGE();
  int st = check_steps(steps, cache, q, k, v, q8_roped, out, block_index, workspace, workspace_bytes, scale, 1);
  if (st != SDVG_OK) return st;
  if (!q_inv_scale || !k_inv_scale || !v_inv_scale || !qk_descale || !v_descale) return SDVG_ERR_INVALID_ARG;
  for (int s = 0; s < steps; ++s) {
    st = sdvg_rope3d_qk_commit_e4m3(cache, q[s], k[s], v[s], q8_roped[s], q_inv_scale, k_inv_scale, v_inv_scale, frames,
                                    grid_h, grid_w, frame_offset, cos_sin_tab, tab_frames, block_index, SDVG_STAGE,
                                    nullptr, stream);
    if (st != SDVG_OK) return st;
    st = sdvg_block_attn_fwd_e4m3(q8_roped[s], nullptr, nullptr, cache, block_index, qk_descale, v_descale, out[s],
                                  nullptr, scale, workspace, workspace_bytes, stream);
    if (st != SDVG_OK) return st;
  }
  return SDVG_OK;
}

int sdvg_block_steps_e4m3_tiled(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                                const void* const* v, void* const* q8_roped, float* const* q_tile_scale,
                                void* const* out, int frames, int grid_h, int grid_w, int frame_offset,
                                const float* cos_sin_tab, int tab_frames, int64_t block_index, float scale,
                                void* workspace, size_t workspace_bytes, void* stream) {
  SDVG_RANGE();
  int st = check_steps(steps, cache, q, k, v, q8_roped, out, block_index, workspace, workspace_bytes, scale, 1);
  if (st != SDVG_OK) return st;
  if (!q_tile_scale) return SDVG_ERR_INVALID_ARG;
  if (!cache->k_tile_scale || !cache->v_tile_scale) return SDVG_ERR_BAD_STATE;
  if (cache->slots > 16) return SDVG_ERR_BAD_SHAPE;
  for (int s = 0; s < steps; ++s) {
    if (!q_tile_scale[s]) return SDVG_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(q_tile_scale[s]) & 3) return SDVG_ERR_MISALIGNED;
  }
  for (int s = 0; s < steps; ++s) {
    st = sdvg_rope3d_qk_commit_e4m3_tiled(cache, q[s], k[s], v[s], q8_roped[s], q_tile_scale[s], frames, grid_h, grid_w,
                                          frame_offset, cos_sin_tab, tab_frames, block_index, SDVG_STAGE, nullptr, stream);
    if (st != SDVG_OK) return st;
    st = sdvg_block_attn_fwd_e4m3_tiled(q8_roped[s], q_tile_scale[s], cache, block_index, out[s], nullptr, scale,
                                        workspace, workspace_bytes, stream);
    if (st != SDVG_OK) return st;
  }
  return SDVG_OK;
}

}  // extern "C"
