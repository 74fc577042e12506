/*
 * sdvg.h — C ABI of the SDVG hot-path library for NVIDIA B200 (sm_100a).
 *
 * The library implements what every drafter and target denoising step of SDVG
 * (speculative decoding for block-autoregressive video diffusion) pays in its
 * attention backbone (Sec. 4.1 "Models": causal attention over a KV cache, rotary
 * positions, bf16) plus the routing rule of Sec. 3:
 *
 *   sdvg_rope3d_qk        3D rotary embedding (frame, row, column) of q and k
 *   sdvg_block_attn_fwd   a block of latent frames attends to itself (all keys
 *                         visible) and to the earlier blocks held in a rolling cache
 *   sdvg_kv_commit        write a block's K/V into its ring slot, evicting the oldest
 *   sdvg_route            worst-frame minimum against tau, block 0 always rejected
 *
 * Conventions
 *   - Every function returns an int status (SDVG_OK == 0).  Nothing throws or
 *     aborts.  All argument and state checks happen on the host before any
 *     launch; a call that returns an error has enqueued nothing.
 *   - "device" pointers are CUDA device memory owned by the caller; "host"
 *     pointers are ordinary host memory.  The library allocates no device memory.
 *   - bf16 tensors are [tokens, heads, head_dim], head_dim contiguous, tokens of
 *     a block ordered frame-major, then grid row, then grid column.  All tensor
 *     pointers must be 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Kernels are enqueued on it; the library never synchronises the device
 *     unless a function says so.
 *   - Functions that take a cache mutate only host metadata of that handle
 *     besides enqueuing work; a handle must not be used from two threads at once.
 */
#ifndef SDVG_H_
#define SDVG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------ */
#define SDVG_OK                   0
#define SDVG_ERR_INVALID_ARG      1   /* NULL pointer, negative size, unknown flag */
#define SDVG_ERR_BAD_SHAPE        2   /* sizes inconsistent or unsupported (head_dim not 64/128, F=0, ...) */
#define SDVG_ERR_MISALIGNED       3   /* a tensor pointer is not 16-byte aligned */
#define SDVG_ERR_BAD_STATE        4   /* block out of order, self not staged, frame outside the table, ... */
#define SDVG_ERR_UNSUPPORTED_ARCH 5   /* current device is not compute capability 10.x */
#define SDVG_ERR_CUDA             6   /* a CUDA call failed: see sdvg_last_cuda_error() */
#define SDVG_ERR_TIMEOUT          7   /* a bounded device-side wait gave up (reported by sdvg_block_attn_status) */

/* ---- commit flags ------------------------------------------------------ */
#define SDVG_STAGE 1   /* write the slot of the block being generated; ring state unchanged */
#define SDVG_FINAL 2   /* write the slot, record the block as committed, advance to the next block */

const char* sdvg_status_string(int status);
/* Last cudaError_t seen by this thread inside the library (0 if none) and its text. */
int         sdvg_last_cuda_error(void);
const char* sdvg_last_cuda_error_string(void);

/* ---- 3D RoPE ----------------------------------------------------------- */
/*
 * Pair split of the head dimension (Sec. 4.1 names RoPE only; the split is the
 * Wan-family convention): height and width own floor(D/6) (even, odd) pairs
 * each, the frame axis the remaining D/2 - 2*floor(D/6).  Pair i of an axis
 * with P pairs rotates by position * 10000^(-i/P).
 */
int sdvg_rope3d_pairs(int head_dim, int* pairs_frame, int* pairs_height, int* pairs_width);

/*
 * (cos, sin) table in fp32, the numeric input that fixes RoPE results to the bit.
 * Layout: for frame positions 0..tab_frames-1, P_f (cos, sin) pairs each; then
 * for rows 0..grid_h-1, P_h pairs each; then for columns 0..grid_w-1, P_w pairs
 * each.  Angles are formed and evaluated in fp64 and rounded once to fp32.
 * sdvg_rope3d_table_floats returns the number of floats (0 on bad arguments);
 * sdvg_rope3d_table fills a HOST buffer of that size.  The caller uploads it.
 */
size_t sdvg_rope3d_table_floats(int head_dim, int tab_frames, int grid_h, int grid_w);
int    sdvg_rope3d_table(float* host_out, int head_dim, int tab_frames, int grid_h, int grid_w);

/*
 * Rotate q and k (device, bf16 [tokens, heads, head_dim]) into q_out, k_out
 * (same layout; in-place allowed, q_out==q and/or k_out==k).  Either pair
 * (q, q_out) or (k, k_out) may be NULL/NULL to rotate only one tensor.
 * tokens must equal frames*grid_h*grid_w; token n sits at frame
 * frame_offset + n/(grid_h*grid_w), row (n/grid_w)%grid_h, column n%grid_w.
 * Arithmetic (per pair, c/s from the table): re' = fl(fl(re*c) - fl(im*s)),
 * im' = fl(fl(re*s) + fl(im*c)) in IEEE fp32 without fused multiply-add,
 * then round-to-nearest-even to bf16.
 * cos_sin_tab: device copy of the table built for (head_dim, tab_frames, grid_h, grid_w).
 * Errors: BAD_SHAPE (head_dim not 64/128, tokens mismatch), BAD_STATE
 * (frame_offset < 0 or frame_offset+frames > tab_frames), MISALIGNED, INVALID_ARG.
 */
int sdvg_rope3d_qk(const void* q, const void* k, void* q_out, void* k_out,
                   int tokens, int heads, int head_dim,
                   int frames, int grid_h, int grid_w, int frame_offset,
                   const float* cos_sin_tab, int tab_frames, void* stream);

/* ---- rolling KV cache (Sec. 3 "Inference flow": K^D and K^T) ------------- */
typedef struct sdvg_cache sdvg_cache;   /* opaque; owns host metadata only */

/* Bytes of ONE buffer (K or V) for the given shape; 0 on bad arguments. */
size_t sdvg_cache_bytes(int slots, int heads, int block_tokens, int head_dim);

/*
 * Bind a cache handle to two caller-owned device buffers of sdvg_cache_bytes()
 * each, 1024-byte aligned.  Physical layout of each buffer (library's choice,
 * readable through sdvg_cache_read_block): [heads][slots][block_tokens][head_dim]
 * bf16, so that one head's ring is one contiguous run of keys.  Block b lives in
 * slot b % slots.  slots = visible earlier blocks + 1.  The buffers are not
 * cleared; empty slots are never read.
 */
int sdvg_cache_create(sdvg_cache** out, void* k_buf, void* v_buf,
                      int slots, int heads, int block_tokens, int head_dim);
int sdvg_cache_reset(sdvg_cache* cache);      /* forget all blocks (host state only) */
int sdvg_cache_destroy(sdvg_cache* cache);    /* frees the handle, not the buffers */
/*
 * Host-side ring state: next block to be generated, slot -> committed block
 * (-1 = empty; slot_block may be NULL or an array of `slots` entries) and the
 * block currently staged (-1 if none; may be NULL).
 */
int sdvg_cache_state(const sdvg_cache* cache, int64_t* next_block, int64_t* slot_block,
                     int64_t* staged_block);
/* Gather one slot back into logical [block_tokens, heads, head_dim] device tensors (either may be NULL). */
int sdvg_cache_read_block(const sdvg_cache* cache, int slot, void* k_out, void* v_out, void* stream);

/*
 * Commit (Sec. 3: the drafter cache is updated with every draft block; the
 * target cache receives the accepted draft block or the regenerated one).
 * Copies k_roped and v (device, bf16 [block_tokens, heads, head_dim]) into slot
 * block_index % slots.  block_index must be the cache's next block.
 * SDVG_STAGE: provisional write used once per denoise step so that attention
 *   can read the block from the ring; the block it overwrites (block_index -
 *   slots) is already outside the window of block_index.
 * SDVG_FINAL: also records the block and advances next_block; *evicted_block
 *   (host, may be NULL) receives the block that left the slot, -1 if it was empty
 *   (always -1 for SDVG_STAGE).
 * Errors: BAD_STATE (out of order), INVALID_ARG (flags), MISALIGNED.
 */
int sdvg_kv_commit(sdvg_cache* cache, const void* k_roped, const void* v,
                   int64_t block_index, int flags, int64_t* evicted_block, void* stream);

/*
 * Fused step prologue: q_out = rope(q); rope(k) and v go straight into the ring
 * slot of block_index with the semantics of `flags` above; k_out (optional)
 * also receives rope(k) in the logical layout.  Bit-identical to
 * sdvg_rope3d_qk followed by sdvg_kv_commit.  frame_offset is the first
 * absolute latent frame of the block.  q/q_out may be NULL/NULL.
 */
int sdvg_rope3d_qk_commit(sdvg_cache* cache, const void* q, const void* k, const void* v,
                          void* q_out, void* k_out,
                          int frames, int grid_h, int grid_w, int frame_offset,
                          const float* cos_sin_tab, int tab_frames,
                          int64_t block_index, int flags, int64_t* evicted_block, void* stream);

/* ---- block attention ---------------------------------------------------- */
/*
 * Device scratch needed by sdvg_block_attn_fwd (a few hundred bytes: a work
 * counter and a status word).  256-byte aligned, caller-owned, must not be
 * shared by calls that overlap on the device.  The status word is STICKY: a
 * kernel whose bounded wait gave up raises it to SDVG_ERR_TIMEOUT and no later
 * launch lowers it again, so one check after a sequence of steps (before their
 * results are committed) is enough.  Clear a new workspace, and a workspace whose
 * error has been handled, with sdvg_block_attn_workspace_reset.
 */
size_t sdvg_block_attn_workspace_bytes(void);

/*
 * Zeroes the workspace on `stream` (a memset, no kernel).  Call it once after
 * allocating the buffer and again after a reported SDVG_ERR_TIMEOUT has been dealt with.
 * Errors: INVALID_ARG (NULL or too small), MISALIGNED, CUDA.
 */
int sdvg_block_attn_workspace_reset(void* workspace, size_t workspace_bytes, void* stream);

/*
 * out[i, h, :] = sum_j softmax_j(scale * <q[i,h,:], K[j,h,:]>) V[j,h,:] where j
 * runs over every token of the committed blocks visible to block_index (the
 * last slots-1 blocks before it) and of block_index itself; no key is masked:
 * bidirectional inside the block, causal across blocks (Sec. 4.1 "Models": both
 * models attend causally over a KV cache; Sec. 1: a block is conditioned on
 * earlier content through that cache).
 *   q, out        device bf16 [block_tokens, heads, head_dim] of the cache's shape
 *   k_self/v_self device bf16, same shape, the block's own roped K and V; both
 *                 NULL means the block was staged (SDVG_STAGE) and is read from the ring
 *   lse           optional device fp32 [heads, block_tokens]: log-sum-exp of the scaled logits
 *   block_index   must be the cache's next block
 * bf16 tensor-core products with fp32 accumulation, fp32 online softmax,
 * probabilities rounded to bf16 before the second product.
 * Errors: BAD_STATE (wrong block, self not staged), BAD_SHAPE, MISALIGNED,
 * INVALID_ARG (workspace too small), UNSUPPORTED_ARCH, CUDA.
 */
int sdvg_block_attn_fwd(const void* q, const void* k_self, const void* v_self,
                        const sdvg_cache* cache, int64_t block_index,
                        void* out, float* lse, float scale,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same attention for `batch` independent problems of one shape in one call (at most 4): the two
 * passes of classifier-free guidance (Sec. 4.1 samples with guidance scale 3.0, i.e. a conditional and an
 * unconditional pass per denoising step), or several videos.  q, k_self, v_self, caches, block_index, out
 * and lse are HOST arrays of `batch` entries holding what sdvg_block_attn_fwd takes for one problem
 * (k_self and v_self may be NULL as arrays = every problem staged; lse may be NULL as an array, or hold
 * NULL entries).  All caches must have the same block_tokens, heads and head_dim.  Problems whose visible
 * key segments agree (same ring fill, same staging: the normal case) are processed by ONE launch whose
 * work items span all problems, which is what fills the GPU at the drafter's shape; otherwise the
 * problems are launched one after the other on `stream`.  Results are those of `batch` separate calls up to
 * the order of one summation: how a launch deals its query tiles to the SMs depends on how many tiles it has, and a
 * tile is either processed whole or with its keys split into two partial results that are merged at the end.
 * Where both launches treat a tile alike (always when neither has more than two tiles per SM) the bits agree.
 * Errors: those of sdvg_block_attn_fwd; BAD_SHAPE for batch > 4 or mismatched cache shapes.
 */
int sdvg_block_attn_fwd_batched(int batch, const void* const* q, const void* const* k_self,
                                const void* const* v_self, const sdvg_cache* const* caches,
                                const int64_t* block_index, void* const* out, float* const* lse, float scale,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronises `stream` and reports the status word of `workspace`: SDVG_OK, or
 * SDVG_ERR_TIMEOUT if a bounded wait inside ANY attention launch on this
 * workspace since its last reset gave up (the outputs of that launch and of
 * everything computed from them are then undefined).  Reading does not clear it.
 */
int sdvg_block_attn_status(const void* workspace, void* stream);

/*
 * Diagnostic: synchronises `stream` and writes to *events (host) how many times, since the last reset of
 * `workspace`, a warp of an attention kernel took the path that rescales the output accumulator because the
 * reference maximum of one of its query rows moved (the online-softmax correction; with the lazy reference
 * it is rare on ordinary data and frequent when the logits keep rising along the keys).  Tests use it to
 * prove that this path ran.
 */
int sdvg_block_attn_rescale_events(const void* workspace, unsigned long long* events, void* stream);

/*
 * Self-test of the bounded device-side wait (no counterpart in the paper; it backs the promise that a
 * stuck attention kernel returns instead of hanging the GPU).  Launches one warp that waits, through the
 * wait the attention kernel uses, for an mbarrier phase that nothing will ever complete, with a limit of
 * limit_ns nanoseconds (1 .. 1e9).  The warp must give up after the limit, record SDVG_ERR_TIMEOUT in the
 * status word of `workspace` and exit normally; sdvg_block_attn_status(workspace) then returns
 * SDVG_ERR_TIMEOUT and the context stays usable.  workspace: as for sdvg_block_attn_fwd.
 */
int sdvg_selftest_bounded_wait(void* workspace, size_t workspace_bytes, unsigned long long limit_ns, void* stream);

/*
 * Same computation as sdvg_block_attn_fwd for callers that cannot allocate device memory
 * (the paper has no counterpart; this is a deployment convenience).  Some hosts of this
 * library run under a fixed memory plan: an inference server that hands every byte of HBM
 * to its own arena at start-up, a plugin called from inside someone else's stream or graph
 * set-up where cudaMalloc would synchronise the device, or a process whose allocator is
 * simply not reachable from the call site.  Such callers have no way to produce the
 * `workspace` buffer, so this entry point brings its own: a 256-byte, 256-byte-aligned array
 * that is part of the library image (every GPU that loads the library holds its own copy
 * until the process exits).  The call itself allocates nothing and frees nothing.
 *
 *   - Limit: the built-in scratch is exactly 256 bytes, which covers every shape the library
 *     supports today.  If a future kernel needed more than that, this function would return
 *     SDVG_ERR_BAD_SHAPE instead of overrunning the array; use sdvg_block_attn_fwd with a
 *     caller-owned workspace in that case.  At most 64 devices per process.
 *   - First call on a device: the function looks up where that device's copy of the array
 *     lives (cudaGetSymbolAddress, with the device current) and remembers it.  Make that first
 *     call outside of any stream capture.
 *   - All calls on a device share the one array and it keeps what the last call left in it.
 *     It starts out zeroed (static initialisation), nothing in it has to be zero at the start
 *     of a call, and the only thing a kernel leaves there is the sticky status word, so no
 *     call clears it.  Two calls that overlap on the GPU (different streams, no ordering
 *     between them) share that word: a timeout is then reported without telling which of
 *     them it was; keep them ordered if that matters.
 *   - *scratch_device_ptr (optional, host) receives the device address of the array, which
 *     can be given to sdvg_block_attn_status to read the status word after the call and to
 *     sdvg_block_attn_workspace_reset (256 bytes) to clear a handled error.
 * Arguments, results and errors are otherwise those of sdvg_block_attn_fwd.
 */
int sdvg_block_attn_fwd_noalloc(const void* q, const void* k_self, const void* v_self,
                                const sdvg_cache* cache, int64_t block_index,
                                void* out, float* lse, float scale,
                                void** scratch_device_ptr, void* stream);

/* ---- router ------------------------------------------------------------- */
/*
 * Eq. (1) and the policy of Sec. 3: q_min[b] = min_i scores[b, i];
 * accept[b] = (first_block_index + b != 0) && (q_min[b] >= tau).
 *   scores        device fp32, flat
 *   frame_offsets device int32 [num_blocks+1] (block b owns scores[offsets[b]..offsets[b+1]))
 *                 or NULL for frames_per_block consecutive scores per block
 *   accept        device u8 [num_blocks]; q_min device fp32 [num_blocks];
 *   argmin        optional device int32 [num_blocks]
 * The minimum is the left-to-right strict-'<' minimum (ties and +0/-0 keep the
 * lowest index); a NaN frame makes q_min that NaN and the block is rejected.
 * With frame_offsets == NULL frames_per_block must be >= 1; with offsets every
 * block must own at least one frame (checked on the device: a block with none
 * gets accept 0, q_min NaN, argmin -1).
 * The offsets must be non-decreasing and the scores buffer must hold at least
 * offsets[num_blocks] floats.  The host cannot read them, so the kernel trusts only
 * the two ends: it never reads outside [offsets[0], offsets[num_blocks]), and a block
 * whose own range runs backwards or leaves that interval is treated as a block
 * without frames.
 * Errors: INVALID_ARG, BAD_SHAPE (num_blocks < 0, frames_per_block < 1).
 */
int sdvg_route(const float* scores, const int32_t* frame_offsets,
               int num_blocks, int frames_per_block, int64_t first_block_index, float tau,
               uint8_t* accept, float* q_min, int32_t* argmin, void* stream);

/*
 * The routing variants of the ablation (Sec. 4.3, Table 2) in one call.
 *   agg     SDVG_AGG_MIN: worst frame, Eq. (1), exactly as sdvg_route;
 *           SDVG_AGG_MEAN: "avg-frame scoring": the frames are added left to right in fp32 (every partial
 *           sum rounded) and the sum is divided by (float)frames with one IEEE division; argmin is -1
 *   signal  SDVG_SIGNAL_REWARD: accept iff aggregate >= tau;
 *           SDVG_SIGNAL_RANDOM: "random routing": accept iff uniforms[b] < accept_prob; the scores only
 *           feed `aggregate`.  The draws are an input (device fp32 [num_blocks], values in [0, 1))
 *   force_first  non-zero: the first block of a video is rejected whatever the signal says ("force-reject
 *           + random" against plain "random routing" in Table 2)
 *   blocks_per_video  0: one stream, only global block 0 is a first block; n > 0: global block g =
 *           first_block_index + b is a first block iff g % n == 0 (a batch of n-block videos, e.g. the
 *           paper's 1003 x 9)
 * accept, aggregate, argmin as in sdvg_route (aggregate takes the place of q_min).
 * Errors: INVALID_ARG (unknown agg/signal, uniforms NULL with SDVG_SIGNAL_RANDOM, blocks_per_video < 0,
 * first_block_index < 0 with blocks_per_video > 0), BAD_SHAPE, MISALIGNED.
 */
#define SDVG_AGG_MIN       0
#define SDVG_AGG_MEAN      1
#define SDVG_SIGNAL_REWARD 0
#define SDVG_SIGNAL_RANDOM 1
int sdvg_route_policy(const float* scores, const int32_t* frame_offsets,
                      int num_blocks, int frames_per_block, int64_t first_block_index, int blocks_per_video,
                      float tau, int agg, int signal, int force_first,
                      const float* uniforms, float accept_prob,
                      uint8_t* accept, float* aggregate, int32_t* argmin, void* stream);

/*
 * Accept-rate statistics with the convention of Tables 1 and 2 (the always-regenerated first block of a
 * video is left out): counts[0] = accepted blocks, counts[1] = routable blocks, both over the blocks that
 * are not first blocks (same first_block_index / blocks_per_video rule as above).  counts: device, two
 * 64-bit integers, 8-byte aligned; cleared by the call on `stream` before the kernel adds to them.
 */
int sdvg_accept_stats(const uint8_t* accept, int num_blocks, int64_t first_block_index, int blocks_per_video,
                      unsigned long long* counts, void* stream);

/* ---- speculative state: snapshot and restore ------------------------------ */
/*
 * Copies `count` device buffers (at most 64) in one launch: dst[i][0 .. bytes[i]) = src[i][0 .. bytes[i]).
 * Sec. 3 "Inference flow": the decoder's cache is cloned before a draft block is decoded and scored, and
 * restored when the router rejects the block; the snapshot is this call, the restore the same call with
 * src and dst exchanged.  src, dst and bytes are HOST arrays; the buffers are device memory, 16-byte aligned,
 * every length a multiple of 16; a source must not overlap a destination.
 * Errors: BAD_SHAPE (count outside 0..64, a length not a multiple of 16), INVALID_ARG, MISALIGNED.
 */
int sdvg_state_copy(const void* const* src, void* const* dst, const size_t* bytes, int count, void* stream);

/* ---- 8-bit (E4M3) variant of the cache and the attention --------------------- */
/*
 * Sec. 2 "Video generation" names quantised attention kernels as speed-ups orthogonal to the method and
 * fixes no number format; this library's choice is the OCP E4M3 byte (1 sign, 4 exponent, 3 mantissa bits,
 * bias 7, no infinities, largest finite value 448) with ONE STATIC SCALE PER HEAD and tensor:
 * x ~ scale[head] * decode(code).  Every routine takes the INVERSE scales for quantising and the plain
 * scales ("descale") for the attention; all scale arrays are device fp32 [heads], positive and finite.
 * The bf16 path above stays the reference path; nothing here changes it.
 */

/*
 * out[t, h, :] = e4m3(x[t, h, :] * inv_scale[h]): the product is one fp32 multiplication (round to nearest),
 * the conversion rounds to nearest even and saturates at +-448 (NaN stays NaN, code 0x7F).
 * x: device bf16 [tokens, heads, head_dim]; out: device bytes, same shape; head_dim 64 or 128.
 * Used for q; k and v go through sdvg_kv_commit_e4m3.  Errors: INVALID_ARG, BAD_SHAPE, MISALIGNED.
 */
int sdvg_quant_e4m3(const void* x, const float* inv_scale, void* out, int tokens, int heads, int head_dim,
                    void* stream);

/* Bytes of ONE of the two buffers of an 8-bit ring (half of sdvg_cache_bytes); 0 unless head_dim is 128. */
size_t sdvg_cache_bytes_e4m3(int slots, int heads, int block_tokens, int head_dim);

/*
 * As sdvg_cache_create, for a ring of E4M3 codes laid out [heads][slots][block_tokens][head_dim] bytes;
 * head_dim must be 128.  The handle works with sdvg_cache_reset / _destroy / _state / _read_block (which
 * then returns bytes), sdvg_kv_commit_e4m3 and sdvg_block_attn_fwd_e4m3; the bf16 entry points answer
 * BAD_SHAPE for it, and the _e4m3 entry points answer BAD_SHAPE for a bf16 ring.
 */
int sdvg_cache_create_e4m3(sdvg_cache** out, void* k_buf, void* v_buf, int slots, int heads, int block_tokens,
                           int head_dim);

/*
 * sdvg_kv_commit for an 8-bit ring: k_roped and v are device bf16 [block_tokens, heads, head_dim] and are
 * quantised on the way into the slot as sdvg_quant_e4m3 does (k with k_inv_scale, v with v_inv_scale).
 * Same ordering rules, flags, eviction report and errors as sdvg_kv_commit.
 */
int sdvg_kv_commit_e4m3(sdvg_cache* cache, const void* k_roped, const void* v, const float* k_inv_scale,
                        const float* v_inv_scale, int64_t block_index, int flags, int64_t* evicted_block,
                        void* stream);

/*
 * sdvg_rope3d_qk_commit for an 8-bit ring, one pass: q8_out = e4m3(rope(q) * q_inv_scale), e4m3(rope(k) *
 * k_inv_scale) and e4m3(v * v_inv_scale) go into the ring slot of block_index.  rope() is the bit-specified
 * rotation of sdvg_rope3d_qk INCLUDING its rounding to bf16, so the result is bit-identical to
 * sdvg_rope3d_qk followed by sdvg_quant_e4m3 (q) and sdvg_kv_commit_e4m3 (k, v).  q, k, v: device bf16
 * [block_tokens, heads, 128]; q8_out: device bytes, same shape; q / q8_out / q_inv_scale may be NULL together.
 * Other arguments and errors as sdvg_rope3d_qk_commit; BAD_SHAPE for a bf16 ring.
 */
int sdvg_rope3d_qk_commit_e4m3(sdvg_cache* cache, const void* q, const void* k, const void* v, void* q8_out,
                               const float* q_inv_scale, const float* k_inv_scale, const float* v_inv_scale,
                               int frames, int grid_h, int grid_w, int frame_offset, const float* cos_sin_tab,
                               int tab_frames, int64_t block_index, int flags, int64_t* evicted_block, void* stream);

/*
 * sdvg_block_attn_fwd on E4M3 operands:
 *   out[i, h, :] = v_descale[h] * sum_j softmax_j(scale * qk_descale[h] * <dec q[i,h,:], dec K[j,h,:]>) dec V[j,h,:]
 * with the same visible keys.  q8, k_self8, v_self8: device bytes [block_tokens, heads, 128] (k_self8 and
 * v_self8 both NULL = the block was staged in the ring); cache: an 8-bit ring; qk_descale[h] = q scale * k
 * scale of head h, v_descale[h] = v scale; out: device bf16; lse as in sdvg_block_attn_fwd (of the
 * descaled logits).  Both products run on the tensor cores in E4M3 with fp32 accumulation; the softmax is
 * fp32 and the probabilities are rounded to E4M3 (relative step 2^-4) before the second product, which is
 * the one approximation beyond the operands' own quantisation.
 * Errors: those of sdvg_block_attn_fwd; BAD_SHAPE for a bf16 ring.
 */
int sdvg_block_attn_fwd_e4m3(const void* q8, const void* k_self8, const void* v_self8, const sdvg_cache* cache,
                             int64_t block_index, const float* qk_descale, const float* v_descale, void* out,
                             float* lse, float scale, void* workspace, size_t workspace_bytes, void* stream);

/*
 * sdvg_block_attn_fwd_batched for 8-bit rings: up to 4 independent problems of one shape (e.g. the conditional
 * and the unconditional pass that a guidance scale of 3.0 implies, Sec. 4.1 "Models"), each with its own ring
 * and its own scale vectors, in one launch when their key segments agree (else one launch each, in stream
 * order).  All arrays are HOST arrays of `batch` entries; k_self8 / v_self8 / lse may be NULL (not given for
 * any problem) or hold NULL entries.  Results are those of separate sdvg_block_attn_fwd_e4m3 calls (see
 * sdvg_block_attn_fwd_batched for what "those" means).
 */
int sdvg_block_attn_fwd_e4m3_batched(int batch, const void* const* q8, const void* const* k_self8,
                                     const void* const* v_self8, const sdvg_cache* const* caches,
                                     const int64_t* block_index, const float* const* qk_descale,
                                     const float* const* v_descale, void* const* out, float* const* lse, float scale,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* ---- 8-bit variant with one scale per tile of 128 tokens ------------------------ */
/*
 * The same number format (Sec. 2 fixes none) with the scales chosen by the library from the data: every tile
 * of 128 consecutive tokens of a block and every head has its own POWER-OF-TWO scale 2^e, e the smallest
 * integer in [-126, 120] with max|x| <= 448 * 2^e over the tile (NaN elements do not count; an infinite
 * maximum takes e = 120); codes are e4m3(x / 2^e), exact up to the one rounding of the conversion.  Nothing
 * has to be calibrated, and a block, or a stretch of one, whose magnitude differs keeps the format's three
 * mantissa bits.  tiles = ceil(block_tokens / 128); the last tile of a block may be short.
 * An 8-bit ring takes such commits once its scale arrays are attached; the static-scale and the tile-scale
 * entry points must not be mixed on one ring (the attention would read scales the other commit never wrote).
 */

/* Floats in ONE of the two scale arrays of a ring: heads * slots * tiles; 0 for a bad shape. */
size_t sdvg_cache_tile_scale_floats(int slots, int heads, int block_tokens);

/*
 * Attaches the scale arrays of an 8-bit ring: device fp32 [heads][slots][tiles] each, caller-owned like the
 * ring buffers and alive as long as the handle.  Errors: INVALID_ARG, BAD_SHAPE (bf16 ring), MISALIGNED
 * (4 bytes).
 */
int sdvg_cache_set_tile_scales(sdvg_cache* cache, float* k_scale, float* v_scale);

/*
 * x: device bf16 [tokens, heads, 128] -> out8: device bytes, same shape, and tile_scale: device fp32
 * [heads][tiles], as defined above.  Used for q when it is already rotated.
 * Errors: INVALID_ARG, BAD_SHAPE (head_dim other than 128), MISALIGNED.
 */
int sdvg_quant_e4m3_tiled(const void* x, void* out8, float* tile_scale, int tokens, int heads, int head_dim,
                          void* stream);

/*
 * sdvg_kv_commit for an 8-bit ring with tile scales: k_roped and v (device bf16 [block_tokens, heads, 128]) are
 * quantised tile by tile into the slot, their scales into the attached arrays.  Same ordering rules, flags,
 * eviction report and errors as sdvg_kv_commit; BAD_STATE also when no scale arrays are attached.
 */
int sdvg_kv_commit_e4m3_tiled(sdvg_cache* cache, const void* k_roped, const void* v, int64_t block_index,
                              int flags, int64_t* evicted_block, void* stream);

/*
 * The fused prologue for such a ring, one pass: rope(q) -> q8_out with q_tile_scale [heads][tiles], rope(k) and
 * v -> the ring slot of block_index with their scales.  rope() is the bit-specified rotation of sdvg_rope3d_qk
 * including its rounding to bf16, so the result is bit-identical to sdvg_rope3d_qk followed by
 * sdvg_quant_e4m3_tiled (q) and sdvg_kv_commit_e4m3_tiled (k, v).  q / q8_out / q_tile_scale may be NULL together.
 * Other arguments and errors as sdvg_rope3d_qk_commit.
 */
int sdvg_rope3d_qk_commit_e4m3_tiled(sdvg_cache* cache, const void* q, const void* k, const void* v, void* q8_out,
                                     float* q_tile_scale, int frames, int grid_h, int grid_w, int frame_offset,
                                     const float* cos_sin_tab, int tab_frames, int64_t block_index, int flags,
                                     int64_t* evicted_block, void* stream);

/*
 * sdvg_block_attn_fwd on such operands:
 *   out[i, h, :] = sum_j softmax_j(scale * <sq_i dec q[i,h,:], sk_j dec K[j,h,:]>) sv_j dec V[j,h,:]
 * with sq_i, sk_j, sv_j the scales of the tiles that query i and key j lie in, over the same visible keys.
 * The block's own K/V must be staged in the ring (commit with SDVG_STAGE first); q8: device bytes
 * [block_tokens, heads, 128]; q_tile_scale: device fp32 [heads][tiles]; out: device bf16; lse optional, as in
 * sdvg_block_attn_fwd.  K's scale enters the logit scale of its key tile, V's scale the exponent of that
 * tile's probabilities before they are rounded to E4M3 (relative to the largest V scale met so far in the row's
 * pass over the keys; the accumulator is rescaled, exactly, when that rises), so the tensor-core work is that
 * of sdvg_block_attn_fwd_e4m3.  Every ring slot is tiled on its own (the short last tile of a block is padded).
 * Errors: those of sdvg_block_attn_fwd; BAD_SHAPE for a bf16 ring or more than 16 slots; BAD_STATE when the
 * block is not staged or no scale arrays are attached.
 */
int sdvg_block_attn_fwd_e4m3_tiled(const void* q8, const float* q_tile_scale, const sdvg_cache* cache,
                                   int64_t block_index, void* out, float* lse, float scale, void* workspace,
                                   size_t workspace_bytes, void* stream);

/* ---- the denoising steps of a block in one call ------------------------------- */
/*
 * Sec. 4.1 "Models": each block takes 4 denoising steps; Sec. 3 "Inference flow": the drafter pays them for
 * every block and the target for every rejected one.  This call enqueues, for s = 0 .. steps-1 and in order,
 *   sdvg_rope3d_qk_commit(cache, q[s], k[s], v[s], q_roped[s], NULL, ..., block_index, SDVG_STAGE)
 *   sdvg_block_attn_fwd(q_roped[s], NULL, NULL, cache, block_index, out[s], NULL, scale, workspace)
 * on `stream`: 2 * steps kernels, nothing else.  The ring state does not change (SDVG_STAGE), so the block's
 * final commit still follows.  The results are those of the separate calls, bit for bit.
 *   q, k, v, q_roped, out   HOST arrays of `steps` device pointers (bf16 [block_tokens, heads, head_dim] each;
 *                           the arrays are read during the call only)
 *   steps                   1 .. 64
 * Every pointer, the workspace, the scale and the block index are checked for all steps before the first
 * launch; grid, table and device are checked by the first prologue, before it launches.
 * Errors: those of the two calls; BAD_SHAPE also for steps outside 1 .. 64 or an 8-bit ring.
 */
int sdvg_block_steps(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                     const void* const* v, void* const* q_roped, void* const* out,
                     int frames, int grid_h, int grid_w, int frame_offset,
                     const float* cos_sin_tab, int tab_frames, int64_t block_index, float scale,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same for an 8-bit ring: sdvg_rope3d_qk_commit_e4m3 (q8_roped[s] receives E4M3 codes, device bytes
 * [block_tokens, heads, 128]) followed by sdvg_block_attn_fwd_e4m3, with the scale vectors of those calls.
 */
int sdvg_block_steps_e4m3(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                          const void* const* v, void* const* q8_roped, void* const* out,
                          const float* q_inv_scale, const float* k_inv_scale, const float* v_inv_scale,
                          const float* qk_descale, const float* v_descale,
                          int frames, int grid_h, int grid_w, int frame_offset,
                          const float* cos_sin_tab, int tab_frames, int64_t block_index, float scale,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same over a tile-scaled 8-bit ring: per step sdvg_rope3d_qk_commit_e4m3_tiled(..., q8_roped[s], q_tile_scale[s],
 * ..., SDVG_STAGE) then sdvg_block_attn_fwd_e4m3_tiled(q8_roped[s], q_tile_scale[s], ...).  q_tile_scale: HOST array of
 * `steps` device fp32 [heads][tiles] arrays.  Errors: those of the two calls, checked for all steps first where they
 * do not depend on the device.
 */
int sdvg_block_steps_e4m3_tiled(int steps, sdvg_cache* cache, const void* const* q, const void* const* k,
                                const void* const* v, void* const* q8_roped, float* const* q_tile_scale,
                                void* const* out, int frames, int grid_h, int grid_w, int frame_offset,
                                const float* cos_sin_tab, int tab_frames, int64_t block_index, float scale,
                                void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SDVG_H_ */
