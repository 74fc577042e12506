"""Thin binding over the C ABI of libsdvg (see include/sdvg.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and the current stream.  There is no
fallback: if the shared library is missing or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdvg.so")

SDVG_OK = 0
SDVG_ERR_INVALID_ARG = 1
SDVG_ERR_BAD_SHAPE = 2
SDVG_ERR_MISALIGNED = 3
SDVG_ERR_BAD_STATE = 4
SDVG_ERR_UNSUPPORTED_ARCH = 5
SDVG_ERR_CUDA = 6
SDVG_ERR_TIMEOUT = 7
SDVG_STAGE = 1
SDVG_FINAL = 2
SDVG_AGG_MIN = 0
SDVG_AGG_MEAN = 1
SDVG_SIGNAL_REWARD = 0
SDVG_SIGNAL_RANDOM = 1

# name -> (restype, argtypes); the list of everything include/sdvg.h declares
_VP, _I, _I64, _SZ, _F = C.c_void_p, C.c_int, C.c_int64, C.c_size_t, C.c_float
SIGNATURES = {
    "sdvg_status_string": (C.c_char_p, [_I]),
    "sdvg_last_cuda_error": (_I, []),
    "sdvg_last_cuda_error_string": (C.c_char_p, []),
    "sdvg_rope3d_pairs": (_I, [_I, C.POINTER(_I), C.POINTER(_I), C.POINTER(_I)]),
    "sdvg_rope3d_table_floats": (_SZ, [_I, _I, _I, _I]),
    "sdvg_rope3d_table": (_I, [_VP, _I, _I, _I, _I]),
    "sdvg_rope3d_qk": (_I, [_VP, _VP, _VP, _VP, _I, _I, _I, _I, _I, _I, _I, _VP, _I, _VP]),
    "sdvg_cache_bytes": (_SZ, [_I, _I, _I, _I]),
    "sdvg_cache_create": (_I, [C.POINTER(_VP), _VP, _VP, _I, _I, _I, _I]),
    "sdvg_cache_reset": (_I, [_VP]),
    "sdvg_cache_destroy": (_I, [_VP]),
    "sdvg_cache_state": (_I, [_VP, C.POINTER(_I64), C.POINTER(_I64), C.POINTER(_I64)]),
    "sdvg_cache_read_block": (_I, [_VP, _I, _VP, _VP, _VP]),
    "sdvg_kv_commit": (_I, [_VP, _VP, _VP, _I64, _I, C.POINTER(_I64), _VP]),
    "sdvg_rope3d_qk_commit": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I, _I64, _I,
                                   C.POINTER(_I64), _VP]),
    "sdvg_block_attn_workspace_bytes": (_SZ, []),
    "sdvg_block_attn_workspace_reset": (_I, [_VP, _SZ, _VP]),
    "sdvg_block_attn_fwd": (_I, [_VP, _VP, _VP, _VP, _I64, _VP, _VP, _F, _VP, _SZ, _VP]),
    "sdvg_block_attn_fwd_batched": (_I, [_I, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _F, _VP, _SZ, _VP]),
    "sdvg_selftest_bounded_wait": (_I, [_VP, _SZ, C.c_ulonglong, _VP]),
    "sdvg_block_attn_status": (_I, [_VP, _VP]),
    "sdvg_block_attn_rescale_events": (_I, [_VP, C.POINTER(C.c_ulonglong), _VP]),
    "sdvg_block_attn_fwd_noalloc": (_I, [_VP, _VP, _VP, _VP, _I64, _VP, _VP, _F, C.POINTER(_VP), _VP]),
    "sdvg_route": (_I, [_VP, _VP, _I, _I, _I64, _F, _VP, _VP, _VP, _VP]),
    "sdvg_route_policy": (_I, [_VP, _VP, _I, _I, _I64, _I, _F, _I, _I, _I, _VP, _F, _VP, _VP, _VP, _VP]),
    "sdvg_accept_stats": (_I, [_VP, _I, _I64, _I, _VP, _VP]),
    "sdvg_state_copy": (_I, [_VP, _VP, _VP, _I, _VP]),
    "sdvg_quant_e4m3": (_I, [_VP, _VP, _VP, _I, _I, _I, _VP]),
    "sdvg_cache_bytes_e4m3": (_SZ, [_I, _I, _I, _I]),
    "sdvg_cache_create_e4m3": (_I, [C.POINTER(_VP), _VP, _VP, _I, _I, _I, _I]),
    "sdvg_kv_commit_e4m3": (_I, [_VP, _VP, _VP, _VP, _VP, _I64, _I, C.POINTER(_I64), _VP]),
    "sdvg_rope3d_qk_commit_e4m3": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I, _I64, _I,
                                        C.POINTER(_I64), _VP]),
    "sdvg_block_attn_fwd_e4m3": (_I, [_VP, _VP, _VP, _VP, _I64, _VP, _VP, _VP, _VP, _F, _VP, _SZ, _VP]),
    "sdvg_cache_tile_scale_floats": (_SZ, [_I, _I, _I]),
    "sdvg_cache_set_tile_scales": (_I, [_VP, _VP, _VP]),
    "sdvg_quant_e4m3_tiled": (_I, [_VP, _VP, _VP, _I, _I, _I, _VP]),
    "sdvg_kv_commit_e4m3_tiled": (_I, [_VP, _VP, _VP, _I64, _I, C.POINTER(_I64), _VP]),
    "sdvg_rope3d_qk_commit_e4m3_tiled": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I, _I64, _I,
                                              C.POINTER(_I64), _VP]),
    "sdvg_block_steps_e4m3_tiled": (_I, [_I, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I, _I64, _F, _VP, _SZ,
                                         _VP]),
    "sdvg_block_attn_fwd_e4m3_tiled": (_I, [_VP, _VP, _VP, _I64, _VP, _VP, _F, _VP, _SZ, _VP]),
    "sdvg_block_attn_fwd_e4m3_batched": (_I, [_I, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _F, _VP, _SZ, _VP]),
    "sdvg_block_steps": (_I, [_I, _VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I, _I64, _F, _VP, _SZ, _VP]),
    "sdvg_block_steps_e4m3": (_I, [_I, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _VP, _I,
                                   _I64, _F, _VP, _SZ, _VP]),
}

_lib = None


class SdvgError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().sdvg_status_string(status).decode()
        if status == SDVG_ERR_CUDA:
            msg += ": " + lib().sdvg_last_cuda_error_string().decode()
        super().__init__(f"{where}: {msg} (status {status})")


def lib() -> C.CDLL:
    """Load libsdvg.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2604_17397_b200.build` first")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(status: int, where: str) -> None:
    if status != SDVG_OK:
        raise SdvgError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _bf16(t: Optional[torch.Tensor], shape=None):
    if t is None:
        return None
    if t.dtype != torch.bfloat16:
        raise ValueError("expected a bfloat16 tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return _ptr(t)


# ---------------------------------------------------------------- RoPE

def sdvg_rope3d_pairs(head_dim: int):
    pf, ph, pw = _I(), _I(), _I()
    _check(lib().sdvg_rope3d_pairs(head_dim, C.byref(pf), C.byref(ph), C.byref(pw)), "sdvg_rope3d_pairs")
    return pf.value, ph.value, pw.value


def sdvg_rope3d_table(head_dim: int, tab_frames: int, grid_h: int, grid_w: int) -> torch.Tensor:
    """Host fp32 (cos, sin) table built by the library; upload it with ``.cuda()``."""
    n = lib().sdvg_rope3d_table_floats(head_dim, tab_frames, grid_h, grid_w)
    if n == 0:
        raise SdvgError(SDVG_ERR_BAD_SHAPE, "sdvg_rope3d_table_floats")
    out = torch.empty(n, dtype=torch.float32)
    _check(lib().sdvg_rope3d_table(out.data_ptr(), head_dim, tab_frames, grid_h, grid_w), "sdvg_rope3d_table")
    return out


def sdvg_rope3d_qk(q, k, q_out, k_out, grid, frame_offset: int, table: torch.Tensor, tab_frames: int,
                   stream=None) -> None:
    ref = q if q is not None else k
    tokens, heads, head_dim = ref.shape
    frames, grid_h, grid_w = grid
    st = lib().sdvg_rope3d_qk(_bf16(q), _bf16(k), _bf16(q_out, None if q is None else q.shape),
                              _bf16(k_out, None if k is None else k.shape), tokens, heads, head_dim,
                              frames, grid_h, grid_w, frame_offset, _ptr(table), tab_frames, _stream(stream))
    _check(st, "sdvg_rope3d_qk")


# ---------------------------------------------------------------- cache

class Cache:
    """Rolling KV cache: torch owns the two device buffers, the library the ring state."""

    def __init__(self, slots: int, heads: int, block_tokens: int, head_dim: int, device="cuda", e4m3: bool = False,
                 tile_scales: bool = False):
        sizer = lib().sdvg_cache_bytes_e4m3 if e4m3 else lib().sdvg_cache_bytes
        nbytes = sizer(slots, heads, block_tokens, head_dim)
        if nbytes == 0:
            raise SdvgError(SDVG_ERR_BAD_SHAPE, "sdvg_cache_bytes")
        self.slots, self.heads, self.block_tokens, self.head_dim = slots, heads, block_tokens, head_dim
        self.e4m3 = e4m3                      # ring of E4M3 codes (8-bit variant) instead of bf16
        # physical layout [heads][slots][tokens][dim]; torch's allocator aligns to 512 B, so over-allocate
        self._k_raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        self._v_raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        self.k_ptr = (self._k_raw.data_ptr() + 1023) & ~1023
        self.v_ptr = (self._v_raw.data_ptr() + 1023) & ~1023
        h = _VP()
        create = lib().sdvg_cache_create_e4m3 if e4m3 else lib().sdvg_cache_create
        _check(create(C.byref(h), self.k_ptr, self.v_ptr, slots, heads, block_tokens, head_dim), "sdvg_cache_create")
        self.handle = h
        # 8-bit ring with one scale per (head, slot, tile of 128 tokens): torch owns the two scale arrays as well
        self.tile_scales = tile_scales
        if tile_scales:
            n = lib().sdvg_cache_tile_scale_floats(slots, heads, block_tokens)
            self.tiles = n // (slots * heads)
            self.k_scale = torch.ones((heads, slots, self.tiles), dtype=torch.float32, device=device)
            self.v_scale = torch.ones((heads, slots, self.tiles), dtype=torch.float32, device=device)
            _check(lib().sdvg_cache_set_tile_scales(h, self.k_scale.data_ptr(), self.v_scale.data_ptr()),
                   "sdvg_cache_set_tile_scales")

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            lib().sdvg_cache_destroy(self.handle)
            self.handle = _VP()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        _check(lib().sdvg_cache_reset(self.handle), "sdvg_cache_reset")

    def state(self):
        """(next_block, [slot -> committed block or -1], staged_block)."""
        nb, sb = _I64(), _I64()
        arr = (_I64 * self.slots)()
        _check(lib().sdvg_cache_state(self.handle, C.byref(nb), arr, C.byref(sb)), "sdvg_cache_state")
        return nb.value, list(arr), sb.value

    def read_block(self, slot: int, stream=None):
        """Logical [tokens, heads, dim] copies of the K and V held in ``slot``."""
        shape = (self.block_tokens, self.heads, self.head_dim)
        k = torch.empty(shape, dtype=torch.uint8 if self.e4m3 else torch.bfloat16, device=self._k_raw.device)
        v = torch.empty_like(k)
        _check(lib().sdvg_cache_read_block(self.handle, slot, k.data_ptr(), v.data_ptr(), _stream(stream)),
               "sdvg_cache_read_block")
        return k, v


def sdvg_kv_commit(cache: Cache, k_roped, v, block_index: int, flags: int, stream=None) -> int:
    """Returns the evicted block (-1 if none)."""
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    ev = _I64(-1)
    st = lib().sdvg_kv_commit(cache.handle, _bf16(k_roped, shape), _bf16(v, shape), block_index, flags,
                              C.byref(ev), _stream(stream))
    _check(st, "sdvg_kv_commit")
    return ev.value


def sdvg_rope3d_qk_commit(cache: Cache, q, k, v, q_out, k_out, grid, frame_offset: int, table, tab_frames: int,
                          block_index: int, flags: int, stream=None) -> int:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    frames, grid_h, grid_w = grid
    ev = _I64(-1)
    st = lib().sdvg_rope3d_qk_commit(cache.handle, _bf16(q, None if q is None else shape), _bf16(k, shape),
                                     _bf16(v, shape), _bf16(q_out, None if q_out is None else shape),
                                     _bf16(k_out, None if k_out is None else shape),
                                     frames, grid_h, grid_w, frame_offset, _ptr(table), tab_frames,
                                     block_index, flags, C.byref(ev), _stream(stream))
    _check(st, "sdvg_rope3d_qk_commit")
    return ev.value


# ---------------------------------------------------------------- attention

def attn_workspace(device="cuda", extra_bytes: int = 0) -> torch.Tensor:
    """A 256-byte-aligned attention workspace on `device`, cleared through the library."""
    n = lib().sdvg_block_attn_workspace_bytes() + extra_bytes
    raw = torch.empty(n + 256, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 256
    ws = raw[off:off + n]
    with torch.cuda.device(ws.device):
        sdvg_block_attn_workspace_reset(ws)
    return ws


def sdvg_block_attn_workspace_reset(workspace, nbytes: Optional[int] = None, stream=None) -> None:
    """Clears the workspace (and with it a sticky SDVG_ERR_TIMEOUT).  `workspace` is a tensor, or an
    integer device address together with `nbytes`."""
    if isinstance(workspace, int):
        ptr, n = workspace, int(nbytes)
    else:
        ptr, n = workspace.data_ptr(), workspace.numel()
    _check(lib().sdvg_block_attn_workspace_reset(ptr, n, _stream(stream)), "sdvg_block_attn_workspace_reset")


def sdvg_block_attn_fwd(q, k_self, v_self, cache: Cache, block_index: int, out, lse, scale: float,
                        workspace: torch.Tensor, stream=None) -> None:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    if lse is not None and (lse.dtype != torch.float32 or tuple(lse.shape) != (cache.heads, cache.block_tokens)):
        raise ValueError("lse must be float32 [heads, block_tokens]")
    st = lib().sdvg_block_attn_fwd(_bf16(q, shape), _bf16(k_self, None if k_self is None else shape),
                                   _bf16(v_self, None if v_self is None else shape), cache.handle, block_index,
                                   _bf16(out, shape), _ptr(lse), scale, workspace.data_ptr(), workspace.numel(),
                                   _stream(stream))
    _check(st, "sdvg_block_attn_fwd")


def sdvg_block_attn_fwd_batched(qs, k_selfs, v_selfs, caches, block_indices, outs, lses, scale: float,
                                workspace: torch.Tensor, stream=None) -> None:
    """Lists of per-problem arguments (k_selfs / v_selfs / lses may be None = not given for any problem)."""
    n = len(qs)
    shape = (caches[0].block_tokens, caches[0].heads, caches[0].head_dim)

    def ptr_array(ts, check):
        if ts is None:
            return None
        return (_VP * n)(*[check(t) for t in ts])

    def lse_ptr(t):
        if t is not None and (t.dtype != torch.float32 or tuple(t.shape) != (shape[1], shape[0])):
            raise ValueError("lse must be float32 [heads, block_tokens]")
        return _ptr(t)

    bf = lambda t: _bf16(t, shape)
    keep = [ptr_array(qs, bf), ptr_array(k_selfs, bf), ptr_array(v_selfs, bf),
            (_VP * n)(*[c.handle.value for c in caches]), (_I64 * n)(*block_indices), ptr_array(outs, bf),
            ptr_array(lses, lse_ptr)]
    st = lib().sdvg_block_attn_fwd_batched(n, *[C.cast(a, _VP) if a is not None else None for a in keep], scale,
                                           workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_attn_fwd_batched")


def sdvg_selftest_bounded_wait(workspace: torch.Tensor, limit_ns: int, stream=None) -> None:
    st = lib().sdvg_selftest_bounded_wait(workspace.data_ptr(), workspace.numel(), limit_ns, _stream(stream))
    _check(st, "sdvg_selftest_bounded_wait")


def sdvg_block_attn_status(workspace, stream=None) -> int:
    """`workspace` is the tensor given to sdvg_block_attn_fwd, or the integer device address
    returned by sdvg_block_attn_fwd_noalloc."""
    ptr = workspace if isinstance(workspace, int) else workspace.data_ptr()
    return lib().sdvg_block_attn_status(ptr, _stream(stream))


def sdvg_block_attn_rescale_events(workspace, stream=None) -> int:
    """Warp-level accumulator-rescale events recorded in the workspace since its last reset."""
    ptr = workspace if isinstance(workspace, int) else workspace.data_ptr()
    n = C.c_ulonglong(0)
    _check(lib().sdvg_block_attn_rescale_events(ptr, C.byref(n), _stream(stream)), "sdvg_block_attn_rescale_events")
    return int(n.value)


def sdvg_block_attn_fwd_noalloc(q, k_self, v_self, cache: Cache, block_index: int, out, lse, scale: float,
                                stream=None) -> int:
    """Attention through the library's built-in scratch: for callers that must not allocate
    device memory.  Returns the device address of that scratch (for sdvg_block_attn_status)."""
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    if lse is not None and (lse.dtype != torch.float32 or tuple(lse.shape) != (cache.heads, cache.block_tokens)):
        raise ValueError("lse must be float32 [heads, block_tokens]")
    scratch = _VP()
    st = lib().sdvg_block_attn_fwd_noalloc(_bf16(q, shape), _bf16(k_self, None if k_self is None else shape),
                                           _bf16(v_self, None if v_self is None else shape), cache.handle,
                                           block_index, _bf16(out, shape), _ptr(lse), scale, C.byref(scratch),
                                           _stream(stream))
    _check(st, "sdvg_block_attn_fwd_noalloc")
    return int(scratch.value)


# ---------------------------------------------------------------- router

def sdvg_route(scores, frame_offsets, num_blocks: int, frames_per_block: int, first_block_index: int, tau: float,
               accept, q_min, argmin=None, stream=None) -> None:
    if scores.dtype != torch.float32 or q_min.dtype != torch.float32 or accept.dtype != torch.uint8:
        raise ValueError("scores/q_min must be float32 and accept uint8")
    if frame_offsets is not None and frame_offsets.dtype != torch.int32:
        raise ValueError("frame_offsets must be int32")
    if argmin is not None and argmin.dtype != torch.int32:
        raise ValueError("argmin must be int32")
    st = lib().sdvg_route(_ptr(scores), _ptr(frame_offsets), num_blocks, frames_per_block, first_block_index, tau,
                          _ptr(accept), _ptr(q_min), _ptr(argmin), _stream(stream))
    _check(st, "sdvg_route")


def sdvg_route_policy(scores, frame_offsets, num_blocks: int, frames_per_block: int, first_block_index: int,
                      blocks_per_video: int, tau: float, agg: int, signal: int, force_first: bool, uniforms,
                      accept_prob: float, accept, aggregate, argmin=None, stream=None) -> None:
    if scores.dtype != torch.float32 or aggregate.dtype != torch.float32 or accept.dtype != torch.uint8:
        raise ValueError("scores/aggregate must be float32 and accept uint8")
    if frame_offsets is not None and frame_offsets.dtype != torch.int32:
        raise ValueError("frame_offsets must be int32")
    if argmin is not None and argmin.dtype != torch.int32:
        raise ValueError("argmin must be int32")
    if uniforms is not None and uniforms.dtype != torch.float32:
        raise ValueError("uniforms must be float32")
    st = lib().sdvg_route_policy(_ptr(scores), _ptr(frame_offsets), num_blocks, frames_per_block, first_block_index,
                                 blocks_per_video, tau, agg, signal, 1 if force_first else 0, _ptr(uniforms),
                                 accept_prob, _ptr(accept), _ptr(aggregate), _ptr(argmin), _stream(stream))
    _check(st, "sdvg_route_policy")


def sdvg_accept_stats(accept, num_blocks: int, first_block_index: int, blocks_per_video: int, counts,
                      stream=None) -> None:
    """counts: device int64 [2] <- (accepted, routable) over the blocks that are not first blocks."""
    if accept.dtype != torch.uint8 or counts.dtype != torch.int64 or counts.numel() < 2:
        raise ValueError("accept must be uint8 and counts int64 [2]")
    st = lib().sdvg_accept_stats(_ptr(accept), num_blocks, first_block_index, blocks_per_video, _ptr(counts),
                                 _stream(stream))
    _check(st, "sdvg_accept_stats")


def sdvg_state_copy(srcs, dsts, stream=None) -> None:
    """dsts[i] <- srcs[i] for lists of contiguous CUDA tensors of equal byte sizes (snapshot or restore)."""
    n = len(srcs)
    if len(dsts) != n:
        raise ValueError("srcs and dsts must have the same length")
    nbytes = []
    for a, b in zip(srcs, dsts):
        if a.numel() * a.element_size() != b.numel() * b.element_size():
            raise ValueError("source and destination sizes differ")
        nbytes.append(a.numel() * a.element_size())
    st = lib().sdvg_state_copy(C.cast((_VP * n)(*[_ptr(t) for t in srcs]), _VP),
                               C.cast((_VP * n)(*[_ptr(t) for t in dsts]), _VP),
                               C.cast((_SZ * n)(*nbytes), _VP), n, _stream(stream))
    _check(st, "sdvg_state_copy")


# ---------------------------------------------------------------- 8-bit (E4M3) variant

def _u8(t: Optional[torch.Tensor], shape=None):
    if t is None:
        return None
    if t.dtype != torch.uint8:
        raise ValueError("expected a uint8 tensor of E4M3 codes")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return _ptr(t)


def _scales(t: torch.Tensor, heads: int):
    if t.dtype != torch.float32 or tuple(t.shape) != (heads,):
        raise ValueError("scales must be float32 [heads]")
    return _ptr(t)


def sdvg_quant_e4m3(x, inv_scale, out, stream=None) -> None:
    tokens, heads, head_dim = x.shape
    st = lib().sdvg_quant_e4m3(_bf16(x), _scales(inv_scale, heads), _u8(out, x.shape), tokens, heads, head_dim,
                               _stream(stream))
    _check(st, "sdvg_quant_e4m3")


def sdvg_kv_commit_e4m3(cache: Cache, k_roped, v, k_inv_scale, v_inv_scale, block_index: int, flags: int,
                        stream=None) -> int:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    ev = _I64(-1)
    st = lib().sdvg_kv_commit_e4m3(cache.handle, _bf16(k_roped, shape), _bf16(v, shape),
                                   _scales(k_inv_scale, cache.heads), _scales(v_inv_scale, cache.heads), block_index,
                                   flags, C.byref(ev), _stream(stream))
    _check(st, "sdvg_kv_commit_e4m3")
    return ev.value


def sdvg_rope3d_qk_commit_e4m3(cache: Cache, q, k, v, q8_out, q_inv_scale, k_inv_scale, v_inv_scale, grid,
                               frame_offset: int, table, tab_frames: int, block_index: int, flags: int, stream=None) -> int:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    frames, grid_h, grid_w = grid
    ev = _I64(-1)
    st = lib().sdvg_rope3d_qk_commit_e4m3(cache.handle, _bf16(q, None if q is None else shape), _bf16(k, shape),
                                          _bf16(v, shape), _u8(q8_out, None if q8_out is None else shape),
                                          None if q_inv_scale is None else _scales(q_inv_scale, cache.heads),
                                          _scales(k_inv_scale, cache.heads), _scales(v_inv_scale, cache.heads),
                                          frames, grid_h, grid_w, frame_offset, _ptr(table), tab_frames, block_index,
                                          flags, C.byref(ev), _stream(stream))
    _check(st, "sdvg_rope3d_qk_commit_e4m3")
    return ev.value


def sdvg_block_attn_fwd_e4m3(q8, k_self8, v_self8, cache: Cache, block_index: int, qk_descale, v_descale, out, lse,
                             scale: float, workspace: torch.Tensor, stream=None) -> None:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    if lse is not None and (lse.dtype != torch.float32 or tuple(lse.shape) != (cache.heads, cache.block_tokens)):
        raise ValueError("lse must be float32 [heads, block_tokens]")
    st = lib().sdvg_block_attn_fwd_e4m3(_u8(q8, shape), _u8(k_self8, None if k_self8 is None else shape),
                                        _u8(v_self8, None if v_self8 is None else shape), cache.handle, block_index,
                                        _scales(qk_descale, cache.heads), _scales(v_descale, cache.heads),
                                        _bf16(out, shape), _ptr(lse), scale, workspace.data_ptr(), workspace.numel(),
                                        _stream(stream))
    _check(st, "sdvg_block_attn_fwd_e4m3")


def _tile_scales(t: Optional[torch.Tensor], heads: int, tokens: int):
    if t is None:
        return None
    if t.dtype != torch.float32 or tuple(t.shape) != (heads, (tokens + 127) // 128) or not t.is_contiguous():
        raise ValueError("tile scales must be contiguous float32 [heads, ceil(tokens / 128)]")
    return _ptr(t)


def sdvg_quant_e4m3_tiled(x, out8, tile_scale, stream=None) -> None:
    tokens, heads, head_dim = x.shape
    st = lib().sdvg_quant_e4m3_tiled(_bf16(x), _u8(out8, x.shape), _tile_scales(tile_scale, heads, tokens), tokens,
                                     heads, head_dim, _stream(stream))
    _check(st, "sdvg_quant_e4m3_tiled")


def sdvg_kv_commit_e4m3_tiled(cache: Cache, k_roped, v, block_index: int, flags: int, stream=None) -> int:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    ev = _I64(-1)
    st = lib().sdvg_kv_commit_e4m3_tiled(cache.handle, _bf16(k_roped, shape), _bf16(v, shape), block_index, flags,
                                         C.byref(ev), _stream(stream))
    _check(st, "sdvg_kv_commit_e4m3_tiled")
    return ev.value


def sdvg_rope3d_qk_commit_e4m3_tiled(cache: Cache, q, k, v, q8_out, q_tile_scale, grid, frame_offset: int, table,
                                     tab_frames: int, block_index: int, flags: int, stream=None) -> int:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    frames, grid_h, grid_w = grid
    ev = _I64(-1)
    st = lib().sdvg_rope3d_qk_commit_e4m3_tiled(cache.handle, _bf16(q, None if q is None else shape), _bf16(k, shape),
                                                _bf16(v, shape), _u8(q8_out, None if q8_out is None else shape),
                                                _tile_scales(q_tile_scale, cache.heads, cache.block_tokens), frames,
                                                grid_h, grid_w, frame_offset, _ptr(table), tab_frames, block_index,
                                                flags, C.byref(ev), _stream(stream))
    _check(st, "sdvg_rope3d_qk_commit_e4m3_tiled")
    return ev.value


def sdvg_block_attn_fwd_e4m3_tiled(q8, q_tile_scale, cache: Cache, block_index: int, out, lse, scale: float,
                                   workspace: torch.Tensor, stream=None) -> None:
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    if lse is not None and (lse.dtype != torch.float32 or tuple(lse.shape) != (cache.heads, cache.block_tokens)):
        raise ValueError("lse must be float32 [heads, block_tokens]")
    st = lib().sdvg_block_attn_fwd_e4m3_tiled(_u8(q8, shape), _tile_scales(q_tile_scale, cache.heads, cache.block_tokens),
                                              cache.handle, block_index, _bf16(out, shape), _ptr(lse), scale,
                                              workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_attn_fwd_e4m3_tiled")


# ---------------------------------------------------------------- the steps of a block in one call

def _ptr_array(ts, check):
    return (_VP * len(ts))(*[check(t) for t in ts])


def sdvg_block_steps(cache: Cache, qs, ks, vs, q_ropeds, outs, grid, frame_offset: int, table, tab_frames: int,
                     block_index: int, scale: float, workspace: torch.Tensor, stream=None) -> None:
    """The denoising steps of one block (lists of per-step tensors): fused rope + stage, then attention, per step."""
    n = len(qs)
    if not (len(ks) == len(vs) == len(q_ropeds) == len(outs) == n):
        raise ValueError("one q, k, v, q_roped and out per step")
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    bf = lambda t: _bf16(t, shape)
    arrays = [_ptr_array(x, bf) for x in (qs, ks, vs, q_ropeds, outs)]
    st = lib().sdvg_block_steps(n, cache.handle, *[C.cast(a, _VP) for a in arrays], grid[0], grid[1], grid[2],
                                frame_offset, _ptr(table), tab_frames, block_index, scale, workspace.data_ptr(),
                                workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_steps")


def sdvg_block_steps_e4m3(cache: Cache, qs, ks, vs, q8_ropeds, outs, q_inv_scale, k_inv_scale, v_inv_scale,
                          qk_descale, v_descale, grid, frame_offset: int, table, tab_frames: int, block_index: int,
                          scale: float, workspace: torch.Tensor, stream=None) -> None:
    """The same over an 8-bit ring (q8_ropeds receive E4M3 codes)."""
    n = len(qs)
    if not (len(ks) == len(vs) == len(q8_ropeds) == len(outs) == n):
        raise ValueError("one q, k, v, q8_roped and out per step")
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    bf = lambda t: _bf16(t, shape)
    u8 = lambda t: _u8(t, shape)
    arrays = [_ptr_array(qs, bf), _ptr_array(ks, bf), _ptr_array(vs, bf), _ptr_array(q8_ropeds, u8), _ptr_array(outs, bf)]
    sc = [_scales(t, cache.heads) for t in (q_inv_scale, k_inv_scale, v_inv_scale, qk_descale, v_descale)]
    st = lib().sdvg_block_steps_e4m3(n, cache.handle, *[C.cast(a, _VP) for a in arrays], *sc, grid[0], grid[1], grid[2],
                                     frame_offset, _ptr(table), tab_frames, block_index, scale, workspace.data_ptr(),
                                     workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_steps_e4m3")


def sdvg_block_steps_e4m3_tiled(cache: Cache, qs, ks, vs, q8_ropeds, q_tile_scales, outs, grid, frame_offset: int, table,
                                tab_frames: int, block_index: int, scale: float, workspace: torch.Tensor,
                                stream=None) -> None:
    """The same over a tile-scaled 8-bit ring (q8_ropeds receive E4M3 codes, q_tile_scales their scales)."""
    n = len(qs)
    if not (len(ks) == len(vs) == len(q8_ropeds) == len(q_tile_scales) == len(outs) == n):
        raise ValueError("one q, k, v, q8_roped, q_tile_scale and out per step")
    shape = (cache.block_tokens, cache.heads, cache.head_dim)
    bf = lambda t: _bf16(t, shape)
    u8 = lambda t: _u8(t, shape)
    ts = lambda t: _tile_scales(t, cache.heads, cache.block_tokens)
    arrays = [_ptr_array(qs, bf), _ptr_array(ks, bf), _ptr_array(vs, bf), _ptr_array(q8_ropeds, u8),
              _ptr_array(q_tile_scales, ts), _ptr_array(outs, bf)]
    st = lib().sdvg_block_steps_e4m3_tiled(n, cache.handle, *[C.cast(a, _VP) for a in arrays], grid[0], grid[1], grid[2],
                                           frame_offset, _ptr(table), tab_frames, block_index, scale,
                                           workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_steps_e4m3_tiled")


def sdvg_block_attn_fwd_e4m3_batched(q8s, k_self8s, v_self8s, caches, block_indices, qk_descales, v_descales, outs, lses,
                                     scale: float, workspace: torch.Tensor, stream=None) -> None:
    """Lists of per-problem arguments over 8-bit rings (k_self8s / v_self8s / lses may be None)."""
    n = len(q8s)
    shape = (caches[0].block_tokens, caches[0].heads, caches[0].head_dim)
    heads = caches[0].heads

    def arr(ts, check):
        return None if ts is None else (_VP * n)(*[check(t) for t in ts])

    def lse_ptr(t):
        if t is not None and (t.dtype != torch.float32 or tuple(t.shape) != (shape[1], shape[0])):
            raise ValueError("lse must be float32 [heads, block_tokens]")
        return _ptr(t)

    u8 = lambda t: _u8(t, shape)
    sc = lambda t: _scales(t, heads)
    keep = [arr(q8s, u8), arr(k_self8s, u8), arr(v_self8s, u8), (_VP * n)(*[c.handle.value for c in caches]),
            (_I64 * n)(*block_indices), arr(qk_descales, sc), arr(v_descales, sc), arr(outs, lambda t: _bf16(t, shape)),
            arr(lses, lse_ptr)]
    st = lib().sdvg_block_attn_fwd_e4m3_batched(n, *[C.cast(a, _VP) if a is not None else None for a in keep], scale,
                                                workspace.data_ptr(), workspace.numel(), _stream(stream))
    _check(st, "sdvg_block_attn_fwd_e4m3_batched")
