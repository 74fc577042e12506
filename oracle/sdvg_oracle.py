"""CPU oracle for the SDVG hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy statement of what the path computes: 3D-RoPE on q/k,
block-causal attention of one block against the rolling KV cache, the ring
commit with eviction, the worst-frame router with a forced rejection of block
0, the per-block speculative schedule that strings them together, and the 8-bit
(E4M3) variant of the cache and the attention, with one static scale per head or one
power-of-two scale per tile of 128 tokens.  Nothing
here is blocked, fused or tuned; library matmul/exp are used as single steps.

Only tests, the smoke check and the bench's ``cpu_baseline`` leg may import
this package.  It shares no code with the CUDA library and never imports it.

bf16 tensors are ``numpy.uint16`` bit patterns, widened exactly to float64.
Token layout of a block tensor is [tokens, heads, head_dim], tokens ordered
frame-major, then grid row, then grid column.

Pins (see tests): every function below is pinned by at least one independent
check (dense-mask brute force, closed forms, invariants, hand-worked router
and ring cases, the accept-rate convention and the cost identity implied by
Table 1).  Parity unpinned: none.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

ROPE_THETA = 10000.0

# --------------------------------------------------------------------------
# bf16 <-> float
# --------------------------------------------------------------------------


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bits, round to nearest even; NaN stays a quiet NaN."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(f)
    if nan.any():
        r = np.where(nan, ((u >> np.uint32(16)) | np.uint32(0x0040)).astype(np.uint16), r)
    return r


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bits through float32 (two RNE roundings; within 1 bf16 ulp of exact)."""
    return f32_to_bf16(np.asarray(x, dtype=np.float64).astype(np.float32))


# --------------------------------------------------------------------------
# 3D RoPE  (Sec. 4.1 "Models": the backbone carries positions by rotary embeddings)
# --------------------------------------------------------------------------


def rope_axis_pairs(head_dim: int) -> tuple[int, int, int]:
    """Number of rotated (even, odd) pairs owned by the frame / height / width axes.

    Height and width each own floor(D/6) pairs, the frame axis the rest of the
    D/2 pairs (D=128 -> 22/21/21, D=64 -> 12/10/10).
    """
    if head_dim <= 0 or head_dim % 2:
        raise ValueError("head_dim must be a positive even number")
    p_hw = head_dim // 6
    return head_dim // 2 - 2 * p_hw, p_hw, p_hw


def token_positions(tokens: int, grid: tuple[int, int, int], frame_offset: int) -> np.ndarray:
    """[tokens, 3] integer (frame, row, column) positions, frame-major order."""
    F, Hg, Wg = grid
    if tokens != F * Hg * Wg:
        raise ValueError("tokens != F*Hg*Wg")
    n = np.arange(tokens, dtype=np.int64)
    f = n // (Hg * Wg) + frame_offset
    y = (n // Wg) % Hg
    x = n % Wg
    return np.stack([f, y, x], axis=1)


def rope_angles(head_dim: int, pos: np.ndarray) -> np.ndarray:
    """[tokens, D/2] fp64 rotation angles: pair i of an axis with P pairs turns by pos*theta^(-i/P)."""
    pf, ph, pw = rope_axis_pairs(head_dim)
    cols = []
    for axis, P in enumerate((pf, ph, pw)):
        i = np.arange(P, dtype=np.float64)
        omega = ROPE_THETA ** (-(i / P))
        cols.append(pos[:, axis:axis + 1].astype(np.float64) * omega[None, :])
    return np.concatenate(cols, axis=1)


def rope_ref(x_bits: np.ndarray, grid: tuple[int, int, int], frame_offset: int) -> np.ndarray:
    """fp64 3D-RoPE of a [tokens, heads, D] bf16 tensor; returns float64 (not rounded).

    Pair p is (x[2p], x[2p+1]) and turns counter-clockwise by its angle.
    """
    T, H, D = x_bits.shape
    x = bf16_to_f64(x_bits)
    a = rope_angles(D, token_positions(T, grid, frame_offset))       # [T, D/2]
    c, s = np.cos(a)[:, None, :], np.sin(a)[:, None, :]
    re, im = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x)
    out[..., 0::2] = re * c - im * s
    out[..., 1::2] = re * s + im * c
    return out


def rope_table(head_dim: int, tab_frames: int, grid_h: int, grid_w: int) -> np.ndarray:
    """fp32 (cos, sin) table, the shared numeric input of the bit-level RoPE.

    Flat float32 array of (cos, sin) pairs: frame positions 0..tab_frames-1 by
    P_f pairs, then grid rows 0..grid_h-1 by P_h pairs, then grid columns
    0..grid_w-1 by P_w pairs.  Angles are formed and evaluated in fp64 and
    rounded once to fp32.
    """
    pf, ph, pw = rope_axis_pairs(head_dim)
    parts = []
    for n_pos, P in ((tab_frames, pf), (grid_h, ph), (grid_w, pw)):
        i = np.arange(P, dtype=np.float64)
        omega = ROPE_THETA ** (-(i / P))
        a = np.arange(n_pos, dtype=np.float64)[:, None] * omega[None, :]
        parts.append(np.stack([np.cos(a), np.sin(a)], axis=-1).reshape(-1))
    return np.concatenate(parts).astype(np.float32)


def rope_bitspec(x_bits: np.ndarray, grid: tuple[int, int, int], frame_offset: int,
                 table: np.ndarray, tab_frames: int) -> np.ndarray:
    """Bit-level RoPE: the fp32 operation sequence that fixes the cache contents.

    With (c, s) read from ``table``:  re' = fl(fl(re*c) - fl(im*s)),
    im' = fl(fl(re*s) + fl(im*c)), every fl() one IEEE fp32 rounding, no fused
    multiply-add, then round-to-nearest-even to bf16.  Returns bf16 bits.
    """
    T, H, D = x_bits.shape
    F, Hg, Wg = grid
    pf, ph, pw = rope_axis_pairs(D)
    if frame_offset < 0 or frame_offset + F > tab_frames:
        raise ValueError("frame positions outside the table")
    tab = np.asarray(table, dtype=np.float32)
    t_f = tab[:tab_frames * pf * 2].reshape(tab_frames, pf, 2)
    t_h = tab[tab_frames * pf * 2: tab_frames * pf * 2 + Hg * ph * 2].reshape(Hg, ph, 2)
    t_w = tab[tab_frames * pf * 2 + Hg * ph * 2:].reshape(Wg, pw, 2)
    pos = token_positions(T, grid, frame_offset)
    cs = np.concatenate([t_f[pos[:, 0]], t_h[pos[:, 1]], t_w[pos[:, 2]]], axis=1)  # [T, D/2, 2]
    c = cs[:, None, :, 0]
    s = cs[:, None, :, 1]
    x = bf16_to_f32(x_bits)
    re, im = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x)
    # numpy float32 ufuncs round every product and sum separately (no contraction)
    out[..., 0::2] = (re * c).astype(np.float32) - (im * s).astype(np.float32)
    out[..., 1::2] = (re * s).astype(np.float32) + (im * c).astype(np.float32)
    return f32_to_bf16(out)


# --------------------------------------------------------------------------
# Block-causal attention over the rolling cache
# --------------------------------------------------------------------------


def visible_blocks(block_index: int, slots: int) -> list[int]:
    """Earlier blocks block ``b`` may attend to: the last slots-1 blocks before it."""
    return list(range(max(0, block_index - (slots - 1)), block_index))


def attn_ref(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, scale: float,
             heads=None, rows=None, row_chunk: int = 1024):
    """Softmax attention of query rows against ALL given keys, in fp64.

    q [Tq, H, D], k/v [Lk, H, D] as bf16 bits (k already roped and rounded, as
    the cache holds it).  For each head h and row i:
      s_j = scale * <q_i, k_j>,  p_j = exp(s_j - max s) / sum,  o = sum_j p_j v_j,
      lse = max s + ln(sum exp(s_j - max s)).
    ``heads`` / ``rows`` restrict the evaluation to a subset (sampling at large
    shapes).  Returns (o [len(rows), len(heads), D] fp64, lse [len(heads), len(rows)] fp64).
    """
    Tq, H, D = q_bits.shape
    heads = list(range(H)) if heads is None else list(heads)
    rows = np.arange(Tq) if rows is None else np.asarray(rows, dtype=np.int64)
    o = np.empty((rows.size, len(heads), D), dtype=np.float64)
    lse = np.empty((len(heads), rows.size), dtype=np.float64)
    for hi, h in enumerate(heads):
        kh = bf16_to_f64(k_bits[:, h, :])
        vh = bf16_to_f64(v_bits[:, h, :])
        for r0 in range(0, rows.size, row_chunk):
            rr = rows[r0:r0 + row_chunk]
            qh = bf16_to_f64(q_bits[rr, h, :])
            s = (qh @ kh.T) * scale
            m = s.max(axis=1, keepdims=True)
            p = np.exp(s - m)
            l = p.sum(axis=1, keepdims=True)
            o[r0:r0 + rr.size, hi, :] = (p @ vh) / l
            lse[hi, r0:r0 + rr.size] = (m + np.log(l))[:, 0]
    return o, lse


def dense_bruteforce(q_blocks, k_blocks, v_blocks, scale: float, slots: int):
    """All blocks as ONE sequence with an explicit block-causal window mask (tiny inputs).

    Key j is visible to query i iff blk(j) <= blk(i) and blk(i)-blk(j) <= slots-1.
    Returns (o [B*T, H, D] fp64, P [H, B*T, B*T] fp64, mask [B*T, B*T] bool).
    """
    B = len(q_blocks)
    T, H, D = q_blocks[0].shape
    q = bf16_to_f64(np.concatenate(q_blocks, axis=0))
    k = bf16_to_f64(np.concatenate(k_blocks, axis=0))
    v = bf16_to_f64(np.concatenate(v_blocks, axis=0))
    blk = np.repeat(np.arange(B), T)
    mask = (blk[None, :] <= blk[:, None]) & ((blk[:, None] - blk[None, :]) <= slots - 1)
    L = B * T
    o = np.zeros((L, H, D))
    P = np.zeros((H, L, L))
    for h in range(H):
        for i in range(L):
            logits = np.full(L, -np.inf)
            for j in range(L):
                if mask[i, j]:
                    logits[j] = scale * float(np.dot(q[i, h], k[j, h]))
            e = np.exp(logits - logits.max())
            P[h, i] = e / e.sum()
            o[i, h] = P[h, i] @ v[:, h, :]
    return o, P, mask


# --------------------------------------------------------------------------
# Ring KV cache (Sec. 3 "Inference flow": K^D updated always, K^T on accept / regenerate)
# --------------------------------------------------------------------------

STAGE = 1
FINAL = 2


class RingCacheRef:
    """Integer model of the rolling cache: block b lives in slot b mod slots.

    ``commit(b, k, v, FINAL)`` requires b == next_block, reports the block that
    was evicted from the slot (-1 if it was empty) and advances next_block.
    ``STAGE`` writes the bits of the provisional block b == next_block into its
    slot (overwriting block b-slots, which b can no longer see) but leaves
    next_block and the slot map alone.  Contents are exact copies of the input.
    """

    def __init__(self, slots: int, heads: int, block_tokens: int, head_dim: int, dtype=np.uint16):
        if min(slots, heads, block_tokens, head_dim) <= 0:
            raise ValueError("bad cache shape")
        self.slots, self.heads, self.T, self.D = slots, heads, block_tokens, head_dim
        self.dtype = np.dtype(dtype)          # uint16: bf16 bits; uint8: E4M3 codes
        self.k = np.zeros((slots, block_tokens, heads, head_dim), dtype=self.dtype)
        self.v = np.zeros_like(self.k)
        self.next_block = 0
        self.slot_block = [-1] * slots

    def slot_of(self, block_index: int) -> int:
        return block_index % self.slots

    def commit(self, block_index: int, k_bits: np.ndarray, v_bits: np.ndarray, flags: int) -> int:
        if flags not in (STAGE, FINAL):
            raise ValueError("flags must be STAGE or FINAL")
        if block_index != self.next_block:
            raise RuntimeError("blocks must be committed in order")
        if k_bits.shape != (self.T, self.heads, self.D) or v_bits.shape != k_bits.shape:
            raise ValueError("bad block shape")
        s = self.slot_of(block_index)
        self.k[s] = k_bits
        self.v[s] = v_bits
        if flags == STAGE:
            return -1
        evicted = self.slot_block[s]
        self.slot_block[s] = block_index
        self.next_block = block_index + 1
        return evicted

    def window(self, block_index: int):
        """Concatenated K, V ([n*T, H, D] bits) of the committed blocks visible to block_index."""
        if block_index != self.next_block:
            raise RuntimeError("attention is defined for the next block only")
        ks, vs = [], []
        for b in visible_blocks(block_index, self.slots):
            s = self.slot_of(b)
            if self.slot_block[s] != b:
                raise RuntimeError("visible block is not in the ring")
            ks.append(self.k[s])
            vs.append(self.v[s])
        if not ks:
            e = np.zeros((0, self.heads, self.D), dtype=self.dtype)
            return e, e.copy()
        return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)


def block_attn_ref(q_bits, k_self_bits, v_self_bits, cache: RingCacheRef, block_index: int,
                   scale: float, heads=None, rows=None):
    """Attention of block b: keys = visible committed blocks + the block itself, all visible."""
    kw, vw = cache.window(block_index)
    k_all = np.concatenate([kw, k_self_bits], axis=0)
    v_all = np.concatenate([vw, v_self_bits], axis=0)
    return attn_ref(q_bits, k_all, v_all, scale, heads=heads, rows=rows)


# --------------------------------------------------------------------------
# 8-bit variant (Sec. 2 "Video generation": quantised attention kernels are named as orthogonal
# speed-ups; the paper fixes no format, so this is the library's choice: OCP E4M3 codes with one
# static scale per head, x ~ scale_h * decode(code))
# --------------------------------------------------------------------------


def e4m3_decode(codes) -> np.ndarray:
    """E4M3 byte -> float64 from the format's definition: 1 sign, 4 exponent (bias 7), 3 mantissa bits;
    exponent field 0 = subnormal (mantissa * 2^-9); no infinities; S.1111.111 is NaN; largest finite 448."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    mag = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7.0))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return sign * mag


def e4m3_encode(x) -> np.ndarray:
    """Nearest E4M3 value, ties to the even code, magnitudes beyond 448 saturate to 448, NaN -> 0x7F.
    One rounding from the exact input (the 127 non-negative finite values are searched directly)."""
    x = np.asarray(x, dtype=np.float64)
    grid = e4m3_decode(np.arange(0x7F, dtype=np.uint8))             # 0 .. 448, increasing with the code
    a = np.minimum(np.abs(np.nan_to_num(x, nan=0.0)), 448.0)
    hi = np.clip(np.searchsorted(grid, a, side="left"), 0, 0x7E)       # first code with value >= a
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = grid[hi] - a, a - grid[lo]
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    code = code | np.where(np.signbit(x), 0x80, 0).astype(np.uint8)
    return np.where(np.isnan(x), np.uint8(0x7F), code).astype(np.uint8)


def quant_e4m3_ref(x_bits: np.ndarray, inv_scale: np.ndarray) -> np.ndarray:
    """bf16 [tokens, heads, dim] -> E4M3 codes: the element times its head's inverse scale as ONE fp32
    multiplication (round to nearest), then the rounding of e4m3_encode."""
    x = bf16_to_f32(x_bits)
    inv = np.asarray(inv_scale, dtype=np.float32).reshape(1, -1, 1)
    with np.errstate(over="ignore"):
        y = (x * inv).astype(np.float32)
    return e4m3_encode(y.astype(np.float64))


def attn_e4m3_ref(q8: np.ndarray, k8: np.ndarray, v8: np.ndarray, qk_descale, v_descale, scale: float,
                  heads=None, rows=None, row_chunk: int = 1024):
    """Attention on dequantised operands, in fp64, nothing else rounded:
      s_j = scale * qk_descale[h] * <dec(q_i), dec(k_j)>,  o = v_descale[h] * sum_j softmax(s)_j dec(v_j).
    qk_descale[h] is the product of the q and k scales of head h, v_descale[h] the v scale.
    Same conventions and return values as attn_ref."""
    Tq, H, D = q8.shape
    heads = list(range(H)) if heads is None else list(heads)
    rows = np.arange(Tq) if rows is None else np.asarray(rows, dtype=np.int64)
    qk_descale = np.asarray(qk_descale, dtype=np.float64)
    v_descale = np.asarray(v_descale, dtype=np.float64)
    o = np.empty((rows.size, len(heads), D), dtype=np.float64)
    lse = np.empty((len(heads), rows.size), dtype=np.float64)
    for hi, h in enumerate(heads):
        kh = e4m3_decode(k8[:, h, :])
        vh = e4m3_decode(v8[:, h, :])
        for r0 in range(0, rows.size, row_chunk):
            rr = rows[r0:r0 + row_chunk]
            qh = e4m3_decode(q8[rr, h, :])
            s = (qh @ kh.T) * (scale * qk_descale[h])
            m = s.max(axis=1, keepdims=True)
            p = np.exp(s - m)
            l = p.sum(axis=1, keepdims=True)
            o[r0:r0 + rr.size, hi, :] = (p @ vh) / l * v_descale[h]
            lse[hi, r0:r0 + rr.size] = (m + np.log(l))[:, 0]
    return o, lse


def block_attn_e4m3_ref(q8, k_self8, v_self8, cache: "RingCacheRef", block_index: int, qk_descale, v_descale,
                        scale: float, heads=None, rows=None):
    """attn_e4m3_ref of block b against a ring of E4M3 codes (RingCacheRef with dtype uint8) and itself."""
    kw, vw = cache.window(block_index)
    k_all = np.concatenate([kw, k_self8], axis=0)
    v_all = np.concatenate([vw, v_self8], axis=0)
    return attn_e4m3_ref(q8, k_all, v_all, qk_descale, v_descale, scale, heads=heads, rows=rows)


# ---- finer scales: one power-of-two scale per tile of 128 consecutive tokens of a block and per head --------
# (the library's choice again, Sec. 2 fixing none: the granularity at which a block's K/V enter the ring, so that
# a block, or a stretch of one, with a different magnitude keeps the format's 3 mantissa bits)

E4M3_TILE_TOKENS = 128
E4M3_SCALE_EXP_MIN, E4M3_SCALE_EXP_MAX = -126, 120


def e4m3_tile_scale_exponent(amax: float) -> int:
    """The smallest integer e in [-126, 120] with amax <= 448 * 2^e: the tile's scale is 2^e, so that its
    largest magnitude lands in (224, 448] whenever e is not clamped.  A non-finite amax takes the largest e."""
    amax = float(amax)
    if not np.isfinite(amax):
        return E4M3_SCALE_EXP_MAX
    for e in range(E4M3_SCALE_EXP_MIN, E4M3_SCALE_EXP_MAX + 1):
        if amax <= 448.0 * 2.0 ** e:
            return e
    return E4M3_SCALE_EXP_MAX


def quant_e4m3_tiled_ref(x_bits: np.ndarray):
    """bf16 [tokens, heads, dim] -> (codes [tokens, heads, dim], scales float32 [heads, tiles]).
    Tile t of head h is tokens [128 t, 128 t + 128) (the last one may be short); its scale is 2^e with e from
    e4m3_tile_scale_exponent of the largest finite-or-infinite magnitude in the tile (NaN elements do not count);
    codes are e4m3_encode(x / scale), the division by a power of two being exact."""
    x = bf16_to_f64(x_bits)
    T, H, D = x.shape
    tiles = (T + E4M3_TILE_TOKENS - 1) // E4M3_TILE_TOKENS
    codes = np.empty((T, H, D), dtype=np.uint8)
    scales = np.empty((H, tiles), dtype=np.float32)
    for h in range(H):
        for t in range(tiles):
            r0, r1 = t * E4M3_TILE_TOKENS, min(T, (t + 1) * E4M3_TILE_TOKENS)
            tile = x[r0:r1, h, :]
            mags = np.abs(tile[~np.isnan(tile)])
            e = e4m3_tile_scale_exponent(mags.max() if mags.size else 0.0)
            scales[h, t] = np.float32(2.0 ** e)
            with np.errstate(over="ignore"):
                codes[r0:r1, h, :] = e4m3_encode(tile * 2.0 ** -e)
    return codes, scales


def e4m3_token_scales(scales: np.ndarray, tokens: int) -> np.ndarray:
    """Tile scales [heads, tiles] -> one scale per token [tokens, heads] (float64)."""
    return np.repeat(np.asarray(scales, dtype=np.float64), E4M3_TILE_TOKENS, axis=1)[:, :tokens].T.copy()


def attn_e4m3_rowscaled_ref(q8, q_scale, k8, k_scale, v8, v_scale, scale: float, heads=None, rows=None,
                            row_chunk: int = 1024):
    """Attention on operands dequantised with one scale per (token, head), in fp64, nothing else rounded:
      q_i = q_scale[i, h] dec(q8_i), k_j = k_scale[j, h] dec(k8_j), v_j = v_scale[j, h] dec(v8_j),
      o_i = sum_j softmax_j(scale <q_i, k_j>) v_j.
    q_scale is [query tokens, heads], k_scale and v_scale [keys, heads].  Same return values as attn_ref."""
    Tq, H, D = q8.shape
    heads = list(range(H)) if heads is None else list(heads)
    rows = np.arange(Tq) if rows is None else np.asarray(rows, dtype=np.int64)
    q_scale, k_scale, v_scale = (np.asarray(a, dtype=np.float64) for a in (q_scale, k_scale, v_scale))
    o = np.empty((rows.size, len(heads), D), dtype=np.float64)
    lse = np.empty((len(heads), rows.size), dtype=np.float64)
    for hi, h in enumerate(heads):
        kh = e4m3_decode(k8[:, h, :]) * k_scale[:, h, None]
        vh = e4m3_decode(v8[:, h, :]) * v_scale[:, h, None]
        for r0 in range(0, rows.size, row_chunk):
            rr = rows[r0:r0 + row_chunk]
            qh = e4m3_decode(q8[rr, h, :]) * q_scale[rr, h, None]
            s = (qh @ kh.T) * scale
            m = s.max(axis=1, keepdims=True)
            p = np.exp(s - m)
            l = p.sum(axis=1, keepdims=True)
            o[r0:r0 + rr.size, hi, :] = (p @ vh) / l
            lse[hi, r0:r0 + rr.size] = (m + np.log(l))[:, 0]
    return o, lse


# --------------------------------------------------------------------------
# Router (Sec. 3: policy pi, Eq. (1) worst-frame aggregation, forced rejection of block 0)
# --------------------------------------------------------------------------


def route_ref(scores: np.ndarray, frame_offsets, num_blocks: int, frames_per_block: int,
              first_block_index: int, tau: float):
    """accept_b = (global block index != 0) and (min_i score[b, i] >= tau), in fp32.

    ``scores`` is flat fp32; block b owns scores[frame_offsets[b]:frame_offsets[b+1]],
    or frames_per_block consecutive values when frame_offsets is None.  The
    minimum is taken left to right with a strict '<', so ties (and +0/-0) keep
    the lowest index; any NaN frame makes q_min that NaN (lowest such index)
    and the block is rejected.  Returns (accept u8[B], q_min f32[B], argmin i32[B]).

    Ragged input the paper does not speak of (Eq. (1) presumes F >= 1 frames): a block
    without frames is rejected with q_min NaN and argmin -1, and so is a block whose
    range runs backwards or leaves [frame_offsets[0], frame_offsets[B]] (the offsets are
    meant to be non-decreasing; only the two ends of the array are trusted).  With a
    fixed frame count such a block cannot occur and frames_per_block < 1 is an error.
    """
    s = np.asarray(scores, dtype=np.float32).reshape(-1)
    tau32 = np.float32(tau)
    accept = np.zeros(num_blocks, dtype=np.uint8)
    q_min = np.zeros(num_blocks, dtype=np.float32)
    argmin = np.zeros(num_blocks, dtype=np.int32)
    if frame_offsets is None and frames_per_block < 1:
        raise ValueError("a block needs at least one frame")
    for b in range(num_blocks):
        if frame_offsets is None:
            lo, hi = b * frames_per_block, (b + 1) * frames_per_block
        else:
            lo, hi = int(frame_offsets[b]), int(frame_offsets[b + 1])
            all_lo, all_hi = int(frame_offsets[0]), int(frame_offsets[num_blocks])
            if not (all_lo <= lo <= hi <= all_hi) or hi == lo:
                q_min[b], argmin[b], accept[b] = np.float32(np.nan), -1, 0
                continue
        m, idx = s[lo], 0
        for i in range(lo + 1, hi):
            x = s[i]
            if np.isnan(m):
                break
            if np.isnan(x) or x < m:
                m, idx = x, i - lo
        q_min[b] = m
        argmin[b] = idx
        accept[b] = 1 if ((first_block_index + b) != 0 and (not np.isnan(m)) and m >= tau32) else 0
    return accept, q_min, argmin


AGG_MIN = 0      # Eq. (1): worst frame
AGG_MEAN = 1     # Table 2 "Avg-frame scoring": mean of the frame scores
SIGNAL_REWARD = 0   # accept iff aggregate >= tau
SIGNAL_RANDOM = 1   # Table 2 "random routing": accept iff a uniform draw < p, the scores are ignored


def route_policy_ref(scores, frame_offsets, num_blocks: int, frames_per_block: int, first_block_index: int,
                     tau: float, agg: int = AGG_MIN, signal: int = SIGNAL_REWARD, force_first: bool = True,
                     blocks_per_video: int = 0, uniforms=None, accept_prob: float = 0.0):
    """Routing policy with the variants of the ablation (Sec. 4.3, Table 2).

    Aggregate per block: the worst frame (AGG_MIN, same rules as ``route_ref``) or the fp32 mean
    (AGG_MEAN): the frames are added left to right, every partial sum rounded to fp32, and the sum is
    divided by float32(F) with one more rounding.  Decision: aggregate >= tau (SIGNAL_REWARD), or
    uniforms[b] < float32(accept_prob) with the scores ignored (SIGNAL_RANDOM; the draws are an input).
    ``force_first`` rejects the first block of every video whatever the signal says: global block
    g = first_block_index + b is a first block iff g == 0 (blocks_per_video == 0, one endless stream) or
    g % blocks_per_video == 0.  "Force-reject + random" and plain "Random routing" of Table 2 differ
    only in that flag.  Returns (accept u8[B], aggregate f32[B], argmin i32[B]; argmin is -1 for AGG_MEAN).
    """
    s = np.asarray(scores, dtype=np.float32).reshape(-1)
    tau32 = np.float32(tau)
    p32 = np.float32(accept_prob)
    accept = np.zeros(num_blocks, dtype=np.uint8)
    aggv = np.zeros(num_blocks, dtype=np.float32)
    argmin = np.full(num_blocks, -1, dtype=np.int32)
    for b in range(num_blocks):
        if frame_offsets is None:
            lo, hi = b * frames_per_block, (b + 1) * frames_per_block
        else:
            lo, hi = int(frame_offsets[b]), int(frame_offsets[b + 1])
            all_lo, all_hi = int(frame_offsets[0]), int(frame_offsets[num_blocks])
            if not (all_lo <= lo <= hi <= all_hi) or hi == lo:
                # no frames, or a malformed range: same reading as route_ref (rejected whatever the signal, NaN, -1)
                aggv[b], argmin[b], accept[b] = np.float32(np.nan), -1, 0
                continue
        if hi <= lo:
            raise ValueError("a block needs at least one frame")
        if agg == AGG_MIN:
            m, idx = s[lo], 0
            for i in range(lo + 1, hi):
                if np.isnan(m):
                    break
                x = s[i]
                if np.isnan(x) or x < m:
                    m, idx = x, i - lo
            argmin[b] = idx
        elif agg == AGG_MEAN:
            acc = np.float32(s[lo])
            with np.errstate(invalid="ignore", over="ignore"):
                for i in range(lo + 1, hi):
                    acc = np.float32(acc + s[i])
                m = np.float32(acc / np.float32(hi - lo))
        else:
            raise ValueError("unknown aggregation")
        aggv[b] = m
        g = first_block_index + b
        first = (g == 0) if blocks_per_video == 0 else (g % blocks_per_video == 0)
        if signal == SIGNAL_REWARD:
            ok = (not np.isnan(m)) and m >= tau32
        elif signal == SIGNAL_RANDOM:
            ok = bool(np.float32(uniforms[b]) < p32)
        else:
            raise ValueError("unknown signal")
        accept[b] = 1 if (ok and not (force_first and first)) else 0
    return accept, aggv, argmin


def accept_stats_ref(accept, first_block_index: int = 0, blocks_per_video: int = 0):
    """(accepted, routable) block counts, the first block of every video left out of both
    (accept-rate convention stated in the captions of Tables 1 and 2: the always-regenerated block 0 is not counted)."""
    a = np.asarray(accept).astype(np.int64)
    g = np.arange(a.size, dtype=np.int64) + first_block_index
    first = (g == 0) if blocks_per_video == 0 else (g % blocks_per_video == 0)
    return int(a[~first].sum()), int((~first).sum())


def accept_rate(accept: np.ndarray, first_block_index: int = 0) -> float:
    """Accept rate with block 0 left out of the count (convention of Tables 1 and 2)."""
    a = np.asarray(accept).astype(np.int64)
    idx = np.arange(a.size) + first_block_index
    keep = idx != 0
    return float(a[keep].sum()) / float(max(1, keep.sum()))


# --------------------------------------------------------------------------
# Per-block speculative schedule (Sec. 3 "Inference flow", Fig. 2)
# --------------------------------------------------------------------------


@dataclass
class TraceResult:
    accept: np.ndarray
    q_min: np.ndarray
    drafter_evicted: list = field(default_factory=list)
    target_evicted: list = field(default_factory=list)
    drafter_attn_calls: int = 0
    target_attn_calls: int = 0
    target_source: list = field(default_factory=list)   # per block: "accepted" or "regenerated"


def schedule_ref(num_blocks: int, steps: int, scores: np.ndarray, tau: float,
                 drafter: RingCacheRef, target: RingCacheRef, provider,
                 grid_d, grid_t, frames_per_block_latent: int,
                 tab_d, tab_t, tab_frames: int, on_attention=None) -> TraceResult:
    """Run the per-block flow with the reference pieces.

    For every block b: the drafter takes ``steps`` denoise steps (each: rope q,k
    at frame offset b*frames -> stage k',v -> attention), then its clean K/V are
    committed to the drafter ring unconditionally.  The router scores the block.
    Accepted: the target-shaped K/V of the draft are committed to the target
    ring.  Rejected (always block 0): the target takes ``steps`` steps of its
    own and commits its clean K/V.  ``provider(model, block, kind, step)``
    returns the (q, k, v) bf16 bits of that call (q is None for clean K/V).
    ``on_attention(model, block, step, q_roped, k_roped, v, cache)`` lets a test
    evaluate sampled attention rows at that point.
    """
    scores = np.asarray(scores, dtype=np.float32)
    accept, q_min, _ = route_ref(scores.reshape(-1), None, num_blocks, scores.shape[1], 0, tau)
    res = TraceResult(accept=accept, q_min=q_min)

    def denoise(model, cache, grid, tab, b, kind):
        calls = 0
        for s in range(steps):
            q, k, v = provider(model, b, kind, s)
            fo = b * frames_per_block_latent
            qr = rope_bitspec(q, grid, fo, tab, tab_frames)
            kr = rope_bitspec(k, grid, fo, tab, tab_frames)
            cache.commit(b, kr, v, STAGE)
            if on_attention is not None:
                on_attention(model, b, s, qr, kr, v, cache)
            calls += 1
        return calls

    for b in range(num_blocks):
        res.drafter_attn_calls += denoise("drafter", drafter, grid_d, tab_d, b, "step")
        _, k, v = provider("drafter", b, "clean", 0)
        kr = rope_bitspec(k, grid_d, b * frames_per_block_latent, tab_d, tab_frames)
        res.drafter_evicted.append(drafter.commit(b, kr, v, FINAL))
        if accept[b]:
            _, k, v = provider("target", b, "accepted", 0)
            res.target_source.append("accepted")
        else:
            res.target_attn_calls += denoise("target", target, grid_t, tab_t, b, "step")
            _, k, v = provider("target", b, "clean", 0)
            res.target_source.append("regenerated")
        kr = rope_bitspec(k, grid_t, b * frames_per_block_latent, tab_t, tab_frames)
        res.target_evicted.append(target.commit(b, kr, v, FINAL))
    return res
