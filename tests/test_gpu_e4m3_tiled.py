"""GPU parity of the 8-bit variant with one power-of-two scale per tile of 128 tokens and head: quantiser, ring
commit and fused prologue bit-exact (codes and scales), attention within the bound that the rounding of P allows,
and the exact invariances that power-of-two scales give."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from gpu_utils import Canaries, to_bits, to_dev

pytestmark = pytest.mark.gpu


def gained(bits: np.ndarray, gain) -> np.ndarray:
    """bf16 tensor [tokens, heads, dim] times a gain broadcast over it (rounded to bf16 again)."""
    return O.f32_to_bf16((O.bf16_to_f32(bits) * np.asarray(gain, dtype=np.float32)).astype(np.float32))


def tile_gain(rng, tokens, heads, lo, hi):
    """A power-of-two gain per (tile, head), as an array broadcastable over [tokens, heads, dim]."""
    tiles = (tokens + 127) // 128
    g = 2.0 ** rng.integers(lo, hi + 1, (tiles, heads))
    return np.repeat(g, 128, axis=0)[:tokens, :, None]


def p_rounding_bound_tiled(q, k, v, v_scale, scale, h, rows):
    """Per-element bound on |out - oracle| for head h; q, k, v are the DEQUANTISED operands (float64), v_scale the
    V scale of every key [keys].

    With p_j = exp(s_j - max s) the kernel rounds P_j = 2^e p_j sv_j / sv_then to E4M3, e in [4, 8] (its reference
    maximum lags by at most 2^4 and the window is shifted up by 2^4) and sv_then the largest V scale met so far,
    at most the largest of all, sv_max.  A normal number moves by at most 2^-4 of itself, anything smaller by at
    most 2^-10; the accumulator is later only multiplied by exact powers of two.  In units of the output that is
    |d o| <= sum_j max(2^-4 p_j, 2^-14 sv_max / sv_j) |v_j| / sum_j p_j.
    """
    s = (q[rows, h, :] @ k[:, h, :].T) * scale
    p = np.exp(s - s.max(axis=1, keepdims=True))
    dp = np.maximum(p * 2.0 ** -4, 2.0 ** -14 * (v_scale.max() / v_scale)[None, :])
    return (dp @ np.abs(v[:, h, :])) / p.sum(axis=1, keepdims=True)


def check_attention(out, o_ref, bound, what):
    got = O.bf16_to_f64(to_bits(out))
    err = np.abs(got - o_ref)
    tol = bound + np.abs(o_ref) * 2.0 ** -8 + 1e-30
    assert np.all(err <= tol), (what, float(err.max()), float((err / tol).max()))
    assert err.mean() <= 0.25 * tol.mean(), (what, float(err.mean()), float(tol.mean()))


def test_tiled_quantiser_bit_exact_codes_and_scales():
    rng = np.random.default_rng(8)
    tokens, heads, dim = 300, 5, 128                       # three tiles, the last of 44 tokens
    x = gained(synth.normal_bf16((tokens, heads, dim), 3, 1), tile_gain(rng, tokens, heads, -20, 20))
    x[0:128, 1] = 0                                        # an all-zero tile
    x[130, 2, 5] = 0x7FC0                                  # a NaN element: does not set the scale, becomes the NaN code
    x[140, 2, 6] = 0xFFC0
    x[260, 3, 0] = 0x7F80                                  # +inf: the tile takes the largest scale, the element saturates
    x[128:256, 4] = synth.f32_to_bf16_bits(np.full((128, dim), 2.0 ** -130, dtype=np.float32))     # bf16 subnormals
    x[129, 0, 3] = synth.f32_to_bf16_bits(np.array([448.0 * 2 ** 7], dtype=np.float32))[0]         # exactly 448 * 2^e
    x[257, 0, 3] = synth.f32_to_bf16_bits(np.array([450.0 * 2 ** 7], dtype=np.float32))[0]         # one bf16 step above
    guard = Canaries()
    out = guard.new((tokens, heads, dim), torch.uint8)
    sc = guard.new((heads, 3), torch.float32, float("nan"))
    api.sdvg_quant_e4m3_tiled(to_dev(x), out, sc)
    codes, scales = O.quant_e4m3_tiled_ref(x)
    assert np.array_equal(sc.cpu().numpy().view(np.uint32), scales.view(np.uint32))
    assert np.array_equal(out.cpu().numpy(), codes)
    assert scales[1, 0] == np.float32(2.0 ** -126) and scales[3, 2] == np.float32(2.0 ** 120) and scales[4, 1] == np.float32(2.0 ** -126)
    guard.check()
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_quant_e4m3_tiled(to_dev(x)[:, :, :64].contiguous(), out[:, :, :64].contiguous(), sc)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE


def test_commit_and_fused_prologue_bit_exact_in_ring_and_scale_arrays():
    sh = synth.Shape("e4m3-tiled-ring", heads=3, head_dim=128, frames=2, grid_h=10, grid_w=13, slots=3)   # 260 tokens: 3 tiles
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tabf = 6 * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    ref_tab = O.rope_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w)
    fused = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True, tile_scales=True)
    apart = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True, tile_scales=True)
    ring = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, dtype=np.uint8)
    ks_ref = np.ones((sh.heads, sh.slots, 3), dtype=np.float32)
    vs_ref = np.ones((sh.heads, sh.slots, 3), dtype=np.float32)
    rng = np.random.default_rng(5)
    guard = Canaries()
    guard.watch_cache(fused)
    for b in range(5):
        q, k, v = (gained(synth.block_tensor(sh, 31, b, 0, t), tile_gain(rng, sh.block_tokens, sh.heads, -9, 9))
                   for t in (synth.Q, synth.K, synth.V))
        fo = b * sh.frames
        qr, kr = O.rope_bitspec(q, grid, fo, ref_tab, tabf), O.rope_bitspec(k, grid, fo, ref_tab, tabf)
        q8_ref, qs_ref = O.quant_e4m3_tiled_ref(qr)
        k8_ref, kt_ref = O.quant_e4m3_tiled_ref(kr)
        v8_ref, vt_ref = O.quant_e4m3_tiled_ref(v)
        slot = b % sh.slots
        # staged first (the ring state must not move), then final
        q8 = guard.new(q.shape, torch.uint8)
        qs = guard.new((sh.heads, 3), torch.float32, float("nan"))
        assert api.sdvg_rope3d_qk_commit_e4m3_tiled(fused, to_dev(q), to_dev(k), to_dev(v), q8, qs, grid, fo, tab, tabf, b,
                                                    api.SDVG_STAGE) == -1
        assert fused.state()[2] == b and fused.state()[0] == b
        assert np.array_equal(q8.cpu().numpy(), q8_ref) and np.array_equal(qs.cpu().numpy(), qs_ref)
        ev = api.sdvg_rope3d_qk_commit_e4m3_tiled(fused, None, to_dev(k), to_dev(v), None, None, grid, fo, tab, tabf, b,
                                                  api.SDVG_FINAL)
        # the same through the separate calls
        dq, dk = torch.empty_like(to_dev(q)), torch.empty_like(to_dev(k))
        api.sdvg_rope3d_qk(to_dev(q), to_dev(k), dq, dk, grid, fo, tab, tabf)
        q8b = torch.zeros_like(q8)
        qsb = torch.zeros_like(qs)
        api.sdvg_quant_e4m3_tiled(dq, q8b, qsb)
        ev2 = api.sdvg_kv_commit_e4m3_tiled(apart, dk, to_dev(v), b, api.SDVG_FINAL)
        assert ev == ev2 == ring.commit(b, k8_ref, v8_ref, O.FINAL)
        assert torch.equal(q8, q8b) and torch.equal(qs, qsb)
        ks_ref[:, slot], vs_ref[:, slot] = kt_ref, vt_ref
        for c in (fused, apart):
            assert c.state()[:2] == (ring.next_block, ring.slot_block)
            for s in range(sh.slots):
                if ring.slot_block[s] >= 0:
                    gk, gv = c.read_block(s)
                    assert np.array_equal(gk.cpu().numpy(), ring.k[s]) and np.array_equal(gv.cpu().numpy(), ring.v[s])
                    assert np.array_equal(c.k_scale[:, s].cpu().numpy(), ks_ref[:, s])
                    assert np.array_equal(c.v_scale[:, s].cpu().numpy(), vs_ref[:, s])
        guard.check()
    # a ring without scale arrays, a bf16 ring, an out-of-order block
    plain = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    bf = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    k = to_dev(synth.block_tensor(sh, 31, 0, 0, synth.K))
    for cache, status in ((plain, api.SDVG_ERR_BAD_STATE), (bf, api.SDVG_ERR_BAD_SHAPE)):
        with pytest.raises(api.SdvgError) as e:
            api.sdvg_kv_commit_e4m3_tiled(cache, k, k, 0, api.SDVG_FINAL)
        assert e.value.status == status
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_kv_commit_e4m3_tiled(fused, k, k, 9, api.SDVG_FINAL)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    for c in (fused, apart, plain, bf):
        c.close()


def run_sequence(sh, nblocks, seed, gain_range, q_std=1.0, rows_per_head=None):
    """Blocks with a magnitude of their own per (tile, head) and tensor through a tile-scaled ring; every block's
    attention (keys: the visible slots, the block itself staged) against the oracle on the dequantised operands."""
    H, T = sh.heads, sh.block_tokens
    tiles = (T + 127) // 128
    cache = api.Cache(sh.slots, H, T, sh.head_dim, e4m3=True, tile_scales=True)
    ring8 = O.RingCacheRef(sh.slots, H, T, sh.head_dim, dtype=np.uint8)
    scales = {}                                  # block -> (k token scales, v token scales) [T, H]
    ws = api.attn_workspace()
    rng = np.random.default_rng(seed)
    guard = Canaries()
    guard.watch_cache(cache)
    lo, hi = gain_range
    for b in range(nblocks):
        q = gained(synth.block_tensor(sh, seed, b, 0, synth.Q, std=q_std), tile_gain(rng, T, H, lo, hi))
        k = gained(synth.block_tensor(sh, seed, b, 0, synth.K), tile_gain(rng, T, H, lo, hi))
        v = gained(synth.block_tensor(sh, seed, b, 0, synth.V), tile_gain(rng, T, H, 2 * lo, 2 * hi))
        q8, qs = O.quant_e4m3_tiled_ref(q)
        k8, ks = O.quant_e4m3_tiled_ref(k)
        v8, vs = O.quant_e4m3_tiled_ref(v)
        dq8 = guard.new(q8.shape, torch.uint8)
        dqs = guard.new((H, tiles), torch.float32)
        api.sdvg_quant_e4m3_tiled(to_dev(q), dq8, dqs)
        assert np.array_equal(dq8.cpu().numpy(), q8) and np.array_equal(dqs.cpu().numpy(), qs)
        api.sdvg_kv_commit_e4m3_tiled(cache, to_dev(k), to_dev(v), b, api.SDVG_STAGE)
        out = guard.new((T, H, sh.head_dim), torch.bfloat16, float("nan"))
        lse = guard.new((H, T), torch.float32, float("nan"))
        api.sdvg_block_attn_fwd_e4m3_tiled(dq8, dqs, cache, b, out, lse, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        scales[b] = (O.e4m3_token_scales(ks, T), O.e4m3_token_scales(vs, T))
        vis = O.visible_blocks(b, sh.slots)
        kw, vw = ring8.window(b)
        k_all, v_all = np.concatenate([kw, k8]), np.concatenate([vw, v8])
        ksc = np.concatenate([scales[n][0] for n in vis] + [scales[b][0]])
        vsc = np.concatenate([scales[n][1] for n in vis] + [scales[b][1]])
        qsc = O.e4m3_token_scales(qs, T)
        qd = O.e4m3_decode(q8) * qsc[:, :, None]
        kd = O.e4m3_decode(k_all) * ksc[:, :, None]
        vd = O.e4m3_decode(v_all) * vsc[:, :, None]
        for h in range(H):
            rows = np.arange(T) if rows_per_head is None else np.sort(rng.choice(T, rows_per_head, replace=False))
            o_ref, lse_ref = O.attn_e4m3_rowscaled_ref(q8, qsc, k_all, ksc, v_all, vsc, sh.scale, heads=[h], rows=rows)
            bound = p_rounding_bound_tiled(qd, kd, vd, vsc[:, h], sh.scale, h, rows)
            check_attention(out[rows, h], o_ref[:, 0], bound, (sh.name, b, h))
            assert np.allclose(lse.cpu().numpy()[h, rows], lse_ref[0], rtol=1e-5, atol=2e-3)
        api.sdvg_kv_commit_e4m3_tiled(cache, to_dev(k), to_dev(v), b, api.SDVG_FINAL)
        ring8.commit(b, k8, v8, O.FINAL)
        guard.check()
    cache.close()


def test_every_fill_level_ragged_tiles_and_wraparound():
    # 230 tokens: two tiles per block, the second of 102 tokens; the ring wraps twice; mild magnitude differences
    sh = synth.Shape("e4m3-tiled-ragged", heads=3, head_dim=128, frames=2, grid_h=5, grid_w=23, slots=3)
    run_sequence(sh, 6, 43, (-1, 1))


def test_odd_tiles_odd_heads_peaked_rows_and_wide_magnitudes():
    # 300 tokens = 3 tiles per head (pairs that straddle heads, a split tile whose two halves end on different
    # V scales); large logits; K per tile over 2^-3 .. 2^3 and V over 2^-6 .. 2^6
    sh = synth.Shape("e4m3-tiled-odd", heads=3, head_dim=128, frames=1, grid_h=12, grid_w=25, slots=4)
    run_sequence(sh, 5, 9, (-3, 3), q_std=2.0)


def test_single_slot_and_single_tile():
    sh = synth.Shape("e4m3-tiled-one", heads=1, head_dim=128, frames=1, grid_h=7, grid_w=11, slots=1)
    run_sequence(sh, 3, 3, (-2, 2))


def _one_block(T, H, q, k, v, scale, ws):
    cache = api.Cache(2, H, T, 128, e4m3=True, tile_scales=True)
    tiles = (T + 127) // 128
    q8 = torch.empty((T, H, 128), dtype=torch.uint8, device="cuda")
    qs = torch.empty((H, tiles), dtype=torch.float32, device="cuda")
    api.sdvg_quant_e4m3_tiled(to_dev(q), q8, qs)
    api.sdvg_kv_commit_e4m3_tiled(cache, to_dev(k), to_dev(v), 0, api.SDVG_STAGE)
    out = torch.full((T, H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((H, T), device="cuda")
    api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, cache, 0, out, lse, scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    cache.close()
    return out, lse


def test_power_of_two_gains_move_through_exactly():
    """Scales are powers of two, so a power-of-two gain on a whole tensor changes the scales and not the codes:
    v * 2^a gives out * 2^a bit for bit, and q * 2^a with k * 2^-a gives the same bits (the logits are unchanged).
    Holds far outside the range one static scale could cover."""
    T, H = 300, 2
    ws = api.attn_workspace()
    q, k, v = (synth.normal_bf16((T, H, 128), 77, i) for i in range(3))
    base, lse0 = _one_block(T, H, q, k, v, 0.09, ws)
    assert not torch.isnan(base.float()).any()
    for a in (-40, -11, 13, 30):
        moved, lse1 = _one_block(T, H, q, k, gained(v, 2.0 ** a), 0.09, ws)
        assert torch.equal((base.float() * 2.0 ** a).to(torch.bfloat16).view(torch.int16), moved.view(torch.int16)), a
        assert torch.equal(lse0, lse1)
        same, lse2 = _one_block(T, H, gained(q, 2.0 ** a), gained(k, 2.0 ** -a), v, 0.09, ws)
        assert torch.equal(base.view(torch.int16), same.view(torch.int16)), a
        assert torch.equal(lse0, lse2)


def test_closed_forms():
    T, H = 300, 2
    ws = api.attn_workspace()
    rng = np.random.default_rng(2)
    # q = 0: every key weighs the same whatever K holds, so the output is the mean of the dequantised V, tiles of
    # different magnitude included (P is a power of two there: no rounding before the output)
    v = gained(synth.normal_bf16((T, H, 128), 5, 0), tile_gain(rng, T, H, -5, 5))
    k = synth.normal_bf16((T, H, 128), 5, 1)
    q0 = np.zeros((T, H, 128), dtype=np.uint16)
    out, lse = _one_block(T, H, q0, k, v, 0.3, ws)
    v8, vs = O.quant_e4m3_tiled_ref(v)
    mean_v = (O.e4m3_decode(v8) * O.e4m3_token_scales(vs, T)[:, :, None]).mean(axis=0)
    got = O.bf16_to_f64(to_bits(out))
    assert np.all(np.abs(got - mean_v[None]) <= np.abs(mean_v[None]) * 2.0 ** -8 + 1e-6 * np.abs(mean_v).max())
    assert np.allclose(lse.cpu().numpy(), np.log(T), atol=1e-5)
    # one key dominates by far: the output is that key's dequantised value bit for bit, also when its tile has a
    # small V scale and the other tiles large ones
    kd = np.zeros((T, H, 128), dtype=np.float32)
    kd[140] = 2.0
    qd = np.ones((T, H, 128), dtype=np.float32)
    vg = np.ones((T, H, 1))
    vg[128:256] = 2.0 ** -7
    v2 = gained(synth.normal_bf16((T, H, 128), 5, 2), vg)
    out, _ = _one_block(T, H, O.f32_to_bf16(qd), O.f32_to_bf16(kd), v2, 0.5, ws)
    v8, vs = O.quant_e4m3_tiled_ref(v2)
    want = O.e4m3_decode(v8[140]) * O.e4m3_token_scales(vs, T)[140][:, None]
    assert np.array_equal(O.bf16_to_f64(to_bits(out)), np.broadcast_to(want[None], (T, H, 128)))


def test_argument_checks():
    sh = synth.Shape("e4m3-tiled-args", heads=2, head_dim=128, frames=1, grid_h=4, grid_w=40, slots=2)
    ws = api.attn_workspace()
    T, H = sh.block_tokens, sh.heads
    q8 = torch.zeros((T, H, 128), dtype=torch.uint8, device="cuda")
    qs = torch.ones((H, 2), device="cuda")
    out = torch.empty((T, H, 128), dtype=torch.bfloat16, device="cuda")
    k = to_dev(synth.block_tensor(sh, 1, 0, 0, synth.K))
    tiled = api.Cache(sh.slots, H, T, 128, e4m3=True, tile_scales=True)
    with pytest.raises(api.SdvgError) as e:                  # the block is not staged
        api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, tiled, 0, out, None, 0.1, ws)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    api.sdvg_kv_commit_e4m3_tiled(tiled, k, k, 0, api.SDVG_STAGE)
    api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, tiled, 0, out, None, 0.1, ws)
    with pytest.raises(api.SdvgError) as e:                  # wrong block
        api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, tiled, 1, out, None, 0.1, ws)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    plain = api.Cache(sh.slots, H, T, 128, e4m3=True)
    inv = torch.ones(H, device="cuda")
    api.sdvg_kv_commit_e4m3(plain, k, k, inv, inv, 0, api.SDVG_STAGE)
    with pytest.raises(api.SdvgError) as e:                  # no scale arrays attached
        api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, plain, 0, out, None, 0.1, ws)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    bf = api.Cache(sh.slots, H, T, 128)
    api.sdvg_kv_commit(bf, k, k, 0, api.SDVG_STAGE)
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, bf, 0, out, None, 0.1, ws)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE
    # tile scales cannot be attached to a bf16 ring
    assert api.lib().sdvg_cache_set_tile_scales(bf.handle, qs.data_ptr(), qs.data_ptr()) == api.SDVG_ERR_BAD_SHAPE
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    for c in (tiled, plain, bf):
        c.close()


def test_full_size_target_shape_sampled_rows():
    # 40 heads x d128, 4680 queries x 7 slots of 37 tiles: the shape the bench times; blocks of different magnitude
    sh = synth.WAN_14B
    H, T = sh.heads, sh.block_tokens
    cache = api.Cache(sh.slots, H, T, sh.head_dim, e4m3=True, tile_scales=True)
    ws = api.attn_workspace()
    pool = synth.TensorPool(sh, 9)
    gains = [1.0, 8.0, 0.25, 1.0, 64.0, 0.5, 2.0]
    for b in range(sh.slots):
        k, v = gained(pool.get(b, 0, synth.K), gains[b] ** 0.5), gained(pool.get(b, 0, synth.V), gains[b])
        api.sdvg_kv_commit_e4m3_tiled(cache, to_dev(k), to_dev(v), b, api.SDVG_FINAL if b < sh.slots - 1 else api.SDVG_STAGE)
    b = sh.slots - 1
    q = pool.get(b, 0, synth.Q)
    q8d = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
    qsd = torch.zeros((H, cache.tiles), dtype=torch.float32, device="cuda")
    api.sdvg_quant_e4m3_tiled(to_dev(q), q8d, qsd)
    out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    api.sdvg_block_attn_fwd_e4m3_tiled(q8d, qsd, cache, b, out, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    assert not torch.isnan(out.float()).any()
    ks, vs = [], []
    for s in range(sh.slots):
        gk, gv = cache.read_block(s)
        ks.append(gk.cpu().numpy())
        vs.append(gv.cpu().numpy())
    k_all, v_all, q8 = np.concatenate(ks), np.concatenate(vs), q8d.cpu().numpy()
    ksc = np.concatenate([O.e4m3_token_scales(cache.k_scale[:, s].cpu().numpy(), T) for s in range(sh.slots)])
    vsc = np.concatenate([O.e4m3_token_scales(cache.v_scale[:, s].cpu().numpy(), T) for s in range(sh.slots)])
    qsc = O.e4m3_token_scales(qsd.cpu().numpy(), T)
    # the ring holds the oracle's codes and scales (one block, one head, checked in full)
    c4, s4 = O.quant_e4m3_tiled_ref(gained(pool.get(4, 0, synth.V), gains[4])[:, 13:14])
    assert np.array_equal(vs[4][:, 13], c4[:, 0]) and np.array_equal(cache.v_scale[13, 4].cpu().numpy(), s4[0])
    rng = np.random.default_rng(0)
    for h in (0, 13, 39):
        rows = np.sort(rng.choice(T, 24, replace=False))
        rows[-1] = T - 1
        o_ref, _ = O.attn_e4m3_rowscaled_ref(q8, qsc, k_all, ksc, v_all, vsc, sh.scale, heads=[h], rows=rows)
        qd = O.e4m3_decode(q8[:, h:h + 1]) * qsc[:, h:h + 1, None]
        kd = O.e4m3_decode(k_all[:, h:h + 1]) * ksc[:, h:h + 1, None]
        vd = O.e4m3_decode(v_all[:, h:h + 1]) * vsc[:, h:h + 1, None]
        bound = p_rounding_bound_tiled(qd, kd, vd, vsc[:, h], sh.scale, 0, rows)
        check_attention(out[rows, h], o_ref[:, 0], bound, ("14b", h))
    cache.close()


def whole_path_errors(gain_q, gain_k, gain_v, heads=2, seed=81):
    """Relative rms error of the whole 8-bit path against the oracle's exact attention on the unquantised bf16
    inputs, at the drafter's window (4680 queries x 14040 keys), for the tile-scaled variant and for the
    static-scale variant whose scales were sized for N(0, 1) tensors (4.5 standard deviations at 448), when the
    tensors arrive multiplied by the given gains."""
    sh = synth.Shape("f8q-tiled", heads=heads, head_dim=128, frames=3, grid_h=30, grid_w=52, slots=3)
    T = sh.block_tokens
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(T, 96, replace=False))
    ct = api.Cache(sh.slots, heads, T, sh.head_dim, e4m3=True, tile_scales=True)
    cs = api.Cache(sh.slots, heads, T, sh.head_dim, e4m3=True)
    ws = api.attn_workspace()
    inv = torch.full((heads,), 448 / 4.5, device="cuda")
    desc = 1.0 / inv
    ks, vs = [], []
    for b in range(sh.slots):
        ks.append(gained(synth.block_tensor(sh, seed, b, 0, synth.K), gain_k))
        vs.append(gained(synth.block_tensor(sh, seed, b, 0, synth.V), gain_v))
        flag = api.SDVG_FINAL if b < sh.slots - 1 else api.SDVG_STAGE
        api.sdvg_kv_commit_e4m3_tiled(ct, to_dev(ks[b]), to_dev(vs[b]), b, flag)
        api.sdvg_kv_commit_e4m3(cs, to_dev(ks[b]), to_dev(vs[b]), inv, inv, b, flag)
    b = sh.slots - 1
    q = gained(synth.block_tensor(sh, seed, b, 0, synth.Q), gain_q)
    q8 = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
    qs = torch.zeros((heads, ct.tiles), device="cuda")
    api.sdvg_quant_e4m3_tiled(to_dev(q), q8, qs)
    out_t = torch.full((T, heads, sh.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    api.sdvg_block_attn_fwd_e4m3_tiled(q8, qs, ct, b, out_t, None, sh.scale, ws)
    q8s = torch.zeros_like(q8)
    api.sdvg_quant_e4m3(to_dev(q), inv, q8s)
    out_s = torch.full_like(out_t, float("nan"))
    api.sdvg_block_attn_fwd_e4m3(q8s, None, None, cs, b, desc * desc, desc, out_s, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    o_ref, _ = O.attn_ref(q, np.concatenate(ks), np.concatenate(vs), sh.scale, rows=rows)
    res = {}
    for name, out in (("tiled", out_t), ("static", out_s)):
        d = O.bf16_to_f64(to_bits(out))[rows] - o_ref
        res[name] = float(np.sqrt((d ** 2).mean() / (o_ref ** 2).mean()))
    ct.close()
    cs.close()
    return res


def test_whole_path_error_does_not_depend_on_the_magnitude_the_data_arrives_with():
    # N(0, 1) data, for which the static scales were sized: both variants cost the format's 3 mantissa bits (about 5%).
    unit = whole_path_errors(1.0, 1.0, 1.0)
    assert unit["tiled"] <= 0.07 and unit["static"] <= 0.07, unit
    # The same data with V 2^11 times smaller and K 2^6 times larger (q 2^-6: the logits are unchanged): the tile
    # scales follow, the result is the same to the bit up to the gain, so the error is the same; the static scales
    # put V below the format's smallest number and saturate K.
    moved = whole_path_errors(2.0 ** -6, 2.0 ** 6, 2.0 ** -11)
    assert abs(moved["tiled"] - unit["tiled"]) <= 1e-3, (unit, moved)
    assert moved["static"] >= 0.5, moved


def test_schedule_with_tile_scaled_rings_follows_the_flow_and_holds_the_oracle_codes_and_scales():
    from paper_2604_17397_b200 import schedule
    from test_gpu_schedule import Provider

    sh_d = synth.Shape("d8t", heads=3, head_dim=128, frames=3, grid_h=4, grid_w=13, slots=3)      # 156 tokens: 2 tiles
    sh_t = synth.Shape("t8t", heads=5, head_dim=128, frames=3, grid_h=4, grid_w=13, slots=4)
    B, steps, tau, seed = 9, 2, -0.7, 61
    tabf = B * sh_t.frames
    scores = synth.calibrated_scores(B, 12, seed)
    prov = Provider(sh_d, sh_t, seed)
    models = {}
    for name, sh in (("drafter", sh_d), ("target", sh_t)):
        cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True, tile_scales=True)
        tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
        models[name] = schedule.ModelState(cache, (sh.frames, sh.grid_h, sh.grid_w), tab, tabf, sh.scale)
    shapes = {"drafter": sh_d, "target": sh_t}
    checked = []

    def on_attention(model, b, s, q8, out):
        if (b + s) % 3:
            return
        m, sh = models[model], shapes[model]
        T = sh.block_tokens
        ks, vs, ksc, vsc = [], [], [], []
        for blk in range(max(0, b - (sh.slots - 1)), b + 1):       # the window as the device ring holds it now
            slot = blk % sh.slots
            gk, gv = m.cache.read_block(slot)
            ks.append(gk.cpu().numpy())
            vs.append(gv.cpu().numpy())
            ksc.append(O.e4m3_token_scales(m.cache.k_scale[:, slot].cpu().numpy(), T))
            vsc.append(O.e4m3_token_scales(m.cache.v_scale[:, slot].cpu().numpy(), T))
        k_all, v_all, ksc, vsc = np.concatenate(ks), np.concatenate(vs), np.concatenate(ksc), np.concatenate(vsc)
        qsc = O.e4m3_token_scales(m.q_tile_scale.cpu().numpy(), T)
        r = np.random.default_rng([seed, b, s])
        h = int(r.integers(sh.heads))
        rows = np.sort(r.choice(T, 16, replace=False))
        q8n = q8.cpu().numpy()
        o_ref, _ = O.attn_e4m3_rowscaled_ref(q8n, qsc, k_all, ksc, v_all, vsc, sh.scale, heads=[h], rows=rows)
        qd = O.e4m3_decode(q8n) * qsc[:, :, None]
        kd = O.e4m3_decode(k_all) * ksc[:, :, None]
        vd = O.e4m3_decode(v_all) * vsc[:, :, None]
        bound = p_rounding_bound_tiled(qd, kd, vd, vsc[:, h], sh.scale, h, rows)
        check_attention(out[torch.from_numpy(rows).cuda(), h], o_ref[:, 0], bound, (model, b, s))
        checked.append((model, b, s))

    res = schedule.run_schedule(B, steps, torch.from_numpy(scores).cuda(), tau, models["drafter"], models["target"],
                                prov.device, on_attention=on_attention)
    for m in models.values():
        assert api.sdvg_block_attn_status(m.workspace) == api.SDVG_OK
    assert len(checked) >= 6 and {c[0] for c in checked} == {"drafter", "target"}
    # the flow is that of the oracle's schedule; its bf16 rings, quantised tile by tile, are what the rings must hold
    rd = O.RingCacheRef(sh_d.slots, sh_d.heads, sh_d.block_tokens, sh_d.head_dim)
    rt = O.RingCacheRef(sh_t.slots, sh_t.heads, sh_t.block_tokens, sh_t.head_dim)
    want = O.schedule_ref(B, steps, scores, tau, rd, rt, prov.bits, (sh_d.frames, sh_d.grid_h, sh_d.grid_w),
                          (sh_t.frames, sh_t.grid_h, sh_t.grid_w), sh_t.frames,
                          O.rope_table(128, tabf, sh_d.grid_h, sh_d.grid_w), O.rope_table(128, tabf, sh_t.grid_h, sh_t.grid_w),
                          tabf)
    assert np.array_equal(res.accept, want.accept) and res.target_source == want.target_source
    assert res.drafter_evicted == want.drafter_evicted and res.target_evicted == want.target_evicted
    assert res.drafter_attn_calls == want.drafter_attn_calls and res.target_attn_calls == want.target_attn_calls
    for name, ref in (("drafter", rd), ("target", rt)):
        cache = models[name].cache
        assert cache.state()[:2] == (ref.next_block, ref.slot_block)
        for s in range(ref.slots):
            gk, gv = cache.read_block(s)
            k8, ks = O.quant_e4m3_tiled_ref(ref.k[s])
            v8, vs = O.quant_e4m3_tiled_ref(ref.v[s])
            assert np.array_equal(gk.cpu().numpy(), k8) and np.array_equal(gv.cpu().numpy(), v8), (name, s)
            assert np.array_equal(cache.k_scale[:, s].cpu().numpy(), ks) and np.array_equal(cache.v_scale[:, s].cpu().numpy(), vs)
        cache.close()


def test_block_steps_of_a_tile_scaled_ring_replayed_from_a_cuda_graph_equal_the_eager_calls():
    from paper_2604_17397_b200 import schedule

    sh = synth.Shape("graph8t", heads=3, head_dim=128, frames=3, grid_h=6, grid_w=11, slots=3)
    tabf, steps = 4 * sh.frames, 3
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True, tile_scales=True)
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    m = schedule.ModelState(cache, (sh.frames, sh.grid_h, sh.grid_w), tab, tabf, sh.scale)
    for b in range(3):                                  # block 2 sees two committed blocks
        if b == 2:
            g = schedule.BlockStepGraph(m, b, steps)
            eager, eager_q8 = [], []
            for s in range(steps):
                q, k, v = (to_dev(synth.block_tensor(sh, 98, b, s, t)) for t in (synth.Q, synth.K, synth.V))
                g.q[s].copy_(q); g.k[s].copy_(k); g.v[s].copy_(v)
                m.stage_and_attend(q, k, v, b, m.q_roped, m.out)
                eager.append(m.out.clone())
                eager_q8.append(m.q_roped.clone())
            for o in g.out:
                o.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert api.sdvg_block_attn_status(m.workspace) == api.SDVG_OK
            for s in range(steps):
                assert torch.equal(g.q_roped[s], eager_q8[s]), s
                assert torch.equal(g.out[s].view(torch.int16), eager[s].view(torch.int16)), s
        k, v = (to_dev(synth.block_tensor(sh, 98, b, 9, t)) for t in (synth.K, synth.V))
        m.commit_final(k, v, b)
    cache.close()
