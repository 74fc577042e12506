"""Pins of the oracle's 8-bit (E4M3) functions against the format's definition, torch's own CPU cast and
the bf16 attention oracle (itself pinned elsewhere)."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from conftest import read_golden_rows


def test_decode_matches_format_table_and_is_monotone():
    for code, value in read_golden_rows("e4m3_format_values.txt"):
        assert O.e4m3_decode(np.array([int(code, 16)], dtype=np.uint8))[0] == float(value)
    pos = O.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0) and pos[0] == 0.0 and pos[-1] == 448.0
    assert np.isnan(O.e4m3_decode(np.array([0x7F, 0xFF], dtype=np.uint8))).all()
    # mirror image for the sign bit, and agreement with torch's decoder for all 256 codes
    assert np.array_equal(O.e4m3_decode(np.arange(0x80, 0xFF, dtype=np.uint8)), -pos)
    t = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.nan_to_num(t, nan=-7.0), np.nan_to_num(O.e4m3_decode(np.arange(256, dtype=np.uint8)), nan=-7.0))


def test_encode_roundtrip_ties_saturation():
    codes = np.concatenate([np.arange(0x7F), np.arange(0x80, 0xFF)]).astype(np.uint8)
    assert np.array_equal(O.e4m3_encode(O.e4m3_decode(codes)), codes)          # every finite code is a fixed point
    # halfway cases go to the even code; just off halfway goes to the nearer one
    assert O.e4m3_encode(np.array([1.0625]))[0] == 0x38      # between 1.0 (0x38) and 1.125 (0x39)
    assert O.e4m3_encode(np.array([1.1875]))[0] == 0x3A      # between 1.125 (0x39) and 1.25 (0x3A)
    assert O.e4m3_encode(np.array([1.0625 + 1e-9]))[0] == 0x39
    assert O.e4m3_encode(np.array([2.0 ** -10]))[0] == 0x00  # halfway between 0 and the smallest subnormal
    assert O.e4m3_encode(np.array([2.0 ** -10 * 1.001]))[0] == 0x01
    assert O.e4m3_encode(np.array([1.9375]))[0] == 0x40      # halfway between 1.875 (0x3F) and 2.0 (0x40): carries into the exponent
    # saturation instead of NaN / infinity; the sign survives, also on zero
    assert list(O.e4m3_encode(np.array([448.0, 464.0, 1e9, np.inf, -465.0, -np.inf]))) == [0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE]
    assert list(O.e4m3_encode(np.array([0.0, -0.0, np.nan]))) == [0x00, 0x80, 0x7F]


def test_encode_matches_torch_cast_for_every_bf16_value_in_range():
    bits = np.arange(65536, dtype=np.uint16)
    x = O.bf16_to_f64(bits)
    keep = np.isfinite(x) & (np.abs(x) < 464.0)              # torch's cast turns what rounds beyond 448 into NaN
    ours = O.e4m3_encode(x[keep])
    theirs = torch.from_numpy(x[keep]).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, theirs)


def test_quant_is_one_fp32_multiply_then_one_rounding():
    rng = np.random.default_rng(5)
    x = O.f32_to_bf16(rng.standard_normal((33, 3, 16)).astype(np.float32) * 3)
    inv = np.array([1.0, 37.3, 0.013], dtype=np.float32)
    got = O.quant_e4m3_ref(x, inv)
    y = (torch.from_numpy(O.bf16_to_f32(x)) * torch.from_numpy(inv).view(1, 3, 1))          # fp32 product
    want = y.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, want)
    assert got.dtype == np.uint8 and got.shape == x.shape
    # scale 1 on values that E4M3 holds exactly is lossless
    exact = O.f32_to_bf16(np.array([[[0.5, -1.75, 448.0, 2.0 ** -9]]], dtype=np.float32))
    assert np.array_equal(O.e4m3_decode(O.quant_e4m3_ref(exact, np.ones(1, np.float32))), O.bf16_to_f64(exact))


def test_attention_e4m3_reduces_to_the_bf16_oracle_on_shared_values():
    # integers in [-8, 8] and halves are exact in both formats: the two oracles must then agree to rounding order
    rng = np.random.default_rng(9)
    T, L, H, D = 17, 45, 3, 16
    qv = rng.integers(-4, 5, (T, H, D)) / 2.0
    kv = rng.integers(-4, 5, (L, H, D)) / 2.0
    vv = rng.integers(-8, 9, (L, H, D)).astype(np.float64)
    q8, k8, v8 = O.e4m3_encode(qv), O.e4m3_encode(kv), O.e4m3_encode(vv)
    assert np.array_equal(O.e4m3_decode(q8), qv)
    ones = np.ones(H)
    o8, lse8 = O.attn_e4m3_ref(q8, k8, v8, ones, ones, 0.21)
    o16, lse16 = O.attn_ref(O.f64_to_bf16(qv), O.f64_to_bf16(kv), O.f64_to_bf16(vv), 0.21)
    np.testing.assert_allclose(o8, o16, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse8, lse16, rtol=0, atol=1e-12)
    # descales: the logit scale can move between `scale` and qk_descale; v_descale is a plain factor per head
    qd = np.array([0.5, 2.0, 1.25])
    vd = np.array([3.0, 0.25, 1.0])
    o_a, lse_a = O.attn_e4m3_ref(q8, k8, v8, qd, vd, 0.21)
    for h in range(H):
        o_h, lse_h = O.attn_e4m3_ref(q8, k8, v8, ones, ones, 0.21 * qd[h], heads=[h])
        np.testing.assert_allclose(o_a[:, h], o_h[:, 0] * vd[h], rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(lse_a[h], lse_h[0], rtol=1e-13, atol=1e-13)
    # one key only: the output is that key's dequantised value, whatever the logits
    o1, _ = O.attn_e4m3_ref(q8, k8[:1], v8[:1], qd, vd, 0.21)
    np.testing.assert_allclose(o1, np.broadcast_to(O.e4m3_decode(v8[:1]) * vd[None, :, None], o1.shape), atol=1e-13)


def test_block_attention_e4m3_sees_the_same_window_as_the_bf16_ring():
    rng = np.random.default_rng(2)
    S, H, T, D = 3, 2, 5, 8
    ring = O.RingCacheRef(S, H, T, D, dtype=np.uint8)
    blocks = [(rng.integers(0, 0x7F, (T, H, D)).astype(np.uint8), rng.integers(0, 0x7F, (T, H, D)).astype(np.uint8))
              for _ in range(6)]
    for b in range(5):
        assert ring.commit(b, blocks[b][0], blocks[b][1], O.FINAL) == (b - S if b >= S else -1)
    q8 = rng.integers(0x20, 0x40, (T, H, D)).astype(np.uint8)
    ones = np.ones(H)
    o, _ = O.block_attn_e4m3_ref(q8, blocks[5][0], blocks[5][1], ring, 5, ones, ones, 0.05)
    k_all = np.concatenate([blocks[3][0], blocks[4][0], blocks[5][0]])
    v_all = np.concatenate([blocks[3][1], blocks[4][1], blocks[5][1]])
    o_direct, _ = O.attn_e4m3_ref(q8, k_all, v_all, ones, ones, 0.05)
    assert np.array_equal(o, o_direct)
    with pytest.raises(RuntimeError):
        O.block_attn_e4m3_ref(q8, blocks[5][0], blocks[5][1], ring, 4, ones, ones, 0.05)


# ---- one power-of-two scale per tile of 128 tokens and head ------------------------------------------------


def test_tile_scale_exponent_on_hand_values():
    # 448 = 0.875 * 2^9 is the largest E4M3 value: amax = 448 fits scale 1, the next bf16 value (450) needs 2
    cases = [(448.0, 0), (450.0, 1), (896.0, 1), (897.0, 2), (1.0, -8), (0.875, -9), (0.876, -8), (224.0, -1), (224.5, 0),
             (3.0, -7), (2.0 ** -140, -126), (0.0, -126), (448.0 * 2.0 ** 120, 120), (3.3e38, 120), (np.inf, 120)]
    for amax, e in cases:
        assert O.e4m3_tile_scale_exponent(amax) == e, amax
    # closed form away from the clamps: e = ceil(log2(amax / 448)), so amax / 2^e lies in (224, 448]
    rng = np.random.default_rng(0)
    for amax in np.exp(rng.uniform(-60, 60, 500)):
        e = O.e4m3_tile_scale_exponent(amax)
        assert 224.0 < amax / 2.0 ** e <= 448.0
        assert e == int(np.ceil(np.log2(amax / 448.0)))


def test_tiled_quantiser_against_torch_cast_and_tile_independence():
    rng = np.random.default_rng(6)
    T, H, D = 300, 3, 16                                  # three tiles, the last one of 44 tokens
    gain = np.exp(rng.uniform(-6, 6, (3, H)))             # every (tile, head) at its own magnitude
    x = rng.standard_normal((T, H, D)) * np.repeat(gain, 128, axis=0)[:T, :, None]
    xb = O.f32_to_bf16(x.astype(np.float32))
    codes, scales = O.quant_e4m3_tiled_ref(xb)
    assert codes.shape == (T, H, D) and codes.dtype == np.uint8 and scales.shape == (H, 3) and scales.dtype == np.float32
    xf = O.bf16_to_f64(xb)
    for h in range(H):
        for t in range(3):
            tile = xf[128 * t:128 * t + 128, h]
            sc = float(scales[h, t])
            assert sc == 2.0 ** round(np.log2(sc))                                        # a power of two
            assert 224.0 < np.abs(tile).max() / sc <= 448.0                               # the tile uses the top binade
            want = torch.from_numpy(tile / sc).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            assert np.array_equal(codes[128 * t:128 * t + 128, h], want)                  # torch's own cast of x / scale
    # dequantised values are within 2^-4 of the input (3 mantissa bits), down to the tile's subnormal step
    deq = O.e4m3_decode(codes) * O.e4m3_token_scales(scales, T)[:, :, None]
    step = O.e4m3_token_scales(scales, T)[:, :, None] * 2.0 ** -10
    assert np.all(np.abs(deq - xf) <= np.maximum(np.abs(xf) * 2.0 ** -4, step))
    # changing one tile changes only that tile's codes and scale
    xb2 = xb.copy()
    xb2[130:140, 1] = O.f32_to_bf16(np.full((10, D), 1e4, dtype=np.float32))
    codes2, scales2 = O.quant_e4m3_tiled_ref(xb2)
    same = np.ones((T, H), dtype=bool)
    same[128:256, 1] = False
    assert np.array_equal(codes2[same], codes[same])
    assert scales2[1, 1] == 32.0 and np.array_equal(np.delete(scales2.ravel(), 1 * 3 + 1), np.delete(scales.ravel(), 1 * 3 + 1))
    # with one magnitude everywhere it is the static quantiser at the same scale
    y = O.f32_to_bf16((rng.standard_normal((T, 1, D)) * 0.5).astype(np.float32))
    y[::128, 0, 0] = O.f32_to_bf16(np.array([3.0], dtype=np.float32))[0]          # every tile's largest magnitude: 3 -> 2^-7
    c3, s3 = O.quant_e4m3_tiled_ref(y)
    assert np.all(s3 == np.float32(2.0 ** -7))
    assert np.array_equal(c3, O.quant_e4m3_ref(y, np.array([2.0 ** 7], dtype=np.float32)))
    # special values: a NaN element does not set the scale and becomes the NaN code; an all-zero tile takes the smallest scale
    z = np.zeros((128, 1, D), dtype=np.uint16)
    cz, sz = O.quant_e4m3_tiled_ref(z)
    assert sz[0, 0] == np.float32(2.0 ** -126) and not cz.any()
    z[3, 0, 2] = 0x7FC0                                      # NaN
    z[5, 0, 1] = O.f32_to_bf16(np.array([1.0], dtype=np.float32))[0]
    cz, sz = O.quant_e4m3_tiled_ref(z)
    assert sz[0, 0] == np.float32(2.0 ** -8) and cz[3, 0, 2] == 0x7F and cz[5, 0, 1] == 0x78       # 256 = 1.0 * 2^8: code 0x78


def test_rowscaled_attention_reduces_to_its_neighbours():
    rng = np.random.default_rng(12)
    T, L, H, D = 9, 300, 2, 16
    q8 = rng.integers(0x28, 0x48, (T, H, D)).astype(np.uint8) | (rng.integers(0, 2, (T, H, D)) * 0x80).astype(np.uint8)
    k8 = rng.integers(0x28, 0x48, (L, H, D)).astype(np.uint8) | (rng.integers(0, 2, (L, H, D)) * 0x80).astype(np.uint8)
    v8 = rng.integers(0x10, 0x60, (L, H, D)).astype(np.uint8) | (rng.integers(0, 2, (L, H, D)) * 0x80).astype(np.uint8)
    # (a) constant scales per head: the static-scale oracle
    sq, sk, sv = np.array([0.5, 2.0]), np.array([0.25, 1.0]), np.array([4.0, 0.125])
    o_a, lse_a = O.attn_e4m3_rowscaled_ref(q8, np.tile(sq, (T, 1)), k8, np.tile(sk, (L, 1)), v8, np.tile(sv, (L, 1)), 0.3)
    o_b, lse_b = O.attn_e4m3_ref(q8, k8, v8, sq * sk, sv, 0.3)
    np.testing.assert_allclose(o_a, o_b, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse_a, lse_b, rtol=1e-12, atol=1e-12)
    # (b) power-of-two scales per tile: code * 2^e is a bf16 number, so the bf16 oracle on those numbers must agree
    qs = O.e4m3_token_scales(2.0 ** rng.integers(-3, 3, (H, 1)), T)
    ks = O.e4m3_token_scales(2.0 ** rng.integers(-3, 3, (H, 3)), L)
    vs = O.e4m3_token_scales(2.0 ** rng.integers(-5, 5, (H, 3)), L)
    o_c, lse_c = O.attn_e4m3_rowscaled_ref(q8, qs, k8, ks, v8, vs, 0.02)
    deq = lambda c, s: O.f64_to_bf16(O.e4m3_decode(c) * s[:, :, None])
    assert np.array_equal(O.bf16_to_f64(deq(k8, ks)), O.e4m3_decode(k8) * ks[:, :, None])          # exactly representable
    o_d, lse_d = O.attn_ref(deq(q8, qs), deq(k8, ks), deq(v8, vs), 0.02)
    np.testing.assert_allclose(o_c, o_d, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse_c, lse_d, rtol=1e-12, atol=1e-12)
    # (c) heads and rows select; a key tile with a vanishing V scale contributes its weight but no value
    o_e, _ = O.attn_e4m3_rowscaled_ref(q8, qs, k8, ks, v8, vs, 0.02, heads=[1], rows=[2, 7])
    np.testing.assert_array_equal(o_e[:, 0], o_c[[2, 7], 1])
    vs0 = vs.copy()
    vs0[:128] = 0.0
    o_f, lse_f = O.attn_e4m3_rowscaled_ref(q8, qs, k8, ks, v8, vs0, 0.02)
    np.testing.assert_allclose(lse_f, lse_c, rtol=0, atol=0)
    s = (O.e4m3_decode(q8[:, 0]) * qs[:, 0, None]) @ (O.e4m3_decode(k8[:, 0]) * ks[:, 0, None]).T * 0.02
    p = np.exp(s - s.max(1, keepdims=True))
    want = (p[:, 128:] @ (O.e4m3_decode(v8[128:, 0]) * vs[128:, 0, None])) / p.sum(1, keepdims=True)
    np.testing.assert_allclose(o_f[:, 0], want, rtol=1e-12, atol=1e-12)
