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
