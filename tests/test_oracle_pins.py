"""Pins of the CPU oracle against things other than itself (CPU only)."""
import math

import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import synth
from conftest import read_golden_rows


# ------------------------------------------------------------------ bf16 packing

def test_bf16_pack_matches_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, np.inf, -np.inf],
                                 dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f32_to_bf16(x), want)
    finite = np.isfinite(x)
    assert np.array_equal(synth.f32_to_bf16_bits(x[finite]), want[finite])
    back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.bf16_to_f64(want), back)


def test_bf16_nan_stays_nan():
    b = O.f32_to_bf16(np.array([np.nan], dtype=np.float32))
    assert np.isnan(O.bf16_to_f64(b))[0]


# ------------------------------------------------------------------ RoPE

def test_rope_axis_split():
    assert O.rope_axis_pairs(128) == (22, 21, 21)
    assert O.rope_axis_pairs(64) == (12, 10, 10)
    for d in (64, 128):
        assert sum(O.rope_axis_pairs(d)) == d // 2


def test_token_positions_frame_major():
    pos = O.token_positions(2 * 4 * 8, (2, 4, 8), 6)
    assert pos[0].tolist() == [6, 0, 0]
    assert pos[7].tolist() == [6, 0, 7]
    assert pos[8].tolist() == [6, 1, 0]
    assert pos[32].tolist() == [7, 0, 0]
    assert pos[63].tolist() == [7, 3, 7]


def test_rope_hand_worked_single_rotation():
    # token at frame 1, row 0, column 0; frame-axis pair 0 has omega = 1 -> turns by 1 rad.
    D = 64
    x = np.zeros((1, 1, D), dtype=np.float32)
    x[0, 0, 0] = 1.0                      # pair 0 = (1, 0)
    x[0, 0, 3] = 2.0                      # pair 1 = (0, 2)
    bits = O.f32_to_bf16(x)
    out = O.rope_ref(bits, (1, 1, 1), frame_offset=1)
    assert out[0, 0, 0] == pytest.approx(0.5403023058681398, abs=1e-15)   # cos 1
    assert out[0, 0, 1] == pytest.approx(0.8414709848078965, abs=1e-15)   # sin 1
    w1 = math.exp(-math.log(10000.0) / 12.0)      # pair 1 of 12 frame pairs
    assert out[0, 0, 2] == pytest.approx(-2.0 * math.sin(w1), abs=1e-15)
    assert out[0, 0, 3] == pytest.approx(2.0 * math.cos(w1), abs=1e-15)
    assert np.all(out[0, 0, 4:] == 0)


def test_rope_last_frame_pair_frequency():
    # D=128: pair 21 of the 22 frame pairs has omega = 10000^(-21/22)
    pos = np.array([[1, 0, 0]])
    a = O.rope_angles(128, pos)
    assert a.shape == (1, 64)
    assert a[0, 21] == pytest.approx(math.exp(-21.0 / 22.0 * math.log(10000.0)), rel=1e-13)
    assert a[0, 0] == 1.0
    assert np.all(a[0, 22:] == 0.0)          # row 0, column 0: other axes do not turn


def test_rope_axes_own_disjoint_pairs():
    sh = synth.TINY
    x = synth.block_tensor(sh, 3, 0, 0, synth.K)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    base = O.rope_ref(x, grid, 0)
    shifted = O.rope_ref(x, grid, 5)          # only the frame position moves
    pf, ph, pw = O.rope_axis_pairs(sh.head_dim)
    assert not np.allclose(base[..., :2 * pf], shifted[..., :2 * pf])
    assert np.array_equal(base[..., 2 * pf:], shifted[..., 2 * pf:])
    # tokens in the same row/frame but different column differ only in the width pairs' angles
    a = O.rope_angles(sh.head_dim, O.token_positions(sh.block_tokens, grid, 0))
    assert np.array_equal(a[0, :pf + ph], a[5, :pf + ph])
    assert not np.array_equal(a[0, pf + ph:], a[5, pf + ph:])


def test_rope_identity_at_origin_and_norms():
    sh = synth.TINY
    x = synth.block_tensor(sh, 4, 0, 0, synth.Q)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    out = O.rope_ref(x, grid, 0)
    xf = O.bf16_to_f64(x)
    assert np.array_equal(out[0], xf[0])                      # token (0,0,0): all angles 0
    n_in = xf[..., 0::2] ** 2 + xf[..., 1::2] ** 2
    n_out = out[..., 0::2] ** 2 + out[..., 1::2] ** 2
    assert np.allclose(n_in, n_out, rtol=1e-14, atol=1e-300)


def test_rope_equals_complex_multiplication():
    sh = synth.TINY
    x = synth.block_tensor(sh, 5, 1, 0, synth.K)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    out = O.rope_ref(x, grid, 2)
    xf = O.bf16_to_f64(x)
    z = xf[..., 0::2] + 1j * xf[..., 1::2]
    a = O.rope_angles(sh.head_dim, O.token_positions(sh.block_tokens, grid, 2))
    w = z * np.exp(1j * a)[:, None, :]
    assert np.allclose(out[..., 0::2], w.real, rtol=0, atol=1e-14)
    assert np.allclose(out[..., 1::2], w.imag, rtol=0, atol=1e-14)


def test_rope_relative_position_invariance():
    # <rope(q, P), rope(k, P')> depends on P - P' only: shifting every frame index leaves logits alone
    sh = synth.TINY
    q = synth.block_tensor(sh, 6, 0, 0, synth.Q)
    k = synth.block_tensor(sh, 6, 0, 0, synth.K)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    l0 = np.einsum("ihd,jhd->hij", O.rope_ref(q, grid, 4), O.rope_ref(k, grid, 0))
    l1 = np.einsum("ihd,jhd->hij", O.rope_ref(q, grid, 11), O.rope_ref(k, grid, 7))
    assert np.allclose(l0, l1, rtol=0, atol=1e-10)
    l2 = np.einsum("ihd,jhd->hij", O.rope_ref(q, grid, 5), O.rope_ref(k, grid, 0))
    assert not np.allclose(l0, l2, atol=1e-3)


def test_rope_bitspec_close_to_ref_and_table_layout():
    for sh, tabf in ((synth.TINY, 8), (synth.Shape("d128", 2, 128, 2, 3, 5, 3), 9)):
        x = synth.block_tensor(sh, 7, 2, 0, synth.K)
        grid = (sh.frames, sh.grid_h, sh.grid_w)
        tab = O.rope_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w)
        pf, ph, pw = O.rope_axis_pairs(sh.head_dim)
        assert tab.size == 2 * (tabf * pf + sh.grid_h * ph + sh.grid_w * pw)
        assert tab[0] == 1.0 and tab[1] == 0.0                        # frame 0, pair 0
        assert tab[2 * pf] == np.float32(math.cos(1.0))               # frame 1, pair 0
        assert tab[2 * pf + 1] == np.float32(math.sin(1.0))
        got = O.rope_bitspec(x, grid, 3, tab, tabf)
        ref = O.rope_ref(x, grid, 3)
        # within one bf16 ulp of the fp64 rotation (relative 2^-8 of the pair's magnitude)
        gotf = O.bf16_to_f64(got)
        mag = np.sqrt(ref[..., 0::2] ** 2 + ref[..., 1::2] ** 2)
        mag = np.repeat(mag, 2, axis=-1)
        assert np.all(np.abs(gotf - ref) <= mag * 2.0 ** -8 + 1e-30)
        # v-like passthrough: a zero-angle token is copied bit for bit
        got0 = O.rope_bitspec(x, grid, 0, tab, tabf)
        assert np.array_equal(got0[0], x[0])


def test_rope_bitspec_is_plain_fp32_ops():
    # scalar re-evaluation of a few elements with Python floats rounded step by step
    sh = synth.TINY
    x = synth.block_tensor(sh, 8, 0, 0, synth.Q)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tab = O.rope_table(sh.head_dim, 4, sh.grid_h, sh.grid_w)
    got = O.rope_bitspec(x, grid, 1, tab, 4)
    pf, ph, pw = O.rope_axis_pairs(sh.head_dim)
    f32 = np.float32
    for (t, h, p) in [(0, 0, 0), (13, 1, 3), (40, 0, 11), (63, 1, 12), (27, 0, 25), (50, 1, 31)]:
        fr, y, xx = O.token_positions(sh.block_tokens, grid, 1)[t]
        if p < pf:
            base = (fr * pf + p) * 2
        elif p < pf + ph:
            base = (4 * pf + y * ph + (p - pf)) * 2
        else:
            base = (4 * pf + sh.grid_h * ph + xx * pw + (p - pf - ph)) * 2
        c, s = f32(tab[base]), f32(tab[base + 1])
        re = f32(O.bf16_to_f64(x[t, h, 2 * p]))
        im = f32(O.bf16_to_f64(x[t, h, 2 * p + 1]))
        r0 = f32(f32(re * c) - f32(im * s))
        r1 = f32(f32(re * s) + f32(im * c))
        want = O.f32_to_bf16(np.array([r0, r1], dtype=np.float32))
        assert got[t, h, 2 * p] == want[0] and got[t, h, 2 * p + 1] == want[1]


# ------------------------------------------------------------------ attention

def _tiny_blocks(seed=0, nblocks=3):
    sh = synth.TINY
    q = [synth.block_tensor(sh, seed, b, 0, synth.Q) for b in range(nblocks)]
    k = [synth.block_tensor(sh, seed, b, 0, synth.K) for b in range(nblocks)]
    v = [synth.block_tensor(sh, seed, b, 0, synth.V) for b in range(nblocks)]
    return sh, q, k, v


def test_attention_matches_dense_mask_bruteforce():
    sh, q, k, v = _tiny_blocks(nblocks=5)
    slots = 3
    o_bf, P, mask = O.dense_bruteforce(q, k, v, sh.scale, slots)
    T = sh.block_tokens
    # the mask is block-causal with a window of slots-1 earlier blocks
    blk = np.repeat(np.arange(5), T)
    for i in (0, T, 2 * T + 5, 4 * T + 63):
        vis = sorted(set(blk[mask[i]]))
        b = blk[i]
        assert vis == list(range(max(0, b - 2), b + 1))
    assert np.allclose(P.sum(axis=2), 1.0, atol=1e-14)
    assert np.all(P[:, ~mask] == 0.0)
    cache = O.RingCacheRef(slots, sh.heads, T, sh.head_dim)
    for b in range(5):
        o, lse = O.block_attn_ref(q[b], k[b], v[b], cache, b, sh.scale)
        assert np.allclose(o, o_bf[b * T:(b + 1) * T], rtol=0, atol=1e-12)
        cache.commit(b, k[b], v[b], O.FINAL)


def test_attention_matches_library_sdpa_fp64():
    sh, q, k, v = _tiny_blocks(seed=2)
    kk = np.concatenate(k, axis=0)
    vv = np.concatenate(v, axis=0)
    o, lse = O.attn_ref(q[2], kk, vv, sh.scale)
    tq = torch.from_numpy(O.bf16_to_f64(q[2])).permute(1, 0, 2)[None]
    tk = torch.from_numpy(O.bf16_to_f64(kk)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(O.bf16_to_f64(vv)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=sh.scale)[0].permute(1, 0, 2).numpy()
    assert np.allclose(o, ref, rtol=0, atol=1e-12)
    logits = torch.einsum("hid,hjd->hij", tq[0], tk[0]) * sh.scale
    assert np.allclose(lse, torch.logsumexp(logits, dim=-1).numpy(), rtol=0, atol=1e-12)


def test_attention_closed_forms():
    sh, q, k, v = _tiny_blocks(seed=3)
    kk, vv = np.concatenate(k[:2]), np.concatenate(v[:2])
    zero_q = np.zeros_like(q[0])
    o, lse = O.attn_ref(zero_q, kk, vv, sh.scale)
    mean_v = O.bf16_to_f64(vv).mean(axis=0)
    assert np.allclose(o, mean_v[None], atol=1e-14)
    assert np.allclose(lse, math.log(kk.shape[0]), atol=1e-14)
    # one visible key: the output is that key's value
    o1, _ = O.attn_ref(q[0], kk[:1], vv[:1], sh.scale)
    assert np.allclose(o1, O.bf16_to_f64(vv[:1]), atol=1e-15)
    # doubling q and halving the scale is exact in bf16/fp64 and changes nothing
    q2 = O.f32_to_bf16(O.bf16_to_f32(q[0]) * np.float32(2))
    oa, la = O.attn_ref(q[0], kk, vv, sh.scale)
    ob, lb = O.attn_ref(q2, kk, vv, sh.scale / 2)
    assert np.array_equal(oa, ob) and np.array_equal(la, lb)
    # a transposed operand or a dropped scale would break this one-hot case:
    D = sh.head_dim
    kq = np.zeros((2, 1, D), dtype=np.float32)
    kq[0, 0, 0] = 8.0
    kq[1, 0, 1] = 8.0
    vq = np.zeros((2, 1, D), dtype=np.float32)
    vq[0, 0, 5] = 1.0
    vq[1, 0, 6] = 1.0
    qq = np.zeros((1, 1, D), dtype=np.float32)
    qq[0, 0, 0] = 1.0
    o, lse = O.attn_ref(O.f32_to_bf16(qq), O.f32_to_bf16(kq), O.f32_to_bf16(vq), 0.125)
    p0 = math.e / (math.e + 1.0)                       # logits (1, 0)
    assert o[0, 0, 5] == pytest.approx(p0, abs=1e-15)
    assert o[0, 0, 6] == pytest.approx(1 - p0, abs=1e-15)
    assert lse[0, 0] == pytest.approx(math.log(math.e + 1.0), abs=1e-15)


def test_attention_subset_rows_heads():
    sh, q, k, v = _tiny_blocks(seed=4)
    kk, vv = np.concatenate(k), np.concatenate(v)
    o, lse = O.attn_ref(q[1], kk, vv, sh.scale)
    rows = np.array([3, 17, 60])
    os_, ls_ = O.attn_ref(q[1], kk, vv, sh.scale, heads=[1], rows=rows)
    assert np.array_equal(os_[:, 0], o[rows, 1])
    assert np.array_equal(ls_[0], lse[1, rows])


def test_mask_by_perturbation_and_slot_rotation():
    sh, q, k, v = _tiny_blocks(seed=5, nblocks=6)
    T = sh.block_tokens

    def run(perturbed_block=None):
        cache = O.RingCacheRef(3, sh.heads, T, sh.head_dim)
        outs = []
        for b in range(6):
            outs.append(O.block_attn_ref(q[b], k[b], v[b], cache, b, sh.scale)[0])
            kk = k[b]
            if b == perturbed_block:
                kk = kk.copy()
                kk[0, 0, 0] ^= 0x8000          # flip a sign in the committed copy of this block
            cache.commit(b, kk, v[b], O.FINAL)
        return outs

    base = run()
    pert = run(perturbed_block=1)
    # block 1 is visible to blocks 2 and 3 only (window of 2 earlier blocks)
    assert np.array_equal(base[0], pert[0]) and np.array_equal(base[1], pert[1])
    assert not np.array_equal(base[2], pert[2]) and not np.array_equal(base[3], pert[3])
    assert np.array_equal(base[4], pert[4]) and np.array_equal(base[5], pert[5])
    # key order does not matter: blocks 4 sees {2,3} stored in slots {2,0}
    kk = np.concatenate([k[3], k[2], k[4]])
    vv = np.concatenate([v[3], v[2], v[4]])
    o_rot, _ = O.attn_ref(q[4], kk, vv, sh.scale)
    assert np.allclose(o_rot, base[4], atol=1e-13)


# ------------------------------------------------------------------ ring cache

def test_ring_hand_worked_trace():
    rows = read_golden_rows("ring_cases.txt")
    cache = O.RingCacheRef(3, 1, 4, 2)
    for blk, slot, evicted, visible in rows:
        b = int(blk)
        assert cache.slot_of(b) == int(slot)
        assert O.visible_blocks(b, 3) == [int(x) for x in visible.split()]
        kb = np.full((4, 1, 2), 100 + b, dtype=np.uint16)
        vb = np.full((4, 1, 2), 200 + b, dtype=np.uint16)
        kw, vw = cache.window(b)
        want = [100 + int(x) for x in visible.split()]
        assert [int(kw[i * 4, 0, 0]) for i in range(len(want))] == want
        assert cache.commit(b, kb, vb, O.FINAL) == int(evicted)
        assert cache.next_block == b + 1
    assert cache.slot_block == [3, 4, 2]


def test_ring_stage_does_not_advance_and_order_is_enforced():
    cache = O.RingCacheRef(2, 1, 2, 2)
    k0 = np.ones((2, 1, 2), dtype=np.uint16)
    assert cache.commit(0, k0, k0, O.STAGE) == -1
    assert cache.next_block == 0 and cache.slot_block == [-1, -1]
    assert np.array_equal(cache.k[0], k0)
    with pytest.raises(RuntimeError):
        cache.commit(1, k0, k0, O.FINAL)
    assert cache.commit(0, k0 * 7, k0, O.FINAL) == -1
    assert np.array_equal(cache.k[0], k0 * 7)
    with pytest.raises(RuntimeError):
        cache.commit(0, k0, k0, O.FINAL)
    with pytest.raises(ValueError):
        cache.commit(1, np.ones((3, 1, 2), dtype=np.uint16), k0, O.FINAL)


# ------------------------------------------------------------------ router

def _parse_scores(txt):
    return np.array([float(t) for t in txt.split()], dtype=np.float32)


def test_route_hand_worked_cases():
    for blk, tau, scores, accept, qmin, argmin in read_golden_rows("route_cases.txt"):
        s = _parse_scores(scores)
        a, q, i = O.route_ref(s, None, 1, s.size, int(blk), float(tau))
        assert int(a[0]) == int(accept), (blk, tau, scores)
        want = np.float32(float(qmin))
        assert (np.isnan(want) and np.isnan(q[0])) or q[0] == want
        assert int(i[0]) == int(argmin)


def test_route_ragged_and_streaming_offsets():
    flat, offs = synth.ragged_scores([9, 12, 12, 3, 1], -0.5, 0.6, 11)
    a, q, i = O.route_ref(flat, offs, 5, 0, 0, -0.7)
    for b in range(5):
        seg = flat[offs[b]:offs[b + 1]]
        assert q[b] == seg.min() and i[b] == int(np.argmin(seg))
        assert a[b] == (1 if (b != 0 and seg.min() >= np.float32(-0.7)) else 0)
    # the same scores seen as blocks 3..7 of a stream: block "0" of the batch is no longer forced
    a2, _, _ = O.route_ref(flat, offs, 5, 0, 3, -5.0)
    assert a2.tolist() == [1, 1, 1, 1, 1]
    a3, _, _ = O.route_ref(flat, offs, 5, 0, 0, -5.0)
    assert a3.tolist() == [0, 1, 1, 1, 1]
    with pytest.raises(ValueError):
        O.route_ref(flat, None, 2, 0, 0, -0.7)                 # a fixed frame count below one


def test_route_malformed_ragged_input_hand_worked():
    # blocks without frames, offsets that run backwards or leave [offsets[0], offsets[B]]: rejected, NaN, -1
    for offsets, scores, tau, accept, qmin, argmin in read_golden_rows("route_malformed_cases.txt"):
        offs = np.array([int(t) for t in offsets.split()], dtype=np.int32)
        s = np.array([float(t) for t in scores.split()], dtype=np.float32)
        a, q, i = O.route_ref(s, offs, offs.size - 1, 0, 1, float(tau))
        want_q = np.array([float(t) for t in qmin.split()], dtype=np.float32)
        assert a.tolist() == [int(t) for t in accept.split()]
        assert i.tolist() == [int(t) for t in argmin.split()]
        assert np.array_equal(np.isnan(q), np.isnan(want_q))
        assert np.array_equal(q[~np.isnan(want_q)], want_q[~np.isnan(want_q)])


def test_route_degenerate_policies_and_accept_rate_convention():
    s = synth.normal_scores(9, 12, -0.5, 0.6, 5)
    a_all, _, _ = O.route_ref(s.reshape(-1), None, 9, 12, 0, -np.inf)     # draft-only except block 0
    a_none, _, _ = O.route_ref(s.reshape(-1), None, 9, 12, 0, np.inf)     # target-only
    assert a_all.tolist() == [0] + [1] * 8 and a_none.sum() == 0
    assert O.accept_rate(a_all) == 1.0          # block 0 is left out of the rate
    assert O.accept_rate(np.array([0, 1, 0, 1, 1, 0, 1, 1, 1])) == pytest.approx(6 / 8)


def test_calibrated_scores_follow_table1_accept_rates():
    s = synth.calibrated_scores(40001, 12, 9)
    for tau, _, rate in read_golden_rows("table1.txt"):
        a, _, _ = O.route_ref(s.reshape(-1), None, s.shape[0], 12, 0, float(tau))
        assert O.accept_rate(a) == pytest.approx(float(rate), abs=0.01)


def _policy_row(row):
    blk, bpv, tau, agg, sig, force, u, p, scores, accept, aggv = row
    s = np.array([float(t) for t in scores.split()], dtype=np.float32)
    kw = dict(agg=O.AGG_MEAN if agg == "mean" else O.AGG_MIN,
              signal=O.SIGNAL_RANDOM if sig == "random" else O.SIGNAL_REWARD, force_first=bool(int(force)),
              blocks_per_video=int(bpv), uniforms=np.array([float(u)], dtype=np.float32), accept_prob=float(p))
    return s, int(blk), float(tau), kw, int(accept), np.float32(float(aggv))


def test_route_policy_hand_worked_cases():
    for row in read_golden_rows("route_policy_cases.txt"):
        s, blk, tau, kw, accept, aggv = _policy_row(row)
        a, v, _ = O.route_policy_ref(s, None, 1, s.size, blk, tau, **kw)
        assert int(a[0]) == accept, row
        assert (np.isnan(aggv) and np.isnan(v[0])) or v[0] == aggv, row


def test_route_policy_reduces_to_the_default_router():
    s = synth.normal_scores(40, 12, -0.5, 0.6, 8)
    for first in (0, 3):
        a, q, i = O.route_ref(s.reshape(-1), None, 40, 12, first, -0.7)
        a2, q2, i2 = O.route_policy_ref(s.reshape(-1), None, 40, 12, first, -0.7)
        assert np.array_equal(a, a2) and np.array_equal(q.view(np.uint32), q2.view(np.uint32)) and np.array_equal(i, i2)


def test_route_policy_mean_against_float64_and_bounds():
    # the fp32 left-to-right mean stays within a few ulp of the exact mean and between min and max
    s = synth.normal_scores(500, 12, -0.5, 0.6, 9)
    _, v, _ = O.route_policy_ref(s.reshape(-1), None, 500, 12, 1, -0.7, agg=O.AGG_MEAN)
    exact = s.astype(np.float64).mean(axis=1)
    assert np.abs(v - exact).max() <= 12 * 2.0 ** -23 * np.abs(s).max()
    assert np.all(v >= s.min(axis=1) - 1e-6) and np.all(v <= s.max(axis=1) + 1e-6)
    # a block of equal frames has exactly that value as its mean, and min == mean
    c = np.full((3, 8), -0.625, dtype=np.float32)
    _, vm, _ = O.route_policy_ref(c.reshape(-1), None, 3, 8, 1, -0.7, agg=O.AGG_MEAN)
    assert np.all(vm == np.float32(-0.625))
    # mean >= min always, so at one tau the mean policy accepts a superset of the min policy (Table 2: higher accept rate)
    a_min, _, _ = O.route_policy_ref(s.reshape(-1), None, 500, 12, 1, -0.7, agg=O.AGG_MIN)
    a_mean, _, _ = O.route_policy_ref(s.reshape(-1), None, 500, 12, 1, -0.7, agg=O.AGG_MEAN)
    assert np.all(a_mean >= a_min)


def test_route_policy_random_signal_and_accept_stats():
    B, V = 9 * 400, 400
    s = synth.normal_scores(B, 12, -0.5, 0.6, 10)
    u = synth.uniform_scores(B, 1, 0.0, 1.0, 11).reshape(-1)
    forced, _, _ = O.route_policy_ref(s.reshape(-1), None, B, 12, 0, -0.7, signal=O.SIGNAL_RANDOM, force_first=True,
                                      blocks_per_video=9, uniforms=u, accept_prob=0.7)
    plain, _, _ = O.route_policy_ref(s.reshape(-1), None, B, 12, 0, -0.7, signal=O.SIGNAL_RANDOM, force_first=False,
                                     blocks_per_video=9, uniforms=u, accept_prob=0.7)
    assert forced.reshape(V, 9)[:, 0].sum() == 0                      # every video's block 0 regenerated
    assert np.array_equal(forced.reshape(V, 9)[:, 1:], plain.reshape(V, 9)[:, 1:])
    assert np.array_equal(plain, (u < np.float32(0.7)).astype(np.uint8))   # the scores play no part
    acc, routable = O.accept_stats_ref(forced, 0, 9)
    assert routable == 8 * V and acc == int(forced.sum())
    assert acc / routable == pytest.approx(0.7, abs=0.03)             # matched accept rate (Table 2: 70.3% / 70.0%)
    # the statistic leaves block 0 out even when it was accepted
    acc2, routable2 = O.accept_stats_ref(plain, 0, 9)
    assert routable2 == routable and acc2 == int(plain.reshape(V, 9)[:, 1:].sum())
    # degenerate probabilities
    none, _, _ = O.route_policy_ref(s.reshape(-1), None, B, 12, 0, 0.0, signal=O.SIGNAL_RANDOM, uniforms=u, accept_prob=0.0)
    every, _, _ = O.route_policy_ref(s.reshape(-1), None, B, 12, 0, 0.0, signal=O.SIGNAL_RANDOM, force_first=False,
                                     uniforms=u, accept_prob=1.0)
    assert none.sum() == 0 and every.sum() == B
    # one stream (blocks_per_video = 0): only global block 0 is a first block
    a1, r1 = O.accept_stats_ref(np.ones(10, dtype=np.uint8), 0, 0)
    a2, r2 = O.accept_stats_ref(np.ones(10, dtype=np.uint8), 5, 0)
    assert (a1, r1) == (9, 9) and (a2, r2) == (10, 10)
    assert O.accept_rate(np.array([1, 1, 0, 1])) == pytest.approx(2 / 3)   # agrees with the older helper


# ------------------------------------------------------------------ schedule

def _tiny_provider(sh_d, sh_t, seed):
    def provider(model, b, kind, step):
        sh = sh_d if model == "drafter" else sh_t
        if kind == "step":
            src = (synth.SRC_DRAFT_STEP if model == "drafter" else synth.SRC_TARGET_STEP) + step
            return tuple(synth.block_tensor(sh, seed, b, src, t) for t in (synth.Q, synth.K, synth.V))
        src = {"clean": synth.SRC_DRAFT_CLEAN if model == "drafter" else synth.SRC_TARGET_CLEAN,
               "accepted": synth.SRC_ACCEPT_CLEAN}[kind]
        return None, synth.block_tensor(sh, seed, b, src, synth.K), synth.block_tensor(sh, seed, b, src, synth.V)
    return provider


def _run_tiny_trace(scores, tau, B=9, S=4, seed=21):
    sh_d = synth.Shape("d", 1, 64, 1, 2, 4, 3)
    sh_t = synth.Shape("t", 2, 64, 1, 2, 4, 7)
    drafter = O.RingCacheRef(sh_d.slots, sh_d.heads, sh_d.block_tokens, sh_d.head_dim)
    target = O.RingCacheRef(sh_t.slots, sh_t.heads, sh_t.block_tokens, sh_t.head_dim)
    tab = O.rope_table(64, B, 2, 4)
    res = O.schedule_ref(B, S, scores, tau, drafter, target, _tiny_provider(sh_d, sh_t, seed),
                         (1, 2, 4), (1, 2, 4), 1, tab, tab, B)
    return res, drafter, target, sh_d, sh_t, tab


def test_schedule_call_counts_reproduce_table1_times():
    # cost identity implied by Table 1: time = T_draft + (1 + (B-1)(1-a)) * T_target / B
    B, S = 9, 4
    t_draft, t_target = 25.7, 97.0
    for tau, secs, rate in read_golden_rows("table1.txt"):
        n_acc = round(float(rate) * (B - 1))
        scores = np.full((B, 12), -5.0, dtype=np.float32)
        scores[1:1 + n_acc] = 1.0
        res, *_ = _run_tiny_trace(scores, -0.7, B, S)
        assert res.drafter_attn_calls == S * B
        n_rej = (B - 1) - n_acc
        assert res.target_attn_calls == S * (1 + n_rej)
        # per-video time predicted from the call counts at the paper's exact (fractional) accept rate
        frac_calls = S * (1 + (B - 1) * (1 - float(rate)))
        pred = t_draft * res.drafter_attn_calls / (S * B) + t_target * frac_calls / (S * B)
        assert 0.0 <= float(secs) - pred <= 2.0, (tau, pred, secs)


def test_schedule_final_caches_hold_the_right_source():
    B = 9
    scores = np.full((B, 12), 1.0, dtype=np.float32)
    scores[3, 4] = -2.0            # block 3 rejected by one bad frame
    scores[6, 0] = -0.71           # block 6 rejected
    res, drafter, target, sh_d, sh_t, tab = _run_tiny_trace(scores, -0.7, B)
    assert res.accept.tolist() == [0, 1, 1, 0, 1, 1, 0, 1, 1]
    assert res.target_source == ["regenerated", "accepted", "accepted", "regenerated", "accepted",
                                 "accepted", "regenerated", "accepted", "accepted"]
    assert res.drafter_evicted == [-1, -1, -1, 0, 1, 2, 3, 4, 5]
    assert res.target_evicted == [-1] * 7 + [0, 1]
    assert drafter.slot_block == [6, 7, 8] and target.slot_block == [7, 8, 2, 3, 4, 5, 6]
    prov = _tiny_provider(sh_d, sh_t, 21)
    for b in range(2, 9):
        kind = "accepted" if res.accept[b] else "clean"
        _, k, v = prov("target", b, kind, 0)
        kr = O.rope_bitspec(k, (1, 2, 4), b, tab, B)
        assert np.array_equal(target.k[b % 7], kr) and np.array_equal(target.v[b % 7], v)
        other = prov("target", b, "clean" if res.accept[b] else "accepted", 0)[2]
        assert not np.array_equal(target.v[b % 7], other)
    for b in range(6, 9):
        _, k, v = prov("drafter", b, "clean", 0)
        assert np.array_equal(drafter.v[b % 3], v)
