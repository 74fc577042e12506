"""sdvg_block_steps: the denoising steps of a block through ONE library call.

The call must give, bit for bit, what the separate fused-prologue and attention calls give, and both must be
the attention the oracle defines on the roped, staged block (Sec. 4.1 "Models": 4 steps per block).
"""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from gpu_utils import ATTN_MAX_ABS, ATTN_MEAN_ABS, to_bits, to_dev

pytestmark = pytest.mark.gpu

STEPS = 4


def _inputs(sh, seed, b):
    return [[synth.block_tensor(sh, seed, b, synth.SRC_DRAFT_STEP + s, t) for t in (synth.Q, synth.K, synth.V)]
            for s in range(STEPS)]


@pytest.mark.parametrize("shape", ["tiny", "ragged"])
def test_block_steps_equal_the_separate_calls_and_the_oracle(shape):
    sh = synth.TINY if shape == "tiny" else synth.Shape("steps", heads=3, head_dim=128, frames=2, grid_h=7, grid_w=23,
                                                        slots=3)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    blocks = 4                                            # one more than the ring holds: the last block evicts
    tabf = blocks * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    ref_tab = O.rope_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w)
    one, sep = (api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2))
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws1, ws2 = api.attn_workspace(), api.attn_workspace()
    for b in range(blocks):
        host = _inputs(sh, 61, b)
        dev = [[to_dev(x) for x in step] for step in host]
        qs, ks, vs = ([step[t] for step in dev] for t in range(3))
        q_r1 = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
        out1 = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
        api.sdvg_block_steps(one, qs, ks, vs, q_r1, out1, grid, b * sh.frames, tab, tabf, b, sh.scale, ws1)
        assert api.sdvg_block_attn_status(ws1) == api.SDVG_OK
        for s in range(STEPS):
            q_r2, out2 = torch.empty_like(qs[s]), torch.full_like(qs[s], float("nan"))
            api.sdvg_rope3d_qk_commit(sep, qs[s], ks[s], vs[s], q_r2, None, grid, b * sh.frames, tab, tabf, b,
                                      api.SDVG_STAGE)
            api.sdvg_block_attn_fwd(q_r2, None, None, sep, b, out2, None, sh.scale, ws2)
            assert torch.equal(q_r1[s], q_r2) and np.array_equal(to_bits(out1[s]), to_bits(out2)), (b, s)
            # the oracle on the same step: rope, stage, attention against the reference ring
            q, k, v = host[s]
            qr = O.rope_bitspec(q, grid, b * sh.frames, ref_tab, tabf)
            kr = O.rope_bitspec(k, grid, b * sh.frames, ref_tab, tabf)
            assert np.array_equal(to_bits(q_r1[s]), qr)
            o_ref, _ = O.block_attn_ref(qr, kr, v, ref, b, sh.scale)
            err = np.abs(O.bf16_to_f64(to_bits(out1[s])) - o_ref)
            assert err.max() <= ATTN_MAX_ABS and err.mean() <= ATTN_MEAN_ABS, (b, s, err.max(), err.mean())
        assert api.sdvg_block_attn_status(ws2) == api.SDVG_OK
        assert one.state() == sep.state()                 # staging leaves the ring state alone, in both
        # the block's final commit (same clean K/V into both rings and the reference)
        k, v = (synth.block_tensor(sh, 61, b, synth.SRC_DRAFT_CLEAN, t) for t in (synth.K, synth.V))
        kr = O.rope_bitspec(k, grid, b * sh.frames, ref_tab, tabf)
        for c in (one, sep):
            api.sdvg_kv_commit(c, to_dev(kr), to_dev(v), b, api.SDVG_FINAL)
        ref.commit(b, kr, v, O.FINAL)
    for s in range(sh.slots):
        (k1, v1), (k2, v2) = one.read_block(s), sep.read_block(s)
        assert torch.equal(k1, k2) and torch.equal(v1, v2)


def test_block_steps_checks_every_step_before_the_first_launch():
    sh = synth.TINY
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tab = api.sdvg_rope3d_table(sh.head_dim, 4 * sh.frames, sh.grid_h, sh.grid_w).cuda()
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    dev = [[to_dev(x) for x in step] for step in _inputs(sh, 62, 0)]
    qs, ks, vs = ([step[t] for step in dev] for t in range(3))
    q_r = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
    out = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
    # wrong block: refused, and nothing ran (the outputs of step 0 are still untouched)
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_steps(cache, qs, ks, vs, q_r, out, grid, 0, tab, 4 * sh.frames, 3, sh.scale, ws)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    # a misaligned pointer in the LAST step: refused before the first step is enqueued
    raw = torch.empty(qs[0].numel() + 8, dtype=torch.bfloat16, device="cuda")
    bad = raw[1:1 + qs[0].numel()].view(qs[0].shape)
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_steps(cache, qs, ks, vs, q_r, out[:-1] + [bad], grid, 0, tab, 4 * sh.frames, 0, sh.scale, ws)
    assert e.value.status == api.SDVG_ERR_MISALIGNED
    torch.cuda.synchronize()
    assert torch.isnan(out[0].float()).all() and torch.isnan(q_r[0].float()).all()
    with pytest.raises(ValueError):
        api.sdvg_block_steps(cache, qs, ks, vs[:-1], q_r, out, grid, 0, tab, 4 * sh.frames, 0, sh.scale, ws)


def test_block_steps_over_an_8_bit_ring_equal_the_separate_calls():
    sh = synth.Shape("steps8", heads=2, head_dim=128, frames=1, grid_h=9, grid_w=31, slots=2)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tabf = 3 * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    one, sep = (api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True) for _ in range(2))
    ws1, ws2 = api.attn_workspace(), api.attn_workspace()
    inv = torch.full((sh.heads,), 448.0 / 6.0, device="cuda")
    qk_d, v_d = 1.0 / (inv * inv), 1.0 / inv
    for b in range(3):
        dev = [[to_dev(x) for x in step] for step in _inputs(sh, 63, b)]
        qs, ks, vs = ([step[t] for step in dev] for t in range(3))
        q8 = [torch.zeros(qs[0].shape, dtype=torch.uint8, device="cuda") for _ in range(STEPS)]
        out1 = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
        api.sdvg_block_steps_e4m3(one, qs, ks, vs, q8, out1, inv, inv, inv, qk_d, v_d, grid, b * sh.frames, tab, tabf, b,
                                  sh.scale, ws1)
        for s in range(STEPS):
            q8b, out2 = torch.zeros_like(q8[s]), torch.full_like(qs[s], float("nan"))
            api.sdvg_rope3d_qk_commit_e4m3(sep, qs[s], ks[s], vs[s], q8b, inv, inv, inv, grid, b * sh.frames, tab, tabf, b,
                                           api.SDVG_STAGE)
            api.sdvg_block_attn_fwd_e4m3(q8b, None, None, sep, b, qk_d, v_d, out2, None, sh.scale, ws2)
            assert torch.equal(q8[s], q8b) and np.array_equal(to_bits(out1[s]), to_bits(out2)), (b, s)
        assert api.sdvg_block_attn_status(ws1) == api.SDVG_OK and api.sdvg_block_attn_status(ws2) == api.SDVG_OK
        for c in (one, sep):
            api.sdvg_kv_commit_e4m3(c, ks[-1], vs[-1], inv, inv, b, api.SDVG_FINAL)


def test_block_steps_over_a_tile_scaled_ring_equal_the_separate_calls():
    sh = synth.Shape("steps8t", heads=2, head_dim=128, frames=1, grid_h=9, grid_w=31, slots=2)     # 279 tokens: 3 tiles
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tabf = 3 * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    one, sep = (api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True, tile_scales=True) for _ in range(2))
    ws1, ws2 = api.attn_workspace(), api.attn_workspace()
    for b in range(3):
        dev = [[to_dev(x) for x in step] for step in _inputs(sh, 64, b)]
        qs, ks, vs = ([step[t] for step in dev] for t in range(3))
        q8 = [torch.zeros(qs[0].shape, dtype=torch.uint8, device="cuda") for _ in range(STEPS)]
        sc = [torch.zeros((sh.heads, one.tiles), device="cuda") for _ in range(STEPS)]
        out1 = [torch.full_like(qs[0], float("nan")) for _ in range(STEPS)]
        api.sdvg_block_steps_e4m3_tiled(one, qs, ks, vs, q8, sc, out1, grid, b * sh.frames, tab, tabf, b, sh.scale, ws1)
        for s in range(STEPS):
            q8b, scb, out2 = torch.zeros_like(q8[s]), torch.zeros_like(sc[s]), torch.full_like(qs[s], float("nan"))
            api.sdvg_rope3d_qk_commit_e4m3_tiled(sep, qs[s], ks[s], vs[s], q8b, scb, grid, b * sh.frames, tab, tabf, b,
                                                 api.SDVG_STAGE)
            api.sdvg_block_attn_fwd_e4m3_tiled(q8b, scb, sep, b, out2, None, sh.scale, ws2)
            assert torch.equal(q8[s], q8b) and torch.equal(sc[s], scb) and np.array_equal(to_bits(out1[s]), to_bits(out2)), (b, s)
            assert not torch.isnan(out2.float()).any()
        assert api.sdvg_block_attn_status(ws1) == api.SDVG_OK and api.sdvg_block_attn_status(ws2) == api.SDVG_OK
        for c in (one, sep):
            api.sdvg_kv_commit_e4m3_tiled(c, ks[-1], vs[-1], b, api.SDVG_FINAL)
        assert torch.equal(one.k_scale, sep.k_scale) and torch.equal(one.v_scale, sep.v_scale)
    plain = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    with pytest.raises(api.SdvgError) as e:                    # no scale arrays attached: refused before anything runs
        api.sdvg_block_steps_e4m3_tiled(plain, qs, ks, vs, q8, sc, out1, grid, 0, tab, tabf, 0, sh.scale, ws1)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
