"""GPU parity: 3D-RoPE, ring commit and their fusion against the oracle, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from gpu_utils import Canaries, to_bits, to_dev

pytestmark = pytest.mark.gpu

ODD = synth.Shape("odd", heads=11, head_dim=128, frames=2, grid_h=5, grid_w=7, slots=4)
ODD64 = synth.Shape("odd64", heads=9, head_dim=64, frames=3, grid_h=3, grid_w=5, slots=2)


def tables(sh, tab_frames):
    ref = O.rope_table(sh.head_dim, tab_frames, sh.grid_h, sh.grid_w)
    mine = api.sdvg_rope3d_table(sh.head_dim, tab_frames, sh.grid_h, sh.grid_w)
    assert np.array_equal(mine.numpy().view(np.uint32), ref.view(np.uint32))
    return ref, mine.cuda()


@pytest.mark.parametrize("sh", [synth.TINY, ODD, ODD64, synth.WAN_1_3B, synth.WAN_14B], ids=lambda s: s.name)
def test_rope_bit_exact(sh):
    tabf = 12
    ref_tab, dev_tab = tables(sh, tabf)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    fo = tabf - sh.frames
    q = synth.block_tensor(sh, 31, 1, 0, synth.Q)
    k = synth.block_tensor(sh, 31, 1, 0, synth.K)
    dq, dk = to_dev(q), to_dev(k)
    guard = Canaries()
    oq, ok = guard.like(dq), guard.like(dk)
    api.sdvg_rope3d_qk(dq, dk, oq, ok, grid, fo, dev_tab, tabf)
    want_q = O.rope_bitspec(q, grid, fo, ref_tab, tabf)
    want_k = O.rope_bitspec(k, grid, fo, ref_tab, tabf)
    assert np.array_equal(to_bits(oq), want_q)
    assert np.array_equal(to_bits(ok), want_k)
    guard.check()
    assert np.array_equal(to_bits(dq), q)              # inputs untouched
    # in place, and k alone
    api.sdvg_rope3d_qk(dq, None, dq, None, grid, fo, dev_tab, tabf)
    assert np.array_equal(to_bits(dq), want_q)
    api.sdvg_rope3d_qk(None, dk, None, dk, grid, fo, dev_tab, tabf)
    assert np.array_equal(to_bits(dk), want_k)


def test_rope_close_to_fp64_rotation_on_gpu_output():
    sh = ODD
    ref_tab, dev_tab = tables(sh, 4)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    k = synth.block_tensor(sh, 32, 0, 0, synth.K)
    out = torch.empty_like(to_dev(k))
    api.sdvg_rope3d_qk(None, to_dev(k), None, out, grid, 2, dev_tab, 4)
    ref = O.rope_ref(k, grid, 2)
    got = O.bf16_to_f64(to_bits(out))
    mag = np.repeat(np.sqrt(ref[..., 0::2] ** 2 + ref[..., 1::2] ** 2), 2, axis=-1)
    assert np.all(np.abs(got - ref) <= mag * 2.0 ** -8 + 1e-30)


@pytest.mark.parametrize("sh", [synth.TINY, ODD, ODD64], ids=lambda s: s.name)
def test_commit_ring_trace_and_contents(sh):
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    guard = Canaries()
    guard.watch_cache(cache)
    nblocks = 2 * sh.slots + 1
    for b in range(nblocks):
        k = synth.block_tensor(sh, 33, b, 0, synth.K)
        v = synth.block_tensor(sh, 33, b, 0, synth.V)
        if b % 2:
            ks = synth.block_tensor(sh, 33, b, 1, synth.K)       # provisional bits first
            assert api.sdvg_kv_commit(cache, to_dev(ks), to_dev(v), b, api.SDVG_STAGE) == -1
            ref.commit(b, ks, v, O.STAGE)
            nb, slots_, staged = cache.state()
            assert nb == ref.next_block == b and slots_ == ref.slot_block and staged == b
            gk, _ = cache.read_block(b % sh.slots)
            assert np.array_equal(to_bits(gk), ks)
        ev = api.sdvg_kv_commit(cache, to_dev(k), to_dev(v), b, api.SDVG_FINAL)
        assert ev == ref.commit(b, k, v, O.FINAL)
        nb, slots_, staged = cache.state()
        assert nb == ref.next_block and slots_ == ref.slot_block and staged == -1
        with pytest.raises(api.SdvgError) as e:
            api.sdvg_kv_commit(cache, to_dev(k), to_dev(v), b, api.SDVG_FINAL)      # same block twice
        assert e.value.status == api.SDVG_ERR_BAD_STATE
    for s in range(sh.slots):
        gk, gv = cache.read_block(s)
        assert np.array_equal(to_bits(gk), ref.k[s]) and np.array_equal(to_bits(gv), ref.v[s])
    guard.check()
    cache.reset()
    assert cache.state() == (0, [-1] * sh.slots, -1)
    cache.close()


@pytest.mark.parametrize("sh", [synth.TINY, ODD, synth.WAN_1_3B], ids=lambda s: s.name)
def test_fused_rope_commit_equals_two_calls_and_oracle(sh):
    tabf = 3 * sh.frames
    ref_tab, dev_tab = tables(sh, tabf)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    fused = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    split = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    guard = Canaries()
    guard.watch_cache(fused)
    for b in range(3):
        q, k, v = (synth.block_tensor(sh, 34, b, 0, t) for t in (synth.Q, synth.K, synth.V))
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        fo = b * sh.frames
        q1, k1 = guard.like(dq), guard.like(dk)
        api.sdvg_rope3d_qk_commit(fused, dq, dk, dv, q1, k1 if b == 1 else None, grid, fo, dev_tab, tabf, b,
                                  api.SDVG_STAGE)
        assert fused.state()[2] == b
        ev1 = api.sdvg_rope3d_qk_commit(fused, None, dk, dv, None, None, grid, fo, dev_tab, tabf, b,
                                        api.SDVG_FINAL)
        q2, k2 = torch.empty_like(dq), torch.empty_like(dk)
        api.sdvg_rope3d_qk(dq, dk, q2, k2, grid, fo, dev_tab, tabf)
        ev2 = api.sdvg_kv_commit(split, k2, dv, b, api.SDVG_FINAL)
        assert ev1 == ev2 == -1
        want_k = O.rope_bitspec(k, grid, fo, ref_tab, tabf)
        assert np.array_equal(to_bits(q1), to_bits(q2))
        assert np.array_equal(to_bits(q1), O.rope_bitspec(q, grid, fo, ref_tab, tabf))
        if b == 1:
            assert np.array_equal(to_bits(k1), want_k)
        for c in (fused, split):
            gk, gv = c.read_block(b % sh.slots)
            assert np.array_equal(to_bits(gk), want_k)
            assert np.array_equal(to_bits(gv), v)
    guard.check()
    assert fused.state() == split.state()
