"""GPU parity: sdvg_block_attn_fwd against the fp64 oracle on the same bits."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from gpu_utils import ATTN_MAX_ABS, ATTN_MEAN_ABS, ATTN_REL_RMS, Canaries, attn_errors, to_bits, to_dev

pytestmark = pytest.mark.gpu


def check(out_bits, ref, what=""):
    mx, mean, rel = attn_errors(out_bits, ref)
    assert mx <= ATTN_MAX_ABS and mean <= ATTN_MEAN_ABS, (what, mx, mean, rel)
    assert rel <= ATTN_REL_RMS, (what, mx, mean, rel)
    return mx, mean, rel


def run_sequence(sh, nblocks, seed, staged, q_scale=1.0, with_lse=True, rows_per_head=None, full_heads=None):
    """Generate nblocks blocks through a ring of sh.slots slots; compare every block's attention."""
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    rng = np.random.default_rng(seed)
    guard = Canaries()                       # guard bytes around every output and around the rings
    guard.watch_cache(cache)
    for b in range(nblocks):
        q = synth.block_tensor(sh, seed, b, 0, synth.Q, std=q_scale)
        k = synth.block_tensor(sh, seed, b, 0, synth.K)
        v = synth.block_tensor(sh, seed, b, 0, synth.V)
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = guard.like(dq, float("nan"))
        lse = guard.new((sh.heads, sh.block_tokens), torch.float32, float("nan")) if with_lse else None
        if staged:
            api.sdvg_kv_commit(cache, dk, dv, b, api.SDVG_STAGE)
            api.sdvg_block_attn_fwd(dq, None, None, cache, b, out, lse, sh.scale, ws)
        else:
            api.sdvg_block_attn_fwd(dq, dk, dv, cache, b, out, lse, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        got = to_bits(out)
        if rows_per_head is None:
            o_ref, lse_ref = O.block_attn_ref(q, k, v, ref, b, sh.scale)
            check(got, o_ref, (sh.name, b, staged))
            if with_lse:
                assert np.allclose(lse.cpu().numpy(), lse_ref, rtol=0, atol=2e-3)
        else:
            for h in range(sh.heads):
                rows = np.arange(sh.block_tokens) if (full_heads and h in full_heads) else \
                    np.sort(rng.choice(sh.block_tokens, rows_per_head, replace=False))
                o_ref, lse_ref = O.block_attn_ref(q, k, v, ref, b, sh.scale, heads=[h], rows=rows)
                check(got[rows, h], o_ref[:, 0], (sh.name, b, h))
                if with_lse:
                    assert np.allclose(lse.cpu().numpy()[h, rows], lse_ref[0], rtol=0, atol=2e-3)
        api.sdvg_kv_commit(cache, dk, dv, b, api.SDVG_FINAL)
        ref.commit(b, k, v, O.FINAL)
        guard.check()
    cache.close()


@pytest.mark.parametrize("staged", [False, True])
def test_config1_tiny_every_fill_level(staged):
    # 2 heads x d64, 64-token blocks, ring of 3: Lk = 64, 128, 192, then wrapped rings
    run_sequence(synth.TINY, 5, 0, staged)


@pytest.mark.parametrize("staged", [False, True])
def test_d128_ragged_tiles_and_wraparound(staged):
    # 2*5*23 = 230 tokens: two query tiles with a ragged tail, key segments with ragged ends
    sh = synth.Shape("ragged128", heads=3, head_dim=128, frames=2, grid_h=5, grid_w=23, slots=3)
    run_sequence(sh, 5, 41, staged)


def test_d64_multi_tile():
    sh = synth.Shape("ragged64", heads=2, head_dim=64, frames=3, grid_h=7, grid_w=19, slots=4)
    run_sequence(sh, 6, 42, True)


@pytest.mark.parametrize("heads,dim", [(3, 128), (1, 64), (5, 64)])
def test_odd_tile_count_with_odd_head_count(heads, dim):
    # 300 tokens = 3 query tiles per head: the third tiles of two heads share a work item, and with an odd
    # number of heads the last such item has a single lane
    sh = synth.Shape("odd-odd", heads=heads, head_dim=dim, frames=1, grid_h=12, grid_w=25, slots=3)
    run_sequence(sh, 4, 45 + heads, True)
    run_sequence(sh, 2, 46 + heads, False)


def test_peaky_logits_keep_the_absolute_tolerance():
    # q scaled x4: softmax concentrates on few keys and outputs are O(1)
    sh = synth.Shape("peaky", heads=2, head_dim=128, frames=1, grid_h=12, grid_w=25, slots=3)
    run_sequence(sh, 4, 43, True, q_scale=4.0)


def test_closed_forms_on_device():
    sh = synth.Shape("cf", heads=2, head_dim=128, frames=1, grid_h=10, grid_w=20, slots=2)
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    k = synth.block_tensor(sh, 44, 0, 0, synth.K)
    v = synth.block_tensor(sh, 44, 0, 0, synth.V)
    q0 = np.zeros_like(k)
    out = torch.empty_like(to_dev(k))
    lse = torch.empty((sh.heads, sh.block_tokens), device="cuda")
    api.sdvg_block_attn_fwd(to_dev(q0), to_dev(k), to_dev(v), cache, 0, out, lse, sh.scale, ws)
    # q = 0: uniform weights, the output is the mean of V and lse = ln(Lk)
    mean_v = O.bf16_to_f64(v).mean(axis=0)
    got = O.bf16_to_f64(to_bits(out))
    assert np.abs(got - mean_v[None]).max() <= 2e-3
    assert np.allclose(lse.cpu().numpy(), np.log(sh.block_tokens), atol=1e-4)


def rows_touching_every_tile(rng, tokens, extra):
    """One random row of every 128-row query tile plus `extra` random rows: no tile of a head goes unsampled."""
    tiles = (tokens + 127) // 128
    one_each = [int(rng.integers(t * 128, min(tokens, (t + 1) * 128))) for t in range(tiles)]
    more = rng.choice(tokens, extra, replace=False)
    return np.unique(np.concatenate([one_each, more]))


def test_config2_wan13b_shape_sampled_and_two_full_heads():
    sh = synth.WAN_1_3B
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    for b in range(2):
        k = synth.block_tensor(sh, 2, b, 0, synth.K)
        v = synth.block_tensor(sh, 2, b, 0, synth.V)
        api.sdvg_kv_commit(cache, to_dev(k), to_dev(v), b, api.SDVG_FINAL)
        ref.commit(b, k, v, O.FINAL)
    q, k, v = (synth.block_tensor(sh, 2, 2, 0, t) for t in (synth.Q, synth.K, synth.V))
    out = torch.full_like(to_dev(q), float("nan"))
    api.sdvg_kv_commit(cache, to_dev(k), to_dev(v), 2, api.SDVG_STAGE)
    api.sdvg_block_attn_fwd(to_dev(q), None, None, cache, 2, out, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    assert not torch.isnan(out.float()).any()                  # every row of every tile was written
    got = to_bits(out)
    rng = np.random.default_rng(2)
    for h in range(sh.heads):
        rows = np.arange(sh.block_tokens) if h in (0, 11) else rows_touching_every_tile(rng, sh.block_tokens, 64)
        o_ref, _ = O.block_attn_ref(q, k, v, ref, 2, sh.scale, heads=[h], rows=rows)
        check(got[rows, h], o_ref[:, 0], ("wan1.3b", h))


def test_config3_wan14b_shape_fused_prologue_cache_bits_and_sampled_attention():
    sh = synth.WAN_14B
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tabf = 7 * sh.frames
    ref_tab = O.rope_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w)
    dev_tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    pool = synth.TensorPool(sh, 3)
    for b in range(6):
        k, v = pool.get(b, 0, synth.K), pool.get(b, 0, synth.V)
        ev = api.sdvg_rope3d_qk_commit(cache, None, to_dev(k), to_dev(v), None, None, grid, b * sh.frames, dev_tab,
                                       tabf, b, api.SDVG_FINAL)
        assert ev == -1
        ref.commit(b, O.rope_bitspec(k, grid, b * sh.frames, ref_tab, tabf), v, O.FINAL)
    b = 6
    q, k, v = (synth.block_tensor(sh, 3, b, 0, t) for t in (synth.Q, synth.K, synth.V))
    dq = to_dev(q)
    q_r = torch.empty_like(dq)
    api.sdvg_rope3d_qk_commit(cache, dq, to_dev(k), to_dev(v), q_r, None, grid, b * sh.frames, dev_tab, tabf, b,
                              api.SDVG_STAGE)
    out = torch.full_like(dq, float("nan"))
    lse = torch.full((sh.heads, sh.block_tokens), float("nan"), device="cuda")
    api.sdvg_block_attn_fwd(q_r, None, None, cache, b, out, lse, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    assert not torch.isnan(out.float()).any() and not torch.isnan(lse).any()      # every row of every tile was written
    qr_ref = O.rope_bitspec(q, grid, b * sh.frames, ref_tab, tabf)
    kr_ref = O.rope_bitspec(k, grid, b * sh.frames, ref_tab, tabf)
    assert np.array_equal(to_bits(q_r), qr_ref)
    # cache contents, bit for bit, all 7 slots (slot 6 holds the staged block)
    for s in range(6):
        gk, gv = cache.read_block(s)
        assert np.array_equal(to_bits(gk), ref.k[s]) and np.array_equal(to_bits(gv), ref.v[s])
    gk, gv = cache.read_block(6)
    assert np.array_equal(to_bits(gk), kr_ref) and np.array_equal(to_bits(gv), v)
    got = to_bits(out)
    rng = np.random.default_rng(3)
    lse_h = lse.cpu().numpy()
    for h in range(sh.heads):
        rows = np.arange(sh.block_tokens) if h in (0, 39) else rows_touching_every_tile(rng, sh.block_tokens, 30)
        o_ref, lse_ref = O.block_attn_ref(qr_ref, kr_ref, v, ref, b, sh.scale, heads=[h], rows=rows)
        check(got[rows, h], o_ref[:, 0], ("wan14b", h))
        assert np.allclose(lse_h[h, rows], lse_ref[0], rtol=0, atol=2e-3)


def test_batched_call_equals_separate_calls_and_the_oracle():
    # cond / uncond pair of one shape: one launch over both problems; bit-identical to two separate calls
    sh = synth.Shape("pair", heads=3, head_dim=128, frames=1, grid_h=12, grid_w=25, slots=3)
    caches = [api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    refs = [O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    ws = api.attn_workspace()
    for b in range(4):
        qkv = [[synth.block_tensor(sh, 60 + n, b, 0, t) for t in (synth.Q, synth.K, synth.V)] for n in range(2)]
        dev = [[to_dev(x) for x in prob] for prob in qkv]
        for n in range(2):
            api.sdvg_kv_commit(caches[n], dev[n][1], dev[n][2], b, api.SDVG_STAGE)
        outs = [torch.full_like(dev[n][0], float("nan")) for n in range(2)]
        lses = [torch.full((sh.heads, sh.block_tokens), float("nan"), device="cuda") for _ in range(2)]
        api.sdvg_block_attn_fwd_batched([d[0] for d in dev], None, None, caches, [b, b], outs, lses, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        for n in range(2):
            one = torch.empty_like(outs[n])
            api.sdvg_block_attn_fwd(dev[n][0], None, None, caches[n], b, one, None, sh.scale, ws)
            assert torch.equal(one.view(torch.int16), outs[n].view(torch.int16))
            o_ref, lse_ref = O.block_attn_ref(*qkv[n], refs[n], b, sh.scale)
            check(to_bits(outs[n]), o_ref, ("batched", b, n))
            assert np.allclose(lses[n].cpu().numpy(), lse_ref, rtol=0, atol=2e-3)
            api.sdvg_kv_commit(caches[n], dev[n][1], dev[n][2], b, api.SDVG_FINAL)
            refs[n].commit(b, qkv[n][1], qkv[n][2], O.FINAL)


def test_batched_call_with_different_ring_fill_falls_back_to_separate_launches():
    sh = synth.Shape("pair2", heads=2, head_dim=64, frames=1, grid_h=10, grid_w=20, slots=3)
    caches = [api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    refs = [O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    ws = api.attn_workspace()
    k0, v0 = synth.block_tensor(sh, 70, 0, 0, synth.K), synth.block_tensor(sh, 70, 0, 0, synth.V)
    api.sdvg_kv_commit(caches[1], to_dev(k0), to_dev(v0), 0, api.SDVG_FINAL)     # problem 1 is one block ahead
    refs[1].commit(0, k0, v0, O.FINAL)
    blocks = [0, 1]
    qkv = [[synth.block_tensor(sh, 71 + n, blocks[n], 0, t) for t in (synth.Q, synth.K, synth.V)] for n in range(2)]
    dev = [[to_dev(x) for x in prob] for prob in qkv]
    outs = [torch.empty_like(dev[n][0]) for n in range(2)]
    api.sdvg_block_attn_fwd_batched([d[0] for d in dev], [d[1] for d in dev], [d[2] for d in dev], caches, blocks,
                                    outs, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    for n in range(2):
        o_ref, _ = O.block_attn_ref(*qkv[n], refs[n], blocks[n], sh.scale)
        check(to_bits(outs[n]), o_ref, ("fallback", n))
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_attn_fwd_batched([dev[0][0]] * 5, None, None, [caches[0]] * 5, [0] * 5, [outs[0]] * 5, None,
                                        sh.scale, ws)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE


def test_bounded_wait_gives_up_reports_timeout_and_leaves_the_context_usable():
    import time
    ws = api.attn_workspace()
    t0 = time.perf_counter()
    api.sdvg_selftest_bounded_wait(ws, 20_000_000)                   # 20 ms limit on a phase nothing completes
    assert api.sdvg_block_attn_status(ws) == api.SDVG_ERR_TIMEOUT    # synchronises the stream
    dt = time.perf_counter() - t0
    assert 0.015 <= dt < 1.0, dt
    assert int(ws.view(torch.int32)[0].item()) == 2                  # the waiting warp ran to its end
    # the device still works: a normal attention call on the same workspace succeeds; the status word is
    # sticky, so the timeout stays visible until the workspace is reset
    sh = synth.TINY
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    q, k, v = (to_dev(synth.block_tensor(sh, 80, 0, 0, t)) for t in (synth.Q, synth.K, synth.V))
    out = torch.full_like(q, float("nan"))
    api.sdvg_block_attn_fwd(q, k, v, cache, 0, out, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_ERR_TIMEOUT
    assert torch.isfinite(out.float()).all()
    api.sdvg_block_attn_workspace_reset(ws)
    api.sdvg_block_attn_fwd(q, k, v, cache, 0, out, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK


def _lazy_raises(tile_max_log2, lazy=8.0):
    """Number of times the lazy reference-maximum policy moves the reference of a row, given the row's
    per-key-tile maxima in the exp2 domain, in the order a lane visits the tiles: the first tile sets the
    reference, a later tile moves it when its maximum exceeds it by more than 2^lazy."""
    ref, n = tile_max_log2[0], 0
    for m in tile_max_log2[1:]:
        if m - ref > lazy:
            ref, n = m, n + 1
    return n


def test_rising_logits_rescale_the_accumulator_at_almost_every_key_tile():
    # Keys whose magnitude grows along the sequence: the row maximum keeps rising by more than the lazy-rescale
    # threshold, so the softmax threads rescale O (and their partial row sums) again and again.
    sh = synth.Shape("rising", heads=2, head_dim=128, frames=3, grid_h=16, grid_w=16, slots=3)   # 768 tokens = 6 key tiles per block
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    ks = []
    for b in range(3):
        q = synth.block_tensor(sh, 90, b, 0, synth.Q, std=1.0)
        # all queries share a direction with the keys so that logits grow with the key index
        base = O.bf16_to_f64(synth.block_tensor(sh, 90, 0, 1, synth.K))[0:1, :, :]
        ramp = (1.0 + 10.0 * (np.arange(sh.block_tokens) + b * sh.block_tokens) / (3 * sh.block_tokens))[:, None, None]
        k = O.f64_to_bf16(base * ramp + 0.05 * O.bf16_to_f64(synth.block_tensor(sh, 90, b, 0, synth.K)))
        q = O.f64_to_bf16(np.abs(O.bf16_to_f64(q)) * np.sign(base) * 1.5)
        v = synth.block_tensor(sh, 90, b, 0, synth.V)
        ks.append(k)
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        out = torch.full_like(dq, float("nan"))
        lse = torch.full((sh.heads, sh.block_tokens), float("nan"), device="cuda")
        api.sdvg_kv_commit(cache, dk, dv, b, api.SDVG_STAGE)
        api.sdvg_block_attn_workspace_reset(ws)
        api.sdvg_block_attn_fwd(dq, None, None, cache, b, out, lse, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        o_ref, lse_ref = O.block_attn_ref(q, k, v, ref, b, sh.scale)
        check(to_bits(out), o_ref, ("rising", b))
        assert np.allclose(lse.cpu().numpy(), lse_ref, rtol=2e-4, atol=2e-3)
        # The rescale path must have run.  From the exact logits: how often does the lazy policy move a row's
        # reference, whether a lane visits every key tile or every second one (a query tile that is worked on by
        # both lanes)?  A warp takes the path when any of its 32 rows moves, and a row has two threads, in two warps.
        kk = np.concatenate([O.bf16_to_f64(x) for x in ks], axis=0)                  # keys in ring order (no wrap yet)
        logit2 = np.einsum("thd,shd->hts", O.bf16_to_f64(q), kk) * sh.scale * 1.4426950408889634
        tile_max = logit2.reshape(sh.heads, sh.block_tokens, -1, 128).max(axis=3)    # [heads, rows, key tiles]
        floor_events = 0
        for h in range(sh.heads):
            per_row = np.array([min(_lazy_raises(tile_max[h, r]), _lazy_raises(tile_max[h, r, 0::2]) +
                                    _lazy_raises(tile_max[h, r, 1::2])) if tile_max.shape[2] > 1 else 0
                                for r in range(sh.block_tokens)])
            floor_events += 2 * int(per_row.reshape(-1, 32).min(axis=1).sum())
        events = api.sdvg_block_attn_rescale_events(ws)
        assert floor_events >= 2 * sh.heads * (sh.block_tokens // 32), floor_events       # the data does force it
        assert events >= floor_events, (events, floor_events)
        api.sdvg_kv_commit(cache, dk, dv, b, api.SDVG_FINAL)
        ref.commit(b, k, v, O.FINAL)


@pytest.mark.parametrize("slots", [1, 2])
@pytest.mark.parametrize("staged", [False, True])
def test_smallest_rings(slots, staged):
    # slots = 1: a block sees only itself; slots = 2: itself and the block before it
    sh = synth.Shape(f"ring{slots}", heads=2, head_dim=64, frames=1, grid_h=9, grid_w=17, slots=slots)
    run_sequence(sh, 4, 95 + slots, staged)


def test_several_rounds_of_pairs_with_odd_tiles_per_head_single_and_batched():
    # 41 heads x 15 tiles = 615 tiles: on a 148-SM GPU two full rounds of pairs (dealt one CTA further on in the
    # second round), pairs that straddle heads in both, 23 key-split singles; two problems in one call double that.
    # Every head is checked on a row of every one of its tiles.
    sh = synth.Shape("rounds", heads=41, head_dim=128, frames=1, grid_h=38, grid_w=50, slots=2)      # 1900 tokens
    caches = [api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    refs = [O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim) for _ in range(2)]
    ws = api.attn_workspace()
    rng = np.random.default_rng(17)
    for n in range(2):
        k0, v0 = synth.block_tensor(sh, 90 + n, 0, 0, synth.K), synth.block_tensor(sh, 90 + n, 0, 0, synth.V)
        api.sdvg_kv_commit(caches[n], to_dev(k0), to_dev(v0), 0, api.SDVG_FINAL)
        refs[n].commit(0, k0, v0, O.FINAL)
    qkv = [[synth.block_tensor(sh, 90 + n, 1, 0, t) for t in (synth.Q, synth.K, synth.V)] for n in range(2)]
    dev = [[to_dev(x) for x in prob] for prob in qkv]
    for n in range(2):
        api.sdvg_kv_commit(caches[n], dev[n][1], dev[n][2], 1, api.SDVG_STAGE)
    one = torch.full_like(dev[0][0], float("nan"))
    api.sdvg_block_attn_fwd(dev[0][0], None, None, caches[0], 1, one, None, sh.scale, ws)
    outs = [torch.full_like(dev[n][0], float("nan")) for n in range(2)]
    api.sdvg_block_attn_fwd_batched([d[0] for d in dev], None, None, caches, [1, 1], outs, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    for o in [one] + outs:
        assert not torch.isnan(o.float()).any()
    for h in range(sh.heads):
        rows = rows_touching_every_tile(rng, sh.block_tokens, 8)
        for n in range(2):
            o_ref, _ = O.block_attn_ref(*qkv[n], refs[n], 1, sh.scale, heads=[h], rows=rows)
            check(to_bits(outs[n])[rows, h], o_ref[:, 0], ("rounds batched", n, h))
            if n == 0:
                check(to_bits(one)[rows, h], o_ref[:, 0], ("rounds single", h))
