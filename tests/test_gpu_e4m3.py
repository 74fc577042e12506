"""GPU parity of the 8-bit (E4M3) variant: quantiser and ring commit bit-exact, attention within the bound
that the one extra rounding (P to E4M3 before the second product) allows."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from gpu_utils import Canaries, f32_dev, to_bits, to_dev

pytestmark = pytest.mark.gpu


def codes_dev(c: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(c)).cuda()


def p_rounding_bound(q8, k8, v8, qk_descale, v_descale, scale, heads, rows):
    """Per-element bound on |out - oracle|.

    With p_j = exp(s_j - max s) (so max p = 1) the kernel rounds 2^e * p_j to E4M3 for some e in [4, 8] (its
    reference maximum lags the true one by at most 2^4, and it shifts the window up by 2^4): a normal number
    moves by at most 2^-4 of itself, a subnormal one (below 2^-6 after scaling) by at most 2^-10 / 2^4 in
    units of p.  So |d o| <= sum_j max(2^-4 p_j, 2^-14) |v_j| / sum_j p_j; on top come the fp32 arithmetic
    (ex2.approx, accumulation: ~1e-5 relative) and the bf16 rounding of the result (2^-9 relative).
    """
    out = np.empty((len(rows), len(heads), q8.shape[2]))
    for hi, h in enumerate(heads):
        s = (O.e4m3_decode(q8[rows, h, :]) @ O.e4m3_decode(k8[:, h, :]).T) * (scale * qk_descale[h])
        p = np.exp(s - s.max(axis=1, keepdims=True))
        dp = np.maximum(p * 2.0 ** -4, 2.0 ** -14)
        out[:, hi, :] = (dp @ np.abs(O.e4m3_decode(v8[:, h, :]))) / p.sum(axis=1, keepdims=True) * v_descale[h]
    return out


def check_attention(out, o_ref, bound, what):
    got = O.bf16_to_f64(to_bits(out))
    err = np.abs(got - o_ref)
    tol = bound + np.abs(o_ref) * 2.0 ** -8 + 1e-6
    assert np.all(err <= tol), (what, float(err.max()), float((err / tol).max()))
    # rounding errors of the thousands of probabilities behind one output are independent: far inside the bound on average
    assert err.mean() <= 0.25 * tol.mean(), (what, float(err.mean()), float(tol.mean()))


@pytest.mark.parametrize("dim", [64, 128])
def test_quantiser_bit_exact_including_special_values(dim):
    rng = np.random.default_rng(3)
    tokens, heads = 257, 5
    x = synth.normal_bf16((tokens, heads, dim), 11, dim, std=2.0)
    special = np.array([0.0, -0.0, 448.0, 464.0, 1e6, -1e6, 2.0 ** -9, 2.0 ** -10, 2.0 ** -10 * 1.01, 1.0625, 1.1875, 1.9375,
                        -0.0146, np.inf, -np.inf, 3e-30], dtype=np.float32)
    x[0, 0, :special.size] = synth.f32_to_bf16_bits(special)        # head 0 has scale 1 below
    inv = np.array([1.0, 37.25, 0.0131, 448.0, 1e-3], dtype=np.float32)
    out = torch.zeros((tokens, heads, dim), dtype=torch.uint8, device="cuda")
    api.sdvg_quant_e4m3(to_dev(x), f32_dev(inv), out)
    assert np.array_equal(out.cpu().numpy(), O.quant_e4m3_ref(x, inv))
    with pytest.raises(api.SdvgError):
        api.sdvg_quant_e4m3(to_dev(x)[:, :, :48].contiguous(), f32_dev(inv), out[:, :, :48].contiguous())   # head_dim 48


def test_ring_commit_quantises_into_the_slots_and_types_do_not_mix():
    sh = synth.Shape("e4m3-ring", heads=3, head_dim=128, frames=1, grid_h=5, grid_w=13, slots=3)
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    ring = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, dtype=np.uint8)
    k_inv = np.array([20.0, 35.5, 70.0], dtype=np.float32)
    v_inv = np.array([64.0, 10.0, 100.0], dtype=np.float32)
    for b in range(5):
        k = synth.block_tensor(sh, 5, b, 0, synth.K)
        v = synth.block_tensor(sh, 5, b, 0, synth.V, std=3.0)
        k8, v8 = O.quant_e4m3_ref(k, k_inv), O.quant_e4m3_ref(v, v_inv)
        assert api.sdvg_kv_commit_e4m3(cache, to_dev(k), to_dev(v), f32_dev(k_inv), f32_dev(v_inv), b, api.SDVG_STAGE) == -1
        assert cache.state()[2] == b
        ev = api.sdvg_kv_commit_e4m3(cache, to_dev(k), to_dev(v), f32_dev(k_inv), f32_dev(v_inv), b, api.SDVG_FINAL)
        assert ev == ring.commit(b, k8, v8, O.FINAL)
        for s in range(sh.slots):
            gk, gv = cache.read_block(s)
            if ring.slot_block[s] >= 0:
                assert np.array_equal(gk.cpu().numpy(), ring.k[s]) and np.array_equal(gv.cpu().numpy(), ring.v[s])
        assert cache.state()[:2] == (ring.next_block, ring.slot_block)
    # out of order, and the two element types are not interchangeable
    k = to_dev(synth.block_tensor(sh, 5, 9, 0, synth.K))
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_kv_commit_e4m3(cache, k, k, f32_dev(k_inv), f32_dev(v_inv), 7, api.SDVG_FINAL)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_kv_commit(cache, k, k, 5, api.SDVG_FINAL)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE
    bf = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_kv_commit_e4m3(bf, k, k, f32_dev(k_inv), f32_dev(v_inv), 0, api.SDVG_FINAL)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE
    ws = api.attn_workspace()
    q8 = torch.zeros((sh.block_tokens, sh.heads, sh.head_dim), dtype=torch.uint8, device="cuda")
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_attn_fwd_e4m3(q8, q8, q8, bf, 0, f32_dev(k_inv), f32_dev(v_inv), torch.empty_like(k), None, 0.1, ws)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE
    with pytest.raises(api.SdvgError):
        api.Cache(sh.slots, sh.heads, sh.block_tokens, 64, e4m3=True)          # the 8-bit ring is built for head_dim 128


def run_sequence(sh, nblocks, seed, q_std=1.0, k_gain=None, rows_per_head=None, staged_only=False):
    """Blocks through an 8-bit ring; every block's attention (staged and with explicit self K/V) against the oracle."""
    H = sh.heads
    cache = api.Cache(sh.slots, H, sh.block_tokens, sh.head_dim, e4m3=True)
    ring = O.RingCacheRef(sh.slots, H, sh.block_tokens, sh.head_dim, dtype=np.uint8)
    ws = api.attn_workspace()
    rng = np.random.default_rng(seed)
    guard = Canaries()                       # guard bytes around the outputs and around the 8-bit rings
    guard.watch_cache(cache)
    k_gain = np.ones(H, dtype=np.float32) if k_gain is None else np.asarray(k_gain, dtype=np.float32)
    # static scales sized for ~4.5 standard deviations of each tensor; different per head
    sq = (4.5 * q_std / 448 * (1 + 0.1 * np.arange(H))).astype(np.float32)
    sk = (4.5 * k_gain / 448).astype(np.float32)
    sv = (4.5 / 448 * (1 + 0.05 * np.arange(H))).astype(np.float32)
    qkd, vd = (sq * sk).astype(np.float32), sv
    for b in range(nblocks):
        q = synth.block_tensor(sh, seed, b, 0, synth.Q, std=q_std)
        k = synth.block_tensor(sh, seed, b, 0, synth.K)
        if not np.all(k_gain == 1):
            k = O.f32_to_bf16(O.bf16_to_f32(k) * k_gain.reshape(1, -1, 1))
        v = synth.block_tensor(sh, seed, b, 0, synth.V)
        q8, k8, v8 = O.quant_e4m3_ref(q, 1 / sq), O.quant_e4m3_ref(k, 1 / sk), O.quant_e4m3_ref(v, 1 / sv)
        dq8 = guard.new(q8.shape, torch.uint8)
        api.sdvg_quant_e4m3(to_dev(q), f32_dev(1 / sq), dq8)
        assert np.array_equal(dq8.cpu().numpy(), q8)
        api.sdvg_kv_commit_e4m3(cache, to_dev(k), to_dev(v), f32_dev(1 / sk), f32_dev(1 / sv), b, api.SDVG_STAGE)
        out = guard.new((sh.block_tokens, H, sh.head_dim), torch.bfloat16, float("nan"))
        lse = guard.new((H, sh.block_tokens), torch.float32, float("nan"))
        api.sdvg_block_attn_fwd_e4m3(dq8, None, None, cache, b, f32_dev(qkd), f32_dev(vd), out, lse, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        outs = [out]
        if not staged_only:
            out2 = torch.full_like(out, float("nan"))
            api.sdvg_block_attn_fwd_e4m3(dq8, codes_dev(k8), codes_dev(v8), cache, b, f32_dev(qkd), f32_dev(vd), out2, None,
                                         sh.scale, ws)
            assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
            # same keys in the same order, whether the block comes from the ring or from its own tensors
            # (bit-identical when the ring part ends on a tile boundary; otherwise the tiles, and with them the
            # reference maxima and the roundings of P, differ, and the second result is checked like the first)
            if ring.window(b)[0].shape[0] % 128 == 0:
                assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
            else:
                outs.append(out2)
        kw, vw = ring.window(b)
        k_all, v_all = np.concatenate([kw, k8]), np.concatenate([vw, v8])
        heads = list(range(H))
        for h in heads:
            rows = np.arange(sh.block_tokens) if rows_per_head is None else \
                np.sort(rng.choice(sh.block_tokens, rows_per_head, replace=False))
            o_ref, lse_ref = O.attn_e4m3_ref(q8, k_all, v_all, qkd.astype(np.float64), vd.astype(np.float64), sh.scale,
                                            heads=[h], rows=rows)
            bound = p_rounding_bound(q8, k_all, v_all, qkd.astype(np.float64), vd.astype(np.float64), sh.scale, [h], rows)
            for o in outs:
                check_attention(o[rows, h], o_ref[:, 0], bound[:, 0], (sh.name, b, h))
            # the logits themselves are exact products of 8-bit numbers accumulated in fp32
            assert np.allclose(lse.cpu().numpy()[h, rows], lse_ref[0], rtol=0, atol=2e-3)
        api.sdvg_kv_commit_e4m3(cache, to_dev(k), to_dev(v), f32_dev(1 / sk), f32_dev(1 / sv), b, api.SDVG_FINAL)
        ring.commit(b, k8, v8, O.FINAL)
        guard.check()
    cache.close()


def test_every_fill_level_ragged_tiles_and_wraparound():
    # 230 tokens: two query tiles with a ragged tail; key segments with ragged ends; the ring wraps twice
    sh = synth.Shape("e4m3-ragged", heads=3, head_dim=128, frames=2, grid_h=5, grid_w=23, slots=3)
    run_sequence(sh, 6, 41)


def test_odd_tiles_odd_heads_and_peaked_rows():
    # 300 tokens = 3 query tiles per head (pairs that straddle heads, a split tile); large logits make a
    # few keys dominate, where the rounding of P is least averaged out; head 2's keys are 3x larger
    sh = synth.Shape("e4m3-odd", heads=3, head_dim=128, frames=1, grid_h=12, grid_w=25, slots=4)
    run_sequence(sh, 5, 7, q_std=3.0, k_gain=[1.0, 0.5, 3.0])


def test_single_slot_and_single_tile():
    sh = synth.Shape("e4m3-one", heads=1, head_dim=128, frames=1, grid_h=7, grid_w=11, slots=1)
    run_sequence(sh, 3, 3)


def test_closed_forms():
    T, H, D = 200, 2, 128
    cache = api.Cache(2, H, T, D, e4m3=True)
    ws = api.attn_workspace()
    ones = torch.ones(H, device="cuda")
    rng = np.random.default_rng(1)
    v8 = rng.integers(0, 0x7F, (T, H, D)).astype(np.uint8) | (rng.integers(0, 2, (T, H, D)).astype(np.uint8) << 7)
    k8 = rng.integers(0x20, 0x48, (T, H, D)).astype(np.uint8)
    out = torch.empty((T, H, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((H, T), device="cuda")
    # q = 0: every key weighs the same (P = 2^4 exactly, no rounding anywhere before the output): the mean of V
    q0 = torch.zeros((T, H, D), dtype=torch.uint8, device="cuda")
    vd = torch.tensor([1.0, 0.25], device="cuda")
    api.sdvg_block_attn_fwd_e4m3(q0, codes_dev(k8), codes_dev(v8), cache, 0, ones, vd, out, lse, 0.3, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    mean_v = O.e4m3_decode(v8).mean(axis=0) * vd.cpu().numpy().reshape(H, 1)
    got = O.bf16_to_f64(to_bits(out))
    assert np.all(np.abs(got - mean_v[None]) <= np.abs(mean_v[None]) * 2.0 ** -8 + 1e-4)
    assert np.allclose(lse.cpu().numpy(), np.log(T), atol=1e-5)
    # one key dominates by far (its logit is 2^7 above the others after scaling): the output is that key's value
    kd = np.full((T, H, D), 0x00, dtype=np.uint8)
    kd[17] = 0x40                                            # 2.0 in every dim
    qd = np.full((T, H, D), 0x38, dtype=np.uint8)            # 1.0 in every dim: logits 256 * scale for key 17, 0 elsewhere
    api.sdvg_block_attn_fwd_e4m3(codes_dev(qd), codes_dev(kd), codes_dev(v8), cache, 0, ones, ones, out, None, 0.5, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    want = O.e4m3_decode(v8[17])
    assert np.array_equal(O.bf16_to_f64(to_bits(out)), np.broadcast_to(want[None], (T, H, D)))
    cache.close()


def test_full_size_target_shape_sampled_rows():
    # 40 heads x d128, 4680 queries x 32760 keys: the launch configuration the bench times; rows sampled per head
    sh = synth.WAN_14B
    H = sh.heads
    cache = api.Cache(sh.slots, H, sh.block_tokens, sh.head_dim, e4m3=True)
    ws = api.attn_workspace()
    pool = synth.TensorPool(sh, 9)
    inv = np.full(H, 448 / 4.5, dtype=np.float32)
    sc = (1 / inv).astype(np.float64)
    ks, vs = [], []
    for b in range(sh.slots):
        k, v = pool.get(b, 0, synth.K), pool.get(b, 0, synth.V)
        flags = api.SDVG_FINAL if b < sh.slots - 1 else api.SDVG_STAGE
        api.sdvg_kv_commit_e4m3(cache, to_dev(k), to_dev(v), f32_dev(inv), f32_dev(inv), b, flags)
    b = sh.slots - 1
    q = pool.get(b, 0, synth.Q)
    dq8 = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
    api.sdvg_quant_e4m3(to_dev(q), f32_dev(inv), dq8)
    out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    api.sdvg_block_attn_fwd_e4m3(dq8, None, None, cache, b, f32_dev(sc * sc), f32_dev(sc), out, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    assert not torch.isnan(out.float()).any()
    for s in range(sh.slots):
        gk, gv = cache.read_block(s)
        ks.append(gk.cpu().numpy())
        vs.append(gv.cpu().numpy())
    k_all, v_all, q8 = np.concatenate(ks), np.concatenate(vs), dq8.cpu().numpy()
    rng = np.random.default_rng(0)
    for h in (0, 13, 39):
        rows = np.sort(rng.choice(sh.block_tokens, 24, replace=False))
        rows[-1] = sh.block_tokens - 1
        assert np.array_equal(ks[3][:, h], O.quant_e4m3_ref(pool.get(3, 0, synth.K), inv)[:, h])   # ring holds the oracle's codes
        o_ref, _ = O.attn_e4m3_ref(q8, k_all, v_all, sc * sc, sc, sh.scale, heads=[h], rows=rows)
        bound = p_rounding_bound(q8, k_all, v_all, sc * sc, sc, sh.scale, [h], rows)
        check_attention(out[rows, h], o_ref[:, 0], bound[:, 0], ("14b", h))
    cache.close()


def test_fused_rope_quantise_stage_is_bit_identical_to_the_separate_calls_and_the_oracle():
    sh = synth.Shape("e4m3-prologue", heads=5, head_dim=128, frames=2, grid_h=6, grid_w=11, slots=3)
    grid = (sh.frames, sh.grid_h, sh.grid_w)
    tabf = 4 * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    ref_tab = O.rope_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w)
    fused = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    apart = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    rng = np.random.default_rng(4)
    q_inv, k_inv, v_inv = (rng.uniform(20, 120, sh.heads).astype(np.float32) for _ in range(3))
    for b in range(4):
        q, k, v = (synth.block_tensor(sh, 21, b, 0, t, std=1.5) for t in (synth.Q, synth.K, synth.V))
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        for flags in (api.SDVG_STAGE, api.SDVG_FINAL):
            q8 = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
            ev = api.sdvg_rope3d_qk_commit_e4m3(fused, dq, dk, dv, q8, f32_dev(q_inv), f32_dev(k_inv), f32_dev(v_inv), grid,
                                                b * sh.frames, tab, tabf, b, flags)
            # the same in three calls
            q_r, k_r = torch.empty_like(dq), torch.empty_like(dk)
            api.sdvg_rope3d_qk(dq, dk, q_r, k_r, grid, b * sh.frames, tab, tabf)
            q8b = torch.zeros_like(q8)
            api.sdvg_quant_e4m3(q_r, f32_dev(q_inv), q8b)
            ev2 = api.sdvg_kv_commit_e4m3(apart, k_r, dv, f32_dev(k_inv), f32_dev(v_inv), b, flags)
            assert ev == ev2 and fused.state() == apart.state()
            assert torch.equal(q8, q8b)
            fk, fv = fused.read_block(b % sh.slots)
            ak, av = apart.read_block(b % sh.slots)
            assert torch.equal(fk, ak) and torch.equal(fv, av)
            # and the oracle: bit-specified rotation rounded to bf16, then the quantiser
            qr = O.rope_bitspec(q, grid, b * sh.frames, ref_tab, tabf)
            kr = O.rope_bitspec(k, grid, b * sh.frames, ref_tab, tabf)
            assert np.array_equal(q8.cpu().numpy(), O.quant_e4m3_ref(qr, q_inv))
            assert np.array_equal(fk.cpu().numpy(), O.quant_e4m3_ref(kr, k_inv))
            assert np.array_equal(fv.cpu().numpy(), O.quant_e4m3_ref(v, v_inv))
    # k and v alone (no q), and a bf16 ring is refused
    api.sdvg_rope3d_qk_commit_e4m3(fused, None, dk, dv, None, None, f32_dev(k_inv), f32_dev(v_inv), grid, 0, tab, tabf, 4,
                                   api.SDVG_STAGE)
    bf = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_rope3d_qk_commit_e4m3(bf, None, dk, dv, None, None, f32_dev(k_inv), f32_dev(v_inv), grid, 0, tab, tabf, 0,
                                       api.SDVG_STAGE)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE


def test_schedule_with_8bit_rings_follows_the_flow_and_holds_the_oracle_codes():
    from paper_2604_17397_b200 import schedule
    from test_gpu_schedule import Provider

    sh_d = synth.Shape("d8", heads=3, head_dim=128, frames=3, grid_h=4, grid_w=13, slots=3)
    sh_t = synth.Shape("t8", heads=5, head_dim=128, frames=3, grid_h=4, grid_w=13, slots=4)
    B, steps, tau, seed = 9, 2, -0.7, 61
    tabf = B * sh_t.frames
    scores = synth.calibrated_scores(B, 12, seed)
    prov = Provider(sh_d, sh_t, seed)
    rng = np.random.default_rng(seed)
    models, inv = {}, {}
    for name, sh in (("drafter", sh_d), ("target", sh_t)):
        inv[name] = [rng.uniform(60, 110, sh.heads).astype(np.float32) for _ in range(3)]
        cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
        tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
        models[name] = schedule.ModelState(cache, (sh.frames, sh.grid_h, sh.grid_w), tab, tabf, sh.scale,
                                           q_inv_scale=f32_dev(inv[name][0]), k_inv_scale=f32_dev(inv[name][1]),
                                           v_inv_scale=f32_dev(inv[name][2]))
    shapes = {"drafter": sh_d, "target": sh_t}
    checked = []

    def on_attention(model, b, s, q8, out):
        if (b + s) % 3:
            return
        m, sh = models[model], shapes[model]
        # the window as the device ring holds it at this moment, the staged block included
        ks, vs = [], []
        for blk in range(max(0, b - (sh.slots - 1)), b + 1):
            gk, gv = m.cache.read_block(blk % sh.slots)
            ks.append(gk.cpu().numpy())
            vs.append(gv.cpu().numpy())
        k_all, v_all = np.concatenate(ks), np.concatenate(vs)
        r = np.random.default_rng([seed, b, s])
        heads = list(np.sort(r.choice(sh.heads, 2, replace=False)))
        rows = np.sort(r.choice(sh.block_tokens, 16, replace=False))
        qkd = 1.0 / (inv[model][0].astype(np.float64) * inv[model][1])
        vd = 1.0 / inv[model][2].astype(np.float64)
        q8n = q8.cpu().numpy()
        o_ref, _ = O.attn_e4m3_ref(q8n, k_all, v_all, qkd, vd, sh.scale, heads=heads, rows=rows)
        bound = p_rounding_bound(q8n, k_all, v_all, qkd, vd, sh.scale, heads, rows)
        got = out[torch.from_numpy(rows).cuda()][:, torch.tensor(heads).cuda()]
        check_attention(got, o_ref, bound, (model, b, s))
        checked.append((model, b, s))

    res = schedule.run_schedule(B, steps, torch.from_numpy(scores).cuda(), tau, models["drafter"], models["target"],
                                prov.device, on_attention=on_attention)
    for m in models.values():
        assert api.sdvg_block_attn_status(m.workspace) == api.SDVG_OK
    assert len(checked) >= 6 and {c[0] for c in checked} == {"drafter", "target"}

    # the flow (routing, branches, evictions, call counts) is that of the oracle's schedule; its bf16 rings,
    # quantised with the same scales, are what the 8-bit rings must hold
    rd = O.RingCacheRef(sh_d.slots, sh_d.heads, sh_d.block_tokens, sh_d.head_dim)
    rt = O.RingCacheRef(sh_t.slots, sh_t.heads, sh_t.block_tokens, sh_t.head_dim)
    want = O.schedule_ref(B, steps, scores, tau, rd, rt, prov.bits, (sh_d.frames, sh_d.grid_h, sh_d.grid_w),
                          (sh_t.frames, sh_t.grid_h, sh_t.grid_w), sh_t.frames,
                          O.rope_table(128, tabf, sh_d.grid_h, sh_d.grid_w), O.rope_table(128, tabf, sh_t.grid_h, sh_t.grid_w),
                          tabf)
    assert np.array_equal(res.accept, want.accept) and res.target_source == want.target_source
    assert 0 < int(want.accept.sum()) < B - 1
    assert res.drafter_evicted == want.drafter_evicted and res.target_evicted == want.target_evicted
    assert res.drafter_attn_calls == want.drafter_attn_calls and res.target_attn_calls == want.target_attn_calls
    for name, ref in (("drafter", rd), ("target", rt)):
        cache = models[name].cache
        assert cache.state()[:2] == (ref.next_block, ref.slot_block)
        for s in range(ref.slots):
            gk, gv = cache.read_block(s)
            assert np.array_equal(gk.cpu().numpy(), O.quant_e4m3_ref(ref.k[s], inv[name][1])), (name, s)
            assert np.array_equal(gv.cpu().numpy(), O.quant_e4m3_ref(ref.v[s], inv[name][2])), (name, s)
        cache.close()


def test_block_steps_of_an_8bit_ring_replayed_from_a_cuda_graph_equal_the_eager_calls():
    from paper_2604_17397_b200 import schedule

    sh = synth.Shape("graph8", heads=3, head_dim=128, frames=3, grid_h=6, grid_w=11, slots=3)
    tabf, steps = 4 * sh.frames, 3
    inv = [f32_dev(np.full(sh.heads, x, dtype=np.float32)) for x in (90.0, 100.0, 80.0)]
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim, e4m3=True)
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    m = schedule.ModelState(cache, (sh.frames, sh.grid_h, sh.grid_w), tab, tabf, sh.scale,
                            q_inv_scale=inv[0], k_inv_scale=inv[1], v_inv_scale=inv[2])
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


def test_batched_call_over_8bit_rings_equals_separate_calls():
    # two problems (the guidance pair) with their own rings and their own scales in one launch
    sh = synth.Shape("pair8", heads=3, head_dim=128, frames=1, grid_h=11, grid_w=29, slots=3)
    H = sh.heads
    ws = api.attn_workspace()
    caches = [api.Cache(sh.slots, H, sh.block_tokens, sh.head_dim, e4m3=True) for _ in range(2)]
    scales = [(4.5 / 448 * (1 + 0.1 * n + 0.05 * np.arange(H))).astype(np.float32) for n in range(2)]
    for b in range(4):
        q8s, outs_one, outs_sep, qkds, vds = [], [], [], [], []
        for n, c in enumerate(caches):
            q, k, v = (to_dev(synth.block_tensor(sh, 70 + n, b, 0, t)) for t in (synth.Q, synth.K, synth.V))
            inv = f32_dev(1 / scales[n])
            api.sdvg_kv_commit_e4m3(c, k, v, inv, inv, b, api.SDVG_STAGE)
            q8 = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
            api.sdvg_quant_e4m3(q, inv, q8)
            q8s.append(q8)
            qkds.append(f32_dev(scales[n] * scales[n]))
            vds.append(f32_dev(scales[n]))
            outs_one.append(torch.full_like(q, float("nan")))
            out = torch.full_like(q, float("nan"))
            api.sdvg_block_attn_fwd_e4m3(q8, None, None, c, b, qkds[n], vds[n], out, None, sh.scale, ws)
            outs_sep.append(out)
        api.sdvg_block_attn_fwd_e4m3_batched(q8s, None, None, caches, [b, b], qkds, vds, outs_one, None, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        for n in range(2):
            assert np.array_equal(to_bits(outs_one[n]), to_bits(outs_sep[n])), (b, n)
            inv = f32_dev(1 / scales[n])
            k, v = (to_dev(synth.block_tensor(sh, 70 + n, b, 0, t)) for t in (synth.K, synth.V))
            api.sdvg_kv_commit_e4m3(caches[n], k, v, inv, inv, b, api.SDVG_FINAL)
    # the host checks every problem before the launch
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_attn_fwd_e4m3_batched(q8s, None, None, caches, [4, 9], qkds, vds, outs_one, None, sh.scale, ws)
    assert e.value.status == api.SDVG_ERR_BAD_STATE


def whole_path_error(q_std, heads=2, seed=81):
    """Relative rms error and cosine of the WHOLE 8-bit path (quantise q, k, v with one scale per head set 10% above
    the largest magnitude, 8-bit products, P rounded to E4M3) against the oracle's exact attention on the unquantised
    bf16 inputs; the bf16 kernel's figures on the same inputs beside it."""
    sh = synth.Shape("f8q", heads=heads, head_dim=128, frames=3, grid_h=30, grid_w=52, slots=3)     # 4680 queries x 14040 keys
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(sh.block_tokens, 96, replace=False))
    c8 = api.Cache(sh.slots, heads, sh.block_tokens, sh.head_dim, e4m3=True)
    c16 = api.Cache(sh.slots, heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    ks, vs = [], []
    for b in range(sh.slots):
        ks.append(synth.block_tensor(sh, seed, b, 0, synth.K))
        vs.append(synth.block_tensor(sh, seed, b, 0, synth.V))
    q = synth.block_tensor(sh, seed, sh.slots - 1, 0, synth.Q, std=q_std)
    k_all, v_all = np.concatenate(ks), np.concatenate(vs)

    def scale_of(x):
        return (np.abs(O.bf16_to_f64(x)).max(axis=(0, 2)) * 1.1 / 448).astype(np.float32)
    sq, sk, sv = scale_of(q), scale_of(k_all), scale_of(v_all)
    for b in range(sh.slots):
        flag = api.SDVG_FINAL if b < sh.slots - 1 else api.SDVG_STAGE
        api.sdvg_kv_commit_e4m3(c8, to_dev(ks[b]), to_dev(vs[b]), f32_dev(1 / sk), f32_dev(1 / sv), b, flag)
        api.sdvg_kv_commit(c16, to_dev(ks[b]), to_dev(vs[b]), b, flag)
    b = sh.slots - 1
    q8 = torch.zeros(q.shape, dtype=torch.uint8, device="cuda")
    api.sdvg_quant_e4m3(to_dev(q), f32_dev(1 / sq), q8)
    out8 = torch.full((sh.block_tokens, heads, sh.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    out16 = torch.full_like(out8, float("nan"))
    api.sdvg_block_attn_fwd_e4m3(q8, None, None, c8, b, f32_dev(sq * sk), f32_dev(sv), out8, None, sh.scale, ws)
    api.sdvg_block_attn_fwd(to_dev(q), None, None, c16, b, out16, None, sh.scale, ws)
    assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
    o_ref, _ = O.attn_ref(q, k_all, v_all, sh.scale, rows=rows)              # exact attention, unquantised inputs
    res = {}
    for name, out in (("e4m3", out8), ("bf16", out16)):
        got = O.bf16_to_f64(to_bits(out))[rows]
        d = got - o_ref
        res[name] = (float(np.sqrt((d ** 2).mean() / (o_ref ** 2).mean())),
                     float((got * o_ref).sum() / np.sqrt((got ** 2).sum() * (o_ref ** 2).sum())))
    c8.close()
    c16.close()
    return res


@pytest.mark.parametrize("q_std,rel_rms_max,cos_min", [(1.0, 0.07, 0.997), (3.0, 0.13, 0.991)])
def test_whole_8bit_path_against_exact_attention_on_the_unquantised_inputs(q_std, rel_rms_max, cos_min):
    # What the variant costs end to end on N(0, 1) data at the drafter's window (queries of unit variance, and three
    # times larger: peaked rows).  Measured 5.3% / 9.7% relative rms: the 3-bit mantissas of q, k, v and P perturb
    # every probability and value by a few percent and the perturbations do not average out relative to an output
    # that is itself a random-sign sum over the keys.  The bounds are set a little above those figures.
    res = whole_path_error(q_std)
    assert res["bf16"][0] <= 0.01 and res["bf16"][1] >= 0.9999, res
    assert res["e4m3"][0] <= rel_rms_max and res["e4m3"][1] >= cos_min, res
