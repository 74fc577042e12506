"""GPU parity: routing variants of the ablation (Sec. 4.3, Table 2) and accept statistics, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from conftest import read_golden_rows

pytestmark = pytest.mark.gpu


def run_policy(scores, offsets, nb, fpb, first, bpv, tau, agg, signal, force, uniforms, p):
    s = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32).reshape(-1)).cuda()
    off = None if offsets is None else torch.from_numpy(np.asarray(offsets, dtype=np.int32)).cuda()
    u = None if uniforms is None else torch.from_numpy(np.ascontiguousarray(uniforms, dtype=np.float32)).cuda()
    acc = torch.full((nb,), 7, dtype=torch.uint8, device="cuda")
    ag = torch.full((nb,), 123.0, dtype=torch.float32, device="cuda")
    am = torch.full((nb,), -7, dtype=torch.int32, device="cuda")
    api.sdvg_route_policy(s, off, nb, fpb, first, bpv, tau, agg, signal, force, u, p, acc, ag, am)
    return acc, ag.cpu().numpy(), am.cpu().numpy()


def assert_same(got, ref):
    assert np.array_equal(got[0].cpu().numpy(), ref[0])
    # A NaN produced by arithmetic (inf - inf in a mean) has no prescribed sign or payload: x86 and the GPU differ.
    # Everything else, NaNs copied from the input by the minimum included, is compared bit for bit.
    made_nan = np.isnan(ref[1]) & (ref[2] < 0)
    assert np.array_equal(np.isnan(got[1]), np.isnan(ref[1]))
    assert np.array_equal(got[1].view(np.uint32)[~made_nan], ref[1].view(np.uint32)[~made_nan])
    assert np.array_equal(got[2], ref[2])


def test_hand_worked_policy_cases():
    for blk, bpv, tau, agg, sig, force, u, p, scores, accept, aggv in read_golden_rows("route_policy_cases.txt"):
        s = np.array([float(t) for t in scores.split()], dtype=np.float32)
        got = run_policy(s, None, 1, s.size, int(blk), int(bpv), float(tau),
                         api.SDVG_AGG_MEAN if agg == "mean" else api.SDVG_AGG_MIN,
                         api.SDVG_SIGNAL_RANDOM if sig == "random" else api.SDVG_SIGNAL_REWARD, bool(int(force)),
                         np.array([float(u)], dtype=np.float32), float(p))
        assert int(got[0].cpu()[0]) == int(accept), (blk, scores)
        want = np.float32(float(aggv))
        assert (np.isnan(want) and np.isnan(got[1][0])) or got[1][0] == want


@pytest.mark.parametrize("agg", [O.AGG_MIN, O.AGG_MEAN])
@pytest.mark.parametrize("signal,force", [(O.SIGNAL_REWARD, True), (O.SIGNAL_RANDOM, True), (O.SIGNAL_RANDOM, False)])
def test_paper_batch_1003_videos_of_9_blocks(agg, signal, force):
    # Table 2 workload: 1003 videos x 9 blocks, 9 decoded frames for a video's first block, 12 for the others
    counts = np.tile(np.array([9] + [12] * 8), 1003)
    flat, offs = synth.ragged_scores(counts, -0.5, 0.6, 23)
    nb = counts.size
    u = synth.uniform_scores(nb, 1, 0.0, 1.0, 24).reshape(-1)
    for tau in (-0.7, -0.2):
        ref = O.route_policy_ref(flat, offs, nb, 0, 0, tau, agg=agg, signal=signal, force_first=force,
                                 blocks_per_video=9, uniforms=u, accept_prob=0.7)
        got = run_policy(flat, offs, nb, 0, 0, 9, tau, agg, signal, force, u, 0.7)
        assert_same(got, ref)
        # accept statistics on the device against the oracle's count
        counts_d = torch.full((2,), -1, dtype=torch.int64, device="cuda")
        api.sdvg_accept_stats(got[0], nb, 0, 9, counts_d)
        assert tuple(counts_d.cpu().tolist()) == O.accept_stats_ref(ref[0], 0, 9)
        assert counts_d[1].item() == 1003 * 8


def test_special_values_fixed_frames_and_streaming_offset():
    rng = np.random.default_rng(5)
    s = synth.normal_scores(20000, 12, -0.5, 0.6, 25).copy()
    flat = s.reshape(-1)
    flat[rng.integers(0, flat.size, 80)] = np.nan
    flat[rng.integers(0, flat.size, 80)] = np.inf
    flat[rng.integers(0, flat.size, 80)] = -np.inf
    for first, bpv in ((0, 0), (4, 0), (13, 9)):
        for agg in (O.AGG_MIN, O.AGG_MEAN):
            ref = O.route_policy_ref(flat, None, 20000, 12, first, -0.6, agg=agg, blocks_per_video=bpv)
            assert_same(run_policy(flat, None, 20000, 12, first, bpv, -0.6, agg, O.SIGNAL_REWARD, True, None, 0.0), ref)
            counts_d = torch.zeros(2, dtype=torch.int64, device="cuda")
            acc = torch.from_numpy(ref[0]).cuda()
            api.sdvg_accept_stats(acc, 20000, first, bpv, counts_d)
            assert tuple(counts_d.cpu().tolist()) == O.accept_stats_ref(ref[0], first, bpv)


def test_default_router_is_the_min_reward_forced_policy():
    s = synth.calibrated_scores(4000, 12, 26)
    acc = torch.empty(4000, dtype=torch.uint8, device="cuda")
    qm = torch.empty(4000, dtype=torch.float32, device="cuda")
    am = torch.empty(4000, dtype=torch.int32, device="cuda")
    api.sdvg_route(torch.from_numpy(s.reshape(-1)).cuda(), None, 4000, 12, 0, -0.7, acc, qm, am)
    got = run_policy(s, None, 4000, 12, 0, 0, -0.7, O.AGG_MIN, O.SIGNAL_REWARD, True, None, 0.0)
    assert torch.equal(acc, got[0]) and np.array_equal(qm.cpu().numpy().view(np.uint32), got[1].view(np.uint32))
    assert np.array_equal(am.cpu().numpy(), got[2])


def test_argument_checks():
    s = torch.zeros(12, device="cuda")
    acc = torch.zeros(1, dtype=torch.uint8, device="cuda")
    ag = torch.zeros(1, device="cuda")
    for kw in (dict(agg=2), dict(signal=3), dict(signal=api.SDVG_SIGNAL_RANDOM), dict(bpv=-1)):
        with pytest.raises(api.SdvgError) as e:
            api.sdvg_route_policy(s, None, 1, 12, 0, kw.get("bpv", 0), -0.7, kw.get("agg", 0), kw.get("signal", 0), True,
                                  None, 0.5, acc, ag, None)
        assert e.value.status == api.SDVG_ERR_INVALID_ARG
    counts = torch.zeros(2, dtype=torch.int64, device="cuda")
    api.sdvg_accept_stats(acc, 0, 0, 0, counts)          # empty batch: counts cleared, nothing else
    assert counts.tolist() == [0, 0]
