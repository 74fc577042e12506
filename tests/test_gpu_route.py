"""GPU parity: sdvg_route against the oracle, bit-exact (accept, q_min bits, argmin)."""
import numpy as np
import pytest
import torch

from oracle import sdvg_oracle as O
from paper_2604_17397_b200 import api, synth
from conftest import read_golden_rows
from gpu_utils import Canaries

pytestmark = pytest.mark.gpu


def run_route(scores, offsets, nb, fpb, first, tau, want_argmin=True):
    s = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32).reshape(-1)).cuda()
    off = None if offsets is None else torch.from_numpy(np.asarray(offsets, dtype=np.int32)).cuda()
    guard = Canaries()                       # guard bytes around the three outputs
    acc = guard.new((nb,), torch.uint8, 7)
    qm = guard.new((nb,), torch.float32, 123.0)
    am = guard.new((nb,), torch.int32, -7) if want_argmin else None
    api.sdvg_route(s, off, nb, fpb, first, tau, acc, qm, am)
    guard.check()
    return acc.cpu().numpy(), qm.cpu().numpy(), None if am is None else am.cpu().numpy()


def assert_same(got, ref):
    ga, gq, gi = got
    ra, rq, ri = ref
    assert np.array_equal(ga, ra)
    assert np.array_equal(gq.view(np.uint32), rq.view(np.uint32))
    if gi is not None:
        assert np.array_equal(gi, ri)


def test_hand_worked_cases():
    for blk, tau, scores, accept, qmin, argmin in read_golden_rows("route_cases.txt"):
        s = np.array([float(t) for t in scores.split()], dtype=np.float32)
        ga, gq, gi = run_route(s, None, 1, s.size, int(blk), float(tau))
        assert int(ga[0]) == int(accept)
        assert int(gi[0]) == int(argmin)
        want = np.float32(float(qmin))
        assert (np.isnan(want) and np.isnan(gq[0])) or gq[0] == want


def test_config1_tiny_router():
    s = synth.uniform_scores(3, 8, -2.0, 1.0, 0)
    assert_same(run_route(s, None, 3, 8, 0, -0.7), O.route_ref(s.reshape(-1), None, 3, 8, 0, -0.7))


def test_config5_trace_scores_three_taus():
    s = synth.normal_scores(16, 12, -0.5, 0.6, 5)
    c = synth.calibrated_scores(16, 12, 5, 1)
    for tau in (-0.9, -0.7, -0.5):
        assert_same(run_route(s, None, 16, 12, 0, tau), O.route_ref(s.reshape(-1), None, 16, 12, 0, tau))
        assert_same(run_route(c, None, 16, 12, 0, tau), O.route_ref(c.reshape(-1), None, 16, 12, 0, tau))


def test_paper_workload_shape_ragged_9_then_12():
    # 1003 videos x 9 blocks; 9 decoded frames for the first block of a video, 12 for the others
    counts = np.tile(np.array([9] + [12] * 8), 1003)
    flat, offs = synth.ragged_scores(counts, -0.5, 0.6, 17)
    nb = counts.size
    ref = O.route_ref(flat, offs, nb, 0, 0, -0.7)
    assert_same(run_route(flat, offs, nb, 0, 0, -0.7), ref)
    assert ref[0][0] == 0


def test_ragged_odd_lengths_special_values_and_streaming_offset():
    rng = np.random.default_rng(3)
    counts = rng.integers(1, 41, size=5000)
    flat, offs = synth.ragged_scores(counts, -0.5, 0.6, 18)
    flat = flat.copy()
    flat[rng.integers(0, flat.size, 60)] = np.nan
    flat[rng.integers(0, flat.size, 60)] = -np.inf
    flat[rng.integers(0, flat.size, 60)] = np.inf
    flat[rng.integers(0, flat.size, 200)] = 0.0
    flat[rng.integers(0, flat.size, 200)] = -0.0
    for first in (0, 3):
        ref = O.route_ref(flat, offs, counts.size, 0, first, -0.7)
        assert_same(run_route(flat, offs, counts.size, 0, first, -0.7), ref)
    # scores starting at an address that is not 16-byte aligned (sub-view of a larger buffer)
    s = torch.from_numpy(np.concatenate([[0.0], flat]).astype(np.float32)).cuda()[1:]
    off = torch.from_numpy(offs).cuda()
    acc = torch.empty(counts.size, dtype=torch.uint8, device="cuda")
    qm = torch.empty(counts.size, dtype=torch.float32, device="cuda")
    api.sdvg_route(s, off, counts.size, 0, 0, -0.7, acc, qm, None)
    ref = O.route_ref(flat, offs, counts.size, 0, 0, -0.7)
    assert np.array_equal(acc.cpu().numpy(), ref[0])
    assert np.array_equal(qm.cpu().numpy().view(np.uint32), ref[1].view(np.uint32))


def test_long_blocks_take_the_unstaged_path_and_empty_block_is_rejected():
    counts = [3, 20000, 5, 9000, 1]
    flat, offs = synth.ragged_scores(counts, 0.0, 1.0, 19)
    assert_same(run_route(flat, offs, 5, 0, 0, -4.5), O.route_ref(flat, offs, 5, 0, 0, -4.5))
    offs2 = np.array([0, 4, 4, 9], dtype=np.int32)       # block 1 owns no frame
    ga, gq, gi = run_route(flat[:9], offs2, 3, 0, 5, -10.0)
    assert ga.tolist() == [1, 0, 1] and np.isnan(gq[1]) and gi[1] == -1


def test_bandwidth_sized_batch_fixed_frames():
    nb = 1 << 18
    s = synth.normal_scores(nb, 12, -0.5, 0.6, 20)
    ga, gq, gi = run_route(s, None, nb, 12, 0, -0.7)
    assert np.array_equal(gq, s.min(axis=1))
    assert np.array_equal(gi, s.argmin(axis=1).astype(np.int32))
    want = (s.min(axis=1) >= np.float32(-0.7)).astype(np.uint8)
    want[0] = 0
    assert np.array_equal(ga, want)
    # spot-check against the oracle proper on a slice that spans several tiles
    ref = O.route_ref(s[:3000].reshape(-1), None, 3000, 12, 0, -0.7)
    assert np.array_equal(ga[:3000], ref[0]) and np.array_equal(gi[:3000], ref[2])


def test_malformed_offsets_read_nothing_out_of_range():
    # Offsets live on the device, so the kernel guards itself: a block whose range runs backwards or leaves
    # [offsets[0], offsets[B]) counts as a block without frames; a block that merely sits outside its tile's
    # range (offsets not sorted) is still read where it is.  Same answers as the oracle's reading.
    for row in read_golden_rows("route_malformed_cases.txt"):
        offsets, scores, tau, accept, qmin, argmin = row
        offs = np.array([int(t) for t in offsets.split()], dtype=np.int32)
        s = np.array([float(t) for t in scores.split()], dtype=np.float32)
        nb = offs.size - 1
        got = run_route(s, offs, nb, 0, 1, float(tau))
        ref = O.route_ref(s, offs, nb, 0, 1, float(tau))
        want_acc = np.array([int(t) for t in accept.split()], dtype=np.uint8)
        want_arg = np.array([int(t) for t in argmin.split()], dtype=np.int32)
        want_q = np.array([float(t) for t in qmin.split()], dtype=np.float32)
        for have in (got, ref):
            assert np.array_equal(have[0], want_acc) and np.array_equal(have[2], want_arg)
            assert np.array_equal(np.isnan(have[1]), np.isnan(want_q))
            assert np.array_equal(have[1][~np.isnan(want_q)], want_q[~np.isnan(want_q)])
    # a long, shuffled offset array: many tiles, most blocks outside their tile's range
    rng = np.random.default_rng(5)
    nb, f = 3000, 7
    s = synth.normal_scores(nb, f, -0.5, 0.6, 6).reshape(-1)
    starts = rng.permutation(nb).astype(np.int32) * f
    offs = np.concatenate([[0], starts[1:], [nb * f]]).astype(np.int32)      # ends fixed, interior shuffled
    got = run_route(s, offs, nb, 0, 1, -0.7)
    ref = O.route_ref(s, offs, nb, 0, 1, -0.7)
    assert np.array_equal(got[0], ref[0]) and np.array_equal(got[2], ref[2])
    assert np.array_equal(got[1].view(np.uint32)[~np.isnan(ref[1])], ref[1].view(np.uint32)[~np.isnan(ref[1])])
    assert np.array_equal(np.isnan(got[1]), np.isnan(ref[1]))


@pytest.mark.parametrize("frames", [4, 8, 12, 16, 20])
def test_vector_path_special_values_at_every_position(frames):
    # fixed frame counts that are multiples of four take the 16-byte vector path: NaN, +-Inf, ties and signed zeros
    # at every frame position must resolve exactly as the sequential left-to-right definition does
    rng = np.random.default_rng(frames)
    nb = 4 * frames * 6 + 37
    s = synth.normal_scores(nb, frames, -0.5, 0.6, 30 + frames)
    specials = [np.nan, np.inf, -np.inf, -0.0, 0.0, -0.7]
    b = 1
    for pos in range(frames):
        for v in specials:
            s[b, pos] = v
            if pos + 1 < frames and v == v:
                s[b, pos + 1] = v                      # a tie right behind it
            b += 1
    for tau in (-0.7, 0.0):
        assert_same(run_route(s, None, nb, frames, 0, tau), O.route_ref(s.reshape(-1), None, nb, frames, 0, tau))
    # the same scores shifted by one float: no longer 16-byte aligned, so the staged path runs; same answers
    flat = np.concatenate([[0.0], s.reshape(-1)]).astype(np.float32)
    d = torch.from_numpy(flat).cuda()[1:]
    acc = torch.empty(nb, dtype=torch.uint8, device="cuda")
    qm = torch.empty(nb, dtype=torch.float32, device="cuda")
    am = torch.empty(nb, dtype=torch.int32, device="cuda")
    api.sdvg_route(d, None, nb, frames, 0, -0.7, acc, qm, am)
    assert_same((acc.cpu().numpy(), qm.cpu().numpy(), am.cpu().numpy()), O.route_ref(s.reshape(-1), None, nb, frames, 0, -0.7))
