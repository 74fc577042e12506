"""GPU parity: snapshot / restore of decoder state (Sec. 3: cache cloned before scoring, restored on rejection)."""
import numpy as np
import pytest
import torch

from paper_2604_17397_b200 import api

pytestmark = pytest.mark.gpu


def make_state(rng, sizes):
    """Feature maps of odd sizes (multiples of 16 bytes), as a causal video decoder keeps between blocks."""
    return [torch.from_numpy(rng.integers(0, 65536, size=n, dtype=np.uint16).view(np.int16)).cuda() for n in sizes]


def test_snapshot_then_restore_brings_back_every_bit():
    rng = np.random.default_rng(7)
    sizes = [8, 8 * 3, 8 * 1001, 8 * 65537, 8 * 12345, 8, 8 * 999999]      # int16 elements
    state = make_state(rng, sizes)
    want = [t.cpu().numpy().copy() for t in state]                          # the definition: a copy
    snap = [torch.full_like(t, -1) for t in state]
    api.sdvg_state_copy(state, snap)
    for t in state:                                                         # the draft block's decode mutates the state
        t.add_(1)
    assert all(not np.array_equal(t.cpu().numpy(), w) for t, w in zip(state, want))
    assert all(np.array_equal(s.cpu().numpy(), w) for s, w in zip(snap, want))
    api.sdvg_state_copy(snap, state)                                        # rejected: roll back
    assert all(np.array_equal(t.cpu().numpy(), w) for t, w in zip(state, want))


def test_neighbours_are_untouched_and_arguments_are_checked():
    rng = np.random.default_rng(8)
    big = torch.from_numpy(rng.integers(0, 255, size=4096, dtype=np.uint8)).cuda()
    dst = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    api.sdvg_state_copy([big[1024:2048]], [dst[2048:3072]])
    got = dst.cpu().numpy()
    assert np.array_equal(got[2048:3072], big.cpu().numpy()[1024:2048])
    assert not got[:2048].any() and not got[3072:].any()
    api.sdvg_state_copy([], [])                                             # empty state: nothing to do
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_state_copy([big[:24]], [dst[:24]])                         # 24 bytes: not a multiple of 16
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_state_copy([big[8:40]], [dst[:32]])                        # source not 16-byte aligned
    assert e.value.status == api.SDVG_ERR_MISALIGNED
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_state_copy([big[:16]] * 65, [dst[:16]] * 65)
    assert e.value.status == api.SDVG_ERR_BAD_SHAPE


def test_copy_rate_of_a_decoder_sized_state():
    # 1 GB in 32 buffers: must run near the copy bandwidth (a loose floor, the bench reports the figure)
    state = [torch.empty(32 * 1024 * 1024, dtype=torch.uint8, device="cuda") for _ in range(32)]
    snap = [torch.empty_like(t) for t in state]
    api.sdvg_state_copy(state, snap)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        api.sdvg_state_copy(state, snap)
    e1.record()
    torch.cuda.synchronize()
    gbs = 5 * 2 * 32 * 32 * 1024 * 1024 / (e0.elapsed_time(e1) * 1e-3) / 1e9
    print("state copy GB/s (read + write):", gbs)
    assert gbs > 3000
