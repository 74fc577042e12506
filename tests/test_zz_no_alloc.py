"""The allocation-free attention entry point must agree with the ordinary one.

Some users of the library cannot call cudaMalloc at the point where they need attention (all of
HBM already belongs to their own arena, or they sit inside a capture or a callback where an
allocation would stall the device), so they cannot supply the workspace buffer.  For them
sdvg_block_attn_fwd_noalloc keeps its scratch inside the library image.  This file is named so
that pytest collects it last: a run that stops at the first failure has then already run every
other test.  It also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2604_17397_b200 import api, synth
from gpu_utils import ATTN_MAX_ABS, ATTN_MEAN_ABS, to_bits, to_dev
from oracle import sdvg_oracle as O

pytestmark = pytest.mark.gpu


def test_noalloc_entry_point_matches_workspace_entry_point_twice_in_a_row():
    sh = synth.Shape("noalloc", heads=3, head_dim=128, frames=2, grid_h=5, grid_w=23, slots=3)
    cache = api.Cache(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ref = O.RingCacheRef(sh.slots, sh.heads, sh.block_tokens, sh.head_dim)
    ws = api.attn_workspace()
    addresses = []
    for b in range(2):                              # two calls in a row share the built-in scratch
        q, k, v = (synth.block_tensor(sh, 77, b, 0, t) for t in (synth.Q, synth.K, synth.V))
        dq, dk, dv = to_dev(q), to_dev(k), to_dev(v)
        want = torch.full_like(dq, float("nan"))
        got = torch.full_like(dq, float("nan"))
        lse_want = torch.empty((sh.heads, sh.block_tokens), device="cuda")
        lse_got = torch.empty_like(lse_want)
        api.sdvg_block_attn_fwd(dq, dk, dv, cache, b, want, lse_want, sh.scale, ws)
        assert api.sdvg_block_attn_status(ws) == api.SDVG_OK
        scratch = api.sdvg_block_attn_fwd_noalloc(dq, dk, dv, cache, b, got, lse_got, sh.scale)
        assert scratch != 0 and api.sdvg_block_attn_status(scratch) == api.SDVG_OK
        addresses.append(scratch)
        # the same kernel on the same inputs, only the scratch differs: the results agree to the bit
        assert np.array_equal(to_bits(got), to_bits(want))
        assert torch.equal(lse_got, lse_want)
        # and both are the attention the oracle defines
        o_ref, lse_ref = O.block_attn_ref(q, k, v, ref, b, sh.scale)
        d = np.abs(O.bf16_to_f64(to_bits(got)) - o_ref)
        assert d.max() <= ATTN_MAX_ABS and d.mean() <= ATTN_MEAN_ABS
        assert np.allclose(lse_got.cpu().numpy(), lse_ref, rtol=2e-4, atol=2e-3)
        api.sdvg_kv_commit(cache, dk, dv, b, api.SDVG_FINAL)
        ref.commit(b, k, v, O.FINAL)
    assert addresses[0] == addresses[1]             # one array per device, found once
    # host-side refusals are the same as for the ordinary entry point
    with pytest.raises(api.SdvgError) as e:
        api.sdvg_block_attn_fwd_noalloc(dq, dk, dv, cache, 7, got, None, sh.scale)
    assert e.value.status == api.SDVG_ERR_BAD_STATE
    cache.close()
