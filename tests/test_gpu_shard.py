"""Head sharding needs no exchange step: running the heads `shard_heads(H, N, r)` through rope + stage ->
attention -> commit on a cache that holds H / N heads reproduces those heads of the unsharded run.

The N ranks of a head-sharded deployment are emulated one after the other on one GPU (they never wait on
one another, so nothing has to run at the same time).  Rope outputs and ring contents are bit-identical by
construction.  The attention output of a query tile depends on how the tile was scheduled: a tile that runs
in a pair visits the keys in one pass, a tile that runs alone has its keys split between the CTA's two lanes
and merged at the end.  With few tiles every tile runs alone in both the sharded and the unsharded launch,
and the outputs are bit-identical as well; at the full target shape the unsharded launch runs pairs and an
8-way shard runs single tiles, and the outputs agree to rounding.
"""
import numpy as np
import pytest
import torch

from paper_2604_17397_b200 import api, dist_util, synth
from gpu_utils import to_bits, to_dev

pytestmark = pytest.mark.gpu


class Replica:
    """One rank's state: a cache of its own heads, the rope table and a workspace."""

    def __init__(self, sh, heads):
        self.sh, self.heads = sh, heads
        self.cache = api.Cache(sh.slots, len(heads), sh.block_tokens, sh.head_dim)
        self.ws = api.attn_workspace()

    def take(self, t):
        """This rank's heads of a full [tokens, heads, dim] tensor, as its own contiguous tensor."""
        return t[:, self.heads.start:self.heads.stop, :].contiguous()

    def step(self, q, k, v, b, tab, tabf):
        sh = self.sh
        grid = (sh.frames, sh.grid_h, sh.grid_w)
        q, k, v = self.take(q), self.take(k), self.take(v)
        q_r, k_r, out = torch.empty_like(q), torch.empty_like(k), torch.full_like(q, float("nan"))
        api.sdvg_rope3d_qk_commit(self.cache, q, k, v, q_r, k_r, grid, b * sh.frames, tab, tabf, b, api.SDVG_STAGE)
        api.sdvg_block_attn_fwd(q_r, None, None, self.cache, b, out, None, sh.scale, self.ws)
        ev = api.sdvg_kv_commit(self.cache, k_r, v, b, api.SDVG_FINAL)
        return q_r, out, ev

    def ring(self):
        """All slots of this rank's ring as logical tensors."""
        return [self.cache.read_block(s) for s in range(self.sh.slots)]


def run(sh, world, blocks, seed):
    """Unsharded run and `world` sharded runs over the same inputs; yields per block what both produced."""
    tabf = blocks * sh.frames
    tab = api.sdvg_rope3d_table(sh.head_dim, tabf, sh.grid_h, sh.grid_w).cuda()
    full = Replica(sh, range(0, sh.heads))
    ranks = [Replica(sh, dist_util.shard_heads(sh.heads, world, r)) for r in range(world)]
    for b in range(blocks):
        q, k, v = (to_dev(synth.block_tensor(sh, seed, b, 0, t)) for t in (synth.Q, synth.K, synth.V))
        fq, fout, fev = full.step(q, k, v, b, tab, tabf)
        assert api.sdvg_block_attn_status(full.ws) == api.SDVG_OK
        for r in ranks:
            rq, rout, rev = r.step(q, k, v, b, tab, tabf)
            assert api.sdvg_block_attn_status(r.ws) == api.SDVG_OK
            assert rev == fev
            yield b, r, r.take(fq), rq, r.take(fout), rout
    # the rings: every slot of every rank equals its heads of the unsharded ring, K and V, to the bit
    fring = full.ring()
    committed = [blk >= 0 for blk in full.cache.state()[1]]       # slots never written hold no defined bits
    for r in ranks:
        assert r.cache.state() == full.cache.state()
        for used, (fk, fv), (rk, rv) in zip(committed, fring, r.ring()):
            if used:
                assert torch.equal(r.take(fk), rk) and torch.equal(r.take(fv), rv)


@pytest.mark.parametrize("world", [2, 4, 8])
def test_head_shards_reproduce_the_unsharded_run_bit_for_bit(world):
    # 8 heads x 4 query tiles: at most 32 tiles per launch, so every tile runs alone in every launch
    sh = synth.Shape("shard", heads=8, head_dim=128, frames=2, grid_h=16, grid_w=16, slots=3)
    for b, r, fq, rq, fout, rout in run(sh, world, blocks=5, seed=41):
        assert torch.equal(fq, rq), (b, r.heads)
        assert np.array_equal(to_bits(fout), to_bits(rout)), (b, r.heads)


def test_head_shards_at_the_target_shape_agree_to_rounding():
    # 40 heads x 37 query tiles: the unsharded launch runs 740 pairs, an 8-way shard 185 single tiles
    sh = synth.WAN_14B
    for b, r, fq, rq, fout, rout in run(sh, 8, blocks=2, seed=43):
        assert torch.equal(fq, rq), (b, r.heads)
        d = (fout.float() - rout.float()).abs()
        scale = fout.float().abs().max().item()
        assert d.max().item() <= 2.0 ** -6 * scale and d.mean().item() <= 2.0 ** -9 * scale, (b, r.heads, d.max().item(), scale)
