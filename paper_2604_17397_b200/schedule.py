"""Per-block speculative schedule (Sec. 3 "Inference flow", Fig. 2) on the device.

Host glue only: it strings the library's entry points together in the order the
paper gives and takes the accept/reject branch on the host.  For every block b

  1. the drafter takes ``steps`` denoise steps; each step is one fused
     rope + stage call and one attention call against the drafter ring K^D;
  2. the drafter's final K/V of the block are committed to K^D unconditionally
     (the drafter always conditions on its own earlier outputs);
  3. the router scores the block (worst frame against tau, global block 0 is
     always rejected);
  4. accepted: the target-shaped K/V of the draft block are committed to the
     target ring K^T.  Rejected: the target takes ``steps`` steps of its own
     against K^T and commits the K/V of the regenerated block.

K^D and K^T are independent rings with their own shapes and window sizes.
The tensors of every call come from a ``provider`` callback, so the same
function drives synthetic traces and a real model.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Optional

import numpy as np
import torch

from . import api


@dataclass
class ModelState:
    """Everything one model (drafter or target) needs for its steps."""
    cache: api.Cache
    grid: tuple                    # (latent frames per block, grid rows, grid columns)
    table: torch.Tensor            # device (cos, sin) table built for tab_frames frame positions
    tab_frames: int
    scale: float
    workspace: torch.Tensor = None
    # 8-bit ring (cache.e4m3): static inverse scales per head, device fp32 [heads]; a ring with tile scales
    # (cache.tile_scales) chooses its scales itself and takes none
    q_inv_scale: torch.Tensor = None
    k_inv_scale: torch.Tensor = None
    v_inv_scale: torch.Tensor = None

    def __post_init__(self):
        if self.workspace is None:
            self.workspace = api.attn_workspace(device=self.table.device)
        shape = (self.cache.block_tokens, self.cache.heads, self.cache.head_dim)
        dev = self.table.device
        self.e4m3 = bool(getattr(self.cache, "e4m3", False))
        self.tiled = bool(getattr(self.cache, "tile_scales", False))
        if self.tiled:
            # scales of the roped queries of the current step, [heads][tiles], written by the fused prologue
            self.q_tile_scale = torch.ones((self.cache.heads, self.cache.tiles), dtype=torch.float32, device=dev)
        elif self.e4m3:
            if self.q_inv_scale is None or self.k_inv_scale is None or self.v_inv_scale is None:
                raise ValueError("an 8-bit ring with static scales needs q, k and v inverse scales")
            self.qk_descale = 1.0 / (self.q_inv_scale * self.k_inv_scale)
            self.v_descale = 1.0 / self.v_inv_scale
        # the roped queries of the current step: bf16, or E4M3 codes for an 8-bit ring
        self.q_roped = torch.empty(shape, dtype=torch.uint8 if self.e4m3 else torch.bfloat16, device=dev)
        self.out = torch.empty(shape, dtype=torch.bfloat16, device=dev)

    @property
    def frames(self) -> int:
        return self.grid[0]

    def new_q_roped(self) -> torch.Tensor:
        return torch.zeros_like(self.q_roped)

    def stage_and_attend(self, q, k, v, block: int, q_roped, out) -> None:
        """One denoise step of `block`: fused rope (+ quantise) + stage, then attention against the ring."""
        if self.tiled:
            api.sdvg_rope3d_qk_commit_e4m3_tiled(self.cache, q, k, v, q_roped, self.q_tile_scale, self.grid,
                                                 block * self.frames, self.table, self.tab_frames, block, api.SDVG_STAGE)
            api.sdvg_block_attn_fwd_e4m3_tiled(q_roped, self.q_tile_scale, self.cache, block, out, None, self.scale,
                                               self.workspace)
        elif self.e4m3:
            api.sdvg_rope3d_qk_commit_e4m3(self.cache, q, k, v, q_roped, self.q_inv_scale, self.k_inv_scale,
                                           self.v_inv_scale, self.grid, block * self.frames, self.table,
                                           self.tab_frames, block, api.SDVG_STAGE)
            api.sdvg_block_attn_fwd_e4m3(q_roped, None, None, self.cache, block, self.qk_descale, self.v_descale, out,
                                         None, self.scale, self.workspace)
        else:
            api.sdvg_rope3d_qk_commit(self.cache, q, k, v, q_roped, None, self.grid, block * self.frames, self.table,
                                      self.tab_frames, block, api.SDVG_STAGE)
            api.sdvg_block_attn_fwd(q_roped, None, None, self.cache, block, out, None, self.scale, self.workspace)

    def block_steps(self, qs, ks, vs, block: int, q_ropeds, outs) -> None:
        """All denoise steps of `block` in ONE library call (per step: fused rope (+ quantise) + stage, attention)."""
        if self.tiled:
            if getattr(self, "_step_scales", None) is None or len(self._step_scales) != len(qs):
                self._step_scales = [torch.ones_like(self.q_tile_scale) for _ in qs]
            api.sdvg_block_steps_e4m3_tiled(self.cache, qs, ks, vs, q_ropeds, self._step_scales, outs, self.grid,
                                            block * self.frames, self.table, self.tab_frames, block, self.scale,
                                            self.workspace)
        elif self.e4m3:
            api.sdvg_block_steps_e4m3(self.cache, qs, ks, vs, q_ropeds, outs, self.q_inv_scale, self.k_inv_scale,
                                      self.v_inv_scale, self.qk_descale, self.v_descale, self.grid, block * self.frames,
                                      self.table, self.tab_frames, block, self.scale, self.workspace)
        else:
            api.sdvg_block_steps(self.cache, qs, ks, vs, q_ropeds, outs, self.grid, block * self.frames, self.table,
                                 self.tab_frames, block, self.scale, self.workspace)

    def check_status(self, where: str) -> None:
        """Raise if an attention kernel of this model gave up on a bounded wait since the workspace was last reset
        (the status word is sticky, so one check covers every launch since then); synchronises the stream."""
        st = api.sdvg_block_attn_status(self.workspace)
        if st != api.SDVG_OK:
            raise api.SdvgError(st, where)

    def commit_final(self, k, v, block: int) -> int:
        """Rope the block's final K and write it with V into the ring (SDVG_FINAL); returns the evicted block."""
        if self.tiled:
            return api.sdvg_rope3d_qk_commit_e4m3_tiled(self.cache, None, k, v, None, None, self.grid,
                                                        block * self.frames, self.table, self.tab_frames, block,
                                                        api.SDVG_FINAL)
        if self.e4m3:
            return api.sdvg_rope3d_qk_commit_e4m3(self.cache, None, k, v, None, None, self.k_inv_scale, self.v_inv_scale,
                                                  self.grid, block * self.frames, self.table, self.tab_frames, block,
                                                  api.SDVG_FINAL)
        return api.sdvg_rope3d_qk_commit(self.cache, None, k, v, None, None, self.grid, block * self.frames, self.table,
                                         self.tab_frames, block, api.SDVG_FINAL)


@dataclass
class TraceResult:
    accept: np.ndarray
    q_min: np.ndarray
    drafter_evicted: list = field(default_factory=list)
    target_evicted: list = field(default_factory=list)
    drafter_attn_calls: int = 0
    target_attn_calls: int = 0
    target_source: list = field(default_factory=list)     # per block: "accepted" or "regenerated"


def _denoise(model: str, m: ModelState, block: int, steps: int, provider, on_attention) -> int:
    for s in range(steps):
        q, k, v = provider(model, block, "step", s)
        m.stage_and_attend(q, k, v, block, m.q_roped, m.out)
        if on_attention is not None:
            on_attention(model, block, s, m.q_roped, m.out)
    return steps


def _commit_clean(m: ModelState, block: int, k, v) -> int:
    return m.commit_final(k, v, block)


def run_schedule(num_blocks: int, steps: int, scores: torch.Tensor, tau: float,
                 drafter: ModelState, target: ModelState,
                 provider: Callable, first_block_index: int = 0,
                 on_attention: Optional[Callable] = None) -> TraceResult:
    """Generate ``num_blocks`` blocks with the drafter/router/target flow.

    scores    device fp32 [num_blocks, frames]: the per-frame reward of every draft block
              (in a real system they appear one block at a time; routing here is also
              done one block at a time, with the block's global index)
    provider  ``provider(model, block, kind, step)`` -> (q, k, v) device bf16 tensors of the
              model's shape; kind is "step" (one denoise step), "clean" (the model's final
              K/V, q is None) or "accepted" (target-shaped K/V of an accepted draft block)
    on_attention  optional ``f(model, block, step, q_roped, out)`` called after each
              attention launch (the tensors are reused by the next step; q_roped holds E4M3
              codes when the model's ring is an 8-bit one)
    A model whose ``cache`` is an 8-bit ring takes every step through the _e4m3 entry points.
    The accept decision is read back to the host once per block, which is the only
    synchronisation point of the flow.
    """
    if scores.dtype != torch.float32 or scores.dim() != 2 or scores.shape[0] != num_blocks:
        raise ValueError("scores must be float32 [num_blocks, frames]")
    frames = scores.shape[1]
    dev = scores.device
    accept_d = torch.zeros(num_blocks, dtype=torch.uint8, device=dev)
    qmin_d = torch.zeros(num_blocks, dtype=torch.float32, device=dev)
    res = TraceResult(accept=np.zeros(num_blocks, dtype=np.uint8), q_min=np.zeros(num_blocks, dtype=np.float32))
    flat = scores.reshape(-1)
    for i in range(num_blocks):
        b = first_block_index + i
        res.drafter_attn_calls += _denoise("drafter", drafter, b, steps, provider, on_attention)
        api.sdvg_route(flat[i * frames:(i + 1) * frames], None, 1, frames, b, tau, accept_d[i:i + 1],
                       qmin_d[i:i + 1], None)
        accepted = bool(accept_d[i].item())               # the flow's one synchronisation point per block
        # a kernel that gave up leaves undefined outputs: stop before anything derived from them enters a ring
        drafter.check_status(f"drafter steps of block {b}")
        _, k, v = provider("drafter", b, "clean", 0)
        res.drafter_evicted.append(_commit_clean(drafter, b, k, v))
        if accepted:
            _, k, v = provider("target", b, "accepted", 0)
            res.target_source.append("accepted")
        else:
            res.target_attn_calls += _denoise("target", target, b, steps, provider, on_attention)
            target.check_status(f"target steps of block {b}")
            _, k, v = provider("target", b, "clean", 0)
            res.target_source.append("regenerated")
        res.target_evicted.append(_commit_clean(target, b, k, v))
    res.accept = accept_d.cpu().numpy()
    res.q_min = qmin_d.cpu().numpy()
    return res


class BlockStepGraph:
    """The S denoising steps of ONE block captured into a CUDA graph (Sec. 4.1: 4 steps per block).

    The capture holds ONE library call (sdvg_block_steps: per step the fused rope + stage kernel followed
    by the attention kernel), reading q, k, v from fixed input tensors (``self.q[s]``, ``self.k[s]``,
    ``self.v[s]``: fill them before ``replay``) and writing ``self.out[s]``.  The ring state does not change inside the loop (SDVG_STAGE leaves it
    alone), so the captured launches stay valid until the block's final commit; a new block needs a
    new capture because its ring slot, frame offset and key segments differ.  One eager pass runs
    first: the library's one-time set-up (kernel attributes, device queries) must not happen during
    capture.
    """

    def __init__(self, m: ModelState, block: int, steps: int):
        shape = (m.cache.block_tokens, m.cache.heads, m.cache.head_dim)
        dev = m.table.device
        new = lambda: torch.zeros(shape, dtype=torch.bfloat16, device=dev)
        self.q, self.k, self.v = ([new() for _ in range(steps)] for _ in range(3))
        self.q_roped = [m.new_q_roped() for _ in range(steps)]
        self.out = [new() for _ in range(steps)]
        self.m, self.block, self.steps = m, block, steps
        self._run()                                   # warm-up, eager
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self._run()

    def _run(self):
        self.m.block_steps(self.q, self.k, self.v, self.block, self.q_roped, self.out)

    def replay(self):
        self.graph.replay()
