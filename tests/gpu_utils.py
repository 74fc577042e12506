"""Helpers shared by the GPU parity tests: bf16 bit patterns <-> device tensors."""
import numpy as np
import torch


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def f32_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def attn_errors(got_bits: np.ndarray, ref: np.ndarray):
    """(max-abs, mean-abs, rms error relative to the reference rms)."""
    from oracle import sdvg_oracle as O
    g = O.bf16_to_f64(got_bits)
    d = np.abs(g - ref)
    return float(d.max()), float(d.mean()), float(np.sqrt((d ** 2).mean()) / max(1e-30, np.sqrt((ref ** 2).mean())))


# spec tolerances for bf16 attention outputs on unit-normal inputs
ATTN_MAX_ABS = 2e-2
ATTN_MEAN_ABS = 2e-3
# extra, relative check: bf16 rounding of P and O keeps the rms error within a few 2^-9
ATTN_REL_RMS = 2e-2


# ---- canaries: guard bytes around device outputs (the stand-in for a memory checker) -------------------
GUARD_BYTES = 256
GUARD_PATTERN = 0xA5


class Canaries:
    """Device outputs allocated between guard regions, and the padding around a cache's rings.

    ``new(shape, dtype, fill)`` returns a tensor that sits 256 bytes inside a larger buffer whose margins
    hold a byte pattern; ``watch_cache(cache)`` records the bytes the cache's raw buffers hold outside the
    two rings.  ``check()`` fails if any kernel has written outside what it was given.
    """

    def __init__(self):
        self.raws, self.ring_pads = [], []

    def new(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((GUARD_BYTES + n + GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8, device="cuda")
        t = raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)
        if fill is not None:
            t.fill_(fill)
        else:
            t.view(torch.uint8).zero_()
        self.raws.append((raw, n))
        return t

    def like(self, ref, fill=None):
        return self.new(tuple(ref.shape), ref.dtype, fill)

    def watch_cache(self, cache):
        for raw, ptr in ((cache._k_raw, cache.k_ptr), (cache._v_raw, cache.v_ptr)):
            lead = ptr - raw.data_ptr()
            used = raw.numel() - 1024
            raw[:lead].fill_(GUARD_PATTERN)
            raw[lead + used:].fill_(GUARD_PATTERN)
            self.ring_pads.append((raw, lead, used))

    def check(self):
        torch.cuda.synchronize()
        for raw, n in self.raws:
            assert bool((raw[:GUARD_BYTES] == GUARD_PATTERN).all()), "write before an output buffer"
            assert bool((raw[GUARD_BYTES + n:] == GUARD_PATTERN).all()), "write past an output buffer"
        for raw, lead, used in self.ring_pads:
            assert bool((raw[:lead] == GUARD_PATTERN).all()), "write before a ring"
            assert bool((raw[lead + used:] == GUARD_PATTERN).all()), "write past a ring"
