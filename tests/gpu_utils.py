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
