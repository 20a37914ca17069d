"""Shared test utilities: tensor <-> numpy bit views, and the level table of a normal-float format built from its
published construction (an input of the 3-bit export, not part of the method's arithmetic)."""
import numpy as np
import scipy.stats
import torch


def f16_bits(t: torch.Tensor) -> np.ndarray:
    """fp16 tensor -> uint16 numpy array of its bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f16_tensor(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.float16)


def normal_float_table(bits=3):
    """Normalized levels of an asymmetric normal-float format, built from its published construction: equally
    spaced probabilities between an offset and 1/2 are sent through the normal quantile function, 2^(bits-1) of
    them on the positive side and 2^(bits-1) - 1 on the negative side, zero added, the lot divided by the
    largest. Returns (table float32 [2^bits] ascending, index of zero)."""
    half = 2 ** (bits - 1)
    offset = 0.5 * ((1 - 1 / (2 * (2 * half - 1))) + (1 - 1 / (2 * 2 * half)))
    pos = scipy.stats.norm.ppf(np.linspace(offset, 0.5, half + 1)[:-1])
    neg = -scipy.stats.norm.ppf(np.linspace(offset, 0.5, half)[:-1])
    t = np.sort(np.concatenate([neg, [0.0], pos]))
    t = t / np.abs(t).max()
    return t.astype(np.float32), int(np.argmin(np.abs(t)))
