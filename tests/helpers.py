"""Shared test utilities: tensor <-> numpy bit views. No arithmetic of the method lives here."""
import numpy as np
import torch


def f16_bits(t: torch.Tensor) -> np.ndarray:
    """fp16 tensor -> uint16 numpy array of its bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f16_tensor(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.float16)
