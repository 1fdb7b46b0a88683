"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch


def words_of(t: torch.Tensor) -> np.ndarray:
    """Raw 16-bit patterns of a bf16/fp16 tensor as a flat numpy uint16 array (host)."""
    return t.detach().reshape(-1).view(torch.int16).cpu().numpy().view(np.uint16)


def tensor_of(words: np.ndarray, dtype: torch.dtype, device="cuda") -> torch.Tensor:
    return torch.from_numpy(words.view(np.int16).copy()).to(device).view(dtype)


def to_dev_bytes(stream: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(stream)).to(device)


def status_tensor():
    return torch.zeros(1, dtype=torch.int32, device="cuda")
