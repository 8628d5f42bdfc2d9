"""Shared test helpers: move seeded host workloads onto the GPU (bit-exact) and compare."""
import numpy as np


def to_device(a: np.ndarray, device):
    """numpy -> torch on `device`; uint16 arrays are reinterpreted as bfloat16 bit patterns."""
    import torch

    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host_f64(t) -> np.ndarray:
    """torch (bf16 / f32) -> numpy float64, exactly."""
    import torch

    return t.detach().to(torch.float64).cpu().numpy()


def bf16_bits(t) -> np.ndarray:
    import torch

    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)
