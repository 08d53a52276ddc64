"""Helpers shared by the GPU parity tests: numpy <-> torch marshalling of bf16 bit patterns."""
import numpy as np
import torch


def bits_to_bf16(a: np.ndarray, device="cuda:0") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device` (same bits)."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    """torch bf16/f32 tensor -> numpy float64 (exact widening)."""
    return t.detach().to(torch.float64).cpu().numpy()


def to_dev(a: np.ndarray, device="cuda:0") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)
