"""Helpers shared by the GPU parity tests: host bit patterns <-> device tensors."""
import numpy as np
import torch


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns (host) -> bf16 CUDA tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits)).cuda().view(torch.bfloat16)


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    torch.cuda.synchronize()
    return t.detach().cpu().numpy()


def status_word() -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def rms(a: np.ndarray) -> float:
    return float(np.sqrt(np.mean(np.square(a.astype(np.float64)))))
