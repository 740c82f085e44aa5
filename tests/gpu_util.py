"""Helpers for the GPU parity tests: numpy <-> torch device buffers, no arithmetic."""
import numpy as np
import torch


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(x: np.ndarray) -> torch.Tensor:
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint32:
        x = x.view(np.int32)
    return torch.from_numpy(x).cuda()


def host_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def f32_bits(x) -> np.ndarray:
    if isinstance(x, torch.Tensor):
        x = x.cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


def poison(shape, dtype) -> torch.Tensor:
    """Output buffer pre-filled with a pattern no correct result contains (0xFF bytes)."""
    t = torch.empty(shape, dtype=dtype, device="cuda")
    t.view(torch.uint8).fill_(0xFF)
    return t


def workspace(nbytes: int) -> torch.Tensor:
    return poison((max(int(nbytes), 256),), torch.uint8)
