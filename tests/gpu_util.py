"""Helpers shared by the GPU parity tests: numpy (oracle side) <-> torch (device side)."""
import numpy as np
import torch

TORCH_VIEW = {"f16": torch.float16, "bf16": torch.bfloat16, "i8": torch.int8}


def to_device(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Stored representation (uint16 bit patterns / int8) -> CUDA tensor of the matching torch dtype."""
    if dtype in ("f16", "bf16"):
        return torch.from_numpy(a.view(np.int16)).cuda().view(TORCH_VIEW[dtype])
    if dtype == "i8":
        return torch.from_numpy(a).cuda()
    if dtype == "f32":
        return torch.from_numpy(a.astype(np.float32)).cuda()
    if dtype == "i32":
        return torch.from_numpy(a.astype(np.int32)).cuda()
    raise ValueError(dtype)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    """CUDA tensor -> numpy stored representation (uint16 bit patterns for 16-bit floats)."""
    if t.dtype in (torch.float16, torch.bfloat16):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def to_host_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype in (torch.float16, torch.bfloat16, torch.float32):
        return t.to(torch.float64).cpu().numpy()
    return t.cpu().numpy()
