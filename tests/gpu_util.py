"""Helpers for the GPU parity tests (device upload of synthetic arrays)."""
import numpy as np
import torch


def require_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device (run them with -m gpu on a B200)"
    return torch.device("cuda:0")


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 CUDA tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(require_cuda())
    return t.view(torch.bfloat16)


def dev_f32(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(require_cuda())
