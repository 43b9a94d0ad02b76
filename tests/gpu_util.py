"""Helpers for the GPU tests: uint16 BF16 bit patterns <-> torch.bfloat16 device tensors."""
import numpy as np
import torch

from paper_2503_14985_b200 import inputs


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 BF16 bit patterns -> CUDA bfloat16 tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(torch.bfloat16)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """CUDA bfloat16 tensor -> float64 numpy (exact)."""
    bits = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return inputs.bf16_bits_to_f64(bits).reshape(tuple(t.shape))


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16).reshape(tuple(t.shape))


def assert_device_healthy():
    import paper_2503_14985_b200 as mlt
    rc, detail = mlt.last_device_error()
    assert rc == 0, f"device status {rc}: {detail}"
