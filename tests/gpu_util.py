"""Helpers shared by the GPU parity tests: move the same bf16 bytes to the device, compare."""
import numpy as np
import torch

from oracle import snip_oracle as orc


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> CUDA bf16 tensor holding the same bytes."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def rel_fro(got: np.ndarray, want: np.ndarray) -> float:
    den = np.linalg.norm(want.astype(np.float64))
    num = np.linalg.norm(got.astype(np.float64) - want.astype(np.float64))
    return float(num / den) if den > 0 else float(num)


def bf16_out_to_f64(t: torch.Tensor) -> np.ndarray:
    return orc.bf16_to_float(bits_of(t))
