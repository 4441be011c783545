"""Helpers shared by the GPU parity tests: device transfer of the synthetic inputs."""
import numpy as np
import torch

from paper_2505_08600_b200 import synth

DEV = "cuda:0"


def to_dev(a: np.ndarray):
    """numpy -> CUDA tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV).view(torch.bfloat16)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).to(DEV)
    return torch.from_numpy(a).to(DEV)


def widen(a: np.ndarray) -> np.ndarray:
    """fp32 or bf16 bit patterns -> float64 values."""
    return (synth.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a).astype(np.float64)


def quantize(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return synth.f32_to_bf16_bits(a) if dtype == "bf16" else a
