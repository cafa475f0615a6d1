"""Helpers shared by the GPU parity tests (host <-> device marshalling, error metrics)."""
import numpy as np
import torch

from paper_2503_14075_b200 import synth

DEV = "cuda:0"


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 CUDA tensor (same bits)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 CUDA tensor -> uint16 bit patterns on the host."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def f64(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_to_f64(bits)


def max_abs(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.max(np.abs(got - want))) if got.size else 0.0


def rel_l2_rows(got: np.ndarray, want: np.ndarray) -> float:
    """Largest relative L2 error over the rows (last axis) of the two arrays."""
    if got.size == 0:
        return 0.0
    num = np.sqrt(np.sum((got - want) ** 2, axis=-1))
    den = np.sqrt(np.sum(want ** 2, axis=-1))
    return float(np.max(num / np.maximum(den, 1e-300)))


# tolerances for bf16-in / fp32-accumulate results against the fp64 oracle
MAX_ABS_TOL = 1e-2
REL_L2_TOL = 5e-3
