"""Shared helpers of the tests: bf16 bit patterns <-> torch / numpy, error norms."""
import numpy as np
import torch

from workloads import from_bf16_bits, to_bf16_bits

TOL = 5e-3          # relative Frobenius error allowed on floating-point outputs


def bits_to_torch(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device` (same bytes)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def torch_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def rel_err(a, b) -> float:
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def f32(bits):
    return from_bf16_bits(bits)


def bf16_round(x):
    return from_bf16_bits(to_bf16_bits(np.asarray(x, np.float32)))
