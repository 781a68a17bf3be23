"""Host <-> device marshalling for the GPU parity tests (no layer arithmetic)."""
import numpy as np
import torch

from paper_2502_01681_b200 import synth


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bfloat16 bit patterns -> CUDA bf16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_f64_of_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def f64_of_bits(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def bf16_weights(w_f32: np.ndarray):
    """float32 draw -> (bits, exact fp64 value of the rounded weights)."""
    bits = synth.f32_to_bf16_bits(w_f32)
    return bits, f64_of_bits(bits)
