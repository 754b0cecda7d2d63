"""Helpers shared by the GPU parity tests (marshalling and the error metric)."""
import numpy as np
import torch

from paper_2105_09377_b200 import synth


def to_bf16_device(x: np.ndarray) -> torch.Tensor:
    """float32 array of bf16-representable values -> bf16 CUDA tensor with the same values."""
    bits = synth.bf16_bits(x).view(np.int16)
    return torch.from_numpy(bits).cuda().view(torch.bfloat16).reshape(x.shape)


def to_f32_device(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |g - r| / max(|r|, rms(r)): relative error that stays defined near zero outputs."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) or 1.0
    return float(np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms)))


REL_TOL = 2e-3
