"""Shared helpers of the GPU parity tests: move seeded inputs to the device, run the
oracle on the exact values the GPU sees (bf16 upcast to fp64)."""
import numpy as np
import torch

from paper_2506_05096_b200 import synth


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).cuda()


def bf16_dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def f64(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_to_f64(bits)
