"""Shared helpers for the parity tests: conversions between the oracle's fp64
numpy arrays and device tensors, and the error metric."""
import numpy as np

from paper_1712_04432_b200 import inputs as I


def rel_fro(got, ref):
    """||got - ref||_F / ||ref||_F in fp64."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (den if den > 0 else 1.0))


def to_dev(a, bf16):
    """numpy float32 (bf16-exact when bf16) -> CUDA tensor of the network dtype."""
    import torch
    a = np.ascontiguousarray(a, np.float32)
    if bf16:
        bits = I.bf16_bits(a).view(np.int16)
        return torch.from_numpy(bits).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_np(t):
    """CUDA tensor (bf16 or f32) -> numpy float64."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    return t.cpu().numpy().astype(np.float64)
