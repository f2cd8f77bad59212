"""Shared helpers of the GPU parity tests (tensor plumbing only)."""
import numpy as np
import torch

from synth.generator import bf16_bits_to_f64


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns [H,N,d] -> CUDA bf16 tensor [1,H,N,d]."""
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()[None].contiguous()


def widen(*bits):
    return tuple(bf16_bits_to_f64(b) for b in bits)


def alloc_lists(hq, nqb, order_stride=None):
    order_stride = order_stride or nqb
    order = torch.full((1, hq, nqb, order_stride), -7, dtype=torch.int32, device="cuda")
    count = torch.full((1, hq, nqb), -7, dtype=torch.int32, device="cuda")
    return order, count


def alloc_outputs(q, order_stride):
    _, hq, n, d = q.shape
    nqb = n // 128
    return dict(out=torch.empty_like(q), lse=torch.empty(1, hq, n, dtype=torch.float32, device="cuda"),
                visited=torch.empty(1, hq, nqb, dtype=torch.int32, device="cuda"),
                scored=torch.empty(1, hq, nqb, dtype=torch.int32, device="cuda"),
                decisions=torch.zeros(1, hq, nqb, (order_stride + 31) // 32, dtype=torch.int32, device="cuda"))
