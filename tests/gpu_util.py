"""Shared helpers of the GPU parity tests: move oracle-side numpy operands to the device."""
import numpy as np
import torch

import paper_2511_16041_b200 as atb


def dev():
    return torch.device("cuda:0")


def bf16_bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev()).view(torch.bfloat16)


def bf16_dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def planes_to_dev(mant: np.ndarray, exp_logical: np.ndarray):
    M, K = mant.shape
    return (torch.from_numpy(np.ascontiguousarray(mant)).to(dev()),
            torch.from_numpy(atb.logical_to_exp_plane(exp_logical, M, K)).to(dev()))


def run_gemm(mant, exp_logical, B_bits, tiling, poison=True):
    """CUDA GEMM through the C ABI on oracle-quantised operands; returns bf16 bit patterns."""
    M, K = mant.shape
    N = B_bits.shape[1]
    md, ed = planes_to_dev(mant, exp_logical)
    Bd = bf16_bits_to_dev(B_bits)
    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev()) if poison else None
    C = atb.atb_gemm(M, N, K, *tiling, md, ed, Bd, C)
    atb.atb_device_status()
    return bf16_dev_to_bits(C)
