"""Shared helpers of the GPU parity tests: host <-> device marshalling and the comparison rules."""
import numpy as np
import torch


def bf16_dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def bf16_bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def canon_fp4(packed):
    """Map the negative-zero nibble 0x8 to 0x0 (FP4 codes are compared by value)."""
    p = np.asarray(packed, dtype=np.uint8)
    lo, hi = p & 15, p >> 4
    lo = np.where(lo == 8, 0, lo)
    hi = np.where(hi == 8, 0, hi)
    return (lo | (hi << 4)).astype(np.uint8)


def rel_row_err(y, ref):
    """max_j |y - ref| / ||ref[i,:]||_2 per row (the parity metric: <= 1e-3)."""
    y = np.asarray(y, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    n = np.linalg.norm(ref, axis=-1)
    n = np.where(n == 0, 1.0, n)
    return np.abs(y - ref).max(axis=-1) / n
