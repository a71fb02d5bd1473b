"""GPU parity: the paper-literal MXFP4 path (E1M2 components, alpha bound 1.859375, beta = alpha/16) against the CPU
oracle run with the same grid and rule."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, bf16_bits, dev

pytestmark = pytest.mark.gpu
TOL = 1e-3
C_BOUND, BETA_SHIFT = oracle.PAPER_E1M2

# E4M3 bytes of 0, .25, ..., 1.75 -> E1M2 code index
_E4M3_TO_CODE = {0x00: 0, 0x28: 1, 0x30: 2, 0x34: 3, 0x38: 4, 0x3A: 5, 0x3C: 6, 0x3E: 7}


def _codes(bytes_, ):
    b = bytes_.cpu().numpy()
    mag = np.vectorize(_E4M3_TO_CODE.__getitem__)(b & 0x7F).astype(np.uint8)
    code = mag | ((b >> 7) << 3)
    code[(mag == 0)] = 0                       # canonical zero
    return code


def _unpack(packed, K):
    lo, hi = packed & 15, packed >> 4
    out = np.empty((packed.shape[0], K), np.uint8)
    out[:, 0::2], out[:, 1::2] = lo, hi
    out[(out & 7) == 0] = 0
    return out


@pytest.mark.parametrize("M,K", [(1, 32), (5, 256), (130, 1024)])
def test_decompose_e1m2_bit_exact(M, K):
    xb = inputs.activations(M, K, seed=M + K)
    if M >= 3:
        xb[1, :] = 0
        xb[2, :64] = 0x8000
    q1, q2, e1, e2 = binding.decompose_mxfp4_e1m2(bf16_dev(xb))
    o1, o2, oe1, oe2 = oracle.decompose_mxfp4(xb, grid=oracle.GRID_E1M2, c_bound=C_BOUND, beta_shift=BETA_SHIFT)
    assert np.array_equal(e1.cpu().numpy(), oe1) and np.array_equal(e2.cpu().numpy(), oe2)
    assert np.array_equal(_codes(q1), _unpack(o1, K)) and np.array_equal(_codes(q2), _unpack(o2, K))
    binding.last_device_status()


@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (64, 512, 1024), (300, 264, 384), (257, 776, 2048)])
def test_gemm_w4a16_e1m2_parity(M, N, K):
    c = inputs.gemm_w4_case(M, N, K, seed=M + K + 1)
    y = binding.gemm_w4a16_e1m2(bf16_dev(c.x), dev(c.w_fp4), dev(c.w_e8m0), out_dtype=torch.float32)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", grid=oracle.GRID_E1M2, c_bound=C_BOUND, beta_shift=BETA_SHIFT)
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= TOL * n + 1e-30), float(np.abs(got - ref).max() / n.max())
    # the E1M2 rule is the more accurate of the two decompositions against unquantized activations (Tab. mxfp4-evolution)
    truth = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="ref")
    e2m1 = binding.gemm_w4a16(bf16_dev(c.x), dev(c.w_fp4), dev(c.w_e8m0), out_dtype=torch.float32).cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - truth) <= np.linalg.norm(e2m1 - truth) * 1.05
