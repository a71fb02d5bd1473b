"""GPU parity: activation decomposition kernels against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, canon_fp4

pytestmark = pytest.mark.gpu


def _cases():
    # (M, K): single block, ragged K (not a multiple of the CTA's stride), config shapes, K beyond the register cache
    return [(1, 16), (3, 48), (16, 4096), (5, 14336), (128, 4096), (2, 40000), (300, 272)]


@pytest.mark.parametrize("M,K", _cases())
def test_decompose_int8_bit_exact(M, K):
    xb = inputs.activations(M, K, seed=M + K)
    if M >= 3:
        xb[1, :] = 0                      # zero row
        xb[2, : K // 2] = 0x8000          # negative zeros
    q1, q2, a, b = binding.decompose_int8(bf16_dev(xb))
    o1, o2, oa, ob = oracle.decompose_int8(xb)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(b.cpu().numpy(), ob)
    assert np.array_equal(q1.cpu().numpy(), o1) and np.array_equal(q2.cpu().numpy(), o2)
    binding.last_device_status()


def test_decompose_int8_special_values_and_strided_rows():
    K = 256
    x = np.zeros((6, K), np.float32)
    x[0, 3] = 1.0
    x[1, :] = -7.5
    x[2, :] = np.linspace(-3, 3, K)
    x[3, 0] = 2.0 ** -120
    x[4, :] = np.random.default_rng(0).standard_normal(K) * 1e4
    x[5, :] = np.random.default_rng(1).standard_normal(K) * 1e-20
    xb = inputs.f32_to_bf16_bits(x)
    wide = np.zeros((6, K + 64), np.uint16)
    wide[:, :K] = xb
    xd = bf16_dev(wide)[:, :K]              # row stride K + 64
    M = 6
    q1 = torch.empty((M, K), dtype=torch.int8, device="cuda")
    q2 = torch.empty_like(q1)
    a = torch.empty(M, dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    code = binding.lib().msd_decompose_int8(xd.data_ptr(), M, K, K + 64, q1.data_ptr(), q2.data_ptr(), a.data_ptr(), b.data_ptr(),
                                            torch.cuda.current_stream().cuda_stream)
    assert code == 0
    o1, o2, oa, ob = oracle.decompose_int8(xb)
    assert np.array_equal(q1.cpu().numpy(), o1) and np.array_equal(q2.cpu().numpy(), o2)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(b.cpu().numpy(), ob)


@pytest.mark.parametrize("M,K", [(1, 32), (4, 8192), (257, 96), (64, 2048)])
def test_decompose_mxfp4_bit_exact(M, K):
    xb = inputs.activations(M, K, seed=K - M)
    if M >= 4:
        xb[1, :32] = 0
        xb[2, :64] = inputs.f32_to_bf16_bits(np.full(64, 4.5, np.float32) * np.float32(2.0 ** -20))
        xb[3, :32] = inputs.f32_to_bf16_bits(np.linspace(-6, 6, 32).astype(np.float32))
    q1, q2, e1, e2 = binding.decompose_mxfp4(bf16_dev(xb))
    o1, o2, oe1, oe2 = oracle.decompose_mxfp4(xb)
    assert np.array_equal(e1.cpu().numpy(), oe1) and np.array_equal(e2.cpu().numpy(), oe2)
    assert np.array_equal(canon_fp4(q1.cpu().numpy()), canon_fp4(o1))
    assert np.array_equal(canon_fp4(q2.cpu().numpy()), canon_fp4(o2))
    binding.last_device_status()


def test_decompose_mxfp4_extreme_exponents():
    K = 64
    x = np.zeros((4, K), np.float32)
    x[0, :] = 3.0e38
    x[1, :32] = 2.0 ** -126
    x[1, 32:] = 2.0 ** -130
    x[2, :] = np.random.default_rng(2).standard_normal(K) * 2.0 ** -120
    x[3, :] = np.random.default_rng(3).standard_normal(K) * 2.0 ** 100
    xb = inputs.f32_to_bf16_bits(x)
    q1, q2, e1, e2 = binding.decompose_mxfp4(bf16_dev(xb))
    o1, o2, oe1, oe2 = oracle.decompose_mxfp4(xb)
    assert np.array_equal(e1.cpu().numpy(), oe1) and np.array_equal(e2.cpu().numpy(), oe2)
    assert np.array_equal(canon_fp4(q1.cpu().numpy()), canon_fp4(o1))
    assert np.array_equal(canon_fp4(q2.cpu().numpy()), canon_fp4(o2))


@pytest.mark.parametrize("M,K", [(3, 48), (16, 4096), (5, 14336)])
def test_decompose_int8_fractional_scaling_bit_exact(M, K):
    """Sec. 3.3: alpha = max/127.49, beta = alpha/254.98 through msd_decompose_int8_ex; an unknown scaling is refused."""
    xb = inputs.activations(M, K, seed=2 * M + K)
    q1, q2, a, b = binding.decompose_int8(bf16_dev(xb), fractional=True)
    o1, o2, oa, ob = oracle.decompose_int8(xb, fractional=True)
    assert np.array_equal(a.cpu().numpy(), oa) and np.array_equal(b.cpu().numpy(), ob)
    assert np.array_equal(q1.cpu().numpy(), o1) and np.array_equal(q2.cpu().numpy(), o2)
    d1, _d2, da, _db = oracle.decompose_int8(xb)
    assert not np.array_equal(oa, da)                      # the flag does change the scales
    x = bf16_dev(xb)
    code = binding.lib().msd_decompose_int8_ex(x.data_ptr(), M, K, K, q1.data_ptr(), q2.data_ptr(), a.data_ptr(), b.data_ptr(), 7,
                                               None)
    assert code == 4                                       # MSD_ERR_UNSUPPORTED
    binding.last_device_status()
