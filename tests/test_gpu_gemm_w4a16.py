"""GPU parity: W4A16 MSD GEMM (two block-scaled FP4 passes accumulated in one FP32 tile) against the CPU oracle's
FP64 sum, within 1e-3 of the row L2 norm; accuracy compared with the single-pass MXFP8 activation baseline."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, bf16_bits, dev

pytestmark = pytest.mark.gpu
TOL = 1e-3


def _run(c, out_dtype):
    y = binding.gemm_w4a16(bf16_dev(c.x), dev(c.w_fp4), dev(c.w_e8m0), out_dtype=out_dtype)
    torch.cuda.synchronize()
    binding.last_device_status()
    return y


def _close(got, ref, bf16):
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    slack = np.abs(ref) * 2.0 ** -8 if bf16 else 0.0
    assert np.all(np.abs(got - ref) <= TOL * n + slack + 1e-30), float(np.abs(got - ref).max() / n.max())


@pytest.mark.parametrize("M,N,K", [(128, 256, 256), (64, 512, 1024), (300, 264, 384), (1, 256, 128), (257, 776, 2048)])
def test_gemm_w4a16_parity_fp32(M, N, K):
    c = inputs.gemm_w4_case(M, N, K, seed=M + K)
    y = _run(c, torch.float32).cpu().numpy().astype(np.float64)
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
    _close(y, ref, False)


def test_gemm_w4a16_bf16_and_accuracy_vs_mxfp8():
    c = inputs.gemm_w4_case(256, 512, 2048, seed=3)
    y = oracle.bf16_bits_to_f64(bf16_bits(_run(c, torch.bfloat16)))
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
    _close(y, ref, True)
    # against X * W_mx4 with unquantized activations the two-pass MXFP4 result beats single-pass MXFP8 activations
    truth = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="ref")
    mx8 = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="mxfp8")
    n = np.linalg.norm(truth)
    assert np.linalg.norm(y - truth) / n < np.linalg.norm(mx8 - truth) / n


def test_scale_handling_extremes():
    """Blocks with very different magnitudes exercise the E8M0 scale path of both operands."""
    rng = np.random.default_rng(0)
    M, N, K = 128, 256, 512
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[:, :128] *= 2.0 ** -30
    x[:, 128:256] *= 2.0 ** 20
    x[5, :] = 0
    w = rng.standard_normal((N, K)).astype(np.float32)
    w[:, 256:384] *= 2.0 ** -12
    xb = inputs.f32_to_bf16_bits(x)
    q, e = inputs.quantize_weight_mxfp4(w)
    y = binding.gemm_w4a16(bf16_dev(xb), dev(q), dev(e), out_dtype=torch.float32)
    torch.cuda.synchronize()
    ref = oracle.gemm_w4a16(xb, q, e, "f64")
    _close(y.cpu().numpy().astype(np.float64), ref, False)


def test_full_size_sampled():
    """The prefill shape at full size (M=4096, K=8192, N=8192, BF16 out); the oracle recomputes sampled rows x columns."""
    M, N, K = 4096, 8192, 8192
    c = inputs.gemm_w4_case(M, N, K, seed=0)
    y = _run(c, torch.bfloat16)
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], rng.integers(0, M, 28)]))
    cols = np.unique(np.concatenate([[0, 255, 256, N - 1], rng.integers(0, N, 60)]))
    ref = oracle.gemm_w4a16(c.x[rows], c.w_fp4[cols], c.w_e8m0[cols], "f64")
    got = oracle.bf16_bits_to_f64(bf16_bits(y))[np.ix_(rows, cols)]
    # sampled columns: the row norm over the sample stands in for the full row norm (it is smaller, so stricter)
    _close(got, ref, True)


@pytest.mark.parametrize("pair", ["0", "1"])
def test_single_cta_and_cta_pair_kernels_agree(pair, monkeypatch):
    """The single-CTA kernel and the CTA-pair kernel (one 256-token tile per pair of CTAs), each forced on every shape,
    including a pair whose second CTA has no rows at all and an odd number of 128-row tiles; both tile widths."""
    binding.debug_set_option("MSD_W4_PAIR", int(pair))
    for (M, N, K) in [(64, 512, 512), (384, 264, 1024), (520, 1032, 768)]:
        c = inputs.gemm_w4_case(M, N, K, seed=7 + M)
        y = _run(c, torch.float32).cpu().numpy().astype(np.float64)
        ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
        _close(y, ref, False)
        binding.debug_set_option("MSD_W4_TILEN", int("256"))
        y = _run(c, torch.float32).cpu().numpy().astype(np.float64)
        binding.debug_set_option("MSD_W4_TILEN", -1)
        _close(y, ref, False)


@pytest.mark.parametrize("M,N,K", [(16, 448, 4096), (100, 1000, 3072), (1, 232, 8192), (128, 264, 2048)])
def test_decode_shapes_with_k_split(M, N, K):
    """Few output tiles and a long K: the K stages are split over several CTAs, the FP32 partial tiles are added by a
    second kernel; only the M rows present are loaded (packed stages).  Ragged last weight tile, M = 1 and M = 128."""
    c = inputs.gemm_w4_case(M, N, K, seed=21 + M)
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
    y = _run(c, torch.float32).cpu().numpy().astype(np.float64)
    _close(y, ref, False)
    yb = _run(c, torch.bfloat16)
    _close(oracle.bf16_bits_to_f64(bf16_bits(yb)), ref, True)


@pytest.mark.parametrize("M,N,K,pair,tile", [(300, 264, 384, -1, -1), (520, 1032, 768, 1, 256), (520, 1032, 768, 1, 224),
                                             (384, 776, 1024, 0, 224), (384, 776, 1024, 0, 256), (16, 448, 4096, -1, -1)])
def test_prepared_weight_scales(M, N, K, pair, tile):
    """Weight scales brought into the blocked layout once (msd_prepare_w4a16_scales) instead of on every call: against
    the oracle, and bit for bit the result of the call that takes the row-major scales; single-CTA, CTA-pair and
    K-split kernels, both tile widths, ragged last weight tile.  The prepared buffer is made once and used twice."""
    c = inputs.gemm_w4_case(M, N, K, seed=3 + M + N)
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
    xd, qd, ed = bf16_dev(c.x), dev(c.w_fp4), dev(c.w_e8m0)
    prepared = binding.prepare_w4a16_scales(ed)
    if pair >= 0:
        binding.debug_set_option("MSD_W4_PAIR", pair)
    if tile >= 0:
        binding.debug_set_option("MSD_W4_TILEN", tile)
    plain = binding.gemm_w4a16(xd, qd, ed, out_dtype=torch.float32)
    for _ in range(2):
        y = binding.gemm_w4a16(xd, qd, None, out_dtype=torch.float32, prepared=prepared)
        torch.cuda.synchronize()
        binding.last_device_status()
        _close(y.cpu().numpy().astype(np.float64), ref, False)
        assert torch.equal(y, plain)
    yb = binding.gemm_w4a16(xd, qd, None, out_dtype=torch.bfloat16, prepared=prepared)
    assert torch.equal(yb, binding.gemm_w4a16(xd, qd, ed, out_dtype=torch.bfloat16))
