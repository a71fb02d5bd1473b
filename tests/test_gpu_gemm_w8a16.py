"""GPU parity: W8A16 MSD GEMM against the CPU oracle (INT32 accumulators bit-exact, outputs within 1e-3 of the
row L2 norm), across tile / split / ragged shapes and at the benchmark's full sizes on sampled columns."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, bf16_bits, dev, rel_row_err

pytestmark = pytest.mark.gpu
TOL = 1e-3          # max |y - y_oracle| <= TOL * ||y_oracle[i,:]||_2


def _run(c, out_dtype, want_acc=True, ws=None):
    x, w, s = bf16_dev(c.x), dev(c.w), dev(c.w_scale)
    res = binding.gemm_w8a16(x, w, s, out_dtype=out_dtype, want_acc=want_acc, ws=ws)
    torch.cuda.synchronize()
    binding.last_device_status()
    return res


def _check(c, out_dtype=torch.float32, ws=None):
    y, acc = _run(c, out_dtype, True, ws)
    ref, oacc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True)
    assert np.array_equal(acc.cpu().numpy(), oacc), "INT32 accumulators differ"
    if out_dtype == torch.float32:
        got = y.cpu().numpy()
    else:
        got = oracle.bf16_bits_to_f64(bf16_bits(y))
    assert rel_row_err(got, ref).max() <= TOL
    if out_dtype == torch.bfloat16:
        # at most one BF16 ulp from the oracle's once-rounded BF16 output
        want = oracle.round_bf16(ref).view(np.int16).astype(np.int32)
        have = bf16_bits(y).view(np.int16).astype(np.int32)
        assert np.abs(want - have).max() <= 1
    return got, ref


@pytest.mark.parametrize("M,N,K", [(1, 128, 128), (8, 256, 512), (16, 4096, 4096), (5, 384, 272), (128, 512, 1024),
                                   (33, 1152, 2048), (1, 14336, 4096), (128, 4096, 2048)])
def test_gemm_w8a16_parity_fp32(M, N, K):
    _check(inputs.gemm_w8_case(M, N, K, seed=0), torch.float32)


@pytest.mark.parametrize("M,N,K", [(4, 1024, 1024), (64, 2048, 512)])
def test_gemm_w8a16_parity_bf16(M, N, K):
    _check(inputs.gemm_w8_case(M, N, K, seed=1), torch.bfloat16)


def test_ragged_n_fp32_and_workspace_reuse():
    c = inputs.gemm_w8_case(7, 200, 400 - 400 % 16, seed=3)
    ws = binding.workspace(binding.gemm_w8a16_workspace_bytes(7, 200, c.x.shape[1]))
    for _ in range(3):                   # the split-K counters must come back to zero after every call
        _check(c, torch.float32, ws)


@pytest.mark.parametrize("ctas", ["1", "3", "37", "148", "200"])
def test_split_schedules(ctas, monkeypatch):
    """Different CTA counts move the tile/segment boundaries; the integer result must not change."""
    binding.debug_set_option("MSD_GEMM_CTAS", int(ctas))
    _check(inputs.gemm_w8_case(16, 640, 1536, seed=5), torch.float32)
    _check(inputs.gemm_w8_case(128, 256, 768, seed=6), torch.bfloat16)


@pytest.mark.parametrize("mode,ctas", [("0", "148"), ("1", "148"), ("1", "100"), ("1", "111")])
def test_row_partition_and_stream_k_agree(mode, ctas, monkeypatch):
    """Tall weights can run either split; band heights (multiples of 8, two sizes) and a ragged last band."""
    binding.debug_set_option("MSD_GEMM_MODE", int(mode))
    binding.debug_set_option("MSD_GEMM_CTAS", int(ctas))
    _check(inputs.gemm_w8_case(16, 12000, 512, seed=8), torch.float32)
    _check(inputs.gemm_w8_case(128, 10004, 256, seed=9), torch.float32)


@pytest.mark.parametrize("ctas", ["148", "40", "24", "9"])
def test_cluster_split_k(ctas, monkeypatch):
    """Few weight tiles: a cluster of CTAs per tile splits K and sums the partial tiles through distributed shared
    memory.  The CTA count sets the cluster size (8, 5 / 4, 3 / 2, ...); token counts cover one finishing CTA (M <= 8),
    fewer owners than CTAs, uneven token groups and the full 128; a ragged last tile; both output types."""
    binding.debug_set_option("MSD_GEMM_MODE", int("2"))
    binding.debug_set_option("MSD_GEMM_CTAS", int(ctas))
    _check(inputs.gemm_w8_case(3, 640, 4096, seed=21), torch.float32)
    _check(inputs.gemm_w8_case(24, 1000, 4096 + 16, seed=22), torch.bfloat16)
    _check(inputs.gemm_w8_case(128, 512, 6144, seed=23), torch.float32)
    _check(inputs.gemm_w8_case(72, 384, 8192, seed=24), torch.bfloat16)


def test_cluster_split_k_comparison_kernel(monkeypatch):
    binding.debug_set_option("MSD_GEMM_MODE", int("2"))
    c = inputs.gemm_w8_case(40, 512, 4096, seed=25)
    y = binding.gemm_dequant_bf16(bf16_dev(c.x), dev(c.w), dev(c.w_scale), out_dtype=torch.float32)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref = oracle.gemm_dequant_bf16_w8(c.x, c.w, c.w_scale)
    assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL


def test_fractional_scaling_layer():
    """msd_gemm_w8a16_ex with the scaling constants of Sec. 3.3 (127.49 / 254.98): accumulators bit-exact against the
    oracle run with the same constants."""
    for (M, N, K, seed) in [(5, 384, 272, 51), (16, 4096, 4096, 52), (128, 512, 1024, 53)]:
        c = inputs.gemm_w8_case(M, N, K, seed=seed)
        y, acc = binding.gemm_w8a16(bf16_dev(c.x), dev(c.w), dev(c.w_scale), out_dtype=torch.float32, want_acc=True, fractional=True)
        torch.cuda.synchronize()
        binding.last_device_status()
        ref, oacc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True, fractional=True)
        assert np.array_equal(acc.cpu().numpy(), oacc)
        assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL
        _, dacc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True)
        assert not np.array_equal(oacc, dacc)


def test_small_m_shapes():
    """M <= 8: one weight band per CTA, a ragged last band, K not a multiple of the stage width; bit for bit."""
    _check(inputs.gemm_w8_case(1, 1152, 2048, seed=11), torch.float32)
    _check(inputs.gemm_w8_case(8, 12000, 528, seed=12), torch.float32)
    _check(inputs.gemm_w8_case(3, 640, 1536 + 16, seed=13), torch.bfloat16)


def test_without_programmatic_dependent_launch(monkeypatch):
    binding.debug_set_option("MSD_NO_PDL", int("1"))
    _check(inputs.gemm_w8_case(16, 1024, 1024, seed=7), torch.float32)


def test_msd_error_not_worse_than_dequant_reference():
    """MSD error against the FP64 dequantized reference stays below the dequantize-to-BF16 path's error."""
    c = inputs.gemm_w8_case(16, 1024, 4096, seed=0)
    y = _run(c, torch.float32, want_acc=False).cpu().numpy()
    ref = oracle.gemm_ref_w8(c.x, c.w, c.w_scale)
    deq = oracle.gemm_dequant_bf16_w8(c.x, c.w, c.w_scale)
    n = np.linalg.norm(ref)
    assert np.linalg.norm(y - ref) / n <= np.linalg.norm(deq - ref) / n


@pytest.mark.parametrize("M", [1, 16, 128])
@pytest.mark.parametrize("N,K", [(14336, 4096), (4096, 14336)])
def test_full_size_sampled_columns(M, N, K):
    """The benchmark's decode shapes in its launch configuration; the oracle recomputes 96 sampled output columns."""
    c = inputs.gemm_w8_case(M, N, K, seed=0)
    y, acc = _run(c, torch.bfloat16, True)
    cols = np.unique(np.concatenate([[0, 127, 128, N - 1], np.random.default_rng(0).integers(0, N, 92)]))
    ref, oacc = oracle.gemm_w8a16(c.x, c.w[cols], c.w_scale[cols], "f64", want_acc=True)
    assert np.array_equal(acc.cpu().numpy()[:, :, cols], oacc)
    got = oracle.bf16_bits_to_f64(bf16_bits(y))[:, cols]
    want = oracle.bf16_bits_to_f64(oracle.round_bf16(ref))
    # sampled columns: compare per element against the BF16 spacing instead of the (unknown) full row norm
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -7 + 1e-30)


def test_host_buffer_entry_point():
    c = inputs.gemm_w8_case(16, 1024, 1024, seed=9)
    M, K = c.x.shape
    N = c.w.shape[0]
    xh = torch.from_numpy(c.x.view(np.int16)).view(torch.bfloat16).pin_memory()
    yh = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    ws = binding.workspace(binding.gemm_w8a16_host_workspace_bytes(M, N, K))
    binding.gemm_w8a16_host(xh, dev(c.w), dev(c.w_scale), yh, ws)
    torch.cuda.synchronize()
    ref = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64")
    assert rel_row_err(oracle.bf16_bits_to_f64(bf16_bits(yh)), ref).max() <= TOL


@pytest.mark.parametrize("M,N,K,ctas", [(16, 1024, 1024, None), (128, 640, 1536, "37"), (5, 12000, 512, None), (1, 4096, 4096, None)])
def test_dequant_bf16_comparison_kernel(M, N, K, ctas, monkeypatch):
    """The path MSD replaces: bf16(s_W * w) written back, then a BF16 x BF16 GEMM with FP32 accumulation."""
    if ctas:
        binding.debug_set_option("MSD_GEMM_CTAS", int(ctas))
    c = inputs.gemm_w8_case(M, N, K, seed=4)
    y = binding.gemm_dequant_bf16(bf16_dev(c.x), dev(c.w), dev(c.w_scale), out_dtype=torch.float32)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref = oracle.gemm_dequant_bf16_w8(c.x, c.w, c.w_scale)
    assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL
    # and it is the less accurate of the two paths against the FP64 product with the dequantized weight
    truth = oracle.gemm_ref_w8(c.x, c.w, c.w_scale)
    msd = binding.gemm_w8a16(bf16_dev(c.x), dev(c.w), dev(c.w_scale), out_dtype=torch.float32).cpu().numpy()
    n = np.linalg.norm(truth)
    assert np.linalg.norm(msd - truth) / n <= np.linalg.norm(y.cpu().numpy() - truth) / n


@pytest.mark.parametrize("M,N,K", [(129, 256, 128), (300, 520, 400), (1000, 264, 2048), (640, 1288, 144)])
def test_prefill_regime_parity_fp32(M, N, K):
    """M > 128 runs the token-major kernel (128 tokens x 256 weight rows per tile, two INT32 accumulators): ragged last
    token tile, ragged last weight tile (also by less than a store chunk), K not a multiple of the stage, several tiles
    per CTA; accumulators bit-exact."""
    _check(inputs.gemm_w8_case(M, N, K, seed=5), torch.float32)


def test_prefill_regime_parity_bf16_and_fractional_scaling():
    c = inputs.gemm_w8_case(777, 1032, 512, seed=6)
    _check(c, torch.bfloat16)
    x, w, s = bf16_dev(c.x), dev(c.w), dev(c.w_scale)
    y, acc = binding.gemm_w8a16(x, w, s, out_dtype=torch.float32, want_acc=True, fractional=True)
    torch.cuda.synchronize()
    binding.last_device_status()
    ref, oacc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True, fractional=True)
    assert np.array_equal(acc.cpu().numpy(), oacc)
    assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL


def test_prefill_full_size_sampled():
    """M = 4096 on the first decode shape (N = 14336, K = 4096), BF16 out; the oracle recomputes sampled rows x columns."""
    M, N, K = 4096, 14336, 4096
    c = inputs.gemm_w8_case(M, N, K, seed=0)
    y = _run(c, torch.bfloat16, want_acc=False)
    rng = np.random.default_rng(2)
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], rng.integers(0, M, 12)]))
    cols = np.unique(np.concatenate([[0, 255, 256, N - 1], rng.integers(0, N, 60)]))
    ref = oracle.gemm_w8a16(c.x[rows], c.w[cols], c.w_scale[cols], "f64")
    got = oracle.bf16_bits_to_f64(bf16_bits(y))[np.ix_(rows, cols)]
    slack = np.abs(ref) * 2.0 ** -8
    n = np.linalg.norm(ref, axis=-1, keepdims=True)      # norm over the sampled columns only: smaller, so stricter
    assert np.all(np.abs(got - ref) <= TOL * n + slack)


@pytest.mark.parametrize("M,N,K", [(256, 512, 4096), (400, 264, 2176), (129, 1032, 8192)])
def test_prefill_regime_with_k_split(M, N, K):
    """A few hundred rows on a narrow layer: few output tiles, so the K stages are split over the CTAs, every work item
    writes s_W (alpha D1 + beta D2) of its K range in FP32 and a second kernel adds the splits (the INT32 accumulators
    are not available in this mode, so outputs only).  Ragged token and weight tiles, a K that is not a multiple of the
    split, FP32 and BF16 outputs."""
    c = inputs.gemm_w8_case(M, N, K, seed=9)
    ref = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64")
    y = _run(c, torch.float32, want_acc=False)
    assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL
    yb = _run(c, torch.bfloat16, want_acc=False)
    got = oracle.bf16_bits_to_f64(bf16_bits(yb))
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(got - ref) <= TOL * n + np.abs(ref) * 2.0 ** -8 + 1e-30)


@pytest.mark.parametrize("pair", ["0", "1"])
@pytest.mark.parametrize("M,N,K", [(129, 256, 128), (300, 520, 400), (1000, 264, 2048), (1290, 1288, 144)])
def test_prefill_single_cta_and_cta_pair_kernels(pair, M, N, K, monkeypatch):
    """The many-row kernel as single CTAs and as CTA pairs (256 tokens per pair of CTAs), each forced on every shape: a
    pair whose second CTA has a single row or none, an odd number of 128-row tiles, ragged weight tiles, several tiles per
    pair; INT32 accumulators bit-exact in both, FP32 and BF16 outputs."""
    binding.debug_set_option("MSD_P8_PAIR", int(pair))
    c = inputs.gemm_w8_case(M, N, K, seed=11)
    _check(c, torch.float32)
    _check(c, torch.bfloat16)


@pytest.mark.parametrize("M,N,K,pair,ksplit", [(129, 256, 128, -1, -1), (300, 520, 448, 0, -1), (300, 520, 448, 1, -1),
                                               (640, 1288, 192, -1, -1), (256, 264, 4096, 0, 4)])
def test_dequant_bf16_comparison_kernel_many_rows(M, N, K, pair, ksplit):
    """The comparison path beyond 128 rows: weights expanded to BF16, then the many-row pipeline as a BF16 x BF16 GEMM
    with FP32 accumulation (single-CTA and CTA-pair kernels, K split): against the oracle's dequantize-to-BF16 product,
    FP32 and BF16 outputs; and MSD is the more accurate of the two against the FP64 product."""
    if pair >= 0:
        binding.debug_set_option("MSD_P8_PAIR", pair)
    if ksplit >= 0:
        binding.debug_set_option("MSD_P8_KSPLIT", ksplit)
    c = inputs.gemm_w8_case(M, N, K, seed=9 + M)
    xd, wd, sd = bf16_dev(c.x), dev(c.w), dev(c.w_scale)
    ref = oracle.gemm_dequant_bf16_w8(c.x, c.w, c.w_scale)
    for _ in range(2):
        y = binding.gemm_dequant_bf16(xd, wd, sd, out_dtype=torch.float32)
        torch.cuda.synchronize()
        binding.last_device_status()
        assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL
    yb = binding.gemm_dequant_bf16(xd, wd, sd, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    got = oracle.bf16_bits_to_f64(bf16_bits(yb))
    n = np.linalg.norm(ref, axis=1, keepdims=True)
    assert np.all(np.abs(got - ref) <= TOL * n + np.abs(ref) * 2.0 ** -8)
    truth = oracle.gemm_ref_w8(c.x, c.w, c.w_scale)
    msd = binding.gemm_w8a16(xd, wd, sd, out_dtype=torch.float32).cpu().numpy()
    assert np.linalg.norm(msd - truth) <= np.linalg.norm(y.cpu().numpy() - truth)


@pytest.mark.parametrize("M,N,K", [(16, 1024, 1024), (1, 4096, 4096), (128, 640, 1536), (5, 12000, 512), (33, 264, 2048),
                                   (16, 14336, 4096), (64, 4096, 2048)])
def test_fused_dequant_comparison_kernel(M, N, K):
    """The stronger comparison arm: INT8 weights converted to BF16 inside the GEMM, scale applied to the FP32 sums.
    Row bands and K-split tiles, ragged last band, M not a multiple of 16.  Against the FP64 product with the
    dequantized weights (the kernel rounds nothing but the FP32 accumulation and the output)."""
    c = inputs.gemm_w8_case(M, N, K, seed=31 + M)
    xd, wd, sd = bf16_dev(c.x), dev(c.w), dev(c.w_scale)
    truth = oracle.gemm_ref_w8(c.x, c.w, c.w_scale)
    for _ in range(2):
        y = binding.gemm_w8a16_fused_dequant(xd, wd, sd, out_dtype=torch.float32)
        torch.cuda.synchronize()
        binding.last_device_status()
        assert rel_row_err(y.cpu().numpy(), truth).max() <= 1e-5
    yb = binding.gemm_w8a16_fused_dequant(xd, wd, sd, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    got = oracle.bf16_bits_to_f64(bf16_bits(yb))
    n = np.linalg.norm(truth, axis=1, keepdims=True)
    assert np.all(np.abs(got - truth) <= 1e-5 * n + np.abs(truth) * 2.0 ** -8)
