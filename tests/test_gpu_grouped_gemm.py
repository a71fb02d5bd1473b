"""GPU parity: grouped W8A16 MSD GEMM (MoE experts) against the CPU oracle run expert by expert."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, bf16_bits, dev, rel_row_err

pytestmark = pytest.mark.gpu
TOL = 1e-3


def _case(sizes, N, K, seed):
    E = len(sizes)
    M = int(sum(sizes))
    x = inputs.activations(max(M, 1), K, seed)[:M]
    ws, ss = [], []
    for e in range(E):
        w, s = inputs.quantize_weight_int8(inputs.weights_f32(N, K, seed * 100 + e))
        ws.append(w)
        ss.append(s)
    return x, np.stack(ws), np.stack(ss)


def _oracle(x, w, s, sizes):
    out = np.zeros((x.shape[0], w.shape[1]), np.float64)
    off = 0
    for e, m in enumerate(sizes):
        if m:
            out[off:off + m] = oracle.gemm_w8a16(x[off:off + m], w[e], s[e], "f64")
        off += m
    return out


@pytest.mark.parametrize("sizes,N,K", [([3, 0, 16, 1], 384, 512), ([128, 5, 0, 0, 64, 7, 9, 2], 1000, 1040),
                                       ([1] * 70 + [0] * 10 + [4] * 5, 256, 256), ([0, 0, 11], 2048, 4096)])
def test_grouped_gemm_matches_per_expert_oracle(sizes, N, K):
    """Uneven groups, empty experts (first, middle, last), more than 64 non-empty groups (two launches), a ragged last
    tile; the workspace is reused for a second call to check that the counters come back to zero."""
    x, w, s = _case(sizes, N, K, seed=len(sizes) + N)
    ref = _oracle(x, w, s, sizes)
    xd, wd, sd = bf16_dev(x), dev(w), dev(s)
    nbytes = int(binding.lib().msd_grouped_gemm_w8a16_workspace_bytes(int(sum(sizes)), max(sizes), len(sizes), N, K))
    ws = binding.workspace(nbytes)
    for _ in range(2):
        y = binding.grouped_gemm_w8a16(xd, wd, sd, sizes, out_dtype=torch.float32, ws=ws)
        torch.cuda.synchronize()
        binding.last_device_status()
        assert rel_row_err(y.cpu().numpy(), ref).max() <= TOL
    yb = binding.grouped_gemm_w8a16(xd, wd, sd, sizes, out_dtype=torch.bfloat16, ws=ws)
    torch.cuda.synchronize()
    got = oracle.bf16_bits_to_f64(bf16_bits(yb))
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(got - ref) <= TOL * n + np.abs(ref) * 2.0 ** -8 + 1e-30)


def test_grouped_equals_ungrouped_bitwise():
    """A group's rows come out exactly as the plain layer computes them (same integer sums, same combine)."""
    sizes = [16, 8]
    x, w, s = _case(sizes, 640, 1536, seed=7)
    y = binding.grouped_gemm_w8a16(bf16_dev(x), dev(w), dev(s), sizes, out_dtype=torch.float32)
    y0 = binding.gemm_w8a16(bf16_dev(x[:16]), dev(w[0]), dev(s[0]), out_dtype=torch.float32)
    y1 = binding.gemm_w8a16(bf16_dev(x[16:]), dev(w[1]), dev(s[1]), out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert torch.equal(y[:16], y0) and torch.equal(y[16:], y1)


def test_bad_group_sizes_are_refused():
    x, w, s = _case([4], 256, 256, seed=1)
    with pytest.raises(binding.MsdError):
        binding.grouped_gemm_w8a16(bf16_dev(np.zeros((129, 256), np.uint16)), dev(w), dev(s), [129], out_dtype=torch.float32)


def _case_w4(sizes, N, K, seed):
    M = int(sum(sizes))
    x = inputs.activations(max(M, 1), K, seed)[:M]
    qs, es = [], []
    for e in range(len(sizes)):
        q, sc = inputs.quantize_weight_mxfp4(inputs.weights_f32(N, K, seed * 100 + e))
        qs.append(q)
        es.append(sc)
    return x, np.stack(qs), np.stack(es)


@pytest.mark.parametrize("sizes,N,K", [([3, 0, 16, 1], 448, 512), ([128, 5, 0, 0, 64, 33, 9, 2], 1000, 1024),
                                       ([1] * 70 + [0] * 10 + [4] * 5, 232, 256), ([0, 0, 11], 2048, 4096)])
def test_grouped_w4a16_matches_per_expert_oracle(sizes, N, K):
    """Grouped W4A16 (MXFP4 weights per expert) against the oracle run expert by expert: uneven groups whose end falls
    inside a warp's 32 output rows (masked stores) and on their boundary (box stores), empty experts, more than 64
    non-empty groups (two launches), ragged last weight tile; FP32 and BF16 outputs; the workspace is reused."""
    x, q, e = _case_w4(sizes, N, K, seed=len(sizes) + N)
    ref = np.zeros((x.shape[0], N), np.float64)
    off = 0
    for g, m in enumerate(sizes):
        if m:
            ref[off:off + m] = oracle.gemm_w4a16(x[off:off + m], q[g], e[g], "f64")
        off += m
    xd, qd, ed = bf16_dev(x), dev(q), dev(e)
    ws = binding.workspace(int(binding.lib().msd_grouped_gemm_w4a16_workspace_bytes(len(sizes), N, K)))
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    for _ in range(2):
        # a canary in the output: rows are written by their own group only
        y = torch.full((x.shape[0], N), 12345.0, dtype=torch.float32, device="cuda")
        binding.grouped_gemm_w4a16(xd, qd, ed, sizes, ws=ws, out=y)
        torch.cuda.synchronize()
        binding.last_device_status()
        assert np.all(np.abs(y.cpu().numpy() - ref) <= TOL * n + 1e-30)
    yb = binding.grouped_gemm_w4a16(xd, qd, ed, sizes, out_dtype=torch.bfloat16, ws=ws)
    torch.cuda.synchronize()
    got = oracle.bf16_bits_to_f64(bf16_bits(yb))
    assert np.all(np.abs(got - ref) <= TOL * n + np.abs(ref) * 2.0 ** -8 + 1e-30)


@pytest.mark.parametrize("sizes,N,K", [([128, 5, 0, 0, 64, 33, 9, 2], 1000, 1024), ([1] * 70 + [0] * 10 + [4] * 5, 232, 256)])
def test_grouped_w4a16_with_prepared_scales(sizes, N, K):
    """All experts' weight scales prepared once: against the per-expert oracle and bit for bit the unprepared call."""
    x, q, e = _case_w4(sizes, N, K, seed=5 + len(sizes))
    ref = np.zeros((x.shape[0], N), np.float64)
    off = 0
    for g, m in enumerate(sizes):
        if m:
            ref[off:off + m] = oracle.gemm_w4a16(x[off:off + m], q[g], e[g], "f64")
        off += m
    xd, qd, ed = bf16_dev(x), dev(q), dev(e)
    prepared = binding.prepare_w4a16_scales(ed)
    plain = binding.grouped_gemm_w4a16(xd, qd, ed, sizes, out_dtype=torch.float32)
    y = binding.grouped_gemm_w4a16(xd, qd, None, sizes, out_dtype=torch.float32, prepared=prepared)
    torch.cuda.synchronize()
    binding.last_device_status()
    n = np.linalg.norm(ref, axis=-1, keepdims=True)
    assert np.all(np.abs(y.cpu().numpy() - ref) <= TOL * n + 1e-30)
    assert torch.equal(y, plain)
