"""The allocation-free W8A16 entry point against the regular one and against the CPU oracle.

Some callers of this library may not allocate device memory at all (a plug-in inside a serving loop that forbids
allocation on its hot path, a host whose memory pool belongs to another runtime); msd_gemm_w8a16_noalloc keeps its
scratch in a fixed array inside the library instead of a caller-provided workspace.  This file is collected last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs
from helpers import bf16_dev, dev

pytestmark = pytest.mark.gpu


def _both(c, out_dtype):
    x, w, s = bf16_dev(c.x), dev(c.w), dev(c.w_scale)
    M, N = c.x.shape[0], c.w.shape[0]
    ref = binding.gemm_w8a16(x, w, s, out_dtype=out_dtype)
    torch.cuda.synchronize()
    got = torch.full((M, N), float("nan"), dtype=out_dtype, device="cuda")
    binding.gemm_w8a16_noalloc(x, w, s, got)
    torch.cuda.synchronize()
    binding.last_device_status()
    return got, ref


@pytest.mark.parametrize("M,N,K", [(16, 4096, 4096), (3, 1000, 2064), (1, 16384, 16384)])
def test_noalloc_matches_regular_entry_point_twice_in_a_row(M, N, K):
    c1 = inputs.gemm_w8_case(M, N, K, seed=21)
    c2 = inputs.gemm_w8_case(M, N, K, seed=22)
    for c in (c1, c2):                      # the second call finds the first call's contents in the shared scratch
        got, ref = _both(c, torch.float32)
        # same kernels on the same inputs: the integer sums are order-free, so the two entry points agree exactly;
        # the tolerance is the one the GEMM parity tests use (1e-3 of the row L2 norm)
        g, r = got.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(g))
        assert np.all(np.abs(g - r) <= 1e-3 * np.linalg.norm(r, axis=1, keepdims=True))
        assert np.array_equal(g, r)
        # and the oracle (Alg. 1 in FP64), on the smaller shapes it finishes in a moment
        if N * K <= 4096 * 4096:
            want = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64")
            assert np.all(np.abs(g - want) <= 1e-3 * np.linalg.norm(want, axis=1, keepdims=True))
    got, ref = _both(c1, torch.bfloat16)
    assert torch.equal(got, ref)


def test_noalloc_rejects_shapes_beyond_its_scratch():
    lib = binding.lib()
    p = C.c_void_p(4096)        # never dereferenced: the size check comes first
    assert lib.msd_gemm_w8a16_noalloc(p, p, p, 17, 4096, 4096, p, 0, None) == 4        # M too large
    assert lib.msd_gemm_w8a16_noalloc(p, p, p, 16, 16384 + 128, 4096, p, 0, None) == 4  # N too large
    assert lib.msd_gemm_w8a16_noalloc(p, p, p, 16, 4096, 16384 + 16, p, 0, None) == 4   # K too large
    assert lib.msd_gemm_w8a16_noalloc(p, p, p, 0, 4096, 4096, p, 0, None) == 2          # bad shape
