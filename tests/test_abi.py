"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments before any launch.
No compute call is made here: these tests run without a GPU."""
import ctypes as C
import os
import re

from paper_2605_13915_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "msd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(msd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = C.CDLL(os.path.join(ROOT, "paper_2605_13915_b200", "libmsd.so")) if os.path.exists(
        os.path.join(ROOT, "paper_2605_13915_b200", "libmsd.so")) else binding.lib()
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    # and the binding knows a signature for each of them
    assert set(names) == set(binding._SIGS)


def test_status_strings():
    lib = binding.lib()
    seen = {lib.msd_status_string(i) for i in range(8)}
    assert len(seen) == 8 and b"ok" in seen


def test_argument_checks_precede_any_launch():
    lib = binding.lib()
    p = C.c_void_p(4096)          # never dereferenced: every call below must fail in the host checks
    null = C.c_void_p(0)
    assert lib.msd_decompose_int8(null, 4, 64, 64, p, p, p, p, None) == 1          # null pointer
    assert lib.msd_decompose_int8(p, 4, 40, 40, p, p, p, p, None) == 2             # K % 16
    assert lib.msd_decompose_int8(C.c_void_p(4098), 4, 64, 64, p, p, p, p, None) == 3   # alignment
    assert lib.msd_decompose_int8(p, 0, 64, 64, p, p, p, p, None) == 0             # M = 0 is a no-op
    assert lib.msd_decompose_mxfp4(p, 4, 48, 48, p, p, p, p, None) == 2            # K % 32
    assert lib.msd_gemm_w8a16(p, p, p, 0, 128, 128, p, 0, None, p, 1 << 30, None) == 2       # M out of range
    assert lib.msd_gemm_w8a16(p, p, p, (1 << 24) + 1, 128, 128, p, 0, None, p, 1 << 30, None) == 2
    assert lib.msd_gemm_w8a16(p, p, p, 300, 130, 128, p, 1, None, p, 1 << 30, None) == 2      # FP32 rows written by TMA: N % 4
    assert lib.msd_gemm_w8a16(p, p, p, 300, 128, 128, p, 0, None, p, 1024, None) == 5         # workspace too small
    assert lib.msd_gemm_w8a16(p, p, p, 4, 128, 128, p, 7, None, p, 1 << 30, None) == 4       # unknown output type
    assert lib.msd_gemm_w8a16(p, p, p, 4, 128, 128, p, 0, None, null, 1 << 30, None) == 1    # null workspace
    assert lib.msd_gemm_w8a16(p, p, p, 4, 128, 128, p, 0, None, C.c_void_p(4096 + 512), 1 << 30, None) == 3
    assert lib.msd_gemm_w8a16(p, p, p, 4, 128, 128, p, 0, None, p, 16, None) == 5            # workspace too small
    assert lib.msd_gemm_w8a16_workspace_bytes(16, 4096, 4096) >= 2 * 16 * 4096
    # E8M0 weight scales are read as 32-bit words: a byte-aligned pointer is refused on the host
    odd = C.c_void_p(4096 + 1)
    assert lib.msd_gemm_w4a16(p, p, odd, 128, 128, 128, p, 0, p, 1 << 30, None) == 3
    assert lib.msd_gemm_w4a16_e1m2(p, p, odd, 128, 128, 128, p, 0, p, 1 << 30, None) == 3
    # beyond K = 131072 the INT32 sums of Alg. 1 could overflow
    assert lib.msd_gemm_w8a16(p, p, p, 4, 128, 131072 + 16, p, 0, None, p, 1 << 40, None) == 4
    # the allocation-free entry point reports bad arguments before it clears its scratch
    assert lib.msd_gemm_w8a16_noalloc(null, p, p, 4, 128, 128, p, 0, None) in (1, 6)
    assert lib.msd_gemm_w8a16_noalloc(p, p, p, 17, 128, 128, p, 0, None) == 4
    # weight scales prepared once: size query, null / misaligned buffers, shape rules as for msd_gemm_w4a16
    assert lib.msd_w4a16_prepared_scales_bytes(1, 8192, 8192) >= 2 * 8192 * 8192 // 32
    assert lib.msd_w4a16_prepared_scales_bytes(1, 8192, 100) == 0
    assert lib.msd_prepare_w4a16_scales(null, 1, 128, 128, p, None) == 1
    assert lib.msd_prepare_w4a16_scales(p, 1, 128, 128, C.c_void_p(4096 + 512), None) == 3
    assert lib.msd_prepare_w4a16_scales(p, 0, 128, 128, p, None) == 2
    assert lib.msd_gemm_w4a16_prepared(p, p, null, 128, 128, 128, p, 0, p, 1 << 30, None) == 1
    assert lib.msd_gemm_w4a16_prepared(p, p, C.c_void_p(4096 + 512), 128, 128, 128, p, 0, p, 1 << 30, None) == 3
    assert lib.msd_gemm_w4a16_prepared(p, p, p, 128, 128, 100, p, 0, p, 1 << 30, None) == 2
    sizes = (C.c_int32 * 2)(4, 4)
    assert lib.msd_grouped_gemm_w4a16_prepared(p, p, null, sizes, 2, 128, 128, p, 0, p, 1 << 30, None) == 1
