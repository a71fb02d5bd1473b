"""CPU oracle for Multi-Scale Dequant: numpy front-end of ``msd_oracle.cpp``.

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do, and it imports
nothing from them.  Arrays are numpy; BF16 travels as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "msd_oracle.cpp")
_LIB = os.path.join(_HERE, "libmsd_oracle.so")

GRID_E2M1 = 0   # values 0, .5, 1, 1.5, 2, 3, 4, 6 (hardware FP4)
GRID_E1M2 = 1   # values 0, .25, ..., 1.75 (the grid the paper states)

# (alpha bound c, log2(alpha/beta)) pairs
PAPER_E1M2 = (1.859375, 4)      # Eq. alpha-mxfp4 / Eq. beta-mxfp4
E2M1_RULE = (4.5, 4)            # the same rule restated on the E2M1 grid


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain C++17, no fused contractions)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.msdo_max_threads.restype = C.c_int
        _lib.msdo_int8_gemm_acc.restype = C.c_int64
        _lib.msdo_gemm_w8a16.restype = C.c_int64
        _lib.msdo_gemm_w8a16_c.restype = C.c_int64
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def max_threads() -> int:
    return int(lib().msdo_max_threads())


def set_threads(n: int) -> None:
    lib().msdo_set_threads(C.c_int(int(n)))


def bf16_bits_to_f64(x_bits):
    x_bits = np.asarray(x_bits, dtype=np.uint16)
    return (x_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_bf16(x64):
    x64 = _c(x64, np.float64)
    out = np.empty(x64.shape, np.uint16)
    lib().msdo_round_bf16(_p(x64), C.c_int64(x64.size), _p(out))
    return out


# --- offline quantizers ------------------------------------------------------
def quantize_weight_int8(w):
    w = _c(w, np.float32)
    N, K = w.shape
    wq = np.empty((N, K), np.int8)
    ws = np.empty(N, np.float32)
    lib().msdo_quantize_weight_int8(_p(w), C.c_int64(N), C.c_int64(K), _p(wq), _p(ws))
    return wq, ws


def quantize_weight_mxfp4(w):
    w = _c(w, np.float32)
    N, K = w.shape
    q = np.empty((N, K // 2), np.uint8)
    e = np.empty((N, K // 32), np.uint8)
    lib().msdo_quantize_weight_mxfp4(_p(w), C.c_int64(N), C.c_int64(K), _p(q), _p(e))
    return q, e


def quantize_rows_int8(x_bits):
    x_bits = _c(x_bits, np.uint16)
    D = x_bits.shape[-1]
    rows = x_bits.size // D
    q = np.empty(x_bits.shape, np.int8)
    s = np.empty(x_bits.shape[:-1], np.float32)
    lib().msdo_quantize_rows_int8(_p(x_bits), C.c_int64(rows), C.c_int64(D), _p(q), _p(s))
    return q, s


# --- decompositions ----------------------------------------------------------
# Scaling constants of the two passes: Eq. alpha / Eq. beta, and the "fractional scaling" pair of Sec. 3.3 (as FP32).
SCALING_DEFAULT = (127.0, 254.0)
SCALING_FRACTIONAL = (127.49, 254.98)


def decompose_int8(x_bits, fractional=False):
    x_bits = _c(x_bits, np.uint16)
    M, K = x_bits.shape
    q1 = np.empty((M, K), np.int8)
    q2 = np.empty((M, K), np.int8)
    a = np.empty(M, np.float32)
    b = np.empty(M, np.float32)
    c1, c2 = SCALING_FRACTIONAL if fractional else SCALING_DEFAULT
    lib().msdo_decompose_int8_c(_p(x_bits), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_float(c1), C.c_float(c2),
                                _p(q1), _p(q2), _p(a), _p(b))
    return q1, q2, a, b


def decompose_int8_f32(x, alpha_fixed=-1.0):
    x = _c(x, np.float32)
    M, K = x.shape
    q1 = np.empty((M, K), np.int8)
    q2 = np.empty((M, K), np.int8)
    a = np.empty(M, np.float32)
    b = np.empty(M, np.float32)
    lib().msdo_decompose_int8_f32(_p(x), C.c_int64(M), C.c_int64(K), C.c_float(alpha_fixed), _p(q1), _p(q2), _p(a), _p(b))
    return q1, q2, a, b


def decompose_mxfp4(x_bits, grid=GRID_E2M1, c_bound=E2M1_RULE[0], beta_shift=E2M1_RULE[1]):
    x_bits = _c(x_bits, np.uint16)
    M, K = x_bits.shape
    assert K % 32 == 0
    q1 = np.empty((M, K // 2), np.uint8)
    q2 = np.empty((M, K // 2), np.uint8)
    e1 = np.empty((M, K // 32), np.uint8)
    e2 = np.empty((M, K // 32), np.uint8)
    lib().msdo_decompose_mxfp4(_p(x_bits), C.c_int64(M), C.c_int64(K), C.c_int64(K), C.c_int(grid),
                               C.c_double(c_bound), C.c_int(beta_shift), _p(q1), _p(q2), _p(e1), _p(e2))
    return q1, q2, e1, e2


def mxfp4_reconstruct(q1, q2, e1, e2, grid=GRID_E2M1):
    q1 = _c(q1, np.uint8)
    M, K2 = q1.shape
    K = 2 * K2
    out = np.empty((M, K), np.float64)
    q2c = None if q2 is None else _c(q2, np.uint8)
    e2c = None if e2 is None else _c(e2, np.uint8)
    e1 = _c(e1, np.uint8)
    lib().msdo_mxfp4_reconstruct(_p(q1), _p(q2c), _p(e1), _p(e2c), C.c_int64(M), C.c_int64(K), C.c_int(grid), _p(out))
    return out


def mxfp8_quantize(x_bits):
    x_bits = _c(x_bits, np.uint16)
    M, K = x_bits.shape
    out = np.empty((M, K), np.float64)
    lib().msdo_mxfp8_quantize(_p(x_bits), C.c_int64(M), C.c_int64(K), C.c_int64(K), _p(out))
    return out


# --- GEMMs ---------------------------------------------------------------------
def int8_gemm_acc(a, w):
    a = _c(a, np.int8)
    w = _c(w, np.int8)
    M, K = a.shape
    N = w.shape[0]
    acc = np.empty((M, N), np.int32)
    ov = lib().msdo_int8_gemm_acc(_p(a), _p(w), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(acc))
    assert ov == 0, "INT32 accumulator overflow"
    return acc


_YT = {"bf16": (0, np.uint16), "f32": (1, np.float32), "f64": (2, np.float64)}


def gemm_w8a16(x_bits, w, w_scale, ytype="f64", want_acc=False, fractional=False):
    x_bits = _c(x_bits, np.uint16)
    w = _c(w, np.int8)
    w_scale = _c(w_scale, np.float32)
    M, K = x_bits.shape
    N = w.shape[0]
    code, dt = _YT[ytype]
    y = np.empty((M, N), dt)
    acc = np.empty((2, M, N), np.int32) if want_acc else None
    c1, c2 = SCALING_FRACTIONAL if fractional else SCALING_DEFAULT
    ov = lib().msdo_gemm_w8a16_c(_p(x_bits), _p(w), _p(w_scale), C.c_int64(M), C.c_int64(N), C.c_int64(K), C.c_float(c1),
                                 C.c_float(c2), _p(y), C.c_int(code), _p(acc))
    assert ov == 0, "INT32 accumulator overflow"
    return (y, acc) if want_acc else y


def gemm_ref_w8(x_bits, w, w_scale):
    x_bits = _c(x_bits, np.uint16)
    w = _c(w, np.int8)
    w_scale = _c(w_scale, np.float32)
    M, K = x_bits.shape
    N = w.shape[0]
    y = np.empty((M, N), np.float64)
    lib().msdo_gemm_ref_w8(_p(x_bits), _p(w), _p(w_scale), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(y))
    return y


def gemm_dequant_bf16_w8(x_bits, w, w_scale):
    x_bits = _c(x_bits, np.uint16)
    w = _c(w, np.int8)
    w_scale = _c(w_scale, np.float32)
    M, K = x_bits.shape
    N = w.shape[0]
    y = np.empty((M, N), np.float64)
    lib().msdo_gemm_dequant_bf16_w8(_p(x_bits), _p(w), _p(w_scale), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(y))
    return y


def gemm_w4a16(x_bits, w_fp4, w_e8m0, ytype="f64", mode="msd", grid=GRID_E2M1, c_bound=E2M1_RULE[0],
               beta_shift=E2M1_RULE[1]):
    """mode: 'msd' two-pass MXFP4 activations, 'mxfp8' single-pass MXFP8 activations, 'ref' unquantized."""
    x_bits = _c(x_bits, np.uint16)
    w_fp4 = _c(w_fp4, np.uint8)
    w_e8m0 = _c(w_e8m0, np.uint8)
    M, K = x_bits.shape
    N = w_fp4.shape[0]
    code, dt = _YT[ytype]
    y = np.empty((M, N), dt)
    m = {"msd": 0, "mxfp8": 1, "ref": 2}[mode]
    lib().msdo_gemm_w4a16(_p(x_bits), _p(w_fp4), _p(w_e8m0), C.c_int64(M), C.c_int64(N), C.c_int64(K), C.c_int(grid),
                          C.c_double(c_bound), C.c_int(beta_shift), C.c_int(m), _p(y), C.c_int(code))
    return y


# --- attention -------------------------------------------------------------------
_ATTN_MODE = {"global": 0, "tiled": 1, "ref": 2, "dequant": 3, "held": 4}


def attn_decode_int8kv(q_bits, k, v, k_scale, v_scale, cu_seqlens, softmax_scale, dv=None, mode="global", tile=0,
                       split_starts=None, want_lse=False, want_s=False, m_margin=0.0, sv_growth=1.0):
    """Decode attention over an INT8 KV cache (Alg. 3, one scale per token per KV head).

    mode: 'global' (definition), 'tiled' (mirrors a tile/split schedule), 'ref' (FP64, no MSD),
    'dequant' (KV -> BF16 comparison path), 'held' (tiled, but the reference maximum and the probability scale
    move only when exceeded: to the tile maximum + ``m_margin`` (natural-log units) and to ``sv_growth`` times the
    tile's largest value scale).  ``v=None`` means V is the first ``dv`` entries of each K row.
    ``split_starts`` ([B, n_splits+1] token offsets relative to each sequence, or [B, Hq, n_splits+1] when the splits
    differ between the query heads) is used by 'tiled' and 'held'.
    """
    q_bits = _c(q_bits, np.uint16)
    B, Hq, D = q_bits.shape
    k = _c(k, np.int8)
    T, Hkv, _ = k.shape
    if v is not None:
        v = _c(v, np.int8)
        dv = v.shape[2]
    assert dv is not None
    k_scale = _c(k_scale, np.float32)
    v_scale = None if v_scale is None else _c(v_scale, np.float32)
    cu = _c(cu_seqlens, np.int32)
    out = np.empty((B, Hq, dv), np.float64)
    lse = np.empty((B, Hq), np.float64) if want_lse else None
    sdbg = np.zeros((2, Hq, T), np.int32) if want_s else None
    m = _ATTN_MODE[mode]
    ns, ss = 0, None
    if m in (1, 4):
        ss = _c(split_starts, np.int32)
        assert ss.shape[:-1] in ((B,), (B, Hq)), ss.shape
        ns = ss.shape[-1] - 1
    lib().msdo_attn_decode_int8kv(_p(q_bits), _p(k), _p(v), _p(k_scale), _p(v_scale), _p(cu), C.c_int32(B),
                                  C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(D), C.c_int32(dv),
                                  C.c_float(softmax_scale), C.c_int(m), C.c_int32(tile), _p(ss), C.c_int32(ns),
                                  _p(out), _p(lse), _p(sdbg), C.c_double(m_margin), C.c_float(sv_growth),
                                  C.c_int32(1 if m in (1, 4) and ss.ndim == 3 else 0))
    res = [out]
    if want_lse:
        res.append(lse)
    if want_s:
        res.append(sdbg)
    return res[0] if len(res) == 1 else tuple(res)
