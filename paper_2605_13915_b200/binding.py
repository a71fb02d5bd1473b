"""Thin ctypes binding of the C ABI in ``include/msd.h``: argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams); every step of the path runs in
the library's kernels.  There is no fallback: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

MSD_OK = 0
OUT_BF16, OUT_FP32 = 0, 1
STATUS = {0: "MSD_OK", 1: "MSD_ERR_NULL_POINTER", 2: "MSD_ERR_BAD_SHAPE", 3: "MSD_ERR_BAD_ALIGNMENT",
          4: "MSD_ERR_UNSUPPORTED", 5: "MSD_ERR_WORKSPACE_TOO_SMALL", 6: "MSD_ERR_CUDA", 7: "MSD_ERR_TIMEOUT"}


class MsdError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)} ({lib().msd_status_string(code).decode()})")


_lib = None
_vp, _i64, _i32, _sz, _f32 = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t, C.c_float

_SIGS = {
    "msd_status_string": (C.c_char_p, [C.c_int]),
    "msd_last_device_status": (C.c_int, [_vp]),
    "msd_workspace_init": (C.c_int, [_vp, _sz, _vp]),
    "msd_decompose_int8": (C.c_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp]),
    "msd_decompose_int8_ex": (C.c_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, C.c_int, _vp]),
    "msd_decompose_mxfp4": (C.c_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp]),
    "msd_gemm_w8a16_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_w8a16": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _vp, _sz, _vp]),
    "msd_gemm_w8a16_ex": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_grouped_gemm_w8a16_workspace_bytes": (_sz, [_i64, _i32, _i32, _i64, _i64]),
    "msd_grouped_gemm_w8a16": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_grouped_gemm_w4a16_workspace_bytes": (_sz, [_i32, _i64, _i64]),
    "msd_grouped_gemm_w4a16": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_gemm_w8a16_noalloc": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp]),
    "msd_debug_set_trace": (None, [_vp]),
    "msd_debug_set_attn_trace": (None, [_vp]),
    "msd_gemm_w8a16_host_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_w8a16_host": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_gemm_dequant_bf16_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_dequant_bf16": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_gemm_w8a16_fused_dequant_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_w8a16_fused_dequant": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_gemm_w4a16_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_w4a16": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_w4a16_prepared_scales_bytes": (_sz, [_i32, _i64, _i64]),
    "msd_prepare_w4a16_scales": (C.c_int, [_vp, _i32, _i64, _i64, _vp, _vp]),
    "msd_gemm_w4a16_prepared": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_grouped_gemm_w4a16_prepared": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_attn_decode_int8kv_workspace_bytes": (_sz, [_i32] * 6),
    "msd_attn_decode_int8kv": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _i32, _i32, _i32, _i32, _f32, _vp, _vp,
                                         _vp, _sz, _vp]),
    "msd_attn_decode_schedule": (C.c_int, [_i32] * 6 + [C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)]),
    "msd_attn_decode_split_starts": (C.c_int, [_i32] * 9 + [C.c_void_p, C.c_void_p]),
    "msd_debug_attn_split_starts": (C.c_int, [_i32] * 9 + [C.c_void_p, C.c_void_p]),
    "msd_attn_decode_softmax_rule": (C.c_int, [_i32] * 6 + [C.POINTER(_f32), C.POINTER(_f32)]),
    "msd_debug_set_attn_dump": (None, [_vp, _vp, _vp]),
    "msd_debug_set_option": (C.c_int, [C.c_char_p, _i32]),
    "msd_debug_reset_options": (None, []),
    "msd_decompose_mxfp4_e1m2": (C.c_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _vp]),
    "msd_gemm_w4a16_e1m2_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "msd_gemm_w4a16_e1m2": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, C.c_int, _vp, _sz, _vp]),
    "msd_attn_decode_int8kv_spec": (C.c_int, [_vp] * 6 + [_i64, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _f32, _vp, _vp, _vp, _sz, _vp]),
    "msd_attn_decode_int8kv_paged": (C.c_int, [_vp] * 7 + [_i64, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _i32, _f32, _vp, _vp, _vp,
                                                _sz, _vp]),
    "msd_debug_timeout_selftest": (C.c_int, [_i64, _vp]),
    "msd_kv_dequant_bf16": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, _i32, _i32, C.c_void_p, C.c_void_p]),
    "msd_attn_decode_bf16kv_workspace_bytes": (_sz, [_i32] * 6),
    "msd_attn_decode_bf16kv": (C.c_int, [_vp, _vp, _vp, _vp, _i64] + [_i32] * 6 + [_f32, _vp, _vp, _vp, _sz, _vp]),
}


def lib():
    """Loads ``libmsd.so`` (building it when the sources are newer); raises when that is impossible."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if _build.needs_build():
            path = _build.build()
        if not os.path.exists(path):
            raise RuntimeError("libmsd.so is missing and could not be built; there is no fallback path")
        h = C.CDLL(path)
        for name, (res, args) in _SIGS.items():
            fn = getattr(h, name)
            fn.restype = res
            fn.argtypes = args
        _lib = h
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code, where):
    if code != MSD_OK:
        raise MsdError(code, where)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("expected contiguous CUDA tensors")


def last_device_status():
    _check(lib().msd_last_device_status(_stream()), "msd_last_device_status")


def _raw_empty(shape, dtype, device):
    return torch.empty(shape, dtype=dtype, device=device)


def _raw_workspace(nbytes, device="cuda"):
    return torch.zeros(max(int(nbytes), 1024) + 1024, dtype=torch.uint8, device=device)


# Every output tensor and workspace the wrappers create comes from these two hooks, so that a test harness can swap in
# an allocator of its own (guard bands around each buffer).
_empty = _raw_empty
_workspace = _raw_workspace


def workspace(nbytes, device="cuda"):
    """A zero-filled, 1024-byte aligned workspace of at least ``nbytes`` bytes."""
    return _workspace(nbytes, device)


def _ws_ptr(ws):
    base = ws.data_ptr()
    al = (base + 1023) // 1024 * 1024
    return C.c_void_p(al), ws.numel() - (al - base)


SCALING_DEFAULT, SCALING_FRACTIONAL = 0, 1


def decompose_int8(x, fractional=False):
    """x [M,K] bfloat16 -> (q1, q2 int8 [M,K], alpha, beta float32 [M]); fractional: scaling constants 127.49 / 254.98."""
    _need_cuda(x)
    M, K = x.shape
    q1 = _empty((M, K), torch.int8, x.device)
    q2 = _empty((M, K), torch.int8, x.device)
    a = _empty(M, torch.float32, x.device)
    b = _empty(M, torch.float32, x.device)
    if fractional:
        _check(lib().msd_decompose_int8_ex(_ptr(x), M, K, x.stride(0) if M else K, _ptr(q1), _ptr(q2), _ptr(a), _ptr(b),
                                           SCALING_FRACTIONAL, _stream()), "msd_decompose_int8_ex")
        return q1, q2, a, b
    _check(lib().msd_decompose_int8(_ptr(x), M, K, x.stride(0) if M else K, _ptr(q1), _ptr(q2), _ptr(a), _ptr(b), _stream()),
           "msd_decompose_int8")
    return q1, q2, a, b


def decompose_mxfp4(x):
    """x [M,K] bfloat16 -> (q1, q2 uint8 [M,K/2], e8m0_1, e8m0_2 uint8 [M,K/32])."""
    _need_cuda(x)
    M, K = x.shape
    q1 = _empty((M, K // 2), torch.uint8, x.device)
    q2 = _empty((M, K // 2), torch.uint8, x.device)
    e1 = _empty((M, K // 32), torch.uint8, x.device)
    e2 = _empty((M, K // 32), torch.uint8, x.device)
    _check(lib().msd_decompose_mxfp4(_ptr(x), M, K, x.stride(0) if M else K, _ptr(q1), _ptr(q2), _ptr(e1), _ptr(e2), _stream()),
           "msd_decompose_mxfp4")
    return q1, q2, e1, e2


def gemm_w8a16_workspace_bytes(M, N, K):
    return int(lib().msd_gemm_w8a16_workspace_bytes(M, N, K))


def gemm_w8a16(x, w, w_scale, out_dtype=torch.bfloat16, ws=None, want_acc=False, out=None, fractional=False):
    """x [M,K] bf16, w [N,K] int8, w_scale [N] f32 -> y [M,N] (bf16 or f32); optional INT32 accumulators [2,M,N]."""
    _need_cuda(x, w, w_scale)
    M, K = x.shape
    N = w.shape[0]
    if ws is None:
        ws = workspace(gemm_w8a16_workspace_bytes(M, N, K), x.device)
    y = out if out is not None else _empty((M, N), out_dtype, x.device)
    acc = _empty((2, M, N), torch.int32, x.device) if want_acc else None
    wp, wb = _ws_ptr(ws)
    yt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32
    if fractional:
        code = lib().msd_gemm_w8a16_ex(_ptr(x), _ptr(w), _ptr(w_scale), M, N, K, _ptr(y), yt, _ptr(acc), SCALING_FRACTIONAL, wp, wb,
                                       _stream())
    else:
        code = lib().msd_gemm_w8a16(_ptr(x), _ptr(w), _ptr(w_scale), M, N, K, _ptr(y), yt, _ptr(acc), wp, wb, _stream())
    _check(code, "msd_gemm_w8a16")
    return (y, acc) if want_acc else y


def grouped_gemm_w8a16(x, w, w_scale, group_sizes, out_dtype=torch.bfloat16, ws=None, out=None):
    """MoE experts: x [M_total,K] bf16 with rows sorted by expert, w [E,N,K] int8, w_scale [E,N] f32, group_sizes: E host ints
    (rows per expert, each <= 128) -> y [M_total,N]."""
    _need_cuda(x, w, w_scale)
    E, N, K = w.shape
    sizes = (C.c_int32 * E)(*[int(v) for v in group_sizes])
    M_total = int(sum(int(v) for v in group_sizes))
    assert x.shape[0] == M_total and x.shape[1] == K
    if ws is None:
        ws = workspace(int(lib().msd_grouped_gemm_w8a16_workspace_bytes(M_total, max(int(v) for v in group_sizes), E, N, K)), x.device)
    y = out if out is not None else _empty((M_total, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    code = lib().msd_grouped_gemm_w8a16(_ptr(x), _ptr(w), _ptr(w_scale), C.cast(sizes, C.c_void_p), E, N, K, _ptr(y),
                                        OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream())
    _check(code, "msd_grouped_gemm_w8a16")
    return y


def grouped_gemm_w4a16(x, w_fp4, w_e8m0, group_sizes, out_dtype=torch.bfloat16, ws=None, out=None, prepared=None):
    """MoE experts with MXFP4 weights: x [M_total,K] bf16 with rows sorted by expert, w_fp4 [E,N,K/2] u8, w_e8m0 [E,N,K/32] u8,
    group_sizes: E host ints (rows per expert, each <= 128) -> y [M_total,N].
    prepared: the result of prepare_w4a16_scales(w_e8m0); w_e8m0 may then be None."""
    _need_cuda(x, w_fp4, prepared if prepared is not None else w_e8m0)
    E, N, K2 = w_fp4.shape
    K = 2 * K2
    sizes = (C.c_int32 * E)(*[int(v) for v in group_sizes])
    M_total = int(sum(int(v) for v in group_sizes))
    assert x.shape[0] == M_total and x.shape[1] == K
    if ws is None:
        ws = workspace(int(lib().msd_grouped_gemm_w4a16_workspace_bytes(E, N, K)), x.device)
    y = out if out is not None else _empty((M_total, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    if prepared is not None:
        code = lib().msd_grouped_gemm_w4a16_prepared(_ptr(x), _ptr(w_fp4), _ptr(prepared), sizes, E, N, K, _ptr(y),
                                                     OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream())
    else:
        code = lib().msd_grouped_gemm_w4a16(_ptr(x), _ptr(w_fp4), _ptr(w_e8m0), sizes, E, N, K, _ptr(y),
                                            OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream())
    _check(code, "msd_grouped_gemm_w4a16")
    return y


def gemm_w8a16_noalloc(x, w, w_scale, out):
    """W8A16 layer through the entry point that owns its scratch (for callers that may not allocate device memory):
    the caller passes inputs and a preallocated output only.  M <= 16, N <= 16384, K <= 16384."""
    _need_cuda(x, w, w_scale, out)
    M, K = x.shape
    N = w.shape[0]
    code = lib().msd_gemm_w8a16_noalloc(_ptr(x), _ptr(w), _ptr(w_scale), M, N, K, _ptr(out),
                                        OUT_BF16 if out.dtype == torch.bfloat16 else OUT_FP32, _stream())
    _check(code, "msd_gemm_w8a16_noalloc")
    return out


def gemm_w8a16_host_workspace_bytes(M, N, K):
    return int(lib().msd_gemm_w8a16_host_workspace_bytes(M, N, K))


def gemm_w8a16_host(x_host, w, w_scale, y_host, ws):
    """Activations and result in pinned host memory; weights resident on the device."""
    M, K = x_host.shape
    N = w.shape[0]
    wp, wb = _ws_ptr(ws)
    code = lib().msd_gemm_w8a16_host(_ptr(x_host), _ptr(w), _ptr(w_scale), M, N, K, _ptr(y_host),
                                     OUT_BF16 if y_host.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream())
    _check(code, "msd_gemm_w8a16_host")
    return y_host


def gemm_dequant_bf16_workspace_bytes(M, N, K):
    return int(lib().msd_gemm_dequant_bf16_workspace_bytes(M, N, K))


def gemm_dequant_bf16(x, w, w_scale, out_dtype=torch.bfloat16, ws=None):
    _need_cuda(x, w, w_scale)
    M, K = x.shape
    N = w.shape[0]
    if ws is None:
        ws = workspace(gemm_dequant_bf16_workspace_bytes(M, N, K), x.device)
    y = _empty((M, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    _check(lib().msd_gemm_dequant_bf16(_ptr(x), _ptr(w), _ptr(w_scale), M, N, K, _ptr(y),
                                       OUT_BF16 if out_dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream()),
           "msd_gemm_dequant_bf16")
    return y


def gemm_w8a16_fused_dequant(x, w, w_scale, out_dtype=torch.bfloat16, ws=None, out=None):
    """Comparison kernel: INT8 weights converted to BF16 inside the GEMM (M <= 128)."""
    _need_cuda(x, w, w_scale)
    M, K = x.shape
    N = w.shape[0]
    if ws is None:
        ws = workspace(max(1024, int(lib().msd_gemm_w8a16_fused_dequant_workspace_bytes(M, N, K))), x.device)
    y = out if out is not None else _empty((M, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    _check(lib().msd_gemm_w8a16_fused_dequant(_ptr(x), _ptr(w), _ptr(w_scale), M, N, K, _ptr(y),
                                              OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream()),
           "msd_gemm_w8a16_fused_dequant")
    return y


def gemm_w4a16_workspace_bytes(M, N, K):
    return int(lib().msd_gemm_w4a16_workspace_bytes(M, N, K))


def prepare_w4a16_scales(w_e8m0):
    """Blocked form of the E8M0 weight scales [N,K/32] (or [E,N,K/32]), made once per weight; pass it as `prepared`."""
    _need_cuda(w_e8m0)
    E = w_e8m0.shape[0] if w_e8m0.dim() == 3 else 1
    N, KB = w_e8m0.shape[-2], w_e8m0.shape[-1]
    nbytes = int(lib().msd_w4a16_prepared_scales_bytes(E, N, 32 * KB))
    if nbytes == 0:
        raise ValueError("msd_w4a16_prepared_scales_bytes: unsupported shape")
    buf = workspace(nbytes + 1024, w_e8m0.device)
    off = (-buf.data_ptr()) % 1024
    prepared = buf[off:off + nbytes]          # a view that starts on a 1024-byte boundary
    _check(lib().msd_prepare_w4a16_scales(_ptr(w_e8m0), E, N, 32 * KB, _ptr(prepared), _stream()), "msd_prepare_w4a16_scales")
    return prepared


def gemm_w4a16(x, w_fp4, w_e8m0, out_dtype=torch.bfloat16, ws=None, out=None, prepared=None):
    """prepared: the result of prepare_w4a16_scales(w_e8m0); w_e8m0 may then be None."""
    _need_cuda(x, w_fp4, prepared if prepared is not None else w_e8m0)
    M, K = x.shape
    N = w_fp4.shape[0]
    if ws is None:
        ws = workspace(gemm_w4a16_workspace_bytes(M, N, K), x.device)
    y = out if out is not None else _empty((M, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    yt = OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32
    if prepared is not None:
        _check(lib().msd_gemm_w4a16_prepared(_ptr(x), _ptr(w_fp4), _ptr(prepared), M, N, K, _ptr(y), yt, wp, wb, _stream()),
               "msd_gemm_w4a16_prepared")
    else:
        _check(lib().msd_gemm_w4a16(_ptr(x), _ptr(w_fp4), _ptr(w_e8m0), M, N, K, _ptr(y), yt, wp, wb, _stream()), "msd_gemm_w4a16")
    return y


def attn_decode_schedule(B, Hq, Hkv, D, Dv, max_seqlen):
    tile, ns, st = _i32(0), _i32(0), _i32(0)
    _check(lib().msd_attn_decode_schedule(B, Hq, Hkv, D, Dv, max_seqlen, C.byref(tile), C.byref(ns), C.byref(st)),
           "msd_attn_decode_schedule")
    return tile.value, ns.value, st.value


def attn_decode_split_starts(seqlens, Hq, Hkv, D, Dv, max_seqlen, q_len=1, paged=False, v_aliased=False, resident_ctas=None):
    """Context splits of a call with these sequence lengths: int32 array [B, Hkv, q_len * Hq // Hkv, n_splits + 1] of
    token offsets (see msd_attn_decode_split_starts), plus the tile size.  resident_ctas: take that many CTAs for the
    balanced schedule's grid instead of asking the device (host arithmetic only)."""
    import numpy as np
    L = np.ascontiguousarray(seqlens, dtype=np.int32)
    B = int(L.shape[0])
    tile, ns, _ = attn_decode_schedule(B, Hq * q_len, Hkv, D, Dv, max(int(max_seqlen), 1))
    starts = np.zeros((B, Hkv, q_len * Hq // Hkv, ns + 1), dtype=np.int32)
    if resident_ctas is None:
        _check(lib().msd_attn_decode_split_starts(B, q_len, Hq, Hkv, D, Dv, max(int(max_seqlen), 1), int(paged), int(v_aliased),
                                                  L.ctypes.data, starts.ctypes.data), "msd_attn_decode_split_starts")
    else:
        _check(lib().msd_debug_attn_split_starts(B, q_len, Hq, Hkv, D, Dv, max(int(max_seqlen), 1), int(v_aliased),
                                                 int(resident_ctas), L.ctypes.data, starts.ctypes.data), "msd_debug_attn_split_starts")
    return starts, tile


def attn_decode_softmax_rule(B, Hq, Hkv, D, Dv, max_seqlen):
    """(m_margin in natural-log units, sv_growth) of the held softmax references the kernel for this shape uses;
    (0, 0): plain running maximum and each tile's own probability scale."""
    m, g = _f32(0), _f32(0)
    _check(lib().msd_attn_decode_softmax_rule(B, Hq, Hkv, D, Dv, max_seqlen, C.byref(m), C.byref(g)), "msd_attn_decode_softmax_rule")
    return m.value, g.value


def debug_set_option(name, value):
    """Sets one of the library's testing / diagnostic switches (the names of msd.h, e.g. "MSD_GEMM_MODE"); -1 unsets it."""
    _check(lib().msd_debug_set_option(name.encode(), int(value)), "msd_debug_set_option")


def debug_reset_options():
    """Back to what the environment says (unset where it says nothing)."""
    lib().msd_debug_reset_options()


def debug_set_attn_dump(q_dbg=None, q_scale_dbg=None, s_dbg=None):
    """Attention launches that follow write the query components [2,rows,D] int8, their scales [2,rows] f32 and the raw
    QK^T sums [2,rows per sequence,T] int32 into these tensors; call without arguments to switch the dumps off."""
    lib().msd_debug_set_attn_dump(_ptr(q_dbg), _ptr(q_scale_dbg), _ptr(s_dbg))


def decompose_mxfp4_e1m2(x):
    """x [M,K] bfloat16 -> (q1, q2 uint8 [M,K] E4M3 bytes of the E1M2 components, e8m0_1, e8m0_2 uint8 [M,K/32])."""
    _need_cuda(x)
    M, K = x.shape
    q1 = _empty((M, K), torch.uint8, x.device)
    q2 = _empty((M, K), torch.uint8, x.device)
    e1 = _empty((M, K // 32), torch.uint8, x.device)
    e2 = _empty((M, K // 32), torch.uint8, x.device)
    _check(lib().msd_decompose_mxfp4_e1m2(_ptr(x), M, K, x.stride(0) if M else K, _ptr(q1), _ptr(q2), _ptr(e1), _ptr(e2), _stream()),
           "msd_decompose_mxfp4_e1m2")
    return q1, q2, e1, e2


def gemm_w4a16_e1m2(x, w_fp4, w_e8m0, out_dtype=torch.bfloat16, ws=None, out=None):
    """W4A16 with the paper-literal E1M2 components (FP8-rate tensor-core path)."""
    _need_cuda(x, w_fp4, w_e8m0)
    M, K = x.shape
    N = w_fp4.shape[0]
    if ws is None:
        ws = workspace(int(lib().msd_gemm_w4a16_e1m2_workspace_bytes(M, N, K)), x.device)
    y = out if out is not None else _empty((M, N), out_dtype, x.device)
    wp, wb = _ws_ptr(ws)
    code = lib().msd_gemm_w4a16_e1m2(_ptr(x), _ptr(w_fp4), _ptr(w_e8m0), M, N, K, _ptr(y),
                                     OUT_BF16 if y.dtype == torch.bfloat16 else OUT_FP32, wp, wb, _stream())
    _check(code, "msd_gemm_w4a16_e1m2")
    return y


def attn_decode_int8kv_spec(q, k, v, k_scale, v_scale, cu_seqlens, max_seqlen, softmax_scale, dv=None, ws=None, want_lse=False):
    """q [B,Sq,Hq,D] bf16: the last Sq tokens of every sequence query its cache causally -> out [B,Sq,Hq,Dv]."""
    _need_cuda(q, k, v, k_scale, v_scale, cu_seqlens)
    B, Sq, Hq, D = q.shape
    Hkv = k.shape[1]
    Dv = v.shape[2] if v is not None else int(dv)
    if ws is None:
        ws = workspace(attn_decode_int8kv_workspace_bytes(B, Hq * Sq, Hkv, D, Dv, max_seqlen), q.device)
    o = _empty((B, Sq, Hq, Dv), torch.bfloat16, q.device)
    lse = _empty((B, Sq, Hq), torch.float32, q.device) if want_lse else None
    wp, wb = _ws_ptr(ws)
    code = lib().msd_attn_decode_int8kv_spec(_ptr(q), _ptr(k), _ptr(v), _ptr(k_scale), _ptr(v_scale), _ptr(cu_seqlens), int(k.shape[0]),
                                             max_seqlen, B, Sq, Hq, Hkv, D, Dv, softmax_scale, _ptr(o), _ptr(lse), wp, wb, _stream())
    _check(code, "msd_attn_decode_int8kv_spec")
    return (o, lse) if want_lse else o


def attn_decode_int8kv_paged(q, k, v, k_scale, v_scale, block_table, seqlens, page_size, max_seqlen, softmax_scale, dv=None,
                             ws=None, want_lse=False, out=None):
    """Paged cache: k [num_blocks*page, Hkv, D] int8, v likewise or None, scales [num_blocks*page, Hkv] f32,
    block_table [B, max_blocks] int32, seqlens [B] int32."""
    _need_cuda(q, k, v, k_scale, v_scale, block_table, seqlens)
    B, Hq, D = q.shape
    Hkv = k.shape[1]
    Dv = v.shape[2] if v is not None else dv
    nblk = k.shape[0] // page_size
    if ws is None:
        ws = workspace(attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, max_seqlen), q.device)
    o = out if out is not None else _empty((B, Hq, Dv), torch.bfloat16, q.device)
    lse = _empty((B, Hq), torch.float32, q.device) if want_lse else None
    wp, wb = _ws_ptr(ws)
    code = lib().msd_attn_decode_int8kv_paged(_ptr(q), _ptr(k), _ptr(v), _ptr(k_scale), _ptr(v_scale), _ptr(block_table), _ptr(seqlens),
                                              nblk, page_size, block_table.shape[1], max_seqlen, B, Hq, Hkv, D, Dv, softmax_scale,
                                              _ptr(o), _ptr(lse), wp, wb, _stream())
    _check(code, "msd_attn_decode_int8kv_paged")
    return (o, lse) if want_lse else o


def kv_dequant_bf16(cache, scale, out=None):
    """cache [T,H,D] int8, scale [T,H] f32 -> bf16(scale * cache) [T,H,D] (the comparison arm's cache expansion)."""
    _need_cuda(cache, scale)
    T, H, D = cache.shape
    if out is None:
        out = _empty((T, H, D), torch.bfloat16, cache.device)
    _check(lib().msd_kv_dequant_bf16(cache.data_ptr(), scale.data_ptr(), T, H, D, out.data_ptr(), _stream()),
           "msd_kv_dequant_bf16")
    return out


def attn_decode_bf16kv(q, k, v, cu_seqlens, max_seqlen, softmax_scale, ws=None, want_lse=False, out=None):
    """The comparison arm's attention: q [B,Hq,D], k [T,Hkv,D], v [T,Hkv,Dv] bf16 (e.g. from kv_dequant_bf16)."""
    _need_cuda(q, k, v, cu_seqlens)
    B, Hq, D = q.shape
    T, Hkv, Dv = v.shape
    if ws is None:
        ws = workspace(int(lib().msd_attn_decode_bf16kv_workspace_bytes(B, Hq, Hkv, D, Dv, max_seqlen)))
    if out is None:
        out = _empty((B, Hq, Dv), torch.bfloat16, q.device)
    lse = _empty((B, Hq), torch.float32, q.device) if want_lse else None
    wp, wb = _ws_ptr(ws)
    _check(lib().msd_attn_decode_bf16kv(_ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), T, max_seqlen, B, Hq, Hkv, D, Dv,
                                        float(softmax_scale), _ptr(out), None if lse is None else _ptr(lse), wp, wb, _stream()),
           "msd_attn_decode_bf16kv")
    return (out, lse) if want_lse else out


def attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, max_seqlen):
    return int(lib().msd_attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, max_seqlen))


def attn_decode_int8kv(q, k, v, k_scale, v_scale, cu_seqlens, max_seqlen, softmax_scale, dv=None, ws=None, want_lse=False,
                       out=None):
    """q [B,Hq,D] bf16; k [T,Hkv,D] int8; v [T,Hkv,Dv] int8 or None; scales [T,Hkv] f32; cu_seqlens [B+1] int32."""
    _need_cuda(q, k, v, k_scale, v_scale, cu_seqlens)
    B, Hq, D = q.shape
    Hkv = k.shape[1]
    Dv = v.shape[2] if v is not None else int(dv)
    if ws is None:
        ws = workspace(attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, max_seqlen), q.device)
    o = out if out is not None else _empty((B, Hq, Dv), torch.bfloat16, q.device)
    lse = _empty((B, Hq), torch.float32, q.device) if want_lse else None
    wp, wb = _ws_ptr(ws)
    code = lib().msd_attn_decode_int8kv(_ptr(q), _ptr(k), _ptr(v), _ptr(k_scale), _ptr(v_scale), _ptr(cu_seqlens), int(k.shape[0]),
                                        max_seqlen, B, Hq, Hkv, D, Dv, softmax_scale, _ptr(o), _ptr(lse), wp, wb, _stream())
    _check(code, "msd_attn_decode_int8kv")
    return (o, lse) if want_lse else o
