"""Seeded synthetic inputs shaped like the paper's workloads.

This module serves both the CUDA path and the CPU oracle and holds none of the method's
arithmetic: it draws activations / weights / KV tensors from seeded generators and applies the
*offline* quantizers that produce the method's inputs (INT8 per-channel weights, MXFP4 weights,
INT8 KV cache with one scale per token per KV head).  The oracle carries its own copy of the
offline quantizers; a CPU test checks that the two agree bit for bit.

Everything is numpy on the host.  BF16 values are ``uint16`` bit patterns.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def _rng(seed, stream=0):
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def f32_to_bf16_bits(x):
    """Round-half-to-even conversion FP32 -> BF16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _normal_f32(rng, shape, std=1.0, chunk=1 << 24):
    """N(0, std) in FP32, drawn in chunks to bound the FP64 temporaries."""
    out = np.empty(int(np.prod(shape)), np.float32)
    for s in range(0, out.size, chunk):
        e = min(out.size, s + chunk)
        out[s:e] = rng.standard_normal(e - s, dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out.reshape(shape)


def activations(M, K, seed=0, outlier_frac=0.01, outlier_scale=50.0):
    """BF16 activations: N(0,1), then floor(K*outlier_frac) channels (seeded, without replacement)
    multiplied by ``outlier_scale`` in every row, then rounded to BF16."""
    rng = _rng(seed, 1)
    x = _normal_f32(rng, (M, K))
    n_out = int(K * outlier_frac)
    if n_out > 0:
        ch = _rng(seed, 2).choice(K, size=n_out, replace=False)
        x[:, ch] *= np.float32(outlier_scale)
    return f32_to_bf16_bits(x)


def weights_f32(N, K, seed=0, std=0.02):
    return _normal_f32(_rng(seed, 3), (N, K), std)


def quantize_weight_int8(w):
    """Symmetric INT8 per output channel: scale = rowmax/127 (FP32), RNE, clamp to +-127."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    m = np.abs(w).max(axis=1)
    s = (m / np.float32(127.0)).astype(np.float32)
    safe = np.where(s > 0, s, np.float32(1.0))
    q = np.rint(w / safe[:, None])
    q = np.clip(q, -127, 127).astype(np.int8)
    q[s == 0] = 0
    return q, s


_E2M1 = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])
# decision thresholds between neighbouring E2M1 codes; a tie goes to the even code
_E2M1_MID = (_E2M1[1:] + _E2M1[:-1]) / 2


def _round_e2m1_codes(s):
    a = np.abs(s)
    lo = np.searchsorted(_E2M1_MID, a, side="left")      # number of midpoints strictly below a
    hi = np.searchsorted(_E2M1_MID, a, side="right")     # number of midpoints <= a
    tie = hi != lo
    code = np.where(tie, np.where(lo % 2 == 0, lo, hi), lo)
    code = np.minimum(code, 7).astype(np.uint8)
    return code | (np.signbit(s).astype(np.uint8) << 3)


def quantize_weight_mxfp4(w):
    """MXFP4 weights: E2M1 values, one E8M0 scale per 32 contiguous K elements,
    scale = 2^(floor(log2(blockmax)) - 2), RNE with saturation; element 2i in the low nibble."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    blk = w.reshape(N, K // 32, 32).astype(np.float64)
    mb = np.abs(blk).max(axis=2)
    _, ex = np.frexp(mb)                         # mb = f * 2^ex, f in [0.5, 1) -> floor(log2) = ex-1
    e = np.where(mb > 0, ex - 1 - 2, -127)
    e = np.clip(e, -127, 127)
    s = np.ldexp(1.0, e)
    codes = _round_e2m1_codes(blk / s[:, :, None]).reshape(N, K)
    packed = (codes[:, 0::2] & 15) | ((codes[:, 1::2] & 15) << 4)
    return packed.astype(np.uint8), (e + 127).astype(np.uint8)


def quantize_rows_int8(x_bits):
    """INT8 rows with one symmetric scale each (KV cache: one scale per token per KV head)."""
    x = bf16_bits_to_f32(x_bits)
    m = np.abs(x).max(axis=-1)
    s = (m / np.float32(127.0)).astype(np.float32)
    safe = np.where(s > 0, s, np.float32(1.0))
    q = np.clip(np.rint(x / safe[..., None]), -127, 127).astype(np.int8)
    q[s == 0] = 0
    return q, s


@dataclass
class GemmW8Case:
    x: np.ndarray          # [M,K] BF16 bits
    w: np.ndarray          # [N,K] INT8
    w_scale: np.ndarray    # [N] FP32


def gemm_w8_case(M, N, K, seed=0):
    w, s = quantize_weight_int8(weights_f32(N, K, seed))
    return GemmW8Case(activations(M, K, seed), w, s)


@dataclass
class GemmW4Case:
    x: np.ndarray          # [M,K] BF16 bits
    w_fp4: np.ndarray      # [N,K/2] packed E2M1
    w_e8m0: np.ndarray     # [N,K/32]


def gemm_w4_case(M, N, K, seed=0):
    q, e = quantize_weight_mxfp4(weights_f32(N, K, seed))
    return GemmW4Case(activations(M, K, seed), q, e)


@dataclass
class AttnCase:
    q: np.ndarray           # [B,Hq,D] BF16 bits
    k: np.ndarray           # [T,Hkv,D] INT8
    v: np.ndarray | None    # [T,Hkv,Dv] INT8, or None when V is the first Dv entries of K rows
    k_scale: np.ndarray     # [T,Hkv] FP32
    v_scale: np.ndarray | None
    cu_seqlens: np.ndarray  # [B+1] int32
    dv: int
    softmax_scale: float

    @property
    def max_seqlen(self):
        return int(np.diff(self.cu_seqlens).max()) if len(self.cu_seqlens) > 1 else 0


def seqlens_uniform(B, lo, hi, seed=0):
    u = _rng(seed, 7).integers(0, 1 << 31, size=B)
    return (lo + (u % (hi - lo + 1))).astype(np.int32)


def gqa_case(B, Hq, Hkv, D, seqlens, seed=0):
    """GQA decode: Q, K, V ~ N(0,1) in BF16; K, V quantized to INT8, one scale per token per KV head."""
    seqlens = np.asarray(seqlens, dtype=np.int32)
    cu = np.zeros(B + 1, np.int32)
    cu[1:] = np.cumsum(seqlens)
    T = int(cu[-1])
    q = f32_to_bf16_bits(_normal_f32(_rng(seed, 4), (B, Hq, D)))
    k, ks = quantize_rows_int8(f32_to_bf16_bits(_normal_f32(_rng(seed, 5), (T, Hkv, D))))
    v, vs = quantize_rows_int8(f32_to_bf16_bits(_normal_f32(_rng(seed, 6), (T, Hkv, D))))
    return AttnCase(q, k, v, ks, vs, cu, D, float(1.0 / np.sqrt(D)))


def mla_case(B, Hq, D, Dv, seqlens, seed=0):
    """MLA-shaped decode: one latent KV head of width D; V is the first Dv entries of the same row."""
    seqlens = np.asarray(seqlens, dtype=np.int32)
    cu = np.zeros(B + 1, np.int32)
    cu[1:] = np.cumsum(seqlens)
    T = int(cu[-1])
    q = f32_to_bf16_bits(_normal_f32(_rng(seed, 4), (B, Hq, D)))
    k, ks = quantize_rows_int8(f32_to_bf16_bits(_normal_f32(_rng(seed, 5), (T, 1, D))))
    return AttnCase(q, k, None, ks, None, cu, Dv, float(1.0 / np.sqrt(D)))


def paginate(case, page_size, seed=0, spare_blocks=3):
    """Scatters a contiguous attention case into a paged cache: blocks of ``page_size`` tokens handed out in a seeded
    random order (as a serving allocator would after some churn), plus unused blocks filled with noise codes.

    Returns (k, v, k_scale, v_scale, block_table [B, max_blocks] int32, seqlens [B] int32); entries of the block table
    past a sequence's last block are -1 and must never be read."""
    seqlens = np.diff(case.cu_seqlens).astype(np.int32)
    B = len(seqlens)
    nblk_seq = (seqlens + page_size - 1) // page_size
    max_blocks = int(max(1, nblk_seq.max()))
    total = int(nblk_seq.sum()) + spare_blocks
    rng = _rng(seed, 11)
    order = rng.permutation(total)
    table = np.full((B, max_blocks), -1, np.int32)
    T, Hkv, D = case.k.shape
    k = rng.integers(-127, 128, size=(total * page_size, Hkv, D), dtype=np.int8)
    ks = (rng.random((total * page_size, Hkv), dtype=np.float32) + 0.5).astype(np.float32)
    v = vs = None
    if case.v is not None:
        v = rng.integers(-127, 128, size=(total * page_size, Hkv, case.v.shape[2]), dtype=np.int8)
        vs = (rng.random((total * page_size, Hkv), dtype=np.float32) + 0.5).astype(np.float32)
    nxt = 0
    for b in range(B):
        t0 = int(case.cu_seqlens[b])
        for j in range(int(nblk_seq[b])):
            blk = int(order[nxt]); nxt += 1
            table[b, j] = blk
            n = min(page_size, int(seqlens[b]) - j * page_size)
            src = slice(t0 + j * page_size, t0 + j * page_size + n)
            dst = slice(blk * page_size, blk * page_size + n)
            k[dst] = case.k[src]
            ks[dst] = case.k_scale[src]
            if v is not None:
                v[dst] = case.v[src]
                vs[dst] = case.v_scale[src]
    return k, v, ks, vs, table, seqlens
