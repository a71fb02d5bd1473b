"""Pins for the attention part of the CPU oracle (Alg. 3 with one scale per token per KV head).

Parity unpinned for the per-token-scale layout: the paper prints no number for it.  What holds the oracle
here: Alg. 3 written out literally in numpy for unit scales, closed-form special cases, the exact softmax on
the dequantized cache, and the ordering MSD error < dequantize-to-BF16 error.
"""
import numpy as np
import pytest

import oracle
from paper_2605_13915_b200 import inputs


def _alg3_literal(q_bits, k, v, scale, m_margin=0.0, a_ref=1.0):
    """Alg. 3 for one head with s_K = s_V = 1: decompose Q; S = (aS1 + bS2)/sqrt(d); P = exp(S - max);
    alpha_P = 1/127; decompose P; O = (alpha_P O1 + beta_P O2)/l.  m_margin / a_ref: the reference sits that far above
    the maximum and alpha_P = a_ref/127 (the held-reference reading; both cancel in O up to the quantisation of P)."""
    q = oracle.bf16_bits_to_f64(q_bits)
    M = np.abs(q).max()
    a = np.float32(M) / np.float32(127)
    q1 = np.clip(np.rint(q.astype(np.float32) / a), -128, 127)
    r = q - float(a) * q1
    b = a / np.float32(254)
    q2 = np.clip(np.rint(r.astype(np.float32) / b), -128, 127)
    S = (float(a) * (k.astype(np.int64) @ q1.astype(np.int64)) + float(b) * (k.astype(np.int64) @ q2.astype(np.int64))) * float(np.float32(scale))
    P = np.exp(S - (S.max() + m_margin))
    ap = np.float32(a_ref) / np.float32(127)
    bp = ap / np.float32(254)
    Pf = P.astype(np.float32)
    p1 = np.clip(np.rint(Pf / ap), -128, 127)
    rp = (Pf.astype(np.float64) - float(ap) * p1).astype(np.float32)
    p2 = np.clip(np.rint(rp / bp), -128, 127)
    O = float(ap) * (p1.astype(np.int64) @ v.astype(np.int64)) + float(bp) * (p2.astype(np.int64) @ v.astype(np.int64))
    return O / P.sum()


def test_reduces_to_alg3_with_unit_scales():
    rng = np.random.default_rng(0)
    L, D = 300, 64
    q = inputs.f32_to_bf16_bits(rng.standard_normal((1, 1, D)).astype(np.float32))
    k = rng.integers(-127, 128, (L, 1, D), dtype=np.int8)
    v = rng.integers(-127, 128, (L, 1, D), dtype=np.int8)
    ones = np.ones((L, 1), np.float32)
    scale = 0.01
    got = oracle.attn_decode_int8kv(q, k, v, ones, ones, [0, L], scale)
    want = _alg3_literal(q[0, 0], k[:, 0], v[:, 0], scale)
    assert np.allclose(got[0, 0], want, rtol=1e-9, atol=1e-9)


def test_closed_form_cases():
    rng = np.random.default_rng(1)
    D = 128
    q = inputs.f32_to_bf16_bits(rng.standard_normal((2, 4, D)).astype(np.float32))
    # (a) single-token context: O = s_V * V_0 (P = 1 maps to code 127 exactly)
    k = rng.integers(-127, 128, (2, 1, D), dtype=np.int8)
    v = rng.integers(-127, 128, (2, 1, D), dtype=np.int8)
    ks = np.array([[0.02], [0.03]], np.float32)
    vs = np.array([[0.5], [0.25]], np.float32)
    out, lse = oracle.attn_decode_int8kv(q, k, v, ks, vs, [0, 1, 2], 0.1, want_lse=True)
    for b in range(2):
        assert np.allclose(out[b], vs[b, 0] * v[b, 0].astype(np.float64)[None, :].repeat(4, 0), rtol=1e-6)
    # (b) all keys identical: every score equal, so O is the mean of the dequantized V rows
    L = 257
    k = np.repeat(rng.integers(-127, 128, (1, 1, D), dtype=np.int8), L, axis=0)
    v = rng.integers(-127, 128, (L, 1, D), dtype=np.int8)
    ks = np.full((L, 1), 0.01, np.float32)
    vs = rng.uniform(0.01, 0.02, (L, 1)).astype(np.float32)
    out = oracle.attn_decode_int8kv(q[:1], k, v, ks, vs, [0, L], 0.05)
    mean = (vs.astype(np.float64) * v[:, 0]).mean(axis=0)
    # P = 1 everywhere; error per element of P~ is at most alpha_P/508, alpha_P = max s_V / 127
    tol = (vs.max() / 127 / 508) * np.abs(v[:, 0].astype(np.float64)).sum(axis=0) / L
    assert np.all(np.abs(out[0] - mean[None, :]) <= tol[None, :] * 1.01 + 1e-12)
    # (c) empty sequence gives zeros and lse = -inf
    out, lse = oracle.attn_decode_int8kv(q[:1], k[:0], v[:0], ks[:0], vs[:0], [0, 0], 0.05, want_lse=True)
    assert not out.any() and np.all(np.isneginf(lse))


@pytest.fixture(scope="module")
def gqa_small():
    return inputs.gqa_case(3, 8, 2, 128, [700, 64, 1500], seed=3)


def test_msd_beats_dequant_bf16(gqa_small):
    c = gqa_small
    args = (c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale)
    ref, lse_ref = oracle.attn_decode_int8kv(*args, mode="ref", want_lse=True)
    msd, lse = oracle.attn_decode_int8kv(*args, mode="global", want_lse=True)
    deq = oracle.attn_decode_int8kv(*args, mode="dequant")
    n = np.linalg.norm(ref)
    e_msd, e_deq = np.linalg.norm(msd - ref) / n, np.linalg.norm(deq - ref) / n
    assert e_msd < 1e-3 and e_msd < 0.5 * e_deq, (e_msd, e_deq)
    assert np.allclose(lse, lse_ref, atol=1e-3)
    # reference softmax against a plain numpy statement for one head
    b, h = 2, 5
    t0, t1 = c.cu_seqlens[b], c.cu_seqlens[b + 1]
    kd = c.k[t0:t1, h // 4].astype(np.float64) * c.k_scale[t0:t1, h // 4, None]
    vd = c.v[t0:t1, h // 4].astype(np.float64) * c.v_scale[t0:t1, h // 4, None]
    s = kd @ oracle.bf16_bits_to_f64(c.q[b, h]) * float(np.float32(c.softmax_scale))
    p = np.exp(s - s.max())
    assert np.allclose(ref[b, h], p @ vd / p.sum(), rtol=1e-10, atol=1e-12)


def test_tiled_mode_tracks_definition(gqa_small):
    c = gqa_small
    args = (c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale)
    glob = oracle.attn_decode_int8kv(*args, mode="global")
    L = np.diff(c.cu_seqlens)
    # one split, one tile covering everything == the definition
    one = oracle.attn_decode_int8kv(*args, mode="tiled", tile=int(L.max()), split_starts=np.stack([0 * L, L], 1))
    assert np.allclose(one, glob, rtol=1e-12, atol=1e-14)
    # three uneven splits walked in 64-token tiles stay within 5e-4 of the row norm
    ss = np.stack([0 * L, L // 3, (2 * L) // 3 + 5, L], 1)
    tiled, lse_t = oracle.attn_decode_int8kv(*args, mode="tiled", tile=64, split_starts=ss, want_lse=True)
    _, lse_g = oracle.attn_decode_int8kv(*args, mode="global", want_lse=True)
    rown = np.linalg.norm(glob, axis=2, keepdims=True)
    assert np.abs(tiled - glob).max() <= 5e-4 * rown.max()
    assert np.all(np.abs(tiled - glob) <= 1e-3 * rown)
    assert np.allclose(lse_t, lse_g, rtol=0, atol=1e-9)
    # splits given per (sequence, head): the same per head as per sequence, and a head with splits of its own gets
    # exactly what a call with those splits for everybody gives that head
    B, Hq = c.q.shape[:2]
    per_head = np.repeat(ss[:, None, :], Hq, axis=1)
    assert np.array_equal(oracle.attn_decode_int8kv(*args, mode="tiled", tile=64, split_starts=per_head), tiled)
    other = np.stack([0 * L, L // 2, L // 2, L], 1)
    mixed = per_head.copy()
    mixed[:, 1] = other
    got = oracle.attn_decode_int8kv(*args, mode="tiled", tile=64, split_starts=mixed)
    alt = oracle.attn_decode_int8kv(*args, mode="tiled", tile=64, split_starts=other)
    assert np.array_equal(got[:, 1], alt[:, 1]) and np.array_equal(got[:, 0], tiled[:, 0]) and np.array_equal(got[:, 2:], tiled[:, 2:])
    assert not np.array_equal(alt[:, 1], tiled[:, 1])


def test_held_references_mode(gqa_small):
    """The tiled mode whose reference maximum and probability scale move only when exceeded (kernels that keep integer
    PV sums across tiles).  Pins: (a) one tile, unit scales: Alg. 3 written out in numpy with the reference m_margin
    above the maximum and alpha_P = sv_growth/127; (b) margin 0, growth 1 and equal value scales: bit for bit the plain
    tiled mode; (c) the margins the CUDA path uses stay within 5e-4 of the row norm of the untiled definition, and the
    log-sum-exp does not depend on them."""
    rng = np.random.default_rng(4)
    L, D = 200, 64
    q = inputs.f32_to_bf16_bits(rng.standard_normal((1, 1, D)).astype(np.float32))
    k = rng.integers(-127, 128, (L, 1, D), dtype=np.int8)
    v = rng.integers(-127, 128, (L, 1, D), dtype=np.int8)
    ones = np.ones((L, 1), np.float32)
    ss = np.array([[0, L]], np.int32)
    for margin, growth in ((0.0, 1.0), (1.3862943611198906, 1.25), (0.5, 2.0)):
        got = oracle.attn_decode_int8kv(q, k, v, ones, ones, [0, L], 0.01, mode="held", tile=L, split_starts=ss,
                                        m_margin=margin, sv_growth=growth)
        want = _alg3_literal(q[0, 0], k[:, 0], v[:, 0], 0.01, m_margin=margin, a_ref=growth)
        assert np.allclose(got[0, 0], want, rtol=1e-9, atol=1e-9), (margin, growth)
    c = gqa_small
    Ls = np.diff(c.cu_seqlens)
    ss = np.stack([0 * Ls, Ls // 3, (2 * Ls) // 3 + 5, Ls], 1)
    const_vs = np.full_like(c.v_scale, 0.0125)
    args = (c.q, c.k, c.v, c.k_scale, const_vs, c.cu_seqlens, c.softmax_scale)
    tiled = oracle.attn_decode_int8kv(*args, mode="tiled", tile=64, split_starts=ss)
    held0 = oracle.attn_decode_int8kv(*args, mode="held", tile=64, split_starts=ss, m_margin=0.0, sv_growth=1.0)
    assert np.array_equal(tiled, held0)
    args = (c.q, c.k, c.v, c.k_scale, c.v_scale, c.cu_seqlens, c.softmax_scale)
    glob, lse_g = oracle.attn_decode_int8kv(*args, mode="global", want_lse=True)
    held, lse_h = oracle.attn_decode_int8kv(*args, mode="held", tile=128, split_starts=ss, m_margin=2 * np.log(2.0),
                                            sv_growth=1.25, want_lse=True)
    rown = np.linalg.norm(glob, axis=2, keepdims=True)
    assert np.abs(held - glob).max() <= 5e-4 * rown.max()
    assert np.all(np.abs(held - glob) <= 1e-3 * rown)
    assert np.allclose(lse_h, lse_g, rtol=0, atol=1e-9)


def test_mla_shape_shares_rows_and_scores_are_exact_integers():
    c = inputs.mla_case(2, 4, 576, 512, [130, 77], seed=5)
    out, s = oracle.attn_decode_int8kv(c.q, c.k, None, c.k_scale, None, c.cu_seqlens, c.softmax_scale, dv=512, want_s=True)
    same = oracle.attn_decode_int8kv(c.q, c.k, np.ascontiguousarray(c.k[:, :, :512]), c.k_scale, c.k_scale, c.cu_seqlens, c.softmax_scale)
    assert np.array_equal(out, same)
    q1, q2, a, b = oracle.decompose_int8(c.q.reshape(-1, 576))
    b_, h = 1, 2
    t0, t1 = c.cu_seqlens[b_], c.cu_seqlens[b_ + 1]
    want1 = c.k[t0:t1, 0].astype(np.int64) @ q1[b_ * 4 + h].astype(np.int64)
    want2 = c.k[t0:t1, 0].astype(np.int64) @ q2[b_ * 4 + h].astype(np.int64)
    assert np.array_equal(s[0, h, t0:t1], want1) and np.array_equal(s[1, h, t0:t1], want2)


def test_vector_op_closed_forms():
    """Tab. attention-complexity closed forms reproduce Tab. decode-vector-examples (a reading check on N, M, d, T_c)."""
    import json, os
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_tables.json")))["tab_decode_vector_examples"]
    d, M, Bc = 128, 8192, 64
    Tc = M // Bc
    for N, key in ((1, "N1"), (32, "N32")):
        deq = 4 * M * d + 4 * N * M + 3 * N * d * Tc
        msd = 6 * N * d + 12 * N * M + 7 * N * d * Tc
        assert abs(deq / 1e6 - gold[key]["dequant"]) < 0.06 and abs(msd / 1e6 - gold[key]["msd"]) < 0.06
