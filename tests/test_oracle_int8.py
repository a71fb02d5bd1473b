"""Pins for the INT8 part of the CPU oracle (two-pass decomposition, exact GEMM, W8A16 layer).

Each test holds the oracle against something other than itself: the paper's theorems and printed
tables, exact integer arithmetic done with Python ints, and special inputs with a closed form.
"""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_13915_b200 import inputs

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_tables.json")))


def _x_rows(M, K, seed, outliers=True):
    return inputs.activations(M, K, seed, outlier_frac=0.01 if outliers else 0.0)


@pytest.mark.parametrize("outliers", [False, True])
def test_theorem1_bound_and_ranges(outliers):
    """Theorem 1: |x - alpha q1 - beta q2| <= M/64516 per element; pass 1 alone <= alpha/2."""
    xb = _x_rows(64, 4096, 3, outliers)
    q1, q2, a, b = oracle.decompose_int8(xb)
    x = oracle.bf16_bits_to_f64(xb)
    M = np.abs(x).max(axis=1)
    rec = a.astype(np.float64)[:, None] * q1 + b.astype(np.float64)[:, None] * q2
    bound = M / GOLD["thm1_int8_bound_divisor"]["value"]
    ratio = np.abs(x - rec).max(axis=1) / bound
    # slack covers the FP32 rounding of alpha, beta and r/beta
    assert ratio.max() <= 1.0 + 2.0 ** -15
    assert ratio.max() > 0.9                      # and the bound is nearly attained
    r1 = np.abs(x - a.astype(np.float64)[:, None] * q1).max(axis=1)
    assert np.all(r1 <= a.astype(np.float64) / 2 * (1 + 1e-4))   # slack: FP32 rounding of the quotient near a tie
    # zero clipping: both passes stay inside [-127, 127] (Discussion, "Clipping vs. Zero-Clipping Trade-off")
    assert q1.min() >= -127 and q1.max() <= 127 and q2.min() >= -127 and q2.max() <= 127
    # the row maximum maps to +-127 (Sec. 3.3 "the extremal element satisfies |x/alpha| = 127 exactly")
    assert np.all(np.abs(q1).max(axis=1) == 127)
    # scales: alpha = M/127, beta = alpha/254 (Eq. alpha, Eq. beta)
    assert np.allclose(a, M / 127, rtol=1e-6) and np.allclose(b, M / 127 / 254, rtol=1e-6)


def test_fractional_scaling_bound_and_extreme_element():
    """Sec. 3.3 "fractional scaling": alpha = M/127.49, beta = alpha/254.98 tightens the bound to M/65015
    (= 127.49 * 254.98 * 2), still without clipping; the extreme element maps to 127 with residual 0.49 alpha,
    i.e. second code round(0.49 * 254.98) = 125; and the default constants stay what they were."""
    xb = _x_rows(64, 4096, 5, True)
    x = oracle.bf16_bits_to_f64(xb)
    M = np.abs(x).max(axis=1)
    q1, q2, a, b = oracle.decompose_int8(xb, fractional=True)
    assert np.allclose(a, M / 127.49, rtol=2e-7) and np.allclose(b, a / 254.98, rtol=2e-7)
    rec = a.astype(np.float64)[:, None] * q1 + b.astype(np.float64)[:, None] * q2
    ratio = np.abs(x - rec).max(axis=1) / (M / (127.49 * 254.98 * 2.0))
    assert ratio.max() <= 1.0 + 2.0 ** -15 and ratio.max() > 0.9
    assert np.abs(q1).max() == 127 and np.abs(q2).max() <= 127
    for i in range(len(M)):
        k = int(np.argmax(np.abs(x[i])))
        assert abs(int(q1[i, k])) == 127 and abs(int(q2[i, k])) == 125
        assert np.sign(q2[i, k]) == np.sign(x[i, k])
    # the tighter bound shows in the data as well, and the default call is untouched by the new parameter
    d1, d2, da, db = oracle.decompose_int8(xb)
    assert np.array_equal(da, (M / 127.0).astype(np.float32)) or np.allclose(da, M / 127.0, rtol=2e-7)
    err_def = np.abs(x - (da.astype(np.float64)[:, None] * d1 + db.astype(np.float64)[:, None] * d2)).max(axis=1)
    assert np.mean(np.abs(x - rec).max(axis=1) / err_def) < 1.0
    # the GEMM with the flag is the stacked integer product of exactly these components
    c = inputs.gemm_w8_case(4, 64, 256, seed=9)
    y, acc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True, fractional=True)
    g1, g2, ga, gb = oracle.decompose_int8(c.x, fractional=True)
    w = c.w.astype(np.int64)
    assert np.array_equal(acc[0], g1.astype(np.int64) @ w.T) and np.array_equal(acc[1], g2.astype(np.int64) @ w.T)
    want = c.w_scale.astype(np.float64)[None, :] * (ga.astype(np.float64)[:, None] * acc[0] + gb.astype(np.float64)[:, None] * acc[1])
    assert np.allclose(y, want, rtol=1e-14, atol=0)


def test_special_rows():
    K = 256
    x = np.zeros((5, K), np.float32)
    x[1, 17] = 3.0                       # one-hot
    x[2, :] = -1.5                       # all equal
    x[3, :] = np.linspace(-2, 2, K)      # ramp
    x[4, 0] = 2.0 ** -100                # small magnitude
    xb = inputs.f32_to_bf16_bits(x)
    q1, q2, a, b = oracle.decompose_int8(xb)
    assert a[0] == 0 and b[0] == 0 and not q1[0].any() and not q2[0].any()
    assert q1[1, 17] == 127 and np.count_nonzero(q1[1]) == 1 and np.count_nonzero(q2[1]) <= 1
    assert np.all(q1[2] == -127) and np.all(np.abs(q2[2]) <= 1)
    assert q1[4, 0] == 127 and np.count_nonzero(q1[4]) == 1
    # monotone input -> monotone first component
    assert np.all(np.diff(q1[3].astype(int)) >= 0)


def test_exact_rational_small():
    """Brute force with exact rationals: the nearest integers to x/alpha and r/beta, ties to even."""
    rng = np.random.default_rng(5)
    xb = inputs.f32_to_bf16_bits(rng.standard_normal((8, 32)).astype(np.float32))
    q1, q2, a, b = oracle.decompose_int8(xb)
    x = inputs.bf16_bits_to_f32(xb)

    def rne(fr):
        fl = fr.numerator // fr.denominator
        rem = fr - fl
        if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
            fl += 1
        return fl

    for i in range(x.shape[0]):
        al, be = Fraction(float(a[i])), Fraction(float(b[i]))
        assert a[i] == np.float32(np.abs(x[i]).max()) / np.float32(127)
        assert b[i] == a[i] / np.float32(254)
        for k in range(x.shape[1]):
            xv = Fraction(float(x[i, k]))
            # the FP32 quotient is the correctly rounded exact quotient, so rounding it to an integer can
            # differ from rounding the exact quotient only when the exact quotient is within one FP32 ulp of
            # a half-integer; accept either neighbour there and require equality elsewhere.
            e1 = rne(xv / al)
            assert abs(int(q1[i, k]) - e1) <= (1 if abs((xv / al) % 1 - Fraction(1, 2)) < Fraction(1, 1 << 16) else 0)
            r = xv - al * int(q1[i, k])
            e2 = max(-128, min(127, rne(r / be)))
            assert abs(int(q2[i, k]) - e2) <= (1 if abs((r / be) % 1 - Fraction(1, 2)) < Fraction(1, 1 << 10) else 0)


def test_int8_gemm_bruteforce():
    rng = np.random.default_rng(11)
    a = rng.integers(-128, 128, (3, 70), dtype=np.int8)
    w = rng.integers(-128, 128, (5, 70), dtype=np.int8)
    acc = oracle.int8_gemm_acc(a, w)
    for i in range(3):
        for n in range(5):
            assert int(acc[i, n]) == sum(int(a[i, k]) * int(w[n, k]) for k in range(70))
    # extreme values do not overflow at the largest K used (14336)
    a = np.full((1, 14336), -128, np.int8)
    w = np.full((1, 14336), -128, np.int8)
    assert int(oracle.int8_gemm_acc(a, w)[0, 0]) == 14336 * 128 * 128


def test_w8a16_identity_weight():
    """W = 127*I with s_W = 1/127 gives y = alpha q1 + beta q2, i.e. x within the Theorem-1 bound."""
    K = 128
    xb = _x_rows(4, K, 9)
    w = (127 * np.eye(K)).astype(np.int8)
    ws = np.full(K, 1 / 127, np.float32)
    y, acc = oracle.gemm_w8a16(xb, w, ws, "f64", want_acc=True)
    q1, q2, a, b = oracle.decompose_int8(xb)
    assert np.array_equal(acc[0], 127 * q1.astype(np.int32)) and np.array_equal(acc[1], 127 * q2.astype(np.int32))
    x = oracle.bf16_bits_to_f64(xb)
    M = np.abs(x).max(axis=1, keepdims=True)
    assert np.all(np.abs(y - x) <= M / 64516 * (1 + 1e-4) + 1e-7 * M)


def test_w8a16_matches_definition_and_output_rounding():
    c = inputs.gemm_w8_case(3, 24, 256, seed=2)
    y64, acc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True)
    q1, q2, a, b = oracle.decompose_int8(c.x)
    # accumulators are the plain integer products of the components
    assert np.array_equal(acc[0], q1.astype(np.int64) @ c.w.astype(np.int64).T)
    assert np.array_equal(acc[1], q2.astype(np.int64) @ c.w.astype(np.int64).T)
    # MSD tracks the FP64 product with the dequantized weight far better than one INT8 pass
    ref = oracle.gemm_ref_w8(c.x, c.w, c.w_scale)
    nrm = np.linalg.norm(ref)
    assert np.linalg.norm(y64 - ref) / nrm < 2e-4
    y32 = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f32")
    assert np.array_equal(y32, y64.astype(np.float32))
    ybf = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "bf16")
    # one rounding to BF16: never further than half a BF16 ulp from the FP64 value
    back = oracle.bf16_bits_to_f64(ybf)
    assert np.all(np.abs(back - y64) <= np.abs(y64) * 2.0 ** -8)
    import torch
    assert np.array_equal(ybf.view(np.int16), torch.from_numpy(y64).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy()) or \
        np.mean(ybf.view(np.int16) != torch.from_numpy(y64).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy()) < 1e-2


def test_paper_ablation_table():
    """Tab. ablation: single scale 0.65 %, dequant-BF16 0.60 %, MSD (K=2) 0.003 % L2 on a 4096x4096 GEMM with
    random INT8 weights, s_W ~ U[0.01, 1] and Gaussian activations (Sec. 6.1 data generation)."""
    rng = np.random.default_rng(0)
    n = 4096
    w = rng.integers(-127, 128, (n, n), dtype=np.int8)
    ws = rng.uniform(0.01, 1.0, n).astype(np.float32)
    x32 = rng.standard_normal((8, n)).astype(np.float32)
    xb = inputs.f32_to_bf16_bits(x32)
    ref = oracle.gemm_ref_w8(xb, w, ws)
    nrm = np.linalg.norm(ref)
    msd = oracle.gemm_w8a16(xb, w, ws, "f64")
    l2_msd = 100 * np.linalg.norm(msd - ref) / nrm
    q1, q2, a, b = oracle.decompose_int8(xb)
    k1 = ws[None, :].astype(np.float64) * (a.astype(np.float64)[:, None] * oracle.int8_gemm_acc(q1, w))
    l2_k1 = 100 * np.linalg.norm(k1 - ref) / nrm
    t = GOLD["tab_ablation"]
    assert 0.6 * t["msd_k2_pct"] <= l2_msd <= 1.5 * t["msd_k2_pct"], l2_msd
    # the single-scale level depends on the max/std ratio of the rows drawn; same order as the table
    assert 0.7 * t["single_scale_k1_pct"] <= l2_k1 <= 1.4 * t["single_scale_k1_pct"], l2_k1
    # the dequantize-to-BF16 path sits at the single-scale level, two orders above MSD (the paper's 0.60 % also
    # counts the BF16 rounding of x itself, which this comparison leaves out by using the BF16 x as the truth)
    deq = oracle.gemm_dequant_bf16_w8(xb, w, ws)
    l2_deq = 100 * np.linalg.norm(deq - ref) / nrm
    assert 0.1 < l2_deq < 1.0 and l2_deq > 30 * l2_msd, l2_deq


def test_offline_quantizers_agree_with_input_module():
    w = inputs.weights_f32(48, 256, seed=4)
    q_o, s_o = oracle.quantize_weight_int8(w)
    q_i, s_i = inputs.quantize_weight_int8(w)
    assert np.array_equal(q_o, q_i) and np.array_equal(s_o, s_i)
    assert np.abs(q_o).max() == 127
    xb = inputs.activations(40, 128, seed=1)
    q_o, s_o = oracle.quantize_rows_int8(xb)
    q_i, s_i = inputs.quantize_rows_int8(xb)
    assert np.array_equal(q_o, q_i) and np.array_equal(s_o, s_i)
