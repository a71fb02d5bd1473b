"""Pins for the MXFP4 part of the CPU oracle: Theorem 2 and the paper's MXFP4 tables on the E1M2 grid the
paper states, and the exhaustive bounds of the same rule restated on the E2M1 grid the tensor cores multiply."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_13915_b200 import inputs

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_tables.json")))
E2M1 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
E1M2 = [0.0, 0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75]


def _codes(packed):
    out = np.empty((packed.shape[0], packed.shape[1] * 2), np.uint8)
    out[:, 0::2] = packed & 15
    out[:, 1::2] = packed >> 4
    return out


def _values(packed, grid):
    c = _codes(packed)
    v = np.array(grid)[c & 7]
    return np.where(c & 8, -v, v)


def _all_bf16_blocks(c_bound):
    """Blocks that pair every BF16 mantissa of the block maximum (binade [1,2)) with every positive BF16 value
    below it down to 2^-9 of the maximum: an exhaustive sweep of the ratios x/M_b the rule can meet."""
    maxima = (np.arange(0x3F80, 0x4000, dtype=np.uint32)).astype(np.uint16)            # 1.0 .. 1.992
    vals = np.arange(0x3B00, 0x4000, dtype=np.uint32).astype(np.uint16)                 # 2^-9 .. 1.992
    blocks = []
    for m in maxima:
        v = vals[vals <= m]
        pad = (-len(v)) % 31
        v = np.concatenate([v, np.full(pad, v[0], np.uint16)]).reshape(-1, 31)
        signs = (np.arange(v.size).reshape(v.shape) % 2).astype(np.uint16) << 15        # alternate signs
        blk = np.concatenate([np.full((v.shape[0], 1), m, np.uint16), v | signs], axis=1)
        blocks.append(blk)
    return np.concatenate(blocks, axis=0)


def test_theorem2_e1m2_exhaustive():
    """Theorem 2: with alpha = 2^ceil(log2(M_b/1.859375)), beta = alpha/16 on the E1M2 grid the pass-1 residual is
    <= alpha/8 and the final error <= alpha/64, and the bound is attained (Tab. mxfp4-bound: ratio up to 1.0000)."""
    c, sh = oracle.PAPER_E1M2
    xb = _all_bf16_blocks(c)
    q1, q2, e1, e2 = oracle.decompose_mxfp4(xb, oracle.GRID_E1M2, c, sh)
    x = oracle.bf16_bits_to_f64(xb)
    alpha = np.ldexp(1.0, e1.astype(int) - 127)
    assert np.all(e2.astype(int) == e1.astype(int) - 4)
    # alpha is the smallest power of two with M_b <= 1.859375 alpha (Eq. alpha-mxfp4)
    mb = np.abs(x).max(axis=1, keepdims=True)
    assert np.all(mb <= c * alpha) and np.all(mb > c * alpha / 2)
    r1 = x - oracle.mxfp4_reconstruct(q1, None, e1, None, oracle.GRID_E1M2)
    assert np.abs(r1 / alpha).max() <= 1 / GOLD["thm2_pass1_residual_divisor"]["value"]
    err = np.abs(x - oracle.mxfp4_reconstruct(q1, q2, e1, e2, oracle.GRID_E1M2)) / alpha
    assert err.max() == 1 / GOLD["thm2_e1m2_bound_divisor"]["value"]


def test_e2m1_rule_exhaustive():
    """The same rule on E2M1 (alpha bound 4.5, beta = alpha/16): pass-1 residual <= alpha/2, final error <= alpha/8
    everywhere and <= alpha/32 for |x| <= 2.25 alpha."""
    c, sh = oracle.E2M1_RULE
    xb = _all_bf16_blocks(c)
    q1, q2, e1, e2 = oracle.decompose_mxfp4(xb)
    x = oracle.bf16_bits_to_f64(xb)
    alpha = np.ldexp(1.0, e1.astype(int) - 127)
    mb = np.abs(x).max(axis=1, keepdims=True)
    assert np.all(mb <= c * alpha) and np.all(mb > c * alpha / 2)
    assert np.all(e2.astype(int) == e1.astype(int) - sh)
    r1 = np.abs(x - oracle.mxfp4_reconstruct(q1, None, e1, None)) / alpha
    assert r1.max() == 0.5
    err = np.abs(x - oracle.mxfp4_reconstruct(q1, q2, e1, e2)) / alpha
    assert err.max() == 1 / 8
    small = np.abs(x) <= 2.25 * alpha
    assert err[small].max() == 1 / 32
    # the first component never uses the top code: |x| <= 4.5 alpha rounds to at most 4
    assert (_codes(q1) & 7).max() == 6


def test_fp4_rounding_ties_and_saturation():
    """Ties go to the code with an even mantissa bit; beyond the top value the result saturates."""
    # a block whose maximum 4.5 gives alpha = 1: the first component is then RNE(x) on the grid
    probe = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 0.26, 0.74, 2.49, 2.51, 3.49, 3.51, -0.25, -2.5, 4.5]
    want = [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 0.5, 0.5, 2.0, 3.0, 3.0, 4.0, -0.0, -2.0, 4.0]
    x = np.zeros((1, 32), np.float32)
    x[0, :len(probe)] = probe
    xb = inputs.f32_to_bf16_bits(x)
    q1, q2, e1, e2 = oracle.decompose_mxfp4(xb)
    assert e1[0, 0] == 127 and e2[0, 0] == 123
    v1 = _values(q1, E2M1)[0, :len(probe)]
    xr = inputs.bf16_bits_to_f32(xb)[0, :len(probe)]
    exact = np.isclose(xr, probe)          # 0.26 etc. are not BF16 numbers; they only need the right side of the tie
    assert np.array_equal(v1[exact], np.array(want)[exact])
    assert np.all(np.abs(v1 - np.array(want)) < 1e-9)
    # second component saturates at +-6 beta when the residual exceeds it
    v2 = _values(q2, E2M1)[0]
    assert v2[14] == 6.0                   # residual 0.5 = 8 beta -> clipped to 6 beta
    # paper grid: uniform step, values above 1.75 clip (Alg. 2 line 4)
    x = np.zeros((1, 32), np.float32)
    x[0, :6] = [1.859375, 1.8, 0.125, 0.375, 0.624, 0.626]
    q1, _, e1, _ = oracle.decompose_mxfp4(inputs.f32_to_bf16_bits(x), oracle.GRID_E1M2, *oracle.PAPER_E1M2)
    assert e1[0, 0] == 127
    assert list(_values(q1, E1M2)[0, :4]) == [1.75, 1.75, 0.0, 0.5]


def test_exact_grid_values_and_scaling_invariance():
    rng = np.random.default_rng(3)
    g = np.array(E2M1)
    x = g[rng.integers(0, 7, (16, 64))] * rng.choice([-1.0, 1.0], (16, 64))
    x[:, 0] = 4.0
    x[:, 32] = 4.0
    xb = inputs.f32_to_bf16_bits(x.astype(np.float32))
    q1, q2, e1, e2 = oracle.decompose_mxfp4(xb)
    assert np.array_equal(_values(q1, E2M1), x) and not (_codes(q2) & 7).any()
    # multiplying a block by a power of two moves only the scale bytes
    y = inputs.activations(8, 128, seed=4)
    yf = inputs.bf16_bits_to_f32(y)
    y2 = inputs.f32_to_bf16_bits(yf * np.float32(2.0 ** -9))
    a = oracle.decompose_mxfp4(y)
    b = oracle.decompose_mxfp4(y2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert np.array_equal(a[2].astype(int) - 9, b[2].astype(int)) and np.array_equal(a[3].astype(int) - 9, b[3].astype(int))
    # zero block: minimum scale codes and zero components
    z = oracle.decompose_mxfp4(np.zeros((1, 32), np.uint16))
    assert z[2][0, 0] == 4 and z[3][0, 0] == 0 and not z[0].any() and not z[1].any()


@pytest.fixture(scope="module")
def gauss_2048():
    rng = np.random.default_rng(1)
    return inputs.f32_to_bf16_bits(rng.standard_normal((2048, 2048)).astype(np.float32))


def _l2(xb, rec):
    x = oracle.bf16_bits_to_f64(xb)
    return np.linalg.norm(x - rec) / np.linalg.norm(x)


def test_paper_evolution_table(gauss_2048):
    """Tab. mxfp4-evolution: v1 (1.75, alpha/8) 0.0182; v2 (1.75, alpha/16) 0.0107; v3 (1.859375, alpha/16) 0.0101."""
    got = {}
    for name, cfg in GOLD["tab_mxfp4_evolution"].items():
        if name == "cite":
            continue
        q1, q2, e1, e2 = oracle.decompose_mxfp4(gauss_2048, oracle.GRID_E1M2, cfg["c"], cfg["shift"])
        got[name] = _l2(gauss_2048, oracle.mxfp4_reconstruct(q1, q2, e1, e2, oracle.GRID_E1M2))
        assert abs(got[name] - cfg["l2"]) <= 0.05 * cfg["l2"], (name, got[name])
        # pass-2 clip rate: none for v1, about one in eight for v2 / v3 (|r/beta| in (1.75, 2])
        x = oracle.bf16_bits_to_f64(gauss_2048)
        r = x - oracle.mxfp4_reconstruct(q1, None, e1, None, oracle.GRID_E1M2)
        beta = np.repeat(np.ldexp(1.0, e2.astype(int) - 127), 32, axis=1)
        clip = 100 * np.mean(np.abs(r / beta) > 1.75)
        if cfg["clip_pct"] == 0:
            assert clip == 0
        else:
            assert 10.0 <= clip <= 14.0, clip
    assert got["v1"] > got["v2"] > got["v3"]


def test_paper_decomp_table(gauss_2048):
    """Tab. mxfp4-decomp: MSD-opt vs single-pass MXFP8 decomposition error across distributions."""
    rng = np.random.default_rng(2)
    n = 2048
    dists = {
        "normal_1.0": None,
        "uniform_3": rng.uniform(-3, 3, (n, n)),
        "laplace_1.0": rng.laplace(0, 1.0, (n, n)),
        "student_t3": rng.standard_t(3, (n, n)),
    }
    for name, data in dists.items():
        xb = gauss_2048 if data is None else inputs.f32_to_bf16_bits(data.astype(np.float32))
        t = GOLD["tab_mxfp4_decomp"][name]
        q1, q2, e1, e2 = oracle.decompose_mxfp4(xb, oracle.GRID_E1M2, *oracle.PAPER_E1M2)
        msd = _l2(xb, oracle.mxfp4_reconstruct(q1, q2, e1, e2, oracle.GRID_E1M2))
        mx8 = _l2(xb, oracle.mxfp8_quantize(xb))
        assert abs(msd - t["msd"]) <= 0.10 * t["msd"], (name, msd)
        assert abs(mx8 - t["mxfp8"]) <= 0.05 * t["mxfp8"], (name, mx8)
        # the E2M1 restatement still beats single-pass MXFP8 (what W4A16 accuracy is compared against)
        q1, q2, e1, e2 = oracle.decompose_mxfp4(xb)
        assert _l2(xb, oracle.mxfp4_reconstruct(q1, q2, e1, e2)) < mx8


def test_w4a16_exact_rational_small():
    """y = sum over blocks of 2^(e_x+e_w) * <q_x, q_w> for both passes, checked with exact rationals."""
    c = inputs.gemm_w4_case(2, 3, 64, seed=6)
    y = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64")
    q1, q2, e1, e2 = oracle.decompose_mxfp4(c.x)
    wv = _values(c.w_fp4, E2M1)
    for i in range(2):
        for n in range(3):
            s = Fraction(0)
            for k in range(64):
                ws = Fraction(2) ** (int(c.w_e8m0[n, k // 32]) - 127)
                for q, e in ((q1, e1), (q2, e2)):
                    xs = Fraction(2) ** (int(e[i, k // 32]) - 127)
                    s += Fraction(float(_values(q, E2M1)[i, k])) * xs * Fraction(float(wv[n, k])) * ws
            assert abs(float(s) - y[i, n]) <= 1e-12 * max(1.0, abs(float(s)))
    # weight quantizer: scale = 2^(floor(log2 blockmax) - 2), so the block maximum lands in [4, 8) before rounding
    w = inputs.weights_f32(4, 64, seed=6)
    q, e = oracle.quantize_weight_mxfp4(w)
    qi, ei = inputs.quantize_weight_mxfp4(w)
    assert np.array_equal(q, qi) and np.array_equal(e, ei)
    s = np.repeat(np.ldexp(1.0, e.astype(int) - 127), 32, axis=1)
    ratio = np.abs(w.astype(np.float64) / s).reshape(4, 2, 32).max(axis=2)
    assert np.all(ratio >= 4) and np.all(ratio < 8)
    assert (_codes(q) & 7).reshape(4, 2, 32).max(axis=2).min() >= 6


def test_w4a16_accuracy_vs_mxfp8():
    """Sec. 6.5: against X * W_mx4 with unquantized X, two-pass MXFP4 activations beat single-pass MXFP8."""
    c = inputs.gemm_w4_case(32, 64, 1024, seed=8)
    ref = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="ref")
    msd = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="msd")
    mx8 = oracle.gemm_w4a16(c.x, c.w_fp4, c.w_e8m0, "f64", mode="mxfp8")
    n = np.linalg.norm(ref)
    assert np.linalg.norm(msd - ref) / n < np.linalg.norm(mx8 - ref) / n < 0.05
