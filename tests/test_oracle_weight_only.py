"""Pins of the oracle's weight-only layer (Section 4.1: integer weights converted to float,
float32 activations; Section 2.2: de-quantize by multiplying with the scale).  No GPU.

The function is the plain definition in double.  It is pinned by exact rational arithmetic on
tiny shapes, by special cases with known answers, and by the identity that ties it to the
(separately pinned) integer path: on activations that are themselves de-quantized codes the float
layer and the integer layer compute the same number.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc


def _rng(seed):
    return np.random.default_rng(seed)


def _sigmoid_frac(z):
    # double precision is enough here: used only for the activation pins
    import math
    return 1.0 / (1.0 + math.exp(-float(z)))


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_equals_exact_rational_arithmetic_on_tiny_shapes(seed):
    """z = s_w * sum_k x * wq + bias evaluated in rationals (every binary32 value is a rational);
    the double result must agree to a few units of 2^-53 of the terms' magnitude."""
    r = _rng(seed)
    M, N, K = 3, 4, 5
    x = r.standard_normal((M, K)).astype(np.float32)
    wq = r.integers(-7, 8, (N, K)).astype(np.int8)
    s_w = (r.random(N) * 0.1 + 0.01).astype(np.float32)
    bias = r.standard_normal(N).astype(np.float32)
    y, z, mag = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, return_parts=True)
    for m in range(M):
        for n in range(N):
            exact = Fraction(float(s_w[n])) * sum(Fraction(float(x[m, k])) * int(wq[n, k]) for k in range(K)) + Fraction(float(bias[n]))
            exact_mag = Fraction(float(s_w[n])) * sum(abs(Fraction(float(x[m, k])) * int(wq[n, k])) for k in range(K))
            assert abs(Fraction(z[m, n]) - exact) <= Fraction(float(mag[m, n]) + abs(float(bias[n]))) * Fraction(8, 2 ** 53)
            assert abs(Fraction(mag[m, n]) - exact_mag) <= exact_mag * Fraction(8, 2 ** 53)
            assert y[m, n] == z[m, n]  # no activation, no residual


def test_identity_codes_scale_the_input():
    """wq = identity codes: z[m][n] = s_w[n] * x[m][n] + bias[n], exactly representable products."""
    r = _rng(3)
    n = 6
    x = r.standard_normal((4, n)).astype(np.float32)
    wq = np.eye(n, dtype=np.int8)
    s_w = np.array([0.5, 2.0, 0.25, 1.0, 4.0, 0.125], dtype=np.float32)
    y = orc.linear_weight_only_f64(x, wq, s_w)
    assert np.array_equal(y, x.astype(np.float64) * s_w.astype(np.float64))


def test_sign_symmetry_and_magnitude():
    r = _rng(4)
    x = r.standard_normal((5, 16)).astype(np.float32)
    wq = r.integers(-127, 128, (8, 16)).astype(np.int8)
    s_w = (r.random(8) + 0.5).astype(np.float32)
    y = orc.linear_weight_only_f64(x, wq, s_w)
    y_neg = orc.linear_weight_only_f64(-x, wq, s_w)
    assert np.array_equal(y_neg, -y)
    # one-signed terms: the magnitude equals the value
    _, z, mag = orc.linear_weight_only_f64(np.abs(x), np.abs(wq).astype(np.int8), s_w, return_parts=True)
    assert np.array_equal(z, mag)
    # and bounds it otherwise
    _, z, mag = orc.linear_weight_only_f64(x, wq, s_w, return_parts=True)
    assert np.all(np.abs(z) <= mag)


@pytest.mark.parametrize("bits_a,bits_w", [(8, 8), (8, 4), (4, 4)])
def test_agrees_with_the_integer_layer_on_dequantized_activations(bits_a, bits_w):
    """If the activations are themselves s_x * codes, then x . (s_w wq) = s_x s_w (xq . wq): the
    float layer must reproduce the integer layer's double-precision epilogue.  With power-of-two
    scales both sides are exact, so the results are equal."""
    r = _rng(10 + bits_a + bits_w)
    M, N, K = 7, 12, 64
    qa, qw = (1 << (bits_a - 1)) - 1, (1 << (bits_w - 1)) - 1
    xq = r.integers(-qa, qa + 1, (M, K)).astype(np.int8)
    wq = r.integers(-qw, qw + 1, (N, K)).astype(np.int8)
    s_x = (2.0 ** r.integers(-6, 3, M)).astype(np.float32)
    s_w = (2.0 ** r.integers(-8, 1, N)).astype(np.float32)
    bias = (r.integers(-8, 9, N) / 4.0).astype(np.float32)
    x = orc.dequantize(xq, s_x, orc.AXIS_ROW)
    acc = orc.int_matmul(xq, wq)
    for act in (orc.ACT_NONE, orc.ACT_SWISH, orc.ACT_GLU, orc.ACT_GLU_SWISH):
        ref = orc.epilogue_f64(acc, s_x, orc.SCALE_ROW, s_w, bias=bias, act=act)
        got = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, act=act)
        assert np.array_equal(got, ref), act
    # general scales: equal up to double rounding of the two evaluation orders
    s_x = (r.random(M) * 0.1 + 0.01).astype(np.float32)
    s_w = (r.random(N) * 0.01 + 0.001).astype(np.float32)
    x = orc.dequantize(xq, s_x, orc.AXIS_ROW)  # binary32 products: x is only approximately s_x * xq
    xd = xq.astype(np.float64) * s_x.astype(np.float64)[:, None]
    err_x = np.abs(x.astype(np.float64) - xd).max()
    assert err_x <= 2.0 ** -24 * np.abs(xd).max()
    got, z, mag = orc.linear_weight_only_f64(x, wq, s_w, return_parts=True)
    ref = orc.epilogue_f64(acc, s_x, orc.SCALE_ROW, s_w)
    assert np.all(np.abs(got - ref) <= 2.0 ** -23 * mag + 1e-300)


def test_activation_and_residual_closed_forms():
    """One input, one weight: z = s_w * x * wq + b by hand; Swish, GLU and residual from their
    textbook definitions."""
    x = np.array([[1.5]], dtype=np.float32)
    wq = np.array([[2], [-3]], dtype=np.int8)
    s_w = np.array([0.5, 0.25], dtype=np.float32)
    bias = np.array([0.25, 1.0], dtype=np.float32)
    z0, z1 = 0.5 * 1.5 * 2 + 0.25, 0.25 * 1.5 * -3 + 1.0  # 1.75, -0.125
    y = orc.linear_weight_only_f64(x, wq, s_w, bias=bias)
    assert y.tolist() == [[z0, z1]]
    y = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, act=orc.ACT_SWISH)
    assert np.allclose(y, [[z0 * _sigmoid_frac(z0), z1 * _sigmoid_frac(z1)]], rtol=1e-15, atol=0)
    y = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, act=orc.ACT_GLU)
    g = z0 * _sigmoid_frac(z1)
    assert np.allclose(y, [[g]], rtol=1e-15, atol=0)
    y = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, act=orc.ACT_GLU_SWISH)
    assert np.allclose(y, [[g * _sigmoid_frac(g)]], rtol=1e-15, atol=0)
    res = np.array([[10.0, -20.0]], dtype=np.float32)
    y = orc.linear_weight_only_f64(x, wq, s_w, bias=bias, residual=res, residual_scale=0.5)
    assert y.tolist() == [[10.0 + 0.5 * z0, -20.0 + 0.5 * z1]]


def test_padded_rows_and_bad_arguments():
    r = _rng(5)
    big = r.standard_normal((4, 24)).astype(np.float32)
    x = big[:, :16]  # row pitch 24
    wq = r.integers(-7, 8, (6, 16)).astype(np.int8)
    s_w = np.ones(6, dtype=np.float32)
    assert np.array_equal(orc.linear_weight_only_f64(x, wq, s_w), orc.linear_weight_only_f64(np.ascontiguousarray(x), wq, s_w))
    with pytest.raises(ValueError):
        orc.linear_weight_only_f64(x, wq[:5], s_w[:5], act=orc.ACT_GLU)  # odd N with GLU
