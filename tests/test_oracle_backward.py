"""Pins of the oracle's straight-through backward of the quantized linear layer.  No GPU.

The paper fixes only that scales carry no gradient (Fig. 2, stop_gradient) and that the forward
is the integer one.  The oracle takes the plain straight-through definition; it is pinned against
the separately pinned forward (the layer is bilinear in the de-quantized operands, so finite
differences of the forward are exact up to double rounding), against exact rational arithmetic on
tiny shapes, and against hand-computed values.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle as orc


def _case(seed, M, N, K, bits_a=8, bits_w=4):
    r = np.random.default_rng(seed)
    qa, qw = (1 << (bits_a - 1)) - 1, (1 << (bits_w - 1)) - 1
    xq = r.integers(-qa, qa + 1, (M, K)).astype(np.int8)
    wq = r.integers(-qw, qw + 1, (N, K)).astype(np.int8)
    s_x = (r.random(M) * 0.05 + 0.01).astype(np.float32)
    s_w = (r.random(N) * 0.01 + 0.001).astype(np.float32)
    dy = r.standard_normal((M, N)).astype(np.float32)
    return xq, wq, s_x, s_w, dy


def _loss(x_hat, wq, s_w, bias, dy):
    """L = sum(dy * y) with y from the forward oracle of the float layer on x_hat."""
    y = orc.linear_weight_only_f64(x_hat, wq, s_w, bias=bias)
    return float(np.sum(dy.astype(np.float64) * y))


def test_gradients_are_the_finite_differences_of_the_forward():
    """y is linear in x_hat, in each de-quantized weight and in the bias, so a finite difference
    of L = <dy, y> is the gradient itself (no truncation error); steps are powers of two so that
    the perturbed inputs are exact."""
    M, N, K = 5, 6, 8
    xq, wq, s_x, s_w, dy = _case(0, M, N, K)
    s_x = (2.0 ** np.arange(-3, M - 3)).astype(np.float32)  # exact de-quantization
    x_hat = orc.dequantize(xq, s_x, orc.AXIS_ROW)
    bias = np.zeros(N, dtype=np.float32)
    dx, dw, db = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w)
    base = _loss(x_hat, wq, s_w, bias, dy)
    for (m, k) in [(0, 0), (2, 5), (4, 7)]:
        xp = x_hat.copy()
        xp[m, k] += np.float32(0.25)
        assert abs((_loss(xp, wq, s_w, bias, dy) - base) / 0.25 - dx[m, k]) <= 1e-12 * max(1.0, abs(dx[m, k]))
    for (n, k) in [(0, 0), (3, 4), (5, 7)]:
        # one code step changes the de-quantized weight by s_w[n]
        wp = wq.copy()
        wp[n, k] += 1 if wp[n, k] < 7 else -1
        step = float(s_w[n]) * (int(wp[n, k]) - int(wq[n, k]))
        assert abs((_loss(x_hat, wp, s_w, bias, dy) - base) / step - dw[n, k]) <= 1e-10 * max(1.0, abs(dw[n, k]))
    for n in (0, 5):
        bp = bias.copy()
        bp[n] = 0.5
        assert abs((_loss(x_hat, wq, s_w, bp, dy) - base) / 0.5 - db[n]) <= 1e-12 * max(1.0, abs(db[n]))


@pytest.mark.parametrize("kind", [orc.SCALE_ROW, orc.SCALE_TENSOR])
def test_equals_exact_rational_arithmetic_on_tiny_shapes(kind):
    M, N, K = 3, 4, 5
    xq, wq, s_x, s_w, dy = _case(1, M, N, K)
    if kind == orc.SCALE_TENSOR:
        s_x = s_x[:1]
    dx, dw, db, mx, mw, mb = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w, s_x_kind=kind, return_mags=True)
    F = lambda v: Fraction(float(v))
    for m in range(M):
        for k in range(K):
            ex = sum(F(dy[m, n]) * F(s_w[n]) * int(wq[n, k]) for n in range(N))
            assert abs(Fraction(dx[m, k]) - ex) <= Fraction(float(mx[m, k])) * Fraction(8, 2 ** 53)
            assert abs(Fraction(mx[m, k]) - sum(abs(F(dy[m, n]) * F(s_w[n]) * int(wq[n, k])) for n in range(N))) <= Fraction(float(mx[m, k])) * Fraction(8, 2 ** 53)
    for n in range(N):
        for k in range(K):
            ex = sum(F(dy[m, n]) * F(s_x[m if kind == orc.SCALE_ROW else 0]) * int(xq[m, k]) for m in range(M))
            assert abs(Fraction(dw[n, k]) - ex) <= Fraction(float(mw[n, k])) * Fraction(8, 2 ** 53)
        assert abs(Fraction(db[n]) - sum(F(dy[m, n]) for m in range(M))) <= Fraction(float(mb[n])) * Fraction(8, 2 ** 53)


def test_hand_computed_one_by_one_and_transposition():
    dy = np.array([[2.0]], dtype=np.float32)
    dx, dw, db = orc.linear_bwd_f64(dy, np.array([[3]], np.int8), np.array([0.5], np.float32), np.array([[-4]], np.int8),
                                    np.array([0.25], np.float32))
    assert dx.tolist() == [[2.0 * 0.25 * -4]] and dw.tolist() == [[2.0 * 0.5 * 3]] and db.tolist() == [2.0]
    # dx is the float layer applied to dy with the transposed, scaled weights: s_w = 1 makes that exact
    xq, wq, s_x, s_w, dy = _case(2, 6, 8, 12, bits_w=8)
    ones = np.ones(8, dtype=np.float32)
    dx, _, _ = orc.linear_bwd_f64(dy, xq, s_x, wq, ones)
    fwd = orc.linear_weight_only_f64(dy, np.ascontiguousarray(wq.T), np.ones(12, dtype=np.float32))
    assert np.array_equal(dx, fwd)
    # and dw is the same construction on the transposed gradient
    _, dw, _ = orc.linear_bwd_f64(dy, xq, np.ones(6, np.float32), wq, s_w)
    fwd = orc.linear_weight_only_f64(np.ascontiguousarray(dy.T), np.ascontiguousarray(xq.T), np.ones(12, dtype=np.float32))
    assert np.array_equal(dw, fwd)


def test_padded_gradient_rows_and_bad_arguments():
    xq, wq, s_x, s_w, dy = _case(3, 4, 6, 8)
    big = np.zeros((4, 10), dtype=np.float32)
    big[:, :6] = dy
    a = orc.linear_bwd_f64(big[:, :6], xq, s_x, wq, s_w)
    b = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w)
    assert all(np.array_equal(u, v) for u, v in zip(a, b))
