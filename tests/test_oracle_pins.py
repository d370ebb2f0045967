"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

The paper prints no worked numeric example of the quantizer, so each part of the oracle is pinned
by invariants, closed forms, brute force on tiny inputs, special cases that reduce to textbook
results, and the model-size tables.  Fixtures with the paper's printed values live in
tests/golden/.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
QMAX = {8: 127, 4: 7}


def _rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- quantizer, Fig. 2

def _read_ties():
    rows = []
    with open(os.path.join(GOLD, "rounding_ties.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                v, a, b = line.split()
                rows.append((float(v), int(a), int(b)))
    return rows


@pytest.mark.parametrize("bits", [8, 4])
def test_ties_follow_each_rounding_rule(bits):
    """Fig. 2 rounds by floor(v + 0.5); the alternative is IEEE nearest-even.  With the row's
    abs-max equal to qmax the scale is exactly 1 and codes are the rounded inputs."""
    ties = _read_ties()
    vals = [v for v, _, _ in ties] + [float(QMAX[bits])]
    x = np.array([vals], dtype=np.float32)
    for rounding, col in ((orc.ROUND_HALF_UP_FLOOR, 1), (orc.ROUND_NEAREST_EVEN, 2)):
        q, s = orc.quantize(x, bits, orc.AXIS_ROW, rounding)
        assert s[0] == np.float32(1.0)
        assert q[0, -1] == QMAX[bits]
        assert q[0, :-1].tolist() == [t[col] for t in ties]


def test_half_up_floor_adds_in_binary32():
    """floor(v + 0.5) with the sum rounded in binary32: v = 0.5 - 2^-25 is below one half, yet
    v + 0.5 rounds to 1.0 (tie to even at spacing 2^-24), so the code is 1.  Nearest-even
    rounding of v itself gives 0."""
    v = np.float32(0.5) - np.float32(2.0 ** -25)
    assert float(v) < 0.5
    x = np.array([[v, 127.0]], dtype=np.float32)
    q, _ = orc.quantize(x, 8, orc.AXIS_ROW, orc.ROUND_HALF_UP_FLOOR)
    assert q[0, 0] == 1
    q, _ = orc.quantize(x, 8, orc.AXIS_ROW, orc.ROUND_NEAREST_EVEN)
    assert q[0, 0] == 0


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("rounding", [orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN])
@pytest.mark.parametrize("axis", [orc.AXIS_ROW, orc.AXIS_COL, orc.AXIS_TENSOR])
def test_quantizer_invariants(bits, rounding, axis):
    """Codes within +-qmax; scale == abs-max / qmax over the reduced axis; the abs-max element
    gets +-qmax; |x/s - q| <= 1/2 (+ rounding slack); |x - s q| <= s/2 (+ slack)."""
    qmax = QMAX[bits]
    x = (_rng(bits * 10 + rounding).standard_normal((37, 53)) * 3.0).astype(np.float32)
    q, s = orc.quantize(x, bits, axis, rounding)
    assert q.dtype == np.int8 and q.min() >= -qmax and q.max() <= qmax
    ax = {orc.AXIS_ROW: 1, orc.AXIS_COL: 0, orc.AXIS_TENSOR: None}[axis]
    amax = np.max(np.abs(x), axis=ax, keepdims=True) if ax is not None else np.max(np.abs(x)).reshape(1, 1)
    s_full = np.broadcast_to(s.reshape(amax.shape), x.shape).astype(np.float64)
    # scale is the correctly rounded binary32 quotient of abs-max and qmax
    exact = amax.astype(np.float64) / qmax
    assert np.all(np.abs(s.reshape(amax.shape).astype(np.float64) - exact) <= np.spacing(exact.astype(np.float32)) / 2)
    v = x.astype(np.float64) / s_full
    slack = qmax * 2.0 ** -22
    assert np.max(np.abs(v - q)) <= 0.5 + slack
    assert np.all(np.abs(x.astype(np.float64) - s_full * q) <= s_full * (0.5 + slack))
    hit = np.abs(x) == np.broadcast_to(amax, x.shape)
    assert np.all(np.abs(q[hit]) == qmax)
    assert np.all(np.sign(q[hit]) == np.sign(x[hit]))


def test_zero_row_and_negative_zero():
    """divide_no_nan: a zero scale yields zero codes; the scale itself is 0."""
    x = np.zeros((3, 16), dtype=np.float32)
    x[1] = np.linspace(-1, 1, 16, dtype=np.float32)
    x[2, 3] = -0.0
    q, s = orc.quantize(x, 8, orc.AXIS_ROW)
    assert s[0] == 0.0 and s[2] == 0.0 and not q[0].any() and not q[2].any()
    assert s[1] == np.float32(1.0) / np.float32(127.0) and abs(q[1, 0]) == 127


def test_subnormal_scale_guard_clip():
    """With a subnormal scale the quotient loses precision and can exceed qmax before the guard
    clip.  In units of the smallest subnormal u: abs-max 190u gives scale 190/127 u -> 1u (the
    scale is rounded to a whole number of u), so x/s = 190 and the clip brings it to 127."""
    u = np.float32(1.401298464324817e-45)
    x = np.array([[190 * u, -190 * u, 37 * u, 0.0]], dtype=np.float32)
    assert x[0, 0] / u == 190
    for rounding in (orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN):
        q, s = orc.quantize(x, 8, orc.AXIS_ROW, rounding)
        assert s[0] == u
        assert q[0].tolist() == [127, -127, 37, 0]
        q, s = orc.quantize(x[:, 2:] * np.float32(1), 4, orc.AXIS_ROW, rounding)   # abs-max 37u: 37/7 -> 5u, 37/5 = 7.4
        assert s[0] == 5 * u and q[0].tolist() == [7, 0]
        q, s = orc.quantize(np.array([[10 * u, -3 * u]], np.float32), 4, orc.AXIS_ROW, rounding)   # 10/7 -> 1u, clip 10 -> 7
        assert s[0] == u and q[0].tolist() == [7, -3]


@pytest.mark.parametrize("bits", [8, 4])
def test_quantize_dequantize_quantize_is_idempotent(bits):
    x = (_rng(5).standard_normal((64, 96)) * 0.7).astype(np.float32)
    for rounding in (orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN):
        q1, s1 = orc.quantize(x, bits, orc.AXIS_ROW, rounding)
        xd = orc.dequantize(q1, s1, orc.AXIS_ROW)
        q2, s2 = orc.quantize(xd, bits, orc.AXIS_ROW, rounding)
        assert np.array_equal(q1, q2)
        assert np.all(np.abs(s1.astype(np.float64) - s2) <= np.spacing(s1))


def test_axis_col_is_axis_row_of_the_transpose():
    """The reduced axis is the argument (reduce_max(..., axis, keepdims=True)); abs-max does not
    depend on memory order, so reducing over rows of W equals reducing over columns of W^T."""
    w = (_rng(11).standard_normal((48, 20)) * 0.05).astype(np.float32)
    qc, sc = orc.quantize(w, 4, orc.AXIS_COL)
    qr, sr = orc.quantize(np.ascontiguousarray(w.T), 4, orc.AXIS_ROW)
    assert np.array_equal(qc.T, qr) and np.array_equal(sc, sr)
    assert sc.shape == (20,)


def test_strided_input_rows():
    big = _rng(3).standard_normal((10, 40)).astype(np.float32)
    view = big[:, :24]
    q1, s1 = orc.quantize(view, 8, orc.AXIS_ROW)
    q2, s2 = orc.quantize(np.ascontiguousarray(view), 8, orc.AXIS_ROW)
    assert np.array_equal(q1, q2) and np.array_equal(s1, s2)


def test_dequantize_multiplies_by_scale():
    q = np.array([[3, -7], [1, 0]], dtype=np.int8)
    assert np.array_equal(orc.dequantize(q, np.array([0.5, 2.0], np.float32), orc.AXIS_ROW),
                          np.array([[1.5, -3.5], [2.0, 0.0]], np.float32))
    assert np.array_equal(orc.dequantize(q, np.array([0.5, 2.0], np.float32), orc.AXIS_COL),
                          np.array([[1.5, -14.0], [0.5, 0.0]], np.float32))


# ----------------------------------------------------------------------------- 4-bit packing

def test_pack_layout_by_hand():
    """Low nibble = even column, high nibble = odd column, two's complement nibbles."""
    q = np.array([[1, -1, -7, 7, 0, -8 + 1]], dtype=np.int8)
    assert orc.pack_int4(q).tolist() == [[0xF1, 0x79, 0x90]]


def test_pack_unpack_all_nibble_pairs():
    pairs = np.array(list(itertools.product(range(-7, 8), repeat=2)), dtype=np.int8)  # 225 x 2
    packed = orc.pack_int4(pairs)
    assert packed.shape == (225, 1)
    assert np.array_equal(orc.unpack_int4(packed, 2), pairs)
    wide = pairs.reshape(5, 90)
    assert orc.pack_int4(wide).nbytes == wide.size // 2
    assert np.array_equal(orc.unpack_int4(orc.pack_int4(wide), 90), wide)
    with pytest.raises(ValueError):
        orc.pack_int4(np.zeros((2, 3), np.int8))


# ----------------------------------------------------------------------------- integer matmul

def test_int_matmul_brute_force_tiny():
    rng = _rng(2)
    for (M, N, K) in [(1, 1, 1), (2, 3, 4), (5, 7, 8), (8, 8, 3)]:
        xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
        wq = rng.integers(-7, 8, (N, K)).astype(np.int8)
        acc = orc.int_matmul(xq, wq)
        for m in range(M):
            for n in range(N):
                assert acc[m, n] == sum(int(xq[m, k]) * int(wq[n, k]) for k in range(K))


def test_int_matmul_enumerates_all_int4_codes_for_k2():
    codes = np.array(list(itertools.product(range(-7, 8), repeat=2)), dtype=np.int8)  # every K=2 vector
    acc = orc.int_matmul(codes, codes)
    a = codes.astype(np.int64)
    expect = a[:, 0][:, None] * a[:, 0][None, :] + a[:, 1][:, None] * a[:, 1][None, :]
    assert np.array_equal(acc, expect)


def test_int_matmul_textbook_cases():
    rng = _rng(4)
    K = 40
    xq = rng.integers(-127, 128, (6, K)).astype(np.int8)
    eye = np.eye(K, dtype=np.int8)
    assert np.array_equal(orc.int_matmul(xq, eye), xq.astype(np.int64))         # W = I
    ones = np.ones((3, K), dtype=np.int8)
    assert np.array_equal(orc.int_matmul(xq, ones), np.repeat(xq.sum(1, dtype=np.int64)[:, None], 3, 1))
    # operand roles: row n of wq is output channel n (not column n)
    w = rng.integers(-7, 8, (5, K)).astype(np.int8)
    assert np.array_equal(orc.int_matmul(xq, w), xq.astype(np.int64) @ w.astype(np.int64).T)
    # extremes: +-qmax everywhere gives +-K qmax_a qmax_w, inside int32 for K = 4096
    K = 4096
    a = np.full((1, K), 127, np.int8)
    b = np.full((2, K), -127, np.int8)
    b[1] = 127
    assert orc.int_matmul(a, b).tolist() == [[-K * 127 * 127, K * 127 * 127]]
    assert K * 127 * 127 < 2 ** 31


def test_int32_overflow_is_reported():
    K = 140000  # 140000 * 127 * 127 > 2^31
    a = np.full((1, K), 127, np.int8)
    with pytest.raises(OverflowError):
        orc.int_matmul(a, a)


def test_factorisation_identity_power_of_two_scales():
    """No zero point (Section 2.2): sum_k (s_a q_a)(s_w q_w) = s_a s_w sum_k q_a q_w.  With
    power-of-two scales every product and sum below is exact in double."""
    rng = _rng(9)
    M, N, K = 7, 5, 64
    xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    wq = rng.integers(-7, 8, (N, K)).astype(np.int8)
    s_a = (2.0 ** rng.integers(-6, 3, M)).astype(np.float32)
    s_w = (2.0 ** rng.integers(-8, 0, N)).astype(np.float32)
    xd = orc.dequantize(xq, s_a, orc.AXIS_ROW).astype(np.float64)
    wd = orc.dequantize(wq, s_w, orc.AXIS_ROW).astype(np.float64)
    ref = xd @ wd.T
    acc = orc.int_matmul(xq, wq)
    y64 = orc.epilogue_f64(acc, s_a, orc.SCALE_ROW, s_w)
    assert np.array_equal(y64, ref)
    y32 = orc.epilogue_f32(acc, s_a, orc.SCALE_ROW, s_w)
    assert np.array_equal(y32.astype(np.float64), ref.astype(np.float32).astype(np.float64))


def test_factorisation_identity_general_scales():
    rng = _rng(10)
    M, N, K = 9, 6, 512
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32)
    xq, s_a = orc.quantize(x, 8, orc.AXIS_ROW)
    wq, s_w = orc.quantize(w, 4, orc.AXIS_ROW)
    xd = xq.astype(np.float64) * s_a[:, None].astype(np.float64)
    wd = wq.astype(np.float64) * s_w[:, None].astype(np.float64)
    ref = xd @ wd.T
    bound = (np.abs(xd) @ np.abs(wd).T) * K * 2.0 ** -52
    y64 = orc.epilogue_f64(orc.int_matmul(xq, wq), s_a, orc.SCALE_ROW, s_w)
    assert np.all(np.abs(y64 - ref) <= bound)


def test_float_emulation_agrees_below_2_24_and_fails_above():
    """Section 1: float emulation of the integer matmul is exact only while results fit the
    binary32 significand (integers up to 2^24)."""
    rng = _rng(12)
    K = 1040                                      # 1040 * 127 * 127 < 2^24
    assert K * 127 * 127 < 2 ** 24
    xq = rng.integers(-127, 128, (4, K)).astype(np.int8)
    wq = rng.integers(-127, 128, (3, K)).astype(np.int8)
    xq[0], wq[0] = 127, 127
    assert np.array_equal(orc.emulated_matmul_f32(xq, wq).astype(np.int64), orc.int_matmul(xq, wq))
    K = 2048                                      # constructed failure: exact sum is odd and > 2^24
    a = np.full((1, K), 127, np.int8)
    b = np.full((1, K), 127, np.int8)
    b[0, -1] = 126
    exact = orc.int_matmul(a, b)[0, 0]
    assert exact == 2047 * 127 * 127 + 127 * 126 == 33032065 and exact % 2 == 1 and exact > 2 ** 24
    assert int(orc.emulated_matmul_f32(a, b)[0, 0]) != exact


# ----------------------------------------------------------------------------- epilogue

def test_epilogue_by_hand():
    acc = np.array([[3, -4], [10, 0]], dtype=np.int64)
    s_x = np.array([0.5, 0.25], np.float32)
    s_w = np.array([0.25, 2.0], np.float32)
    bias = np.array([1.0, -1.0], np.float32)
    y = orc.epilogue_f32(acc, s_x, orc.SCALE_ROW, s_w, bias)
    assert y.tolist() == [[1.375, -5.0], [1.625, -1.0]]
    y = orc.epilogue_f32(acc, np.array([0.5], np.float32), orc.SCALE_TENSOR, s_w, None)
    assert y.tolist() == [[0.375, -4.0], [1.25, 0.0]]
    res = np.array([[10.0, 20.0], [30.0, 40.0]], np.float32)
    y = orc.epilogue_f32(acc, s_x, orc.SCALE_ROW, s_w, bias, residual=res, residual_scale=0.5)
    assert y.tolist() == [[10.6875, 17.5], [30.8125, 39.5]]
    y64 = orc.epilogue_f64(acc, s_x, orc.SCALE_ROW, s_w, bias, residual=res, residual_scale=0.5)
    assert y64.tolist() == [[10.6875, 17.5], [30.8125, 39.5]]


def test_epilogue_f32_is_within_two_roundings_of_f64():
    rng = _rng(14)
    M, N = 33, 40
    acc = rng.integers(-(2 ** 24), 2 ** 24, (M, N)).astype(np.int64)
    s_x = rng.uniform(1e-3, 1e-1, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 1e-2, N).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    y32 = orc.epilogue_f32(acc, s_x, orc.SCALE_ROW, s_w, bias).astype(np.float64)
    y64 = orc.epilogue_f64(acc, s_x, orc.SCALE_ROW, s_w, bias)
    mag = np.maximum(np.abs(y64), np.abs(acc * s_x[:, None].astype(np.float64) * s_w[None, :]))
    assert np.all(np.abs(y32 - y64) <= 2.0 ** -23 * mag)


def test_swish_closed_forms():
    """Swish(z) = z sigmoid(z): Swish(0) = 0, Swish(ln 3) = (3/4) ln 3, Swish(z) - Swish(-z) = z."""
    z = np.array([0.0, math.log(3.0), -math.log(3.0), 5.0, -5.0, 20.0, -20.0, 90.0, -90.0])
    # acc = round(z * 2^20), scales 2^-10 * 2^-10: pre-activation is an exactly known binary32
    acc = np.round(z * 2 ** 20).astype(np.int64).reshape(1, -1)
    zq = (acc[0] * 2.0 ** -20).astype(np.float32)
    s = np.array([2.0 ** -10], np.float32)
    y, pre = orc.epilogue_f32(acc, s, orc.SCALE_TENSOR, np.full(z.size, 2.0 ** -10, np.float32), act=orc.ACT_SWISH,
                              return_preact=True)
    assert np.array_equal(pre[0], zq)
    y = y[0].astype(np.float64)
    assert y[0] == 0.0
    assert abs(y[1] - 0.75 * zq[1]) <= 1e-6 * abs(zq[1]) and abs(y[2] + 0.25 * zq[1]) <= 1e-6
    for i in (1, 3, 5, 7):
        assert abs((y[i] - y[i + 1]) - zq[i]) <= 2.0 ** -22 * abs(zq[i])
    assert y[7] == zq[7] and abs(y[8]) < 1e-35
    y64 = orc.epilogue_f64(acc, s, orc.SCALE_TENSOR, np.full(z.size, 2.0 ** -10, np.float32), act=orc.ACT_SWISH)[0]
    assert np.all(np.abs(y - y64) <= 2.0 ** -23 * np.abs(y64) + 1e-45)


def test_glu_closed_forms():
    """GLU: out[j] = z[j] sigmoid(z[j + N/2]); gate 0 halves the value, gate ln 3 scales by 3/4;
    first half are values, second half are gates."""
    one = 2 ** 20
    g3 = int(round(math.log(3.0) * one))
    acc = np.array([[3 * one, -2 * one, one, 0, g3, -40 * one]], dtype=np.int64)   # values 3,-2,1 ; gates 0, ln3, -40
    s = np.array([2.0 ** -10], np.float32)
    sw = np.full(6, 2.0 ** -10, np.float32)
    y = orc.epilogue_f32(acc, s, orc.SCALE_TENSOR, sw, act=orc.ACT_GLU)
    assert y.shape == (1, 3)
    assert y[0, 0] == 1.5 and abs(y[0, 1] + 1.5) < 1e-6 and 0 < y[0, 2] < 1e-17
    ys = orc.epilogue_f32(acc, s, orc.SCALE_TENSOR, sw, act=orc.ACT_GLU_SWISH)
    g = 1.5
    assert abs(ys[0, 0] - g / (1 + math.exp(-g))) < 1e-7
    y64 = orc.epilogue_f64(acc, s, orc.SCALE_TENSOR, sw, act=orc.ACT_GLU_SWISH)
    assert np.all(np.abs(ys - y64) <= 2.0 ** -23 * np.abs(y64) + 1e-45)
    with pytest.raises(ValueError):
        orc.epilogue_f32(acc[:, :5], s, orc.SCALE_TENSOR, sw[:5], act=orc.ACT_GLU)


# ----------------------------------------------------------------------------- whole layer

def test_linear_fwd_is_the_composition_and_close_to_float_matmul():
    """Whole layer = quantize -> integer matmul -> epilogue; and, because scaling is by abs-max
    with round-to-nearest, it approximates the float layer with error bounded by the code grid."""
    rng = _rng(21)
    M, K, N = 12, 256, 24
    x = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    wq, s_w = orc.quantize(w, 8, orc.AXIS_ROW)
    y, xq, sx, acc = orc.linear_fwd(x, wq, s_w, bias=bias, return_parts=True)
    xq2, sx2 = orc.quantize(x, 8, orc.AXIS_ROW)
    assert np.array_equal(xq, xq2) and np.array_equal(sx, sx2)
    assert np.array_equal(acc, orc.int_matmul(xq, wq))
    assert np.array_equal(y, orc.epilogue_f32(acc, sx, orc.SCALE_ROW, s_w, bias))
    ref = x.astype(np.float64) @ w.astype(np.float64).T + bias
    # each operand is within s/2 of its grid point: |err| <= sum_k (|x| s_w/2 + |w| s_a/2 + s_a s_w/4)
    bound = (np.abs(x).astype(np.float64) @ np.ones((K, 1))) * (s_w[None, :] / 2.0) \
        + (sx[:, None] / 2.0) * (np.abs(w).astype(np.float64) @ np.ones((K, 1))).T \
        + K * sx[:, None] * s_w[None, :] / 4.0
    assert np.all(np.abs(y - ref) <= bound * (1 + 1e-5) + 1e-6)
    assert np.max(np.abs(y - ref)) < 0.05 * np.std(ref) + 0.05


def test_linear_fwd_per_tensor_scale():
    rng = _rng(22)
    x = rng.standard_normal((8, 32)).astype(np.float32)
    wq = rng.integers(-127, 128, (4, 32)).astype(np.int8)
    s_w = rng.uniform(0.001, 0.01, 4).astype(np.float32)
    y, xq, sx, acc = orc.linear_fwd(x, wq, s_w, a_scale_kind=orc.SCALE_TENSOR, return_parts=True)
    assert sx.shape == (1,) and sx[0] == np.float32(np.abs(x).max()) / np.float32(127.0)
    assert np.array_equal(y, orc.epilogue_f32(acc, sx, orc.SCALE_TENSOR, s_w))


# ----------------------------------------------------------------------------- model sizes (Tables 1, 2)

def _read_sizes():
    t1, t2, params, ratios = {}, {}, {}, {}
    with open(os.path.join(GOLD, "model_sizes.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            p = line.split()
            if p[0] == "table1":
                t1[p[1]] = tuple(float(v) for v in p[2:5])
            elif p[0] == "table2":
                t2[p[1]] = float(p[2])
            elif p[0] == "params":
                params[p[1]] = float(p[2])
            else:
                ratios[p[1]] = float(p[2])
    return t1, t2, params, ratios


def _mb(n_params_m: float, bits: int) -> float:
    """Size in MB (10^6 bytes) of n_params_m million weights stored as one [K, 1000] matrix."""
    K = int(round(n_params_m * 1e6 / 1000))
    return orc.weight_bytes(K, 1000, bits) / 1e6


def test_weight_bytes_closed_form():
    assert orc.weight_bytes(512, 2048, 8) == 512 * 2048 + 4 * 2048
    assert orc.weight_bytes(512, 2048, 4) == 512 * 2048 // 2 + 4 * 2048
    assert orc.weight_bytes(512, 2048, 32) == 4 * 512 * 2048
    q = np.zeros((2048, 512), np.int8)
    assert orc.pack_int4(q).nbytes + 4 * 2048 == orc.weight_bytes(512, 2048, 4)


def test_table2_sizes_follow_from_parameter_counts():
    """Table 2 with the parameter counts of Section 2.1: both encoders quantized, decoders kept
    at int8 in every quantized model; sizes agree with the printed ones within 3 %."""
    _, t2, p, ratios = _read_sizes()
    dec = 2 * p["decoder"]
    size = {
        "B0": _mb(p["causal"], 32) + _mb(p["noncausal"], 32) + _mb(dec, 32),
        "E0": _mb(p["causal"], 8) + _mb(p["noncausal"], 8) + _mb(dec, 8),
        "E3": _mb(p["causal"], 4) + _mb(p["noncausal"], 4) + _mb(dec, 8),
        "E4": _mb(p["causal"], 4) + _mb(p["noncausal"], 8) + _mb(dec, 8),
        "E5": _mb(p["causal"], 8) + _mb(p["noncausal"], 4) + _mb(dec, 8),
    }
    for k, v in size.items():
        assert abs(v - t2[k]) <= 0.03 * t2[k], (k, v, t2[k])
    # E10: int4 in the first 3 of 7 causal and 3 of 6 non-causal layers (the first 3 causal
    # layers have no self-attention, so equal layer sizes over-estimate the saving slightly)
    e10 = size["E0"] - (_mb(p["causal"] * 3 / 7, 8) - _mb(p["causal"] * 3 / 7, 4)) \
        - (_mb(p["noncausal"] * 3 / 6, 8) - _mb(p["noncausal"] * 3 / 6, 4))
    assert abs(e10 - t2["E10"]) <= 0.05 * t2["E10"]
    assert abs(t2["E10"] / t2["E0"] - ratios["E10_over_int8"]) < 0.01
    assert abs(t2["E10"] / t2["B0"] - ratios["E10_over_float"]) < 0.01


def test_table1_int4_size_follows_from_int8_size():
    """Table 1: the quantized fraction f of the parameters that explains float -> int8 also
    predicts the int4 column (4 bits per quantized weight, 32 per unquantized one)."""
    t1, _, _, ratios = _read_sizes()
    for name, (f32, i8, i4) in t1.items():
        n = f32 / 4.0                                     # million parameters
        lo, hi = 0.0, 1.0
        for _ in range(60):                               # bisection on f
            f = (lo + hi) / 2
            if _mb(n * f, 8) + _mb(n * (1 - f), 32) > i8:
                lo = f
            else:
                hi = f
        pred = _mb(n * f, 4) + _mb(n * (1 - f), 32)
        assert abs(pred - i4) <= 1.5, (name, f, pred, i4)
    assert abs(t1["L"][0] / t1["L"][2] - ratios["L_float_over_int4"]) < 0.05
