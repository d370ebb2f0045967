"""Parity of the weight-only layer (Section 4.1: I8W / I4W -- integer weights converted to float,
float32 activations) against the CPU oracle, through the C ABI (needs a B200).

The kernel is a float matmul on the tensor cores: weight codes are exact as floats, every
activation enters with the upper ten fraction bits of its binary32 value, products are exact,
sums are binary32.  Tolerance, derived from that arithmetic, per pre-activation z:
    |z - z_ref| <= (2^-10 + K * 2^-24) * mag + 2^-23 * |z_ref|,   mag = s_w * sum_k |x * wq|
(2^-10: dropping thirteen fraction bits of x by truncation; K * 2^-24: K binary32 additions; the
last term: the epilogue's one fma).  Where every operand is a tf32 value and no partial sum needs
more than 24 bits nothing is rounded and the result must be equal bit for bit.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle as orc
from paper_2203_15952_b200 import binding as aqt
from paper_2203_15952_b200 import inputs as gen

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _weights(seed, N, K, bits):
    wt = gen.normal(seed, 900 + bits, N, K, std=1.0 / np.sqrt(K))
    wq, s_w = orc.quantize(wt, bits, orc.AXIS_ROW)
    return wq, s_w, (orc.pack_int4(wq) if bits == 4 else wq)


def _sig(v):
    return 1.0 / (1.0 + np.exp(-v))


def _bound_out(act, z, dz, residual_scale, has_res, y_ref):
    """Propagates the pre-activation bound dz through the activation (Lipschitz constants of the
    textbook functions: |Swish'| <= 1.1, sigmoid' <= 1/4) and the residual fma."""
    n_out = y_ref.shape[1]
    if act == orc.ACT_NONE:
        d = dz
    elif act == orc.ACT_SWISH:
        d = 1.1 * dz
    else:
        zv, zg, dv, dg = z[:, :n_out], z[:, n_out:], dz[:, :n_out], dz[:, n_out:]
        d = dv + (np.abs(zv) + dv) * 0.25 * dg
        if act == orc.ACT_GLU_SWISH:
            d = 1.1 * d
    d = d + 4e-7 * np.abs(z[:, :n_out]) + 1e-30  # the kernel's sigmoid is within 3e-7 of |z|
    if has_res:
        d = abs(residual_scale) * d
    return d + 2.0 ** -23 * np.abs(y_ref)


def _check(M, N, K, bits_w, act, seed=0, residual=False, bias=True, ldx=None, x_scale=1.0, precision=aqt.FLOAT_TF32):
    x = gen.normal(seed, 17, M, K, std=x_scale)
    wq, s_w, w_dev = _weights(seed, N, K, bits_w)
    b = gen.normal(seed, 19, 1, N, std=0.05)[0] if bias else None
    n_out = N // 2 if act >= 2 else N
    res = gen.normal(seed, 23, M, n_out) if residual else None
    y_ref, z, mag = orc.linear_weight_only_f64(x, wq, s_w, bias=b, residual=res, residual_scale=0.5, act=act, return_parts=True)
    if ldx is None:
        xd = _dev(x)
    else:
        buf = torch.full((M, ldx), 7.0, dtype=torch.float32, device=DEV)  # the padding must not be read into the sum
        buf[:, :K] = _dev(x)
        xd = buf[:, :K]
    y = torch.full((M, n_out), float("nan"), dtype=torch.float32, device=DEV)
    aqt.aqt_linear_fwd_weight_only(xd, _dev(w_dev), _dev(s_w), None if b is None else _dev(b), None if res is None else _dev(res), 0.5,
                                   bits_w=bits_w, precision=precision, act=act, y=y)
    assert aqt.aqt_device_status() == 0
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    # two-term form: the dropped part of lo is below 2^-10 of lo, itself below 2^-10 of x; 2K summands
    operand = 2.0 ** -10 if precision == aqt.FLOAT_TF32 else 2.0 ** -20
    terms = K if precision == aqt.FLOAT_TF32 else 2 * K
    dz = (operand + terms * 2.0 ** -24) * mag + 2.0 ** -23 * np.abs(z)
    tol = _bound_out(act, z, dz, 0.5, residual, y_ref)
    err = np.abs(got - y_ref)
    assert np.all(err <= tol), "max err/tol %.3g at %s" % ((err / tol).max(), np.unravel_index((err / tol).argmax(), err.shape))
    return err, tol, mag


@pytest.mark.parametrize("bits_w", [8, 4])
@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (300, 512, 512), (1000, 2048, 512), (257, 512, 2048), (129, 136, 100),
                                   (50, 96, 36), (16, 64, 4), (3, 1024, 1024)])
def test_weight_only_within_the_tf32_bound(M, N, K, bits_w):
    _check(M, N, K, bits_w, orc.ACT_NONE)


@pytest.mark.parametrize("act", [orc.ACT_SWISH, orc.ACT_GLU, orc.ACT_GLU_SWISH])
@pytest.mark.parametrize("bits_w", [8, 4])
def test_weight_only_activations_and_residual(act, bits_w):
    _check(391, 1024, 512, bits_w, act, seed=1)
    _check(200, 512, 256, bits_w, act, seed=2, residual=True)


def test_weight_only_residual_no_bias_and_padded_rows():
    _check(700, 512, 2048, 4, orc.ACT_NONE, seed=3, residual=True, bias=False)
    _check(130, 256, 100, 8, orc.ACT_NONE, seed=4, ldx=128)
    _check(130, 256, 512, 4, orc.ACT_SWISH, seed=5, ldx=516)


@pytest.mark.parametrize("bits_w", [8, 4])
@pytest.mark.parametrize("M,N,K", [(300, 512, 512), (257, 512, 2048), (129, 136, 100), (16, 64, 4)])
def test_weight_only_two_term_form(M, N, K, bits_w):
    _check(M, N, K, bits_w, orc.ACT_NONE, precision=aqt.FLOAT_TF32X2)
    _check(M, N, K, bits_w, orc.ACT_SWISH, seed=1, residual=True, ldx=K + 8, precision=aqt.FLOAT_TF32X2)


def test_weight_only_two_term_form_is_far_more_accurate():
    """x = hi + lo exactly, hi a tf32 value: the operand error of the two-term form is about 2^-20
    of the terms against 2^-10 for one term.  Measured against the same oracle values."""
    e1, _, mag = _check(512, 512, 1024, 8, orc.ACT_NONE, seed=6, bias=False)
    e2, _, _ = _check(512, 512, 1024, 8, orc.ACT_NONE, seed=6, bias=False, precision=aqt.FLOAT_TF32X2)
    assert (e2 / mag).max() < 2.0 ** -18
    assert np.median(e2 / mag) < np.median(e1 / mag) / 64


def test_weight_only_error_is_of_tf32_size_not_larger():
    """The bound is not slack by orders of magnitude: the observed error is a sizeable fraction of
    2^-10 * mag / sqrt(K) (random signs) and far above binary32 rounding, i.e. the test would
    notice both a kernel that is less accurate than stated and a bound that hides a wrong term."""
    err, tol, mag = _check(512, 512, 1024, 8, orc.ACT_NONE, seed=6, bias=False)
    rel = err / mag
    assert rel.max() < 2.0 ** -10
    assert np.median(rel) > 2.0 ** -24


@pytest.mark.parametrize("bits_w", [8, 4])
def test_weight_only_is_exact_on_tf32_inputs(bits_w):
    """x small integers times a power of two (tf32 values), power-of-two channel scales, dyadic
    bias: every product and partial sum fits 24 bits, so the float layer equals the oracle bit for
    bit -- and equals the integer layer on the same codes."""
    r = np.random.default_rng(11)
    M, N, K = 300, 384, 640
    qw = 127 if bits_w == 8 else 7
    xi = r.integers(-15, 16, (M, K))
    x = (xi * 0.125).astype(np.float32)
    wq = r.integers(-qw, qw + 1, (N, K)).astype(np.int8)
    s_w = (2.0 ** r.integers(-6, 2, N)).astype(np.float32)
    bias = (r.integers(-64, 65, N) / 16.0).astype(np.float32)
    y_ref = orc.linear_weight_only_f64(x, wq, s_w, bias=bias)
    assert np.array_equal(y_ref, y_ref.astype(np.float32).astype(np.float64))
    w_dev = orc.pack_int4(wq) if bits_w == 4 else wq
    y = aqt.aqt_linear_fwd_weight_only(_dev(x), _dev(w_dev), _dev(s_w), _dev(bias), bits_w=bits_w)
    assert aqt.aqt_device_status() == 0
    assert np.array_equal(y.cpu().numpy(), y_ref.astype(np.float32))
    # the integer layer on the same numbers: x = 0.125 * codes
    acc = orc.int_matmul(xi.astype(np.int8), wq)
    y_int = orc.epilogue_f32(acc, np.array([0.125], np.float32), orc.SCALE_TENSOR, s_w, bias=bias)
    assert np.array_equal(y.cpu().numpy(), y_int)


def test_weight_only_full_size_ffn_layer_sampled_rows():
    """The first FFN layer at its full size (M = 12 800, 512 -> 2048, int4 weights, Swish), rows
    sampled for the oracle."""
    M, N, K = 12800, 2048, 512
    x = gen.normal(7, 17, M, K)
    wq, s_w, w_dev = _weights(7, N, K, 4)
    y = aqt.aqt_linear_fwd_weight_only(_dev(x), _dev(w_dev), _dev(s_w), None, bits_w=4, act=orc.ACT_SWISH)
    assert aqt.aqt_device_status() == 0
    rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(M - 130, M), np.random.default_rng(0).integers(0, M, 200)]))
    y_ref, z, mag = orc.linear_weight_only_f64(x[rows], wq, s_w, act=orc.ACT_SWISH, return_parts=True)
    dz = (2.0 ** -10 + K * 2.0 ** -24) * mag + 2.0 ** -23 * np.abs(z)
    tol = _bound_out(orc.ACT_SWISH, z, dz, 1.0, False, y_ref)
    assert np.all(np.abs(y.cpu().numpy()[rows].astype(np.float64) - y_ref) <= tol)


@pytest.mark.parametrize("N,K,act,residual", [(512, 512, orc.ACT_NONE, True), (512, 2048, orc.ACT_NONE, False), (1024, 256, orc.ACT_SWISH, False),
                                              (1024, 256, orc.ACT_GLU_SWISH, False), (512, 128, orc.ACT_GLU, True)])
def test_weight_only_many_rows_take_cta_pairs(N, K, act, residual):
    """M = 19 072 rows: from 18 944 rows on (two rounds of 256-row tiles over the SM pairs) the
    float kind runs on CTA pairs, with the eight-warp or (deep K, no activation) four-warp
    epilogue.  Sampled rows against the oracle."""
    M = 19072
    x = gen.normal(9, 17, M, K)
    wq, s_w, w_dev = _weights(9, N, K, 4)
    n_out = N // 2 if act >= 2 else N
    res = gen.normal(9, 23, M, n_out) if residual else None
    y = aqt.aqt_linear_fwd_weight_only(_dev(x), _dev(w_dev), _dev(s_w), None, None if res is None else _dev(res), 0.5, bits_w=4, act=act)
    assert aqt.aqt_device_status() == 0
    rows = np.unique(np.concatenate([np.arange(0, 260), np.arange(M - 260, M), np.random.default_rng(2).integers(0, M, 200)]))
    y_ref, z, mag = orc.linear_weight_only_f64(x[rows], wq, s_w, residual=None if res is None else res[rows], residual_scale=0.5, act=act,
                                               return_parts=True)
    dz = (2.0 ** -10 + K * 2.0 ** -24) * mag + 2.0 ** -23 * np.abs(z)
    tol = _bound_out(act, z, dz, 0.5, residual, y_ref)
    assert np.all(np.abs(y.cpu().numpy()[rows].astype(np.float64) - y_ref) <= tol)


def test_weight_only_argument_errors():
    L = aqt.lib()
    i64, vp, f = ctypes.c_int64, ctypes.c_void_p, ctypes.c_float(1.0)
    one = vp(256)

    def call(M, N, K, bits_w=8, act=0, x=one, ldx=None, ldy=None, ws=one, wsb=1 << 30, precision=0):
        ldx = K if ldx is None else ldx
        ldy = N if ldy is None else ldy
        return L.aqt_linear_fwd_weight_only(x, i64(ldx), one, one, None, None, i64(0), f, i64(M), i64(N), i64(K), bits_w, precision,
                                            act, one, i64(ldy), ws, ctypes.c_size_t(wsb), None)
    assert call(128, 256, 130) == -1            # K not a multiple of 4
    assert call(128, 250, 128) == -1            # N not a multiple of 4
    assert call(128, 260, 128, act=2) == -1     # GLU needs N % 8 == 0
    assert call(128, 256, 128, bits_w=5) == -1
    assert call(128, 256, 128, ldx=64) == -1    # pitch smaller than the row
    assert call(128, 256, 128, ldx=130) == -2   # pitch not a multiple of 4 floats
    assert call(128, 256, 128, x=vp(260)) == -2  # x not 16-byte aligned
    assert call(128, 256, 128, ws=None) == -4
    assert call(128, 256, 128, wsb=1000) == -4
    assert call(128, 256, 128, precision=2) == -1
    assert call(128, 256, 128, precision=1, wsb=4 * 256 * 128) == -4  # the two-term form needs the split activations too
    assert call(0, 256, 128) == 0               # empty: no-op
    assert aqt.aqt_workspace_bytes(aqt.OP_LINEAR_WEIGHT_ONLY, 128, 256, 128, 0, 4) == 4 * 256 * 128
    assert aqt.aqt_workspace_bytes(aqt.OP_LINEAR_WEIGHT_ONLY_X2, 128, 256, 128, 0, 4) == 8 * 256 * 128 + 8 * 128 * 128
