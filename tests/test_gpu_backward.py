"""Parity of the straight-through backward (aqt_linear_bwd) against the CPU oracle, through the
C ABI (needs a B200).

dx and dw are float matmuls on the tensor cores with tf32 operands: the upstream gradient and the
scaled codes (a binary32 product of scale and code) each enter with their upper ten fraction
bits, products are exact, sums binary32.  Tolerance per element, from that arithmetic:
    |g - g_ref| <= (2^-9 + 2^-23 + depth * 2^-24) * mag,   mag = sum of |terms|, depth = N (dx) or M (dw)
dbias is a binary32 sum in a fixed order: |db - db_ref| <= M * 2^-24 * sum |dy|, and the same bits
on every run.  With tf32-exact operands and small integers nothing rounds and results are equal.
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


def _case(seed, M, N, K, bits_a, bits_w):
    r = np.random.default_rng(seed)
    qa, qw = (1 << (bits_a - 1)) - 1, (1 << (bits_w - 1)) - 1
    xq = r.integers(-qa, qa + 1, (M, K)).astype(np.int8)
    wq = r.integers(-qw, qw + 1, (N, K)).astype(np.int8)
    s_x = (r.random(M) * 0.05 + 0.01).astype(np.float32)
    s_w = (r.random(N) * 0.01 + 0.001).astype(np.float32)
    dy = gen.normal(seed, 31, M, N)
    return xq, wq, s_x, s_w, dy


def _check(M, N, K, bits_a=8, bits_w=4, seed=0, kind=aqt.SCALE_ROW, lddy=None):
    xq, wq, s_x, s_w, dy = _case(seed, M, N, K, bits_a, bits_w)
    if kind == aqt.SCALE_TENSOR:
        s_x = s_x[:1]
    dx_ref, dw_ref, db_ref, mx, mw, mb = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w, s_x_kind=kind, return_mags=True)
    xq_d = _dev(orc.pack_int4(xq)) if bits_a == 4 else _dev(xq)
    wq_d = _dev(orc.pack_int4(wq)) if bits_w == 4 else _dev(wq)
    if lddy is None:
        dy_d = _dev(dy)
    else:
        buf = torch.full((M, lddy), 3.0, dtype=torch.float32, device=DEV)  # the padding must stay out of every sum
        buf[:, :N] = _dev(dy)
        dy_d = buf[:, :N]
    dx, dw, db = aqt.aqt_linear_bwd(dy_d, xq_d, _dev(s_x), wq_d, _dev(s_w), K=K, bits_a=bits_a, bits_w=bits_w, s_x_kind=kind)
    assert aqt.aqt_device_status() == 0
    dx, dw, db = dx.cpu().numpy().astype(np.float64), dw.cpu().numpy().astype(np.float64), db.cpu().numpy().astype(np.float64)
    ex = np.abs(dx - dx_ref) / ((2.0 ** -9 + 2.0 ** -23 + N * 2.0 ** -24) * mx + 1e-300)
    ew = np.abs(dw - dw_ref) / ((2.0 ** -9 + 2.0 ** -23 + M * 2.0 ** -24) * mw + 1e-300)
    eb = np.abs(db - db_ref) / (M * 2.0 ** -24 * mb + 1e-300)
    assert ex.max() <= 1.0, "dx %.3g" % ex.max()
    assert ew.max() <= 1.0, "dw %.3g" % ew.max()
    assert eb.max() <= 1.0, "db %.3g" % eb.max()
    return ex, ew


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (300, 512, 512), (1000, 2048, 512), (257, 512, 2048), (129, 136, 100),
                                   (50, 96, 36), (7, 64, 4), (4100, 128, 128)])
@pytest.mark.parametrize("bits_a,bits_w", [(8, 8), (8, 4), (4, 4)])
def test_backward_within_the_tf32_bound(M, N, K, bits_a, bits_w):
    _check(M, N, K, bits_a, bits_w)


def test_backward_per_tensor_scale_padded_gradient_and_partial_outputs():
    _check(200, 256, 128, kind=aqt.SCALE_TENSOR, seed=1)
    _check(333, 512, 256, lddy=520, seed=2)
    xq, wq, s_x, s_w, dy = _case(3, 100, 128, 64, 8, 8)
    dx, dw, db = aqt.aqt_linear_bwd(_dev(dy), None, None, _dev(wq), _dev(s_w), K=64, want_dw=False, want_dbias=False)
    assert dw is None and db is None
    ref = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w, return_mags=True)
    assert np.all(np.abs(dx.cpu().numpy() - ref[0]) <= 2.0 ** -8 * ref[3] + 1e-30)
    dx, dw, db = aqt.aqt_linear_bwd(_dev(dy), _dev(xq), _dev(s_x), None, None, K=64, want_dx=False)
    assert dx is None
    assert np.all(np.abs(dw.cpu().numpy() - ref[1]) <= 2.0 ** -8 * ref[4] + 1e-30)


def test_backward_error_is_of_tf32_size():
    ex, ew = _check(512, 1024, 512, 8, 8, seed=4)
    assert np.median(ex) > 2.0 ** -14 and np.median(ew) > 2.0 ** -14   # the bound is not slack by orders of magnitude


def test_backward_is_exact_on_tf32_inputs_and_deterministic():
    """dy small integers times a power of two, power-of-two scales: every scaled code and every
    partial sum is exact in binary32, so dx, dw and dbias equal the oracle bit for bit."""
    r = np.random.default_rng(5)
    M, N, K = 260, 384, 256
    xq = r.integers(-127, 128, (M, K)).astype(np.int8)
    wq = r.integers(-7, 8, (N, K)).astype(np.int8)
    s_x = (2.0 ** r.integers(-5, 1, M)).astype(np.float32)
    s_w = (2.0 ** r.integers(-6, 1, N)).astype(np.float32)
    dy = (r.integers(-7, 8, (M, N)) * 0.25).astype(np.float32)
    ref = orc.linear_bwd_f64(dy, xq, s_x, wq, s_w)
    assert all(np.array_equal(g, g.astype(np.float32).astype(np.float64)) for g in ref)
    args = (_dev(dy), _dev(xq), _dev(s_x), _dev(orc.pack_int4(wq)), _dev(s_w))
    got = aqt.aqt_linear_bwd(*args, K=K, bits_a=8, bits_w=4)
    assert aqt.aqt_device_status() == 0
    for g, g_ref in zip(got, ref):
        assert np.array_equal(g.cpu().numpy(), g_ref.astype(np.float32))
    again = aqt.aqt_linear_bwd(*args, K=K, bits_a=8, bits_w=4)
    for g, h in zip(got, again):
        assert torch.equal(g.view(torch.int32), h.view(torch.int32))


def test_backward_full_size_ffn_layer_sampled():
    """The first FFN layer at its full size (M = 12 800, 512 -> 2048): sampled rows of dx and
    sampled weight rows of dw against the oracle."""
    M, N, K = 12800, 2048, 512
    xq, wq, s_x, s_w, dy = _case(6, M, N, K, 8, 4)
    dx, dw, db = aqt.aqt_linear_bwd(_dev(dy), _dev(xq), _dev(s_x), _dev(orc.pack_int4(wq)), _dev(s_w), K=K, bits_a=8, bits_w=4)
    assert aqt.aqt_device_status() == 0
    rows = np.unique(np.concatenate([np.arange(0, 40), np.arange(M - 40, M), np.random.default_rng(0).integers(0, M, 60)]))
    dx_ref, _, _, mx, _, _ = orc.linear_bwd_f64(dy[rows], xq[rows], s_x[rows], wq, s_w, return_mags=True)
    assert np.all(np.abs(dx.cpu().numpy()[rows] - dx_ref) <= (2.0 ** -9 + 2.0 ** -23 + N * 2.0 ** -24) * mx)
    cols = np.unique(np.concatenate([np.arange(0, 20), np.arange(N - 20, N), np.random.default_rng(1).integers(0, N, 40)]))
    _, dw_ref, db_ref, _, mw, mb = orc.linear_bwd_f64(np.ascontiguousarray(dy[:, cols]), xq, s_x, wq[cols], s_w[cols], return_mags=True)
    assert np.all(np.abs(dw.cpu().numpy()[cols] - dw_ref) <= (2.0 ** -9 + 2.0 ** -23 + M * 2.0 ** -24) * mw)
    assert np.all(np.abs(db.cpu().numpy()[cols] - db_ref) <= M * 2.0 ** -24 * mb)


def test_backward_argument_errors():
    L = aqt.lib()
    i64, vp = ctypes.c_int64, ctypes.c_void_p
    one = vp(256)

    def call(M, N, K, bits_a=8, bits_w=8, kind=0, dy=one, lddy=None, dx=one, lddx=None, dw=one, ws=one, wsb=1 << 40, xq=one):
        lddy = N if lddy is None else lddy
        lddx = K if lddx is None else lddx
        return L.aqt_linear_bwd(dy, i64(lddy), xq, one, kind, bits_a, one, one, bits_w, i64(M), i64(N), i64(K), dx, i64(lddx), dw,
                                i64(K), None, ws, ctypes.c_size_t(wsb), None)
    assert call(128, 256, 130) == -1              # K not a multiple of 4
    assert call(128, 250, 128) == -1              # N not a multiple of 4
    assert call(128, 256, 128, bits_a=5) == -1
    assert call(128, 256, 128, kind=3) == -1
    assert call(128, 256, 128, lddy=128) == -1    # pitch smaller than the row
    assert call(128, 256, 128, lddy=258) == -2    # pitch not a multiple of 4 floats
    assert call(128, 256, 128, dx=vp(260)) == -2  # dx not 16-byte aligned
    assert call(128, 256, 128, xq=None) == -1     # dw wanted without the activation codes
    assert call(128, 256, 128, ws=None) == -4
    assert call(128, 256, 128, wsb=1000) == -4
    assert call(0, 256, 128) == 0                 # empty: no-op
    assert aqt.aqt_workspace_bytes(aqt.OP_LINEAR_BWD, 128, 256, 128, 0, 0) >= 4 * (128 * 256 + (256 + 128) * 128)
