"""Parity of the matmul that quantizes its own output rows (Fig. 2 applied in the epilogue) against
the CPU oracle, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2203_15952_b200 import binding as aqt

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _codes(rng, rows, K, bits):
    qm = 127 if bits == 8 else 7
    return rng.integers(-qm, qm + 1, (rows, K)).astype(np.int8)


def _run(M, N, K, bits_a, bits_w, act, with_bias, with_res, bits_out, rounding, pack_out, special_rows=False,
         may_refuse_without_y=False):
    rng = np.random.default_rng(7 + 1000 * M + N + K + bits_out)
    xq = _codes(rng, M, K, bits_a)
    wq = _codes(rng, N, K, bits_w)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    if special_rows:
        xq[0, :] = 0                       # with no bias: an all-zero output row (scale 0, codes 0)
        if M > 2:
            s_x[1] = 1e-37                 # a row whose maximum is far below the fast-division range
            s_x[2] = 3e33                  # and one far above it
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32) if with_bias else None
    res = rng.standard_normal((M, N)).astype(np.float32) if with_res else None
    acc_ref = orc.int_matmul(xq, wq)
    y_ref = orc.epilogue_f32(acc_ref, s_x, aqt.SCALE_ROW, s_w, bias, res, 0.5, act)
    y64 = orc.epilogue_f64(acc_ref, s_x, aqt.SCALE_ROW, s_w, bias, res, 0.5, act)

    xq_d = _dev(orc.pack_int4(xq)) if bits_a == 4 else _dev(xq)
    wq_d = _dev(orc.pack_int4(wq)) if bits_w == 4 else _dev(wq)
    args = (xq_d, _dev(s_x), wq_d, _dev(s_w), None if bias is None else _dev(bias), None if res is None else _dev(res), 0.5)
    kw = dict(K=K, bits_a=bits_a, bits_w=bits_w, act=act, bits_out=bits_out, rounding=rounding, pack_out=pack_out)
    q_shape = (M, N // 2) if pack_out else (M, N)
    q_d = torch.full(q_shape, 0x55, dtype=torch.uint8 if pack_out else torch.int8, device=DEV)
    s_d = torch.full((M,), float("nan"), dtype=torch.float32, device=DEV)
    y_d = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    aqt.aqt_qmatmul_requant(*args, **kw, q_out=q_d, s_out=s_d, y=y_d)
    assert aqt.aqt_device_status() == 0
    y = y_d.cpu().numpy()
    q = q_d.cpu().numpy()
    s = s_d.cpu().numpy()

    # the fp32 output: the same bar as the plain matmul
    if act == aqt.ACT_NONE:
        assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))
    else:
        assert np.isfinite(y).all()
        z = orc.epilogue_f64(acc_ref, s_x, aqt.SCALE_ROW, s_w, None, None, 0.0, aqt.ACT_NONE)
        mag = np.maximum(np.abs(y64), np.abs(z))
        if bias is not None:
            mag = np.maximum(mag, np.abs(bias)[None, :])
        if res is not None:
            mag = np.maximum(mag, np.abs(res))
        assert np.all(np.abs(y - y64) <= 1e-6 * mag + 1e-30), float(np.max(np.abs(y - y64) / (mag + 1e-30)))

    # codes and scales: the oracle's quantizer on the rows the kernel itself produced, bit for bit
    q_ref, s_ref = orc.quantize(y, bits_out, orc.AXIS_ROW, rounding)
    assert np.array_equal(s.view(np.uint32), s_ref.reshape(-1).view(np.uint32)), "scales differ in %d rows" % (s != s_ref.reshape(-1)).sum()
    q_cmp = orc.pack_int4(q_ref) if pack_out else q_ref
    assert np.array_equal(q, q_cmp), "codes differ: %d of %d" % ((q != q_cmp).sum(), q.size)
    if act == aqt.ACT_NONE:
        q_ref2, s_ref2 = orc.quantize(y_ref, bits_out, orc.AXIS_ROW, rounding)   # nothing of the kernel's in the reference
        assert np.array_equal(q_ref2, q_ref) and np.array_equal(s_ref2, s_ref)

    # without the fp32 output the codes are the same ones
    if res is None:
        q2_d = torch.full(q_shape, 0x55, dtype=q_d.dtype, device=DEV)
        s2_d = torch.full((M,), float("nan"), dtype=torch.float32, device=DEV)
        try:
            _, _, y_none = aqt.aqt_qmatmul_requant(*args, **kw, q_out=q2_d, s_out=s2_d)
        except aqt.AqtError as e:
            # shapes no fused kernel takes need the fp32 output as the hand-over between the two steps
            assert may_refuse_without_y and e.status == -3
            return
        assert y_none is None
        assert aqt.aqt_device_status() == 0
        assert torch.equal(q2_d, q_d) and torch.equal(s2_d.view(torch.int32), s_d.view(torch.int32))


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (128, 256, 128), (256, 512, 512), (300, 2048, 512), (1000, 512, 256),
                                   (40, 144, 144), (5000, 1024, 384), (129, 2064, 96)])
@pytest.mark.parametrize("act", [aqt.ACT_NONE, aqt.ACT_SWISH])
def test_requant_w8a8(M, N, K, act):
    _run(M, N, K, 8, 8, act, True, False, 8, aqt.ROUND_NEAREST_EVEN, False)


@pytest.mark.parametrize("bits_a,bits_w,bits_out,pack_out", [(8, 4, 8, False), (4, 4, 4, True), (8, 4, 4, False), (4, 8, 8, False)])
@pytest.mark.parametrize("rounding", [aqt.ROUND_NEAREST_EVEN, aqt.ROUND_HALF_UP_FLOOR])
def test_requant_bit_widths_and_rounding(bits_a, bits_w, bits_out, pack_out, rounding):
    _run(700, 1024, 512, bits_a, bits_w, aqt.ACT_SWISH, True, False, bits_out, rounding, pack_out)
    _run(333, 512, 256, bits_a, bits_w, aqt.ACT_NONE, False, False, bits_out, rounding, pack_out, special_rows=True)


@pytest.mark.parametrize("M,N,K", [(256, 512, 512), (1300, 512, 128), (77, 1024, 512)])
@pytest.mark.parametrize("act", [aqt.ACT_NONE, aqt.ACT_SWISH])
def test_requant_with_residual_stream(M, N, K, act):
    _run(M, N, K, 8, 4, act, True, True, 8, aqt.ROUND_NEAREST_EVEN, False)


def test_requant_with_residual_stream_many_tiles_per_cta():
    """Six tiles per CTA with residual and fp32 output: the sets overlap, so chunks of the residual
    of several tiles are wanted at the same time while the residual ring holds two."""
    _run(6000, 2048, 128, 8, 4, aqt.ACT_SWISH, True, True, 8, aqt.ROUND_NEAREST_EVEN, False)
    _run(5000, 512, 256, 8, 8, aqt.ACT_NONE, False, True, 4, aqt.ROUND_HALF_UP_FLOOR, True)


def test_requant_many_tiles_per_cta():
    """More m-tiles than groups of CTAs: every TMEM buffer and both exchange slots are reused."""
    _run(12800, 2048, 512, 8, 4, aqt.ACT_SWISH, False, False, 8, aqt.ROUND_NEAREST_EVEN, False)


@pytest.mark.parametrize("M,N,K,bits_w,act", [(300, 1024, 1024, 4, aqt.ACT_SWISH), (1500, 4096, 1024, 4, aqt.ACT_SWISH),
                                               (129, 512, 640, 8, aqt.ACT_NONE), (700, 2048, 1024, 8, aqt.ACT_SWISH),
                                               (260, 1024, 768, 4, aqt.ACT_NONE)])
def test_requant_deep_k_form(M, N, K, bits_w, act):
    """512 < K <= 1024 (the d = 1024 encoder): the fused kernel with an eight-k-block weight slab
    takes the call when only codes and scales are wanted.  _run checks the two-step path (with y)
    against the oracle and then the fused path (without y) against it, bit for bit."""
    _run(M, N, K, 8, bits_w, act, True, False, 8, aqt.ROUND_NEAREST_EVEN, False)
    # (the huge-scale special row stays finite only with 4-bit weights at this depth)
    _run(M, N, K, 8, bits_w, act, False, False, 4, aqt.ROUND_HALF_UP_FLOOR, True, special_rows=(bits_w == 4))


@pytest.mark.parametrize("act", [aqt.ACT_GLU, aqt.ACT_GLU_SWISH])
@pytest.mark.parametrize("M,N,K,bits_w", [(128, 128, 128, 8), (300, 1024, 512, 4), (1000, 2048, 256, 4), (77, 288, 144, 8),
                                           (2600, 1024, 512, 8), (129, 4224, 64, 4), (300, 2048, 1024, 4), (129, 512, 640, 8)])
def test_requant_glu_forms(act, M, N, K, bits_w):
    """The GLU forms (a tile = 64 value + 64 gate channels -> 64 output columns).  With y the call
    runs matmul + quantizer through y, which is checked against the oracle like every other form;
    without y the fused kernel must give the very same codes and scales."""
    for rounding, bits_out in ((aqt.ROUND_NEAREST_EVEN, 8), (aqt.ROUND_HALF_UP_FLOOR, 4)):
        rng = np.random.default_rng(11 + M + N + K + bits_out)
        xq, wq = _codes(rng, M, K, 8), _codes(rng, N, K, bits_w)
        s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
        s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
        bias = (rng.standard_normal(N) * 0.1).astype(np.float32)
        acc_ref = orc.int_matmul(xq, wq)
        y64 = orc.epilogue_f64(acc_ref, s_x, aqt.SCALE_ROW, s_w, bias, None, 0.0, act)
        z = orc.epilogue_f64(acc_ref, s_x, aqt.SCALE_ROW, s_w, None, None, 0.0, aqt.ACT_NONE)
        wq_d = _dev(orc.pack_int4(wq)) if bits_w == 4 else _dev(wq)
        args = (_dev(xq), _dev(s_x), wq_d, _dev(s_w), _dev(bias), None, 1.0)
        kw = dict(K=K, bits_a=8, bits_w=bits_w, act=act, bits_out=bits_out, rounding=rounding, pack_out=False)
        n_out = N // 2
        q_y, s_y, y_d = aqt.aqt_qmatmul_requant(*args, **kw, want_y=True)          # two steps through y
        q_d = torch.full((M, n_out), 0x55, dtype=torch.int8, device=DEV)
        s_d = torch.full((M,), float("nan"), dtype=torch.float32, device=DEV)
        _, _, y_none = aqt.aqt_qmatmul_requant(*args, **kw, q_out=q_d, s_out=s_d)    # the fused kernel
        assert y_none is None and aqt.aqt_device_status() == 0
        y = y_d.cpu().numpy()
        mag = np.maximum(np.maximum(np.abs(y64), np.abs(z[:, :n_out])), np.abs(bias)[None, :n_out])
        assert np.all(np.abs(y - y64) <= 1e-6 * mag + 1e-30)
        q_ref, s_ref = orc.quantize(y, bits_out, orc.AXIS_ROW, rounding)
        assert np.array_equal(s_y.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)) and np.array_equal(q_y.cpu().numpy(), q_ref)
        assert np.array_equal(s_d.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)), "fused scales differ"
        assert np.array_equal(q_d.cpu().numpy(), q_ref), "fused codes differ: %d" % (q_d.cpu().numpy() != q_ref).sum()


@pytest.mark.parametrize("M,N,K,act", [(300, 1024, 1024, aqt.ACT_NONE), (1500, 1024, 1024, aqt.ACT_SWISH), (129, 1040, 640, aqt.ACT_NONE),
                                       (2000, 2064, 896, aqt.ACT_NONE)])
def test_requant_deep_k_with_residual_stream(M, N, K, act):
    """The d = 1024 encoder's attention output and second pointwise layers: 512 < K <= 1024 with
    residual and fp32 output next to the codes (matmul, then the row quantizer, inside the one
    call); N with a ragged last tile."""
    _run(M, N, K, 8, 4, act, True, True, 8, aqt.ROUND_NEAREST_EVEN, False)
    _run(M, N, K, 8, 8, act, False, True, 4, aqt.ROUND_NEAREST_EVEN, N % 32 == 0)


@pytest.mark.parametrize("seed", range(24))
def test_requant_random_shapes(seed):
    """Seeded random shapes inside the limits of the call (K a multiple of 16, output width a
    multiple of 32): every form it dispatches to (fused K <= 512, eight-k-block, CTA pairs from
    K = 2048, matmul + quantizer in between) against the oracle."""
    rng = np.random.default_rng(400 + seed)
    K = int(rng.choice([16, 64, 144, 256, 512, 640, 1024, 1536, 2048, 4096]))
    N = 32 * int(rng.integers(1, 65))
    M = int(rng.integers(1, 3000))
    while M * N * K > 3e8:
        if N > 128:
            N = 32 * max(1, (N // 32) // 2)
        else:
            M = max(1, M // 2)
    bits_a, bits_w = [(8, 8), (8, 4), (4, 4), (4, 8)][int(rng.integers(0, 4))]
    act = [aqt.ACT_NONE, aqt.ACT_SWISH][int(rng.integers(0, 2))]
    bits_out = [8, 4][int(rng.integers(0, 2))]
    pack_out = bits_out == 4 and bool(rng.integers(0, 2))
    rounding = [aqt.ROUND_NEAREST_EVEN, aqt.ROUND_HALF_UP_FLOOR][int(rng.integers(0, 2))]
    _run(M, N, K, bits_a, bits_w, act, bool(rng.integers(0, 2)), bool(rng.integers(0, 2)), bits_out, rounding, pack_out,
         may_refuse_without_y=K > 1024)


def test_requant_unfused_shapes_go_through_y():
    """K > 1024 (and K > 512 or the GLU forms with an fp32 output) are not taken by the fused
    kernel: the call runs the two steps through y."""
    _run(200, 512, 2048, 8, 4, aqt.ACT_NONE, True, True, 8, aqt.ROUND_NEAREST_EVEN, False)
    rng = np.random.default_rng(3)
    xq, wq = _codes(rng, 64, 2048, 8), _codes(rng, 256, 2048, 8)
    with pytest.raises(aqt.AqtError) as e:
        aqt.aqt_qmatmul_requant(_dev(xq), _dev(np.ones(64, np.float32)), _dev(wq), _dev(np.ones(256, np.float32)), K=2048)
    assert e.value.status == -3


@pytest.mark.parametrize("M,N,K", [(1, 512, 512), (16, 2048, 256), (127, 640, 128), (129, 2304, 512), (260, 4224, 64), (3000, 128, 512)])
def test_requant_edge_shapes(M, N, K):
    """One row, fewer m-tiles than groups of CTAs, a ragged last m-tile, more than sixteen n-tiles
    (the exchange warp then reads the row maxima in several batches), a single n-tile."""
    _run(M, N, K, 8, 8, aqt.ACT_SWISH, True, False, 8, aqt.ROUND_NEAREST_EVEN, False)
    _run(M, N, K, 8, 4, aqt.ACT_NONE, False, M > 100, 4, aqt.ROUND_HALF_UP_FLOOR, True)


def test_requant_argument_checks():
    z8 = torch.zeros((64, 64), dtype=torch.int8, device=DEV)
    w8 = torch.zeros((48, 64), dtype=torch.int8, device=DEV)
    one = torch.ones(64, device=DEV)
    with pytest.raises(aqt.AqtError) as e:   # N_out not a multiple of 16
        aqt.aqt_qmatmul_requant(z8, one, w8[:40], one[:40], K=64)
    assert e.value.status == -1
    with pytest.raises(aqt.AqtError) as e:   # packing needs 4-bit output codes
        aqt.aqt_qmatmul_requant(z8, one, w8, one[:48], K=64, bits_out=8, pack_out=True)
    assert e.value.status == -1
    with pytest.raises(aqt.AqtError) as e:   # packed rows need N_out % 32 == 0
        aqt.aqt_qmatmul_requant(z8, one, w8, one[:48], K=64, bits_out=4, pack_out=True)
    assert e.value.status == -1
    q, s_, y = aqt.aqt_qmatmul_requant(z8[:0], one[:0], w8, one[:48], K=64)   # empty batch: nothing to do
    assert q.shape == (0, 48) and y is None
    assert aqt.aqt_device_status() == 0


@pytest.mark.parametrize("M,N,K,act,with_res", [(600, 512, 2048, aqt.ACT_NONE, True), (700, 1024, 4096, aqt.ACT_SWISH, False),
                                                 (300, 768, 2048, aqt.ACT_NONE, True), (513, 256, 4096, aqt.ACT_SWISH, True),
                                                 (129, 1536, 1024, aqt.ACT_NONE, False)])
def test_requant_second_ffn_layers_small(M, N, K, act, with_res):
    """K = 1024 .. 4096 (the second feed-forward layers): the CTA-pair kernel quantizes its output
    rows in the epilogue, with the fp32 output (a residual stream) and without it.  Row maxima
    come from several warps and, beyond 512 columns, several CTA pairs."""
    _run(M, N, K, 8, 4, act, True, with_res, 8, aqt.ROUND_NEAREST_EVEN, False, special_rows=True)
    _run(M, N, K, 8, 8 if K <= 2048 else 4, act, False, with_res, 4, aqt.ROUND_HALF_UP_FLOOR, False)


@pytest.mark.parametrize("M,N,K,plan", [(25600, 512, 2048, "pair256s4e8"), (12800, 512, 2048, "pair512s3e16"),
                                        (30000, 1024, 4096, "pair256s6e4")])
def test_requant_second_ffn_layers_full_size_sampled_rows(M, N, K, plan):
    """The second feed-forward layers at the workloads' sizes: fp32 output with residual + codes
    and scales, sampled rows against the oracle; every row's largest |code| is 127."""
    from paper_2203_15952_b200 import inputs as gen
    rng = np.random.default_rng(M + N)
    xq = gen.random_codes(41, M, K, 8)
    wq = gen.random_codes(42, N, K, 4)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    res = rng.standard_normal((M, N), dtype=np.float32)
    xq_d, wq_d, res_d = _dev(xq), _dev(wq), _dev(res)
    y_d = torch.full((M, N), float("nan"), dtype=torch.float32, device=DEV)
    q_d, s_d, _ = aqt.aqt_qmatmul_requant(xq_d, _dev(s_x), wq_d, _dev(s_w), None, res_d, 0.5, K=K, bits_a=8, bits_w=aqt.BITS_4_UNPACKED,
                                          bits_out=8, y=y_d)
    q2_d, s2_d, y_none = aqt.aqt_qmatmul_requant(xq_d, _dev(s_x), wq_d, _dev(s_w), None, None, 0.5, K=K, bits_a=8,
                                                 bits_w=aqt.BITS_4_UNPACKED, bits_out=8)
    assert aqt.aqt_device_status() == 0 and y_none is None
    rows = sorted(set([0, 127, 128, 255, 256, 511, M - 257, M - 129, M - 1]) | set(rng.integers(0, M, 30).tolist()))
    acc_ref = orc.int_matmul(xq[rows], wq)
    y_ref = orc.epilogue_f32(acc_ref, s_x[rows], aqt.SCALE_ROW, s_w, None, res[rows], 0.5, aqt.ACT_NONE)
    assert np.array_equal(y_d[rows].cpu().numpy().view(np.uint32), y_ref.view(np.uint32))
    q_ref, s_ref = orc.quantize(y_ref, 8, orc.AXIS_ROW)
    assert np.array_equal(q_d[rows].cpu().numpy(), q_ref) and np.array_equal(s_d[rows].cpu().numpy(), s_ref.reshape(-1))
    # without residual and fp32 output
    u_ref = orc.epilogue_f32(acc_ref, s_x[rows], aqt.SCALE_ROW, s_w, None, None, 0.0, aqt.ACT_NONE)
    q_ref2, s_ref2 = orc.quantize(u_ref, 8, orc.AXIS_ROW)
    assert np.array_equal(q2_d[rows].cpu().numpy(), q_ref2) and np.array_equal(s2_d[rows].cpu().numpy(), s_ref2.reshape(-1))
    assert int(q_d.abs().max(dim=1).values.min()) == 127 and int(q2_d.abs().max(dim=1).values.min()) == 127
    # the GPU row quantizer on the fp32 output gives the same codes everywhere
    q3, s3 = aqt.aqt_quantize(y_d, 8, aqt.AXIS_ROW)
    assert torch.equal(q3, q_d) and torch.equal(s3.view(torch.int32), s_d.view(torch.int32))
