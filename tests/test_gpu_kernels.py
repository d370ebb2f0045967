"""Parity of each CUDA kernel against the CPU oracle, through the C ABI (needs a B200)."""
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


def _status_ok():
    assert aqt.aqt_device_status() == 0


# ----------------------------------------------------------------------------- quantizer

@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("rounding", [orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN])
@pytest.mark.parametrize("shape", [(64, 256), (300, 512), (131, 1024), (70, 2048), (33, 4096), (40, 96), (17, 4100), (9, 37), (5, 8192)])
def test_quantize_rows_bit_exact(bits, rounding, shape):
    x = gen.normal(1, 100 + bits, shape[0], shape[1], std=1.7)
    x[0, :] = 0.0                                     # zero row
    x[1, 0] = 1e-41                                   # subnormal element
    if shape[0] > 3:
        x[2, :] *= 1e-30                              # tiny row (slow division path)
        x[3, :] *= 1e25                               # huge row
    q_ref, s_ref = orc.quantize(x, bits, orc.AXIS_ROW, rounding)
    q, s = aqt.aqt_quantize(_dev(x), bits, aqt.AXIS_ROW, rounding)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), q_ref)
    if shape[1] % 2 == 0 and bits == 4:
        qp, s2 = aqt.aqt_quantize(_dev(x), 4, aqt.AXIS_ROW, rounding, pack=True)
        assert np.array_equal(qp.cpu().numpy(), orc.pack_int4(q_ref))
        assert np.array_equal(s2.cpu().numpy(), s_ref)


def test_quantize_ties_and_half_ulp_cases():
    """Exact ties and values one ulp either side of them, on the GPU's division sequence."""
    base = np.arange(-127, 127, dtype=np.float32) + 0.5
    vals = np.concatenate([base, np.nextafter(base, np.float32(1e9)), np.nextafter(base, np.float32(-1e9)), [127.0]]).astype(np.float32)
    vals = np.concatenate([vals, np.zeros((-len(vals)) % 4, np.float32)])
    x = np.stack([vals, vals * np.float32(3.0), vals * np.float32(0.1), vals * np.float32(1e-3)])
    for rounding in (orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN):
        q_ref, s_ref = orc.quantize(x, 8, orc.AXIS_ROW, rounding)
        q, s = aqt.aqt_quantize(_dev(x), 8, aqt.AXIS_ROW, rounding)
        assert np.array_equal(s.cpu().numpy(), s_ref) and np.array_equal(q.cpu().numpy(), q_ref)


def test_quantize_strided_rows():
    big = gen.normal(2, 5, 50, 640)
    xd = _dev(big)[:, :512]
    q_ref, s_ref = orc.quantize(np.ascontiguousarray(big[:, :512]), 8, orc.AXIS_ROW)
    q, s = aqt.aqt_quantize(xd, 8, aqt.AXIS_ROW)
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)


@pytest.mark.parametrize("axis", [orc.AXIS_COL, orc.AXIS_TENSOR])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("shape", [(64, 256), (512, 2048), (37, 53), (1000, 6)])
def test_quantize_col_and_tensor_axes_bit_exact(axis, bits, shape):
    x = gen.normal(3, 7, shape[0], shape[1], std=0.05)
    for rounding in (orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN):
        q_ref, s_ref = orc.quantize(x, bits, axis, rounding)
        q, s = aqt.aqt_quantize(_dev(x), bits, axis, rounding)
        assert np.array_equal(s.cpu().numpy(), s_ref) and np.array_equal(q.cpu().numpy(), q_ref)
    if bits == 4 and shape[1] % 2 == 0:
        qp, _ = aqt.aqt_quantize(_dev(x), 4, axis, orc.ROUND_NEAREST_EVEN, pack=True)
        assert np.array_equal(qp.cpu().numpy(), orc.pack_int4(orc.quantize(x, 4, axis)[0]))


def test_quantize_heavy_tailed_rows():
    x = gen.student_t3(0, 77, 256, 1024)
    q_ref, s_ref = orc.quantize(x, 8, orc.AXIS_ROW)
    q, s = aqt.aqt_quantize(_dev(x), 8, aqt.AXIS_ROW)
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)


# ----------------------------------------------------------------------------- pack / unpack

@pytest.mark.parametrize("shape", [(225, 2), (7, 90), (128, 512), (3, 4098), (1, 16)])
def test_pack_unpack_bit_exact(shape):
    rng = np.random.default_rng(shape[0])
    q = rng.integers(-7, 8, shape).astype(np.int8)
    packed_ref = orc.pack_int4(q)
    packed = aqt.aqt_pack_int4(_dev(q))
    assert np.array_equal(packed.cpu().numpy(), packed_ref)
    assert np.array_equal(aqt.aqt_unpack_int4(packed, shape[1]).cpu().numpy(), q)
    assert np.array_equal(aqt.aqt_unpack_int4(_dev(packed_ref), shape[1]).cpu().numpy(), orc.unpack_int4(packed_ref, shape[1]))


# ----------------------------------------------------------------------------- integer matmul + epilogue

def _codes(rng, rows, K, bits):
    qm = 127 if bits == 8 else 7
    return rng.integers(-qm, qm + 1, (rows, K)).astype(np.int8)


def _run_qmatmul(M, N, K, bits_a, bits_w, act, with_bias, with_res, s_x_kind=aqt.SCALE_ROW, seed=0, extremes=False, plan=None,
                 unpacked4=False):
    """One aqt_qmatmul call against the oracle.  plan: a kernel configuration by name instead of
    the library's choice.  unpacked4: 4-bit codes handed over in int8 containers (AQT_BITS_4_UNPACKED)."""
    rng = np.random.default_rng(seed + 1000 * M + N + K)
    xq = _codes(rng, M, K, bits_a)
    wq = _codes(rng, N, K, bits_w)
    if extremes:
        xq[0, :] = 127 if bits_a == 8 else 7
        wq[0, :] = 127 if bits_w == 8 else 7
        wq[1 % N, :] = -wq[0, :]
    s_x = rng.uniform(1e-3, 5e-2, M if s_x_kind == aqt.SCALE_ROW else 1).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.1).astype(np.float32) if with_bias else None
    n_out = N // 2 if act in (aqt.ACT_GLU, aqt.ACT_GLU_SWISH) else N
    res = rng.standard_normal((M, n_out)).astype(np.float32) if with_res else None
    acc_ref = orc.int_matmul(xq, wq)
    y_ref = orc.epilogue_f32(acc_ref, s_x, s_x_kind, s_w, bias, res, 0.5, act)
    y64 = orc.epilogue_f64(acc_ref, s_x, s_x_kind, s_w, bias, res, 0.5, act)

    xq_d = _dev(orc.pack_int4(xq)) if (bits_a == 4 and not unpacked4) else _dev(xq)
    wq_d = _dev(orc.pack_int4(wq)) if (bits_w == 4 and not unpacked4) else _dev(wq)
    arg_a = aqt.BITS_4_UNPACKED if (bits_a == 4 and unpacked4) else bits_a
    arg_w = aqt.BITS_4_UNPACKED if (bits_w == 4 and unpacked4) else bits_w
    acc_d = torch.full((M, N), -12345, dtype=torch.int32, device=DEV)
    y_d = torch.full((M, n_out), float("nan"), dtype=torch.float32, device=DEV)
    aqt.aqt_qmatmul(xq_d, _dev(s_x), wq_d, _dev(s_w), None if bias is None else _dev(bias),
                    None if res is None else _dev(res), 0.5, K=K, bits_a=arg_a, bits_w=arg_w, act=act,
                    s_x_kind=s_x_kind, y=y_d, acc_debug=acc_d, plan=plan)
    _status_ok()
    # the production instantiation (no accumulator dump) writes the same output bits
    y_p = torch.full((M, n_out), float("nan"), dtype=torch.float32, device=DEV)
    aqt.aqt_qmatmul(xq_d, _dev(s_x), wq_d, _dev(s_w), None if bias is None else _dev(bias),
                    None if res is None else _dev(res), 0.5, K=K, bits_a=arg_a, bits_w=arg_w, act=act,
                    s_x_kind=s_x_kind, y=y_p, plan=plan)
    _status_ok()
    assert torch.equal(y_p.view(torch.int32), y_d.view(torch.int32))
    acc = acc_d.cpu().numpy()
    y = y_d.cpu().numpy()
    assert np.array_equal(acc.astype(np.int64), acc_ref), "accumulators differ: %d of %d" % ((acc != acc_ref).sum(), acc.size)
    if act == aqt.ACT_NONE:
        assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))          # only IEEE ops: bit-exact
    else:
        assert np.isfinite(y).all()
        # float tolerance: 1e-6 relative to the larger of the result and the terms it is formed from
        # (the de-quantized sum acc * s_x * s_w and the bias, which may cancel; the residual)
        z = orc.epilogue_f64(acc_ref, s_x, s_x_kind, s_w, None, None, 0.0, aqt.ACT_NONE)
        mag = np.maximum(np.abs(y64), np.abs(z[:, :n_out]))
        if bias is not None:
            mag = np.maximum(mag, np.abs(bias[:n_out])[None, :])
        if res is not None:
            mag = np.maximum(mag, np.abs(res))
        assert np.all(np.abs(y - y64) <= 1e-6 * mag + 1e-30), float(np.max(np.abs(y - y64) / (mag + 1e-30)))


@pytest.mark.parametrize("M,N,K", [(128, 64, 128), (128, 128, 128), (128, 256, 128), (128, 256, 512), (256, 512, 256)])
def test_qmatmul_single_tiles_int8(M, N, K):
    _run_qmatmul(M, N, K, 8, 8, aqt.ACT_NONE, False, False, extremes=True)


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (200, 192, 96), (1000, 520, 160), (129, 36, 32), (1, 4, 32), (333, 1536, 512)])
def test_qmatmul_ragged_shapes(M, N, K):
    _run_qmatmul(M, N, K, 8, 8, aqt.ACT_NONE, True, True)


@pytest.mark.parametrize("bits_a,bits_w", [(8, 4), (4, 4), (4, 8)])
@pytest.mark.parametrize("M,N,K", [(384, 512, 512), (130, 200, 2048)])
def test_qmatmul_int4_operands(bits_a, bits_w, M, N, K):
    _run_qmatmul(M, N, K, bits_a, bits_w, aqt.ACT_NONE, True, False, extremes=True)


@pytest.mark.parametrize("act", [aqt.ACT_SWISH, aqt.ACT_GLU, aqt.ACT_GLU_SWISH])
@pytest.mark.parametrize("M,N,K", [(256, 512, 256), (300, 1024, 512), (100, 136, 64)])
def test_qmatmul_activations(act, M, N, K):
    if act != aqt.ACT_SWISH and M > 128:
        assert aqt.aqt_plan_qmatmul(M, N, K, 8, 4, act) == "ws128e8"      # the GLU forms of the weight-stationary kernel
    _run_qmatmul(M, N, K, 8, 4, act, True, True)


@pytest.mark.parametrize("plan", ["stream128s4e8", "stream256s3e16"])
def test_qmatmul_glu_streaming_plan_named(plan):
    """GLU on the streaming kernel (K > 512: value and gate rows of a tile are two boxes of the ring)."""
    _run_qmatmul(600, 1024, 1024, 8, 4, aqt.ACT_GLU_SWISH, True, True, plan=plan)
    _run_qmatmul(300, 512, 640, 8, 8, aqt.ACT_GLU, False, False, plan=plan)


@pytest.mark.parametrize("M", [4, 200, 1300])
@pytest.mark.parametrize("N,K,act,bits_a,bits_w", [(576, 144, aqt.ACT_SWISH, 8, 4), (144, 576, aqt.ACT_NONE, 8, 4), (144, 144, aqt.ACT_NONE, 4, 4),
                                                    (288, 144, aqt.ACT_GLU_SWISH, 8, 8), (144, 1168, aqt.ACT_NONE, 8, 4)])
def test_qmatmul_conformer_s_widths(M, N, K, act, bits_a, bits_w):
    """Model width 144 (the paper's Conformer S, Section 3.2): K is a multiple of 16 but not of 32 or
    128, so the last k-block is partly outside the tensor and packed rows are 72 bytes."""
    _run_qmatmul(M, N, K, bits_a, bits_w, act, True, True, extremes=True)


def test_linear_fwd_conformer_s_width():
    M, K, N = 333, 144, 576
    x = gen.normal(8, 1, M, K)
    wt = gen.weight(8, 2, K, N)
    wq, s_w = orc.quantize(wt, 4, orc.AXIS_ROW)
    y_ref = orc.linear_fwd(x, wq, s_w)
    wq_d, sw_d = aqt.aqt_quantize(_dev(wt), 4, aqt.AXIS_ROW, pack=True)
    assert np.array_equal(wq_d.cpu().numpy(), orc.pack_int4(wq))
    y = aqt.aqt_linear_fwd(_dev(x), wq_d, sw_d, bits_a=8, bits_w=4)
    _status_ok()
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


def _random_matmul_case(seed, row_quantizing=False):
    """A seeded random shape and operand mix inside the documented limits (K a multiple of 16, N a
    multiple of 16 or, for the GLU forms, 32), small enough for the oracle: M N K <= 3e8."""
    rng = np.random.default_rng(900 + seed)
    act = [aqt.ACT_NONE, aqt.ACT_SWISH, aqt.ACT_GLU, aqt.ACT_GLU_SWISH][int(rng.integers(0, 4))]
    K = int(rng.choice([16, 48, 96, 128, 144, 256, 384, 512, 640, 768, 1024, 1536, 2048, 4096]))
    n_step = 64 if act in (aqt.ACT_GLU, aqt.ACT_GLU_SWISH) else 32
    N = n_step * int(rng.integers(1, 2304 // n_step + 1))
    M = int(rng.integers(1, 2600))
    while M * N * K > 3e8:
        if N > 4 * n_step:
            N = n_step * max(1, (N // n_step) // 2)
        else:
            M = max(1, M // 2)
    bits_a, bits_w = [(8, 8), (8, 4), (4, 4), (4, 8)][int(rng.integers(0, 4))]
    return M, N, K, bits_a, bits_w, act, bool(rng.integers(0, 2)), bool(rng.integers(0, 2))


@pytest.mark.parametrize("seed", range(24))
def test_qmatmul_random_shapes(seed):
    """Shapes nobody picked by hand: whatever kernel configuration the library chooses for them
    must give the oracle's accumulators and outputs."""
    M, N, K, bits_a, bits_w, act, with_bias, with_res = _random_matmul_case(seed)
    _run_qmatmul(M, N, K, bits_a, bits_w, act, with_bias, with_res, seed=seed)


def test_qmatmul_per_tensor_scale_and_deep_k():
    _run_qmatmul(256, 256, 4096, 8, 8, aqt.ACT_NONE, True, False, s_x_kind=aqt.SCALE_TENSOR, extremes=True)


def test_qmatmul_many_tiles_persistent_loop():
    """More tiles than SMs, so every CTA walks several tiles and both accumulator buffers."""
    _run_qmatmul(128 * 40, 2048, 512, 8, 8, aqt.ACT_SWISH, False, False)
    _run_qmatmul(128 * 37 + 5, 512, 2048, 8, 8, aqt.ACT_NONE, False, True)


@pytest.mark.parametrize("M", [1, 3, 8, 9, 16, 17])
@pytest.mark.parametrize("N,K,act,bits_a,bits_w", [(2048, 512, aqt.ACT_SWISH, 8, 4), (512, 2048, aqt.ACT_NONE, 8, 4),
                                                    (1024, 512, aqt.ACT_GLU_SWISH, 8, 8), (136, 96, aqt.ACT_GLU, 4, 4),
                                                    (260, 4096, aqt.ACT_NONE, 4, 8)])
def test_qmatmul_small_batch(M, N, K, act, bits_a, bits_w):
    """A few rows (streaming use): the weight-bandwidth-bound kernel, packed operands read directly."""
    _run_qmatmul(M, N, K, bits_a, bits_w, act, True, True, extremes=(M > 1))
    _run_qmatmul(M, N, K, bits_a, bits_w, act, False, False, s_x_kind=aqt.SCALE_TENSOR)


@pytest.mark.parametrize("M", [1, 5, 16, 17, 33, 48, 64])
@pytest.mark.parametrize("N,K,act,bits_a,bits_w,kind,rounding", [
    (256, 256, aqt.ACT_NONE, 8, 8, aqt.SCALE_TENSOR, orc.ROUND_NEAREST_EVEN),
    (2048, 512, aqt.ACT_NONE, 8, 4, aqt.SCALE_ROW, orc.ROUND_HALF_UP_FLOOR),
    (144, 144, aqt.ACT_NONE, 4, 4, aqt.SCALE_ROW, orc.ROUND_NEAREST_EVEN),
    (512, 1024, aqt.ACT_NONE, 4, 8, aqt.SCALE_TENSOR, orc.ROUND_HALF_UP_FLOOR),
    (1024, 512, aqt.ACT_GLU_SWISH, 8, 4, aqt.SCALE_ROW, orc.ROUND_NEAREST_EVEN),
    (576, 16, aqt.ACT_SWISH, 8, 8, aqt.SCALE_ROW, orc.ROUND_NEAREST_EVEN)])
def test_linear_fwd_few_rows(M, N, K, act, bits_a, bits_w, kind, rounding):
    """One to 64 rows of fp32 activations (a streaming step) through the whole layer, across the
    threshold between the small-batch and the tensor-core matmul.  Outputs bit-exact without a
    transcendental, within the float bar with one; a zero row and a row of tiny values ride along."""
    x = gen.normal(60 + M, 1, M, K)
    if M > 2:
        x[1, :] = 0.0
        x[2, :] *= 1e-30
    wt = gen.weight(60 + M, 2, K, N)
    bias = gen.normal(60 + M, 3, 1, N, std=0.01)[0]
    n_out = N // 2 if act in (aqt.ACT_GLU, aqt.ACT_GLU_SWISH) else N
    res = gen.normal(60 + M, 4, M, n_out)
    wq, s_w = orc.quantize(wt, bits_w, orc.AXIS_ROW, rounding)
    y_ref, xq, sx, acc = orc.linear_fwd(x, wq, s_w, bias=bias, residual=res, residual_scale=0.5, bits_a=bits_a, a_scale_kind=kind,
                                        rounding=rounding, act=act, return_parts=True)
    wq_d = _dev(orc.pack_int4(wq)) if bits_w == 4 else _dev(wq)
    y = aqt.aqt_linear_fwd(_dev(x), wq_d, _dev(s_w), _dev(bias), _dev(res), 0.5, bits_a=bits_a, bits_w=bits_w, a_scale_kind=kind,
                           rounding=rounding, act=act)
    _status_ok()
    y = y.cpu().numpy()
    if act == aqt.ACT_NONE:
        assert np.array_equal(y.view(np.uint32), y_ref.view(np.uint32))
    else:
        y64 = orc.epilogue_f64(acc, sx, kind, s_w, bias, res, 0.5, act)
        z = np.abs(orc.epilogue_f64(acc, sx, kind, s_w, None, None, 0.0, aqt.ACT_NONE))
        mag = np.maximum(np.maximum(np.abs(y64), z[:, :n_out]), np.maximum(np.abs(bias[:n_out])[None, :], np.abs(res)))
        assert np.all(np.abs(y - y64) <= 1e-6 * mag + 1e-30)


def test_linear_fwd_small_batch_matches_oracle():
    M, K, N = 5, 512, 2048
    x = gen.normal(6, 1, M, K)
    wt = gen.weight(6, 2, K, N)
    wq, s_w = orc.quantize(wt, 4, orc.AXIS_ROW)
    y_ref = orc.linear_fwd(x, wq, s_w)
    y = aqt.aqt_linear_fwd(_dev(x), _dev(orc.pack_int4(wq)), _dev(s_w), bits_a=8, bits_w=4)
    _status_ok()
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


PAIR_PLANS = ["pair256s4e8", "pair256s6e4", "pair128s6e8", "pair128s8e4"]


@pytest.mark.parametrize("plan", PAIR_PLANS + ["pair512s3e16"])
def test_qmatmul_cta_pair_plans_named(plan):
    """Every two-CTA (cta_group::2) configuration of the streaming kernel, named explicitly, on
    shapes that would otherwise take one CTA per tile: ragged M (the second CTA's rows partly or
    wholly outside), ragged N, residual, several tiles per pair, 4-bit operands in both layouts."""
    _run_qmatmul(130, 200, 2048, 8, 8, aqt.ACT_NONE, True, True, extremes=True, plan=plan)
    _run_qmatmul(700, 384, 640, 8, 8, aqt.ACT_SWISH, True, False, plan=plan)
    _run_qmatmul(256 * 80 + 37, 256, 2048, 8, 8, aqt.ACT_NONE, False, True, plan=plan)
    _run_qmatmul(512, 1024, 4096, 4, 4, aqt.ACT_NONE, False, False, s_x_kind=aqt.SCALE_TENSOR, plan=plan)
    _run_qmatmul(1000, 1536, 1024, 8, 4, aqt.ACT_NONE, True, True, plan=plan, unpacked4=True)


@pytest.mark.parametrize("plan", ["pair256s4e8", "pair256s6e4", "pair128s6e8", "pair128s8e4"])
def test_qmatmul_cta_pair_plans_glu(plan):
    """GLU halves split across the pair (value rows in the leader, gate rows in its peer)."""
    _run_qmatmul(256, 512, 1024, 8, 4, aqt.ACT_GLU_SWISH, True, True, plan=plan)
    _run_qmatmul(900, 1024, 512, 8, 8, aqt.ACT_GLU, False, True, plan=plan)


@pytest.mark.parametrize("plan", ["stream256s3e16", "stream256s4e4", "stream128s4e16", "stream128s6e4", "stream64s5e8", "stream64s8e4",
                                  "ws128e16"])
def test_qmatmul_single_cta_plans_named(plan):
    """The one-CTA-per-tile configurations by name, on one shallow shape all of them can take."""
    _run_qmatmul(777, 640, 512, 8, 4, aqt.ACT_SWISH, True, True, plan=plan)
    _run_qmatmul(300, 256, 384, 8, 8, aqt.ACT_NONE, True, False, plan=plan, extremes=True)


def test_qmatmul_wide_pair_tiles_ffn_second_layer_shape():
    """The benchmark's second matmul (12 800 x 2048 -> 512, 4-bit weights kept unpacked by the
    caller): the plan the library picks is the 256 x 512 pair tile; full size, sampled rows."""
    M, N, K = 12800, 512, 2048
    assert aqt.aqt_plan_qmatmul(M, N, K, 8, aqt.BITS_4_UNPACKED) == "pair512s3e16"
    xq = gen.random_codes(11, M, K, 8)
    wq = gen.random_codes(12, N, K, 4)
    rng = np.random.default_rng(13)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    acc_d = torch.empty((M, N), dtype=torch.int32, device=DEV)
    args = (_dev(xq), _dev(s_x), _dev(wq), _dev(s_w), None, _dev(res), 0.5)
    y = aqt.aqt_qmatmul(*args, K=K, bits_a=8, bits_w=aqt.BITS_4_UNPACKED)
    y2 = aqt.aqt_qmatmul(*args, K=K, bits_a=8, bits_w=aqt.BITS_4_UNPACKED, acc_debug=acc_d)
    y3 = aqt.aqt_qmatmul(_dev(xq), _dev(s_x), _dev(orc.pack_int4(wq)), _dev(s_w), None, _dev(res), 0.5, K=K, bits_a=8, bits_w=4)
    _status_ok()
    rows = sorted(set([0, 127, 128, 255, 256, 511, 512, M - 257, M - 129, M - 1]) | set(rng.integers(0, M, 40).tolist()))
    acc_ref = orc.int_matmul(xq[rows], wq)
    assert np.array_equal(acc_d.cpu().numpy()[rows].astype(np.int64), acc_ref)
    y_ref = orc.epilogue_f32(acc_ref, s_x[rows], orc.SCALE_ROW, s_w, None, res[rows], 0.5, orc.ACT_NONE)
    assert np.array_equal(y.cpu().numpy()[rows].view(np.uint32), y_ref.view(np.uint32))
    assert torch.equal(y.view(torch.int32), y2.view(torch.int32)) and torch.equal(y.view(torch.int32), y3.view(torch.int32))


def test_qmatmul_cta_pairs_large_deep_k_sampled_rows():
    """A shape that takes CTA pairs by itself (deep K, many tiles per pair): 19 200 x 1024 x 2048.
    Accumulators and outputs are compared with the oracle on sampled rows."""
    M, N, K = 19200, 1024, 2048
    assert aqt.aqt_plan_qmatmul(M, N, K, 8, 4) == "pair128s6e8"
    rng = np.random.default_rng(7)
    xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
    wq = rng.integers(-7, 8, (N, K)).astype(np.int8)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    acc_d = torch.empty((M, N), dtype=torch.int32, device=DEV)
    y = aqt.aqt_qmatmul(_dev(xq), _dev(s_x), _dev(orc.pack_int4(wq)), _dev(s_w), None, _dev(res), 0.5, K=K, bits_a=8, bits_w=4,
                        acc_debug=acc_d)
    y2 = aqt.aqt_qmatmul(_dev(xq), _dev(s_x), _dev(orc.pack_int4(wq)), _dev(s_w), None, _dev(res), 0.5, K=K, bits_a=8, bits_w=4)
    _status_ok()
    rows = sorted(set([0, 127, 128, 255, 256, M - 257, M - 129, M - 1]) | set(rng.integers(0, M, 40).tolist()))
    acc_ref = orc.int_matmul(xq[rows], wq)
    assert np.array_equal(acc_d.cpu().numpy()[rows].astype(np.int64), acc_ref)
    y_ref = orc.epilogue_f32(acc_ref, s_x[rows], orc.SCALE_ROW, s_w, None, res[rows], 0.5, orc.ACT_NONE)
    assert np.array_equal(y.cpu().numpy()[rows].view(np.uint32), y_ref.view(np.uint32))
    assert torch.equal(y.view(torch.int32), y2.view(torch.int32))


# ----------------------------------------------------------------------------- whole layer

@pytest.mark.parametrize("bits_a,bits_w,kind", [(8, 8, aqt.SCALE_TENSOR), (8, 4, aqt.SCALE_ROW), (4, 4, aqt.SCALE_ROW)])
@pytest.mark.parametrize("rounding", [orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN])
def test_linear_fwd_matches_oracle(bits_a, bits_w, kind, rounding):
    M, K, N = 200, 512, 384
    x = gen.normal(4, 1, M, K)
    wt = gen.weight(4, 2, K, N)
    bias = gen.normal(4, 3, 1, N, std=0.01)[0]
    wq, s_w = orc.quantize(wt, bits_w, orc.AXIS_ROW, rounding)
    y_ref = orc.linear_fwd(x, wq, s_w, bias=bias, bits_a=bits_a, a_scale_kind=kind, rounding=rounding)
    # weights prepared on the GPU as well: quantize over K per output channel, pack if 4-bit
    wq_d, sw_d = aqt.aqt_quantize(_dev(wt), bits_w, aqt.AXIS_ROW, rounding, pack=(bits_w == 4))
    assert np.array_equal(sw_d.cpu().numpy(), s_w)
    y = aqt.aqt_linear_fwd(_dev(x), wq_d, sw_d, _dev(bias), bits_a=bits_a, bits_w=bits_w, a_scale_kind=kind,
                           rounding=rounding)
    _status_ok()
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


@pytest.mark.parametrize("seed", range(12))
def test_linear_fwd_random_shapes(seed):
    """The whole layer (fp32 in, fp32 out, act = NONE so every output bit is fixed) on seeded
    random shapes, scale kinds, bit widths and rounding rules, weights prepared on the GPU."""
    rng = np.random.default_rng(1300 + seed)
    K = 16 * int(rng.integers(1, 129))
    N = 16 * int(rng.integers(1, 97))
    M = int(rng.integers(1, 1500))
    while M * N * K > 2e8:
        M = max(1, M // 2)
    bits_a, bits_w = [(8, 8), (8, 4), (4, 4), (4, 8)][int(rng.integers(0, 4))]
    kind = [aqt.SCALE_ROW, aqt.SCALE_TENSOR][int(rng.integers(0, 2))]
    rounding = [orc.ROUND_HALF_UP_FLOOR, orc.ROUND_NEAREST_EVEN][int(rng.integers(0, 2))]
    x = gen.normal(40 + seed, 1, M, K)
    wt = gen.weight(40 + seed, 2, K, N)
    bias = gen.normal(40 + seed, 3, 1, N, std=0.01)[0] if rng.integers(0, 2) else None
    res = gen.normal(40 + seed, 4, M, N) if rng.integers(0, 2) else None
    wq, s_w = orc.quantize(wt, bits_w, orc.AXIS_ROW, rounding)
    y_ref = orc.linear_fwd(x, wq, s_w, bias=bias, residual=res, residual_scale=0.5, bits_a=bits_a, a_scale_kind=kind, rounding=rounding)
    wq_d, sw_d = aqt.aqt_quantize(_dev(wt), bits_w, aqt.AXIS_ROW, rounding, pack=(bits_w == 4))
    assert np.array_equal(sw_d.cpu().numpy(), s_w)
    y = aqt.aqt_linear_fwd(_dev(x), wq_d, sw_d, None if bias is None else _dev(bias), None if res is None else _dev(res), 0.5,
                           bits_a=bits_a, bits_w=bits_w, a_scale_kind=kind, rounding=rounding)
    _status_ok()
    assert np.array_equal(y.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))


def test_linear_fwd_host_buffers():
    M, K, N = 256, 256, 256
    x = gen.normal(5, 1, M, K)
    wt = gen.weight(5, 2, K, N)
    wq, s_w = orc.quantize(wt, 8, orc.AXIS_ROW)
    y_ref = orc.linear_fwd(x, wq, s_w, act=orc.ACT_SWISH)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty((M, N), dtype=torch.float32).pin_memory()
    ws = torch.empty(aqt.linear_fwd_host_workspace_bytes(M, N, K, 8, 8, aqt.ACT_SWISH), dtype=torch.uint8, device=DEV)
    aqt.aqt_linear_fwd_host(xh, _dev(wq), _dev(s_w), None, yh, ws, act=aqt.ACT_SWISH)
    _status_ok()
    y = yh.numpy()
    assert np.all(np.abs(y - y_ref) <= 1e-6 * np.maximum(np.abs(y_ref), 1e-3) + 1e-30)


def test_bounded_wait_gives_up_and_reports_timeout():
    """A wait on a barrier nothing signals runs out after its limit: the kernel returns, the
    status word says AQT_ERR_TIMEOUT once, and the context keeps working."""
    assert aqt.aqt_device_status() == 0
    assert aqt.aqt_selftest_bounded_wait(2_000_000) is True
    assert aqt.aqt_device_status() == -6
    assert aqt.aqt_device_status() == 0                      # cleared by the read
    x = torch.ones((4, 32), dtype=torch.float32, device=DEV)
    q, s = aqt.aqt_quantize(x, 8, aqt.AXIS_ROW)              # the context is still usable
    assert int(q.min()) == 127 and aqt.aqt_device_status() == 0


def test_status_codes_on_device():
    x = torch.zeros((128, 128), dtype=torch.int8, device=DEV)
    s = torch.ones(128, dtype=torch.float32, device=DEV)
    with pytest.raises(aqt.AqtError) as e:
        aqt.aqt_qmatmul(x, s, torch.zeros((128, 64), dtype=torch.uint8, device=DEV), s, K=128, bits_w=4,
                        workspace=torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.status == -4
