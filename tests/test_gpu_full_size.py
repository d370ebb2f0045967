"""Parity at the full size of the large encoder configuration (M = 128 x 512 = 65 536 rows, d = 1024,
ff = 4096), in the kernel configurations that those sizes select (needs a B200).

The oracle cannot run 65 536 rows in seconds, and does not have to: every row of a layer with
per-row activation scales is independent of every other row, so the oracle is run on sampled rows
(tile edges, the last rows, random rows) and compared with the same rows of the full-size GPU
result -- accumulators, codes and scales bit for bit, float outputs bit for bit where the layer
has no transcendental and within 1e-6 of the larger of result and terms otherwise.  Properties
that hold at any size (every row's largest |code| is the largest code; the accumulator-dumping and
the production instantiation agree on every element) cover the rest of the tensor.
"""
import numpy as np
import pytest
import torch

import oracle as orc
from oracle import conformer_ref as ref
from paper_2203_15952_b200 import binding as aqt
from paper_2203_15952_b200 import inputs as gen
from paper_2203_15952_b200.encoder import ConformerBlockLinears, QuantLinear

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
M_FULL = gen.WORKLOADS[5].M


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _rows(M, rng, n_random=40, tail=257):
    fixed = [0, 127, 128, 255, 256, 511, 512] + list(range(M - tail, M))
    return sorted(set(fixed) | set(rng.integers(0, M, n_random).tolist()))


def _float_close(y, y64, mag):
    err = np.abs(y - y64)
    assert np.all(err <= 1e-6 * mag + 1e-30), float(np.max(err / (mag + 1e-30)))


@pytest.mark.parametrize("N,plan", [(1024, "pair256s6e4"), (384, "pair128s8e4")])
def test_large_encoder_ffn_second_layer_matmul(N, plan):
    """65 536 x 4096 -> N, int8 activations, int4 weights, fp32 residual: the deep-K CTA-pair
    configurations with the four-warp epilogue.  First the production instantiation, then the
    accumulator-dumping one."""
    M, K = M_FULL, 4096
    assert aqt.aqt_plan_qmatmul(M, N, K, 8, 4) == plan
    rng = np.random.default_rng(N)
    xq = gen.random_codes(21, M, K, 8)
    wq = gen.random_codes(22, N, K, 4)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    res = rng.standard_normal((M, N), dtype=np.float32)
    xq_d, wq_d, res_d = _dev(xq), _dev(orc.pack_int4(wq)), _dev(res)
    y = aqt.aqt_qmatmul(xq_d, _dev(s_x), wq_d, _dev(s_w), None, res_d, 0.5, K=K, bits_a=8, bits_w=4)
    acc_d = torch.empty((M, N), dtype=torch.int32, device=DEV)
    y2 = aqt.aqt_qmatmul(xq_d, _dev(s_x), wq_d, _dev(s_w), None, res_d, 0.5, K=K, bits_a=8, bits_w=4, acc_debug=acc_d)
    assert aqt.aqt_device_status() == 0
    rows = _rows(M, rng)
    acc_ref = orc.int_matmul(xq[rows], wq)
    assert np.array_equal(acc_d[rows].cpu().numpy().astype(np.int64), acc_ref)
    y_ref = orc.epilogue_f32(acc_ref, s_x[rows], orc.SCALE_ROW, s_w, None, res[rows], 0.5, orc.ACT_NONE)
    assert np.array_equal(y[rows].cpu().numpy().view(np.uint32), y_ref.view(np.uint32))
    assert torch.equal(y.view(torch.int32), y2.view(torch.int32))


@pytest.mark.parametrize("N,act", [(4096, aqt.ACT_SWISH), (2048, aqt.ACT_GLU_SWISH)])
def test_large_encoder_first_layers_quantize_their_rows(N, act):
    """65 536 x 1024 -> 4096 Swish and -> 2048 GLU + Swish with the output rows quantized in the
    epilogue (codes and scales only).  The fp32 tensor the codes stand for is the one aqt_qmatmul
    writes; it is checked against the oracle on sampled rows, and the fused codes and scales must
    be the oracle's quantizer applied to those rows, and the GPU quantizer's output everywhere."""
    M, K = M_FULL, 1024
    n_out = N // 2 if act == aqt.ACT_GLU_SWISH else N
    rng = np.random.default_rng(N + 1)
    xq = gen.random_codes(31, M, K, 8)
    wq = gen.random_codes(32, N, K, 4)
    s_x = rng.uniform(1e-3, 5e-2, M).astype(np.float32)
    s_w = rng.uniform(1e-4, 5e-3, N).astype(np.float32)
    xq_d, wq_d, sx_d, sw_d = _dev(xq), _dev(orc.pack_int4(wq)), _dev(s_x), _dev(s_w)
    q, s, _ = aqt.aqt_qmatmul_requant(xq_d, sx_d, wq_d, sw_d, K=K, bits_a=8, bits_w=4, act=act, bits_out=8)
    u = aqt.aqt_qmatmul(xq_d, sx_d, wq_d, sw_d, K=K, bits_a=8, bits_w=4, act=act)
    q2, s2 = aqt.aqt_quantize(u, 8, aqt.AXIS_ROW)
    assert aqt.aqt_device_status() == 0
    assert q.shape == (M, n_out)
    assert torch.equal(q, q2) and torch.equal(s.view(torch.int32), s2.view(torch.int32))
    rows = _rows(M, rng, n_random=24, tail=130)
    acc_ref = orc.int_matmul(xq[rows], wq)
    u_rows = u[rows].cpu().numpy()
    u64 = orc.epilogue_f64(acc_ref, s_x[rows], orc.SCALE_ROW, s_w, None, None, 0.0, act)
    z = np.abs(orc.epilogue_f64(acc_ref, s_x[rows], orc.SCALE_ROW, s_w, None, None, 0.0, orc.ACT_NONE))
    _float_close(u_rows, u64, np.maximum(np.abs(u64), z[:, :n_out]))
    q_ref, s_ref = orc.quantize(u_rows, 8, orc.AXIS_ROW)
    assert np.array_equal(q[rows].cpu().numpy(), q_ref) and np.array_equal(s[rows].cpu().numpy(), s_ref)
    # any size: the row's largest magnitude takes the largest code
    assert int(q.abs().max(dim=1).values.min()) == 127


def _layers(w, block, specs):
    gpu, cpu = [], []
    for i, sp in enumerate(specs):
        wt = gen.layer_weight(w, block, i, sp)
        ql = QuantLinear.from_float(sp, _dev(wt))
        wq, sw = ref.prepare_weight(wt, sp.bits_w)
        assert np.array_equal(ql.wq.cpu().numpy().view(np.uint8), orc.pack_int4(wq)) and np.array_equal(ql.s_w.cpu().numpy(), sw)
        gpu.append(ql)
        cpu.append((wq, sw, None))
    return gpu, cpu


def _check_layer(spec, cpu_w, x_rows, y_rows, residual_rows=None, rs=1.0):
    wq, sw, bias = cpu_w
    y_ref, xq, sx, acc = orc.linear_fwd(x_rows, wq, sw, bias=bias, residual=residual_rows, residual_scale=rs,
                                        bits_a=spec.bits_a, act=spec.act, return_parts=True)
    if spec.act == gen.ACT_NONE:
        assert np.array_equal(y_rows.view(np.uint32), y_ref.view(np.uint32)), spec.name
        return
    y64 = orc.epilogue_f64(acc, sx, orc.SCALE_ROW, sw, bias, residual_rows, rs, spec.act)
    z = np.abs(orc.epilogue_f64(acc, sx, orc.SCALE_ROW, sw, None, None, 0.0, orc.ACT_NONE))
    mag = np.maximum(np.abs(y64), z[:, :y64.shape[1]])
    if residual_rows is not None:
        mag = np.maximum(mag, np.abs(residual_rows))
    _float_close(y_rows, y64, mag)


def test_large_encoder_block_full_batch_layerwise():
    """One block of the d = 1024 encoder on the whole 65 536-row batch of heavy-tailed (Student-t,
    3 degrees of freedom) inputs: every one of the ten linears is compared with the oracle on
    sampled rows, the oracle being fed the GPU's own fp32 input rows of that layer.  The block is
    then run as the benchmark runs it (intermediates handed on as codes) and must give the same bits."""
    w = gen.WORKLOADS[5]
    specs = gen.workload_layers(w)
    M = w.M
    gpu, cpu = _layers(w, 0, specs)
    x = gen.workload_input(w)
    rng = np.random.default_rng(5)
    rows = sorted(set([0, 127, 128, 255, 256, M // 2, M - 257, M - 129, M - 128, M - 1]) | set(rng.integers(0, M, 10).tolist()))
    blk = ConformerBlockLinears(M, w.d, w.ff, gpu, DEV)
    xd = _dev(x)
    h_out = torch.empty((M, w.d), dtype=torch.float32, device=DEV)
    keep = {}
    blk.forward(gpu, xd, h_out, keep=keep)
    assert aqt.aqt_device_status() == 0
    g = {k: v[rows].cpu().numpy() for k, v in keep.items()}
    del keep
    n = [sp.name for sp in specs]
    h_in = x[rows]
    _check_layer(specs[0], cpu[0], h_in, g[n[0]])
    _check_layer(specs[1], cpu[1], g[n[0]], g[n[1]], residual_rows=h_in, rs=0.5)
    for i in (2, 3, 4):
        _check_layer(specs[i], cpu[i], g[n[1]], g[n[i]])
    _check_layer(specs[5], cpu[5], g[n[4]], g[n[5]], residual_rows=g[n[1]], rs=1.0)
    _check_layer(specs[6], cpu[6], g[n[5]], g[n[6]])
    _check_layer(specs[7], cpu[7], g[n[6]], g[n[7]], residual_rows=g[n[5]], rs=1.0)
    _check_layer(specs[8], cpu[8], g[n[7]], g[n[8]])
    _check_layer(specs[9], cpu[9], g[n[8]], g[n[9]], residual_rows=g[n[7]], rs=0.5)
    h_fused = torch.empty_like(h_out)
    blk.forward(gpu, xd, h_fused)
    assert aqt.aqt_device_status() == 0
    assert torch.equal(h_fused.view(torch.int32), h_out.view(torch.int32))
    # the kernel configurations this batch size selects for the block's matmuls
    assert aqt.aqt_plan_qmatmul(M, w.d, w.ff, 8, aqt.BITS_4_UNPACKED) == "pair256s6e4"      # second FFN layers
    assert aqt.aqt_plan_qmatmul(M, 3 * w.d, w.d, 8, aqt.BITS_4_UNPACKED) == "stream256s3e16"  # q, k, v in one matmul
