"""The allocation-free matmul entry point gives the same result as aqt_qmatmul.

Collected last on purpose (file name): if it fails under `pytest -x`, every other test has
already run.  It must pass alone in a fresh process and after the other tests.

aqt_qmatmul_w4_noalloc exists for callers that cannot get device scratch memory (no cudaMalloc
inside a capture, a host application that owns all allocations, a fixed memory budget): the
sign-extended weights go into an array built into the library instead of a caller workspace.
All calls share that array and it keeps the previous call's bytes, so the test makes two calls in
a row with different weights and a smaller second shape, and checks both against aqt_qmatmul
and against the CPU oracle.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2203_15952_b200 import binding as aqt

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, M, N, K, act, with_res):
    g = torch.Generator(device="cpu").manual_seed(seed)
    xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8).to(DEV)
    wq = torch.randint(0, 256, (N, K // 2), generator=g, dtype=torch.uint8).to(DEV)   # any nibble pair
    s_x = (torch.rand(M, generator=g) * 1e-2 + 1e-3).to(DEV)
    s_w = (torch.rand(N, generator=g) * 1e-3 + 1e-4).to(DEV)
    bias = (torch.randn(N, generator=g) * 0.1).to(DEV)
    n_out = N // 2 if act in (aqt.ACT_GLU, aqt.ACT_GLU_SWISH) else N
    res = torch.randn((M, n_out), generator=g).to(DEV) if with_res else None
    return xq, s_x, wq, s_w, bias, res, n_out


def _oracle_rows(xq, s_x, wq, s_w, bias, res, act, rows):
    """The oracle's result for the given rows (codes unpacked by the oracle's own routine)."""
    import oracle as orc
    wq_i8 = orc.unpack_int4(wq.cpu().numpy(), 2 * wq.shape[1])
    acc = orc.int_matmul(xq.cpu().numpy()[rows], wq_i8)
    r = None if res is None else res.cpu().numpy()[rows]
    args = (acc, s_x.cpu().numpy()[rows], orc.SCALE_ROW, s_w.cpu().numpy(), bias.cpu().numpy(), r, 0.5, act)
    return orc.epilogue_f32(*args), orc.epilogue_f64(*args), np.abs(orc.epilogue_f64(acc, args[1], orc.SCALE_ROW, args[3], None, None, 0.0, 0))


# Every shape has K > 512, so the weights always go through the built-in scratch array (smaller K
# is sign-extended in shared memory and would not touch it).  The second call of a pair is
# smaller than the first and uses other weights: it runs over the first call's stale bytes.
@pytest.mark.parametrize("first,second", [((300, 512, 2048, aqt.ACT_NONE, True), (129, 136, 1024, aqt.ACT_SWISH, False)),
                                          ((256, 1024, 2048, aqt.ACT_GLU_SWISH, True), (200, 256, 640, aqt.ACT_NONE, False))])
def test_noalloc_matches_workspace_entry_point_and_oracle_twice_in_a_row(first, second):
    for seed, (M, N, K, act, with_res) in enumerate((first, second)):
        xq, s_x, wq, s_w, bias, res, n_out = _case(seed, M, N, K, act, with_res)
        y_ref = aqt.aqt_qmatmul(xq, s_x, wq, s_w, bias, res, 0.5, K=K, bits_a=8, bits_w=4, act=act)
        y = torch.full((M, n_out), float("nan"), dtype=torch.float32, device=DEV)
        aqt.aqt_qmatmul_w4_noalloc(xq, s_x, wq, s_w, bias, res, 0.5, K=K, act=act, y=y)
        assert aqt.aqt_device_status() == 0
        # same kernels on the same codes: identical bits (stricter than the 1e-6 used against the oracle)
        assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32))
        # and against the CPU oracle on rows across the tile edges
        rows = sorted(set([0, 1, 127, 128, M - 1]) | set(range(0, M, 37)))
        y32, y64, z = _oracle_rows(xq, s_x, wq, s_w, bias, res, act, rows)
        got = y.cpu().numpy()[rows]
        if act == aqt.ACT_NONE:
            assert np.array_equal(got.view(np.uint32), y32.view(np.uint32))
        else:
            mag = np.maximum(np.maximum(np.abs(y64), z[:, :n_out]), np.abs(bias.cpu().numpy()[:n_out])[None, :])
            if res is not None:
                mag = np.maximum(mag, np.abs(res.cpu().numpy()[rows]))
            assert np.all(np.abs(got - y64) <= 1e-6 * mag + 1e-30)


def test_noalloc_rejects_weights_larger_than_the_builtin_scratch():
    N, K = 4096, 2048                                       # 8 MiB of codes > 4 MiB built in
    assert N * K > aqt.NOALLOC_MAX_WEIGHT_BYTES
    xq = torch.zeros((128, K), dtype=torch.int8, device=DEV)
    wq = torch.zeros((N, K // 2), dtype=torch.uint8, device=DEV)
    s = torch.ones(N, dtype=torch.float32, device=DEV)
    y = torch.zeros((128, N), dtype=torch.float32, device=DEV)
    with pytest.raises(aqt.AqtError) as e:
        aqt.aqt_qmatmul_w4_noalloc(xq, s[:128], wq, s, K=K, y=y)
    assert e.value.status == -3


def test_noalloc_largest_accepted_weights_use_the_whole_scratch():
    """N * K equal to the built-in limit, random codes: a tail or overrun error at the end of the
    array would change the last output channels."""
    K = 2048
    N = aqt.NOALLOC_MAX_WEIGHT_BYTES // K
    xq, s_x, wq, s_w, bias, res, n_out = _case(5, 160, N, K, aqt.ACT_NONE, False)
    y_ref = aqt.aqt_qmatmul(xq, s_x, wq, s_w, bias, None, 0.5, K=K, bits_a=8, bits_w=4)
    y = torch.full((160, N), float("nan"), dtype=torch.float32, device=DEV)
    aqt.aqt_qmatmul_w4_noalloc(xq, s_x, wq, s_w, bias, None, 0.5, K=K, y=y)
    assert aqt.aqt_device_status() == 0
    assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32))
    rows = [0, 127, 128, 159]
    y32, _, _ = _oracle_rows(xq, s_x, wq, s_w, bias, None, aqt.ACT_NONE, rows)
    assert np.array_equal(y.cpu().numpy()[rows].view(np.uint32), y32.view(np.uint32))
