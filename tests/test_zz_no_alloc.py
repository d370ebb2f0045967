"""The allocation-free matmul entry point gives the same result as aqt_qmatmul.

Collected last on purpose (file name): if it fails under `pytest -x`, every other test has
already run.  It must pass alone in a fresh process and after the other tests.

aqt_qmatmul_w4_noalloc exists for callers that cannot get device scratch memory (no cudaMalloc
inside a capture, a host application that owns all allocations, a fixed memory budget): the
sign-extended weights go into an array built into the library instead of a caller workspace.
All calls share that array and it keeps the previous call's bytes, so the test makes two calls in
a row with different weights and a smaller second shape, and checks both against aqt_qmatmul.
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


@pytest.mark.parametrize("first,second", [((300, 512, 512, aqt.ACT_NONE, True), (129, 136, 96, aqt.ACT_SWISH, False)),
                                          ((256, 1024, 2048, aqt.ACT_GLU_SWISH, True), (256, 1024, 2048, aqt.ACT_NONE, False))])
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(first, second):
    for seed, (M, N, K, act, with_res) in enumerate((first, second)):
        xq, s_x, wq, s_w, bias, res, n_out = _case(seed, M, N, K, act, with_res)
        y_ref = aqt.aqt_qmatmul(xq, s_x, wq, s_w, bias, res, 0.5, K=K, bits_a=8, bits_w=4, act=act)
        y = torch.full((M, n_out), float("nan"), dtype=torch.float32, device=DEV)
        aqt.aqt_qmatmul_w4_noalloc(xq, s_x, wq, s_w, bias, res, 0.5, K=K, act=act, y=y)
        assert aqt.aqt_device_status() == 0
        # same kernels on the same codes: identical bits (stricter than the 1e-6 used against the oracle)
        assert torch.equal(y.view(torch.int32), y_ref.view(torch.int32))


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
    # the largest accepted size still works
    N2 = aqt.NOALLOC_MAX_WEIGHT_BYTES // K
    y2 = torch.zeros((128, N2), dtype=torch.float32, device=DEV)
    aqt.aqt_qmatmul_w4_noalloc(xq, s[:128], wq[:N2], s[:N2], K=K, y=y2)
    assert aqt.aqt_device_status() == 0 and float(y2.abs().max()) == 0.0
