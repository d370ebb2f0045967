"""The oracle's chain driver (FFN pair, block, stack) is the composition of single layers."""
import numpy as np

import oracle as orc
from oracle import conformer_ref as ref
from paper_2203_15952_b200 import inputs as gen


def _weights(w, block, specs):
    out = []
    for i, s in enumerate(specs):
        wq, sw = ref.prepare_weight(gen.layer_weight(w, block, i, s), s.bits_w)
        out.append((wq, sw, gen.layer_bias(w, block, i, s)))
    return out


def test_ffn_pair_is_two_layers():
    w = gen.WORKLOADS[2]
    specs = gen.workload_layers(w)
    wts = _weights(w, 0, specs)
    x = gen.workload_input(w, row_subset=list(range(0, 12800, 1600)))
    out = ref.ffn_pair(specs, wts, x)
    u = orc.linear_fwd(x, wts[0][0], wts[0][1], act=orc.ACT_SWISH)
    y = orc.linear_fwd(u, wts[1][0], wts[1][1])
    assert np.array_equal(out["u"], u) and np.array_equal(out["y"], y)
    assert out["y"].shape == (8, 512) and np.isfinite(out["y"]).all()
    # int4 weights: codes inside [-7, 7] and at least one +-7 per output channel
    assert np.abs(wts[0][0]).max() == 7 and np.all(np.abs(wts[0][0]).max(axis=1) == 7)


def test_block_dataflow_and_row_independence():
    """With per-row activation scales every row is independent: running a subset of rows gives
    the same bits as those rows of a larger run."""
    w = gen.WORKLOADS[3]
    specs = gen.workload_layers(w)
    wts = _weights(w, 0, specs)
    rows = [3, 77, 4000, 12799]
    x = gen.workload_input(w, row_subset=rows)
    full = ref.block(specs, wts, x)
    half = ref.block(specs, wts, x[1:3])
    assert np.array_equal(full["h"][1:3], half["h"])
    # residual structure: h after ffn_a2 = x + 0.5 * (ffn_a2 output without residual)
    u = orc.linear_fwd(x, wts[0][0], wts[0][1], bits_a=4, act=orc.ACT_SWISH)
    y_nores = orc.linear_fwd(u, wts[1][0], wts[1][1], bits_a=4)
    assert np.allclose(full["ffn_a2"], x + 0.5 * y_nores, rtol=0, atol=1e-6)
    assert full["conv_pw1"].shape == (4, 512) and full["attn_q"].shape == (4, 512)
    assert np.isfinite(full["h"]).all()


def test_stack_runs_blocks_in_sequence():
    w = gen.WORKLOADS[4]
    specs = gen.workload_layers(w)
    x = gen.workload_input(w, row_subset=[0, 1])
    cache = {}

    def wob(b):
        if b not in cache:
            cache[b] = _weights(w, b, specs)
        return cache[b]

    outs = ref.stack(specs, wob, x, 2, keep=[0, 1])
    h0 = ref.block(specs, wob(0), x)["h"]
    h1 = ref.block(specs, wob(1), h0)["h"]
    assert np.array_equal(outs[0], h0) and np.array_equal(outs[1], h1)
