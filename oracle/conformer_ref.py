"""Oracle-side driver for chains of quantized linears (FFN pair, Conformer block, encoder stack).

TEST INFRASTRUCTURE ONLY.  Calls nothing but the oracle's C functions; imports nothing from the
product package.  The layer tables it walks are passed in by the caller.

Only the weight-bearing linears of a Conformer block are on the quantized path (Section 3.3:
encoders are quantized, decoders and convolution kernels are not).  The parts of a block that are
not linears (attention scores, depthwise convolution, normalisation) are replaced by the identity
in this stand-in dataflow, which the CUDA driver follows step for step:

    h <- h + 1/2 * W_a2 . Swish(W_a1 . h)          feed-forward module a
    q, k, v <- W_q . h, W_k . h, W_v . h            attention projections (q, k only produced)
    h <- h + W_o . v
    c <- Swish(GLU(W_pw1 . h))                      convolution module, pointwise 1
    h <- h + W_pw2 . c                              pointwise 2
    h <- h + 1/2 * W_b2 . Swish(W_b1 . h)          feed-forward module b

Residual adds are fp32 and belong to the epilogue of the producing linear.
"""
from __future__ import annotations

from typing import Callable, Dict, List, Optional, Tuple

import numpy as np

from . import (AXIS_ROW, ROUND_NEAREST_EVEN, SCALE_ROW, SCALE_TENSOR, linear_fwd, quantize)


def prepare_weight(wt: np.ndarray, bits: int, rounding: int = ROUND_NEAREST_EVEN) -> Tuple[np.ndarray, np.ndarray]:
    """Per-output-channel weight quantization: wt is W^T [N, K]; reduce over K (Section 2.2,
    channel-wise).  Returns (codes int8 [N, K], scales fp32 [N])."""
    return quantize(np.ascontiguousarray(wt, dtype=np.float32), bits, AXIS_ROW, rounding)


def run_layer(spec, wq, s_w, bias, x, residual=None, residual_scale=1.0, a_scale="row",
              rounding=ROUND_NEAREST_EVEN, return_parts=False):
    kind = SCALE_ROW if a_scale == "row" else SCALE_TENSOR
    return linear_fwd(x, wq, s_w, bias=bias, residual=residual, residual_scale=residual_scale,
                      bits_a=spec.bits_a, a_scale_kind=kind, rounding=rounding, act=spec.act,
                      return_parts=return_parts)


def ffn_pair(specs, weights, x, a_scale="row", rounding=ROUND_NEAREST_EVEN) -> Dict[str, np.ndarray]:
    """y = W_2 . Swish(W_1 . x): two linears, the second re-quantizes the first's output."""
    (wq1, sw1, b1), (wq2, sw2, b2) = weights
    u = run_layer(specs[0], wq1, sw1, b1, x, a_scale=a_scale, rounding=rounding)
    y = run_layer(specs[1], wq2, sw2, b2, u, a_scale=a_scale, rounding=rounding)
    return {"u": u, "y": y}


def block(specs, weights, h, a_scale="row", rounding=ROUND_NEAREST_EVEN) -> Dict[str, np.ndarray]:
    """One block of the stand-in dataflow.  specs/weights: the ten linears in execution order.
    Returns every intermediate, keyed by the layer that produced it, and the block output 'h'."""
    out: Dict[str, np.ndarray] = {}

    def L(i, x, residual=None, rs=1.0):
        wq, sw, b = weights[i]
        y = run_layer(specs[i], wq, sw, b, x, residual=residual, residual_scale=rs, a_scale=a_scale, rounding=rounding)
        out[specs[i].name] = y
        return y

    u = L(0, h)
    h = L(1, u, residual=h, rs=0.5)
    L(2, h)
    L(3, h)
    v = L(4, h)
    h = L(5, v, residual=h, rs=1.0)
    c = L(6, h)
    h = L(7, c, residual=h, rs=1.0)
    u = L(8, h)
    h = L(9, u, residual=h, rs=0.5)
    out["h"] = h
    return out


def stack(specs, weights_of_block: Callable[[int], list], h, n_blocks: int, a_scale="row",
          rounding=ROUND_NEAREST_EVEN, keep: Optional[List[int]] = None) -> Dict[int, np.ndarray]:
    """n_blocks blocks in sequence; returns {block index: h after that block} for blocks in keep
    (default: the last one)."""
    keep = [n_blocks - 1] if keep is None else keep
    outs = {}
    for b in range(n_blocks):
        h = block(specs, weights_of_block(b), h, a_scale=a_scale, rounding=rounding)["h"]
        if b in keep:
            outs[b] = h
    return outs
