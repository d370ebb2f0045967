"""Chains of quantized linears on the GPU: FFN pair, Conformer block, encoder stack.

Every arithmetic step is a call into the C ABI (binding.aqt_*); this module only owns buffers and
the order of calls.  The dataflow is the stand-in block used by the workloads: the parts of a
Conformer block that are not weight-bearing linears (attention scores, depthwise convolution,
normalisation) are not on the quantized path (Section 3.3 quantizes the encoder's linears only)
and are replaced by the identity:

    h <- h + 1/2 * W_a2 . Swish(W_a1 . h)          feed-forward module a
    q, k, v <- W_q . h, W_k . h, W_v . h            attention projections
    h <- h + W_o . v
    c <- Swish(GLU(W_pw1 . h))                      convolution module, pointwise 1
    h <- h + W_pw2 . c                              pointwise 2
    h <- h + 1/2 * W_b2 . Swish(W_b1 . h)          feed-forward module b

Residual adds are fp32 and are fused into the epilogue of the producing linear.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from . import binding as aqt
from .inputs import LinearSpec


@dataclass
class QuantLinear:
    """Pre-quantized weights of one linear: codes W^T [N, K] (nibble-packed when 4-bit), one
    fp32 scale per output channel (Section 2.2, channel-wise), optional fp32 bias."""
    spec: LinearSpec
    wq: torch.Tensor
    s_w: torch.Tensor
    bias: Optional[torch.Tensor]

    @classmethod
    def from_float(cls, spec: LinearSpec, wt: torch.Tensor, bias: Optional[torch.Tensor] = None,
                   rounding: int = aqt.ROUND_NEAREST_EVEN) -> "QuantLinear":
        """wt: fp32 W^T [N, K] on the GPU.  Quantizes over K per output channel with the same
        quantizer the activations use (Fig. 2), packing 4-bit codes two per byte."""
        assert wt.shape == (spec.N, spec.K)
        wq, s_w = aqt.aqt_quantize(wt, spec.bits_w, aqt.AXIS_ROW, rounding, pack=(spec.bits_w == 4))
        return cls(spec, wq, s_w, bias)

    @property
    def weight_bytes(self) -> int:
        return self.wq.numel() + 4 * self.s_w.numel()


class LayerRunner:
    """Owns the scratch workspace shared by all layers of a workload and runs single layers."""

    def __init__(self, M: int, layers: List[QuantLinear], device, a_scale_kind: int = aqt.SCALE_ROW,
                 rounding: int = aqt.ROUND_NEAREST_EVEN):
        self.M, self.device, self.a_scale_kind, self.rounding = M, device, a_scale_kind, rounding
        need = max(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_FWD, M, 3 * l.spec.N, l.spec.K, l.spec.bits_a, l.spec.bits_w) for l in layers)
        self.workspace = torch.empty(need, dtype=torch.uint8, device=device)

    def quantize_input(self, x: torch.Tensor, bits_a: int):
        """Activation codes (int8 containers) and scales of x, for several layers that read the
        same tensor (the attention projections): one quantizer pass instead of one per layer."""
        M, K = x.shape
        if getattr(self, "_shared_q", None) is None or self._shared_q.shape != (M, K):
            self._shared_q = torch.empty((M, K), dtype=torch.int8, device=x.device)
            self._shared_s = torch.empty(M if self.a_scale_kind == aqt.SCALE_ROW else 1, dtype=torch.float32, device=x.device)
        axis = aqt.AXIS_ROW if self.a_scale_kind == aqt.SCALE_ROW else aqt.AXIS_TENSOR
        aqt.aqt_quantize(x, bits_a, axis, self.rounding, q_out=self._shared_q, scale_out=self._shared_s)
        return self._shared_q, self._shared_s

    def matmul(self, layer: QuantLinear, xq: torch.Tensor, s_x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
        """Integer matmul + epilogue of `layer` on already-quantized activations (int8 containers)."""
        s = layer.spec
        return aqt.aqt_qmatmul(xq, s_x, layer.wq, layer.s_w, layer.bias, None, 1.0, K=s.K, bits_a=8, bits_w=s.bits_w, act=s.act,
                               s_x_kind=self.a_scale_kind, y=y, workspace=self.workspace)

    def __call__(self, layer: QuantLinear, x: torch.Tensor, y: torch.Tensor, residual: Optional[torch.Tensor] = None,
                 residual_scale: float = 1.0) -> torch.Tensor:
        s = layer.spec
        return aqt.aqt_linear_fwd(x, layer.wq, layer.s_w, layer.bias, residual, residual_scale, bits_a=s.bits_a,
                                  bits_w=s.bits_w, a_scale_kind=self.a_scale_kind, rounding=self.rounding, act=s.act,
                                  y=y, workspace=self.workspace)


class FfnPair:
    """y = W_2 . Swish(W_1 . x): the second layer re-quantizes the first layer's fp32 output."""

    def __init__(self, M: int, layers: List[QuantLinear], device, **kw):
        assert len(layers) == 2
        self.layers = layers
        self.run = LayerRunner(M, layers, device, **kw)
        self.u = torch.empty((M, layers[0].spec.n_out), dtype=torch.float32, device=device)

    def forward(self, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
        self.run(self.layers[0], x, self.u)
        return self.run(self.layers[1], self.u, y)

    @property
    def ops(self) -> int:
        return sum(2 * self.run.M * l.spec.N * l.spec.K for l in self.layers)


class ConformerBlockLinears:
    """The ten linears of one block in the stand-in dataflow above.  Buffers are allocated once
    and shared by every block of a stack."""

    def __init__(self, M: int, d: int, ff: int, layers_for_sizing: List[QuantLinear], device, **kw):
        self.M, self.d, self.ff = M, d, ff
        self.run = LayerRunner(M, layers_for_sizing, device, **kw)
        f32 = dict(dtype=torch.float32, device=device)
        self.u = torch.empty((M, ff), **f32)
        # q, k, v come out of one GEMM over the concatenated projection weights (N = 3d)
        self.qkv = torch.empty((M, 3 * d), **f32)
        self.q, self.k, self.v = self.qkv[:, 0:d], self.qkv[:, d:2 * d], self.qkv[:, 2 * d:3 * d]
        self._qkv_weights: Dict[int, tuple] = {}
        self.c = torch.empty((M, d), **f32)
        self.h_a = torch.empty((M, d), **f32)
        self.h_b = torch.empty((M, d), **f32)

    def forward(self, layers: List[QuantLinear], h_in: torch.Tensor, h_out: torch.Tensor,
                keep: Optional[Dict[str, torch.Tensor]] = None) -> torch.Tensor:
        """h_in -> h_out (distinct buffers, neither h_a nor h_b).  `keep`, if given, receives
        clones of every intermediate keyed by layer name (for parity checks)."""
        L, run = layers, self.run

        def note(name, t):
            if keep is not None:
                keep[name] = t.clone()

        run(L[0], h_in, self.u); note(L[0].spec.name, self.u)
        run(L[1], self.u, self.h_a, residual=h_in, residual_scale=0.5); note(L[1].spec.name, self.h_a)
        # q, k, v read the same h: quantize it once (the codes do not depend on the consumer) and
        # run the three projections as one matmul over their concatenated output channels
        hq, hs = run.quantize_input(self.h_a, L[2].spec.bits_a)
        wq, s_w, bias = self._fused_qkv(L)
        aqt.aqt_qmatmul(hq, hs, wq, s_w, bias, None, 1.0, K=self.d, bits_a=8, bits_w=L[2].spec.bits_w, act=aqt.ACT_NONE,
                        s_x_kind=run.a_scale_kind, y=self.qkv, workspace=run.workspace)
        note(L[2].spec.name, self.q); note(L[3].spec.name, self.k); note(L[4].spec.name, self.v)
        run(L[5], self.v, self.h_b, residual=self.h_a, residual_scale=1.0); note(L[5].spec.name, self.h_b)
        run(L[6], self.h_b, self.c); note(L[6].spec.name, self.c)
        run(L[7], self.c, self.h_a, residual=self.h_b, residual_scale=1.0); note(L[7].spec.name, self.h_a)
        run(L[8], self.h_a, self.u); note(L[8].spec.name, self.u)
        run(L[9], self.u, h_out, residual=self.h_a, residual_scale=0.5); note(L[9].spec.name, h_out)
        return h_out

    def _fused_qkv(self, L: List[QuantLinear]):
        """Codes, scales and bias of the q, k, v projections stacked along the output channels
        (built once per block and kept)."""
        key = id(L[2])
        if key not in self._qkv_weights:
            q, k, v = L[2], L[3], L[4]
            assert q.spec.bits_w == k.spec.bits_w == v.spec.bits_w and q.spec.act == k.spec.act == v.spec.act == aqt.ACT_NONE
            bias = None if q.bias is None else torch.cat([q.bias, k.bias, v.bias]).contiguous()
            self._qkv_weights[key] = (torch.cat([q.wq, k.wq, v.wq]).contiguous(), torch.cat([q.s_w, k.s_w, v.s_w]).contiguous(), bias)
        return self._qkv_weights[key]

    def ops(self, layers: List[QuantLinear]) -> int:
        return sum(2 * self.M * l.spec.N * l.spec.K for l in layers)


class EncoderStack:
    """n_blocks blocks in sequence, ping-ponging the residual stream between two buffers."""

    def __init__(self, M: int, d: int, ff: int, blocks: List[List[QuantLinear]], device, **kw):
        self.blocks = blocks
        self.block = ConformerBlockLinears(M, d, ff, blocks[0], device, **kw)
        self.h0 = torch.empty((M, d), dtype=torch.float32, device=device)
        self.h1 = torch.empty((M, d), dtype=torch.float32, device=device)

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        """x is read only; the result lives in one of the stack's own buffers."""
        src = x
        for b, layers in enumerate(self.blocks):
            dst = self.h0 if b % 2 == 0 else self.h1
            self.block.forward(layers, src, dst)
            src = dst
        return src

    @property
    def ops(self) -> int:
        return sum(self.block.ops(layers) for layers in self.blocks)
