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

Residual adds are fp32 and are fused into the epilogue of the producing linear.  Where a linear
with K <= 512 feeds another quantized linear, its epilogue also quantizes its output rows
(aqt_qmatmul_requant): the fp32 tensor between the two is then written only if it is needed as
well (the residual stream, or a parity check; the GLU layer only fuses when it is not).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from . import binding as aqt
from .inputs import LinearSpec


def _container_bits(bits_a: int) -> int:
    """Activation codes travel between kernels in int8 containers (as Fig. 2 casts them)."""
    return 8 if bits_a == 8 else aqt.BITS_4_UNPACKED


@dataclass
class QuantLinear:
    """Pre-quantized weights of one linear: codes W^T [N, K] (nibble-packed when 4-bit), one
    fp32 scale per output channel (Section 2.2, channel-wise), optional fp32 bias."""
    spec: LinearSpec
    wq: torch.Tensor
    s_w: torch.Tensor
    bias: Optional[torch.Tensor]
    wq_unpacked: Optional[torch.Tensor] = None

    @classmethod
    def from_float(cls, spec: LinearSpec, wt: torch.Tensor, bias: Optional[torch.Tensor] = None,
                   rounding: int = aqt.ROUND_NEAREST_EVEN) -> "QuantLinear":
        """wt: fp32 W^T [N, K] on the GPU.  Quantizes over K per output channel with the same
        quantizer the activations use (Fig. 2), packing 4-bit codes two per byte."""
        assert wt.shape == (spec.N, spec.K)
        wq, s_w = aqt.aqt_quantize(wt, spec.bits_w, aqt.AXIS_ROW, rounding, pack=(spec.bits_w == 4))
        return cls(spec, wq, s_w, bias).prepare()

    def prepare(self) -> "QuantLinear":
        """Packed 4-bit weights deeper than the weight-stationary kernel's 512 (which sign-extends
        them itself in shared memory) would be sign-extended into the workspace on every call:
        do it once here and hand the matmuls the int8 containers instead."""
        s = self.spec
        if s.bits_w == 4 and (s.K > 512 or s.K % 32 != 0) and self.wq_unpacked is None:
            self.wq_unpacked = aqt.aqt_unpack_int4(self.wq, s.K)
        return self

    @property
    def mm_weight(self) -> torch.Tensor:
        """The codes as handed to the matmul entry points."""
        return self.wq if self.wq_unpacked is None else self.wq_unpacked

    @property
    def mm_bits(self) -> int:
        return self.spec.bits_w if self.wq_unpacked is None else aqt.BITS_4_UNPACKED

    @property
    def weight_bytes(self) -> int:
        return self.wq.numel() + 4 * self.s_w.numel()


class WeightArena:
    """The float weights W^T [N_i, K] of many linears kept in one tensor per (K, bit width), one
    below the other, so that re-quantizing all of them (every training step when the model is
    trained quantized from scratch, Section 2.2) is one quantizer call per group instead of one
    per weight: the quantizer reduces over K row by row (one scale per output channel), so the
    rows of different weights do not interact and the codes and scales are those of the
    per-weight calls.  `float_view(i)` is weight i's slice of the arena (the optimizer writes
    there); `quantize()` fills the code and scale arenas; `linear(i)` wraps weight i's slices."""

    def __init__(self, specs: List[LinearSpec], device):
        self.specs = list(specs)
        self.groups: Dict[tuple, List[int]] = {}
        for i, sp in enumerate(self.specs):
            self.groups.setdefault((sp.K, sp.bits_w), []).append(i)
        self.float_arena: Dict[tuple, torch.Tensor] = {}
        self.code_arena: Dict[tuple, torch.Tensor] = {}
        self.scale_arena: Dict[tuple, torch.Tensor] = {}
        self._row0: Dict[int, int] = {}
        for key, members in self.groups.items():
            K, bits = key
            rows = 0
            for i in members:
                self._row0[i] = rows
                rows += self.specs[i].N
            self.float_arena[key] = torch.empty((rows, K), dtype=torch.float32, device=device)
            self.code_arena[key] = torch.empty((rows, K // 2 if bits == 4 else K), dtype=torch.uint8 if bits == 4 else torch.int8,
                                               device=device)
            self.scale_arena[key] = torch.empty(rows, dtype=torch.float32, device=device)

    def _slice(self, arena: Dict[tuple, torch.Tensor], i: int) -> torch.Tensor:
        sp = self.specs[i]
        r0 = self._row0[i]
        return arena[(sp.K, sp.bits_w)][r0:r0 + sp.N]

    def float_view(self, i: int) -> torch.Tensor:
        return self._slice(self.float_arena, i)

    def quantize(self, rounding: int = aqt.ROUND_NEAREST_EVEN, stream=None) -> int:
        """One quantizer call per group; returns the number of calls."""
        for key, wt in self.float_arena.items():
            aqt.aqt_quantize(wt, key[1], aqt.AXIS_ROW, rounding, pack=(key[1] == 4), q_out=self.code_arena[key],
                             scale_out=self.scale_arena[key], stream=stream)
        return len(self.float_arena)

    def linear(self, i: int, bias: Optional[torch.Tensor] = None) -> "QuantLinear":
        return QuantLinear(self.specs[i], self._slice(self.code_arena, i), self._slice(self.scale_arena, i), bias).prepare()

    @property
    def algorithmic_bytes(self) -> int:
        """fp32 weights read, codes and scales written."""
        return sum(4 * w.numel() + self.code_arena[k].numel() + 4 * self.scale_arena[k].numel() for k, w in self.float_arena.items())


class LayerRunner:
    """Owns the scratch workspace shared by all layers of a workload and runs single layers."""

    def __init__(self, M: int, layers: List[QuantLinear], device, a_scale_kind: int = aqt.SCALE_ROW,
                 rounding: int = aqt.ROUND_NEAREST_EVEN):
        self.M, self.device, self.a_scale_kind, self.rounding = M, device, a_scale_kind, rounding
        need = max(max(aqt.aqt_workspace_bytes(op, M, 3 * l.spec.N, l.spec.K, l.spec.bits_a, l.spec.bits_w)
                       for op in (aqt.OP_LINEAR_FWD, aqt.OP_QMATMUL_REQUANT)) for l in layers)
        self.workspace = torch.empty(need, dtype=torch.uint8, device=device)
        self._codes: Dict[str, tuple] = {}

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

    def matmul(self, layer: QuantLinear, xq: torch.Tensor, s_x: torch.Tensor, y: torch.Tensor,
               residual: Optional[torch.Tensor] = None, residual_scale: float = 1.0) -> torch.Tensor:
        """Integer matmul + epilogue of `layer` on already-quantized activations (int8 containers)."""
        s = layer.spec
        return aqt.aqt_qmatmul(xq, s_x, layer.mm_weight, layer.s_w, layer.bias, residual, residual_scale, K=s.K, bits_a=_container_bits(s.bits_a),
                               bits_w=layer.mm_bits, act=s.act, s_x_kind=self.a_scale_kind, y=y, workspace=self.workspace)

    def fuses_requant(self, layer: QuantLinear, with_y: bool = True) -> bool:
        """True if `layer`'s matmul can quantize its own output rows in its epilogue (the GLU
        forms and 512 < K <= 1024 only when the fp32 output is not wanted as well; 1024 < K < 2048
        not at all)."""
        s = layer.spec
        ok = self.a_scale_kind == aqt.SCALE_ROW and s.K % 16 == 0 and s.n_out % 32 == 0 and s.N <= 128 * 148
        glu = s.act in (aqt.ACT_GLU, aqt.ACT_GLU_SWISH)
        if s.K >= 2048:
            # deep K: the CTA-pair kernel quantizes its rows (no GLU; at most 16 column parts per row)
            return ok and not glu and self.M > 128 and s.N <= 2048
        if glu or s.K > 512:
            return ok and not with_y and s.K <= 1024
        return ok

    def code_buffers(self, role: str, cols: int):
        """Codes (int8 containers) and row scales of an activation tensor, one pair of buffers per role."""
        if role not in self._codes or self._codes[role][0].shape[1] != cols:
            self._codes[role] = (torch.empty((self.M, cols), dtype=torch.int8, device=self.device),
                                 torch.empty(self.M, dtype=torch.float32, device=self.device))
        return self._codes[role]

    def matmul_requant(self, layer: QuantLinear, xq: torch.Tensor, s_x: torch.Tensor, bits_out: int, role: str,
                       y: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None, residual_scale: float = 1.0):
        """`layer` on quantized activations, its output rows quantized to `bits_out` bits in the
        epilogue.  Returns (codes, scales); y (fp32) is written too if given."""
        s = layer.spec
        q, sc = self.code_buffers(role, s.n_out)
        aqt.aqt_qmatmul_requant(xq, s_x, layer.mm_weight, layer.s_w, layer.bias, residual, residual_scale, K=s.K, bits_a=_container_bits(s.bits_a),
                                bits_w=layer.mm_bits, act=s.act, s_x_kind=self.a_scale_kind, bits_out=bits_out,
                                rounding=self.rounding, pack_out=False, q_out=q, s_out=sc, y=y, workspace=self.workspace)
        return q, sc

    def __call__(self, layer: QuantLinear, x: torch.Tensor, y: torch.Tensor, residual: Optional[torch.Tensor] = None,
                 residual_scale: float = 1.0) -> torch.Tensor:
        s = layer.spec
        return aqt.aqt_linear_fwd(x, layer.mm_weight, layer.s_w, layer.bias, residual, residual_scale, bits_a=s.bits_a,
                                  bits_w=layer.mm_bits, a_scale_kind=self.a_scale_kind, rounding=self.rounding, act=s.act,
                                  y=y, workspace=self.workspace)


class FfnPair:
    """y = W_2 . Swish(W_1 . x).  The second layer consumes the first layer's output as codes and
    row scales; the first matmul produces them in its epilogue when it can (`fused`), and the fp32
    hidden tensor u is then written only with keep_u (parity checks)."""

    def __init__(self, M: int, layers: List[QuantLinear], device, fused: bool = True, keep_u: bool = False, **kw):
        assert len(layers) == 2
        self.layers = layers
        self.run = LayerRunner(M, layers, device, **kw)
        self.fused = fused and self.run.fuses_requant(layers[0], with_y=keep_u)
        self.keep_u = keep_u or not self.fused
        self.u = torch.empty((M, layers[0].spec.n_out), dtype=torch.float32, device=device) if self.keep_u else None

    def forward(self, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
        if not self.fused:
            self.run(self.layers[0], x, self.u)
            return self.run(self.layers[1], self.u, y)
        l0, l1 = self.layers
        xq, xs = self.run.quantize_input(x, l0.spec.bits_a)
        uq, us = self.run.matmul_requant(l0, xq, xs, l1.spec.bits_a, "u", y=self.u)
        return self.run.matmul(l1, uq, us, y)

    @property
    def launches_per_step(self) -> int:
        """Kernels of the library launched by one forward()."""
        l0, l1 = self.layers
        return 3 if self.fused else 4

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
                keep: Optional[Dict[str, torch.Tensor]] = None, in_codes=None, next_bits: Optional[int] = None):
        """h_in -> h_out (distinct buffers, neither h_a nor h_b).  `keep`, if given, receives
        clones of every intermediate keyed by layer name (for parity checks).  in_codes: (codes,
        scales) of h_in if the producer already quantized its rows.  next_bits: if given, the last
        matmul also quantizes the rows of h_out to that width for the next block, and the codes and
        scales are returned with h_out (None where the shape does not allow it)."""
        L, run = layers, self.run

        def note(name, t):
            if keep is not None:
                keep[name] = t.clone()

        parity = keep is not None  # then every fp32 intermediate is written as well
        hq, hs = self._ffn(L[0], L[1], h_in, self.h_a, 0.5, parity, note, xq=in_codes[0] if in_codes else None,
                           xs=in_codes[1] if in_codes else None, out_role="ha", out_bits=L[2].spec.bits_a)
        note(L[1].spec.name, self.h_a)
        # q, k, v read the same h: its codes come out of the second feed-forward matmul's epilogue
        # (or one quantizer pass; the codes do not depend on the consumer), and the three
        # projections run as one matmul over their concatenated output channels
        if hq is None:
            hq, hs = run.quantize_input(self.h_a, L[2].spec.bits_a)
        wq, s_w, bias = self._fused_qkv(L)
        aqt.aqt_qmatmul(hq, hs, wq, s_w, bias, None, 1.0, K=self.d, bits_a=_container_bits(L[2].spec.bits_a), bits_w=L[2].mm_bits, act=aqt.ACT_NONE,
                        s_x_kind=run.a_scale_kind, y=self.qkv, workspace=run.workspace)
        note(L[2].spec.name, self.q); note(L[3].spec.name, self.k); note(L[4].spec.name, self.v)
        # h_b = h_a + W_o v is needed both as fp32 (residual stream) and as codes (pointwise 1)
        bq = bs = cq = cs = None
        if run.fuses_requant(L[5]):
            vq, vs = run.quantize_input(self.v, L[5].spec.bits_a)
            bq, bs = run.matmul_requant(L[5], vq, vs, L[6].spec.bits_a, "h", y=self.h_b, residual=self.h_a, residual_scale=1.0)
        else:
            run(L[5], self.v, self.h_b, residual=self.h_a, residual_scale=1.0)
        note(L[5].spec.name, self.h_b)
        # c = Swish(GLU(W_pw1 h_b)) is only read by pointwise 2: it leaves pointwise 1 as codes when it can
        if not parity and run.fuses_requant(L[6], with_y=False):
            if bq is None:
                bq, bs = run.quantize_input(self.h_b, L[6].spec.bits_a)
            cq, cs = run.matmul_requant(L[6], bq, bs, L[7].spec.bits_a, "c")
        elif bq is not None:
            run.matmul(L[6], bq, bs, self.c)
        else:
            run(L[6], self.h_b, self.c)
        if cq is None:
            note(L[6].spec.name, self.c)
        # h_a = h_b + W_pw2 c, again as fp32 and as codes (first layer of feed-forward module b)
        if run.fuses_requant(L[7]):
            if cq is None:
                cq, cs = run.quantize_input(self.c, L[7].spec.bits_a)
            aq, as_ = run.matmul_requant(L[7], cq, cs, L[8].spec.bits_a, "h", y=self.h_a, residual=self.h_b, residual_scale=1.0)
            note(L[7].spec.name, self.h_a)
            out_codes = self._ffn(L[8], L[9], self.h_a, h_out, 0.5, parity, note, xq=aq, xs=as_, out_role="hb", out_bits=next_bits)
        else:
            if cq is not None:
                run.matmul(L[7], cq, cs, self.h_a, residual=self.h_b, residual_scale=1.0)
            else:
                run(L[7], self.c, self.h_a, residual=self.h_b, residual_scale=1.0)
            note(L[7].spec.name, self.h_a)
            out_codes = self._ffn(L[8], L[9], self.h_a, h_out, 0.5, parity, note, out_role="hb", out_bits=next_bits)
        note(L[9].spec.name, h_out)
        if next_bits is not None:
            return h_out, (out_codes if out_codes[0] is not None else None)
        return h_out

    def _ffn(self, l0: QuantLinear, l1: QuantLinear, h: torch.Tensor, out: torch.Tensor, rs: float, parity: bool, note,
             xq: Optional[torch.Tensor] = None, xs: Optional[torch.Tensor] = None, out_role: str = "ha",
             out_bits: Optional[int] = None):
        """out = h + rs * W_1 . Swish(W_0 . h); xq, xs: codes and scales of h if already at hand.
        out_bits: also quantize the rows of `out` to that width in the second matmul's epilogue
        where it can; returns (codes, scales) of out, or (None, None)."""
        run = self.run
        fuse_out = out_bits is not None and run.fuses_requant(l1, with_y=True)
        if run.fuses_requant(l0, with_y=parity):
            if xq is None:
                xq, xs = run.quantize_input(h, l0.spec.bits_a)
            uq, us = run.matmul_requant(l0, xq, xs, l1.spec.bits_a, "u", y=self.u if parity else None)
            if parity:
                note(l0.spec.name, self.u)
        else:
            run(l0, h, self.u); note(l0.spec.name, self.u)
            if not fuse_out:
                run(l1, self.u, out, residual=h, residual_scale=rs)
                return None, None
            uq, us = run.code_buffers("u", l0.spec.n_out)
            aqt.aqt_quantize(self.u, l1.spec.bits_a, aqt.AXIS_ROW, run.rounding, q_out=uq, scale_out=us)
        if fuse_out:
            return run.matmul_requant(l1, uq, us, out_bits, out_role, y=out, residual=h, residual_scale=rs)
        run.matmul(l1, uq, us, out, residual=h, residual_scale=rs)
        return None, None

    def _fused_qkv(self, L: List[QuantLinear]):
        """Codes, scales and bias of the q, k, v projections stacked along the output channels
        (built once per block and kept)."""
        key = id(L[2])
        if key not in self._qkv_weights:
            q, k, v = L[2], L[3], L[4]
            assert q.spec.bits_w == k.spec.bits_w == v.spec.bits_w and q.spec.act == k.spec.act == v.spec.act == aqt.ACT_NONE
            bias = None if q.bias is None else torch.cat([q.bias, k.bias, v.bias]).contiguous()
            self._qkv_weights[key] = (torch.cat([q.mm_weight, k.mm_weight, v.mm_weight]).contiguous(),
                                      torch.cat([q.s_w, k.s_w, v.s_w]).contiguous(), bias)
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
        src, codes = x, None
        for b, layers in enumerate(self.blocks):
            dst = self.h0 if b % 2 == 0 else self.h1
            nxt = self.blocks[b + 1][0].spec.bits_a if b + 1 < len(self.blocks) else None
            if nxt is None:
                self.block.forward(layers, src, dst, in_codes=codes)
                codes = None
            else:
                _, codes = self.block.forward(layers, src, dst, in_codes=codes, next_bits=nxt)
            src = dst
        return src

    @property
    def ops(self) -> int:
        return sum(self.block.ops(layers) for layers in self.blocks)
