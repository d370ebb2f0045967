"""Seeded synthetic inputs for the quantized-linear hot path.

This module is the only code shared by the CPU oracle's tests and the CUDA path.  It holds no
quantizer, matmul or epilogue arithmetic: it produces float32 arrays (activations, weights,
biases) and the shape tables of the workloads.

Every value is a pure function of (seed, tensor id, element index), so any row subset of a tensor
can be produced without materialising the whole tensor, and both sides of a parity test see the
same bits.

The paper trains on LibriSpeech and a private corpus (Section 3.1); neither is needed for this
path, whose cost depends only on shapes, bit widths and, for abs-max scaling, on the tails of the
value distribution.  The tensors here take the Conformer-L shapes of Section 3.2 (17 blocks, model
width 512, 8 heads) and stand in for those workloads.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)
_TID = np.uint64(0xD6E8FEB86659FD93)


def _mix64(z: np.ndarray) -> np.ndarray:
    """64-bit finaliser (xor-shift-multiply); a bijection on uint64."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        a = _mix64(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)]) + _GOLDEN)
        b = _mix64(np.array([np.uint64(tensor_id & 0xFFFFFFFFFFFFFFFF)]) * _TID + _C1)
        return _mix64(a ^ b)[0]


def uniform01(seed: int, tensor_id: int, index: np.ndarray) -> np.ndarray:
    """Doubles strictly inside (0, 1), one per counter value in ``index``."""
    key = _stream_key(seed, tensor_id)
    with np.errstate(over="ignore"):
        z = _mix64(np.asarray(index, dtype=np.uint64) * _GOLDEN + key)
    return ((z >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_f64(seed: int, tensor_id: int, index: np.ndarray) -> np.ndarray:
    """Standard normal via Box-Muller in double precision, counters 2i and 2i+1."""
    idx = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        u1 = uniform01(seed, tensor_id, idx * np.uint64(2))
        u2 = uniform01(seed, tensor_id, idx * np.uint64(2) + np.uint64(1))
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def _index_grid(rows: int, cols: int, row_subset: Optional[Sequence[int]]) -> np.ndarray:
    r = np.arange(rows, dtype=np.uint64) if row_subset is None else np.asarray(row_subset, dtype=np.uint64)
    c = np.arange(cols, dtype=np.uint64)
    return r[:, None] * np.uint64(cols) + c[None, :]


def _for_each_chunk(n_rows: int, chunk_rows: int, fill) -> None:
    """fill(a, b) for consecutive row ranges; large tensors on a few threads (the numpy kernels
    release the interpreter lock, and every element is a function of its own counter only, so the
    result does not depend on how the rows are cut)."""
    starts = list(range(0, n_rows, chunk_rows))
    threads = min(len(starts), os.cpu_count() or 1, 16)
    if threads <= 1:
        for a in starts:
            fill(a, min(a + chunk_rows, n_rows))
        return
    with ThreadPoolExecutor(max_workers=threads) as pool:
        list(pool.map(lambda a: fill(a, min(a + chunk_rows, n_rows)), starts))


def normal(seed: int, tensor_id: int, rows: int, cols: int, std: float = 1.0,
           row_subset: Optional[Sequence[int]] = None, chunk_rows: int = 2048) -> np.ndarray:
    """float32 [rows, cols] (or [len(row_subset), cols]) ~ N(0, std^2)."""
    sel = np.arange(rows) if row_subset is None else np.asarray(row_subset)
    out = np.empty((len(sel), cols), dtype=np.float32)

    def fill(a, b):
        idx = _index_grid(rows, cols, sel[a:b])
        out[a:b] = (_normal_f64(seed, tensor_id, idx) * std).astype(np.float32)
    _for_each_chunk(len(sel), chunk_rows, fill)
    return out


def student_t3(seed: int, tensor_id: int, rows: int, cols: int,
               row_subset: Optional[Sequence[int]] = None, chunk_rows: int = 1024) -> np.ndarray:
    """float32 heavy-tailed activations: Student-t with 3 degrees of freedom, unit variance.

    t = z0 / sqrt((z1^2 + z2^2 + z3^2) / 3), divided by sqrt(3) (the variance of t_3 is 3).
    Four independent normal streams are taken from sub-ids of ``tensor_id``.
    """
    sel = np.arange(rows) if row_subset is None else np.asarray(row_subset)
    out = np.empty((len(sel), cols), dtype=np.float32)

    def fill(a, b):
        idx = _index_grid(rows, cols, sel[a:b])
        z = [_normal_f64(seed, tensor_id * 4 + j + (1 << 60), idx) for j in range(4)]
        t = z[0] / np.sqrt((z[1] ** 2 + z[2] ** 2 + z[3] ** 2) / 3.0)
        out[a:b] = (t / np.sqrt(3.0)).astype(np.float32)
    _for_each_chunk(len(sel), chunk_rows, fill)
    return out


def random_codes(seed: int, rows: int, cols: int, bits: int) -> np.ndarray:
    """int8 [rows, cols] quantization codes drawn uniformly from [-qmax, qmax] (qmax = 127 at 8
    bits, 7 at 4), for tests that start from codes instead of from float tensors.  One sequential
    stream per seed (numpy's PCG64), so the full tensor is generated and rows are picked from it."""
    qmax = 127 if bits == 8 else 7
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(-qmax, qmax + 1, size=(rows, cols), dtype=np.int8)


def tensor_id(config: int, block: int = 0, layer: int = 0, role: int = 0) -> int:
    """Tensor id from (config, block, layer, role); role: 0 x, 1 W, 2 bias, 3 residual."""
    return (config << 40) | (block << 24) | (layer << 8) | role


ROLE_X, ROLE_W, ROLE_BIAS, ROLE_RES = 0, 1, 2, 3

# Epilogue activations (numeric values match the C ABI's AQT_ACT_* constants).
ACT_NONE, ACT_SWISH, ACT_GLU, ACT_GLU_SWISH = 0, 1, 2, 3


@dataclass(frozen=True)
class LinearSpec:
    """One weight-bearing linear of a Conformer block: y = act(x W + b), W is [K, N]."""
    name: str
    K: int
    N: int
    act: int = ACT_NONE
    bits_w: int = 4
    bits_a: int = 8

    @property
    def n_out(self) -> int:
        return self.N // 2 if self.act in (ACT_GLU, ACT_GLU_SWISH) else self.N


def weight(seed: int, tid: int, K: int, N: int, std: Optional[float] = None) -> np.ndarray:
    """W^T as float32 [N, K] (output channel major, K contiguous), entries ~ N(0, 1/fan_in).

    Element (k, n) of the [K, N] matrix W has counter k*N + n, so the [K, N] view and this
    transposed view hold the same numbers.
    """
    std = (1.0 / np.sqrt(K)) if std is None else std
    return np.ascontiguousarray(normal(seed, tid, K, N, std=std).T)


def block_linears(d: int, ff: int, bits_ffn_w: int, bits_attn_w: int, bits_a: int) -> list:
    """The ten linears of one Conformer block, in execution order.

    FFN module a (d->ff Swish, ff->d), attention projections Q, K, V, O (d->d), convolution
    module pointwise 1 (d->2d, GLU, then Swish) and pointwise 2 (d->d), FFN module b.
    Which layers are quantized follows Section 3.3 (encoder layers only); per-layer bit widths
    are arguments because Table 2 mixes int4 and int8 by layer.
    """
    f, a = bits_ffn_w, bits_attn_w
    return [
        LinearSpec("ffn_a1", d, ff, ACT_SWISH, f, bits_a),
        LinearSpec("ffn_a2", ff, d, ACT_NONE, f, bits_a),
        LinearSpec("attn_q", d, d, ACT_NONE, a, bits_a),
        LinearSpec("attn_k", d, d, ACT_NONE, a, bits_a),
        LinearSpec("attn_v", d, d, ACT_NONE, a, bits_a),
        LinearSpec("attn_o", d, d, ACT_NONE, a, bits_a),
        LinearSpec("conv_pw1", d, 2 * d, ACT_GLU_SWISH, a, bits_a),
        LinearSpec("conv_pw2", d, d, ACT_NONE, a, bits_a),
        LinearSpec("ffn_b1", d, ff, ACT_SWISH, f, bits_a),
        LinearSpec("ffn_b2", ff, d, ACT_NONE, f, bits_a),
    ]


@dataclass(frozen=True)
class Workload:
    """A benchmark/parity configuration: shapes, bit widths, scale kinds, input distribution."""
    cfg: int
    name: str
    M: int
    d: int
    ff: int
    blocks: int
    bits_ffn_w: int
    bits_attn_w: int
    bits_a: int
    a_scale: str          # "row" | "tensor"
    x_dist: str           # "normal" | "student_t3"
    kind: str             # "single" | "ffn_pair" | "block" | "stack"


WORKLOADS = {
    1: Workload(1, "single_linear_64x256x256_w8a8_tensor", 64, 256, 256, 1, 8, 8, 8, "tensor", "normal", "single"),
    2: Workload(2, "conformer_ffn_pair_d512_ff2048_M12800_w4a8", 12800, 512, 2048, 1, 4, 4, 8, "row", "normal", "ffn_pair"),
    3: Workload(3, "conformer_block_d512_M12800_w4a4", 12800, 512, 2048, 1, 4, 4, 4, "row", "normal", "block"),
    4: Workload(4, "conformer_stack17_d512_M25600_mixed_w4w8_a8", 25600, 512, 2048, 17, 4, 8, 8, "row", "normal", "stack"),
    5: Workload(5, "conformer_stack17_d1024_M65536_w4a8_student_t3", 65536, 1024, 4096, 17, 4, 4, 8, "row", "student_t3", "stack"),
}


def workload_input(w: Workload, seed: int = 0, row_subset: Optional[Sequence[int]] = None) -> np.ndarray:
    """Block-0 input activations x [M, d] (or the given rows of it)."""
    tid = tensor_id(w.cfg, 0, 0, ROLE_X)
    if w.x_dist == "student_t3":
        return student_t3(seed, tid, w.M, w.d, row_subset=row_subset)
    return normal(seed, tid, w.M, w.d, row_subset=row_subset)


def workload_layers(w: Workload) -> list:
    if w.kind == "single":
        return [LinearSpec("linear", w.d, w.ff, ACT_NONE, w.bits_ffn_w, w.bits_a)]
    if w.kind == "ffn_pair":
        return [LinearSpec("ffn_1", w.d, w.ff, ACT_SWISH, w.bits_ffn_w, w.bits_a),
                LinearSpec("ffn_2", w.ff, w.d, ACT_NONE, w.bits_ffn_w, w.bits_a)]
    return block_linears(w.d, w.ff, w.bits_ffn_w, w.bits_attn_w, w.bits_a)


def layer_weight(w: Workload, block: int, layer: int, spec: LinearSpec, seed: int = 0) -> np.ndarray:
    """float32 W^T [N, K] for layer ``layer`` of block ``block``."""
    std = 0.05 if w.cfg == 1 else None
    return weight(seed, tensor_id(w.cfg, block, layer, ROLE_W), spec.K, spec.N, std=std)


def layer_bias(w: Workload, block: int, layer: int, spec: LinearSpec, seed: int = 0) -> Optional[np.ndarray]:
    """float32 bias [N]: N(0, 0.01^2) for the single-linear workload, none (zero) elsewhere."""
    if w.cfg != 1:
        return None
    return normal(seed, tensor_id(w.cfg, block, layer, ROLE_BIAS), 1, spec.N, std=0.01)[0]
