"""ctypes front end of the CPU oracle (oracle/aqt_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  Nothing in the product package imports this module, and this module imports
nothing from the product package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aqt_oracle.c")
_LIB = os.path.join(_HERE, "libaqt_oracle.so")

AXIS_ROW, AXIS_COL, AXIS_TENSOR = 0, 1, 2
ROUND_HALF_UP_FLOOR, ROUND_NEAREST_EVEN = 0, 1
ACT_NONE, ACT_SWISH, ACT_GLU, ACT_GLU_SWISH = 0, 1, 2, 3
SCALE_ROW, SCALE_TENSOR = 0, 1

CFLAGS = ["-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than the source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_weight_bytes.restype = ctypes.c_int64
        L.orc_int_matmul.restype = ctypes.c_int64
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def num_threads() -> int:
    return int(lib().orc_num_threads())


def quantize(x: np.ndarray, bits: int, axis: int, rounding: int = ROUND_NEAREST_EVEN):
    """Fig. 2 quantize(input, axis): returns (codes int8 [rows, cols], scales fp32)."""
    assert x.dtype == np.float32 and x.ndim == 2 and x.strides[1] == 4
    rows, cols = x.shape
    ld = x.strides[0] // 4 if rows > 1 else cols
    q = np.empty((rows, cols), dtype=np.int8)
    n_scale = rows if axis == AXIS_ROW else (cols if axis == AXIS_COL else 1)
    s = np.empty(n_scale, dtype=np.float32)
    rc = lib().orc_quantize(_p(x), _i64(rows), _i64(cols), _i64(ld), bits, axis, rounding, _p(q), _p(s))
    if rc != 0:
        raise ValueError("orc_quantize: bad argument")
    return q, s


def dequantize(q: np.ndarray, scale: np.ndarray, axis: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    out = np.empty(q.shape, dtype=np.float32)
    lib().orc_dequantize(_p(q), _i64(q.shape[0]), _i64(q.shape[1]), _p(np.ascontiguousarray(scale, dtype=np.float32)), axis, _p(out))
    return out


def pack_int4(q: np.ndarray) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    rows, cols = q.shape
    out = np.empty((rows, cols // 2), dtype=np.uint8)
    if lib().orc_pack_int4(_p(q), _i64(rows), _i64(cols), _p(out)) != 0:
        raise ValueError("orc_pack_int4: cols must be even")
    return out


def unpack_int4(packed: np.ndarray, cols: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    rows = packed.shape[0]
    out = np.empty((rows, cols), dtype=np.int8)
    if lib().orc_unpack_int4(_p(packed), _i64(rows), _i64(cols), _p(out)) != 0:
        raise ValueError("orc_unpack_int4: cols must be even")
    return out


def weight_bytes(K: int, N: int, bits: int) -> int:
    return int(lib().orc_weight_bytes(_i64(K), _i64(N), bits))


def int_matmul(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """acc[m, n] = sum_k xq[m, k] * wq[n, k] (int64).  Raises if any result leaves int32."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = xq.shape
    N, K2 = wq.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int64)
    over = lib().orc_int_matmul(_p(xq), _p(wq), _i64(M), _i64(N), _i64(K), _p(acc))
    if over != 0:
        raise OverflowError("%d accumulators outside int32" % over)
    return acc


def emulated_matmul_f32(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = xq.shape
    N = wq.shape[0]
    out = np.empty((M, N), dtype=np.float32)
    lib().orc_emulated_matmul_f32(_p(xq), _p(wq), _i64(M), _i64(N), _i64(K), _p(out))
    return out


def _n_out(N: int, act: int) -> int:
    return N // 2 if act in (ACT_GLU, ACT_GLU_SWISH) else N


def epilogue_f32(acc, s_x, s_x_kind, s_w, bias=None, residual=None, residual_scale=1.0, act=ACT_NONE,
                 return_preact=False):
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    M, N = acc.shape
    y = np.empty((M, _n_out(N, act)), dtype=np.float32)
    z = np.empty((M, N), dtype=np.float32) if return_preact else None
    s_x = np.ascontiguousarray(s_x, dtype=np.float32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    residual = None if residual is None else np.ascontiguousarray(residual, dtype=np.float32)
    rc = lib().orc_epilogue_f32(_p(acc), _p(s_x), s_x_kind, _p(s_w), _p(bias), _p(residual), _i64(y.shape[1]),
                                ctypes.c_float(residual_scale), _i64(M), _i64(N), act, _p(y), _i64(y.shape[1]), _p(z))
    if rc != 0:
        raise ValueError("orc_epilogue_f32: bad argument")
    return (y, z) if return_preact else y


def epilogue_f64(acc, s_x, s_x_kind, s_w, bias=None, residual=None, residual_scale=1.0, act=ACT_NONE):
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    M, N = acc.shape
    y = np.empty((M, _n_out(N, act)), dtype=np.float64)
    s_x = np.ascontiguousarray(s_x, dtype=np.float32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    residual = None if residual is None else np.ascontiguousarray(residual, dtype=np.float32)
    rc = lib().orc_epilogue_f64(_p(acc), _p(s_x), s_x_kind, _p(s_w), _p(bias), _p(residual), _i64(y.shape[1]),
                                ctypes.c_float(residual_scale), _i64(M), _i64(N), act, _p(y))
    if rc != 0:
        raise ValueError("orc_epilogue_f64: bad argument")
    return y


def linear_fwd(x, wq, s_w, bias=None, residual=None, residual_scale=1.0, bits_a=8, a_scale_kind=SCALE_ROW,
               rounding=ROUND_NEAREST_EVEN, act=ACT_NONE, return_parts=False):
    """Whole layer: quantize x, integer matmul against codes wq [N, K], epilogue.

    With return_parts also returns (xq, s_x, acc)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = x.shape
    N = wq.shape[0]
    assert wq.shape[1] == K
    y = np.empty((M, _n_out(N, act)), dtype=np.float32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    residual = None if residual is None else np.ascontiguousarray(residual, dtype=np.float32)
    xq = np.empty((M, K), dtype=np.int8) if return_parts else None
    sx = np.empty(M if a_scale_kind == SCALE_ROW else 1, dtype=np.float32) if return_parts else None
    acc = np.empty((M, N), dtype=np.int64) if return_parts else None
    rc = lib().orc_linear_fwd(_p(x), _i64(K), _p(wq), _p(s_w), _p(bias), _p(residual), _i64(y.shape[1]),
                              ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K), bits_a, a_scale_kind,
                              rounding, act, _p(y), _i64(y.shape[1]), _p(xq), _p(sx), _p(acc))
    if rc == -2:
        raise OverflowError("accumulator outside int32")
    if rc != 0:
        raise ValueError("orc_linear_fwd: bad argument")
    return (y, xq, sx, acc) if return_parts else y


def linear_weight_only_f64(x, wq, s_w, bias=None, residual=None, residual_scale=1.0, act=ACT_NONE, return_parts=False):
    """The weight-only layer (float activations, integer weights de-quantized by their channel
    scale) in double.  With return_parts also returns (z, mag): pre-activations and the magnitude
    s_w * sum_k |x * wq| of each."""
    x = np.asarray(x, dtype=np.float32)
    assert x.ndim == 2 and x.strides[1] == 4
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    M, K = x.shape
    ldx = x.strides[0] // 4 if M > 1 else K
    N = wq.shape[0]
    assert wq.shape[1] == K
    y = np.empty((M, _n_out(N, act)), dtype=np.float64)
    z = np.empty((M, N), dtype=np.float64) if return_parts else None
    mag = np.empty((M, N), dtype=np.float64) if return_parts else None
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    residual = None if residual is None else np.ascontiguousarray(residual, dtype=np.float32)
    rc = lib().orc_linear_weight_only_f64(_p(x), _i64(ldx), _p(wq), _p(s_w), _p(bias), _p(residual), _i64(y.shape[1]),
                                          ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K), act, _p(y), _p(z), _p(mag))
    if rc != 0:
        raise ValueError("orc_linear_weight_only_f64: bad argument")
    return (y, z, mag) if return_parts else y


def linear_bwd_f64(dy, xq, s_x, wq, s_w, s_x_kind=SCALE_ROW, return_mags=False):
    """Straight-through backward of the quantized linear layer in double: returns (dx [M, K],
    dw [N, K], db [N]); with return_mags also the sums of absolute values of the same terms."""
    dy = np.asarray(dy, dtype=np.float32)
    assert dy.ndim == 2 and dy.strides[1] == 4
    M, N = dy.shape
    lddy = dy.strides[0] // 4 if M > 1 else N
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    K = xq.shape[1]
    assert xq.shape == (M, K) and wq.shape == (N, K)
    s_x = np.ascontiguousarray(s_x, dtype=np.float32)
    s_w = np.ascontiguousarray(s_w, dtype=np.float32)
    dx, dw, db = np.empty((M, K)), np.empty((N, K)), np.empty(N)
    mags = (np.empty((M, K)), np.empty((N, K)), np.empty(N)) if return_mags else (None, None, None)
    rc = lib().orc_linear_bwd_f64(_p(dy), _i64(lddy), _p(xq), _p(s_x), s_x_kind, _p(wq), _p(s_w), _i64(M), _i64(N), _i64(K),
                                  _p(dx), _p(dw), _p(db), _p(mags[0]), _p(mags[1]), _p(mags[2]))
    if rc != 0:
        raise ValueError("orc_linear_bwd_f64: bad argument")
    return (dx, dw, db) + (mags if return_mags else ())
