"""Thin Python binding of the C ABI in include/aqt.h: same names, argument marshalling only.

Every step of the quantized linear layer runs in the CUDA library; torch is used here for device
memory and the current stream.  There is no CPU fallback: if the shared library is missing the
import of any entry point fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

# enums of include/aqt.h
AQT_OK = 0
AXIS_ROW, AXIS_COL, AXIS_TENSOR = 0, 1, 2
ROUND_HALF_UP_FLOOR, ROUND_NEAREST_EVEN = 0, 1
SCALE_ROW, SCALE_TENSOR = 0, 1
ACT_NONE, ACT_SWISH, ACT_GLU, ACT_GLU_SWISH = 0, 1, 2, 3
OP_QMATMUL, OP_LINEAR_FWD, OP_QMATMUL_REQUANT, OP_LINEAR_WEIGHT_ONLY, OP_LINEAR_WEIGHT_ONLY_X2, OP_LINEAR_BWD, OP_FFN_FWD = 1, 2, 3, 4, 5, 6, 7
FLOAT_TF32, FLOAT_TF32X2 = 0, 1
BITS_4_UNPACKED = 48  # 4-bit codes, one per int8 container
STATIC_WEIGHTS = 0x100  # OR into bits_w: the weights were complete before the preceding work on the stream was enqueued

EXPORTS = ("aqt_version", "aqt_status_string", "aqt_quantize", "aqt_pack_int4", "aqt_unpack_int4", "aqt_qmatmul",
           "aqt_linear_fwd", "aqt_linear_fwd_host", "aqt_workspace_bytes", "aqt_device_status", "aqt_qmatmul_w4_noalloc",
           "aqt_selftest_bounded_wait", "aqt_qmatmul_requant", "aqt_linear_fwd_weight_only", "aqt_linear_bwd",
           "aqt_plan_qmatmul", "aqt_qmatmul_with_plan", "aqt_ffn_fwd", "aqt_selftest_sfu_rate")
NOALLOC_MAX_WEIGHT_BYTES = 4 << 20


class AqtError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (fn, status, status_string(status)))


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load libaqt.so (built in-tree by paper_2203_15952_b200.build).  Never falls back."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise ImportError("CUDA library %s is missing; build it with `python -m paper_2203_15952_b200.build` "
                              "(needs nvcc). There is no CPU fallback." % path)
        L = ctypes.CDLL(path)
        L.aqt_status_string.restype = ctypes.c_char_p
        L.aqt_workspace_bytes.restype = ctypes.c_size_t
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().aqt_status_string(int(status)).decode()


def _check(fn: str, status: int) -> None:
    if status != AQT_OK:
        raise AqtError(fn, status)


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _i64(v) -> ctypes.c_int64:
    return ctypes.c_int64(int(v))


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _n_out(N: int, act: int) -> int:
    return N // 2 if act in (ACT_GLU, ACT_GLU_SWISH) else N


def bind(fn_name: str, *cargs):
    """Pre-marshalled call: returns a zero-argument callable that invokes entry point `fn_name`
    with the given ctypes arguments and raises AqtError on a non-zero status.  For launch-rate
    sensitive loops (the arguments, including the stream, are fixed at bind time)."""
    fn = getattr(lib(), fn_name)

    def call():
        st = fn(*cargs)
        if st != AQT_OK:
            raise AqtError(fn_name, st)
    return call


def bind_quantize(x, bits, axis, rounding, pack, q_out, scale_out, stream=None):
    rows, cols = x.shape
    return bind("aqt_quantize", _ptr(x), _i64(rows), _i64(cols), _i64(x.stride(0)), int(bits), int(axis), int(rounding),
                int(bool(pack)), _ptr(q_out), _ptr(scale_out), _stream(stream))


def bind_qmatmul(xq, s_x, wq, s_w, bias, residual, residual_scale, K, bits_a, bits_w, act, s_x_kind, y, workspace,
                 stream=None):
    M, N = xq.shape[0], wq.shape[0]
    return bind("aqt_qmatmul", _ptr(xq), _ptr(s_x), int(s_x_kind), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
                _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N),
                _i64(K), int(bits_a), int(bits_w), int(act), _ptr(y), _i64(y.stride(0)), _ptr(None), _ptr(workspace),
                ctypes.c_size_t(0 if workspace is None else workspace.numel()), _stream(stream))


def bind_qmatmul_requant(xq, s_x, wq, s_w, bias, residual, residual_scale, K, bits_a, bits_w, act, s_x_kind, bits_out, rounding,
                         pack_out, q_out, s_out, y, workspace, stream=None):
    M, N = xq.shape[0], wq.shape[0]
    return bind("aqt_qmatmul_requant", _ptr(xq), _ptr(s_x), int(s_x_kind), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
                _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N),
                _i64(K), int(bits_a), int(bits_w), int(act), int(bits_out), int(rounding), int(bool(pack_out)), _ptr(q_out),
                _ptr(s_out), _ptr(y), _i64(y.stride(0) if y is not None else 0), _ptr(workspace),
                ctypes.c_size_t(workspace.numel()), _stream(stream))


def bind_linear_fwd(x, wq, s_w, bias, residual, residual_scale, bits_a, bits_w, a_scale_kind, rounding, act, y, workspace,
                    stream=None):
    M, K = x.shape
    N = wq.shape[0]
    return bind("aqt_linear_fwd", _ptr(x), _i64(x.stride(0)), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
                _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N),
                _i64(K), int(bits_a), int(bits_w), int(a_scale_kind), int(rounding), int(act), _ptr(y), _i64(y.stride(0)),
                _ptr(workspace), ctypes.c_size_t(workspace.numel()), _stream(stream))


def bind_linear_fwd_weight_only(x, wq, s_w, bias, residual, residual_scale, bits_w, act, y, workspace, stream=None,
                                precision=FLOAT_TF32):
    M, K = x.shape
    N = wq.shape[0]
    return bind("aqt_linear_fwd_weight_only", _ptr(x), _i64(x.stride(0)), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
                _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N),
                _i64(K), int(bits_w), int(precision), int(act), _ptr(y), _i64(y.stride(0)), _ptr(workspace),
                ctypes.c_size_t(workspace.numel()), _stream(stream))


def aqt_version() -> int:
    return int(lib().aqt_version())


def aqt_workspace_bytes(op: int, M: int, N: int, K: int, bits_a: int, bits_w: int) -> int:
    return int(lib().aqt_workspace_bytes(int(op), _i64(M), _i64(N), _i64(K), int(bits_a), int(bits_w)))


def aqt_plan_qmatmul(M: int, N: int, K: int, bits_a: int = 8, bits_w: int = 8, act: int = ACT_NONE, float_kind: bool = False,
                     sm_count: int = 0) -> str:
    """Name of the kernel configuration the library launches for this shape (host-only)."""
    buf = ctypes.create_string_buffer(64)
    _check("aqt_plan_qmatmul", lib().aqt_plan_qmatmul(_i64(M), _i64(N), _i64(K), int(bits_a), int(bits_w), int(act),
                                                      int(bool(float_kind)), int(sm_count), buf, ctypes.c_size_t(64)))
    return buf.value.decode()


def aqt_device_status(stream=None) -> int:
    out = ctypes.c_int(0)
    _check("aqt_device_status", lib().aqt_device_status(_stream(stream), ctypes.byref(out)))
    return out.value


def aqt_selftest_bounded_wait(limit_ns: int = 1_000_000, stream=None) -> bool:
    """Runs the bounded-wait self-test; True if the wait gave up as it must.  Leaves
    AQT_ERR_TIMEOUT in the device status word for the next aqt_device_status()."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check("aqt_selftest_bounded_wait", lib().aqt_selftest_bounded_wait(ctypes.c_uint64(limit_ns), _ptr(flag), _stream(stream)))
    torch.cuda.synchronize()
    return bool(flag.item() == 1)


def aqt_selftest_sfu_rate(iterations: int = 4096, repeats: int = 3) -> float:
    """Special-function operations per second (in Gop/s) of the current device, measured with a
    kernel that runs only 2^x and reciprocal chains; best of `repeats` timed launches."""
    sink = torch.zeros(1, dtype=torch.float32, device="cuda")
    ops = ctypes.c_int64(0)
    stream = torch.cuda.current_stream()
    best = 0.0
    for i in range(repeats + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        _check("aqt_selftest_sfu_rate", lib().aqt_selftest_sfu_rate(int(iterations), _ptr(sink), ctypes.byref(ops), _stream(stream)))
        e1.record(stream)
        torch.cuda.synchronize()
        if i > 0:
            best = max(best, ops.value / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    return best


def aqt_quantize(x: torch.Tensor, bits: int, axis: int = AXIS_ROW, rounding: int = ROUND_NEAREST_EVEN,
                 pack: bool = False, q_out: Optional[torch.Tensor] = None, scale_out: Optional[torch.Tensor] = None,
                 stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Fig. 2 quantize(input, axis) on the GPU.  x: fp32 [rows, cols] (last dim contiguous)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and (x.shape[1] <= 1 or x.stride(1) == 1)
    rows, cols = x.shape
    ld = x.stride(0) if rows > 1 else max(cols, 1)
    if q_out is None:
        q_out = torch.empty((rows, cols // 2), dtype=torch.uint8, device=x.device) if pack else \
            torch.empty((rows, cols), dtype=torch.int8, device=x.device)
    n_scale = rows if axis == AXIS_ROW else (cols if axis == AXIS_COL else 1)
    if scale_out is None:
        scale_out = torch.empty(n_scale, dtype=torch.float32, device=x.device)
    _check("aqt_quantize", lib().aqt_quantize(_ptr(x), _i64(rows), _i64(cols), _i64(ld), int(bits), int(axis), int(rounding),
                                              int(bool(pack)), _ptr(q_out), _ptr(scale_out), _stream(stream)))
    return q_out, scale_out


def aqt_pack_int4(q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    assert q.is_cuda and q.dtype == torch.int8 and q.dim() == 2 and q.is_contiguous()
    rows, cols = q.shape
    if out is None:
        out = torch.empty((rows, cols // 2), dtype=torch.uint8, device=q.device)
    _check("aqt_pack_int4", lib().aqt_pack_int4(_ptr(q), _i64(rows), _i64(cols), _ptr(out), _stream(stream)))
    return out


def aqt_unpack_int4(packed: torch.Tensor, cols: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    assert packed.is_cuda and packed.dtype == torch.uint8 and packed.dim() == 2 and packed.is_contiguous()
    rows = packed.shape[0]
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.int8, device=packed.device)
    _check("aqt_unpack_int4", lib().aqt_unpack_int4(_ptr(packed), _i64(rows), _i64(cols), _ptr(out), _stream(stream)))
    return out


def _workspace(need: int, workspace: Optional[torch.Tensor], device) -> Optional[torch.Tensor]:
    if need == 0:
        return workspace
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace


def aqt_qmatmul(xq: torch.Tensor, s_x: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor,
                bias: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None, residual_scale: float = 1.0,
                *, K: int, bits_a: int = 8, bits_w: int = 8, act: int = ACT_NONE, s_x_kind: int = SCALE_ROW,
                y: Optional[torch.Tensor] = None, acc_debug: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream=None, plan: Optional[str] = None) -> torch.Tensor:
    """Integer matmul on codes + de-quantizing epilogue.  xq [M, K] int8 or [M, K/2] uint8 packed;
    wq [N, K] int8 or [N, K/2] uint8 packed.  Returns y fp32 [M, N_out].  plan: a kernel
    configuration by name (aqt_qmatmul_with_plan) instead of the library's own choice."""
    M, N = xq.shape[0], wq.shape[0]
    n_out = _n_out(N, act)
    if y is None:
        y = torch.empty((M, n_out), dtype=torch.float32, device=xq.device)
    need = aqt_workspace_bytes(OP_QMATMUL, M, N, K, bits_a, bits_w)
    workspace = _workspace(need, workspace, xq.device)
    args = (_ptr(xq), _ptr(s_x), int(s_x_kind), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
            _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K),
            int(bits_a), int(bits_w), int(act), _ptr(y), _i64(y.stride(0)), _ptr(acc_debug), _ptr(workspace),
            ctypes.c_size_t(0 if workspace is None else workspace.numel()), _stream(stream))
    if plan is None:
        _check("aqt_qmatmul", lib().aqt_qmatmul(*args))
    else:
        _check("aqt_qmatmul_with_plan", lib().aqt_qmatmul_with_plan(ctypes.c_char_p(plan.encode()), *args))
    return y


def aqt_qmatmul_requant(xq: torch.Tensor, s_x: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor,
                        bias: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None,
                        residual_scale: float = 1.0, *, K: int, bits_a: int = 8, bits_w: int = 8, act: int = ACT_NONE,
                        s_x_kind: int = SCALE_ROW, bits_out: int = 8, rounding: int = ROUND_NEAREST_EVEN, pack_out: bool = False,
                        want_y: bool = False, q_out: Optional[torch.Tensor] = None, s_out: Optional[torch.Tensor] = None,
                        y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """aqt_qmatmul whose output rows leave the kernel already quantized for the next layer.
    Returns (q_out, s_out, y); y is None unless want_y (or a residual / y tensor is given)."""
    M, N = xq.shape[0], wq.shape[0]
    n_out = _n_out(N, act)
    if q_out is None:
        q_out = torch.empty((M, n_out // 2 if pack_out else n_out), dtype=torch.uint8 if pack_out else torch.int8,
                            device=xq.device)
    if s_out is None:
        s_out = torch.empty((M,), dtype=torch.float32, device=xq.device)
    if y is None and (want_y or residual is not None):
        y = torch.empty((M, n_out), dtype=torch.float32, device=xq.device)
    need = aqt_workspace_bytes(OP_QMATMUL_REQUANT, M, N, K, bits_a, bits_w)
    workspace = _workspace(need, workspace, xq.device)
    _check("aqt_qmatmul_requant", lib().aqt_qmatmul_requant(
        _ptr(xq), _ptr(s_x), int(s_x_kind), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
        _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K),
        int(bits_a), int(bits_w), int(act), int(bits_out), int(rounding), int(bool(pack_out)), _ptr(q_out), _ptr(s_out),
        _ptr(y), _i64(y.stride(0) if y is not None else 0), _ptr(workspace),
        ctypes.c_size_t(0 if workspace is None else workspace.numel()), _stream(stream)))
    return q_out, s_out, y


def aqt_qmatmul_w4_noalloc(xq: torch.Tensor, s_x: torch.Tensor, wq_packed: torch.Tensor, s_w: torch.Tensor,
                           bias: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None,
                           residual_scale: float = 1.0, *, K: int, act: int = ACT_NONE, s_x_kind: int = SCALE_ROW,
                           y: torch.Tensor, stream=None) -> torch.Tensor:
    """aqt_qmatmul for int8 activations and packed 4-bit weights with no workspace: for callers that
    cannot allocate device memory.  The scratch is a fixed array inside the library (N*K must not
    exceed NOALLOC_MAX_WEIGHT_BYTES); calls on one device share it, so calls that overlap on the
    GPU race.  The output tensor `y` must be supplied by the caller: this wrapper allocates nothing."""
    M, N = xq.shape[0], wq_packed.shape[0]
    _check("aqt_qmatmul_w4_noalloc", lib().aqt_qmatmul_w4_noalloc(
        _ptr(xq), _ptr(s_x), int(s_x_kind), _ptr(wq_packed), _ptr(s_w), _ptr(bias), _ptr(residual),
        _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K),
        int(act), _ptr(y), _i64(y.stride(0)), _stream(stream)))
    return y


def aqt_linear_fwd(x: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                   residual: Optional[torch.Tensor] = None, residual_scale: float = 1.0, *, bits_a: int = 8,
                   bits_w: int = 8, a_scale_kind: int = SCALE_ROW, rounding: int = ROUND_NEAREST_EVEN,
                   act: int = ACT_NONE, y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   stream=None) -> torch.Tensor:
    """The whole layer: dynamic activation quantization, integer matmul, epilogue.  x fp32 [M, K]."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    N = wq.shape[0]
    n_out = _n_out(N, act)
    if y is None:
        y = torch.empty((M, n_out), dtype=torch.float32, device=x.device)
    need = aqt_workspace_bytes(OP_LINEAR_FWD, M, N, K, bits_a, bits_w)
    workspace = _workspace(need, workspace, x.device)
    _check("aqt_linear_fwd", lib().aqt_linear_fwd(
        _ptr(x), _i64(x.stride(0)), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
        _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K),
        int(bits_a), int(bits_w), int(a_scale_kind), int(rounding), int(act), _ptr(y), _i64(y.stride(0)), _ptr(workspace),
        ctypes.c_size_t(workspace.numel()), _stream(stream)))
    return y


def aqt_linear_fwd_weight_only(x: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor, bias: Optional[torch.Tensor] = None,
                               residual: Optional[torch.Tensor] = None, residual_scale: float = 1.0, *, bits_w: int = 8,
                               precision: int = FLOAT_TF32, act: int = ACT_NONE, y: Optional[torch.Tensor] = None,
                               workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """The weight-only layer (int8 / int4 weights, float activations): x fp32 [M, K] against the
    codes wq [N, K] int8 or [N, K/2] uint8 packed, de-quantized by s_w after the float matmul."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    N = wq.shape[0]
    if y is None:
        y = torch.empty((M, _n_out(N, act)), dtype=torch.float32, device=x.device)
    need = aqt_workspace_bytes(OP_LINEAR_WEIGHT_ONLY_X2 if precision == FLOAT_TF32X2 else OP_LINEAR_WEIGHT_ONLY, M, N, K, 0, bits_w)
    workspace = _workspace(need, workspace, x.device)
    _check("aqt_linear_fwd_weight_only", lib().aqt_linear_fwd_weight_only(
        _ptr(x), _i64(x.stride(0)), _ptr(wq), _ptr(s_w), _ptr(bias), _ptr(residual),
        _i64(residual.stride(0) if residual is not None else 0), ctypes.c_float(residual_scale), _i64(M), _i64(N), _i64(K),
        int(bits_w), int(precision), int(act), _ptr(y), _i64(y.stride(0)), _ptr(workspace), ctypes.c_size_t(workspace.numel()),
        _stream(stream)))
    return y


def aqt_linear_bwd(dy: torch.Tensor, xq: Optional[torch.Tensor], s_x: Optional[torch.Tensor], wq: Optional[torch.Tensor],
                   s_w: Optional[torch.Tensor], *, K: int, bits_a: int = 8, bits_w: int = 8, s_x_kind: int = SCALE_ROW,
                   want_dx: bool = True, want_dw: bool = True, want_dbias: bool = True,
                   workspace: Optional[torch.Tensor] = None, stream=None):
    """Straight-through backward of the quantized linear layer: returns (dx [M, K], dw [N, K],
    dbias [N]), None for the ones not wanted.  dy fp32 [M, N]; codes and scales as in the forward."""
    assert dy.is_cuda and dy.dtype == torch.float32 and dy.dim() == 2 and dy.stride(1) == 1
    M, N = dy.shape
    f32 = dict(dtype=torch.float32, device=dy.device)
    dx = torch.empty((M, K), **f32) if want_dx else None
    dw = torch.empty((N, K), **f32) if want_dw else None
    db = torch.empty((N,), **f32) if want_dbias else None
    need = aqt_workspace_bytes(OP_LINEAR_BWD, M, N, K, 0, 0)
    workspace = _workspace(need, workspace, dy.device)
    _check("aqt_linear_bwd", lib().aqt_linear_bwd(
        _ptr(dy), _i64(dy.stride(0)), _ptr(xq), _ptr(s_x), int(s_x_kind), int(bits_a), _ptr(wq), _ptr(s_w), int(bits_w),
        _i64(M), _i64(N), _i64(K), _ptr(dx), _i64(K), _ptr(dw), _i64(K), _ptr(db), _ptr(workspace),
        ctypes.c_size_t(0 if workspace is None else workspace.numel()), _stream(stream)))
    return dx, dw, db


def linear_fwd_host_workspace_bytes(M: int, N: int, K: int, bits_a: int, bits_w: int, act: int,
                                    x_on_host: bool = True, y_on_host: bool = True) -> int:
    r256 = lambda v: (v + 255) // 256 * 256
    need = r256(aqt_workspace_bytes(OP_LINEAR_FWD, M, N, K, bits_a, bits_w))
    if x_on_host:
        need += r256(4 * M * K)
    if y_on_host:
        need += r256(4 * M * _n_out(N, act))
    return need


def aqt_linear_fwd_host(x: torch.Tensor, wq: torch.Tensor, s_w: torch.Tensor, bias: Optional[torch.Tensor],
                        y: torch.Tensor, workspace: torch.Tensor, *, bits_a: int = 8, bits_w: int = 8,
                        a_scale_kind: int = SCALE_ROW, rounding: int = ROUND_NEAREST_EVEN, act: int = ACT_NONE,
                        stream=None) -> torch.Tensor:
    """aqt_linear_fwd with x and/or y in (pinned) host memory; copies are enqueued on the stream.
    Whether a tensor is on the host is read from the tensor itself."""
    assert x.is_contiguous() and y.is_contiguous() and x.dtype == torch.float32 and y.dtype == torch.float32
    M, K = x.shape
    N = wq.shape[0]
    _check("aqt_linear_fwd_host", lib().aqt_linear_fwd_host(
        _ptr(x), int(not x.is_cuda), _ptr(wq), _ptr(s_w), _ptr(bias), _i64(M), _i64(N), _i64(K), int(bits_a), int(bits_w),
        int(a_scale_kind), int(rounding), int(act), _ptr(y), int(not y.is_cuda), _ptr(workspace),
        ctypes.c_size_t(workspace.numel()), _stream(stream)))
    return y


def bind_ffn_fwd(x, w1q, s_w1, bits_w1, w2q, s_w2, bits_w2, y, workspace, *, bits_a=8, rounding=ROUND_NEAREST_EVEN, act=ACT_SWISH,
                 stream=None):
    """Pre-marshalled aqt_ffn_fwd (see bind): x, y fp32 [M, d] on the host (pinned) or the device."""
    M, d = x.shape
    ff = w1q.shape[0]
    return bind("aqt_ffn_fwd", _ptr(x), int(not x.is_cuda), _ptr(w1q), _ptr(s_w1), _ptr(None), int(bits_w1), _ptr(w2q), _ptr(s_w2),
                _ptr(None), int(bits_w2), _i64(M), _i64(d), _i64(ff), int(bits_a), int(rounding), int(act), _ptr(y), int(not y.is_cuda),
                _ptr(workspace), ctypes.c_size_t(workspace.numel()), _stream(stream))


def aqt_ffn_fwd(x, w1q, s_w1, bits_w1, w2q, s_w2, bits_w2, y, workspace=None, **kw):
    """y = W2 . act(W1 . x) through two quantized layers (aqt_ffn_fwd); x / y may be pinned host tensors."""
    M, d = x.shape
    ff = w1q.shape[0]
    if workspace is None:
        workspace = torch.empty(aqt_workspace_bytes(OP_FFN_FWD, M, ff, d, kw.get("bits_a", 8), 4), dtype=torch.uint8,
                                device=w1q.device)
    bind_ffn_fwd(x, w1q, s_w1, bits_w1, w2q, s_w2, bits_w2, y, workspace, **kw)()
    return y
