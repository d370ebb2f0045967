"""The C-ABI library builds, loads without a GPU, and exports every symbol include/aqt.h declares."""
import ctypes
import os
import re

import pytest

from paper_2203_15952_b200 import build as aqt_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "aqt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aqt_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_named_calls():
    names = _declared_symbols()
    for required in ("aqt_quantize", "aqt_pack_int4", "aqt_unpack_int4", "aqt_qmatmul", "aqt_linear_fwd",
                     "aqt_workspace_bytes", "aqt_version", "aqt_status_string"):
        assert required in names


def test_library_exports_every_declared_symbol():
    path = aqt_build.build()
    L = ctypes.CDLL(path)
    for name in _declared_symbols():
        assert hasattr(L, name), name
    from paper_2203_15952_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_symbols()


def test_host_only_calls():
    from paper_2203_15952_b200 import binding as b
    assert b.aqt_version() >= 100
    assert b.status_string(0) == "ok" and "workspace" in b.status_string(-4)
    # 4-bit operands need a sign-extended copy; 8-bit ones do not
    assert b.aqt_workspace_bytes(b.OP_QMATMUL, 128, 256, 512, 8, 8) == 0
    assert b.aqt_workspace_bytes(b.OP_QMATMUL, 128, 256, 512, 8, 4) == 256 * 512
    assert b.aqt_workspace_bytes(b.OP_QMATMUL, 128, 256, 512, 4, 4) == 128 * 512 + 256 * 512
    assert b.aqt_workspace_bytes(b.OP_LINEAR_FWD, 100, 256, 512, 8, 8) == 100 * 512 + 512
    assert b.aqt_workspace_bytes(99, 1, 1, 1, 8, 8) == 0


def test_argument_errors_are_reported_before_any_cuda_call():
    """Bad arguments return a status synchronously; no device is touched (none exists here)."""
    L = ctypes.CDLL(aqt_build.build())
    i64, vp = ctypes.c_int64, ctypes.c_void_p
    one = vp(16)
    # quantize: unknown bit width, pack with 8 bits, odd cols for packing, ld < cols
    assert L.aqt_quantize(one, i64(4), i64(8), i64(8), 5, 0, 1, 0, one, one, None) == -1
    assert L.aqt_quantize(one, i64(4), i64(8), i64(8), 8, 0, 1, 1, one, one, None) == -1
    assert L.aqt_quantize(one, i64(4), i64(7), i64(7), 4, 0, 1, 1, one, one, None) == -1
    assert L.aqt_quantize(one, i64(4), i64(8), i64(4), 8, 0, 1, 0, one, one, None) == -1
    assert L.aqt_quantize(one, i64(4), i64(8), i64(8), 8, 3, 1, 0, one, one, None) == -1
    assert L.aqt_quantize(one, i64(0), i64(8), i64(8), 8, 0, 1, 0, one, one, None) == 0      # empty: no-op
    assert L.aqt_pack_int4(one, i64(2), i64(3), one, None) == -1
    assert L.aqt_unpack_int4(one, i64(2), i64(3), one, None) == -1
    f = ctypes.c_float(1.0)

    def mm(M, N, K, ba, bw, act, xq=one, ldy=None, ws=None, wsb=0, kind=0):
        ldy = N if ldy is None else ldy
        return L.aqt_qmatmul(xq, one, kind, one, one, None, None, i64(0), f, i64(M), i64(N), i64(K), ba, bw, act, one,
                             i64(ldy), None, ws, ctypes.c_size_t(wsb), None)
    assert mm(128, 256, 100, 8, 8, 0) == -1          # K not a multiple of 16
    assert mm(128, 250, 128, 8, 8, 0) == -1          # N not a multiple of 4
    assert mm(128, 260, 128, 8, 8, 2) == -1          # GLU needs N % 8 == 0
    assert mm(128, 256, 128, 3, 8, 0) == -1
    assert mm(128, 256, 128, 8, 8, 7) == -1
    assert mm(128, 256, 128, 8, 8, 0, kind=5) == -1
    assert mm(0, 256, 128, 8, 8, 0) == 0             # empty: no-op
    assert mm(128, 256, 128, 8, 8, 0, xq=vp(8)) == -2     # misaligned codes
    assert mm(128, 256, 128, 8, 8, 0, ldy=258) == -2      # pitch not a multiple of 4 floats
    assert mm(128, 256, 128, 8, 8, 0, ldy=128) == -1      # pitch smaller than the row
    assert mm(128, 256, 128, 8, 4, 0) == -4               # int4 weights need workspace
    assert mm(128, 256, 128, 8, 4, 0, ws=vp(256), wsb=100) == -4
    assert mm(1 << 31, 256, 128, 8, 8, 0) == -3


def test_argument_errors_of_the_float_entry_points_need_no_device():
    """The weight-only layer and the backward report bad arguments before any CUDA call too."""
    L = ctypes.CDLL(aqt_build.build())
    i64, vp, f = ctypes.c_int64, ctypes.c_void_p, ctypes.c_float(1.0)
    one = vp(256)

    def wo(M, N, K, bits_w=8, prec=0, act=0, ldx=None, ws=one, wsb=1 << 40):
        return L.aqt_linear_fwd_weight_only(one, i64(K if ldx is None else ldx), one, one, None, None, i64(0), f, i64(M), i64(N), i64(K),
                                            bits_w, prec, act, one, i64(N), ws, ctypes.c_size_t(wsb), None)
    assert wo(128, 256, 130) == -1 and wo(128, 250, 128) == -1 and wo(128, 256, 128, bits_w=3) == -1
    assert wo(128, 256, 128, prec=7) == -1 and wo(128, 256, 128, act=9) == -1
    assert wo(128, 256, 128, ldx=130) == -2 and wo(128, 256, 128, ws=None) == -4 and wo(0, 256, 128) == 0

    def bwd(M, N, K, kind=0, lddy=None, ws=one, wsb=1 << 40, xq=one):
        return L.aqt_linear_bwd(one, i64(N if lddy is None else lddy), xq, one, kind, 8, one, one, 4, i64(M), i64(N), i64(K), one, i64(K),
                                one, i64(K), None, ws, ctypes.c_size_t(wsb), None)
    assert bwd(128, 256, 130) == -1 and bwd(128, 250, 128) == -1 and bwd(128, 256, 128, kind=2) == -1
    assert bwd(128, 256, 128, lddy=258) == -2 and bwd(128, 256, 128, xq=None) == -1
    assert bwd(128, 256, 128, ws=None) == -4 and bwd(128, 256, 128, wsb=10) == -4 and bwd(0, 256, 128) == 0
    L.aqt_workspace_bytes.restype = ctypes.c_size_t
    assert L.aqt_workspace_bytes(4, i64(128), i64(256), i64(128), 0, 4) == 4 * 256 * 128
    assert L.aqt_workspace_bytes(5, i64(128), i64(256), i64(128), 0, 4) == 8 * 256 * 128 + 8 * 128 * 128
    assert L.aqt_workspace_bytes(6, i64(12800), i64(2048), i64(512), 0, 0) > 4 * (512 * 2048 + (2048 + 512) * 12800)


def test_plan_query_and_new_entry_points_reject_bad_arguments():
    """The plan query is host-only; the entry points added beside the named calls validate like them."""
    import ctypes
    from paper_2203_15952_b200 import binding as b
    L = ctypes.CDLL(aqt_build.build())
    i64, vp = ctypes.c_int64, ctypes.c_void_p
    one = vp(256)
    buf = ctypes.create_string_buffer(64)
    assert L.aqt_plan_qmatmul(i64(1000), i64(512), i64(512), 8, 4, 0, 0, 148, buf, ctypes.c_size_t(64)) == 0 and buf.value == b"ws128e16"
    assert L.aqt_plan_qmatmul(i64(1000), i64(512), i64(512), 8, 4, 0, 0, 148, buf, ctypes.c_size_t(4)) == -1      # name does not fit
    assert L.aqt_plan_qmatmul(i64(0), i64(512), i64(512), 8, 4, 0, 0, 148, buf, ctypes.c_size_t(64)) == -1
    assert L.aqt_plan_qmatmul(i64(8), i64(512), i64(512), 8, 5, 0, 0, 148, buf, ctypes.c_size_t(64)) == -1         # unknown width
    assert b.aqt_plan_qmatmul(8, 512, 512, 8, b.BITS_4_UNPACKED) == "small_m"
    # a named plan that does not exist; the 4-bit-in-container width and the static-weights flag pass validation
    f = ctypes.c_float(1.0)
    args = (one, one, 0, one, one, None, None, i64(0), f, i64(256), i64(256), i64(256), 8, b.BITS_4_UNPACKED | b.STATIC_WEIGHTS, 0, one,
            i64(256), None, None, ctypes.c_size_t(0), None)
    assert L.aqt_qmatmul_with_plan(ctypes.c_char_p(b"no_such_plan"), *args) == -1
    bad = list(args); bad[13] = 5
    assert L.aqt_qmatmul(*bad) == -1
    # aqt_ffn_fwd: activation other than none / Swish, missing workspace
    ffn = lambda act, ws, wsb: L.aqt_ffn_fwd(one, 0, one, one, None, 4, one, one, None, 4, i64(256), i64(512), i64(2048), 8, 1, act, one, 0,
                                             ws, ctypes.c_size_t(wsb), None)
    assert ffn(2, one, 1 << 30) == -1
    assert ffn(1, None, 0) == -4
    assert b.aqt_workspace_bytes(b.OP_FFN_FWD, 256, 2048, 512, 8, 4) > 2 * 4 * 256 * 512 + 256 * 2048
    ops = ctypes.c_int64(0)
    assert L.aqt_selftest_sfu_rate(0, one, ctypes.byref(ops), None) == -1
