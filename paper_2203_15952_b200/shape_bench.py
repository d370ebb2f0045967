"""Time one entry point of the library on one shape (CUDA events, rotating buffers).

    python -m paper_2203_15952_b200.shape_bench qmatmul M N K [--act 0..3] [--bits-w 4|8] [--residual]
                                                 [--iters I] [--sustain SECONDS]
    python -m paper_2203_15952_b200.shape_bench requant M N K [--act 0|1] [--bits-w 4|8] [--bits 4|8] [--with-y] [--residual]
    python -m paper_2203_15952_b200.shape_bench quantize M K [--bits 4|8]
    python -m paper_2203_15952_b200.shape_bench linear M N K [--act ..] [--bits-w ..] [--bits 4|8] [--per-tensor]
    python -m paper_2203_15952_b200.shape_bench wonly M N K [--act ..] [--bits-w 4|8] [--residual] [--x2]
    python -m paper_2203_15952_b200.shape_bench bwd M N K [--bits-w 4|8]

Inputs are random codes / normals drawn on the GPU (seeded); several buffer sets are rotated so
that consecutive launches do not find their inputs in L2.  With --sustain the call is repeated for
that many seconds while nvidia-smi samples clocks and power (power-capped throughput).
Prints one line: time per call, TOPS or GB/s (algorithmic bytes), and with --sustain the clocks.
"""
from __future__ import annotations

import argparse
import statistics
import subprocess
import sys
import time

import torch

from . import binding as aqt


def _time(calls, iters):
    for c in calls:
        c()
    for c in calls:
        c()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        calls[i % len(calls)]()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3  # us


def _time_graph(make_calls, iters):
    """The same calls captured in a CUDA graph (no host launch cost between kernels)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        calls = make_calls(side)
        for c in calls:
            c()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for i in range(iters):
            calls[i % len(calls)]()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def _sustain(calls, seconds):
    q = "clocks.sm,power.draw,clocks_event_reasons.sw_power_cap"
    proc = subprocess.Popen(["nvidia-smi", "-i", str(torch.cuda.current_device()), "--query-gpu=" + q, "--format=csv,noheader,nounits",
                             "-lms", "100"], stdout=subprocess.PIPE, text=True)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n, t0 = 0, time.time()
    e0.record()
    while time.time() - t0 < seconds:
        for _ in range(50):
            calls[n % len(calls)]()
            n += 1
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    proc.terminate()
    out, _ = proc.communicate()
    rows = [l.split(",") for l in out.strip().splitlines()][3:]
    clk = [float(r[0]) for r in rows] or [float("nan")]
    pw = [float(r[1]) for r in rows] or [float("nan")]
    capped = sum(("Active" in r[2]) and ("Not" not in r[2]) for r in rows)
    return e0.elapsed_time(e1) / n * 1e3, " sustained %.1f s: SM clock median %.0f MHz, power max %.0f W, power cap active in %d/%d samples" % (
        seconds, statistics.median(clk), max(pw), capped, len(rows))


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("op", choices=["qmatmul", "requant", "quantize", "linear", "wonly", "bwd"])
    ap.add_argument("dims", type=int, nargs="+")
    ap.add_argument("--act", type=int, default=0)
    ap.add_argument("--bits-w", type=int, default=8)
    ap.add_argument("--bits", type=int, default=8)
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--with-y", action="store_true", help="requant: also write the fp32 output")
    ap.add_argument("--per-tensor", action="store_true", help="linear: one activation scale for the whole tensor")
    ap.add_argument("--x2", action="store_true", help="wonly: two-term (hi + lo) form of the float activations")
    ap.add_argument("--iters", type=int, default=30)
    ap.add_argument("--sets", type=int, default=4)
    ap.add_argument("--sustain", type=float, default=0.0)
    ap.add_argument("--graph", action="store_true", help="replay the calls from a CUDA graph (kernel time without host launch cost)")
    a = ap.parse_args(argv)
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(0)
    keep = []
    if a.op == "qmatmul":
        M, N, K = a.dims
        n_out = N // 2 if a.act >= 2 else N
        wq = torch.randint(-7, 8, (N, K if a.bits_w == 8 else K // 2), generator=g, dtype=torch.int8, device=dev)
        if a.bits_w == 4:
            wq = wq.view(torch.uint8)
        sw = torch.rand(N, generator=g, device=dev) * 1e-3
        ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_QMATMUL, M, N, K, 8, a.bits_w) + 256, dtype=torch.uint8, device=dev)
        sets = []
        for _ in range(a.sets):
            xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8, device=dev)
            sx = torch.rand(M, generator=g, device=dev) * 1e-2
            y = torch.empty((M, n_out), dtype=torch.float32, device=dev)
            rr = torch.randn((M, n_out), generator=g, device=dev) if a.residual else None
            sets.append((xq, sx, y, rr))

        def make_calls(stream=None):
            return [aqt.bind_qmatmul(xq, sx, wq, sw, None, rr, 0.5, K, 8, a.bits_w, a.act, aqt.SCALE_ROW, y, ws, stream)
                    for (xq, sx, y, rr) in sets]
        ops = 2.0 * M * N * K
        nbytes = M * K + N * K * a.bits_w // 8 + 8 * N + 4 * M + 4 * M * n_out * (2 if a.residual else 1)
        label = "qmatmul M%d N%d K%d act%d w%d res%d" % (M, N, K, a.act, a.bits_w, int(a.residual))
    elif a.op == "requant":
        # matmul whose epilogue quantizes the output rows (--bits: width of the output codes)
        M, N, K = a.dims
        wq = torch.randint(-7, 8, (N, K if a.bits_w == 8 else K // 2), generator=g, dtype=torch.int8, device=dev)
        if a.bits_w == 4:
            wq = wq.view(torch.uint8)
        sw = torch.rand(N, generator=g, device=dev) * 1e-3
        ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_QMATMUL_REQUANT, M, N, K, 8, a.bits_w) + 256, dtype=torch.uint8, device=dev)
        pack = a.bits == 4
        sets = []
        for _ in range(a.sets):
            xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8, device=dev)
            sx = torch.rand(M, generator=g, device=dev) * 1e-2
            q = torch.empty((M, N // 2 if pack else N), dtype=torch.uint8 if pack else torch.int8, device=dev)
            so = torch.empty(M, device=dev)
            y = torch.empty((M, N), dtype=torch.float32, device=dev) if (a.with_y or a.residual) else None
            rr = torch.randn((M, N), generator=g, device=dev) if a.residual else None
            sets.append((xq, sx, q, so, y, rr))

        def make_calls(stream=None):
            return [aqt.bind_qmatmul_requant(xq, sx, wq, sw, None, rr, 0.5, K, 8, a.bits_w, a.act, aqt.SCALE_ROW, a.bits,
                                             aqt.ROUND_NEAREST_EVEN, pack, q, so, y, ws, stream)
                    for (xq, sx, q, so, y, rr) in sets]
        ops = 2.0 * M * N * K
        nbytes = (M * K + N * K * a.bits_w // 8 + 8 * N + 8 * M + M * N * a.bits // 8
                  + 4 * M * N * ((1 if (a.with_y or a.residual) else 0) + (1 if a.residual else 0)))
        label = "requant M%d N%d K%d act%d w%d out%d y%d res%d" % (M, N, K, a.act, a.bits_w, a.bits, int(a.with_y or a.residual), int(a.residual))
    elif a.op == "linear":
        M, N, K = a.dims
        n_out = N // 2 if a.act >= 2 else N
        wq = torch.randint(-7, 8, (N, K if a.bits_w == 8 else K // 2), generator=g, dtype=torch.int8, device=dev)
        if a.bits_w == 4:
            wq = wq.view(torch.uint8)
        sw = torch.rand(N, generator=g, device=dev) * 1e-3
        ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_FWD, M, N, K, a.bits, a.bits_w) + 256, dtype=torch.uint8, device=dev)
        kind = aqt.SCALE_TENSOR if a.per_tensor else aqt.SCALE_ROW
        sets = [(torch.randn((M, K), generator=g, device=dev), torch.empty((M, n_out), dtype=torch.float32, device=dev))
                for _ in range(a.sets)]

        def make_calls(stream=None):
            return [aqt.bind_linear_fwd(x, wq, sw, None, None, 1.0, a.bits, a.bits_w, kind, aqt.ROUND_NEAREST_EVEN, a.act, y, ws, stream)
                    for (x, y) in sets]
        ops = 2.0 * M * N * K
        nbytes = 4 * M * K + N * K * a.bits_w // 8 + 8 * N + 4 * M * n_out
        label = "linear M%d N%d K%d act%d a%d w%d %s" % (M, N, K, a.act, a.bits, a.bits_w, "per-tensor" if a.per_tensor else "per-row")
    elif a.op == "bwd":
        # straight-through backward: dx, dw and dbias of one layer from dy and the forward's codes
        import ctypes
        M, N, K = a.dims
        wq = torch.randint(-7, 8, (N, K if a.bits_w == 8 else K // 2), generator=g, dtype=torch.int8, device=dev)
        if a.bits_w == 4:
            wq = wq.view(torch.uint8)
        sw = torch.rand(N, generator=g, device=dev) * 1e-3
        xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8, device=dev)
        sx = torch.rand(M, generator=g, device=dev) * 1e-2
        ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_BWD, M, N, K, 0, 0) + 256, dtype=torch.uint8, device=dev)
        sets = [(torch.randn((M, N), generator=g, device=dev), torch.empty((M, K), device=dev), torch.empty((N, K), device=dev),
                 torch.empty(N, device=dev)) for _ in range(a.sets)]

        def make_calls(stream=None):
            return [aqt.bind("aqt_linear_bwd", aqt._ptr(dy), aqt._i64(N), aqt._ptr(xq), aqt._ptr(sx), aqt.SCALE_ROW, 8, aqt._ptr(wq),
                             aqt._ptr(sw), int(a.bits_w), aqt._i64(M), aqt._i64(N), aqt._i64(K), aqt._ptr(dx), aqt._i64(K), aqt._ptr(dw),
                             aqt._i64(K), aqt._ptr(db), aqt._ptr(ws), ctypes.c_size_t(ws.numel()), aqt._stream(stream))
                    for (dy, dx, dw, db) in sets]
        ops = 4.0 * M * N * K
        nbytes = 4 * M * N + M * K + N * K * a.bits_w // 8 + 4 * M * K + 4 * N * K + 4 * (M + 2 * N)
        label = "bwd M%d N%d K%d w%d" % (M, N, K, a.bits_w)
    elif a.op == "wonly":
        # weight-only layer: fp32 activations against integer weights (float matmul, tf32 operands)
        M, N, K = a.dims
        n_out = N // 2 if a.act >= 2 else N
        wq = torch.randint(-7, 8, (N, K if a.bits_w == 8 else K // 2), generator=g, dtype=torch.int8, device=dev)
        if a.bits_w == 4:
            wq = wq.view(torch.uint8)
        sw = torch.rand(N, generator=g, device=dev) * 1e-3
        prec = aqt.FLOAT_TF32X2 if a.x2 else aqt.FLOAT_TF32
        ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_WEIGHT_ONLY_X2 if a.x2 else aqt.OP_LINEAR_WEIGHT_ONLY, M, N, K, 0, a.bits_w) + 256,
                         dtype=torch.uint8, device=dev)
        sets = []
        for _ in range(a.sets):
            x = torch.randn((M, K), generator=g, device=dev)
            y = torch.empty((M, n_out), dtype=torch.float32, device=dev)
            rr = torch.randn((M, n_out), generator=g, device=dev) if a.residual else None
            sets.append((x, y, rr))

        def make_calls(stream=None):
            return [aqt.bind_linear_fwd_weight_only(x, wq, sw, None, rr, 0.5, a.bits_w, a.act, y, ws, stream, precision=prec)
                    for (x, y, rr) in sets]
        ops = 2.0 * M * N * K
        nbytes = 4 * M * K + N * K * a.bits_w // 8 + 8 * N + 4 * M * n_out * (2 if a.residual else 1)
        label = "wonly%s M%d N%d K%d act%d w%d res%d" % ("-x2" if a.x2 else "", M, N, K, a.act, a.bits_w, int(a.residual))
    else:
        M, K = a.dims
        sets = []
        for _ in range(a.sets):
            x = torch.randn((M, K), generator=g, device=dev)
            q = torch.empty((M, K), dtype=torch.int8, device=dev)
            s = torch.empty(M, device=dev)
            sets.append((x, q, s))

        def make_calls(stream=None):
            return [aqt.bind_quantize(x, a.bits, aqt.AXIS_ROW, aqt.ROUND_NEAREST_EVEN, False, q, s, stream) for (x, q, s) in sets]
        ops = 0.0
        nbytes = 5 * M * K + 4 * M
        label = "quantize M%d K%d bits%d" % (M, K, a.bits)
    calls = make_calls()
    extra = ""
    if a.sustain > 0:
        t, extra = _sustain(calls, a.sustain)
    elif a.graph:
        t = _time_graph(make_calls, a.iters)
        extra = " (graph replay)"
    else:
        t = _time(calls, a.iters)
    if aqt.aqt_device_status() != 0:
        raise SystemExit("device status reports a failed wait")
    print("%s: %8.2f us  %8.1f TOPS  %7.1f GB/s%s" % (label, t, ops / t / 1e6, nbytes / t / 1e3, extra), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
