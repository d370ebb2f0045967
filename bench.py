#!/usr/bin/env python
"""Benchmark of the quantized linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 \
        --master-port P bench.py --gpus N --steps K --warmup W

Workload: the Conformer feed-forward pair (d_model 512 -> 2048 Swish -> 512, batch 32 x 400
frames, int4 per-channel weights, int8 per-row dynamic activations), synthetic seeded inputs.
One step = one pass of the whole path over one batch:
    quantize(x) -> integer GEMM + de-quantize + Swish -> quantize(u) -> integer GEMM + de-quantize.
Prints ONE JSON line (rank 0).  With N > 1 every rank runs the same batch size on its own GPU
(rows are independent under per-row scales, so the path shards with no collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "quantized Conformer linear TOPS (int4 weights, int8 activations)"
UNIT = "TOPS"
CFG = 2  # the Conformer FFN pair; fits one GPU many times over
NCU_CAPTURE_VERSION = 201  # library version the ncu traffic figures below were captured at
# call index -> DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the
# ncu summaries under profiles/ (qgemm_requant_ffn1_ncu.md, qgemm_i8_ffn2_ncu.md); the quantizer of the
# 12 800 x 512 input has no capture of its own (its 33 MB stay inside L2 under the profiler)
NCU_TRAFFIC = {1: 7704320 + 2560, 2: 27355904 + 73984}
INT8_NOMINAL_TOPS = 4500.0  # dense int8 tensor peak of the part, nominal


def _peaks():
    """Measured denominators (HBM copy GB/s, bf16 TFLOP/s burst and sustained) and where they come from."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "kind": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "kind": "fallback"}


def _capture(fn, stream_ctx_torch, warm: int = 1):
    """Run fn() on a side stream once (warm-up), then capture it into a CUDA graph."""
    torch = stream_ctx_torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(warm):
            fn(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        fn(side)
    return graph


def _time_replays(torch, graph, replays: int, min_seconds: float = 0.0, warm: int = 2):
    """Milliseconds per replay (CUDA events on the current stream); at least `replays` replays
    and at least `min_seconds` of them.  Returns (ms_per_replay, replays_done)."""
    stream = torch.cuda.current_stream()
    for _ in range(warm):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    done = 0
    e0.record(stream)
    t0 = time.perf_counter()
    while True:
        for _ in range(replays):
            graph.replay()
        done += replays
        if min_seconds <= 0.0:
            break
        torch.cuda.synchronize()          # only the sustained runs look at the wall clock
        if time.perf_counter() - t0 >= min_seconds:
            break
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / done, done


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc, self.gpu = None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        for line in out.strip().splitlines():
            f = [v.strip() for v in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power), "samples": len(sm),
                "reasons": sorted(reasons)}


def _dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores

def _oracle_weights(w, specs):
    from oracle import conformer_ref as ref
    from paper_2203_15952_b200 import inputs as gen
    out = []
    for i, s in enumerate(specs):
        wq, sw = ref.prepare_weight(gen.layer_weight(w, 0, i, s), s.bits_w)
        out.append((wq, sw, gen.layer_bias(w, 0, i, s)))
    return out


def _oracle_time_rows(w, specs, wts, rows: int, offset: int = 0) -> float:
    """Seconds the oracle takes for the whole path on `rows` rows of the workload."""
    from oracle import conformer_ref as ref
    from paper_2203_15952_b200 import inputs as gen
    sel = [(offset + i) % w.M for i in range(rows)]
    x = gen.workload_input(w, row_subset=sel)
    t0 = time.perf_counter()
    ref.ffn_pair(specs, wts, x)
    return time.perf_counter() - t0


def cpu_baseline(budget_s: float = 15.0):
    """Oracle throughput on a bounded row sample (rows are independent under per-row scales, so
    rows / time is the oracle's rate for this path, not an extrapolation of other work)."""
    import oracle as orc
    from paper_2203_15952_b200 import inputs as gen
    w = gen.WORKLOADS[CFG]
    specs = gen.workload_layers(w)
    wts = _oracle_weights(w, specs)
    probe_rows = 128
    t_probe = _oracle_time_rows(w, specs, wts, probe_rows)
    # 10-30 s of CPU work: as many rows as the budget allows, in passes of at most M rows
    rows_total = int(max(probe_rows, probe_rows * budget_s / max(t_probe, 1e-6))) // 64 * 64
    rows, t, off = 0, 0.0, probe_rows
    while rows < rows_total and t < 2 * budget_s:
        n = min(w.M, rows_total - rows)
        t += _oracle_time_rows(w, specs, wts, n, offset=off)
        rows += n
        off += n
    ops_per_row = sum(2 * s.N * s.K for s in specs)
    return {"value": rows * ops_per_row / t / 1e12, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": "%d rows (batch of %d, rows cycled) of the FFN pair, whole path (quantize, int matmul, epilogue, twice), %.1f s" % (rows, w.M, t),
            "frames_per_s": rows / t}


def run_reference(args):
    rank, world, _ = _dist_env()
    if rank != 0:
        return 0
    import oracle as orc
    from paper_2203_15952_b200 import inputs as gen
    w = gen.WORKLOADS[CFG]
    specs = gen.workload_layers(w)
    wts = _oracle_weights(w, specs)
    ops_per_row = sum(2 * s.N * s.K for s in specs)
    t_probe = _oracle_time_rows(w, specs, wts, 128)
    # a step = a row sample sized so that warm-up + steps finish within about two minutes
    per_step_budget = args.ref_budget_s / max(1, args.steps + args.warmup)
    rows = int(max(64, min(w.M, 128 * per_step_budget / max(t_probe, 1e-6)))) // 64 * 64
    for i in range(args.warmup):
        _oracle_time_rows(w, specs, wts, rows, offset=i * rows)
    t = 0.0
    for i in range(args.steps):
        t += _oracle_time_rows(w, specs, wts, rows, offset=(args.warmup + i) * rows)
    value = args.steps * rows * ops_per_row / t / 1e12
    sample = "%d of %d rows per step, whole FFN-pair path on the CPU oracle" % (rows, w.M)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": w.name, "rows_per_step": rows, "note": "CPU oracle on host cores; bounded row sample"},
            "frames_per_s": args.steps * rows / t,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------------
# our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2203_15952_b200 import binding as aqt
    from paper_2203_15952_b200 import inputs as gen
    from paper_2203_15952_b200.encoder import QuantLinear

    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = gen.WORKLOADS[CFG]
    specs = gen.workload_layers(w)
    M = w.M
    # every rank works on its own batch of M rows (seeded by rank): weak scaling, no collective
    seed = rank
    layers = []
    for i, s in enumerate(specs):
        wt = torch.from_numpy(gen.layer_weight(w, 0, i, s, seed=0)).to(dev)
        layers.append(QuantLinear.from_float(s, wt))   # packed int4; W2 (K = 2048) also kept sign-extended, once
    R = 6  # rotating input/output sets: the six x and six y tensors (315 MB) exceed the 126 MB L2
    x_host = gen.workload_input(w, seed=seed)
    xs = [torch.from_numpy(x_host).to(dev) for _ in range(R)]
    ys = [torch.empty((M, specs[1].N), dtype=torch.float32, device=dev) for _ in range(R)]
    q1 = torch.empty((M, specs[0].K), dtype=torch.int8, device=dev)
    q2 = torch.empty((M, specs[1].K), dtype=torch.int8, device=dev)
    s1 = torch.empty(M, dtype=torch.float32, device=dev)
    s2 = torch.empty(M, dtype=torch.float32, device=dev)
    ws = torch.empty(max(max(aqt.aqt_workspace_bytes(op, M, s.N, s.K, s.bits_a, s.bits_w) for s in specs)
                         for op in (aqt.OP_QMATMUL, aqt.OP_QMATMUL_REQUANT)) + 256, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    # One step = the whole FFN pair: the hidden tensor u = Swish(W1 x) is quantized per row inside
    # the first matmul's epilogue and only ever exists as codes + row scales.
    names = ["quantize(x) 12800x512", "qmatmul 512->2048 swish + quantize(u) rows (one kernel)", "qmatmul 2048->512"]
    NC = len(names)
    l0, l1 = layers

    # pre-marshalled C-ABI calls (one set per rotating buffer) so that Python stays ahead of the GPU
    def make_calls(st, rounding=aqt.ROUND_NEAREST_EVEN):
        out = []
        for r in range(R):
            out.append((
                aqt.bind_quantize(xs[r], specs[0].bits_a, aqt.AXIS_ROW, rounding, False, q1, s1, st),
                aqt.bind_qmatmul_requant(q1, s1, l0.mm_weight, l0.s_w, None, None, 1.0, specs[0].K, 8, l0.mm_bits | aqt.STATIC_WEIGHTS,
                                         specs[0].act, aqt.SCALE_ROW, specs[1].bits_a, rounding, False, q2, s2, None, ws, st),
                aqt.bind_qmatmul(q2, s2, l1.mm_weight, l1.s_w, None, None, 1.0, specs[1].K, 8, l1.mm_bits,
                                 specs[1].act, aqt.SCALE_ROW, ys[r], ws, st)))
        return out

    calls = make_calls(stream)

    def step(i):
        for f in calls[i % R]:
            f()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    if aqt.aqt_device_status() != 0:
        raise SystemExit("device status reports a failed wait during warm-up")

    # R consecutive steps captured in a CUDA graph (launch latency out of the way; consecutive
    # kernels overlap their set-up with the tail of the one before by programmatic dependent launch).
    graph = None
    if not args.no_graph:
        def run_plain(st):
            for c3 in make_calls(st):
                for c in c3:
                    c()
        graph = _capture(run_plain, torch)
        for _ in range(2):
            graph.replay()
        # the steps left over when --steps is not a multiple of R: a graph of their own, so that the
        # whole timed region is replayed from graphs whatever the step count
        rem = args.steps % R
        graph_rem = None
        if rem:
            def run_rem(st):
                for c3 in make_calls(st)[:rem]:
                    for c in c3:
                        c()
            graph_rem = _capture(run_rem, torch)
            graph_rem.replay()
        barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # ---- the timed region: exactly args.steps steps
    barrier()
    e_begin.record(stream)
    replays, i = 0, 0
    if graph is not None:
        for k in range(args.steps // R):
            graph.replay()
            replays += 1
            i += R
        if graph_rem is not None:
            graph_rem.replay()
            i += rem
    while i < args.steps:
        step(i); i += 1
    e_end.record(stream)
    barrier()
    total_ms = e_begin.elapsed_time(e_end)
    status = aqt.aqt_device_status()

    # ---- duration of each call of the step: the same call on the R rotating buffer sets, back to
    # back in a graph of its own (an event between two kernels of the step's graph would keep them
    # from overlapping and adds several microseconds per node, so the step itself carries none).
    # Inputs sit where the step leaves them: x in HBM, the codes a call reads in L2.
    per_call_ms = []
    for j in range(NC):
        def run_one(st, j=j):
            for c3 in make_calls(st):
                c3[j]()
        if graph is not None:
            gj = _capture(run_one, torch)
            per_call_ms.append(_time_replays(torch, gj, 10)[0] / R)
            del gj
        else:
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            run_one(stream)
            torch.cuda.synchronize()
            evs[0].record(stream)
            for _ in range(4):
                run_one(stream)
            evs[1].record(stream)
            torch.cuda.synchronize()
            per_call_ms.append(evs[0].elapsed_time(evs[1]) / (4 * R))

    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    ops_step = sum(2 * M * s.N * s.K for s in specs)
    value = world * args.steps * ops_step / (total_ms * 1e-3) / 1e12

    # ---- the same step for at least half a second (thousands of steps): the clock samples of the
    # JSON line are taken while this and the timed region run
    sustained = None
    if graph is not None and world == 1 and not args.no_sustained:
        ms_rep, n_rep = _time_replays(torch, graph, 200, min_seconds=0.6)
        sustained = {"value": ops_step / (ms_rep / R * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_rep / R, "steps": n_rep * R,
                     "seconds": ms_rep * n_rep * 1e-3}
    clocks = sampler.stop() if rank == 0 else None

    # ---- the same step with the rounding of Fig. 2, floor(v + 0.5), in both quantizers (the headline
    # uses nearest-even, which the workload definitions ask for); graph replay, same buffers
    fig2_ms = None
    if graph is not None and world == 1:
        def run_fig2(st):
            for c3 in make_calls(st, aqt.ROUND_HALF_UP_FLOOR):
                for c in c3:
                    c()
        g2 = _capture(run_fig2, torch)
        fig2_ms = _time_replays(torch, g2, 20)[0] / R

    # ---- end to end: host buffers through the C ABI (aqt_ffn_fwd: copy in, quantize, both matmuls
    # with the hidden tensor kept as codes, copy out), copies inside the timed region (per rank).
    # Every step copies its own input from pinned host memory and its own result back.  Steps
    # alternate between two streams (each with its own buffers) so that the host-to-device copy
    # of one step, the kernels of the previous one and the device-to-host copy of the one before
    # overlap; the timed region ends when the last result has landed on the host.
    n_lanes = 2
    lanes = []
    for _ in range(n_lanes):
        ln = {"stream": torch.cuda.Stream(), "xh": torch.from_numpy(x_host).clone().pin_memory(),
              "yh": torch.empty((M, specs[1].N), dtype=torch.float32).pin_memory(),
              "ws": torch.empty(aqt.aqt_workspace_bytes(aqt.OP_FFN_FWD, M, w.ff, w.d, 8, 4) + 256, dtype=torch.uint8, device=dev)}
        ln["call"] = aqt.bind_ffn_fwd(ln["xh"], l0.mm_weight, l0.s_w, l0.mm_bits, l1.mm_weight, l1.s_w, l1.mm_bits, ln["yh"], ln["ws"],
                                      bits_a=8, act=specs[0].act, stream=ln["stream"])
        lanes.append(ln)

    for i in range(4):
        lanes[i % n_lanes]["call"]()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for ln in lanes:
        ln["stream"].wait_event(e0)
    for i in range(args.steps):
        lanes[i % n_lanes]["call"]()
    for ln in lanes:
        stream.wait_stream(ln["stream"])
    e1.record(stream)
    barrier()
    te = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(te, op=dist.ReduceOp.MAX)
    e2e_value = world * args.steps * ops_step / (float(te.item()) * 1e-3) / 1e12
    e2e_status = aqt.aqt_device_status()

    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return 0
    # ---- roofline of the dominant call (largest share of the step), and every call's own figures
    pk = _peaks()
    s0, s1_ = specs
    alg_bytes = [
        4 * M * s0.K + M * s0.K + 4 * M,                                              # quantize(x): read fp32, write codes + scales
        M * s0.K + s0.K * s0.N // 2 + 8 * s0.N + 4 * M + M * s0.N + 4 * M,            # GEMM 1: codes, int4 weights, scales in; codes + scales out
        M * s1_.K + s1_.K * s1_.N + 8 * s1_.N + 4 * M + 4 * M * s1_.N,                # GEMM 2: codes, weights (int4 codes in int8 containers), scales in; fp32 out
    ]
    alg_ops = [0, 2 * M * s0.N * s0.K, 2 * M * s1_.N * s1_.K]
    sm_mhz = (clocks or {}).get("sm_mhz") or 1965.0
    sm_max_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    kernels = []
    for j in range(NC):
        sec = per_call_ms[j] * 1e-3
        k = {"call": names[j], "ms": per_call_ms[j], "algorithmic_bytes": alg_bytes[j], "gbs": alg_bytes[j] / sec / 1e9,
             "hbm_frac": alg_bytes[j] / sec / 1e9 / pk["hbm_gbs"], "share": per_call_ms[j] / sum(per_call_ms),
             "plan": ("quantize_rows", "requant ws128 (weight stationary, rows quantized in the epilogue)",
                      aqt.aqt_plan_qmatmul(M, s1_.N, s1_.K, 8, aqt.BITS_4_UNPACKED, s1_.act))[j]}
        if alg_ops[j]:
            tops = alg_ops[j] / sec / 1e12
            k.update({"tops": tops, "tensor_frac_nominal_int8": tops / INT8_NOMINAL_TOPS,
                      "tensor_frac_2x_bf16_" + pk["kind"]: tops / (2.0 * pk["bf16"]),
                      "tensor_frac_at_sampled_clock": tops / (INT8_NOMINAL_TOPS * sm_mhz / sm_max_mhz)})
        kernels.append(k)
    # DRAM traffic per launch from the committed ncu captures (dram__bytes_read.sum +
    # dram__bytes_write.sum); the write part undercounts what is still in L2 when the kernel ends.
    ncu_traffic = NCU_TRAFFIC if aqt.aqt_version() == NCU_CAPTURE_VERSION else {}
    dom = max(range(NC), key=lambda j: per_call_ms[j])
    props = torch.cuda.get_device_properties(dev)
    if dom == 1:
        # The fused kernel moves 33 MB (5 us of HBM time) and is bound by arithmetic instead: the
        # Swish needs two special-function operations (2^x, reciprocal) per element.  peak = the
        # special-function rate measured in this run by a kernel that does nothing else
        # (aqt_selftest_sfu_rate); the nominal 16 op/clk/SM x SMs x the maximum SM clock beside it.
        sfu_nominal = 16 * props.multi_processor_count * sm_max_mhz * 1e6 / 1e9      # Gop/s
        sfu_measured = aqt.aqt_selftest_sfu_rate()
        sfu_achieved = 2.0 * M * s0.N / (per_call_ms[1] * 1e-3) / 1e9
        roofline = {"bound": "alu", "kernel": names[1], "achieved": sfu_achieved, "peak": sfu_measured, "unit": "Gop/s",
                    "frac": sfu_achieved / sfu_measured,
                    "peak_source": "special-function unit, measured in this run by aqt_selftest_sfu_rate (2^x and reciprocal chains only)",
                    "peak_nominal": sfu_nominal, "frac_of_nominal": sfu_achieved / sfu_nominal,
                    "peak_nominal_source": "16 op/clk/SM x %d SMs x %d MHz" % (props.multi_processor_count, sm_max_mhz),
                    "hbm_frac": kernels[1]["hbm_frac"], "tensor_frac_nominal_int8": kernels[1]["tensor_frac_nominal_int8"],
                    "traffic": ncu_traffic.get(1), "calls": kernels}
    elif dom == 2 and kernels[2]["tensor_frac_nominal_int8"] > kernels[2]["hbm_frac"]:
        roofline = {"bound": "tensor", "kernel": names[2], "achieved": kernels[2]["tops"], "peak": INT8_NOMINAL_TOPS, "unit": "TOP/s",
                    "frac": kernels[2]["tensor_frac_nominal_int8"], "peak_source": "nominal dense int8 (no measured int8 peak exists)",
                    "hbm_frac": kernels[2]["hbm_frac"], "traffic": ncu_traffic.get(2), "calls": kernels}
    else:
        achieved = kernels[dom]["gbs"]
        roofline = {"bound": "hbm", "kernel": names[dom], "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / pk["hbm_gbs"], "peak_source": "of " + pk["kind"], "traffic": ncu_traffic.get(dom), "calls": kernels}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int8", "data": "synthetic",
            "config": {"workload": w.name, "M": M, "d_model": w.d, "ff": w.ff, "bits_w": 4, "bits_a": 8, "a_scale": "per-row",
                       "rounding": "nearest-even", "l2": "rotating %d input/output sets (x and y: 315 MB) exceed the 126 MB L2" % R,
                       "parallelism": "replicas x%d (rows sharded, no collective)" % world},
            "frames_per_s": world * args.steps * M / (total_ms * 1e-3),
            "clocks": clocks, "device_status": status,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * M * s0.K, "d2h_bytes_per_step": 4 * M * s1_.N,
                    "ms_per_step": float(te.item()) / args.steps, "streams": n_lanes, "api": "aqt_ffn_fwd", "device_status": e2e_status},
            "gpu_launches": args.steps * NC, "sum_call_ms_per_step": sum(per_call_ms),
            "launch_mode": ("cuda graph of %d steps x %d replays + one graph of the %d steps left over; per-call durations from one graph per call" %
                            (R, replays, args.steps - replays * R))
            if graph is not None else "call by call",
            "roofline": roofline}
    if sustained is not None:
        line["sustained"] = sustained
    if fig2_ms is not None:
        line["fig2_rounding"] = {"rounding": "floor(v + 0.5)", "ms_per_step": fig2_ms, "value": ops_step / (fig2_ms * 1e-3) / 1e12,
                                 "unit": UNIT}
    if world == 1 and not args.no_legs:
        line["quantizer"] = quantizer_leg(dev)
        line["encoder"] = encoder_frames_per_s(dev)
        line["weight_only"] = weight_only_ffn_pair(dev)
        line["weight_quantizer"] = weight_quantizer_leg(dev)
        line["backward"] = backward_ffn_layer(dev)
        # last: seconds of dense work that pull the clocks down (the part is power-limited)
        line["large_gemm"] = large_gemm_leg(dev)
        line["encoder_large"] = encoder_frames_per_s(dev, steps=2, cfg=5)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line), flush=True)
    return 0


def encoder_frames_per_s(dev, steps: int = 5, cfg: int = 4):
    """Second half of the metric: frames/s of the 17-block Conformer-encoder linear stack
    (cfg 4: d = 512, ff = 2048, batch 64 x 400 frames, FFN weights int4, attention / pointwise weights
    int8; cfg 5: d = 1024, ff = 4096, batch 128 x 512 frames, int4 weights; int8 per-row activations,
    fp32 residual adds fused into the epilogues).  170 linears per step, replayed from a CUDA graph.
    Weights are N(0, 1/fan_in) drawn on the GPU (seeded)."""
    import torch
    from paper_2203_15952_b200 import inputs as gen
    from paper_2203_15952_b200.encoder import EncoderStack, QuantLinear
    w = gen.WORKLOADS[cfg]
    specs = gen.workload_layers(w)
    g = torch.Generator(device=dev).manual_seed(4)
    blocks = []
    for _ in range(w.blocks):
        blocks.append([QuantLinear.from_float(s, torch.randn((s.N, s.K), generator=g, device=dev) * (s.K ** -0.5)) for s in specs])
    stack = EncoderStack(w.M, w.d, w.ff, blocks, dev)
    x = torch.randn((w.M, w.d), generator=g, device=dev)
    if w.x_dist == "student_t3":  # heavy-tailed block-0 input: Student-t with 3 degrees of freedom, unit variance
        chi = sum(torch.randn((w.M, w.d), generator=g, device=dev) ** 2 for _ in range(3)) / 3.0
        x = x / torch.sqrt(chi) / (3.0 ** 0.5)
        del chi
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        stack.forward(x)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        stack.forward(x)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return {"workload": w.name, "frames_per_s": w.M / (ms * 1e-3), "ms_per_step": ms, "tops": stack.ops / (ms * 1e-3) / 1e12,
            "steps": steps, "linears_per_step": len(specs) * w.blocks, "launch_mode": "cuda graph"}


def quantizer_leg(dev, replays: int = 10):
    """The activation quantizer alone on tensors far larger than L2 (row-wise abs-max, scale,
    round, cast / nibble pack): GB/s of the bytes the method itself must move, 4 per element in,
    1 (int8) or 1/2 (packed int4) out, 4 per row of scales, against the measured HBM copy rate.
    Two input tensors alternate, so nothing is served from L2."""
    import torch
    from paper_2203_15952_b200 import binding as aqt
    pk = _peaks()
    out = []
    g = torch.Generator(device=dev).manual_seed(7)
    for (M, K) in ((65536, 4096), (65536, 1024)):
        xs = [torch.randn((M, K), generator=g, device=dev) for _ in range(2)]
        for bits, pack in ((8, False), (4, True)):
            q = torch.empty((M, K // 2 if pack else K), dtype=torch.uint8 if pack else torch.int8, device=dev)
            sc = torch.empty(M, dtype=torch.float32, device=dev)

            def run(st):
                for x in xs:
                    aqt.bind_quantize(x, bits, aqt.AXIS_ROW, aqt.ROUND_NEAREST_EVEN, pack, q, sc, st)()
            graph = _capture(run, torch)
            ms = _time_replays(torch, graph, replays)[0] / len(xs)
            nbytes = 4 * M * K + M * K * bits // 8 + 4 * M
            gbs = nbytes / (ms * 1e-3) / 1e9
            out.append({"rows": M, "cols": K, "bits": bits, "packed": pack, "ms": ms, "algorithmic_bytes": nbytes,
                        "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                                     "peak_source": "of " + pk["kind"], "traffic": None}})
            del graph
        del xs
    return out


def weight_quantizer_leg(dev, replays: int = 10):
    """The weight quantizer as a per-step leg (training from scratch re-quantizes the float weights
    every step, Section 2.2): aqt_quantize over K per output channel with nibble packing, for the ten
    weights of every block of the d = 512 encoder (17 blocks, 357 MB of fp32 weights: beyond L2).
    Timed twice: the float weights in one arena per contraction depth (rows of different weights
    below one another, one call per arena: the rows are quantized independently, so the codes are
    the same), and one call per weight."""
    import torch
    from paper_2203_15952_b200 import binding as aqt
    from paper_2203_15952_b200 import encoder as enc
    from paper_2203_15952_b200 import inputs as gen
    pk = _peaks()
    w = gen.WORKLOADS[4]
    specs = gen.block_linears(w.d, w.ff, 4, 4, 8) * w.blocks
    arena = enc.WeightArena(specs, dev)
    g = torch.Generator(device=dev).manual_seed(8)
    for i, sp in enumerate(specs):
        arena.float_view(i).copy_(torch.randn((sp.N, sp.K), generator=g, device=dev) * (sp.K ** -0.5))
    nbytes = arena.algorithmic_bytes

    def run_arena(st):
        arena.quantize(stream=st)
    ms = _time_replays(torch, _capture(run_arena, torch), replays)[0]
    outs = {}
    for sp in specs:
        outs.setdefault((sp.N, sp.K), (torch.empty((sp.N, sp.K // 2), dtype=torch.uint8, device=dev),
                                       torch.empty(sp.N, dtype=torch.float32, device=dev)))

    def run_each(st):
        for i, sp in enumerate(specs):
            q, sc = outs[(sp.N, sp.K)]
            aqt.bind_quantize(arena.float_view(i), 4, aqt.AXIS_ROW, aqt.ROUND_NEAREST_EVEN, True, q, sc, st)()
    ms_each = _time_replays(torch, _capture(run_each, torch), replays)[0]
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": "int4 weight quantizer, 10 weights x %d blocks, d = %d, one arena per contraction depth" % (w.blocks, w.d),
            "ms_per_step": ms, "ms_per_block": ms / w.blocks, "launches_per_step": len(arena.float_arena), "algorithmic_bytes": nbytes,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs / pk["hbm_gbs"],
                         "peak_source": "of " + pk["kind"], "traffic": None},
            "one_call_per_weight": {"ms_per_step": ms_each, "launches_per_step": len(specs),
                                    "gbs": nbytes / (ms_each * 1e-3) / 1e9, "hbm_frac": nbytes / (ms_each * 1e-3) / 1e9 / pk["hbm_gbs"]}}


def large_gemm_leg(dev, burst_replays: int = 20, sustained_seconds: float = 2.0):
    """The integer matmul on the large shapes of the d = 1024 encoder (M = 65 536, int8 activation
    codes, int4 weights): burst (20 graph replays) and sustained (2 s back to back, with the SM clock
    and power sampled meanwhile).  TOPS against the nominal dense int8 peak, against twice the
    measured bf16 rates (no int8 peak has been measured on this machine) and scaled to the sampled clock."""
    import torch
    from paper_2203_15952_b200 import binding as aqt
    pk = _peaks()
    M = 65536
    out = []
    g = torch.Generator(device=dev).manual_seed(9)
    for (N, K, act, with_res, what) in ((1024, 4096, aqt.ACT_NONE, False, "ffn second layer"),
                                        (1024, 4096, aqt.ACT_NONE, True, "ffn second layer + residual"),
                                        (4096, 1024, aqt.ACT_SWISH, False, "ffn first layer, Swish")):
        time.sleep(1.0)  # let the clocks recover before the burst figure
        xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8, device=dev)
        wq = torch.randint(-7, 8, (N, K), generator=g, dtype=torch.int8, device=dev)
        s_x = torch.rand(M, generator=g, device=dev) * 1e-2 + 1e-3
        s_w = torch.rand(N, generator=g, device=dev) * 1e-3 + 1e-4
        ys = [torch.empty((M, N), dtype=torch.float32, device=dev) for _ in range(2)]
        res = torch.randn((M, N), generator=g, device=dev) if with_res else None

        def run(st):
            for y in ys:
                aqt.bind_qmatmul(xq, s_x, wq, s_w, None, res, 1.0, K, 8, aqt.BITS_4_UNPACKED, act, aqt.SCALE_ROW, y, None, st)()
        graph = _capture(run, torch)
        ops = 2.0 * M * N * K
        burst_ms = _time_replays(torch, graph, burst_replays // 2)[0] / len(ys)
        sampler = ClockSampler(torch.cuda.current_device())
        sampler.start()
        time.sleep(0.2)
        sus_ms, n = _time_replays(torch, graph, 20, min_seconds=sustained_seconds, warm=0)
        sus_ms /= len(ys)
        clocks = sampler.stop()
        mhz = clocks.get("sm_mhz") or 1965.0
        mx = clocks.get("sm_max_mhz") or 1965.0
        tb, ts = ops / (burst_ms * 1e-3) / 1e12, ops / (sus_ms * 1e-3) / 1e12
        nbytes = M * K + N * K // 2 + 8 * N + 4 * M + 4 * M * N * (2 if with_res else 1)
        out.append({"shape": "%d x %d -> %d" % (M, K, N), "what": what, "plan": aqt.aqt_plan_qmatmul(M, N, K, 8, 4, act),
                    "burst": {"ms": burst_ms, "tops": tb, "frac_nominal_int8": tb / INT8_NOMINAL_TOPS,
                              "frac_2x_bf16_burst_" + pk["kind"]: tb / (2 * pk["bf16"])},
                    "sustained": {"ms": sus_ms, "tops": ts, "seconds": sus_ms * n * len(ys) * 1e-3, "frac_nominal_int8": ts / INT8_NOMINAL_TOPS,
                                  "frac_2x_bf16_sustained_" + pk["kind"]: ts / (2 * pk["bf16_sustained"]),
                                  "frac_of_int8_peak_at_sampled_clock": ts / (INT8_NOMINAL_TOPS * mhz / mx), "clocks": clocks},
                    "hbm_frac_burst": nbytes / (burst_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                    "roofline": {"bound": "tensor", "achieved": tb, "peak": INT8_NOMINAL_TOPS, "unit": "TOP/s", "frac": tb / INT8_NOMINAL_TOPS,
                                 "peak_source": "nominal dense int8; twice the measured bf16 burst beside it", "traffic": None}})
        del graph, xq, wq, ys, res
    return out


def weight_only_ffn_pair(dev, steps: int = 20):
    """The same FFN pair in the weight-only configuration of Section 4.1 (I4W: int4 weights, fp32
    activations): two aqt_linear_fwd_weight_only calls per step (float matmul on the tensor cores'
    tf32 kind, Swish between), replayed from a CUDA graph over rotating buffers.  Reported against
    the tensor roofline of that kind: the measured bf16 rate times the nominal tf32 : bf16 ratio of 1/2."""
    import torch
    from paper_2203_15952_b200 import binding as aqt
    from paper_2203_15952_b200 import inputs as gen
    from paper_2203_15952_b200.encoder import QuantLinear
    w = gen.WORKLOADS[CFG]
    specs = gen.workload_layers(w)
    M = w.M
    g = torch.Generator(device=dev).manual_seed(5)
    layers = [QuantLinear.from_float(s, torch.randn((s.N, s.K), generator=g, device=dev) * (s.K ** -0.5)) for s in specs]
    R = 3
    xs = [torch.randn((M, specs[0].K), generator=g, device=dev) for _ in range(R)]
    ys = [torch.empty((M, specs[1].N), dtype=torch.float32, device=dev) for _ in range(R)]
    u = torch.empty((M, specs[0].N), dtype=torch.float32, device=dev)  # 105 MB between the two layers
    ws = torch.empty(max(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_WEIGHT_ONLY_X2, M, s.N, s.K, 0, s.bits_w) for s in specs) + 256,
                     dtype=torch.uint8, device=dev)

    def timed(precision):
        def run(st):
            for r in range(R):
                aqt.bind_linear_fwd_weight_only(xs[r], layers[0].wq, layers[0].s_w, None, None, 1.0, specs[0].bits_w, specs[0].act, u, ws,
                                                st, precision=precision)()
                aqt.bind_linear_fwd_weight_only(u, layers[1].wq, layers[1].s_w, None, None, 1.0, specs[1].bits_w, specs[1].act, ys[r], ws,
                                                st, precision=precision)()
        return _time_replays(torch, _capture(run, torch), steps)[0] / R
    ms = timed(aqt.FLOAT_TF32)
    ms_x2 = timed(aqt.FLOAT_TF32X2)
    flops = sum(2.0 * M * s.N * s.K for s in specs)
    tflops = flops / (ms * 1e-3) / 1e12
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    bf16, kind = 1589.0, "fallback"
    if os.path.exists(path):
        with open(path) as f:
            bf16, kind = float(json.load(f)["bf16_tflops"]), "measured"
    peak = 0.5 * bf16
    return {"workload": w.name + "_i4w_fp32_activations", "value": tflops, "unit": "TFLOP/s", "ms_per_step": ms,
            "frames_per_s": M / (ms * 1e-3), "dtype": "tf32", "gpu_launches_per_step": 4, "launch_mode": "cuda graph",
            "two_term": {"what": "every activation split exactly into its tf32 part and the rest, both multiplied (operand error 2^-20 "
                                 "instead of 2^-10 of the terms): the fp32-grade form", "ms_per_step": ms_x2,
                         "value": flops / (ms_x2 * 1e-3) / 1e12, "unit": "TFLOP/s of the layer's own 2MNK flops",
                         "tensor_flops_frac_of_peak": 2.0 * flops / (ms_x2 * 1e-3) / 1e12 / peak},
            "roofline": {"bound": "tensor", "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
                         "peak_source": "bf16 burst of %s x nominal tf32 : bf16 ratio 1/2" % kind, "traffic": None}}


def backward_ffn_layer(dev, steps: int = 20):
    """Straight-through backward (dx, dw, dbias) of the pair's first layer (M = 12 800, 512 -> 2048,
    int4 weights, int8 activation codes) through aqt_linear_bwd, replayed from a CUDA graph over
    rotating gradient buffers; 2 * 2 * M * N * K flops per call on the tensor cores' tf32 kind."""
    import ctypes
    import torch
    from paper_2203_15952_b200 import binding as aqt
    from paper_2203_15952_b200 import inputs as gen
    w = gen.WORKLOADS[CFG]
    s0 = gen.workload_layers(w)[0]
    M, N, K = w.M, s0.N, s0.K
    g = torch.Generator(device=dev).manual_seed(6)
    wq = torch.randint(-7, 8, (N, K // 2), generator=g, dtype=torch.int8, device=dev).view(torch.uint8)
    sw = torch.rand(N, generator=g, device=dev) * 1e-3
    xq = torch.randint(-127, 128, (M, K), generator=g, dtype=torch.int8, device=dev)
    sx = torch.rand(M, generator=g, device=dev) * 1e-2
    ws = torch.empty(aqt.aqt_workspace_bytes(aqt.OP_LINEAR_BWD, M, N, K, 0, 0) + 256, dtype=torch.uint8, device=dev)
    R = 3
    sets = [(torch.randn((M, N), generator=g, device=dev), torch.empty((M, K), device=dev), torch.empty((N, K), device=dev),
             torch.empty(N, device=dev)) for _ in range(R)]
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        calls = [aqt.bind("aqt_linear_bwd", aqt._ptr(dy), aqt._i64(N), aqt._ptr(xq), aqt._ptr(sx), aqt.SCALE_ROW, 8, aqt._ptr(wq),
                          aqt._ptr(sw), 4, aqt._i64(M), aqt._i64(N), aqt._i64(K), aqt._ptr(dx), aqt._i64(K), aqt._ptr(dw), aqt._i64(K),
                          aqt._ptr(db), aqt._ptr(ws), ctypes.c_size_t(ws.numel()), aqt._stream(side)) for (dy, dx, dw, db) in sets]
        for c in calls:
            c()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for c in calls:
            c()
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / (steps * R)
    tflops = 4.0 * M * N * K / (ms * 1e-3) / 1e12
    return {"workload": "ffn_first_layer_M%d_N%d_K%d_w4a8_dx_dw_dbias" % (M, N, K), "value": tflops, "unit": "TFLOP/s", "ms_per_step": ms,
            "dtype": "tf32", "gpu_launches_per_step": 9, "launch_mode": "cuda graph"}


def run_case(args):
    """One call of the library, a few times over, for profiler captures (ncu -k ... -c ...): small
    enough to finish in seconds, inputs larger than L2 where the kernel's DRAM figures matter."""
    import torch
    from paper_2203_15952_b200 import binding as aqt
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    g = torch.Generator(device=dev).manual_seed(11)
    name, it = args.case, args.iters
    codes = lambda r, c, q: torch.randint(-q, q + 1, (r, c), generator=g, dtype=torch.int8, device=dev)
    scales = lambda n, a: torch.rand(n, generator=g, device=dev) * a + a * 0.1
    if name in ("quantize_ffn", "quantize_large"):
        M, K = (12800, 512) if name == "quantize_ffn" else (65536, 1024)
        xs = [torch.randn((M, K), generator=g, device=dev) for _ in range(2 if name == "quantize_large" else 6)]
        for i in range(it):
            aqt.aqt_quantize(xs[i % len(xs)], 8, aqt.AXIS_ROW)
    elif name in ("requant_ffn1", "requant_large"):
        M, N, K = (12800, 2048, 512) if name == "requant_ffn1" else (32768, 4096, 1024)
        xq, wq = codes(M, K, 127), torch.randint(0, 256, (N, K // 2), generator=g, dtype=torch.uint8, device=dev)
        w_arg, bits_w = (wq, 4) if K <= 512 else (aqt.aqt_unpack_int4(wq, K), aqt.BITS_4_UNPACKED)
        s_x, s_w = scales(M, 1e-2), scales(N, 1e-3)
        for i in range(it):
            aqt.aqt_qmatmul_requant(xq, s_x, w_arg, s_w, K=K, bits_a=8, bits_w=bits_w, act=aqt.ACT_SWISH, bits_out=8)
    elif name in ("gemm_ffn2", "gemm_large_ffn2", "gemm_large_ffn1"):
        M, N, K, act = {"gemm_ffn2": (12800, 512, 2048, aqt.ACT_NONE), "gemm_large_ffn2": (32768, 1024, 4096, aqt.ACT_NONE),
                        "gemm_large_ffn1": (32768, 4096, 1024, aqt.ACT_SWISH)}[name]
        xq, wq, s_x, s_w = codes(M, K, 127), codes(N, K, 7), scales(M, 1e-2), scales(N, 1e-3)
        y = torch.empty((M, N), dtype=torch.float32, device=dev)
        for i in range(it):
            aqt.aqt_qmatmul(xq, s_x, wq, s_w, K=K, bits_a=8, bits_w=aqt.BITS_4_UNPACKED, act=act, y=y)
    elif name == "weight_only_ffn1":
        M, N, K = 12800, 2048, 512
        x, wq, s_w = torch.randn((M, K), generator=g, device=dev), torch.randint(0, 256, (N, K // 2), generator=g, dtype=torch.uint8, device=dev), scales(N, 1e-3)
        for i in range(it):
            aqt.aqt_linear_fwd_weight_only(x, wq, s_w, bits_w=4, act=aqt.ACT_SWISH)
    elif name == "bwd_ffn1":
        M, N, K = 12800, 2048, 512
        dy, xq, wq = torch.randn((M, N), generator=g, device=dev), codes(M, K, 127), torch.randint(0, 256, (N, K // 2), generator=g, dtype=torch.uint8, device=dev)
        s_x, s_w = scales(M, 1e-2), scales(N, 1e-3)
        for i in range(it):
            aqt.aqt_linear_bwd(dy, xq, s_x, wq, s_w, K=K, bits_a=8, bits_w=4)
    else:
        raise SystemExit("unknown case " + name)
    torch.cuda.synchronize()
    print(json.dumps({"case": name, "iters": it, "device_status": aqt.aqt_device_status()}), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-budget-s", type=float, default=100.0, help="--impl reference: CPU seconds for warm-up + steps together")
    ap.add_argument("--no-legs", "--no-encoder", dest="no_legs", action="store_true",
                    help="skip the legs beside the headline (quantizer, encoder stacks, weight-only, backward, large matmuls)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the half-second sustained run of the headline step")
    ap.add_argument("--no-graph", action="store_true", help="launch every step call by call (no CUDA graph replay)")
    ap.add_argument("--case", default=None, help="run one library call a few times and exit (for profiler captures): quantize_ffn, "
                    "quantize_large, requant_ffn1, requant_large, gemm_ffn2, gemm_large_ffn2, gemm_large_ffn1, weight_only_ffn1, bwd_ffn1")
    ap.add_argument("--iters", type=int, default=4, help="--case: number of calls")
    args = ap.parse_args()
    if args.case is not None:
        return run_case(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
