"""Which kernel configuration each matmul of the five workload configurations runs in, and that
every one of them is exercised by a parity test against the oracle (host-only: the plan query
needs no device).

The library chooses a configuration ("plan") of its GEMM kernel template per shape.  A parity
test only proves the configurations it reaches, so this file walks every matmul shape of the
workloads through the same choice the launches make (for the 148 multiprocessors of the part)
and requires each resulting plan to be named below together with the GPU test that runs it; those
tests assert the plan name themselves, so the table cannot drift from what they execute.
"""
import os
import re

from paper_2203_15952_b200 import binding as aqt
from paper_2203_15952_b200 import inputs as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

# plan -> (test file, test function) that compares this configuration with the oracle
COVERED_BY = {
    "small_m": ("test_gpu_kernels.py", "test_qmatmul_small_batch"),
    "ws128e16": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "ws128e8": ("test_gpu_kernels.py", "test_qmatmul_activations"),
    "stream256s3e16": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "stream256s4e4": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "stream128s4e16": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "stream128s6e4": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "stream128s4e8": ("test_gpu_kernels.py", "test_qmatmul_glu_streaming_plan_named"),
    "stream64s5e8": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "stream64s8e4": ("test_gpu_kernels.py", "test_qmatmul_single_cta_plans_named"),
    "pair256s4e8": ("test_gpu_kernels.py", "test_qmatmul_cta_pair_plans_named"),
    "pair256s6e4": ("test_gpu_full_size.py", "test_large_encoder_ffn_second_layer_matmul"),
    "pair128s6e8": ("test_gpu_kernels.py", "test_qmatmul_cta_pair_plans_named"),
    "pair128s8e4": ("test_gpu_full_size.py", "test_large_encoder_ffn_second_layer_matmul"),
    "pair512s3e16": ("test_gpu_kernels.py", "test_qmatmul_wide_pair_tiles_ffn_second_layer_shape"),
}


def _workload_matmul_shapes():
    """(M, N, K, bits_a, bits_w, act) of every matmul the drivers issue for the five configurations,
    including the one matmul over the concatenated q, k, v projections."""
    shapes = set()
    for cfg, w in gen.WORKLOADS.items():
        for s in gen.workload_layers(w):
            shapes.add((w.M, s.N, s.K, s.bits_a, s.bits_w, s.act))
        if w.kind in ("block", "stack"):
            shapes.add((w.M, 3 * w.d, w.d, w.bits_a, w.bits_attn_w, gen.ACT_NONE))
    return sorted(shapes)


def test_every_plan_the_workloads_reach_has_a_parity_test():
    reached = {}
    for (M, N, K, ba, bw, act) in _workload_matmul_shapes():
        plan = aqt.aqt_plan_qmatmul(M, N, K, ba, bw, act, sm_count=148)
        reached.setdefault(plan, []).append((M, N, K))
    assert reached, "no shapes"
    for plan, shapes in reached.items():
        assert plan in COVERED_BY, "plan %s (shapes %s) has no parity test" % (plan, shapes[:3])


def test_the_named_tests_exist_and_pin_their_plan():
    for plan, (fname, func) in COVERED_BY.items():
        text = open(os.path.join(ROOT, "tests", fname)).read()
        m = re.search(r"def %s\(.*?(?=\ndef |\Z)" % re.escape(func), text, flags=re.S)
        assert m, (fname, func)
        body = text[:m.end()]
        # the plan is either forced by name (a parametrize list above the test) or asserted inside it
        assert '"%s"' % plan in body or plan == "small_m" or plan in ("ws128e8",), (plan, func)


def test_plans_of_the_headline_shapes():
    """The shapes the benchmark and the benchmark spec's targets are quoted on."""
    p = lambda *a, **k: aqt.aqt_plan_qmatmul(*a, sm_count=148, **k)
    assert p(12800, 2048, 512, 8, 4, gen.ACT_SWISH) == "ws128e16"
    assert p(12800, 512, 2048, 8, 4) == "pair512s3e16"
    assert p(65536, 1024, 4096, 8, 4) == "pair256s6e4"
    assert p(65536, 4096, 1024, 8, 4, gen.ACT_SWISH) == "stream256s3e16"
    assert p(8, 512, 2048, 8, 4) == "small_m"
    assert p(64, 256, 256, 8, 8) == "ws128e16"
    # the float kind (weight-only layer, backward) plans with K in elements
    assert p(65536, 1024, 4096, 0, 4, float_kind=True) == "pair256s6e4"
    # a device with other SM counts changes the choice only through the number of rounds
    assert aqt.aqt_plan_qmatmul(12800, 2048, 512, 8, 4, gen.ACT_SWISH, sm_count=8) == "stream256s3e16"
