"""The seeded input generator: deterministic, subset-addressable, with the stated distributions."""
import numpy as np

from paper_2203_15952_b200 import inputs as gen


def test_row_subset_equals_rows_of_full_tensor():
    full = gen.normal(0, 7, 300, 64)
    rows = [0, 5, 17, 299]
    assert np.array_equal(gen.normal(0, 7, 300, 64, row_subset=rows), full[rows])
    assert np.array_equal(gen.normal(0, 7, 300, 64), full)
    t_full = gen.student_t3(0, 9, 200, 32)
    assert np.array_equal(gen.student_t3(0, 9, 200, 32, row_subset=rows[:3]), t_full[rows[:3]])


def test_streams_differ_by_seed_and_tensor_id():
    a = gen.normal(0, 1, 8, 8)
    assert not np.array_equal(a, gen.normal(1, 1, 8, 8))
    assert not np.array_equal(a, gen.normal(0, 2, 8, 8))


def test_normal_moments():
    x = gen.normal(0, 3, 2000, 512).astype(np.float64)
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3
    assert abs(np.mean(x ** 4) - 3.0) < 0.05
    assert x.dtype == np.float64 and gen.normal(0, 3, 2, 2).dtype == np.float32


def test_student_t3_is_heavy_tailed_with_unit_scale():
    x = gen.student_t3(0, 4, 4000, 512).astype(np.float64)
    # t_3 / sqrt(3): the quartiles of t_3 are +-0.7649, so the scaled ones are +-0.4416
    q1, q3 = np.percentile(x, [25, 75])
    assert abs(q3 - 0.4416) < 5e-3 and abs(q1 + 0.4416) < 5e-3
    assert np.abs(x).max() > 20.0            # far beyond any Gaussian sample of this size
    row_max = np.abs(x).max(axis=1)
    assert np.median(row_max) > 4.0


def test_weight_is_the_transpose_view_with_fan_in_scaling():
    wt = gen.weight(0, 11, 512, 64)
    assert wt.shape == (64, 512) and wt.flags["C_CONTIGUOUS"]
    assert np.array_equal(wt.T, gen.normal(0, 11, 512, 64, std=1.0 / np.sqrt(512)))
    assert abs(wt.std() * np.sqrt(512) - 1.0) < 0.02


def test_workload_tables():
    w2 = gen.WORKLOADS[2]
    specs = gen.workload_layers(w2)
    assert [(s.K, s.N, s.act, s.bits_w, s.bits_a) for s in specs] == [(512, 2048, gen.ACT_SWISH, 4, 8), (2048, 512, gen.ACT_NONE, 4, 8)]
    w4 = gen.WORKLOADS[4]
    specs = gen.workload_layers(w4)
    assert len(specs) == 10 and w4.M == 64 * 400 and w4.blocks == 17
    assert {s.name: s.bits_w for s in specs}["ffn_a1"] == 4 and {s.name: s.bits_w for s in specs}["attn_q"] == 8
    pw1 = [s for s in specs if s.name == "conv_pw1"][0]
    assert pw1.N == 1024 and pw1.n_out == 512
    w5 = gen.WORKLOADS[5]
    assert w5.M == 128 * 512 and w5.d == 1024 and w5.ff == 4096 and w5.x_dist == "student_t3"
    x = gen.workload_input(gen.WORKLOADS[1])
    assert x.shape == (64, 256)
    assert gen.layer_bias(gen.WORKLOADS[1], 0, 0, gen.workload_layers(gen.WORKLOADS[1])[0]).shape == (256,)
