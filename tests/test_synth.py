"""The seeded input generator: determinism and the structure the recipe promises."""
import numpy as np

from paper_2406_17276_b200 import synth


def test_bf16_round_trip_and_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0], np.float32)   # 1+2^-8 ties to even, 1+3*2^-8 rounds up
    b = synth.f32_to_bf16_bits(x)
    assert synth.bf16_bits_to_f32(b).tolist() == [1.0, 1.0, 1.015625, -2.5, 0.0]


def test_tables_are_deterministic_and_disagree_on_the_stated_fraction():
    w = synth.Workload("t", 4, 1000, 8, 4, 4, 3.0, 1.1, 0.20, H=200, seed=3)
    ld, lt = synth.make_tables(w)
    ld2, lt2 = synth.make_tables(w)
    assert np.array_equal(ld, ld2) and np.array_equal(lt, lt2)
    assert ld.shape == (200, 1000) and ld.dtype == np.uint16
    fd = synth.bf16_bits_to_f32(ld); ft = synth.bf16_bits_to_f32(lt)
    assert int((fd.argmax(1) != ft.argmax(1)).sum()) == 40
    assert np.array_equal(np.sort(ld, axis=1), np.sort(lt, axis=1))     # same multiset per row
    assert abs(float(fd.std()) - 3.0) < 0.1
    assert np.all(fd.max(1) > 6.0)                                      # every row carries a peak


def test_root_tokens_in_range_and_seeded():
    a = synth.root_tokens(32, 32000, 1); b = synth.root_tokens(32, 32000, 1); c = synth.root_tokens(32, 32000, 2)
    assert a.dtype == np.int32 and a.min() >= 0 and a.max() < 32000
    assert np.array_equal(a, b) and not np.array_equal(a, c)


def test_named_workloads_match_the_five_configurations():
    w = synth.WORKLOADS
    assert (w["c1"].batch, w["c1"].V, w["c1"].n, w["c1"].k, w["c1"].max_depth) == (1, 32000, 10, 10, 6)
    assert (w["c2"].batch, w["c2"].V, w["c2"].n, w["c2"].k, w["c2"].max_depth) == (1, 32000, 50, 10, 10)
    assert (w["c3"].batch, w["c3"].V, w["c3"].n, w["c3"].k, w["c3"].max_depth) == (1, 128256, 64, 16, 12)
    assert (w["c4"].batch, w["c4"].V, w["c4"].n, w["c4"].k, w["c4"].max_depth) == (32, 32000, 64, 10, 10)
    assert (w["c5"].batch, w["c5"].V, w["c5"].n, w["c5"].k, w["c5"].max_depth) == (64, 152064, 256, 32, 20)
