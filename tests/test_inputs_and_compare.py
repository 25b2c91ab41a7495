"""Host-side test infrastructure: the seeded generators and the comparators.  CPU only."""
from __future__ import annotations

import numpy as np
import pytest

import compare
import oracle
from oracle import BF16, F32
from paper_2512_09196_b200 import inputs


def test_generator_is_a_pure_function_of_index():
    w = inputs.Workload("t", "layernorm", BF16, 64, 96, seed=11, x_mean=0.5, x_std=3.0)
    full = w.generate()
    part = w.generate(row0=17, nrows=9)
    np.testing.assert_array_equal(full["x"][17:26], part["x"])
    np.testing.assert_array_equal(full["gamma"], part["gamma"])
    again = w.generate()
    np.testing.assert_array_equal(full["x"], again["x"])
    other = inputs.Workload("t", "layernorm", BF16, 64, 96, seed=12, x_mean=0.5, x_std=3.0).generate()
    assert (other["x"] != full["x"]).mean() > 0.9


def test_distributions_have_the_stated_moments():
    x = inputs.normal((2000, 500), F32, seed=5, stream=0, mean=0.5, std=3.0).astype(np.float64)
    assert abs(x.mean() - 0.5) < 0.02 and abs(x.std() - 3.0) < 0.02
    # Box-Muller pairs are uncorrelated and the tails are populated
    assert abs(np.corrcoef(x.ravel()[0::2], x.ravel()[1::2])[0, 1]) < 0.01
    assert (np.abs(x - 0.5) > 12.0).any()
    u = inputs.uniform((100000,), F32, seed=5, stream=1, lo=0.5, hi=1.5).astype(np.float64)
    assert u.min() >= 0.5 and u.max() <= 1.5 and abs(u.mean() - 1.0) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    w = inputs.config(2)
    xo = compare.bf16_to_f64(inputs.normal_outliers((512, 8192), BF16, 2, 0.0, 1.0, 0.01, 100.0))
    frac = (np.abs(xo) > 6.0).mean()          # |N(0,1)| > 6 never happens at this size; outliers mostly do
    assert 0.008 < frac < 0.011
    assert w.op == "rmsnorm" and w.rows == 16384 and w.cols == 8192


def test_tail_mask_layout():
    w = inputs.Workload("m", "softmax", BF16, 40, 256, seed=3, x_std=10.0, mask_step=32)
    x = w.generate()["x"]
    for r in range(40):
        k = (r * 32) % 256
        assert (x[r, 256 - k:] == 0xFF80).all()
        assert (x[r, :256 - k] != 0xFF80).all()
    np.testing.assert_array_equal(w.generate(row0=9, nrows=3)["x"], x[9:12])
    c3 = inputs.config(3)
    assert (c3.rows - 1) * 32 % c3.cols == c3.cols - 32      # the last row keeps 32 live columns


def test_sweep_rows_floor():
    rows = {(w.dt, w.cols): w.rows for w in inputs.sweep() if w.op == "softmax"}
    assert rows[(F32, 1000)] == 67108 and rows[(BF16, 1000)] == 134217
    assert rows[(F32, 5120)] == 13107 and rows[(BF16, 12288)] == 10922
    assert rows[(F32, 64)] == 1048576 and rows[(BF16, 65536)] == 2048
    assert len(inputs.sweep()) == 84


def test_algorithmic_bytes():
    assert inputs.config(0).algorithmic_bytes() == 8388608
    assert inputs.config(1).algorithmic_bytes() == 134299648
    assert inputs.config(2).algorithmic_bytes() == 536887296
    assert inputs.config(3).algorithmic_bytes() == 2147483648


def test_shard_rows_partitions():
    for rows, world in ((8192, 8), (10, 4), (3, 8), (0, 2)):
        got = [inputs.shard_rows(rows, r, world) for r in range(world)]
        assert sum(n for _, n in got) == rows
        pos = 0
        for r0, n in got:
            assert r0 == pos
            pos += n
    with pytest.raises(ValueError):
        inputs.shard_rows(4, 4, 4)


# ------------------------------------------------------------------ comparators discriminate

def test_bf16_comparator_flags_two_ulp_but_not_one():
    rng = np.random.default_rng(0)
    v = rng.normal(0, 1, (8, 128))
    o = oracle.bf16_from_double(v)
    assert compare.compare_values(o, o, v, BF16).ok
    one = o.copy(); one[3, 5] += 1
    assert compare.compare_values(one, o, v, BF16).ok
    two = o.copy(); two[3, 5] += 2
    r = compare.compare_values(two, o, v, BF16)
    assert not r.ok and r["first_bad"] == (3, 5)
    # across zero: +min-subnormal vs -min-subnormal is 2 apart, +0 vs -0 is 0 apart
    assert compare.bf16_ulp_dist(np.array([0x0001], np.uint16), np.array([0x8001], np.uint16))[0] == 2
    assert compare.bf16_ulp_dist(np.array([0x0000], np.uint16), np.array([0x8000], np.uint16))[0] == 0
    nan = o.copy(); nan[0, 0] = 0x7FC0
    assert not compare.compare_values(nan, o, v, BF16).ok


def test_f32_comparator_threshold():
    v = np.array([[1.0, -2.0, 1e-30, 0.0]])
    o = v.astype(np.float32)
    assert compare.compare_values(o, o, v, F32).ok
    g = o.copy(); g[0, 0] = np.float32(1.0 + 5e-6)
    assert compare.compare_values(g, o, v, F32).ok
    g[0, 0] = np.float32(1.0 + 2e-5)
    assert not compare.compare_values(g, o, v, F32).ok
    g = o.copy(); g[0, 3] = 1e-40
    assert not compare.compare_values(g, o, v, F32).ok
    g = o.copy(); g[0, 1] = np.nan
    assert not compare.compare_values(g, o, v, F32).ok


def test_softmax_comparator_wants_positive_zero_under_the_mask():
    x = np.array([[0.0, -np.inf]], np.float32)
    y, y64 = oracle.softmax(x, F32, want64=True)
    assert compare.compare_softmax(y, y, y64, x, F32).ok
    g = y.copy(); g[0, 1] = -0.0
    assert not compare.compare_softmax(g, y, y64, x, F32).ok


def test_layernorm_condition_scale_only_relaxes_near_cancellation():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 1, (4, 64)).astype(np.float32)
    g = rng.uniform(0.5, 1.5, 64).astype(np.float32)
    b = rng.uniform(0.5, 1.5, 64).astype(np.float32)
    y, mean, rstd, y64, st = oracle.layernorm(x, g, b, 1e-5, F32, want64=True)
    assert compare.compare_layernorm(y, y, y64, x, g, b, st, F32).ok
    cond = compare.layernorm_cond(x, g, b, st, F32)
    assert (cond >= np.abs(y64) * (1 - 1e-12)).all()
    bad = y.copy(); bad[2, 7] += np.float32(1e-3) * np.float32(cond[2, 7])
    assert not compare.compare_layernorm(bad, y, y64, x, g, b, st, F32).ok
    assert compare.compare_mean(mean, st, x, F32).ok and compare.compare_rstd(rstd, st[:, 1]).ok
    assert not compare.compare_rstd(rstd * np.float32(1.0001), st[:, 1]).ok
