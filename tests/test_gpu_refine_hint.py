"""The tuner's refinement hint reads a signal (registers, resident CTAs, waves and tail of the grid, bytes in flight, the
distance to the streaming copy) and orders the knobs by a rule table: forced incumbents that are short of occupancy, end
in a part-empty wave, or keep too little in flight make the matching rule fire and its knobs come first; a plan that
already runs at the copy ceiling ends the tuning at once; the winner of a tuned shape still matches the oracle."""
from __future__ import annotations

import pytest

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu
BF16, F32 = inputs.BF16, inputs.F32


def _knobs(plan: str) -> dict:
    return {k: int(v) for k, v in (kv.split("=") for kv in plan.split(":", 1)[1].split(","))}


def test_low_occupancy_incumbent_fires_the_register_rule_first():
    plan = "pipe:threads=512,lanes=64,vpt=8,rpg=1,stages=2,chunk=8192,persist=1"       # 126 registers, one CTA of 16 warps per SM
    h = tf.tf_refine_hint("layernorm", 8192, 4096, BF16, plan)
    assert h["rule"] == "occupancy", h
    assert h["regs"] > 96 and h["occupancy"] <= 0.25 and h["ctas_per_sm"] == 1
    base = _knobs(plan)
    for first in h["first"]:
        k = _knobs(first)
        assert k["vpt"] < base["vpt"] or k["threads"] < base["threads"] or k["rpg"] < base["rpg"], (first, h)
    assert any(_knobs(f)["vpt"] < base["vpt"] for f in h["first"]), h          # the same row on fewer registers per thread


def test_part_empty_last_wave_fires_the_tail_rule():
    plan = "twopass:threads=512,cache=0,persist=0,regcap=1"                             # 1024 CTAs on 3 x 148 resident ones: 2.3 waves
    h = tf.tf_refine_hint("softmax", 1024, 131072, BF16, plan)
    assert h["rule"] == "tail", h
    assert 2.0 < h["waves"] < 3.0 and h["tail"] > 0.15
    for first in h["first"]:
        k = _knobs(first)
        assert k["persist"] > 0 or k["cluster"] > 1 or k["threads"] < 512, (first, h)


def test_little_in_flight_fires_the_inflight_rule():
    plan = "cta:threads=64,vpt=1,cluster=1,persist=0"                                   # 32 CTAs x 64 threads x one 16-byte load per SM
    h = tf.tf_refine_hint("rmsnorm", 100000, 256, F32, plan)
    assert h["rule"] == "inflight", h
    assert h["inflight_kb"] < 40
    for first in h["first"]:
        k = _knobs(first)
        assert k["threads"] > 64 or k["persist"] > 0, (first, h)


def test_tuning_stops_at_the_copy_ceiling_and_the_winner_matches_the_oracle():
    tf.tf_clear_cache()
    # a shape whose default plan runs at the rate of the streaming copy: nothing to refine
    res = tf.tf_tune("softmax", 262144, 256, F32)
    h = tf.tf_tune_last_hint()
    assert h["vs_copy"] > 0 and h["regs"] > 0 and h["ctas_per_sm"] > 0, h
    n = len(tf.tf_candidates("softmax", 262144, 256, F32))
    if h["rule"] == "ceiling":
        assert res["timed"] == 1, (res, h)
    assert res["timed"] <= n + 8 * 12
    # a shape with room: LayerNorm bf16 mid-width; whatever wins, it reproduces the oracle
    w = inputs.Workload("hint-tuned", "layernorm", BF16, 2000, 4096, seed=17, x_mean=0.5, x_std=3.0, eps=1e-5)
    res = tf.tf_tune(w.op, w.rows, w.cols, w.dt)
    assert res["best_us"] <= res["heuristic_us"]
    assert tf.tf_query_choice(w.op, w.rows, w.cols, w.dt) == res["plan"]
    assert not parity.parity(w)
    tf.tf_clear_cache()
