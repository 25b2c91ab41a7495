"""The tuner's cache file (environment variable TF_TUNE_CACHE): a tuned plan is written to the file, forgotten with the
in-memory cache, read back from the file on the next call, and gone once the file is."""
from __future__ import annotations

import os

import pytest

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs

pytestmark = pytest.mark.gpu


def test_tuned_plan_survives_through_the_cache_file(tmp_path):
    path = tmp_path / "tf_tune_cache.txt"
    op, rows, cols, dt = "rmsnorm", 3000, 2048, inputs.BF16
    old = os.environ.get("TF_TUNE_CACHE")
    os.environ["TF_TUNE_CACHE"] = str(path)
    try:
        tf.tf_clear_cache()
        default = tf.tf_query_choice(op, rows, cols, dt)
        # make the cached plan recognisable whatever the tuner would pick: tune, then overwrite the file's plan with a
        # valid one that differs from the default
        tuned = tf.tf_tune(op, rows, cols, dt)
        lines = path.read_text().splitlines()
        assert len(lines) == 1 and lines[0].split()[3:5] == [str(rows), str(cols)]
        assert lines[0].split()[5] == tuned["plan"]
        assert tf.tf_query_choice(op, rows, cols, dt) == tuned["plan"]
        marker = "cta:threads=96,vpt=4,cluster=1,persist=0"
        assert marker != default
        path.write_text(" ".join(lines[0].split()[:5] + [marker]) + "\n")
        tf.tf_clear_cache()                                         # forgets the plans in memory; the file is read again
        assert tf.tf_query_choice(op, rows, cols, dt) == marker
        assert tf.tf_query_choice(op, rows + 1, cols, dt) != marker  # the key holds the exact shape
        # a second shape is appended without losing the first
        tf.tf_tune("softmax", 500, 1024, inputs.F32)
        assert len(path.read_text().splitlines()) == 2
        tf.tf_clear_cache()
        assert tf.tf_query_choice(op, rows, cols, dt) == marker
        # lines that do not parse are skipped, not fatal
        path.write_text("garbage\n0 9 9 1 1 nonsense:threads=1\n")
        tf.tf_clear_cache()
        assert tf.tf_query_choice(op, rows, cols, dt) == default
        path.unlink()
        tf.tf_clear_cache()
        assert tf.tf_query_choice(op, rows, cols, dt) == default
    finally:
        if old is None:
            os.environ.pop("TF_TUNE_CACHE", None)
        else:
            os.environ["TF_TUNE_CACHE"] = old
        tf.tf_clear_cache()
