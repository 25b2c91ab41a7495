"""The time-out path of the bounded waits, exercised without faulting or hanging anything: a wait on a barrier that cannot
complete runs out of a one-millisecond budget, the kernel records it and returns; the host reads TF_ERR_TIMEOUT once, the
next ordinary call is correct, and the tuner drops a candidate for which the word is set."""
from __future__ import annotations

import pytest
import torch

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_records_it_and_the_device_stays_usable():
    tf.tf_device_status()                                           # clean before
    src = torch.arange(64, dtype=torch.float32, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    assert tf.tf_debug_wait_probe(src, 2_000_000) is True           # about a millisecond of SM clocks
    t1.record()
    torch.cuda.synchronize()
    assert 0.2 < t0.elapsed_time(t1) < 100.0                        # it waited for its budget, and only for that
    with pytest.raises(tf.TfError) as e:
        tf.tf_device_status()
    assert e.value.status == 4                                      # TF_ERR_TIMEOUT
    tf.tf_device_status()                                           # read once: cleared
    # the next ordinary calls are unaffected, staged variants included
    for plan in (None, "pipe:threads=256,lanes=32,vpt=8,rpg=1,stages=2,chunk=8192,persist=1", "ring:threads=128,vpt=8,cluster=2,stages=2,persist=1,psmem=0"):
        tf.tf_force_plan("softmax", plan)
        try:
            assert not parity.parity(inputs.Workload("after", "softmax", inputs.BF16, 300, 2048, seed=11, x_std=3.0))
        finally:
            tf.tf_force_plan("softmax", None)
    tf.tf_device_status()


def test_probe_rejects_bad_arguments():
    L = tf.lib()
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    src = torch.zeros(16, device="cuda")
    assert L.tf_debug_wait_probe(None, 1000, flag.data_ptr(), None) == 1
    assert L.tf_debug_wait_probe(src.data_ptr() + 4, 1000, flag.data_ptr(), None) == 1
    assert L.tf_debug_wait_probe(src.data_ptr(), 0, flag.data_ptr(), None) == 1
    assert L.tf_debug_wait_probe(src.data_ptr(), 1000, None, None) == 1


def test_tuner_drops_candidates_whose_wait_gave_up():
    # an L2-resident shape: the tuner has no copy ceiling to finish early at, so the free run times its whole list
    op, rows, cols, dt = "rmsnorm", 512, 4096, inputs.F32
    tf.tf_clear_cache()
    heur = tf.tf_query_choice(op, rows, cols, dt)
    free = tf.tf_tune(op, rows, cols, dt)
    tf.tf_clear_cache()
    names = tf.tf_candidates(op, rows, cols, dt)
    # fail every candidate of the kinds the heuristic plan is not: the winner must then be of the heuristic's kind
    kind = heur.split(":")[0]
    others = sorted({n.split(":")[0] for n in names} - {kind})
    assert others, names
    try:
        timed = []
        for prefix in others:
            tf.tf_debug_tune_inject_timeout(prefix + ":")
            res = tf.tf_tune(op, rows, cols, dt)
            assert not res["plan"].startswith(prefix + ":"), (prefix, res)
            timed.append(res["timed"])
            tf.tf_device_status()                                   # the tuner cleared the word it was shown
            tf.tf_clear_cache()
        assert min(timed) < free["timed"], (timed, free)            # dropped candidates are never timed
    finally:
        tf.tf_debug_tune_inject_timeout(None)
        tf.tf_clear_cache()
    assert not parity.parity(inputs.Workload("after-tune", op, dt, 64, cols, seed=3, eps=1e-6))
