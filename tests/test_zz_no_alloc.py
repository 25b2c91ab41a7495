"""The entry point for callers that cannot allocate device memory (a server that handed all free memory to its own
pool at start-up, a latency-critical loop): `tf_softmax_fwd_noalloc` keeps its scratch in a fixed array inside the
library.  Checked through the C ABI against the ordinary `tf_softmax_fwd` on two calls in a row -- the second with a
different shape and contents, so that partials left over from the first call would show -- and against the CPU oracle.
This file is collected last on purpose."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import compare
import oracle
import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu


def _both(w):
    data = w.generate()
    x = parity.to_dev(data["x"], w.dt)
    y_new = torch.empty_like(x)
    L = tf.lib()
    stream = torch.cuda.current_stream().cuda_stream
    st = L.tf_softmax_fwd_noalloc(x.data_ptr(), y_new.data_ptr(), w.rows, w.cols, w.dt, stream)
    assert st == 0, tf.STATUS_NAMES.get(st, st)
    y_old = torch.empty_like(x)
    st = L.tf_softmax_fwd(x.data_ptr(), y_old.data_ptr(), w.rows, w.cols, w.dt, stream)
    assert st == 0
    torch.cuda.synchronize()
    tf.tf_device_status()
    return data, parity.to_host(y_new, w.dt), parity.to_host(y_old, w.dt)


@pytest.mark.parametrize("dt", [inputs.BF16, inputs.F32])
def test_noalloc_softmax_matches_the_ordinary_entry_point_twice_in_a_row(dt):
    tf.tf_force_plan("softmax", None)
    first = inputs.Workload("noalloc_a", "softmax", dt, 6, 150016, seed=21, x_std=10.0, mask_step=20011)
    second = inputs.Workload("noalloc_b", "softmax", dt, 37, 4104, seed=22, x_mean=-3.0, x_std=2.0)
    for w in (first, second):
        data, y_new, y_old = _both(w)
        # each result is within the parity tolerance of the exact one, so the two may differ by twice that
        if dt == inputs.BF16:
            assert int(compare.bf16_ulp_dist(y_new, y_old).max()) <= 2
        else:
            a, b = y_new.astype(np.float64), y_old.astype(np.float64)
            assert np.all(np.abs(a - b) <= 2e-5 * np.maximum(np.abs(a), np.abs(b)) + 2 * compare.F32_QUANTUM)
        ref, ref64 = oracle.softmax(data["x"], dt, want64=True, nthreads=8)
        r = compare.compare_softmax(y_new, ref, ref64, data["x"], dt)
        assert r.ok, str(r)


def test_noalloc_rejects_what_it_cannot_hold():
    L = tf.lib()
    x = torch.zeros((8, 4096), device="cuda")
    p = x.data_ptr()
    assert L.tf_softmax_fwd_noalloc(p, p, 8193, 4096, 0, None) == 2            # more rows than the fixed scratch covers
    assert L.tf_softmax_fwd_noalloc(p + 4, p, 4, 4096, 0, None) == 2           # misaligned
    assert L.tf_softmax_fwd_noalloc(p, p, 4, 4095, 0, None) == 2               # cols * 4 not a multiple of 16
    assert L.tf_softmax_fwd_noalloc(None, p, 4, 4096, 0, None) == 1
    assert L.tf_softmax_fwd_noalloc(p, p, 0, 4096, 0, None) == 0
